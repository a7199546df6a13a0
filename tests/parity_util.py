"""Helpers of the GPU parity tests: run the CUDA library on a workload group and
compare it with the CPU oracle under the stated rules.

Comparison rules
  * window scores: |gpu - oracle| <= 1e-3 * |oracle|  (fp32 accumulation from bf16/fp32 inputs)
  * window indices: list of length k, strictly ascending, in range; the symmetric
    difference with the oracle's set may only contain "ambiguous" windows, i.e.
    windows whose oracle fp32 score is within 1e-5 relative of the k-th largest score
  * compact K/V: bit-exact against the oracle's gather run with the indices the
    GPU chose (which equal the oracle's unless an ambiguous swap happened);
    rows the method does not write keep the pre-launch fill
"""
from __future__ import annotations

import numpy as np
import torch

import oracle
from paper_2503_17922_b200 import binding
from paper_2503_17922_b200 import workloads as wl

SCORE_RTOL = 1e-3
TIE_RTOL = 1e-5
FILL_BYTE = 0xA5


def oracle_kwargs(w, grp):
    return dict(n_kv_heads=w.n_kv_heads, l_obs=w.l_obs, window=w.window, task=w.task, top_p=w.top_p,
                max_seqlen=w.max_seqlen, budgets=grp["budgets"], cu_seqlens=grp["cu_seqlens"])


def fill_pattern(dtype: str) -> int:
    return 0xA5A5A5A5 if dtype == "f32" else 0xA5A5


def lse_obs_reference(w, grp) -> np.ndarray:
    """Eq. 1's normalisers as a prefill attention would hand them over: natural log of the sum of
    exp(q_i . k_j / sqrt(d)) over the keys j <= position(i), for every observation row, float32
    [B, H_q, alpha].  Plain numpy in float64, written out from the definition."""
    q = wl.to_f32(grp["q_obs"]).astype(np.float64)          # [B, H_q, alpha, d]
    k = wl.to_f32(grp["k_layers"][0]).astype(np.float64)
    G = w.n_q_heads // w.n_kv_heads
    out = np.zeros((w.batch, w.n_q_heads, w.l_obs), dtype=np.float32)
    for b in range(w.batch):
        n = int(grp["seqlens"][b])
        if n <= w.l_obs:
            continue                                         # nothing is scored for such a sequence
        if grp["cu_seqlens"] is not None:
            lo = int(grp["cu_seqlens"][b])
            kb = k[lo:lo + n].transpose(1, 0, 2)             # packed [T, H_kv, d] -> [H_kv, n, d]
        else:
            kb = k[b, :, :n]
        for hq in range(w.n_q_heads):
            logits = q[b, hq] @ kb[hq // G].T / np.sqrt(w.head_dim)      # [alpha, n]
            for i in range(w.l_obs):
                row = logits[i, :n - w.l_obs + i + 1]
                m = row.max()
                out[b, hq, i] = m + np.log(np.exp(row - m).sum())
    return out


def run_gpu_group(w, grp, score_impl=binding.WKV_SCORE_AUTO, staged=False, want_tokens=False, lse_obs=None):
    """Runs the whole group on the GPU. `staged` uses the three stage entry points
    instead of wkv_compress_group; `lse_obs` (host float32 [B, H_q, alpha]) the entry points
    that take the normalisers from the caller.  Returns host copies of every output."""
    prob = binding.Problem.from_workload(w, score_impl=score_impl)
    q = binding.to_device(grp["q_obs"])
    ks = [binding.to_device(x) for x in grp["k_layers"]]
    vs = [binding.to_device(x) for x in grp["v_layers"]]
    out = prob.alloc_outputs(len(ks), fill_byte=FILL_BYTE)
    work = prob.alloc_workspace()
    tok = None
    lse = None if lse_obs is None else torch.from_numpy(np.ascontiguousarray(lse_obs)).cuda()
    if staged:
        if want_tokens:
            tok = torch.full((w.batch, w.n_kv_heads, prob.nr_max), float("nan"), dtype=torch.float32, device="cuda")
        if lse is None:
            binding.wkv_score_windows(prob, q, ks[0], out["window_scores"], tok, work)
        else:
            binding.wkv_score_windows_lse(prob, q, ks[0], lse, out["window_scores"], tok, work)
        binding.wkv_select_topk_windows(prob, out["window_scores"], out["window_idx"], out["kept_len"])
        binding.wkv_gather_kv(prob, ks, vs, out["window_idx"], out["k_out"], out["v_out"],
                              keep_capacity=out["keep_capacity"])
    elif lse is None:
        binding.wkv_compress_group(prob, q, ks, vs, out["k_out"], out["v_out"], out["window_scores"],
                                   out["window_idx"], out["kept_len"], work, keep_capacity=out["keep_capacity"])
    else:
        binding.wkv_compress_group_lse(prob, q, lse, ks, vs, out["k_out"], out["v_out"], out["window_scores"],
                                       out["window_idx"], out["kept_len"], work,
                                       keep_capacity=out["keep_capacity"])
    torch.cuda.synchronize()
    assert binding.device_status(work) == 0, "a kernel reported an expired wait"
    return {
        "prob": prob,
        "window_scores": out["window_scores"].cpu().numpy(),
        "window_idx": out["window_idx"].cpu().numpy(),
        "kept_len": out["kept_len"].cpu().numpy(),
        "k_out": [binding.to_host_bits(t) for t in out["k_out"]],
        "v_out": [binding.to_host_bits(t) for t in out["v_out"]],
        "token_scores": None if tok is None else tok.cpu().numpy(),
    }


def check_selection(w, grp, gpu, ref, units=None):
    """Score tolerance + index rule for every unit (or the listed (b, h) units).
    Returns (max relative score error, number of ambiguous swaps)."""
    seqlens = grp["seqlens"]
    max_rel, swaps = 0.0, 0
    todo = units if units is not None else [(b, h) for b in range(w.batch) for h in range(w.n_kv_heads)]
    for b, h in todo:
        n = int(seqlens[b])
        kw = oracle.num_windows(n, w.l_obs, w.window)
        k = oracle.num_selected(n, w.l_obs, w.window, int(grp["budgets"][b]))
        s_ref = ref["window_scores"][b, h, :kw].astype(np.float64)
        s_gpu = gpu["window_scores"][b, h, :kw].astype(np.float64)
        if kw:
            assert np.isfinite(s_gpu).all(), f"unit ({b},{h}): non-finite window score"
            rel = np.abs(s_gpu - s_ref) / np.maximum(np.abs(s_ref), 1e-30)
            assert rel.max() <= SCORE_RTOL, f"unit ({b},{h}): score error {rel.max():.3e} at window {rel.argmax()}"
            max_rel = max(max_rel, float(rel.max()))
        gi = gpu["window_idx"][b, h]
        ri = ref["window_idx"][b, h]
        assert (gi[k:] == -1).all(), f"unit ({b},{h}): padding not -1"
        sel = gi[:k]
        if k:
            assert (np.diff(sel) > 0).all() and sel[0] >= 0 and sel[-1] < kw, f"unit ({b},{h}): indices not ascending/in range"
            tau = np.sort(s_ref)[-k]
            amb = np.abs(s_ref - tau) <= TIE_RTOL * np.maximum(np.abs(s_ref), abs(tau))
            diff = set(sel.tolist()) ^ set(ri[:k].tolist())
            assert all(amb[x] for x in diff), f"unit ({b},{h}): index mismatch outside the near-tie band: {sorted(diff)}"
            swaps += len(diff) // 2
        n_r = max(n - w.l_obs, 0)
        rows = sum(min((int(i) + 1) * w.window, n_r) - int(i) * w.window for i in sel) + min(w.l_obs, n)
        assert int(gpu["kept_len"][b, h]) == rows, f"unit ({b},{h}): kept_len"
    return max_rel, swaps


def check_gather(w, grp, gpu, layers=None):
    """Compact caches bit-exact against the oracle's gather fed with the GPU's indices."""
    prob = gpu["prob"]
    kw = dict(n_kv_heads=w.n_kv_heads, l_obs=w.l_obs, window=w.window, max_seqlen=w.max_seqlen,
              budgets=grp["budgets"], keep_max=prob.keep_max, cu_seqlens=grp["cu_seqlens"],
              fill=fill_pattern(w.dtype))
    for layer in (range(len(grp["k_layers"])) if layers is None else layers):
        for name, src, got in (("K", grp["k_layers"][layer], gpu["k_out"][layer]),
                               ("V", grp["v_layers"][layer], gpu["v_out"][layer])):
            exp = oracle.gather_layer(src, gpu["window_idx"], **kw)
            assert got.shape == exp.shape
            if not np.array_equal(got, exp):
                bad = np.argwhere(got != exp)[0]
                raise AssertionError(f"layer {layer} {name}: first mismatch at {tuple(bad)}")


def full_check(w, group=0, score_impl=binding.WKV_SCORE_AUTO, staged=False, given_lse=False):
    grp = wl.make_group(w, group)
    ref = oracle.select_leader(grp["q_obs"], grp["k_layers"][0], **oracle_kwargs(w, grp))
    gpu = run_gpu_group(w, grp, score_impl=score_impl, staged=staged,
                        lse_obs=lse_obs_reference(w, grp) if given_lse else None)
    stats = check_selection(w, grp, gpu, ref)
    check_gather(w, grp, gpu)
    return grp, ref, gpu, stats
