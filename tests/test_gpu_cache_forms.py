"""GPU tests of the two further forms of the compact cache (section 2.2.2 as driven during prefill, section
2.1's decode cache): compaction inside the layer's own buffer, and gather into a paged cache through a
block table.  Both are bit-exact against the oracle's gather on the same indices."""
import numpy as np
import pytest
import torch

import oracle
from paper_2503_17922_b200 import binding
from paper_2503_17922_b200 import workloads as wl

import parity_util as pu

pytestmark = pytest.mark.gpu


def _case(**kw):
    base = dict(name="cache-forms", dtype="bf16", batch=2, n_layers=2, gamma=2, n_q_heads=8, n_kv_heads=2,
                head_dim=128, max_seqlen=1337, l_obs=16, window=8, top_p=4, budget_frac=0.2, n_planted=5, config_id=12)
    base.update(kw)
    return wl.scaled(wl.llama8b_single_group(), **base)


def _indices(w, grp, prob, pattern):
    """Window lists chosen by the test (ascending, k per sequence): 'selected' = the oracle's selection;
    'shift' = windows 1..k (every output window lies on the source of the next slot); 'tail' = the last k
    windows (the longest moves, ragged last window included); 'front' = windows 0..k-1 (nothing moves)."""
    if pattern == "selected":
        ref = oracle.select_leader(grp["q_obs"], grp["k_layers"][0], **pu.oracle_kwargs(w, grp))
        return np.ascontiguousarray(ref["window_idx"], dtype=np.int32)
    idx = np.full((w.batch, w.n_kv_heads, prob.k_max), -1, dtype=np.int32)
    for b in range(w.batch):
        n = int(grp["seqlens"][b])
        kw = oracle.num_windows(n, w.l_obs, w.window)
        k = oracle.num_selected(n, w.l_obs, w.window, int(grp["budgets"][b]))
        for h in range(w.n_kv_heads):
            if pattern == "shift":
                lo = 1 if k < kw else 0
            elif pattern == "tail":
                lo = kw - k
            else:
                lo = 0
            idx[b, h, :k] = np.arange(lo, lo + k)
    return idx


@pytest.mark.parametrize("pattern", ["selected", "shift", "tail", "front"])
@pytest.mark.parametrize("case", [
    dict(),                                                    # dense [B, H_kv, N, d]
    dict(layout="bnhd", window=16, max_seqlen=777),            # token-major rows
    dict(ragged=True, batch=3, max_seqlen=900),                # packed [T, H_kv, d]
    dict(dtype="f32", head_dim=64, n_q_heads=4, l_obs=8),
    dict(budget_frac=0.9, max_seqlen=2100),                    # most rows kept: many batches per unit, short moves
    dict(budget_frac=None, budget_tokens=10 ** 6),             # everything kept: nothing moves
], ids=lambda c: "-".join(f"{k}{v}" for k, v in c.items()) or "base")
def test_compaction_in_place(case, pattern):
    case = dict(case)
    layout = case.pop("layout", "bhnd")
    w = _case(**case)
    grp = wl.make_group(w, 0)
    prob = binding.Problem(dtype=w.dtype, batch=w.batch, n_q_heads=w.n_q_heads, n_kv_heads=w.n_kv_heads,
                           head_dim=w.head_dim, l_obs=w.l_obs, window=w.window, task=w.task, top_p=w.top_p,
                           max_seqlen=w.max_seqlen, budgets=grp["budgets"], cu_seqlens=grp["cu_seqlens"],
                           kv_layout=layout)
    idx = _indices(w, grp, prob, pattern)

    def dev(x):
        return binding.to_device(np.ascontiguousarray(x.transpose(0, 2, 1, 3)) if layout == "bnhd" else x)
    ks = [dev(x) for x in grp["k_layers"]]
    vs = [dev(x) for x in grp["v_layers"]]
    before = [binding.to_host_bits(t) for t in ks + vs]
    binding.wkv_compact_kv_inplace(prob, ks, vs, torch.from_numpy(idx).cuda())
    torch.cuda.synchronize()
    kw_ = dict(n_kv_heads=w.n_kv_heads, l_obs=w.l_obs, window=w.window, max_seqlen=w.max_seqlen,
               budgets=grp["budgets"], keep_max=prob.keep_max, cu_seqlens=grp["cu_seqlens"], fill=0)
    moved = 0
    for layer in range(w.gamma):
        for src, got_t, old in ((grp["k_layers"][layer], ks[layer], before[layer]),
                                (grp["v_layers"][layer], vs[layer], before[w.gamma + layer])):
            exp = oracle.gather_layer(src, idx, **kw_)                  # dense [B, H_kv, keep_max, d]
            got = binding.to_host_bits(got_t)
            for b in range(w.batch):
                n = int(grp["seqlens"][b])
                n_r = max(n - w.l_obs, 0)
                k = oracle.num_selected(n, w.l_obs, w.window, int(grp["budgets"][b]))
                for h in range(w.n_kv_heads):
                    kept = sum(min((int(i) + 1) * w.window, n_r) - int(i) * w.window for i in idx[b, h, :k]) + min(w.l_obs, n)
                    if grp["cu_seqlens"] is not None:
                        lo = int(grp["cu_seqlens"][b])
                        unit_rows, old_rows = got[lo:lo + n, h], old[lo:lo + n, h]
                    elif layout == "bnhd":
                        unit_rows, old_rows = got[b, :n, h], old[b, :n, h]
                    else:
                        unit_rows, old_rows = got[b, h, :n], old[b, h, :n]
                    np.testing.assert_array_equal(unit_rows[:kept], exp[b, h, :kept])
                    # rows behind the compact cache are leftovers: each still equals some row of the old tensor
                    # at the same position (never written) - the kernel writes nothing at or beyond kept
                    np.testing.assert_array_equal(unit_rows[kept:], old_rows[kept:])
                    moved += int((unit_rows[:kept] != old_rows[:kept]).any())
    if pattern in ("shift", "tail", "selected") and case.get("budget_tokens") is None:
        assert moved > 0


@pytest.mark.parametrize("pool_layout", ["heads-outer", "token-major"])
@pytest.mark.parametrize("case", [
    dict(),
    dict(ragged=True, batch=3, max_seqlen=900, window=16),
    dict(dtype="f32", head_dim=64, n_q_heads=4, l_obs=8),
], ids=lambda c: "-".join(f"{k}{v}" for k, v in c.items()) or "base")
def test_gather_into_a_paged_cache(case, pool_layout):
    """Pages of 24 rows (not a multiple of the window length, so windows straddle pages), a block table
    that scatters every sequence's pages over the pool, one table for all layers and for K and V."""
    w = _case(**case)
    grp = wl.make_group(w, 0)
    prob = binding.Problem.from_workload(w)
    ref = oracle.select_leader(grp["q_obs"], grp["k_layers"][0], **pu.oracle_kwargs(w, grp))
    idx = np.ascontiguousarray(ref["window_idx"], dtype=np.int32)
    ps = 24
    max_pages = -(-prob.keep_max // ps)
    num_pages = w.batch * max_pages + 5
    g = np.random.Generator(np.random.Philox(key=99))
    table = g.permutation(num_pages)[: w.batch * max_pages].reshape(w.batch, max_pages).astype(np.int32)
    H, d = w.n_kv_heads, w.head_dim
    tdt = torch.float32 if w.dtype == "f32" else torch.bfloat16
    if pool_layout == "heads-outer":
        shape, strides = (num_pages, H, ps, d), (H * ps * d, ps * d, d)
    else:
        shape, strides = (num_pages, ps, H, d), (ps * H * d, d, H * d)
    ks = [binding.to_device(x) for x in grp["k_layers"]]
    vs = [binding.to_device(x) for x in grp["v_layers"]]
    pools = [[torch.empty(shape, dtype=tdt, device="cuda") for _ in range(w.gamma)] for _ in range(2)]
    for t in pools[0] + pools[1]:
        t.view(torch.uint8).fill_(pu.FILL_BYTE)
    binding.wkv_gather_kv_paged(prob, ks, vs, torch.from_numpy(idx).cuda(), pools[0], pools[1],
                                torch.from_numpy(table).cuda(), ps, num_pages, *strides)
    torch.cuda.synchronize()
    fill = pu.fill_pattern(w.dtype)
    kw_ = dict(n_kv_heads=H, l_obs=w.l_obs, window=w.window, max_seqlen=w.max_seqlen, budgets=grp["budgets"],
               keep_max=prob.keep_max, cu_seqlens=grp["cu_seqlens"], fill=fill)
    for layer in range(w.gamma):
        for src, pool in ((grp["k_layers"][layer], pools[0][layer]), (grp["v_layers"][layer], pools[1][layer])):
            exp = oracle.gather_layer(src, idx, **kw_)                  # dense [B, H, keep_max, d], fill behind kept
            got = binding.to_host_bits(pool)
            want = np.empty(got.shape, dtype=got.dtype)                 # the pool as the definition of the layout gives it
            want.view(np.uint32 if w.dtype == "f32" else np.uint16)[...] = fill
            for b in range(w.batch):
                for h in range(H):
                    kept = int(ref["kept_len"][b, h])
                    for r in range(kept):
                        page, slot = int(table[b, r // ps]), r % ps
                        if pool_layout == "heads-outer":
                            want[page, h, slot] = exp[b, h, r]
                        else:
                            want[page, slot, h] = exp[b, h, r]
            np.testing.assert_array_equal(got, want)


def test_paged_cache_argument_checks():
    w = _case()
    grp = wl.make_group(w, 0)
    prob = binding.Problem.from_workload(w)
    z = torch.zeros(64, dtype=torch.int32, device="cuda")
    t = [torch.zeros(8, dtype=torch.bfloat16, device="cuda")]
    with pytest.raises(binding.WkvError) as e:          # two pages of 24 rows cannot hold keep_max rows
        binding.wkv_gather_kv_paged(prob, t, None, z, [torch.zeros(8, dtype=torch.bfloat16, device="cuda")], None,
                                    z.view(2, 32)[:, :2].contiguous(), 24, 10, 24 * 128 * 2, 24 * 128, 128)
    assert e.value.status == 2
