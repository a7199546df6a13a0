"""Pins for the CPU oracle: each check compares the oracle with something the
paper's equations or plain mathematics fix, never with the oracle's own formula
retyped.  (Eq. numbers refer to the paper's section 2.2.1.)"""
import itertools
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

import oracle
from paper_2503_17922_b200 import workloads as wl

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "handworked_eq1_4.txt")


def _rand(shape, seed, dtype="f32"):
    x = np.random.Generator(np.random.Philox(key=seed)).standard_normal(shape, dtype=np.float32)
    return x if dtype == "f32" else wl.f32_to_bf16_bits(x)


# ------------------------------------------------------------------ Eq. 1-2
def _parse_golden():
    cases, cur = [], None
    for line in open(GOLDEN):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        if line.startswith("case"):
            cur = {"name": line.split()[1]}
            cases.append(cur)
            continue
        key, val = [x.strip() for x in line.split("=")]
        cur[key] = val.split()
    return cases


@pytest.mark.parametrize("case", _parse_golden(), ids=lambda c: c["name"])
def test_handworked_rational_examples(case):
    n, alpha, G, omega = (int(case[x][0]) for x in ("n", "alpha", "G", "omega"))
    q = np.array([float(x) for x in case["q"]], dtype=np.float32).reshape(G, alpha, 1)
    k = np.log(np.array([float(x) for x in case["key_weights"]], dtype=np.float64)).astype(np.float32).reshape(n, 1)
    t, mass, _ = oracle.token_scores_unit(q, k)
    t_exp = np.array([float(Fraction(x)) for x in case["t"]])
    np.testing.assert_allclose(t, t_exp, rtol=2e-6)
    for p in (1, 2):
        s = oracle.window_scores(t, omega, p)
        np.testing.assert_allclose(s, [float(Fraction(x)) for x in case[f"s_p{p}"]], rtol=2e-6)
    # whole path through the batch entry, p = omega (localization)
    budget = int(case["budget"][0])
    qb = q.reshape(1, G, alpha, 1)
    kb = k.reshape(1, 1, n, 1)
    sel = oracle.select_leader(qb, kb, n_kv_heads=1, l_obs=alpha, window=omega, task=wl.TASK_LOCALIZATION,
                               top_p=0, max_seqlen=n, budgets=np.array([budget], dtype=np.int32))
    k_sel = len(case["idx_p2"])
    assert list(sel["window_idx"][0, 0, :k_sel]) == [int(x) for x in case["idx_p2"]]
    assert int(sel["kept_len"][0, 0]) == int(case["kept_len_p2"][0])


@pytest.mark.parametrize("G,alpha,n,d", [(1, 1, 9, 4), (4, 8, 100, 16), (2, 5, 37, 8)])
def test_identical_keys_closed_form(G, alpha, n, d):
    # all keys equal => every causal row is uniform over its i+1 keys =>
    # t_j = G * sum_{i=n-alpha}^{n-1} 1/(i+1) for every review token
    q = _rand((G, alpha, d), 1)
    k = np.tile(_rand((1, d), 2), (n, 1))
    t, mass, _ = oracle.token_scores_unit(q, k)
    expect = G * sum(1.0 / (i + 1) for i in range(n - alpha, n))
    np.testing.assert_allclose(t, np.full(n - alpha, expect), rtol=1e-12)
    # zero queries give the same uniform rows whatever the keys are
    t0, _, _ = oracle.token_scores_unit(np.zeros_like(q), _rand((n, d), 3))
    np.testing.assert_allclose(t0, np.full(n - alpha, expect), rtol=1e-12)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_row_sum_invariant(dtype):
    # softmax rows sum to one: review mass + observation mass = G * alpha
    G, alpha, n, d = 4, 8, 300, 32
    q, k = _rand((G, alpha, d), 4, dtype), _rand((n, d), 5, dtype)
    t, mass, _ = oracle.token_scores_unit(q, k)
    assert abs(t.sum() + mass - G * alpha) < 1e-10
    assert mass > 0 and (t > 0).all()


def test_shift_invariance():
    # an extra key component that is constant over keys adds a per-row constant to the
    # logits (once sqrt(d) is held fixed by zero padding) and must not change t
    G, alpha, n, d = 2, 4, 64, 16
    q = _rand((G, alpha, d), 6)
    k = _rand((n, d), 7)
    q0 = q.copy(); q0[..., -1] = 0
    k0 = k.copy(); k0[..., -1] = 0
    t_ref, _, _ = oracle.token_scores_unit(q0, k0)
    k1 = k0.copy(); k1[..., -1] = 3.0      # constant over keys
    q1 = q0.copy(); q1[..., -1] = _rand((G, alpha), 8)
    t_shift, _, _ = oracle.token_scores_unit(q1, k1)
    np.testing.assert_allclose(t_shift, t_ref, rtol=1e-9)


def test_dominant_key_takes_all_mass():
    G, alpha, n, d = 2, 4, 50, 8
    q = np.ones((G, alpha, d), dtype=np.float32)
    k = np.zeros((n, d), dtype=np.float32)
    k[17] = 60.0 * np.sqrt(d) / d          # logit +60 for every row
    t, mass, _ = oracle.token_scores_unit(q, k)
    assert abs(t[17] - G * alpha) < 1e-20 * 1e3 + 1e-15
    assert np.delete(t, 17).max() < 1e-24


@pytest.mark.parametrize("dtype,G,alpha,n,d", [("f32", 4, 8, 257, 64), ("bf16", 4, 32, 515, 128),
                                                ("f32", 1, 1, 33, 8)])
def test_token_scores_against_library_softmax(dtype, G, alpha, n, d):
    # t = softmax(Q K^T / sqrt(d) + causal mask).sum(rows), evaluated by torch on the CPU
    q, k = _rand((G, alpha, d), 9, dtype), _rand((n, d), 10, dtype)
    t, _, lse = oracle.token_scores_unit(q, k, want_lse=True)
    qt = torch.from_numpy(wl.to_f32(q)).double().reshape(G * alpha, d)
    kt = torch.from_numpy(wl.to_f32(k)).double()
    logits = qt @ kt.T / d ** 0.5
    pos = (n - alpha) + torch.arange(alpha).repeat(G)             # absolute position of each row
    mask = torch.arange(n)[None, :] > pos[:, None]
    logits = logits.masked_fill(mask, float("-inf"))
    a = torch.softmax(logits, dim=-1)
    np.testing.assert_allclose(t, a[:, : n - alpha].sum(0).numpy(), rtol=1e-10)
    np.testing.assert_allclose(lse, torch.logsumexp(logits, dim=-1).numpy(), rtol=1e-10, atol=1e-11)
    if G == 1 and alpha == 1:     # a single softmax row
        np.testing.assert_allclose(t, a[0, : n - 1].numpy(), rtol=1e-12)


def test_causal_mask_matters():
    # a mistake that lets row i see keys beyond its own position would change the result:
    # make the last key huge; only the last observation row may see it
    G, alpha, n, d = 1, 2, 6, 1
    q = np.ones((G, alpha, d), dtype=np.float32)
    k = np.zeros((n, d), dtype=np.float32)
    k[n - 1] = 50.0
    t, mass, _ = oracle.token_scores_unit(q, k)
    # row n-2 is uniform over n-1 keys, row n-1 puts ~all its mass on key n-1
    np.testing.assert_allclose(t, np.full(n - alpha, 1.0 / (n - 1)), rtol=1e-9, atol=1e-20)


# ------------------------------------------------------------------ Eq. 3-4
@pytest.mark.parametrize("omega", [4, 8, 16, 32])
def test_pooling_special_cases_against_library(omega):
    t = np.abs(_rand((omega * 13,), 11)).astype(np.float64)
    tt = torch.from_numpy(t)[None, None]
    avg = torch.nn.functional.avg_pool1d(tt, omega, omega)[0, 0].numpy()
    mx = torch.nn.functional.max_pool1d(tt, omega, omega)[0, 0].numpy()
    np.testing.assert_allclose(oracle.window_scores(t, omega, omega), avg, rtol=1e-14)
    np.testing.assert_allclose(oracle.window_scores(t, omega, 1), mx, rtol=0)
    # p > omega behaves like p = omega (divisor min(p, omega))
    np.testing.assert_allclose(oracle.window_scores(t, omega, omega + 5), avg, rtol=1e-14)
    prev = mx
    for p in range(2, omega + 1):          # monotone non-increasing in p, between mean and max
        cur = oracle.window_scores(t, omega, p)
        assert (cur <= prev + 1e-15).all() and (cur >= avg - 1e-15).all()
        prev = cur
    # top-p equals sorting each window by a library sort
    p = omega // 2
    srt = np.sort(t.reshape(-1, omega), axis=1)[:, ::-1][:, :p].mean(axis=1)
    np.testing.assert_allclose(oracle.window_scores(t, omega, p), srt, rtol=1e-14)


def test_pooling_ragged_last_window_handworked():
    # n_r = omega + 3, omega = 4: windows {1,5,2,4} and {9,3,6}
    t = np.array([1, 5, 2, 4, 9, 3, 6], dtype=np.float64)
    np.testing.assert_allclose(oracle.window_scores(t, 4, 4), [12 / 4, 18 / 3])
    np.testing.assert_allclose(oracle.window_scores(t, 4, 2), [9 / 2, 15 / 2])
    np.testing.assert_allclose(oracle.window_scores(t, 4, 3), [11 / 3, 18 / 3])
    np.testing.assert_allclose(oracle.window_scores(t, 4, 1), [5, 9])


# ------------------------------------------------------------------ selection
def test_integer_formulas():
    assert oracle.num_windows(1024, 8, 8) == 127
    assert oracle.num_windows(8, 8, 8) == 0 and oracle.num_windows(5, 8, 8) == 0
    assert oracle.num_windows(9, 8, 8) == 1
    assert oracle.num_selected(1024, 8, 8, 128) == 15          # (128-8)/8
    assert oracle.num_selected(8192, 32, 8, 983) == 118
    assert oracle.num_selected(32768, 32, 16, 3932) == 243
    assert oracle.num_selected(100, 8, 8, 5) == 0              # budget below alpha
    assert oracle.num_selected(100, 8, 8, 10 ** 6) == 12       # budget above n: every window
    for n, a, w, b in itertools.product([1, 7, 64, 100], [1, 8], [3, 8], [0, 8, 9, 40, 1000]):
        k = oracle.num_selected(n, a, w, b)
        assert 0 <= k <= oracle.num_windows(n, a, w)
        if b >= a:
            assert k * w + a <= max(b, a) or k == 0


@pytest.mark.parametrize("seed", range(6))
def test_topk_bruteforce_subset_enumeration(seed):
    g = np.random.Generator(np.random.Philox(key=100 + seed))
    kw = int(g.integers(2, 13))
    k = int(g.integers(1, kw + 1))
    # few distinct values => many exact ties
    scores = g.integers(0, 4, size=kw).astype(np.float32) / 4
    idx = oracle.select_topk(scores, k)
    assert len(idx) == k and (np.diff(idx) > 0).all() and idx.min() >= 0 and idx.max() < kw
    best = None
    for sub in itertools.combinations(range(kw), k):
        tot = float(scores[list(sub)].astype(np.float64).sum())
        key = (-tot, sub)                  # max total, then lexicographically smallest
        if best is None or key < best:
            best = key
    assert tuple(idx) == best[1]


def test_topk_invariants_and_equivariance():
    g = np.random.Generator(np.random.Philox(key=200))
    s = g.standard_normal(500).astype(np.float32)
    k = 37
    idx = oracle.select_topk(s, k)
    thr = np.sort(s)[-k]
    assert set(idx) == set(np.nonzero(s >= thr)[0])            # no ties in Gaussian draws
    np.testing.assert_array_equal(oracle.select_topk(np.ones(20, np.float32), 5), np.arange(5))
    perm = g.permutation(500)
    idx_p = oracle.select_topk(s[perm], k)
    assert set(perm[idx_p]) == set(idx)
    assert len(oracle.select_topk(s, 0)) == 0
    np.testing.assert_array_equal(oracle.select_topk(s, 10 ** 6), np.arange(500))


# ------------------------------------------------------------------ gather + whole path
def _small_group(dtype="bf16", ragged=False, seed_cfg=2):
    base = wl.llama8b_single_group()
    return wl.scaled(base, name="small", dtype=dtype, n_q_heads=4, n_kv_heads=2, head_dim=32,
                     max_seqlen=203 if not ragged else 256, l_obs=8, window=8, n_layers=2, gamma=2,
                     n_planted=3, batch=3 if ragged else 2, ragged=ragged, budget_frac=0.3)


@pytest.mark.parametrize("ragged", [False, True])
def test_gather_spot_checks_and_budget_invariants(ragged):
    w = _small_group(ragged=ragged)
    grp = wl.make_group(w, 0)
    res = oracle.compress_group(grp["q_obs"], grp["k_layers"], grp["v_layers"], n_kv_heads=w.n_kv_heads,
                                l_obs=w.l_obs, window=w.window, task=w.task, top_p=w.top_p,
                                max_seqlen=w.max_seqlen, budgets=grp["budgets"], cu_seqlens=grp["cu_seqlens"],
                                fill=0xABCD)
    seqlens, cu = grp["seqlens"], grp["cu_seqlens"]
    for b in range(w.batch):
        n = int(seqlens[b]); n_r = n - w.l_obs
        ksel = oracle.num_selected(n, w.l_obs, w.window, int(grp["budgets"][b]))
        assert ksel * w.window + w.l_obs <= grp["budgets"][b]
        for h in range(w.n_kv_heads):
            idx = res["window_idx"][b, h]
            sel = idx[:ksel]
            assert (idx[ksel:] == -1).all() and (np.diff(sel) > 0).all()
            assert sel.min() >= 0 and sel.max() < oracle.num_windows(n, w.l_obs, w.window)
            # source row of each output row, derived independently of the gather loop
            rows = np.concatenate([np.arange(i * w.window, min((i + 1) * w.window, n_r)) for i in sel]
                                  + [np.arange(n_r, n)])
            assert res["kept_len"][b, h] == len(rows)
            for layer in range(w.gamma):
                for src, out in ((grp["k_layers"][layer], res["k_out"][layer]),
                                 (grp["v_layers"][layer], res["v_out"][layer])):
                    src_u = src[cu[b]:cu[b + 1], h] if ragged else src[b, h]
                    np.testing.assert_array_equal(out[b, h, : len(rows)], src_u[rows])
                    assert (out[b, h, len(rows):] == 0xABCD).all()
            planted = wl.planted_windows(w, b, h, n)
            assert set(planted) <= set(sel), "planted windows must be retained"


@pytest.mark.parametrize("ragged", [False, True])
def test_gather_into_the_packed_output_layout(ragged):
    """The packed compact cache [T_out, H_kv, d]: sequence b starts at row cu_seqlens_out[b], its rows
    are token-major with the KV heads interleaved.  Every output element is located here by index
    arithmetic written independently of the oracle's gather loop, on given (not selected) indices
    that differ per head and include the ragged last window; slack rows between sequences and rows
    behind a unit's kept length must keep the fill."""
    w = _small_group(ragged=ragged)
    grp = wl.make_group(w, 0)
    seqlens, cu = grp["seqlens"], grp["cu_seqlens"]
    H, d = w.n_kv_heads, w.head_dim
    ks = [oracle.num_selected(int(n), w.l_obs, w.window, int(b)) for n, b in zip(seqlens, grp["budgets"])]
    k_max = max(ks)
    idx = np.full((w.batch, H, k_max), -1, dtype=np.int32)
    for b in range(w.batch):
        kw = oracle.num_windows(int(seqlens[b]), w.l_obs, w.window)
        for h in range(H):
            # head 0: every other window and the (short) last one; head 1: the first k windows
            cand = np.unique(np.concatenate([np.arange(h, kw, 2)[: ks[b] - 1], [kw - 1]]))[: ks[b]] if h == 0 \
                else np.arange(ks[b])
            assert len(cand) == ks[b]
            idx[b, h, : ks[b]] = cand
    slack = [3, 0, 5][: w.batch]                       # unused rows behind each sequence's share
    cu_out = np.zeros(w.batch + 1, dtype=np.int32)
    for b in range(w.batch):
        cu_out[b + 1] = cu_out[b] + ks[b] * w.window + w.l_obs + slack[b]
    FILL = 0x5A5A
    src = grp["v_layers"][1]
    out = oracle.gather_layer(src, idx, n_kv_heads=H, l_obs=w.l_obs, window=w.window, max_seqlen=w.max_seqlen,
                              budgets=grp["budgets"], keep_max=0, cu_seqlens=cu, cu_seqlens_out=cu_out, fill=FILL)
    assert out.shape == (int(cu_out[-1]), H, d)
    flat = out.reshape(-1)                              # element (row, h, c) at (row * H + h) * d + c
    written = np.zeros(out.shape[:2], dtype=bool)
    for b in range(w.batch):
        n = int(seqlens[b]); n_r = n - w.l_obs
        for h in range(H):
            rows = np.concatenate([np.arange(i * w.window, min((i + 1) * w.window, n_r)) for i in idx[b, h, : ks[b]]]
                                  + [np.arange(n_r, n)])
            src_u = src[cu[b]:cu[b + 1], h] if ragged else src[b, h]
            for r, j in enumerate(rows):
                base = ((int(cu_out[b]) + r) * H + h) * d
                np.testing.assert_array_equal(flat[base: base + d], src_u[j])
                written[int(cu_out[b]) + r, h] = True
            # head 0 holds the short last window, head 1 does not: the kept lengths differ
            assert len(rows) == ks[b] * w.window + w.l_obs - (w.window - (n_r - (oracle.num_windows(n, w.l_obs, w.window) - 1) * w.window) if h == 0 else 0)
    assert (out[~written] == FILL).all() and (~written).sum() > 0


@pytest.mark.parametrize("ragged", [False, True])
def test_batch_driver_maps_heads_and_sequences_as_the_library_softmax_does(ragged):
    """The batch driver (`select_leader`) has to pick, for unit (b, h), sequence b's rows of the packed or
    dense K, KV head h's keys, and the query heads h*G .. h*G+G-1 (grouped-query attention).  Pinned
    against an independent library computation per unit: torch CPU softmax with a causal mask, summed
    over exactly those rows, then average / max pooling by torch for the window scores.  A wrong head
    mapping, sequence offset or stride gives other scores."""
    w = wl.scaled(_small_group(ragged=ragged), n_q_heads=6, n_kv_heads=3, task=wl.TASK_LOCALIZATION)
    grp = wl.make_group(w, 0)
    res = oracle.select_leader(grp["q_obs"], grp["k_layers"][0], n_kv_heads=w.n_kv_heads, l_obs=w.l_obs,
                               window=w.window, task=w.task, top_p=w.top_p, max_seqlen=w.max_seqlen,
                               budgets=grp["budgets"], cu_seqlens=grp["cu_seqlens"], want_tokens=True)
    q = torch.from_numpy(wl.to_f32(grp["q_obs"])).double()            # [B, H_q, alpha, d]
    k = torch.from_numpy(wl.to_f32(grp["k_layers"][0])).double()
    G, a = w.n_q_heads // w.n_kv_heads, w.l_obs
    for b in range(w.batch):
        n = int(grp["seqlens"][b])
        for h in range(w.n_kv_heads):
            kb = k[int(grp["cu_seqlens"][b]): int(grp["cu_seqlens"][b]) + n, h] if ragged else k[b, h, :n]
            t = torch.zeros(n - a, dtype=torch.float64)
            for g in range(G):
                logits = q[b, h * G + g] @ kb.T / w.head_dim ** 0.5                       # [alpha, n]
                pos = torch.arange(n - a, n).view(a, 1)
                logits = logits.masked_fill(torch.arange(n).view(1, n) > pos, float("-inf"))
                t += torch.softmax(logits, dim=-1)[:, : n - a].sum(0)
            np.testing.assert_allclose(res["token_scores"][b, h, : n - a], t.numpy(), rtol=1e-10, atol=0)
            full = (n - a) // w.window
            pooled = torch.nn.functional.avg_pool1d(t.view(1, 1, -1), w.window, w.window).view(-1).numpy()
            np.testing.assert_allclose(res["window_scores_f64"][b, h, :full], pooled[:full], rtol=1e-10, atol=0)


def test_budget_above_context_is_identity_copy():
    w = wl.scaled(_small_group(), budget_frac=None, budget_tokens=10 ** 6)
    grp = wl.make_group(w, 0)
    res = oracle.compress_group(grp["q_obs"], grp["k_layers"], grp["v_layers"], n_kv_heads=w.n_kv_heads,
                                l_obs=w.l_obs, window=w.window, task=w.task, top_p=w.top_p,
                                max_seqlen=w.max_seqlen, budgets=grp["budgets"])
    n = w.max_seqlen
    assert (res["kept_len"] == n).all()
    np.testing.assert_array_equal(res["k_out"][1][:, :, :n], grp["k_layers"][1])
    np.testing.assert_array_equal(res["v_out"][0][:, :, :n], grp["v_layers"][0])


def test_budget_below_alpha_keeps_only_observation_rows():
    w = wl.scaled(_small_group(), budget_frac=None, budget_tokens=3)
    grp = wl.make_group(w, 0)
    res = oracle.compress_group(grp["q_obs"], grp["k_layers"], grp["v_layers"], n_kv_heads=w.n_kv_heads,
                                l_obs=w.l_obs, window=w.window, task=w.task, top_p=w.top_p,
                                max_seqlen=w.max_seqlen, budgets=grp["budgets"])
    assert (res["kept_len"] == w.l_obs).all()
    np.testing.assert_array_equal(res["k_out"][0][:, :, : w.l_obs], grp["k_layers"][0][:, :, -w.l_obs:])


def test_config1_planted_windows_selected():
    w = wl.tiny()
    grp = wl.make_group(w, 0)
    res = oracle.compress_group(grp["q_obs"], grp["k_layers"], grp["v_layers"], n_kv_heads=w.n_kv_heads,
                                l_obs=w.l_obs, window=w.window, task=w.task, top_p=w.top_p,
                                max_seqlen=w.max_seqlen, budgets=grp["budgets"], want_tokens=True)
    assert res["k_max"] == 15 and res["keep_max"] == 128
    for h in range(w.n_kv_heads):
        assert set(wl.planted_windows(w, 0, h, 1024)) <= set(res["window_idx"][0, h])
        assert np.nanmin(res["token_scores"][0, h]) > 1e-30


def test_aggregation_differs_from_localization_only_through_p():
    w = _small_group()
    grp = wl.make_group(w, 0)
    common = dict(n_kv_heads=w.n_kv_heads, l_obs=w.l_obs, window=w.window, max_seqlen=w.max_seqlen,
                  budgets=grp["budgets"], want_tokens=True)
    loc = oracle.select_leader(grp["q_obs"], grp["k_layers"][0], task=wl.TASK_LOCALIZATION, top_p=3, **common)
    agg = oracle.select_leader(grp["q_obs"], grp["k_layers"][0], task=wl.TASK_AGGREGATION, top_p=3, **common)
    np.testing.assert_array_equal(loc["token_scores"], agg["token_scores"])
    t = loc["token_scores"][1, 0][: w.max_seqlen - w.l_obs]
    np.testing.assert_allclose(loc["window_scores_f64"][1, 0][: len(t) // 8 + 1], oracle.window_scores(t, 8, 8))
    np.testing.assert_allclose(agg["window_scores_f64"][1, 0][: len(t) // 8 + 1], oracle.window_scores(t, 8, 3))
    assert oracle.effective_p(wl.TASK_AGGREGATION, 8, 0) == 4 and oracle.effective_p(wl.TASK_LOCALIZATION, 8, 3) == 8


def test_workload_shapes_match_the_configs():
    c2, c3, c5 = wl.llama8b_single_group(), wl.llama8b_full(), wl.batched_ragged()
    assert int(c2.budgets()[0]) == 983 and int(c3.budgets()[0]) == 3932
    assert c3.rows == 128 and c5.rows == 256 and wl.mistral_needle(4096).rows == 64
    n5 = c5.seqlens()
    assert n5.min() >= 32768 and n5.max() <= 65536 and len(n5) == 8
    x = np.array([1.0, 1.00390625, 1.01171875, -3.0e-40, np.inf], dtype=np.float32)
    back = wl.bf16_bits_to_f32(wl.f32_to_bf16_bits(x))
    tx = torch.from_numpy(x).to(torch.bfloat16).float().numpy()      # library rounding
    np.testing.assert_array_equal(back, tx)


# ------------------------------------------------------------------ Eq. 5-7: pyramid budgets
def test_group_budgets_closed_forms():
    from fractions import Fraction
    # the configuration of the paper's main experiments: 32 layers, groups of 8, lambda = 14, and an
    # average of 2048 tokens per layer.  Hand-derived from Eq. 6-7: b^3 = 65536/56, b^0 = 32768 - b^3.
    r = oracle.group_budgets(32, 8, 32 * 2048, 14)
    assert r["group"][3] == Fraction(65536, 56) and r["group"][0] == Fraction(32768) - Fraction(65536, 56)
    assert [round(float(x), 1) for x in r["per_layer"]] == [3949.7, 2681.9, 1414.1, 146.3]
    for n_layers, gamma, total, lam in [(32, 8, 65536, 14), (28, 7, 28 * 512, 14), (32, 4, 32 * 1024, Fraction(7, 2)),
                                        (32, 1, 32 * 2048, 14), (8, 8, 4096, 14)]:
        r = oracle.group_budgets(n_layers, gamma, total, lam)
        b, H = r["group"], n_layers // gamma
        assert sum(b) == total                                            # Eq. 5
        if H > 1:
            assert b[-1] * lam * H == total                               # Eq. 6
            assert len({b[h] - b[h + 1] for h in range(H - 1)}) == 1      # Eq. 7: arithmetic sequence
            assert b[0] >= b[-1]
        ints = r["per_layer_int"]
        assert 0 <= total - gamma * sum(ints) < gamma                     # nothing above the budget, < gamma lost
        assert all(ints[h] == int(r["per_layer"][h]) for h in range(1, H))


def test_group_budgets_library_matches_oracle():
    from fractions import Fraction
    from paper_2503_17922_b200 import binding, build
    build.build_library()
    for n_layers, gamma, total, num, den in [(32, 8, 65536, 14, 1), (28, 7, 14336, 14, 1), (32, 4, 32768, 7, 2),
                                             (32, 1, 65536, 14, 1), (8, 8, 4096, 14, 1), (32, 8, 12345, 3, 1),
                                             (64, 4, 10 ** 9, 14, 1), (32, 8, 0, 14, 1), (32, 8, 100, 1, 1)]:
        got = binding.wkv_group_budgets(n_layers, gamma, total, num, den)
        exp = oracle.group_budgets(n_layers, gamma, total, Fraction(num, den))["per_layer_int"]
        assert got.tolist() == exp, (n_layers, gamma, total, num, den)
    with pytest.raises(binding.WkvError):
        binding.wkv_group_budgets(30, 8, 1000)
    with pytest.raises(binding.WkvError):
        binding.wkv_group_budgets(32, 8, 1000, 1, 2)      # lambda < 1
