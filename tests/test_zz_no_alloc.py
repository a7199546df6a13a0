"""The allocation-free scoring entry point (collected last on purpose: a failure here must not hide
any other test from a run that stops at the first failure).

wkv_score_windows_static serves hosts that cannot hand the library a workspace: an inference
engine that reserved all device memory for its own pools, or code that runs where cudaMalloc is not
allowed.  It must give the results of wkv_score_windows, call after call, out of one built-in
scratch area that keeps whatever the previous call left in it."""
import ctypes

import numpy as np
import oracle
import pytest
import torch

from paper_2503_17922_b200 import binding
from paper_2503_17922_b200 import workloads as wl

import parity_util as pu


def _case(**kw):
    base = dict(name="no-alloc", batch=2, n_layers=1, gamma=1, n_q_heads=8, n_kv_heads=2, head_dim=128,
                max_seqlen=2500, l_obs=16, window=8, top_p=4, budget_frac=0.2, n_planted=5, config_id=11)
    base.update(kw)
    return wl.scaled(wl.llama8b_single_group(), **base)


@pytest.mark.gpu
def test_static_scratch_matches_workspace_entry_twice_in_a_row():
    # two different problems back to back: the second call finds the first one's statistics in the
    # shared area (more rows, more chunks) and must not be disturbed by them.  Each call is held
    # against the CPU oracle's window and token scores (the 1e-3 rule) and, bit for bit, against
    # the entry point that takes a caller workspace: both run the same kernels in a fixed order.
    for w in (_case(n_q_heads=16, l_obs=32, max_seqlen=4000), _case(task=wl.TASK_AGGREGATION)):
        grp = wl.make_group(w, 0)
        prob = binding.Problem.from_workload(w)
        assert prob.workspace_bytes <= binding.WKV_STATIC_SCRATCH_BYTES
        q = binding.to_device(grp["q_obs"])
        k = binding.to_device(grp["k_layers"][0])
        shape = (w.batch, w.n_kv_heads, prob.kw_max)
        expected = torch.full(shape, float("nan"), dtype=torch.float32, device="cuda")
        tok_expected = torch.full((w.batch, w.n_kv_heads, prob.nr_max), float("nan"), dtype=torch.float32, device="cuda")
        work = prob.alloc_workspace()
        binding.wkv_score_windows(prob, q, k, expected, tok_expected, work)
        ref = oracle.select_leader(grp["q_obs"], grp["k_layers"][0], want_tokens=True, **pu.oracle_kwargs(w, grp))
        for call in range(2):
            got = torch.full(shape, float("nan"), dtype=torch.float32, device="cuda")
            tok = torch.full_like(tok_expected, float("nan"))
            status = torch.full((1,), -1, dtype=torch.int32, device="cuda")
            binding.wkv_score_windows_static(prob, q, k, got, tok, status)
            torch.cuda.synchronize()
            assert int(status.item()) == 0
            e, g = expected.cpu().numpy(), got.cpu().numpy()
            valid = ~np.isnan(e)
            assert valid.any() and (np.isnan(g) == ~valid).all()
            o = ref["window_scores"].astype(np.float64)
            assert (~np.isnan(o) == valid).all()
            np.testing.assert_allclose(g[valid], o[valid], rtol=pu.SCORE_RTOL, atol=0)
            np.testing.assert_array_equal(g[valid], e[valid])
            te, tg, to = tok_expected.cpu().numpy(), tok.cpu().numpy(), ref["token_scores"]
            tv = ~np.isnan(te)
            assert (~np.isnan(to) == tv).all()
            np.testing.assert_allclose(tg[tv], to[tv], rtol=pu.SCORE_RTOL, atol=0)
            np.testing.assert_array_equal(tg[tv], te[tv])
        assert binding.device_status(work) == 0


def test_static_scratch_refuses_shapes_beyond_its_size():
    # host-side check only: nothing is enqueued, so this also runs without a GPU
    binding.lib()
    s = binding.WkvShape()
    s.struct_size = ctypes.sizeof(binding.WkvShape)
    s.dtype, s.batch, s.n_q_heads, s.n_kv_heads, s.head_dim = binding.WKV_BF16, 8, 32, 8, 128
    s.l_obs, s.window, s.top_p, s.task, s.max_seqlen, s.budget = 64, 32, 16, 1, 65536, 7000
    s.stride_b, s.stride_h, s.stride_t = 8 * 65536 * 128, 65536 * 128, 128
    s.q_stride_b, s.q_stride_h, s.q_stride_t = 32 * 64 * 128, 64 * 128, 128
    L = binding.lib()
    assert L.wkv_workspace_bytes(ctypes.byref(s)) > binding.WKV_STATIC_SCRATCH_BYTES
    st = L.wkv_score_windows_static(ctypes.byref(s), 0x1000, 0x1000, 0x1000, None, None, None)
    assert st == 9 and b"built-in area" in L.wkv_last_error_detail()
