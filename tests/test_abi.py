"""CPU-only checks of the C-ABI library: it loads, exports what the header declares,
its host-side integer helpers agree with the oracle's, and argument errors are
reported before anything touches a GPU."""
import ctypes
import os
import re

import numpy as np
import pytest

import oracle
from paper_2503_17922_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def L():
    build.build_library()
    return binding.lib()


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "wkv.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(wkv_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(L):
    names = _declared_functions()
    assert len(names) >= 10
    for n in names:
        assert hasattr(L, n), f"{n} declared in wkv.h but not exported"
    assert sorted(binding.EXPORTED_SYMBOLS) == names


def test_struct_mirror_size(L):
    # 14 int32 + 4 pointers + 6 int64
    assert ctypes.sizeof(binding.WkvShape) == 14 * 4 + 4 * 8 + 6 * 8


def test_integer_helpers_match_oracle(L):
    for n in (1, 7, 8, 9, 100, 1024, 32768):
        for a in (1, 8, 32):
            for w in (1, 3, 8, 16, 32):
                assert L.wkv_num_windows(n, a, w) == oracle.num_windows(n, a, w)
                for b in (0, a, a + w - 1, a + w, 983, 10 ** 6):
                    assert L.wkv_num_selected(n, a, w, b) == oracle.num_selected(n, a, w, b)


def _shape(**kw):
    s = binding.WkvShape()
    s.struct_size = ctypes.sizeof(binding.WkvShape)
    s.dtype, s.batch, s.n_q_heads, s.n_kv_heads, s.head_dim = binding.WKV_BF16, 1, 4, 2, 64
    s.l_obs, s.window, s.top_p, s.task, s.max_seqlen, s.budget = 8, 8, 0, 0, 1024, 128
    s.stride_b, s.stride_h, s.stride_t = 2 * 1024 * 64, 1024 * 64, 64
    s.q_stride_b, s.q_stride_h, s.q_stride_t = 4 * 8 * 64, 8 * 64, 64
    for k, v in kw.items():
        setattr(s, k, v)
    return s


def test_leading_sizes(L):
    s = _shape()
    assert L.wkv_kw_max(ctypes.byref(s)) == 127
    assert L.wkv_k_max(ctypes.byref(s)) == 15
    assert L.wkv_keep_max(ctypes.byref(s)) == 128
    assert L.wkv_workspace_bytes(ctypes.byref(s)) > 0
    cu = np.array([0, 5, 905], dtype=np.int32)
    bud = np.array([64, 100], dtype=np.int32)
    s = _shape(batch=2, cu_seqlens_host=cu.ctypes.data, cu_seqlens_dev=0x1000,
               budgets_host=bud.ctypes.data, budgets_dev=0x2000, stride_b=0, stride_h=64, stride_t=128)
    assert L.wkv_kw_max(ctypes.byref(s)) == oracle.num_windows(900, 8, 8)
    assert L.wkv_k_max(ctypes.byref(s)) == 11
    assert L.wkv_keep_max(ctypes.byref(s)) == oracle.keep_max([5, 900], [64, 100], 8, 8) == 96


@pytest.mark.parametrize("kw,status", [
    (dict(struct_size=8), 2), (dict(dtype=5), 3), (dict(batch=0), 2), (dict(n_q_heads=3), 2),
    (dict(head_dim=4), 6), (dict(stride_t=68), 6), (dict(budget=-1), 4), (dict(task=2), 2),
    (dict(score_impl=9), 2), (dict(cu_seqlens_host=0x10), 1), (dict(l_obs=0), 2),
])
def test_argument_errors_are_host_side(L, kw, status):
    s = _shape(**kw)
    st = L.wkv_score_windows(ctypes.byref(s), 0x100, 0x100, 0x100, None, 0x100, 1 << 30, None)
    assert st == status, L.wkv_last_error_detail()
    assert L.wkv_workspace_bytes(ctypes.byref(s)) == 0
    assert len(L.wkv_status_string(st)) > 0 and len(L.wkv_last_error_detail()) > 0


def test_null_workspace_alignment_and_limits(L):
    s = _shape()
    need = L.wkv_workspace_bytes(ctypes.byref(s))
    assert L.wkv_score_windows(ctypes.byref(s), None, 0x100, 0x100, None, 0x100, need, None) == 1
    assert L.wkv_score_windows(ctypes.byref(s), 0x100, 0x100, 0x100, None, None, need, None) == 5
    assert L.wkv_score_windows(ctypes.byref(s), 0x100, 0x100, 0x100, None, 0x100, need - 1, None) == 5
    assert L.wkv_score_windows(ctypes.byref(s), 0x100, 0x100, 0x100, None, 0x110, need, None) == 5
    assert L.wkv_score_windows(ctypes.byref(s), 0x108, 0x100, 0x100, None, 0x100, need, None) == 6
    ptrs = (ctypes.c_void_p * 40)(*([0x100] * 40))
    assert L.wkv_gather_kv(ctypes.byref(s), 33, ptrs, ptrs, 0x100, ptrs, ptrs, None, 128, None) == 9
    assert L.wkv_gather_kv(ctypes.byref(s), 2, ptrs, ptrs, 0x100, ptrs, ptrs, None, 127, None) == 2
    assert L.wkv_gather_kv(ctypes.byref(s), 2, ptrs, ptrs, None, ptrs, ptrs, None, 128, None) == 1
    assert L.wkv_launch_count() == 0


def test_missing_library_fails_loudly(monkeypatch):
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", "/nonexistent/libwkv.so")
    with pytest.raises(RuntimeError, match="no other implementation"):
        binding.lib()
