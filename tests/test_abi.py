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


def test_keep_len_matches_the_oracle_formulas(L):
    k = ctypes.c_int32(-5)
    for n in (1, 7, 8, 9, 17, 100, 1024, 1027, 32768):
        for a in (1, 8, 32):
            for w in (1, 3, 8, 16, 32):
                for b in (0, a, a + w - 1, a + w, 983, 10 ** 6):
                    rows = L.wkv_keep_len(n, a, w, b, ctypes.byref(k))
                    k_ref = oracle.num_selected(n, a, w, b)
                    assert k.value == k_ref
                    n_r = max(n - a, 0)
                    # the largest set of k windows in rows: the k first ones (all full unless k == K_w)
                    assert rows == min(k_ref * w, n_r) + min(a, n)
                    assert rows == oracle.keep_max([n], [b], a, w) or k_ref == oracle.num_windows(n, a, w)
                    assert rows <= n and (b < a or rows <= max(b, min(a, n)))
    assert L.wkv_keep_len(100, 8, 8, 64, None) == 64      # k = 7 windows of 8 + 8 observation rows
    assert L.wkv_keep_len(-1, 8, 8, 64, None) == -1 and L.wkv_keep_len(10, 0, 8, 64, None) == -1


def test_sync_word_helper(L):
    s = _shape()
    t, a = ctypes.c_size_t(0), ctypes.c_size_t(0)
    need = L.wkv_workspace_bytes(ctypes.byref(s))
    seen = set()
    for unit in range(2):
        assert L.wkv_workspace_sync_words(ctypes.byref(s), unit, ctypes.byref(t), ctypes.byref(a)) == 0
        assert 4 <= t.value < a.value < need and t.value % 4 == 0 and a.value % 4 == 0
        seen |= {t.value, a.value}
    assert len(seen) == 4
    assert L.wkv_workspace_sync_words(ctypes.byref(s), 2, ctypes.byref(t), ctypes.byref(a)) == 2
    assert L.wkv_workspace_sync_words(ctypes.byref(s), 0, None, None) == 0


def test_host_entry_refuses_byte_counts_that_disagree_with_the_shape(L):
    """wkv_compress_group_host copies caller-sized byte ranges: sizes that do not cover the tensors
    of the shape, or an output size that is not exactly one dense compact cache, are refused on the
    host before any copy is enqueued (no GPU needed to see the refusal)."""
    s = _shape()
    ptrs = (ctypes.c_void_p * 4)(*([0x1000] * 4))
    kv_bytes = 2 * 1024 * 64 * 2
    q_bytes = 4 * 8 * 64 * 2
    cap = L.wkv_keep_max(ctypes.byref(s))
    out_bytes = 2 * cap * 64 * 2
    need = L.wkv_workspace_bytes(ctypes.byref(s))

    def call(qb=q_bytes, kb=kv_bytes, ob=out_bytes, capacity=cap):
        return L.wkv_compress_group_host(ctypes.byref(s), 2, 0x1000, qb, ptrs, ptrs, kb, ptrs, ptrs, ob, 0x1000, 0x1000,
                                         0x1000, ptrs, ptrs, ptrs, ptrs, 0x1000, 0x1000, capacity, 0x1000, need, None)
    assert call(kb=kv_bytes - 2) == 2 and b"bytes_per_layer" in L.wkv_last_error_detail()
    assert call(qb=q_bytes - 2) == 2
    assert call(ob=out_bytes - 2) == 2 and b"out_bytes_per_layer" in L.wkv_last_error_detail()
    assert call(ob=out_bytes + 128) == 2
    assert call(capacity=cap - 1, ob=2 * (cap - 1) * 64 * 2) == 2
    assert L.wkv_launch_count() == 0


def test_gather_refuses_a_cache_that_is_its_own_input(L):
    s = _shape()
    a = (ctypes.c_void_p * 2)(0x1000, 0x2000)
    b = (ctypes.c_void_p * 2)(0x3000, 0x2000)      # layer 1: output == input
    assert L.wkv_gather_kv(ctypes.byref(s), 2, a, None, 0x100, b, None, None, 128, None) == 2
    assert b"must not be the input" in L.wkv_last_error_detail()


def test_jaccard_of_index_sets(L):
    """Section 3.2's similarity measure: closed cases (identical, disjoint, nested, both empty), and the
    library's merge walk against the oracle's set arithmetic on random selections."""
    pad = lambda xs, k: np.array(list(xs) + [-1] * (k - len(xs)), dtype=np.int32)
    a = np.stack([pad([0, 3, 5, 9], 6), pad([1, 2], 6), pad([0, 1, 2, 3], 6), pad([], 6), pad([4], 6)])
    b = np.stack([pad([0, 3, 5, 9], 6), pad([3, 4], 6), pad([1, 2], 6), pad([], 6), pad([], 6)])
    per_unit, mean = binding.wkv_jaccard_windows(a, b)
    assert per_unit.tolist() == [1.0, 0.0, 0.5, 1.0, 0.0] and abs(mean - 0.5) < 1e-15
    np.testing.assert_array_equal(per_unit, oracle.jaccard_windows(a, b))
    g = np.random.Generator(np.random.Philox(key=5))
    A = np.full((3, 4, 40), -1, dtype=np.int32)
    B = np.full((3, 4, 40), -1, dtype=np.int32)
    for pos in np.ndindex(3, 4):
        for M in (A, B):
            n = int(g.integers(0, 41))
            M[pos][:n] = np.sort(g.choice(100, size=n, replace=False))
    per_unit, mean = binding.wkv_jaccard_windows(A, B)
    ref = oracle.jaccard_windows(A, B)
    np.testing.assert_allclose(per_unit, ref, rtol=0, atol=1e-15)
    assert abs(mean - ref.mean()) < 1e-12
    # symmetric, and 1 only for equal sets
    np.testing.assert_array_equal(per_unit, binding.wkv_jaccard_windows(B, A)[0])
    bad = a.copy()
    bad[0, :2] = [3, 3]
    with pytest.raises(binding.WkvError):
        binding.wkv_jaccard_windows(bad, b)


def test_missing_library_fails_loudly(monkeypatch):
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", "/nonexistent/libwkv.so")
    with pytest.raises(RuntimeError, match="no other implementation"):
        binding.lib()
