"""Thin ctypes binding of the C-ABI library (include/wkv.h).

Argument marshalling only: every step of the path runs in the library's CUDA
kernels.  Tensors are torch CUDA tensors used purely as device memory; their
`data_ptr()` and the current stream's handle are what crosses the boundary.
There is no CPU fallback: if the shared library is missing, loading fails.
"""
from __future__ import annotations

import ctypes
import os
from typing import List, Optional, Sequence

import numpy as np

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libwkv.so")

WKV_F32, WKV_BF16 = 0, 1
WKV_TASK_LOCALIZATION, WKV_TASK_AGGREGATION = 0, 1
WKV_SCORE_AUTO, WKV_SCORE_SIMT, WKV_SCORE_TCGEN05, WKV_SCORE_TCGEN05_PIPELINED = 0, 1, 2, 3
WKV_MAX_GROUP_LAYERS = 32

EXPORTED_SYMBOLS = [
    "wkv_num_windows", "wkv_num_selected", "wkv_keep_len", "wkv_workspace_sync_words", "wkv_kw_max", "wkv_k_max", "wkv_keep_max", "wkv_group_budgets", "wkv_jaccard_windows",
    "wkv_workspace_bytes", "wkv_score_windows", "wkv_score_windows_static", "wkv_select_topk_windows", "wkv_gather_kv", "wkv_gather_kv_paged", "wkv_compact_kv_inplace",
    "wkv_compress_group", "wkv_compress_group_host", "wkv_score_windows_lse", "wkv_compress_group_lse",
    "wkv_select_leader_windows", "wkv_probe_ex2_rate", "wkv_probe_colsum_rate", "wkv_group_plan_create", "wkv_group_plan_launch", "wkv_group_plan_destroy", "wkv_status_string", "wkv_last_error_detail",
    "wkv_launch_count",
]


class WkvShape(ctypes.Structure):
    """Mirror of `wkv_shape`."""
    _fields_ = [
        ("struct_size", ctypes.c_uint32),
        ("dtype", ctypes.c_int32),
        ("batch", ctypes.c_int32),
        ("n_q_heads", ctypes.c_int32),
        ("n_kv_heads", ctypes.c_int32),
        ("head_dim", ctypes.c_int32),
        ("l_obs", ctypes.c_int32),
        ("window", ctypes.c_int32),
        ("top_p", ctypes.c_int32),
        ("task", ctypes.c_int32),
        ("max_seqlen", ctypes.c_int32),
        ("budget", ctypes.c_int32),
        ("score_impl", ctypes.c_int32),
        ("reserved", ctypes.c_int32),
        ("cu_seqlens_host", ctypes.c_void_p),
        ("cu_seqlens_dev", ctypes.c_void_p),
        ("budgets_host", ctypes.c_void_p),
        ("budgets_dev", ctypes.c_void_p),
        ("stride_b", ctypes.c_int64),
        ("stride_h", ctypes.c_int64),
        ("stride_t", ctypes.c_int64),
        ("q_stride_b", ctypes.c_int64),
        ("q_stride_h", ctypes.c_int64),
        ("q_stride_t", ctypes.c_int64),
    ]


class WkvError(RuntimeError):
    def __init__(self, status: int, what: str, detail: str):
        super().__init__(f"{what}: status {status} ({detail})")
        self.status = status


_lib = None


def lib() -> ctypes.CDLL:
    """Loads libwkv.so; raises if it has not been built (no fallback exists)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2503_17922_b200.build` "
                           "(needs nvcc); this package has no other implementation of the path")
    L = ctypes.CDLL(LIB_PATH)
    vp, i32, sz = ctypes.c_void_p, ctypes.c_int32, ctypes.c_size_t
    sp = ctypes.POINTER(WkvShape)
    L.wkv_num_windows.restype = i32
    L.wkv_num_windows.argtypes = [i32, i32, i32]
    L.wkv_num_selected.restype = i32
    L.wkv_num_selected.argtypes = [i32, i32, i32, i32]
    L.wkv_keep_len.restype = i32
    L.wkv_keep_len.argtypes = [i32, i32, i32, i32, ctypes.POINTER(i32)]
    L.wkv_workspace_sync_words.restype = ctypes.c_int
    L.wkv_workspace_sync_words.argtypes = [sp, i32, ctypes.POINTER(sz), ctypes.POINTER(sz)]
    for name in ("wkv_kw_max", "wkv_k_max", "wkv_keep_max"):
        getattr(L, name).restype = i32
        getattr(L, name).argtypes = [sp]
    L.wkv_group_budgets.restype = ctypes.c_int
    L.wkv_group_budgets.argtypes = [i32, i32, ctypes.c_int64, i32, i32, vp]
    L.wkv_jaccard_windows.restype = ctypes.c_int
    L.wkv_jaccard_windows.argtypes = [vp, vp, i32, i32, vp, ctypes.POINTER(ctypes.c_double)]
    L.wkv_workspace_bytes.restype = sz
    L.wkv_workspace_bytes.argtypes = [sp]
    L.wkv_score_windows.restype = ctypes.c_int
    L.wkv_score_windows.argtypes = [sp, vp, vp, vp, vp, vp, sz, vp]
    L.wkv_score_windows_static.restype = ctypes.c_int
    L.wkv_score_windows_static.argtypes = [sp, vp, vp, vp, vp, vp, vp]
    L.wkv_select_topk_windows.restype = ctypes.c_int
    L.wkv_select_topk_windows.argtypes = [sp, vp, vp, vp, vp]
    L.wkv_gather_kv.restype = ctypes.c_int
    L.wkv_gather_kv.argtypes = [sp, i32, vp, vp, vp, vp, vp, vp, i32, vp]
    L.wkv_gather_kv_paged.restype = ctypes.c_int
    L.wkv_gather_kv_paged.argtypes = [sp, i32, vp, vp, vp, vp, vp, vp, i32, i32, i32, ctypes.c_int64, ctypes.c_int64,
                                      ctypes.c_int64, vp]
    L.wkv_compact_kv_inplace.restype = ctypes.c_int
    L.wkv_compact_kv_inplace.argtypes = [sp, i32, vp, vp, vp, vp]
    L.wkv_compress_group.restype = ctypes.c_int
    L.wkv_compress_group.argtypes = [sp, i32, vp, vp, vp, vp, vp, vp, vp, vp, vp, i32, vp, sz, vp]
    L.wkv_score_windows_lse.restype = ctypes.c_int
    L.wkv_score_windows_lse.argtypes = [sp, vp, vp, vp, vp, vp, vp, sz, vp]
    L.wkv_compress_group_lse.restype = ctypes.c_int
    L.wkv_compress_group_lse.argtypes = [sp, i32, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, i32, vp, sz, vp]
    L.wkv_select_leader_windows.restype = ctypes.c_int
    L.wkv_select_leader_windows.argtypes = [sp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
    L.wkv_group_plan_create.restype = ctypes.c_int
    L.wkv_group_plan_create.argtypes = [sp, i32, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, i32, vp, sz,
                                        ctypes.POINTER(vp)]
    L.wkv_group_plan_launch.restype = ctypes.c_int
    L.wkv_group_plan_launch.argtypes = [vp, vp]
    L.wkv_group_plan_destroy.restype = None
    L.wkv_group_plan_destroy.argtypes = [vp]
    L.wkv_compress_group_host.restype = ctypes.c_int
    L.wkv_compress_group_host.argtypes = [sp, i32, vp, sz, vp, vp, sz, vp, vp, sz, vp, vp,
                                          vp, vp, vp, vp, vp, vp, vp, i32, vp, sz, vp]
    L.wkv_probe_ex2_rate.restype = ctypes.c_int
    L.wkv_probe_ex2_rate.argtypes = [vp, i32, i32, i32, ctypes.POINTER(ctypes.c_int64), vp]
    L.wkv_probe_colsum_rate.restype = ctypes.c_int
    L.wkv_probe_colsum_rate.argtypes = [vp, i32, i32, i32, ctypes.POINTER(ctypes.c_int64), vp]
    L.wkv_status_string.restype = ctypes.c_char_p
    L.wkv_status_string.argtypes = [ctypes.c_int]
    L.wkv_last_error_detail.restype = ctypes.c_char_p
    L.wkv_last_error_detail.argtypes = []
    L.wkv_launch_count.restype = ctypes.c_uint64
    L.wkv_launch_count.argtypes = []
    _lib = L
    return L


def _check(status: int, what: str) -> None:
    if status != 0:
        L = lib()
        raise WkvError(status, what, f"{L.wkv_status_string(status).decode()}: "
                                     f"{L.wkv_last_error_detail().decode()}")


def _ptr(t) -> Optional[int]:
    """Device (or host) address of a torch tensor / numpy array / int / None."""
    if t is None:
        return None
    if isinstance(t, int):
        return t
    if isinstance(t, np.ndarray):
        return t.ctypes.data
    return t.data_ptr()


def _stream(stream) -> Optional[int]:
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    return stream if isinstance(stream, int) else stream.cuda_stream


def _ptr_array(tensors: Optional[Sequence]) -> Optional[ctypes.Array]:
    if tensors is None:
        return None
    arr = (ctypes.c_void_p * len(tensors))()
    for i, t in enumerate(tensors):
        arr[i] = _ptr(t)
    return arr


class Problem:
    """A `wkv_shape` together with the host/device arrays it points to (kept alive here)."""

    def __init__(self, *, dtype: str, batch: int, n_q_heads: int, n_kv_heads: int, head_dim: int,
                 l_obs: int, window: int, task: int, top_p: int, max_seqlen: int,
                 budgets: Sequence[int], cu_seqlens: Optional[Sequence[int]] = None,
                 kv_layout: str = "bhnd", score_impl: int = WKV_SCORE_AUTO, device=None):
        import torch
        self.dtype = dtype
        self.elem_bytes = 4 if dtype == "f32" else 2
        self.torch_dtype = torch.float32 if dtype == "f32" else torch.bfloat16
        self.device = device if device is not None else torch.device("cuda", torch.cuda.current_device())
        s = WkvShape()
        s.struct_size = ctypes.sizeof(WkvShape)
        s.dtype = WKV_F32 if dtype == "f32" else WKV_BF16
        s.batch, s.n_q_heads, s.n_kv_heads, s.head_dim = batch, n_q_heads, n_kv_heads, head_dim
        s.l_obs, s.window, s.top_p, s.task = l_obs, window, top_p, task
        s.max_seqlen = max_seqlen
        s.score_impl = score_impl
        self.budgets_host = np.ascontiguousarray(budgets, dtype=np.int32)
        assert len(self.budgets_host) == batch
        self.budgets_dev = torch.from_numpy(self.budgets_host).to(self.device)
        s.budget = int(self.budgets_host[0])
        s.budgets_host = self.budgets_host.ctypes.data
        s.budgets_dev = self.budgets_dev.data_ptr()
        self.packed = cu_seqlens is not None
        if self.packed:
            self.cu_host = np.ascontiguousarray(cu_seqlens, dtype=np.int32)
            self.cu_dev = torch.from_numpy(self.cu_host).to(self.device)
            s.cu_seqlens_host = self.cu_host.ctypes.data
            s.cu_seqlens_dev = self.cu_dev.data_ptr()
            s.stride_b, s.stride_h, s.stride_t = 0, head_dim, n_kv_heads * head_dim
            self.seqlens = np.diff(self.cu_host)
        else:
            self.cu_host = self.cu_dev = None
            if kv_layout == "bhnd":
                s.stride_b, s.stride_h, s.stride_t = n_kv_heads * max_seqlen * head_dim, max_seqlen * head_dim, head_dim
            elif kv_layout == "bnhd":
                s.stride_b, s.stride_h, s.stride_t = max_seqlen * n_kv_heads * head_dim, head_dim, n_kv_heads * head_dim
            else:
                raise ValueError(kv_layout)
            self.seqlens = np.full(batch, max_seqlen, dtype=np.int32)
        s.q_stride_b, s.q_stride_h, s.q_stride_t = n_q_heads * l_obs * head_dim, l_obs * head_dim, head_dim
        self.shape = s
        L = lib()
        self.kw_max = L.wkv_kw_max(ctypes.byref(s))
        self.k_max = L.wkv_k_max(ctypes.byref(s))
        self.keep_max = L.wkv_keep_max(ctypes.byref(s))
        self.workspace_bytes = L.wkv_workspace_bytes(ctypes.byref(s))
        if self.kw_max == 0:
            raise WkvError(-1, "wkv_shape", L.wkv_last_error_detail().decode())
        self.units = batch * n_kv_heads
        self.nr_max = max(1, max_seqlen - l_obs)

    @classmethod
    def from_workload(cls, w, score_impl: int = WKV_SCORE_AUTO, device=None) -> "Problem":
        """Builds the shape of a `workloads.Workload`."""
        return cls(dtype=w.dtype, batch=w.batch, n_q_heads=w.n_q_heads, n_kv_heads=w.n_kv_heads,
                   head_dim=w.head_dim, l_obs=w.l_obs, window=w.window, task=w.task, top_p=w.top_p,
                   max_seqlen=w.max_seqlen, budgets=w.budgets(),
                   cu_seqlens=w.cu_seqlens() if w.ragged else None, score_impl=score_impl, device=device)

    # ---- caller-side allocations (torch is the allocator, nothing else) ----
    def alloc_workspace(self):
        """Zero-filled scratch; its first int32 is the device status word (see `device_status`)."""
        import torch
        return torch.zeros(max(self.workspace_bytes, 256), dtype=torch.uint8, device=self.device)

    def alloc_outputs(self, n_layers: int, fill_byte: Optional[int] = None, keep_capacity: Optional[int] = None):
        import torch
        cap = self.keep_max if keep_capacity is None else keep_capacity
        B, H, d = self.shape.batch, self.shape.n_kv_heads, self.shape.head_dim

        def mk():
            t = torch.empty((B, H, cap, d), dtype=self.torch_dtype, device=self.device)
            if fill_byte is not None:
                t.view(torch.uint8).fill_(fill_byte)
            return t
        return {
            "window_scores": torch.full((B, H, self.kw_max), float("nan"), dtype=torch.float32, device=self.device),
            "window_idx": torch.full((B, H, self.k_max), -7, dtype=torch.int32, device=self.device),
            "kept_len": torch.full((B, H), -7, dtype=torch.int32, device=self.device),
            "k_out": [mk() for _ in range(n_layers)],
            "v_out": [mk() for _ in range(n_layers)],
            "keep_capacity": cap,
        }


def wkv_score_windows(prob: Problem, q_obs, k_leader, window_scores, token_scores, workspace, stream=None) -> None:
    _check(lib().wkv_score_windows(ctypes.byref(prob.shape), _ptr(q_obs), _ptr(k_leader), _ptr(window_scores),
                                   _ptr(token_scores), _ptr(workspace), workspace.numel(), _stream(stream)),
           "wkv_score_windows")


WKV_STATIC_SCRATCH_BYTES = 4 << 20


def wkv_score_windows_static(prob: Problem, q_obs, k_leader, window_scores, token_scores=None,
                             device_status=None, stream=None) -> None:
    """Scoring without a caller workspace: for hosts that may not allocate device memory.  The
    scratch is a fixed area inside the library (at most WKV_STATIC_SCRATCH_BYTES; larger shapes
    raise), shared by all calls on the device, so overlapping calls must be serialised."""
    _check(lib().wkv_score_windows_static(ctypes.byref(prob.shape), _ptr(q_obs), _ptr(k_leader),
                                          _ptr(window_scores), _ptr(token_scores), _ptr(device_status),
                                          _stream(stream)), "wkv_score_windows_static")


def wkv_select_topk_windows(prob: Problem, window_scores, window_idx, kept_len, stream=None) -> None:
    _check(lib().wkv_select_topk_windows(ctypes.byref(prob.shape), _ptr(window_scores), _ptr(window_idx),
                                         _ptr(kept_len), _stream(stream)), "wkv_select_topk_windows")


def wkv_gather_kv(prob: Problem, k_layers, v_layers, window_idx, k_out_layers, v_out_layers,
                  cu_seqlens_out=None, keep_capacity: int = 0, stream=None) -> None:
    _check(lib().wkv_gather_kv(ctypes.byref(prob.shape), len(k_layers), _ptr_array(k_layers),
                               _ptr_array(v_layers), _ptr(window_idx), _ptr_array(k_out_layers),
                               _ptr_array(v_out_layers), _ptr(cu_seqlens_out), keep_capacity, _stream(stream)),
           "wkv_gather_kv")


def wkv_gather_kv_paged(prob: Problem, k_layers, v_layers, window_idx, k_pools, v_pools, block_table, page_size: int,
                        num_pages: int, page_stride: int, head_stride: int, row_stride: int, stream=None) -> None:
    """Gather into paged pools: row r of unit (b, h) -> page block_table[b, r // page_size], slot r % page_size."""
    _check(lib().wkv_gather_kv_paged(ctypes.byref(prob.shape), len(k_layers), _ptr_array(k_layers), _ptr_array(v_layers),
                                     _ptr(window_idx), _ptr_array(k_pools), _ptr_array(v_pools), _ptr(block_table),
                                     block_table.shape[-1], page_size, num_pages, page_stride, head_stride, row_stride,
                                     _stream(stream)), "wkv_gather_kv_paged")


def wkv_compact_kv_inplace(prob: Problem, k_layers, v_layers, window_idx, stream=None) -> None:
    """Moves every unit's retained rows to the front of its own rows, inside the given tensors."""
    _check(lib().wkv_compact_kv_inplace(ctypes.byref(prob.shape), len(k_layers), _ptr_array(k_layers),
                                        _ptr_array(v_layers), _ptr(window_idx), _stream(stream)),
           "wkv_compact_kv_inplace")


def wkv_compress_group(prob: Problem, q_obs_leader, k_layers, v_layers, k_out_layers, v_out_layers,
                       window_scores, window_idx, kept_len, workspace, cu_seqlens_out=None,
                       keep_capacity: int = 0, stream=None) -> None:
    _check(lib().wkv_compress_group(ctypes.byref(prob.shape), len(k_layers), _ptr(q_obs_leader),
                                    _ptr_array(k_layers), _ptr_array(v_layers), _ptr_array(k_out_layers),
                                    _ptr_array(v_out_layers), _ptr(window_scores), _ptr(window_idx),
                                    _ptr(kept_len), _ptr(cu_seqlens_out), keep_capacity, _ptr(workspace),
                                    workspace.numel(), _stream(stream)), "wkv_compress_group")


def wkv_score_windows_lse(prob: Problem, q_obs, k_leader, lse_obs, window_scores, token_scores, workspace,
                          stream=None) -> None:
    """Scoring with the observation rows' softmax normalisers (natural-log LSE, float [B, H_q, alpha])
    supplied by the caller, e.g. from the leader layer's prefill attention."""
    _check(lib().wkv_score_windows_lse(ctypes.byref(prob.shape), _ptr(q_obs), _ptr(k_leader), _ptr(lse_obs),
                                       _ptr(window_scores), _ptr(token_scores), _ptr(workspace), workspace.numel(),
                                       _stream(stream)), "wkv_score_windows_lse")


def wkv_select_leader_windows(prob: Problem, q_obs_leader, k_leader, window_scores, window_idx, kept_len, workspace,
                              lse_obs=None, stream=None) -> None:
    """Layer-by-layer use: score + pool + select on the leader layer only; the layers of the group are
    then gathered one by one with wkv_gather_kv as their K/V appear."""
    _check(lib().wkv_select_leader_windows(ctypes.byref(prob.shape), _ptr(q_obs_leader), _ptr(k_leader),
                                           _ptr(lse_obs), _ptr(window_scores), _ptr(window_idx), _ptr(kept_len),
                                           _ptr(workspace), workspace.numel(), _stream(stream)),
           "wkv_select_leader_windows")


def _group_lse_args(prob, q_obs_leader, lse_obs, k_layers, v_layers, k_out_layers, v_out_layers, window_scores,
                    window_idx, kept_len, workspace, cu_seqlens_out, keep_capacity, stream):
    arrs = (_ptr_array(k_layers), _ptr_array(v_layers), _ptr_array(k_out_layers), _ptr_array(v_out_layers))
    args = (ctypes.byref(prob.shape), len(k_layers), _ptr(q_obs_leader), _ptr(lse_obs), arrs[0], arrs[1], arrs[2],
            arrs[3], _ptr(window_scores), _ptr(window_idx), _ptr(kept_len), _ptr(cu_seqlens_out), keep_capacity,
            _ptr(workspace), workspace.numel(), _stream(stream))
    return args, arrs


def wkv_compress_group_lse(prob: Problem, q_obs_leader, lse_obs, k_layers, v_layers, k_out_layers, v_out_layers,
                           window_scores, window_idx, kept_len, workspace, cu_seqlens_out=None,
                           keep_capacity: int = 0, stream=None) -> None:
    args, _keep = _group_lse_args(prob, q_obs_leader, lse_obs, k_layers, v_layers, k_out_layers, v_out_layers,
                                  window_scores, window_idx, kept_len, workspace, cu_seqlens_out, keep_capacity,
                                  stream)
    _check(lib().wkv_compress_group_lse(*args), "wkv_compress_group_lse")


class GroupPlan:
    """wkv_group_plan: the group call recorded once, replayed by `launch(stream)`.  Keeps the tensors
    it was created with alive."""

    def __init__(self, prob: Problem, q_obs_leader, k_layers, v_layers, k_out_layers, v_out_layers, window_scores,
                 window_idx, kept_len, workspace, lse_obs=None, cu_seqlens_out=None, keep_capacity: int = 0):
        args, arrs = _group_lse_args(prob, q_obs_leader, lse_obs, k_layers, v_layers, k_out_layers, v_out_layers,
                                     window_scores, window_idx, kept_len, workspace, cu_seqlens_out, keep_capacity,
                                     None)
        self._keep = (prob, arrs, q_obs_leader, lse_obs, k_layers, v_layers, k_out_layers, v_out_layers,
                      window_scores, window_idx, kept_len, workspace, cu_seqlens_out)
        handle = ctypes.c_void_p()
        _check(lib().wkv_group_plan_create(*args[:-1], ctypes.byref(handle)), "wkv_group_plan_create")
        self._handle = handle
        self._launch = lib().wkv_group_plan_launch

    def launch(self, stream=None) -> None:
        st = self._launch(self._handle, _stream(stream))
        if st != 0:
            _check(st, "wkv_group_plan_launch")

    def close(self) -> None:
        if self._handle:
            lib().wkv_group_plan_destroy(self._handle)
            self._handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


class PreparedCall:
    """A C-ABI call with its arguments marshalled once (pointer tables, shape, stream): `run()` is a
    single foreign call, so that a loop over many groups is not bound by Python."""

    def __init__(self, fn, what: str, args: tuple, keep: tuple):
        self._fn, self._what, self._args, self._keep = fn, what, args, keep

    def run(self) -> None:
        st = self._fn(*self._args)
        if st != 0:
            _check(st, self._what)


def prepare_compress_group(prob: Problem, q_obs_leader, k_layers, v_layers, k_out_layers, v_out_layers,
                           window_scores, window_idx, kept_len, workspace, cu_seqlens_out=None,
                           keep_capacity: int = 0, stream=None) -> PreparedCall:
    arrs = (_ptr_array(k_layers), _ptr_array(v_layers), _ptr_array(k_out_layers), _ptr_array(v_out_layers))
    args = (ctypes.byref(prob.shape), len(k_layers), _ptr(q_obs_leader), arrs[0], arrs[1], arrs[2], arrs[3],
            _ptr(window_scores), _ptr(window_idx), _ptr(kept_len), _ptr(cu_seqlens_out), keep_capacity,
            _ptr(workspace), workspace.numel(), _stream(stream))
    return PreparedCall(lib().wkv_compress_group, "wkv_compress_group", args,
                        (prob, q_obs_leader, k_layers, v_layers, k_out_layers, v_out_layers, window_scores,
                         window_idx, kept_len, workspace, cu_seqlens_out, arrs))


def prepare_compress_group_lse(prob: Problem, q_obs_leader, lse_obs, k_layers, v_layers, k_out_layers,
                               v_out_layers, window_scores, window_idx, kept_len, workspace, cu_seqlens_out=None,
                               keep_capacity: int = 0, stream=None) -> PreparedCall:
    args, arrs = _group_lse_args(prob, q_obs_leader, lse_obs, k_layers, v_layers, k_out_layers, v_out_layers,
                                 window_scores, window_idx, kept_len, workspace, cu_seqlens_out, keep_capacity,
                                 stream)
    return PreparedCall(lib().wkv_compress_group_lse, "wkv_compress_group_lse", args,
                        (prob, arrs, q_obs_leader, lse_obs, k_layers, v_layers, k_out_layers, v_out_layers,
                         window_scores, window_idx, kept_len, workspace, cu_seqlens_out))


def prepare_score_windows(prob: Problem, q_obs, k_leader, window_scores, token_scores, workspace,
                          stream=None) -> PreparedCall:
    args = (ctypes.byref(prob.shape), _ptr(q_obs), _ptr(k_leader), _ptr(window_scores), _ptr(token_scores),
            _ptr(workspace), workspace.numel(), _stream(stream))
    return PreparedCall(lib().wkv_score_windows, "wkv_score_windows", args,
                        (prob, q_obs, k_leader, window_scores, token_scores, workspace))


def prepare_select_leader_windows(prob: Problem, q_obs_leader, k_leader, window_scores, window_idx, kept_len,
                                  workspace, lse_obs=None, stream=None) -> PreparedCall:
    args = (ctypes.byref(prob.shape), _ptr(q_obs_leader), _ptr(k_leader), _ptr(lse_obs), _ptr(window_scores),
            _ptr(window_idx), _ptr(kept_len), _ptr(workspace), workspace.numel(), _stream(stream))
    return PreparedCall(lib().wkv_select_leader_windows, "wkv_select_leader_windows", args,
                        (prob, q_obs_leader, k_leader, lse_obs, window_scores, window_idx, kept_len, workspace))


def prepare_select_topk_windows(prob: Problem, window_scores, window_idx, kept_len, stream=None) -> PreparedCall:
    args = (ctypes.byref(prob.shape), _ptr(window_scores), _ptr(window_idx), _ptr(kept_len), _stream(stream))
    return PreparedCall(lib().wkv_select_topk_windows, "wkv_select_topk_windows", args,
                        (prob, window_scores, window_idx, kept_len))


def prepare_gather_kv(prob: Problem, k_layers, v_layers, window_idx, k_out_layers, v_out_layers,
                      cu_seqlens_out=None, keep_capacity: int = 0, stream=None) -> PreparedCall:
    arrs = (_ptr_array(k_layers), _ptr_array(v_layers), _ptr_array(k_out_layers), _ptr_array(v_out_layers))
    args = (ctypes.byref(prob.shape), len(k_layers), arrs[0], arrs[1], _ptr(window_idx), arrs[2], arrs[3],
            _ptr(cu_seqlens_out), keep_capacity, _stream(stream))
    return PreparedCall(lib().wkv_gather_kv, "wkv_gather_kv", args,
                        (prob, k_layers, v_layers, window_idx, k_out_layers, v_out_layers, cu_seqlens_out, arrs))


def wkv_compress_group_host(prob: Problem, q_obs_host, k_layers_host, v_layers_host, k_out_host, v_out_host,
                            window_idx_host, kept_len_host, q_obs_dev, k_layers_dev, v_layers_dev,
                            k_out_dev, v_out_dev, window_idx_dev, kept_len_dev, keep_capacity, workspace,
                            stream=None) -> None:
    """Host-buffer entry: copies in, compresses, copies out, synchronises (host tensors: torch CPU, pinned)."""
    nbytes = lambda t: t.numel() * t.element_size()
    _check(lib().wkv_compress_group_host(
        ctypes.byref(prob.shape), len(k_layers_host), _ptr(q_obs_host), nbytes(q_obs_host),
        _ptr_array(k_layers_host), _ptr_array(v_layers_host), nbytes(k_layers_host[0]),
        _ptr_array(k_out_host), _ptr_array(v_out_host), nbytes(k_out_host[0]),
        _ptr(window_idx_host), _ptr(kept_len_host), _ptr(q_obs_dev), _ptr_array(k_layers_dev),
        _ptr_array(v_layers_dev), _ptr_array(k_out_dev), _ptr_array(v_out_dev), _ptr(window_idx_dev),
        _ptr(kept_len_dev), keep_capacity, _ptr(workspace), workspace.numel(), _stream(stream)),
        "wkv_compress_group_host")


def wkv_keep_len(n: int, alpha: int, omega: int, budget: int):
    """(row capacity of one unit's compact cache, k) for a sequence of n tokens."""
    k = ctypes.c_int32(0)
    rows = lib().wkv_keep_len(n, alpha, omega, budget, ctypes.byref(k))
    return int(rows), int(k.value)


def workspace_sync_words(prob: "Problem", unit: int):
    """Byte offsets (ticket word, arrival word) of a unit's synchronisation words in the workspace."""
    t, a = ctypes.c_size_t(0), ctypes.c_size_t(0)
    _check(lib().wkv_workspace_sync_words(ctypes.byref(prob.shape), unit, ctypes.byref(t), ctypes.byref(a)),
           "wkv_workspace_sync_words")
    return int(t.value), int(a.value)


def wkv_probe_ex2_rate(scratch, blocks: int, threads: int, iters: int, stream=None) -> int:
    """Launches the ex2 rate probe; returns the number of exponentials the launch evaluates."""
    n = ctypes.c_int64(0)
    _check(lib().wkv_probe_ex2_rate(_ptr(scratch), blocks, threads, iters, ctypes.byref(n), _stream(stream)),
           "wkv_probe_ex2_rate")
    return int(n.value)


def wkv_probe_colsum_rate(scratch, blocks: int, threads: int, iters: int, stream=None) -> int:
    """Launches the cross-lane column-sum probe; returns the number of block elements it reduces."""
    n = ctypes.c_int64(0)
    _check(lib().wkv_probe_colsum_rate(_ptr(scratch), blocks, threads, iters, ctypes.byref(n), _stream(stream)),
           "wkv_probe_colsum_rate")
    return int(n.value)


def device_status(workspace) -> int:
    """The workspace's status word (synchronises): 0, or the OR of the error bits a kernel has set."""
    return int(workspace[:4].view(__import__("torch").int32).item())


def wkv_group_budgets(n_layers: int, gamma: int, b_total: int, lambda_num: int = 14, lambda_den: int = 1) -> np.ndarray:
    """Eq. 5-7: per-layer budget of each of the n_layers / gamma groups (host arithmetic, exact)."""
    out = np.zeros(max(n_layers // max(gamma, 1), 1), dtype=np.int32)
    _check(lib().wkv_group_budgets(n_layers, gamma, b_total, lambda_num, lambda_den, out.ctypes.data),
           "wkv_group_budgets")
    return out


def wkv_jaccard_windows(idx_a: np.ndarray, idx_b: np.ndarray):
    """Section 3.2's similarity of two selections: (per-unit Jaccard [units], mean).  Host arrays
    [..., k_max] of ascending window indices padded with negative entries."""
    a = np.ascontiguousarray(idx_a, dtype=np.int32)
    b = np.ascontiguousarray(idx_b, dtype=np.int32)
    assert a.shape == b.shape
    k_max = a.shape[-1]
    units = a.size // k_max
    per_unit = np.zeros(units, dtype=np.float64)
    mean = ctypes.c_double(0.0)
    _check(lib().wkv_jaccard_windows(a.ctypes.data, b.ctypes.data, units, k_max, per_unit.ctypes.data,
                                     ctypes.byref(mean)), "wkv_jaccard_windows")
    return per_unit.reshape(a.shape[:-1]), float(mean.value)


def wkv_launch_count() -> int:
    return int(lib().wkv_launch_count())


def to_device(x: np.ndarray, device=None):
    """numpy workload tensor (float32, or bf16 bits as uint16) -> torch CUDA tensor of that dtype."""
    import torch
    if x.dtype == np.uint16:
        t = torch.from_numpy(x.view(np.int16)).view(torch.bfloat16)
    else:
        t = torch.from_numpy(x)
    return t.to(device if device is not None else "cuda")


def to_host_bits(t) -> np.ndarray:
    """torch tensor -> numpy array in the workload convention (bf16 as uint16 bits)."""
    import torch
    t = t.detach().cpu().contiguous()
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view(np.uint16)
    return t.numpy()
