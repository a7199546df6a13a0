"""Python face of the CPU oracle (TEST INFRASTRUCTURE ONLY).

Only tests, the smoke check and the benchmark's cpu-baseline leg may import
this package.  It compiles `wkv_oracle.c` with gcc on first use and exposes the
paper's steps on numpy arrays:

  token_scores_unit   Eq. 1-2 for one (sequence, KV head)
  window_scores       Eq. 3-4
  select_topk         budgeted selection, ties to the lower index
  num_windows / num_selected   integer formulas (Eq. 3, budget sentence)
  select_leader       Eq. 1-4 + selection for every unit of a batch
  gather_layer        compacted cache of one layer from shared indices
  compress_group      the whole group (leader selection + gamma gathers)
  jaccard_windows     similarity of two index selections (section 3.2)

bf16 tensors are passed as uint16 bit patterns, fp32 as float32.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Dict, List, Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "wkv_oracle.c")
_LIB = os.path.join(_HERE, "libwkv_oracle.so")

F32, BF16 = 0, 1


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (plain -O2, OpenMP over independent units)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["gcc", "-O2", "-std=c99", "-fopenmp", "-fPIC", "-shared",
                               "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        i64, vp = ctypes.c_int64, ctypes.c_void_p
        _lib.wkvo_num_threads.restype = ctypes.c_int
        _lib.wkvo_num_windows.restype = i64
        _lib.wkvo_num_windows.argtypes = [i64, i64, i64]
        _lib.wkvo_num_selected.restype = i64
        _lib.wkvo_num_selected.argtypes = [i64, i64, i64, i64]
        _lib.wkvo_token_scores_unit.restype = None
        _lib.wkvo_token_scores_unit.argtypes = [ctypes.c_int, vp, i64, i64, vp, i64, i64, i64, i64, i64,
                                                vp, vp, vp]
        _lib.wkvo_window_scores.restype = None
        _lib.wkvo_window_scores.argtypes = [vp, i64, i64, i64, vp]
        _lib.wkvo_select_topk.restype = None
        _lib.wkvo_select_topk.argtypes = [vp, i64, i64, vp]
        _lib.wkvo_gather_unit.restype = i64
        _lib.wkvo_gather_unit.argtypes = [ctypes.c_int, vp, i64, vp, i64, i64, i64, i64, i64, vp, i64]
        _lib.wkvo_select_leader.restype = None
        _lib.wkvo_select_leader.argtypes = [ctypes.c_int, vp, vp] + [i64] * 8 + [vp, vp] + [i64] * 9 + [vp] * 6
        _lib.wkvo_gather_layer.restype = None
        _lib.wkvo_gather_layer.argtypes = [ctypes.c_int, vp, vp] + [i64] * 6 + [vp] + [i64] * 3 + \
                                          [vp, i64, vp, i64, vp]
    return _lib


def num_threads() -> int:
    return int(lib().wkvo_num_threads())


def _dtype_code(a: np.ndarray) -> int:
    if a.dtype == np.float32:
        return F32
    if a.dtype == np.uint16:
        return BF16
    raise TypeError(f"oracle takes float32 or bf16 bits (uint16), got {a.dtype}")


def _ptr(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def num_windows(n: int, alpha: int, omega: int) -> int:
    return int(lib().wkvo_num_windows(n, alpha, omega))


def num_selected(n: int, alpha: int, omega: int, budget: int) -> int:
    return int(lib().wkvo_num_selected(n, alpha, omega, budget))


def effective_p(task: int, omega: int, top_p: int) -> int:
    """p of Eq. 4: omega for localization (task 0); for aggregation the caller's
    value, or ceil(omega/2) when it passes 0."""
    if task == 0:
        return omega
    return top_p if top_p > 0 else (omega + 1) // 2


def token_scores_unit(q: np.ndarray, k: np.ndarray, want_lse: bool = False):
    """Eq. 1-2.  q [G, alpha, d], k [n, d] (same dtype).  Returns (t [n-alpha] float64,
    observation mass, lse [G*alpha] or None)."""
    q = np.ascontiguousarray(q)
    k = np.ascontiguousarray(k)
    G, alpha, d = q.shape
    n = k.shape[0]
    assert k.shape[1] == d and _dtype_code(q) == _dtype_code(k)
    t = np.zeros(max(n - alpha, 0), dtype=np.float64)
    mass = ctypes.c_double(0.0)
    lse = np.zeros(G * alpha, dtype=np.float64) if want_lse else None
    lib().wkvo_token_scores_unit(_dtype_code(q), _ptr(q), alpha * d, d, _ptr(k), d, n, alpha, G, d,
                                 _ptr(t), ctypes.cast(ctypes.byref(mass), ctypes.c_void_p), _ptr(lse))
    return t, mass.value, lse


def window_scores(t: np.ndarray, omega: int, p: int) -> np.ndarray:
    """Eq. 3-4 on a vector of token scores; returns float64 [ceil(len/omega)]."""
    t = np.ascontiguousarray(t, dtype=np.float64)
    kw = -(-len(t) // omega)
    s = np.zeros(kw, dtype=np.float64)
    if kw:
        lib().wkvo_window_scores(_ptr(t), len(t), omega, p, _ptr(s))
    return s


def select_topk(scores: np.ndarray, k: int) -> np.ndarray:
    """Indices (ascending) of the k largest fp32 scores; ties to the lower index."""
    s = np.ascontiguousarray(scores, dtype=np.float32)
    k = min(int(k), len(s))
    idx = np.zeros(max(k, 0), dtype=np.int32)
    if k > 0:
        lib().wkvo_select_topk(_ptr(s), len(s), k, _ptr(idx))
    return idx


def _layout(w_batch: int, n_kv_heads: int, d: int, max_seqlen: int, packed: bool):
    """(stride_b, stride_h, stride_t) in elements for the two layouts."""
    if packed:
        return 0, d, n_kv_heads * d
    return n_kv_heads * max_seqlen * d, max_seqlen * d, d


def select_leader(q_obs: np.ndarray, k: np.ndarray, *, n_kv_heads: int, l_obs: int, window: int,
                  task: int, top_p: int, max_seqlen: int, budgets: np.ndarray,
                  cu_seqlens: Optional[np.ndarray] = None, want_tokens: bool = False,
                  unit_mask: Optional[np.ndarray] = None) -> Dict[str, np.ndarray]:
    """Eq. 1-4 and the budgeted selection for every (sequence, KV head)."""
    q_obs = np.ascontiguousarray(q_obs)
    k = np.ascontiguousarray(k)
    B, Hq, alpha, d = q_obs.shape
    assert alpha == l_obs
    packed = cu_seqlens is not None
    sb, sh, st = _layout(B, n_kv_heads, d, max_seqlen, packed)
    budgets = np.ascontiguousarray(budgets, dtype=np.int32)
    cu = None if cu_seqlens is None else np.ascontiguousarray(cu_seqlens, dtype=np.int32)
    seqlens = np.full(B, max_seqlen) if cu is None else np.diff(cu)
    kw_max = max(1, max(num_windows(int(n), alpha, window) for n in seqlens))
    nr_max = max(1, int(max(seqlens)) - alpha)
    k_max = max(1, max(num_selected(int(n), alpha, window, int(b)) for n, b in zip(seqlens, budgets)))
    units = B * n_kv_heads
    sd = np.full((B, n_kv_heads, kw_max), np.nan, dtype=np.float64)
    sf = np.full((B, n_kv_heads, kw_max), np.nan, dtype=np.float32)
    tok = np.full((B, n_kv_heads, nr_max), np.nan, dtype=np.float64) if want_tokens else None
    idx = np.full((B, n_kv_heads, k_max), -1, dtype=np.int32)
    kept = np.zeros((B, n_kv_heads), dtype=np.int32)
    mask = None if unit_mask is None else np.ascontiguousarray(unit_mask, dtype=np.uint8).reshape(units)
    p = effective_p(task, window, top_p)
    lib().wkvo_select_leader(_dtype_code(k), _ptr(q_obs), _ptr(k), B, Hq, n_kv_heads, d, alpha, window, p,
                             max_seqlen, _ptr(cu), _ptr(budgets), sb, sh, st,
                             Hq * alpha * d, alpha * d, d, kw_max, nr_max, k_max,
                             _ptr(sd), _ptr(sf), _ptr(tok), _ptr(idx), _ptr(kept), _ptr(mask))
    return {"window_scores_f64": sd, "window_scores": sf, "token_scores": tok,
            "window_idx": idx, "kept_len": kept, "k_max": k_max, "kw_max": kw_max}


def gather_layer(src: np.ndarray, window_idx: np.ndarray, *, n_kv_heads: int, l_obs: int, window: int,
                 max_seqlen: int, budgets: np.ndarray, keep_max: int,
                 cu_seqlens: Optional[np.ndarray] = None,
                 cu_seqlens_out: Optional[np.ndarray] = None, fill: int = 0) -> np.ndarray:
    """Compacted cache of one layer.  Dense output [B,H_kv,keep_max,d] or, with
    `cu_seqlens_out`, packed [T_out,H_kv,d].  Rows the method does not write keep `fill`
    (a byte pattern for the element's integer view)."""
    src = np.ascontiguousarray(src)
    d = src.shape[-1]
    packed = cu_seqlens is not None
    B = len(budgets)
    sb, sh, st = _layout(B, n_kv_heads, d, max_seqlen, packed)
    widx = np.ascontiguousarray(window_idx, dtype=np.int32)
    k_max = widx.shape[-1]
    budgets = np.ascontiguousarray(budgets, dtype=np.int32)
    cu = None if cu_seqlens is None else np.ascontiguousarray(cu_seqlens, dtype=np.int32)
    cuo = None if cu_seqlens_out is None else np.ascontiguousarray(cu_seqlens_out, dtype=np.int32)
    if cuo is None:
        dst = np.empty((B, n_kv_heads, keep_max, d), dtype=src.dtype)
    else:
        dst = np.empty((int(cuo[-1]), n_kv_heads, d), dtype=src.dtype)
    dst.view(np.uint32 if src.dtype == np.float32 else np.uint16)[...] = fill
    lib().wkvo_gather_layer(_dtype_code(src), _ptr(src), _ptr(dst), B, n_kv_heads, d, l_obs, window,
                            max_seqlen, _ptr(cu), sb, sh, st, _ptr(widx), k_max, _ptr(budgets),
                            keep_max, _ptr(cuo))
    return dst


def group_budgets(n_layers: int, gamma: int, b_total: int, lam) -> Dict[str, object]:
    """Eq. 5-7 in exact rational arithmetic.  Returns the real-valued group budgets b^h (Fractions),
    the real-valued per-layer budgets b^h / gamma, and the integer per-layer budgets: floor, with
    the tokens lost to the flooring given to group 0 in whole multiples of gamma."""
    from fractions import Fraction
    H = n_layers // gamma
    T, lam = Fraction(b_total), Fraction(lam)
    if H == 1:
        b = [T]
    else:
        b_top = T / (lam * H)                      # Eq. 6, top group
        b_bottom = 2 * T / H - b_top               # Eq. 6, bottom group
        b = [b_bottom - (b_bottom - b_top) / (H - 1) * h for h in range(H)]   # Eq. 7
    per_layer = [x / gamma for x in b]
    ints = [int(x // 1) for x in per_layer]
    ints[0] += (b_total - gamma * sum(ints)) // gamma
    return {"group": b, "per_layer": per_layer, "per_layer_int": ints}


def jaccard_windows(idx_a: np.ndarray, idx_b: np.ndarray) -> np.ndarray:
    """Section 3.2: Jaccard similarity |A n B| / |A u B| of two retained-window sets per unit, written
    out with Python sets.  idx_* are [..., k_max] index lists padded with negative entries; two empty
    sets count as identical."""
    a = np.asarray(idx_a)
    b = np.asarray(idx_b)
    out = np.zeros(a.shape[:-1], dtype=np.float64)
    for pos in np.ndindex(*a.shape[:-1]):
        A = {int(x) for x in a[pos] if x >= 0}
        B = {int(x) for x in b[pos] if x >= 0}
        out[pos] = 1.0 if not (A | B) else len(A & B) / len(A | B)
    return out


def keep_max(seqlens: Sequence[int], budgets: Sequence[int], l_obs: int, window: int) -> int:
    """Row capacity of the dense compact cache: max over sequences of k*omega + min(alpha, n)."""
    return max(num_selected(int(n), l_obs, window, int(b)) * window + min(l_obs, int(n))
               for n, b in zip(seqlens, budgets))


def compress_group(q_obs: np.ndarray, k_layers: List[np.ndarray], v_layers: List[np.ndarray], *,
                   n_kv_heads: int, l_obs: int, window: int, task: int, top_p: int, max_seqlen: int,
                   budgets: np.ndarray, cu_seqlens: Optional[np.ndarray] = None,
                   cu_seqlens_out: Optional[np.ndarray] = None, fill: int = 0,
                   want_tokens: bool = False) -> Dict[str, object]:
    """Leader selection on k_layers[0], then the shared-index gather of every layer."""
    sel = select_leader(q_obs, k_layers[0], n_kv_heads=n_kv_heads, l_obs=l_obs, window=window, task=task,
                        top_p=top_p, max_seqlen=max_seqlen, budgets=budgets, cu_seqlens=cu_seqlens,
                        want_tokens=want_tokens)
    seqlens = np.full(len(budgets), max_seqlen) if cu_seqlens is None else np.diff(cu_seqlens)
    km = keep_max(seqlens, budgets, l_obs, window)
    kw = dict(n_kv_heads=n_kv_heads, l_obs=l_obs, window=window, max_seqlen=max_seqlen, budgets=budgets,
              keep_max=km, cu_seqlens=cu_seqlens, cu_seqlens_out=cu_seqlens_out, fill=fill)
    sel["k_out"] = [gather_layer(x, sel["window_idx"], **kw) for x in k_layers]
    sel["v_out"] = [gather_layer(x, sel["window_idx"], **kw) for x in v_layers]
    sel["keep_max"] = km
    return sel
