"""Seeded synthetic workloads for the WindowKV prefill-compression path.

This module only *generates inputs*: shapes, value distributions and planted
structure of the five benchmark configurations.  It contains none of the
method's arithmetic (no softmax, pooling, selection or gather) and imports
neither the CUDA binding nor the CPU oracle, so both sides can be fed the very
same bits.

All randomness comes from numpy's counter-based Philox generator, keyed by
(seed, config id, layer, tensor id); the float32 draws are rounded to bf16 with
round-to-nearest-even in integer arithmetic, so the bits do not depend on the
machine.

Layouts produced (d contiguous everywhere):
  * Q_obs  : [B, H_q, alpha, d]      observation-window queries of the leader
  * K, V   : dense  [B, H_kv, N, d]   (configs 1-4)
             packed [T, H_kv, d] + cu_seqlens [B+1]   (config 5, ragged)
Element type: np.float32, or np.uint16 holding bf16 bit patterns.
"""
from __future__ import annotations

import dataclasses
from concurrent.futures import ThreadPoolExecutor
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np

TASK_LOCALIZATION = 0
TASK_AGGREGATION = 1

BASE_SEED = 0x5EED0000


# --------------------------------------------------------------------------
# bf16 helpers (pure bit manipulation)
# --------------------------------------------------------------------------
def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 -> bf16 (round-to-nearest-even), returned as uint16 bits."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    r = u + np.uint32(0x7FFF) + lsb
    return (r >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns to float32."""
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def to_f32(x: np.ndarray) -> np.ndarray:
    """Exact float32 view of a workload tensor (float32 or bf16 bits)."""
    return bf16_bits_to_f32(x) if x.dtype == np.uint16 else np.asarray(x, dtype=np.float32)


# --------------------------------------------------------------------------
# configuration
# --------------------------------------------------------------------------
@dataclasses.dataclass(frozen=True)
class Workload:
    """One benchmark configuration (shapes follow the paper's notation:
    alpha = observation window, omega = review window, gamma = layers/group)."""

    name: str
    config_id: int
    dtype: str                 # "f32" | "bf16"
    batch: int
    n_layers: int
    gamma: int                 # layers per group
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    max_seqlen: int            # N
    l_obs: int                 # alpha
    window: int                # omega
    task: int
    top_p: int                 # p for the aggregation task (ignored for localization)
    budget_frac: Optional[float] = None   # per-layer budget as a fraction of n_b ...
    budget_tokens: Optional[int] = None   # ... or as a token count
    ragged: bool = False       # packed layout, n_b ~ U[N/2, N]
    n_planted: int = 0         # planted windows per (sequence, KV head); <0 => fraction in percent
    needle: Optional[Tuple[int, float]] = None   # (needle length in tokens, depth in [0,1])
    key_norm_sigma: float = 0.0                  # lognormal sigma of per-token key scale
    plant_rise: float = 5.0    # target mean logit rise of planted keys

    @property
    def n_groups(self) -> int:
        return self.n_layers // self.gamma

    @property
    def group_size(self) -> int:
        return self.n_q_heads // self.n_kv_heads

    @property
    def rows(self) -> int:
        return self.group_size * self.l_obs

    def seqlens(self) -> np.ndarray:
        """Per-sequence context lengths n_b (deterministic)."""
        if not self.ragged:
            return np.full(self.batch, self.max_seqlen, dtype=np.int32)
        g = np.random.Generator(np.random.Philox(key=BASE_SEED + self.config_id * 256 + 255))
        lo = self.max_seqlen // 2
        return g.integers(lo, self.max_seqlen + 1, size=self.batch).astype(np.int32)

    def cu_seqlens(self) -> np.ndarray:
        cu = np.zeros(self.batch + 1, dtype=np.int32)
        cu[1:] = np.cumsum(self.seqlens())
        return cu

    def budgets(self) -> np.ndarray:
        """Per-sequence, per-layer KV budget in tokens (includes the observation window)."""
        n = self.seqlens().astype(np.int64)
        if self.budget_tokens is not None:
            return np.full(self.batch, self.budget_tokens, dtype=np.int32)
        # integer arithmetic: floor(frac * n) with frac given in 1/10000
        num = int(round(self.budget_frac * 10000))
        return ((n * num) // 10000).astype(np.int32)


def tiny() -> Workload:
    return Workload("C1-tiny", 1, "f32", 1, 2, 2, 4, 2, 64, 1024, 8, 8, TASK_LOCALIZATION, 0,
                    budget_tokens=128, n_planted=4)


def llama8b_single_group(task: int = TASK_LOCALIZATION) -> Workload:
    return Workload("C2-8B-single-group", 2, "bf16", 1, 4, 4, 32, 8, 128, 8192, 32, 8, task, 4,
                    budget_frac=0.12, n_planted=32)


def llama8b_full() -> Workload:
    return Workload("C3-8B-32K", 3, "bf16", 1, 32, 4, 32, 8, 128, 32768, 32, 16, TASK_AGGREGATION, 8,
                    budget_frac=0.12, key_norm_sigma=0.5)


def mistral_needle(n: int = 4096, depth: float = 0.5) -> Workload:
    budget = {4096: 128, 16384: 512, 32768: 2048}[n]
    return Workload(f"C4-needle-{n}-{int(depth * 100)}", 4, "bf16", 1, 32, 4, 32, 8, 128, n, 16, 8,
                    TASK_LOCALIZATION, 0, budget_tokens=budget, needle=(64, depth))


def batched_ragged() -> Workload:
    return Workload("C5-batched-ragged", 5, "bf16", 8, 32, 8, 32, 8, 128, 65536, 64, 32,
                    TASK_AGGREGATION, 16, budget_frac=0.12, ragged=True, n_planted=-1)


def batched_ragged_small() -> Workload:
    """Config 5's shape (256 observation rows per unit, packed ragged batch, 8 layers per group) cut down
    to 4 sequences of 8-16 K tokens and one group: a case small enough for counter captures."""
    return scaled(batched_ragged(), name="C5-small", batch=4, max_seqlen=16384, n_layers=8, config_id=13)


def qwen_small(l_obs: int = 16, n: int = 8192) -> Workload:
    """The paper's second model family (section 4.1: 7 layers per group, review window 32,
    observation window 4 or 16), with the shape of a 1.5 B model of that family: 28 layers,
    12 query heads over 2 KV heads (G = 6, so R = 24 or 96 observation rows), head dimension 128.
    Not one of the five benchmark configurations: a parity case for G != 4 and gamma = 7."""
    return Workload(f"qwen-small-a{l_obs}", 6, "bf16", 1, 28, 7, 12, 2, 128, n, l_obs, 32, TASK_AGGREGATION, 16,
                    budget_frac=0.12, n_planted=16)


def scaled(w: Workload, **kw) -> Workload:
    """A copy of a workload with some fields replaced (smaller parity cases)."""
    return dataclasses.replace(w, **kw)


ALL_CONFIGS = {
    "C1": tiny,
    "C2": llama8b_single_group,
    "C3": llama8b_full,
    "C4": mistral_needle,
    "C5": batched_ragged,
}


# --------------------------------------------------------------------------
# generation
# --------------------------------------------------------------------------
def _rng(w: Workload, layer: int, tensor: int, seq: int = 0) -> np.random.Generator:
    key = (BASE_SEED + w.config_id * 256 + layer) & 0xFFFFFFFFFFFFFFFF
    return np.random.Generator(np.random.Philox(key=[key, (tensor << 32) | seq]))


def _round(w: Workload, x: np.ndarray) -> np.ndarray:
    return x if w.dtype == "f32" else f32_to_bf16_bits(x)


def planted_windows(w: Workload, b: int, h: int, n_b: int) -> np.ndarray:
    """Window indices (ascending) that the recipe boosts for unit (b, h)."""
    n_r = n_b - w.l_obs
    if n_r <= 0:
        return np.zeros(0, dtype=np.int64)
    k_w = -(-n_r // w.window)
    if w.needle is not None:
        length, depth = w.needle
        per = length // w.window
        first = int(depth * (k_w - per))
        first = max(0, min(first, k_w - per))
        return np.arange(first, first + per, dtype=np.int64)
    if w.n_planted == 0:
        return np.zeros(0, dtype=np.int64)
    count = w.n_planted if w.n_planted > 0 else max(1, (k_w * (-w.n_planted)) // 100)
    full = n_r // w.window          # only full windows are planted
    count = min(count, full)
    g = np.random.Generator(np.random.Philox(key=[BASE_SEED + w.config_id * 256 + 254, (b << 16) | h]))
    return np.sort(g.choice(full, size=count, replace=False)).astype(np.int64)


def make_q_obs(w: Workload, group: int) -> np.ndarray:
    """Observation-window queries of the group's leader layer, [B, H_q, alpha, d]."""
    layer = group * w.gamma
    x = _rng(w, layer, 0).standard_normal((w.batch, w.n_q_heads, w.l_obs, w.head_dim), dtype=np.float32)
    return _round(w, x)


def _plant_direction(w: Workload, q_obs: np.ndarray, b: int, h: int) -> np.ndarray:
    g = w.group_size
    q = to_f32(q_obs[b, h * g:(h + 1) * g]).astype(np.float64)     # [G, alpha, d]
    s = q.sum(axis=(0, 1))
    nrm = np.linalg.norm(s)
    return (s / nrm if nrm > 0 else s).astype(np.float32)


def make_layer_kv(w: Workload, layer: int, q_obs: Optional[np.ndarray] = None,
                  want_v: bool = True) -> Tuple[np.ndarray, Optional[np.ndarray]]:
    """K and V of one layer.  Planted structure is added to K only, and only when
    `q_obs` (the leader's observation queries) is given."""
    d, hk = w.head_dim, w.n_kv_heads
    seqlens = w.seqlens()
    cu = w.cu_seqlens()
    total = int(cu[-1])

    def fill(tensor: int) -> np.ndarray:
        if w.ragged:
            out = np.empty((total, hk, d), dtype=np.float32)
            for b in range(w.batch):
                _rng(w, layer, tensor, b).standard_normal(dtype=np.float32, out=out[cu[b]:cu[b + 1]].reshape(-1))
            return out
        out = np.empty((w.batch, hk, w.max_seqlen, d), dtype=np.float32)
        for b in range(w.batch):
            _rng(w, layer, tensor, b).standard_normal(dtype=np.float32, out=out[b].reshape(-1))
        return out

    k = fill(1)
    if w.key_norm_sigma > 0:
        sg = w.key_norm_sigma
        for b in range(w.batch):
            n_b = int(seqlens[b])
            z = _rng(w, layer, 3, b).standard_normal((hk, n_b), dtype=np.float32)
            scale = np.exp(sg * z - 0.5 * sg * sg).astype(np.float32)
            if w.ragged:
                k[cu[b]:cu[b + 1]] *= scale.T[:, :, None]
            else:
                k[b] *= scale[:, :, None]
    if q_obs is not None and (w.n_planted != 0 or w.needle is not None):
        beta = w.plant_rise * np.sqrt(w.rows / d)          # mean rise = beta * sqrt(d / R)
        for b in range(w.batch):
            n_b = int(seqlens[b])
            for h in range(hk):
                u = _plant_direction(w, q_obs, b, h) * np.float32(beta * np.sqrt(d))
                for win in planted_windows(w, b, h, n_b):
                    lo = int(win) * w.window
                    hi = min(lo + w.window, n_b - w.l_obs)
                    if w.ragged:
                        k[cu[b] + lo:cu[b] + hi, h] += u
                    else:
                        k[b, h, lo:hi] += u
    k = _round(w, k)
    v = _round(w, fill(2)) if want_v else None
    return k, v


def make_group(w: Workload, group: int, n_threads: int = 8) -> Dict[str, object]:
    """All inputs of one layer group: leader queries, gamma layers of K and V,
    sequence lengths and budgets."""
    q_obs = make_q_obs(w, group)
    layers = [group * w.gamma + i for i in range(w.gamma)]

    def one(layer: int):
        return make_layer_kv(w, layer, q_obs if layer == layers[0] else None)

    if n_threads > 1 and len(layers) > 1:
        with ThreadPoolExecutor(max_workers=min(n_threads, len(layers))) as ex:
            kv = list(ex.map(one, layers))
    else:
        kv = [one(l) for l in layers]
    return {
        "workload": w,
        "group": group,
        "q_obs": q_obs,
        "k_layers": [x[0] for x in kv],
        "v_layers": [x[1] for x in kv],
        "seqlens": w.seqlens(),
        "cu_seqlens": w.cu_seqlens() if w.ragged else None,
        "budgets": w.budgets(),
    }
