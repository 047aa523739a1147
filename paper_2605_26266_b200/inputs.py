"""Seeded synthetic inputs for the five workloads.

This module only draws random numbers and rounds them once to BF16; it holds
none of the method's arithmetic (no rotation, no quantization, no attention).
Both the CUDA path and the CPU checker consume the BF16 bit patterns it
returns, so the two always see identical inputs.

The workloads are synthetic stand-ins for the activations of chunk-wise
autoregressive video-diffusion transformers (several thousand tokens per chunk,
head dim 128, group size 32/64/128, a handful to dozens of cached chunks); the
models and prompt suites used in the paper's experiments are not reproduced.

Every tensor is drawn from numpy.random.default_rng(SeedSequence([seed, cfg_id,
tensor_id, chunk_index])) as float32 and rounded to BF16 with
round-to-nearest-even.  Tensors are laid out [batch, heads, tokens, head_dim].
"""
from __future__ import annotations

from dataclasses import dataclass, replace

import numpy as np

T_Q, T_K, T_V, T_AUX = 0, 1, 2, 3


@dataclass(frozen=True)
class Workload:
    name: str
    cfg_id: int
    batch: int
    heads: int
    head_dim: int
    chunk: int            # tokens per chunk (= queries M = current keys N_R)
    cached_chunks: int    # number of earlier chunks in the cache when attention runs
    bits: int
    group: int
    seed: int
    k_dist: str = "normal"        # "normal" | "student_t3"
    k_outliers: int = 0           # outlier channels per head (fixed over tokens)
    k_outlier_scale: float = 1.0
    head_scale: bool = False      # q, k scaled per head by U[0.5, 2]

    @property
    def n_cached(self) -> int:
        return self.chunk * self.cached_chunks

    @property
    def groups(self) -> int:
        return self.head_dim // self.group

    @property
    def capacity(self) -> int:
        """Cache capacity in tokens: room for cached_chunks + 1 chunks, rounded up to 128."""
        n = self.chunk * (self.cached_chunks + 1)
        return (n + 127) // 128 * 128

    def flops(self, n_cached=None) -> float:
        """Tensor FLOPs of one attention call: QK^T and PV only."""
        ns = self.n_cached if n_cached is None else n_cached
        return 4.0 * self.batch * self.heads * self.chunk * (ns + self.chunk) * self.head_dim

    def attn_bytes(self, n_cached=None) -> float:
        """Algorithmic HBM bytes of one attention call: packed codes + scales + zeros of the
        attended window (K and V), Q, K_R, V_R read and O written."""
        ns = self.n_cached if n_cached is None else n_cached
        per_tok = 2 * (self.head_dim * self.bits // 8 + 3 * self.groups)
        cur = 4 * self.chunk * self.head_dim * 2
        return float(self.batch * self.heads * (ns * per_tok + cur))

    def append_bytes(self) -> float:
        """Algorithmic HBM bytes of one quantize-append call: BF16 K, V read; packed codes,
        scales and zeros written."""
        per_tok = 2 * (self.head_dim * 2) + 2 * (self.head_dim * self.bits // 8 + 3 * self.groups)
        return float(self.batch * self.heads * self.chunk * per_tok)


WORKLOADS = {
    "tiny": Workload("tiny", 1, 1, 2, 64, 256, 4, 2, 64, 0),
    "sweep_int4": Workload("sweep_int4", 2, 1, 16, 128, 1560, 4, 4, 128, 0,
                           k_outliers=4, k_outlier_scale=8.0),
    "sweep_int2": Workload("sweep_int2", 2, 1, 16, 128, 1560, 4, 2, 128, 0,
                           k_outliers=4, k_outlier_scale=8.0),
    "dit": Workload("dit", 3, 1, 24, 128, 4680, 8, 2, 64, 0, head_scale=True),
    "long": Workload("long", 4, 1, 24, 128, 4680, 32, 2, 128, 0),
    "pipeline": Workload("pipeline", 5, 2, 32, 128, 2048, 15, 2, 32, 1,
                         k_dist="student_t3", k_outliers=8, k_outlier_scale=10.0),
    # short query chunk over a long prefix (the partial-prefill regime): 32 units of 514 key tiles, split over all SMs
    "prefix": Workload("prefix", 6, 1, 32, 128, 256, 256, 2, 128, 0, k_outliers=4, k_outlier_scale=8.0),
}


def with_seed(w: Workload, seed: int) -> Workload:
    return replace(w, seed=seed)


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to BF16 (nearest, ties to even); returns the uint16 bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = (u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)
    return r.astype(np.uint16)


def _rng(w: Workload, tensor_id: int, chunk_index: int):
    return np.random.default_rng(np.random.SeedSequence([w.seed, w.cfg_id, tensor_id, chunk_index]))


def _head_aux(w: Workload):
    """Per-head constants fixed over tokens and chunks: outlier channel indices and
    per-head scales of q and k."""
    r = np.random.default_rng(np.random.SeedSequence([w.seed, w.cfg_id, T_AUX]))
    idx = np.stack([r.choice(w.head_dim, size=max(w.k_outliers, 1), replace=False)
                    for _ in range(w.heads)])
    uq = r.uniform(0.5, 2.0, size=w.heads).astype(np.float32)
    uk = r.uniform(0.5, 2.0, size=w.heads).astype(np.float32)
    return idx, uq, uk


def make_chunk(w: Workload, chunk_index: int, tokens: int | None = None, need_q: bool = True):
    """Q, K, V of chunk `chunk_index` as BF16 bit patterns, each [batch, heads, tokens, head_dim].
    need_q=False skips the query draw (Q comes back as None): every tensor has its own generator, so K and V
    are the same bits either way.  Cached chunks only ever contribute K and V."""
    n = w.chunk if tokens is None else tokens
    shape = (w.batch, w.heads, n, w.head_dim)
    idx, uq, uk = _head_aux(w)
    q = _rng(w, T_Q, chunk_index).standard_normal(shape, dtype=np.float32) if need_q else None
    if w.k_dist == "student_t3":
        k = _rng(w, T_K, chunk_index).standard_t(3.0, size=shape).astype(np.float32)
    else:
        k = _rng(w, T_K, chunk_index).standard_normal(shape, dtype=np.float32)
    v = _rng(w, T_V, chunk_index).standard_normal(shape, dtype=np.float32)
    if w.k_outliers:
        for h in range(w.heads):
            k[:, h, :, idx[h, :w.k_outliers]] *= np.float32(w.k_outlier_scale)
    if w.head_scale:
        if need_q:
            q *= uq[None, :, None, None]
        k *= uk[None, :, None, None]
    return (f32_to_bf16_bits(q) if need_q else None), f32_to_bf16_bits(k), f32_to_bf16_bits(v)


def sample_rows(m: int, tile: int = 128, n_random: int = 64, seed: int = 0) -> np.ndarray:
    """Query rows that touch every row tile: first, middle and last row of each tile of
    `tile` rows (the ragged tail tile included) plus `n_random` random rows."""
    rows = set()
    for t0 in range(0, m, tile):
        t1 = min(t0 + tile, m) - 1
        rows.update((t0, (t0 + t1) // 2, t1))
    r = np.random.default_rng(np.random.SeedSequence([seed, m, tile]))
    rows.update(int(x) for x in r.integers(0, m, size=n_random))
    return np.array(sorted(rows), dtype=np.int64)
