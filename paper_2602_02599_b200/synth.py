"""Seeded synthetic inputs for the RAP decode path (shapes of the paper's 3B-14B workloads).

This module only draws random numbers and names workload shapes.  It holds none of the
method's arithmetic (no top-k, no RoPE, no rounding, no attention) so that the CUDA
path and the CPU oracle can both be fed from it without sharing any computation.
It imports NumPy only.

Streams: np.random.default_rng([seed, tag, layer(, extra)]) so every layer can be
regenerated on its own.  Tags: 1 pair scores, 2 V-channel scores, 3 weights,
4 hidden states, 5 cache fill, 6 low-rank comparator factors, 7 bias, 8 output projection.
"""
from __future__ import annotations

from dataclasses import dataclass, replace

import numpy as np

TAG_KSCORE, TAG_VSCORE, TAG_W, TAG_X, TAG_CACHE, TAG_LOWRANK, TAG_BIAS, TAG_WO = 1, 2, 3, 4, 5, 6, 7, 8


@dataclass(frozen=True)
class Workload:
    """Shape of one attention stack and its decode batch."""
    name: str
    n_layers: int
    hidden: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    rope_theta: float
    rho: float
    n_pairs: int        # P, retained RoPE pairs per KV head
    n_vch: int          # d_v', retained V channels per KV head
    batch: int
    seq: int            # cached tokens before the timed step
    dtype: str          # 'f32' or 'bf16'
    seed: int
    pairing: int = 0    # 0 = (i, i + D/2), 1 = (2i, 2i + 1)

    @property
    def group(self):
        return self.n_q_heads // self.n_kv_heads

    @property
    def n_out(self):
        return (self.n_q_heads + self.n_kv_heads) * 2 * self.n_pairs + self.n_kv_heads * self.n_vch

    @property
    def elem_bytes(self):
        return 4 if self.dtype == "f32" else 2


# Retained counts at head_dim 128 for the swept retain ratios.
SWEEP_COUNTS = {1.0: (64, 128), 0.9: (58, 115), 0.8: (51, 102), 0.7: (45, 90), 0.5: (32, 64)}

TINY = Workload("tiny-fp32", 1, 256, 4, 2, 64, 10000.0, 0.75, 24, 48, 1, 128, "f32", 0)
LLAMA_3B = Workload("llama3.2-3b-shape", 28, 3072, 24, 8, 128, 500000.0, 0.9, 58, 115, 16, 8192, "bf16", 2000)
LLAMA_8B = Workload("llama3.1-8b-shape", 32, 4096, 32, 8, 128, 500000.0, 0.7, 45, 90, 32, 32768, "bf16", 3000)
QWEN_14B = Workload("qwen2.5-14b-shape", 48, 5120, 40, 8, 128, 1000000.0, 0.7, 45, 90, 4, 100000, "bf16", 4000)


def sweep_workload(rho):
    """One point of the retain-ratio sweep on the 8B shape (batch 16, 16384-token cache)."""
    P, dv = SWEEP_COUNTS[rho]
    return replace(LLAMA_8B, name=f"sweep-8b-rho{rho}", rho=rho, n_pairs=P, n_vch=dv,
                   batch=16, seq=16384, seed=5000)


CONFIGS = {
    "tiny": TINY,
    "3b": LLAMA_3B,
    "8b": LLAMA_8B,
    "14b": QWEN_14B,
    **{f"sweep{rho}": sweep_workload(rho) for rho in SWEEP_COUNTS},
}


def scaled_down(w, n_layers=2, batch=2, seq=512, hidden=None):
    """Same heads / dims / retain ratio as w on a stack the oracle finishes in seconds."""
    return replace(w, name=w.name + "-small", n_layers=n_layers, batch=batch, seq=seq,
                   hidden=w.hidden if hidden is None else hidden)


def draw_scores(w):
    """Lognormal(0, 1) stand-ins for the root-Fisher scores: pairs [L][H_kv][D/2], V [L][H_kv][D]."""
    ks = np.empty((w.n_layers, w.n_kv_heads, w.head_dim // 2))
    vs = np.empty((w.n_layers, w.n_kv_heads, w.head_dim))
    for l in range(w.n_layers):
        ks[l] = np.random.default_rng([w.seed, TAG_KSCORE, l]).lognormal(0.0, 1.0, ks[l].shape)
        vs[l] = np.random.default_rng([w.seed, TAG_VSCORE, l]).lognormal(0.0, 1.0, vs[l].shape)
    return ks, vs


def draw_full_weights(w, layer):
    """Dense W_q [H_q*D][hidden], W_k, W_v [H_kv*D][hidden], N(0, 0.02^2), fp32."""
    rng = np.random.default_rng([w.seed, TAG_W, layer])
    D = w.head_dim
    Wq = rng.normal(0.0, 0.02, (w.n_q_heads * D, w.hidden)).astype(np.float32)
    Wk = rng.normal(0.0, 0.02, (w.n_kv_heads * D, w.hidden)).astype(np.float32)
    Wv = rng.normal(0.0, 0.02, (w.n_kv_heads * D, w.hidden)).astype(np.float32)
    return Wq, Wk, Wv


def draw_packed_weights(w, layer):
    """Shrunken W~_qkv [N_out][hidden] drawn directly (a row selection of iid rows is iid)."""
    rng = np.random.default_rng([w.seed, TAG_W, layer, 1])
    return rng.standard_normal((w.n_out, w.hidden), dtype=np.float32) * np.float32(0.02)


def draw_wo(w, layer):
    """Dense output projection W_o [hidden][H_q*D], N(0, 0.02^2), fp32 (weights stored [out][in])."""
    rng = np.random.default_rng([w.seed, TAG_WO, layer])
    return rng.standard_normal((w.hidden, w.n_q_heads * w.head_dim), dtype=np.float32) * np.float32(0.02)


def draw_bias(w, layer, n):
    return np.random.default_rng([w.seed, TAG_BIAS, layer]).normal(0.0, 0.1, n).astype(np.float32)


def draw_hidden(w, layer, step, rows):
    """Hidden states N(0, 1), [rows][hidden], fp32; one independent draw per (layer, step)."""
    rng = np.random.default_rng([w.seed, TAG_X, layer, step])
    return rng.standard_normal((rows, w.hidden), dtype=np.float32)


def draw_cache_rows(w, layer, b, h, rows, width, which):
    """iid N(0, hidden * 0.02^2) rows -- the law of projected hidden states -- for cache fills."""
    rng = np.random.default_rng([w.seed, TAG_CACHE, layer, b, h, which])
    sigma = np.float32(np.sqrt(w.hidden) * 0.02)
    return rng.standard_normal((rows, width), dtype=np.float32) * sigma


def draw_lowrank_factor(w, layer, rank):
    """B_k [H_kv][rank][D] ~ N(0, 1/rank) for the low-rank comparator."""
    rng = np.random.default_rng([w.seed, TAG_LOWRANK, layer])
    return (rng.standard_normal((w.n_kv_heads, rank, w.head_dim)) / np.sqrt(rank)).astype(np.float32)


def ragged_lengths(w, seq=None):
    """Per-sequence cached lengths for the ragged parity variant: S - 37 b (at least 1)."""
    s = w.seq if seq is None else seq
    return np.maximum(1, s - 37 * np.arange(w.batch)).astype(np.int32)
