"""Seeded synthetic KV-cache inputs shaped like LLaMA-2 / Mistral decode workloads.

Holds no arithmetic of the compression method: only random draws.  Both the
CPU oracle's tests and the CUDA path's tests / benchmark take their inputs
from here, so that the two sides see identical arrays.

Recipe (stand-in for real model KV caches, which need weights and datasets):
  K[b,h,i,j] = fp16( N(0,1) * c[h,j] * o ),  c[h,j] ~ lognormal(0,1) fixed per
               (head, channel) and shared over batch and tokens -- a few key
               channels carry much larger magnitudes than the rest;
  V[b,h,i,j] = fp16( N(0,1) * o );
  o = 20 with probability 0.01, independently per entry, else 1;
  q ~ fp16 N(0,1);   B0 (power-iteration start) ~ fp32 N(0,1).
Generators: numpy PCG64 seeded with SeedSequence([0x6EA2, config_id, stream]).
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np

STREAM_K, STREAM_V, STREAM_MASK_K, STREAM_Q, STREAM_B0, STREAM_APPEND, STREAM_CHAN, STREAM_MASK_V = range(8)


@dataclass(frozen=True)
class Workload:
    """One of the benchmark configurations (sizes only)."""
    config_id: int
    name: str
    batch: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    n: int               # prefill / context tokens
    bits: int
    group: int
    s_pct: float
    rank: int
    buffer_cap: int
    power_iters: int = 3


WORKLOADS = {
    1: Workload(1, "C1 single head n=256 4-bit g64 s2 r4 nb16", 1, 1, 1, 128, 256, 4, 64, 2.0, 4, 16),
    2: Workload(2, "C2 LLaMA-2-7B layer B8 H32 n4096 2-bit g64 s2 r4 nb64", 8, 32, 32, 128, 4096, 2, 64, 2.0, 4, 64),
    3: Workload(3, "C3 LLaMA-2-13B layer B16 H40 n8192 4-bit g64 s1 r8 nb64", 16, 40, 40, 128, 8192, 4, 64, 1.0, 8, 64),
    32: Workload(32, "C3 LLaMA-2-13B layer B16 H40 n8192 2-bit g64 s1 r8 nb64", 16, 40, 40, 128, 8192, 2, 64, 1.0, 8, 64),
    4: Workload(4, "C4 Mistral-7B GQA layer B4 Hq32 Hkv8 n32768 2-bit g128 s2 r4 nb64", 4, 32, 8, 128, 32768, 2, 128, 2.0, 4, 64),
    # per-vector grouping (group 0): the KCVT backbone with the paper's 4-bit setting (Section 4, "Implementation
    # details": s = 2 %, r = 4, n_b = 20)
    6: Workload(6, "C6 LLaMA-2-7B layer B8 H32 n4096 4-bit per-vector (KCVT) s2 r4 nb20", 8, 32, 32, 128, 4096, 4, 0, 2.0, 4, 20),
    # parity-only shapes that land in other branches of the decode kernel's work split (many warps per unit)
    21: Workload(21, "T1 B2 H32 n4096 2-bit g64 s2 r4 nb64", 2, 32, 32, 128, 4096, 2, 64, 2.0, 4, 64),
    22: Workload(22, "T2 B4 H32 n4096 4-bit g64 s2 r4 nb64", 4, 32, 32, 128, 4096, 4, 64, 2.0, 4, 64),
}


def rng(config_id: int, stream: int, extra: int = 0) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64(np.random.SeedSequence([0x6EA2, config_id, stream, extra])))


def channel_scale(config_id: int, n_kv_heads: int, head_dim: int) -> np.ndarray:
    """c[h, j] ~ lognormal(0, 1), float64 [H_kv, d_H]."""
    return rng(config_id, STREAM_CHAN).lognormal(0.0, 1.0, size=(n_kv_heads, head_dim))


def _spikes(gen, shape):
    return np.where(gen.random(shape) < 0.01, 20.0, 1.0)


def make_kv(config_id: int, batch: int, n_kv_heads: int, n: int, head_dim: int, extra: int = 0):
    """K, V fp16 [B, H_kv, n, d_H]."""
    shape = (batch, n_kv_heads, n, head_dim)
    c = channel_scale(config_id, n_kv_heads, head_dim)[None, :, None, :]
    k = rng(config_id, STREAM_K, extra).standard_normal(shape) * c * _spikes(rng(config_id, STREAM_MASK_K, extra), shape)
    v = rng(config_id, STREAM_V, extra).standard_normal(shape) * _spikes(rng(config_id, STREAM_MASK_V, extra), shape)
    return k.astype(np.float16), v.astype(np.float16)


def make_query(config_id: int, batch: int, n_q_heads: int, head_dim: int, extra: int = 0) -> np.ndarray:
    """q fp16 [B, H_q, d_H]."""
    return rng(config_id, STREAM_Q, extra).standard_normal((batch, n_q_heads, head_dim)).astype(np.float16)


def make_b0(config_id: int, batch: int, n_kv_heads: int, head_dim: int, rank: int, extra: int = 0) -> np.ndarray:
    """Power-iteration start, fp32 [B, H_kv, 2 (K, V), d_H, rank]."""
    return rng(config_id, STREAM_B0, extra).standard_normal((batch, n_kv_heads, 2, head_dim, max(rank, 1))).astype(np.float32)[..., :rank]


def make_appended(config_id: int, batch: int, n_kv_heads: int, head_dim: int, steps: int):
    """Tokens pushed during decoding: k, v fp16 [steps, B, H_kv, d_H], same distribution."""
    k, v = make_kv(config_id, batch, n_kv_heads, steps, head_dim, extra=STREAM_APPEND + 1000)
    return np.ascontiguousarray(k.transpose(2, 0, 1, 3)), np.ascontiguousarray(v.transpose(2, 0, 1, 3))
