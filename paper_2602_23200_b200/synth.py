"""Seeded synthetic inputs for the InnerQ decode path.

This module only draws numbers.  It holds none of the method's arithmetic (no
quantisation, no normalisation, no attention), so both the CPU oracle's tests and
the CUDA path's tests/bench may import it without sharing method code.

Every tensor is generated on the host, per (batch, KV head) unit, from a Philox
stream keyed by (base seed, workload id, tensor id, unit, step), so any subset of a
workload can be produced independently and reproducibly.  Values are drawn in
float32, shaped by the workload's recipe, and rounded once to fp16 (clamped to the
finite fp16 range).

The recipes stand in for the KV cache of one decoder layer of 7B/8B-class models at
the paper's sequence lengths (Section "Latency"): Gaussian bulk, a few large-magnitude
key channels per head (the channel outliers that motivate the per-channel key
normalisation, Section "Per-channel Normalization of K"), heavy-tailed values.
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import Optional, Tuple

import numpy as np

BASE_SEED = 26022320
FP16_MAX = 65504.0

# tensor ids for the Philox key
_T_K, _T_V, _T_Q, _T_KNEW, _T_VNEW, _T_AUX = 1, 2, 3, 4, 5, 6

SYM, ASYM, HYBRID = 0, 1, 2
INNER, OUTER, FP16 = 0, 1, 2


@dataclass(frozen=True)
class Workload:
    """Shape, quantisation setting and data recipe of one synthetic workload."""
    name: str
    wid: int                 # workload id (part of the random key)
    batch: int
    n_q_heads: int
    n_kv_heads: int
    n_tokens: int
    head_dim: int = 128
    group: int = 32
    k_bits: int = 2
    v_bits: int = 2
    k_mode: int = HYBRID
    v_mode: int = HYBRID
    w_sink: int = 4
    w_recent: int = 128
    sym_variant: int = 0
    grouping: int = INNER
    k_normalize: int = 1
    # data recipe
    k_dist: str = "normal"       # "normal" | "lognormal_channels"
    v_dist: str = "normal"       # "normal" | "student_t4"
    outlier_channels: Tuple[int, ...] = ()   # fixed outlier key channels (all heads)
    n_hashed_outliers: int = 0   # outlier key channels drawn per KV head
    outlier_lo: float = 20.0     # multiplier range for outlier channels
    outlier_hi: float = 20.0
    append_scale: float = 1.0    # multiplier on appended k/v tokens

    @property
    def n_units(self) -> int:
        return self.batch * self.n_kv_heads

    @property
    def q_per_kv(self) -> int:
        return self.n_q_heads // self.n_kv_heads

    def with_(self, **kw) -> "Workload":
        return replace(self, **kw)


def _rng(w: Workload, tensor: int, unit: int, step: int = 0) -> np.random.Generator:
    ss = np.random.SeedSequence([BASE_SEED, w.wid, tensor, unit, step])
    return np.random.Generator(np.random.Philox(ss))


def _to_fp16(x: np.ndarray) -> np.ndarray:
    return np.clip(x, -FP16_MAX, FP16_MAX).astype(np.float16)


def key_channel_scale(w: Workload, unit: int) -> np.ndarray:
    """Per-channel multiplier applied to the keys of one (batch, KV head) unit.

    The multiplier depends on the KV head only (not on the batch index), like a
    property of the model's key projection would."""
    D = w.head_dim
    head = unit % w.n_kv_heads
    g = np.random.Generator(np.random.Philox(np.random.SeedSequence([BASE_SEED, w.wid, _T_AUX, head])))
    scale = np.ones(D, dtype=np.float32)
    if w.k_dist == "lognormal_channels":
        scale = np.clip(np.exp(g.standard_normal(D, dtype=np.float32)), 0.05, 50.0).astype(np.float32)
    for c in w.outlier_channels:
        scale[c % D] *= np.float32(w.outlier_lo)
    if w.n_hashed_outliers:
        chans = g.permutation(D)[: w.n_hashed_outliers]
        mult = g.uniform(w.outlier_lo, w.outlier_hi, size=w.n_hashed_outliers).astype(np.float32)
        scale[chans] *= mult
    return scale


def _draw(g: np.random.Generator, dist: str, shape) -> np.ndarray:
    if dist in ("normal", "lognormal_channels"):
        return g.standard_normal(shape, dtype=np.float32)
    if dist == "student_t4":
        z = g.standard_normal(shape, dtype=np.float32)
        chi = np.zeros(shape, dtype=np.float32)
        for _ in range(4):
            n = g.standard_normal(shape, dtype=np.float32)
            chi += n * n
        return z / np.sqrt(chi / np.float32(4.0))
    raise ValueError(dist)


def kv_unit(w: Workload, unit: int, n_tokens: Optional[int] = None) -> Tuple[np.ndarray, np.ndarray]:
    """fp16 K[N, D] and V[N, D] of one (batch, KV head) unit."""
    N = w.n_tokens if n_tokens is None else n_tokens
    D = w.head_dim
    k = _draw(_rng(w, _T_K, unit), w.k_dist, (N, D)) * key_channel_scale(w, unit)[None, :]
    v = _draw(_rng(w, _T_V, unit), w.v_dist, (N, D))
    return _to_fp16(k), _to_fp16(v)


def kv_all(w: Workload, n_tokens: Optional[int] = None) -> Tuple[np.ndarray, np.ndarray]:
    """fp16 K, V of shape [batch, n_kv_heads, N, D] (all units)."""
    N = w.n_tokens if n_tokens is None else n_tokens
    K = np.empty((w.n_units, N, w.head_dim), dtype=np.float16)
    V = np.empty_like(K)
    for u in range(w.n_units):
        K[u], V[u] = kv_unit(w, u, N)
    shape = (w.batch, w.n_kv_heads, N, w.head_dim)
    return K.reshape(shape), V.reshape(shape)


def query(w: Workload, step: int = 0) -> np.ndarray:
    """fp16 q[batch, n_q_heads, D] for decode step `step`."""
    g = _rng(w, _T_Q, 0, step)
    return _to_fp16(g.standard_normal((w.batch, w.n_q_heads, w.head_dim), dtype=np.float32))


def new_token(w: Workload, step: int) -> Tuple[np.ndarray, np.ndarray]:
    """fp16 k_new, v_new of shape [batch, n_kv_heads, D] appended at decode step `step`."""
    D = w.head_dim
    k = np.empty((w.n_units, D), dtype=np.float32)
    v = np.empty((w.n_units, D), dtype=np.float32)
    for u in range(w.n_units):
        k[u] = _draw(_rng(w, _T_KNEW, u, step), w.k_dist, (D,)) * key_channel_scale(w, u)
        v[u] = _draw(_rng(w, _T_VNEW, u, step), w.v_dist, (D,))
    k *= np.float32(w.append_scale)
    v *= np.float32(w.append_scale)
    shape = (w.batch, w.n_kv_heads, D)
    return _to_fp16(k).reshape(shape), _to_fp16(v).reshape(shape)


# --- the named workloads (shapes and settings of the benchmark configurations) ----------------

def config1() -> Workload:
    """Single head, 4096 tokens, 2-bit, G=32, four fixed outlier key channels x20."""
    return Workload("c1_single_head_4k", 1, batch=1, n_q_heads=1, n_kv_heads=1, n_tokens=4096,
                    group=32, k_bits=2, v_bits=2, w_sink=4, w_recent=128,
                    outlier_channels=(7, 42, 77, 112), outlier_lo=20.0, outlier_hi=20.0)


def config2() -> Workload:
    """7B-class MHA decode: 32 heads, 32768 tokens, 2-bit, G=32; 2% outlier key channels x10-30."""
    return Workload("c2_mha32_32k", 2, batch=1, n_q_heads=32, n_kv_heads=32, n_tokens=32768,
                    group=32, k_bits=2, v_bits=2, w_sink=4, w_recent=128,
                    n_hashed_outliers=3, outlier_lo=10.0, outlier_hi=30.0)


def config3(bits: int = 4) -> Workload:
    """8B-class GQA decode: 32/8 heads, batch 16, 8192 tokens, G=64; t(4) values, heavy-tailed key channel scales."""
    return Workload(f"c3_gqa_b16_8k_{bits}bit", 3, batch=16, n_q_heads=32, n_kv_heads=8, n_tokens=8192,
                    group=64, k_bits=bits, v_bits=bits, w_sink=4, w_recent=128,
                    k_dist="lognormal_channels", v_dist="student_t4")


def config4() -> Workload:
    """Long-context GQA decode: 32/8 heads, batch 4, 131072 tokens, 2-bit, G=128; 2% outlier key channels x20."""
    return Workload("c4_gqa_b4_128k", 4, batch=4, n_q_heads=32, n_kv_heads=8, n_tokens=131072,
                    group=128, k_bits=2, v_bits=2, w_sink=4, w_recent=256,
                    n_hashed_outliers=3, outlier_lo=20.0, outlier_hi=20.0)


def config5(bits: int, group: int, mode: int = HYBRID, grouping: int = INNER, sym_variant: int = 0) -> Workload:
    """Sweep point on the config-3 shape and data."""
    w = config3(bits)
    if grouping == OUTER:
        mode = ASYM
    return w.with_(name=f"c5_b{bits}_g{group}_m{mode}_grp{grouping}", group=group, k_bits=bits, v_bits=bits,
                   k_mode=mode, v_mode=mode, grouping=grouping, sym_variant=sym_variant,
                   k_normalize=1 if grouping == INNER else 0)


def tiny(**kw) -> Workload:
    """Small multi-tile workload with a ragged tail, for fast parity tests."""
    base = Workload("tiny", 9, batch=2, n_q_heads=4, n_kv_heads=2, n_tokens=333,
                    group=32, k_bits=2, v_bits=2, w_sink=4, w_recent=16,
                    n_hashed_outliers=3, outlier_lo=10.0, outlier_hi=30.0)
    return base.with_(**kw)
