"""Seeded synthetic inputs for the LoCoCo chunk step.

This module only draws random tensors and rounds them to the storage type.
It contains none of the method's arithmetic and imports neither the CUDA
binding nor the CPU oracle, so both sides can be fed from it.

The paper's workloads (Llama-2-7B key/value states, block size 512, memory
size 128..512, kernel width 21, contexts up to 32K; Section 4.1 and
Section 4.3) supply only shapes; the tensors here are seeded stand-ins.

Draw order per sequence (fixed): Q, K, V.  Conv weights G and the loss
projections P_O, P_K, P_V come from separate, named streams so that adding a
sequence never changes the weights.
"""
from __future__ import annotations

from dataclasses import dataclass, replace

import numpy as np


@dataclass(frozen=True)
class Workload:
    """One chunk-loop problem in the paper's notation (Algorithm 2)."""

    name: str
    index: int            # 1-based position in the list of configurations
    batch: int
    heads: int
    d: int                # head dimension
    M: int                # cache slots
    B: int                # chunk (segment) size
    k: int                # conv kernel width, odd
    L: int                # tokens per sequence
    dtype: str            # "f32" or "bf16" storage
    weights_per_head: bool
    qkv_scale: float      # multiplies the N(0,1) draws of Q, K, V
    g_std: float = 0.02
    heavy_tail_p: float = 0.0    # Bernoulli rate of key rows scaled by heavy_tail_x
    heavy_tail_x: float = 1.0
    c_in_mult: int = 1           # conv input channels = c_in_mult * d (1: keys, 2: keys||values)
    seed0: int | None = None     # overrides 1000*index

    @property
    def c_in(self) -> int:
        return self.c_in_mult * self.d

    @property
    def n_chunks(self) -> int:
        return -(-self.L // self.B)

    def seed(self, sequence: int) -> int:
        base = self.seed0 if self.seed0 is not None else 1000 * self.index
        return base + sequence

    def slice(self, **kw) -> "Workload":
        """A smaller problem with the same value recipe (fewer heads, shorter L ...)."""
        return replace(self, **kw)


CONFIGS = {
    # Tiny fp32 reference case.
    "cfg1": Workload("cfg1", 1, batch=1, heads=1, d=64, M=16, B=16, k=5, L=256, dtype="f32",
                     weights_per_head=False, qkv_scale=1.0, seed0=0),
    # Llama-2-7B-shaped inference layer.
    "cfg2": Workload("cfg2", 2, batch=1, heads=32, d=128, M=128, B=512, k=21, L=4096, dtype="bf16",
                     weights_per_head=True, qkv_scale=128.0 ** -0.5),
    # Streaming batch.
    "cfg3": Workload("cfg3", 3, batch=16, heads=32, d=128, M=128, B=64, k=21, L=8192, dtype="bf16",
                     weights_per_head=False, qkv_scale=1.0),
    # Fine-tuning-shaped forward, heavy-tailed keys.
    "cfg4": Workload("cfg4", 4, batch=1, heads=32, d=128, M=512, B=4096, k=21, L=32768, dtype="bf16",
                     weights_per_head=False, qkv_scale=1.0, heavy_tail_p=0.05, heavy_tail_x=4.0),
    # Same shapes, used with the backward pass.
    "cfg5": Workload("cfg5", 5, batch=1, heads=32, d=128, M=512, B=4096, k=21, L=32768, dtype="bf16",
                     weights_per_head=False, qkv_scale=1.0, heavy_tail_p=0.05, heavy_tail_x=4.0),
}


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """Round float32 to the nearest bfloat16 (ties to even); result is float32 holding the
    rounded value (low 16 bits zero)."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32)
    bias = np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))
    r = (u + bias) & np.uint32(0xFFFF0000)
    nan = np.isnan(x)
    if nan.any():
        r = np.where(nan, u | np.uint32(0x00400000), r)
    return r.view(np.float32)


def bf16_bits(x_rounded: np.ndarray) -> np.ndarray:
    """The 16-bit patterns of values already rounded by round_to_bf16."""
    return (np.ascontiguousarray(x_rounded, dtype=np.float32).view(np.uint32) >> np.uint32(16)).astype(np.uint16)


def bits_to_f32(bits: np.ndarray) -> np.ndarray:
    return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32)


def _store(x: np.ndarray, dtype: str) -> np.ndarray:
    if dtype == "bf16":
        return round_to_bf16(x)
    if dtype == "f32":
        return np.ascontiguousarray(x, dtype=np.float32)
    raise ValueError(dtype)


def make_sequence(w: Workload, sequence: int):
    """Q, K, V of one sequence: float32 arrays [heads, L, d] whose values are exactly
    representable in the storage dtype."""
    rng = np.random.Generator(np.random.PCG64(w.seed(sequence)))
    shape = (w.heads, w.L, w.d)
    q = rng.standard_normal(shape, dtype=np.float32) * np.float32(w.qkv_scale)
    k = rng.standard_normal(shape, dtype=np.float32) * np.float32(w.qkv_scale)
    v = rng.standard_normal(shape, dtype=np.float32) * np.float32(w.qkv_scale)
    if w.heavy_tail_p > 0.0:
        mask = rng.random((w.heads, w.L, 1)) < w.heavy_tail_p
        k = np.where(mask, k * np.float32(w.heavy_tail_x), k)
    return _store(q, w.dtype), _store(k, w.dtype), _store(v, w.dtype)


def make_qkv(w: Workload):
    """Q, K, V for the whole batch: float32 [batch, heads, L, d]."""
    qs, ks, vs = zip(*(make_sequence(w, s) for s in range(w.batch)))
    return np.stack(qs), np.stack(ks), np.stack(vs)


def make_weights(w: Workload, with_bias: bool = False):
    """Conv weights G [heads|1, M, c_in, k] (and optionally a bias [heads|1, M])."""
    rng = np.random.Generator(np.random.PCG64([w.seed(0), 0x6C6F636F]))
    hg = w.heads if w.weights_per_head else 1
    g = rng.standard_normal((hg, w.M, w.c_in, w.k), dtype=np.float32) * np.float32(w.g_std)
    bias = None
    if with_bias:
        bias = rng.standard_normal((hg, w.M), dtype=np.float32) * np.float32(w.g_std)
        bias = _store(bias, w.dtype)
    return _store(g, w.dtype), bias


def make_loss_projections(w: Workload):
    """P_O [batch, heads, L, d], P_K and P_V [batch, heads, M, d] of the scalar loss
    <P_O, O> + <P_K, K_cache_final> + <P_V, V_cache_final>."""
    rng = np.random.Generator(np.random.PCG64([w.seed(0), 0x6C6F7373]))
    p_o = rng.standard_normal((w.batch, w.heads, w.L, w.d), dtype=np.float32)
    p_k = rng.standard_normal((w.batch, w.heads, w.M, w.d), dtype=np.float32)
    p_v = rng.standard_normal((w.batch, w.heads, w.M, w.d), dtype=np.float32)
    return _store(p_o, w.dtype), _store(p_k, w.dtype), _store(p_v, w.dtype)
