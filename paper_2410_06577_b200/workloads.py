"""Seeded synthetic inputs for the DDTS recurrence.

This module holds NONE of the method's arithmetic: it only draws random numbers in a
fixed order and rounds them to the dtype the GPU consumes, so that the CPU oracle and
the CUDA library see identical bits.  Both the tests and the benchmark import it.

Draw order for every workload: q, k, v, x (gate pre-activation), y (temperature
pre-activation), s0 (if any); the gradients fed to the backward pass come from a generator of
their own (d_o, then dL/dS_T if any).  Varlen lengths are drawn first from their own generator.
All arrays are returned as float32 whose values are exactly representable in ``dtype``.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Optional

import numpy as np


def round_to_bf16(a: np.ndarray) -> np.ndarray:
    """Round float32 to the nearest bfloat16 (ties to even); result stays float32."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    u = a.view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) & 0xFFFF0000
    return u.astype(np.uint32).view(np.float32).reshape(a.shape)


def _round(a: np.ndarray, dtype: str) -> np.ndarray:
    a = a.astype(np.float32)
    return round_to_bf16(a) if dtype == "bf16" else a


@dataclass
class PrefillInputs:
    dtype: str                      # "bf16" or "f32": dtype of q,k,v,x,y,o on the GPU
    q: np.ndarray                   # [B,H,T,dk]
    k: np.ndarray
    x: np.ndarray                   # gate pre-activation
    y: np.ndarray                   # temperature pre-activation
    v: np.ndarray                   # [B,H,T,dv]
    s0: Optional[np.ndarray] = None  # [B|N,H,dk,dv] float32
    cu_seqlens: Optional[np.ndarray] = None  # int32 [N+1]
    name: str = ""
    meta: dict = field(default_factory=dict)

    @property
    def shape(self):
        B, H, T, dk = self.q.shape
        return B, H, T, dk, self.v.shape[-1]

    @property
    def tokens(self) -> int:
        B, _, T, _ = self.q.shape
        return B * T


@dataclass
class DecodeInputs:
    dtype: str
    q: np.ndarray                   # [R,Nseq,H,dk]: a ring of R distinct token inputs
    k: np.ndarray
    x: np.ndarray
    y: np.ndarray
    v: np.ndarray                   # [R,Nseq,H,dv]
    state: np.ndarray               # [Nseq,H,dk,dv] float32
    name: str = ""


def make_prefill(seed: int, B: int, H: int, T: int, dk: int, dv: int, dtype: str = "bf16",
                 gate_mean: float = -3.0, s0_std: Optional[float] = None,
                 cu_seqlens: Optional[np.ndarray] = None, name: str = "") -> PrefillInputs:
    """q,k ~ N(0,1)/sqrt(dk); v ~ N(0,1); x ~ N(gate_mean,1); y ~ N(0,1); s0 ~ N(0,s0_std)."""
    rng = np.random.default_rng(seed)
    shape_k = (B, H, T, dk)
    q = _round(rng.standard_normal(shape_k, dtype=np.float32) / np.float32(np.sqrt(dk)), dtype)
    k = _round(rng.standard_normal(shape_k, dtype=np.float32) / np.float32(np.sqrt(dk)), dtype)
    v = _round(rng.standard_normal((B, H, T, dv), dtype=np.float32), dtype)
    x = _round(rng.standard_normal(shape_k, dtype=np.float32) + np.float32(gate_mean), dtype)
    y = _round(rng.standard_normal(shape_k, dtype=np.float32), dtype)
    s0 = None
    if s0_std is not None:
        nseq = B if cu_seqlens is None else len(cu_seqlens) - 1
        s0 = (rng.standard_normal((nseq, H, dk, dv), dtype=np.float32) * np.float32(s0_std))
    cu = None if cu_seqlens is None else np.ascontiguousarray(cu_seqlens, dtype=np.int32)
    return PrefillInputs(dtype, q, k, x, y, v, s0, cu, name)


def make_grads(seed: int, p: PrefillInputs, with_state: bool = True, state_std: float = 0.1):
    """Incoming gradients for the backward pass: dL/do ~ N(0,1) in the workload's dtype and, if
    asked for, dL/dS_T ~ N(0, state_std) in float32.  Returns (d_o [B,H,T,dv], d_sT or None)."""
    rng = np.random.default_rng(seed)
    B, H, T, dk, dv = p.shape
    d_o = _round(rng.standard_normal((B, H, T, dv), dtype=np.float32), p.dtype)
    d_sT = None
    if with_state:
        nseq = B if p.cu_seqlens is None else len(p.cu_seqlens) - 1
        d_sT = rng.standard_normal((nseq, H, dk, dv), dtype=np.float32) * np.float32(state_std)
    return d_o, d_sT


def make_value_decay(seed: int, shape, dtype: str, low: float = 0.8) -> np.ndarray:
    """Value-side decay factors beta_t for the ablation arm: uniform in (low, 1], rounded to the
    workload's dtype."""
    rng = np.random.default_rng(seed)
    return _round(np.float32(1.0) - np.float32(1.0 - low) * rng.random(shape, dtype=np.float32), dtype)


def make_swska(seed: int, B: int, H: int, T: int, d: int = 128, dtype: str = "bf16"):
    """Inputs of the sliding-window shared-key attention: q [B,H,T,d], the shared k [B,T,d] and
    v [B,H,T,d], all ~ N(0,1), rounded to ``dtype`` (draw order q, k, v)."""
    rng = np.random.default_rng(seed)
    q = _round(rng.standard_normal((B, H, T, d), dtype=np.float32), dtype)
    k = _round(rng.standard_normal((B, T, d), dtype=np.float32), dtype)
    v = _round(rng.standard_normal((B, H, T, d), dtype=np.float32), dtype)
    return q, k, v


def varlen_lengths(seed: int, n_seq: int, lo: int, hi: int) -> np.ndarray:
    """Lengths uniform in [lo, hi] and their exclusive prefix sum (int32 [n_seq+1])."""
    rng = np.random.default_rng(seed)
    lens = rng.integers(lo, hi + 1, n_seq)
    cu = np.zeros(n_seq + 1, dtype=np.int32)
    cu[1:] = np.cumsum(lens)
    return cu


def make_decode(seed: int, Nseq: int, H: int, dk: int, dv: int, ring: int = 16,
                dtype: str = "bf16", gate_mean: float = -3.0, state_std: float = 0.1,
                name: str = "") -> DecodeInputs:
    rng = np.random.default_rng(seed)
    sk = (ring, Nseq, H, dk)
    q = _round(rng.standard_normal(sk, dtype=np.float32) / np.float32(np.sqrt(dk)), dtype)
    k = _round(rng.standard_normal(sk, dtype=np.float32) / np.float32(np.sqrt(dk)), dtype)
    v = _round(rng.standard_normal((ring, Nseq, H, dv), dtype=np.float32), dtype)
    x = _round(rng.standard_normal(sk, dtype=np.float32) + np.float32(gate_mean), dtype)
    y = _round(rng.standard_normal(sk, dtype=np.float32), dtype)
    state = rng.standard_normal((Nseq, H, dk, dv), dtype=np.float32) * np.float32(state_std)
    return DecodeInputs(dtype, q, k, x, y, v, state, name)


# The five named workloads.  ``shrink`` divides the large dimension so that the oracle can
# check every element in seconds while still spanning several tiles and a ragged tail.
def config(idx: int, shrink: int = 1):
    if idx == 0:
        return make_prefill(0, 1, 1, 256, 64, 64, "f32", name="cfg0_single_f32")
    if idx == 1:
        return make_prefill(1, max(1, 4 // shrink), max(1, 16 // shrink), 2048, 128, 256, "bf16",
                            name="cfg1_layer_prefill")
    if idx == 2:
        return make_prefill(2, 1, max(1, 16 // shrink), 32768 // shrink, 128, 256, "bf16",
                            gate_mean=-4.0, s0_std=0.1, name="cfg2_long_context")
    if idx == 3:
        return make_decode(3, max(1, 256 // shrink), max(1, 16 // shrink), 128, 256,
                           name="cfg3_decode")
    if idx == 4:
        n_seq = max(2, 64 // shrink)
        cu = varlen_lengths(4, n_seq, 128, 4096 // shrink if shrink > 1 else 4096)
        T = int(cu[-1])
        p = make_prefill(4, 1, max(1, 16 // shrink), T, 128, 256, "bf16", cu_seqlens=cu,
                         name="cfg4_varlen")
        return p
    raise ValueError(f"no such config: {idx}")
