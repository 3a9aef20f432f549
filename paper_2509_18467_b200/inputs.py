"""Seeded synthetic inputs for the LAWCAT layer, shared by the tests, the benchmark and the smoke check.

This module holds no arithmetic of the method: it draws random tensors of the layer's shapes from a counter-based
generator (numpy's Philox), optionally rounds them to bfloat16 values (round-to-nearest-even, done on the host so
that the CPU oracle and the GPU see identical bits), and names the benchmark configurations.

Recipe: q, k, v ~ N(0,1); gate logits ~ N(0,1); mix weights W_h ~ N(0, 1/d_k); conv taps ~ N(0, 1/conv_k);
upstream gradients ~ N(0,1). Tensor i of configuration c uses seed BASE_SEED + 16*c + i.
Gate function (two low-rank linear layers in front of the gate): hidden states x ~ N(0,1), first layer ~ N(0, 1/d_model),
second layer ~ N(0, 1/rank), bias ~ N(0, 1/4), so that the logits are about N(0, 1.25); seeds BASE_SEED + 2^20 + 16*c + i.
"""
from __future__ import annotations

from dataclasses import dataclass, replace

import numpy as np

BASE_SEED = 0x250918467000

# tensor indices (the "+ i" of the seed)
_IDX = dict(q=0, k=1, v=2, gate=3, w_q=4, w_k=5, W=6, dO=7, cache_q=8, cache_k=9, S0=10, z0=11, d_qdot=12,
            d_kdot=13)


@dataclass(frozen=True)
class LayerShape:
    """Shape and options of one workload; field names follow the C parameter block."""
    B: int
    T: int
    H: int
    H_kv: int
    d_k: int
    d_v: int
    conv_k: int = 4
    gate_dim: int = 0        # 0 -> d_k (one decay per key channel)
    dtype: str = "bf16"      # "f32" | "bf16"
    gate_tau: float = 16.0
    config_id: int = 0
    name: str = ""

    @property
    def gd(self) -> int:
        return self.gate_dim or self.d_k


# The benchmark configurations (index = position in the baseline's list of configurations).
CONFIGS = {
    "c1": LayerShape(1, 512, 4, 4, 64, 64, dtype="f32", config_id=1, name="c1-fp32-T512-H4-d64"),
    "c2": LayerShape(1, 8192, 32, 8, 64, 64, config_id=2, name="c2-llama3.2-1b-T8192"),
    "c3": LayerShape(1, 32768, 32, 8, 128, 128, config_id=3, name="c3-mistral-7b-T32768"),
    "c4": LayerShape(8, 1024, 32, 8, 64, 64, config_id=4, name="c4-distill-llama3.2-1b-B8-T1024"),
    "c5-decode": LayerShape(64, 1, 32, 8, 128, 128, config_id=5, name="c5-decode-mistral-7b-B64"),
}


def with_T(shape: LayerShape, T: int) -> LayerShape:
    return replace(shape, T=T)


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """Round float32 values to the nearest bfloat16 (ties to even); the result is still float32."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32)
    r = ((u >> 16) & 1) + np.uint32(0x7FFF)
    return ((u + r) & np.uint32(0xFFFF0000)).view(np.float32)


def bf16_bits(x: np.ndarray) -> np.ndarray:
    """uint16 bit patterns of float32 values that are already exactly representable in bfloat16."""
    return (np.ascontiguousarray(x, dtype=np.float32).view(np.uint32) >> 16).astype(np.uint16)


def bits_to_f32(b: np.ndarray) -> np.ndarray:
    """float32 values of bfloat16 bit patterns (uint16)."""
    return (b.astype(np.uint32) << 16).view(np.float32)


def _normal(seed: int, shape, scale: float = 1.0) -> np.ndarray:
    g = np.random.Generator(np.random.Philox(key=seed))
    a = g.standard_normal(size=shape, dtype=np.float32)
    if scale != 1.0:
        a *= np.float32(scale)
    return a


def make(shape: LayerShape, names, seed_offset: int = 0) -> dict:
    """Draw the named tensors (subset of q k v gate w_q w_k W dO cache_q cache_k S0 z0 d_qdot d_kdot) as float32
    arrays; for dtype 'bf16' every tensor except the fp32 states S0, z0 holds bf16-representable values."""
    s = shape
    K = s.conv_k
    shp = dict(
        q=(s.B, s.T, s.H, s.d_k), k=(s.B, s.T, s.H_kv, s.d_k), v=(s.B, s.T, s.H_kv, s.d_v),
        gate=(s.B, s.T, s.H, s.gd), w_q=(s.H * s.d_k, K), w_k=(s.H_kv * s.d_k, K), W=(s.H, s.d_k, s.d_k),
        dO=(s.B, s.T, s.H, s.d_v), cache_q=(s.B, K - 1, s.H * s.d_k), cache_k=(s.B, K - 1, s.H_kv * s.d_k),
        S0=(s.B, s.H, s.d_k, s.d_v), z0=(s.B, s.H, s.d_k), d_qdot=(s.B, s.T, s.H, s.d_k),
        d_kdot=(s.B, s.T, s.H, s.d_k))
    scale = dict(W=1.0 / np.sqrt(s.d_k), w_q=1.0 / np.sqrt(K), w_k=1.0 / np.sqrt(K))
    out = {}
    for n in names:
        a = _normal(BASE_SEED + 16 * s.config_id + _IDX[n] + 1024 * seed_offset, shp[n], scale.get(n, 1.0))
        if n in ("S0", "z0"):
            a = np.abs(a)  # a state reached from positive features is positive; keeps denominators away from 0
        elif s.dtype == "bf16":
            a = round_to_bf16(a)
        out[n] = a
    return out


def make_gate_fn(shape: LayerShape, d_model: int, rank: int, seed_offset: int = 0) -> dict:
    """Inputs of the gate function for a workload: x [B,T,d_model], A1 [rank,d_model], A2 [H*gate_dim,rank],
    bias [H*gate_dim], float32 arrays (bf16-representable values for dtype 'bf16')."""
    s = shape
    n_out = s.H * s.gd
    shp = dict(x=(s.B, s.T, d_model), A1=(rank, d_model), A2=(n_out, rank), bias=(n_out,))
    scale = dict(x=1.0, A1=1.0 / np.sqrt(d_model), A2=1.0 / np.sqrt(rank), bias=0.5)
    out = {}
    for i, n in enumerate(("x", "A1", "A2", "bias")):
        a = _normal(BASE_SEED + (1 << 20) + 16 * s.config_id + i + 1024 * seed_offset, shp[n], scale[n])
        out[n] = round_to_bf16(a) if s.dtype == "bf16" else a
    return out
