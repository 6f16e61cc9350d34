"""Seeded synthetic inputs shaped like the paper's workloads.

Pure numpy.  This module holds no arithmetic of the hot path (no unpacking,
de-quantisation, contraction or rotation): it only draws random tensors,
quantises them into codes / scales / zero-points (the offline step that
produces the artefact the hot path consumes, Section 3.4) and names the layer
shapes and channel maps of the benchmark configurations.  Both the CUDA tests
and the CPU oracle's tests are fed from here so that they see identical bits.

Draw order per tensor is fixed: a workload draws W (per matrix, in the order
listed), then x, then the outlier channel set, then pos, then idx.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List, Optional, Tuple

import numpy as np

GROUP = 128
Family = Tuple[int, int, int, int]  # (start, period, keep, count) in stored coordinates


# ----------------------------------------------------------------------------- numeric helpers
def bf16_round(a: np.ndarray) -> np.ndarray:
    """Round fp32 values to the nearest bf16 (ties to even); result stays fp32."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    u = a.view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) & 0xFFFF0000
    return u.astype(np.uint32).view(np.float32)


def to_dtype_values(a: np.ndarray, dtype: str) -> np.ndarray:
    """fp32 array whose values are exactly representable in `dtype` ('f16'|'bf16')."""
    if dtype == "f16":
        return np.asarray(a, dtype=np.float32).astype(np.float16).astype(np.float32)
    if dtype == "bf16":
        return bf16_round(a)
    raise ValueError(dtype)


def bf16_bits(a: np.ndarray) -> np.ndarray:
    """uint16 bit patterns of bf16-representable fp32 values."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    return (a.view(np.uint32) >> 16).astype(np.uint16)


def keep_count(rate: float, D: int) -> int:
    """Channels kept at a keep rate: nearest multiple of 4 (the paper fixes no rule;
    this one yields head dims 128/108/96/84 at 1.0/0.85/0.75/0.65)."""
    return int(4 * round(rate * D / 4.0))


# ----------------------------------------------------------------------------- quantisers
def quantize_asym_u4(W: np.ndarray, group: int = GROUP):
    """Asymmetric uint4, group-wise along K: s=(max-min)/15, z=clamp(rint(-min/s),0,15),
    code=clamp(rint(w/s)+z,0,15); s is stored in fp16 and the codes are computed
    against that stored value.  A constant group gets s=1."""
    N, K = W.shape
    G = K // group
    Wg = W.reshape(N, G, group).astype(np.float64)
    lo, hi = Wg.min(axis=2), Wg.max(axis=2)
    s = (hi - lo) / 15.0
    s = np.where(s > 0, s, 1.0)
    s16 = s.astype(np.float16)
    s16 = np.where(s16 > 0, s16, np.float16(6.1e-5))
    sd = s16.astype(np.float64)
    z = np.clip(np.rint(-lo / sd), 0, 15)
    codes = np.clip(np.rint(Wg / sd[:, :, None]) + z[:, :, None], 0, 15).astype(np.uint8)
    return codes.reshape(N, K), s16, z.astype(np.float16)


def quantize_sym_u4(W: np.ndarray, group: int = GROUP):
    """The paper's symmetric quantiser (Section 3.4): codes clamp(rint(W/s),-8,7),
    s=max|W|/7, stored as code+8 with zero-point 8."""
    N, K = W.shape
    G = K // group
    Wg = W.reshape(N, G, group).astype(np.float64)
    s = np.abs(Wg).max(axis=2) / 7.0
    s = np.where(s > 0, s, 1.0)
    s16 = s.astype(np.float16)
    s16 = np.where(s16 > 0, s16, np.float16(6.1e-5))
    q = np.clip(np.rint(Wg / s16.astype(np.float64)[:, :, None]), -8, 7)
    codes = (q + 8).astype(np.uint8)
    return codes.reshape(N, K), s16, np.full((N, G), 8.0, dtype=np.float16)


# ----------------------------------------------------------------------------- random draws
def draw_weight(rng: np.random.Generator, N: int, K: int, std: float = 0.02) -> np.ndarray:
    return (rng.standard_normal((N, K), dtype=np.float32) * np.float32(std))


def draw_x(rng: np.random.Generator, M: int, K: int, dtype: str = "f16",
           outlier_frac: float = 0.01, outlier_scale: float = 20.0) -> np.ndarray:
    """Activations ~N(0,1); a fraction of the channels (same set for every row) is
    scaled up, as LLM hidden states have a few large channels."""
    x = rng.standard_normal((M, K), dtype=np.float32)
    n_out = int(round(outlier_frac * K))
    if n_out > 0:
        ch = rng.choice(K, size=n_out, replace=False)
        x[:, ch] *= np.float32(outlier_scale)
    return to_dtype_values(x, dtype)


def draw_pos(rng: np.random.Generator, M: int, max_pos: int = 8192) -> np.ndarray:
    return rng.integers(0, max_pos, size=M, dtype=np.int32)


def draw_idx(rng: np.random.Generator, n_kv_heads: int, head_dim: int, head_keep: int,
             kind: str = "perm") -> np.ndarray:
    """Retained ORIGINAL pair indices per KV head: the leading head_keep/2 entries of
    a permutation of 0..head_dim/2-1 (random, identity or reversed)."""
    half, keep = head_dim // 2, head_keep // 2
    out = np.empty((n_kv_heads, keep), dtype=np.int32)
    for g in range(n_kv_heads):
        if kind == "perm":
            p = rng.permutation(half)
        elif kind == "identity":
            p = np.arange(half)
        elif kind == "reversed":
            p = np.arange(half)[::-1]
        else:
            raise ValueError(kind)
        out[g] = p[:keep]
    return out


@dataclass
class QWeight:
    """A quantised matrix in the interchange format, un-packed: codes [N,K] in 0..15,
    fp16 scales and zero-points [N, K/128].  Packing is left to the side under test."""
    codes: np.ndarray
    scales: np.ndarray
    zeros: np.ndarray

    @property
    def N(self) -> int:
        return self.codes.shape[0]

    @property
    def K(self) -> int:
        return self.codes.shape[1]


def draw_qweight(rng: np.random.Generator, N: int, K: int, std: float = 0.02,
                 symmetric: bool = False) -> QWeight:
    W = draw_weight(rng, N, K, std)
    c, s, z = (quantize_sym_u4 if symmetric else quantize_asym_u4)(W)
    return QWeight(c, s, z)


def random_qweight_fast(rng: np.random.Generator, N: int, K: int) -> QWeight:
    """Large-matrix variant for throughput runs: uniform random codes and scales of the
    magnitude the quantiser yields for N(0,0.02) weights (values do not affect timing)."""
    codes = rng.integers(0, 16, size=(N, K), dtype=np.uint8)
    G = K // GROUP
    s = (0.0075 * (1.0 + 0.1 * rng.standard_normal((N, G), dtype=np.float32))).astype(np.float16)
    z = rng.integers(6, 10, size=(N, G)).astype(np.float16)
    return QWeight(codes, s, z)


# ----------------------------------------------------------------------------- channel maps
def map_leading(k: int) -> List[Family]:
    return [(0, max(k, 1), k, 1)]


def map_per_head(n_heads: int, head_dim: int, head_keep: int, start: int = 0) -> List[Family]:
    return [(start, head_dim, head_keep, n_heads)]


def map_qk_halfheads(n_heads: int, head_dim: int, head_keep: int) -> List[Family]:
    """Symmetric-sorted Q/K rows: leading head_keep/2 of each half head."""
    return [(0, head_dim // 2, head_keep // 2, 2 * n_heads)]


def map_mamba_in_proj(d_inner: int, headdim: int, head_keep: int, d_state: int, ngroups: int,
                      nheads: int, state_keep: Optional[int] = None) -> List[Family]:
    """Mamba2 in_proj rows in the order z, x, B, C, dt; z and x pruned per SSM head.  With state_keep the
    state dimension D_s is pruned too: every group of B and of C keeps its leading state_keep rows."""
    if state_keep is None or state_keep == d_state:
        bc_dt = 2 * ngroups * d_state + nheads
        return [(0, headdim, head_keep, nheads), (d_inner, headdim, head_keep, nheads),
                (2 * d_inner, bc_dt, bc_dt, 1)]
    b0 = 2 * d_inner
    c0 = b0 + ngroups * d_state
    dt0 = c0 + ngroups * d_state
    return [(0, headdim, head_keep, nheads), (d_inner, headdim, head_keep, nheads),
            (b0, d_state, state_keep, ngroups), (c0, d_state, state_keep, ngroups), (dt0, nheads, nheads, 1)]


def map_size(fams: List[Family]) -> int:
    return sum(keep * count for (_, _, keep, count) in fams)


# ----------------------------------------------------------------------------- model shapes
@dataclass
class LayerShapes:
    name: str
    hidden: int
    intermediate: int = 0
    n_q_heads: int = 0
    n_kv_heads: int = 0
    head_dim: int = 128
    theta: float = 10000.0
    extra: Dict[str, int] = field(default_factory=dict)


LLAMA3_8B = LayerShapes("llama3-8b", hidden=4096, intermediate=14336, n_q_heads=32, n_kv_heads=8,
                        head_dim=128, theta=500000.0)
QWEN25_7B = LayerShapes("qwen2.5-7b", hidden=3584, intermediate=18944, n_q_heads=28, n_kv_heads=4,
                        head_dim=128, theta=1000000.0)
MAMBA2_2P7B = LayerShapes("mamba2-2.7b", hidden=2560,
                          extra=dict(d_inner=5120, d_state=128, ngroups=1, headdim=64, nheads=80,
                                     in_proj_rows=10576))

KEEP_RATES = (1.0, 0.85, 0.75, 0.65)
