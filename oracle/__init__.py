"""UniQL hot-path ORACLE (Python face) -- test infrastructure, not product code.

Thin ctypes wrapper over ``uniql_oracle.c`` (plain scalar fp64 C).  Only the
tests, the smoke check and the benchmark's CPU-baseline leg may import this
package; the CUDA library and its binding never do, and nothing here touches
the CUDA path.  All arithmetic of the method lives in the C file; this module
only converts array types, expands channel maps into explicit index lists and
calls it.

Parity status: every function is pinned by ``tests/test_oracle_pins.py``.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Iterable, Optional, Sequence, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "uniql_oracle.c")
_LIB = os.path.join(_HERE, "_liboracle.so")

GROUP = 128  # quantisation group size along the input channels (Section 3.4)


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (-O2, OpenMP) next to its source."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".%d.tmp" % os.getpid()
        subprocess.check_call(
            ["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        i64, vp = ctypes.c_int64, ctypes.c_void_p
        _lib.uniql_oracle_threads.restype = ctypes.c_int
        _lib.uniql_oracle_pack_u4.argtypes = [vp, i64, i64, vp]
        _lib.uniql_oracle_unpack_u4.argtypes = [vp, i64, i64, vp]
        _lib.uniql_oracle_dequant.argtypes = [vp, vp, vp, i64, i64, i64, vp]
        _lib.uniql_oracle_qlinear.argtypes = [vp, i64, i64, vp, vp, vp, vp, i64, i64, i64,
                                              vp, i64, vp, i64, vp, i64, vp]
        _lib.uniql_oracle_rope.argtypes = [vp, i64, i64, i64, i64, i64, vp, vp,
                                           ctypes.c_double, vp, vp]
        _lib.uniql_oracle_swiglu.argtypes = [vp, vp, i64, vp]
    return _lib


def threads() -> int:
    return int(_load().uniql_oracle_threads())


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _f64(a) -> np.ndarray:
    """Exact widening of fp16 / bf16-valued fp32 / fp64 arrays to contiguous fp64."""
    return np.ascontiguousarray(np.asarray(a), dtype=np.float64)


def pack_u4(codes: np.ndarray) -> np.ndarray:
    codes = np.ascontiguousarray(codes, dtype=np.uint8)
    N, K = codes.shape
    out = np.empty((N, K // 2), dtype=np.uint8)
    rc = _load().uniql_oracle_pack_u4(_p(codes), N, K, _p(out))
    if rc:
        raise ValueError("pack_u4: bad argument (K odd or code > 15)")
    return out


def unpack_u4(packed: np.ndarray) -> np.ndarray:
    packed = np.ascontiguousarray(packed, dtype=np.uint8)
    N, Kh = packed.shape
    out = np.empty((N, 2 * Kh), dtype=np.uint8)
    rc = _load().uniql_oracle_unpack_u4(_p(packed), N, 2 * Kh, _p(out))
    if rc:
        raise ValueError("unpack_u4: bad argument")
    return out


def dequant(packed: np.ndarray, scales, zeros, group: int = GROUP) -> np.ndarray:
    packed = np.ascontiguousarray(packed, dtype=np.uint8)
    N, Kh = packed.shape
    K = 2 * Kh
    s, z = _f64(scales), _f64(zeros)
    assert s.shape == (N, K // group) and z.shape == s.shape
    w = np.empty((N, K), dtype=np.float64)
    rc = _load().uniql_oracle_dequant(_p(packed), _p(s), _p(z), N, K, group, _p(w))
    if rc:
        raise ValueError("dequant: bad argument")
    return w


Family = Tuple[int, int, int, int]  # (start, period, keep, count), stored coordinates


def expand_map(families: Iterable[Family]) -> np.ndarray:
    """Retained channels of a channel map, in compact order.

    A map is a list of periodic families: family (start, period, keep, count)
    keeps the leading ``keep`` channels of each of ``count`` blocks that begin
    at start, start+period, ...  The compact order is the concatenation of the
    families, block after block (Section 3.4: per matrix the trailing sorted
    channels of D_int, of every head's D_hd, of D_s are dropped)."""
    out = []
    for start, period, keep, count in families:
        for h in range(count):
            for i in range(keep):
                out.append(start + h * period + i)
    return np.asarray(out, dtype=np.int32)


def leading(k: int) -> np.ndarray:
    return np.arange(k, dtype=np.int32)


def qlinear(x, packed: np.ndarray, scales, zeros, O: Sequence[int], I: Sequence[int],
            bias=None, rows: Optional[Sequence[int]] = None, group: int = GROUP) -> np.ndarray:
    """fp64 accumulators [R, len(O)] of the pruned quantised linear layer."""
    packed = np.ascontiguousarray(packed, dtype=np.uint8)
    N, Kh = packed.shape
    K = 2 * Kh
    xd = _f64(x)
    assert xd.ndim == 2
    M, ldx = xd.shape
    O = np.ascontiguousarray(O, dtype=np.int32)
    I = np.ascontiguousarray(I, dtype=np.int32)
    assert ldx >= len(I)
    s, z = _f64(scales), _f64(zeros)
    assert s.shape == (N, K // group) and z.shape == s.shape
    b = None if bias is None else _f64(bias)
    r = None if rows is None else np.ascontiguousarray(rows, dtype=np.int32)
    R = M if r is None else len(r)
    acc = np.empty((R, len(O)), dtype=np.float64)
    rc = _load().uniql_oracle_qlinear(_p(xd), M, ldx, _p(packed), _p(s), _p(z), _p(b), N, K, group,
                                      _p(O), len(O), _p(I), len(I), _p(r), 0 if r is None else len(r),
                                      _p(acc))
    if rc:
        raise ValueError("qlinear: bad argument (rc=%d)" % rc)
    return acc


def rope(acc: np.ndarray, n_heads: int, n_kv_heads: int, head_dim: int, head_keep: int,
         idx: np.ndarray, pos: Sequence[int], theta: float,
         inv_freq: Optional[np.ndarray] = None) -> np.ndarray:
    """Rotate fp64 accumulators [R, n_heads*head_keep]; pos has R entries."""
    a = _f64(acc)
    R = a.shape[0]
    assert a.shape[1] == n_heads * head_keep
    idx = np.ascontiguousarray(idx, dtype=np.int32)
    assert idx.shape == (n_kv_heads, head_keep // 2)
    pos = np.ascontiguousarray(pos, dtype=np.int32)
    assert pos.shape == (R,)
    f = None if inv_freq is None else _f64(inv_freq)
    out = np.empty_like(a)
    rc = _load().uniql_oracle_rope(_p(a), R, n_heads, n_kv_heads, head_dim, head_keep, _p(idx),
                                   _p(pos), float(theta), _p(f), _p(out))
    if rc:
        raise ValueError("rope: bad argument (rc=%d)" % rc)
    return out


def qk_halfhead_map(n_heads: int, head_dim: int, head_keep: int) -> list:
    """Output-channel map of a symmetric-sorted Q or K matrix truncated to
    head_keep dims per head: the leading head_keep/2 rows of every half head
    (Algorithm 2: idx_sym = [argsort, D_hd/2 + argsort], so pairs stay intact)."""
    return [(0, head_dim // 2, head_keep // 2, 2 * n_heads)]


def swiglu(g, u) -> np.ndarray:
    """silu(g) * u element by element in fp64 (MLP paragraph of Section 3.2, SiLU gate)."""
    gd, ud = _f64(g), _f64(u)
    assert gd.shape == ud.shape
    out = np.empty_like(gd)
    rc = _load().uniql_oracle_swiglu(_p(gd), _p(ud), gd.size, _p(out))
    if rc:
        raise ValueError("swiglu: bad argument (rc=%d)" % rc)
    return out


def round_bf16(a: np.ndarray) -> np.ndarray:
    """Nearest bfloat16 (8 significand bits, ties to even) of every element, returned in fp64: the value is
    first taken to fp32, whose upper 16 bits are the bfloat16 format, then rounded on the integer pattern."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) & 0xFFFF0000
    return u.astype(np.uint32).view(np.float32).astype(np.float64)


def mlp_swiglu(x, wg, sg, zg, wu, su, zu, wd, sd, zd, k_int: int,
               out_rows: Optional[Sequence[int]] = None, h_dtype: str = "f16") -> Tuple[np.ndarray, np.ndarray]:
    """The pruned SwiGLU MLP block, one call of the oracle per step:
    g = x Wg[:k_int]^T, u = x Wu[:k_int]^T, h = silu(g) * u, y = fp16(h) Wd[:, :k_int]^T.
    The gated activations are a stored fp16 tensor of the model, so they are rounded to
    fp16 (a type conversion, no arithmetic) before the down projection; h_dtype = "bf16"
    for a model whose activations are stored in bfloat16.
    Returns (h in fp64 before that rounding, y in fp64); `out_rows` samples output channels of y."""
    hidden = 2 * np.asarray(wg).shape[1]
    O, I = leading(k_int), leading(hidden)
    g = qlinear(x, wg, sg, zg, O, I)
    u = qlinear(x, wu, su, zu, O, I)
    h = swiglu(g, u)
    h16 = h.astype(np.float16).astype(np.float64) if h_dtype == "f16" else round_bf16(h)
    n_out = np.asarray(wd).shape[0]
    Od = leading(n_out) if out_rows is None else np.ascontiguousarray(out_rows, dtype=np.int32)
    y = qlinear(h16, wd, sd, zd, Od, leading(k_int))
    return h, y
