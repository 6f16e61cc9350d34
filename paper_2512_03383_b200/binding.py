"""ctypes binding of libuniql.so: argument marshalling only.

Function names follow the C ABI (include/uniql.h).  Tensors are torch CUDA tensors used
as device buffers; the current torch stream is passed unless one is given.  There is no
fallback: if the CUDA library is missing or fails to load, importing this module raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import List, Optional, Sequence, Tuple

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libuniql.so")

UNIQL_F16, UNIQL_BF16 = 0, 1
PATH_AUTO, PATH_GENERIC, PATH_DECODE, PATH_PREFILL, PATH_GEMV = 0, 1, 2, 3, 4
MAX_FAMILIES, MAX_JOBS = 8, 4

Family = Tuple[int, int, int, int]


class UniqlError(RuntimeError):
    def __init__(self, status: int, what: str):
        super().__init__("%s: status %d (%s)" % (what, status, status_string(status)))
        self.status = status


class _Family(ctypes.Structure):
    _fields_ = [("start", ctypes.c_int32), ("period", ctypes.c_int32), ("keep", ctypes.c_int32),
                ("count", ctypes.c_int32)]


class _ChanMap(ctypes.Structure):
    _fields_ = [("n_fam", ctypes.c_int32), ("fam", _Family * MAX_FAMILIES)]


class _Job(ctypes.Structure):
    _fields_ = [("packed_w", ctypes.c_void_p), ("scales", ctypes.c_void_p), ("zeros", ctypes.c_void_p),
                ("bias", ctypes.c_void_p), ("N", ctypes.c_int32), ("k_out", ctypes.c_int32),
                ("out_map", ctypes.POINTER(_ChanMap)), ("y", ctypes.c_void_p), ("ldy", ctypes.c_int32)]


if not os.path.exists(LIB_PATH):
    raise ImportError("libuniql.so is not built (run `python -m paper_2512_03383_b200.build`); "
                      "there is no fallback path")
_lib = ctypes.CDLL(LIB_PATH)

_vp, _i, _i64, _sz, _d = ctypes.c_void_p, ctypes.c_int, ctypes.c_int64, ctypes.c_size_t, ctypes.c_double
_lib.uniql_version.restype = _i
_lib.uniql_status_string.restype = ctypes.c_char_p
_lib.uniql_status_string.argtypes = [_i]
_lib.uniql_set_path.argtypes = [_i]
_lib.uniql_pack_u4.argtypes = [_vp, _i64, _i64, _vp, _vp]
_lib.uniql_unpack_u4.argtypes = [_vp, _i64, _i64, _vp, _vp]
_lib.uniql_dequant.argtypes = [_vp, _vp, _vp, _i64, _i64, _i, _vp, _vp]
_lib.uniql_workspace_bytes.restype = _sz
_lib.uniql_workspace_bytes.argtypes = [_i, _i, _i]
_lib.uniql_workspace_init.argtypes = [_vp, _sz, _vp]
_lib.uniql_workspace_status.argtypes = [_vp, ctypes.POINTER(_i)]
_lib.uniql_qlinear.argtypes = [_vp, _vp, _vp, _vp, _i, _i, _i, _i, _i, _vp, _vp]
_lib.uniql_qkv_rope_proj.argtypes = [_vp, _i, _i, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _i, _i, _i,
                                     _i, _i, _i, _i, _vp, _vp, _d, ctypes.POINTER(_d), _vp, _i, _vp, _i, _vp, _i,
                                     _vp, _sz, _vp]
_lib.uniql_embed_rows.argtypes = [_vp, _vp, _vp, _i64, _i64, _vp, _i64, _i, _vp, _i64, _vp, _vp]
_lib.uniql_mlp_workspace_bytes.restype = _sz
_lib.uniql_mlp_workspace_bytes.argtypes = [_i, _i, _i]
_lib.uniql_mlp_swiglu_decode.argtypes = [_vp, _i, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _i, _i, _i, _i,
                                         _vp, _i, _vp, _i, _i, _vp, _sz, _vp]
_lib.uniql_mlp_swiglu.argtypes = [_vp, _i, _i, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _i, _i, _i, _i,
                                  _vp, _i, _vp, _i, _vp, _sz, _vp]
_lib.uniql_qlinear_noalloc.argtypes = [_vp, _vp, _vp, _vp, _i, _i, _i, _i, _i, _vp, _vp]
_lib.uniql_qlinear_ex.argtypes = [_vp, _i, _i, _vp, _vp, _vp, _vp, _i, _i, _i, ctypes.POINTER(_ChanMap), _i,
                                  ctypes.POINTER(_ChanMap), _i, _vp, _i, _vp, _sz, _vp]
_lib.uniql_qlinear_multi.argtypes = [_vp, _i, _i, _i, _i, ctypes.POINTER(_ChanMap), _i, _i,
                                     ctypes.POINTER(_Job), _vp, _sz, _vp]
_lib.uniql_qk_rope_proj.argtypes = [_vp, _i, _i, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _i, _i, _i, _i, _i, _i,
                                    _vp, _vp, _d, ctypes.POINTER(_d), _vp, _i, _vp, _i, _vp, _sz, _vp]
for _n in ("uniql_set_path", "uniql_pack_u4", "uniql_unpack_u4", "uniql_dequant", "uniql_workspace_init",
           "uniql_workspace_status", "uniql_qlinear", "uniql_qlinear_noalloc", "uniql_noalloc_status", "uniql_qlinear_ex", "uniql_qlinear_multi", "uniql_qk_rope_proj",
           "uniql_mlp_swiglu_decode", "uniql_mlp_swiglu", "uniql_qkv_rope_proj", "uniql_embed_rows"):
    getattr(_lib, _n).restype = _i


_lib.uniql_set_option.argtypes = [ctypes.c_char_p, _i]
_lib.uniql_set_option.restype = _i
_lib.uniql_noalloc_status.argtypes = [ctypes.POINTER(_i)]

OPTION_DEFAULTS = {"pdl": 1, "decode_kp": 0, "decode_rp": 0, "decode_stages": 0, "decode_narrow": -1,
                   "decode_xstream": -1, "decode_xcluster": -1, "decode_i8": 1, "decode_split_batch": 2,
                   "prefill_grid": 0, "prefill_convert": 0, "prefill_streamk": -1, "prefill_dual": -1, "prefill_helpers": 1, "gemv_first": 0, "gemv_depth": 0,
                   "wait_shift": 0}


def set_option(name: str, value: int) -> None:
    """uniql_set_option: a tuning / test option of the process (see include/uniql.h)."""
    _check(_lib.uniql_set_option(name.encode(), int(value)), "uniql_set_option")


def reset_options() -> None:
    for k, v in OPTION_DEFAULTS.items():
        set_option(k, v)


def lib() -> ctypes.CDLL:
    return _lib


def version() -> int:
    return int(_lib.uniql_version())


def status_string(status: int) -> str:
    return _lib.uniql_status_string(int(status)).decode()


def _check(status: int, what: str) -> None:
    if status != 0:
        raise UniqlError(status, what)


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream(stream) -> ctypes.c_void_p:
    if stream is None:
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream))


def _dt(t: torch.Tensor) -> int:
    if t.dtype == torch.float16:
        return UNIQL_F16
    if t.dtype == torch.bfloat16:
        return UNIQL_BF16
    raise TypeError("activations must be float16 or bfloat16, got %s" % t.dtype)


def chanmap(families: Optional[Sequence[Family]]) -> Optional[_ChanMap]:
    if families is None:
        return None
    if len(families) > MAX_FAMILIES:
        raise ValueError("at most %d families" % MAX_FAMILIES)
    m = _ChanMap()
    m.n_fam = len(families)
    for i, (start, period, keep, count) in enumerate(families):
        m.fam[i] = _Family(start, period, keep, count)
    return m


def _mapref(m: Optional[_ChanMap]):
    return None if m is None else ctypes.byref(m)


def set_path(path: int) -> None:
    _check(_lib.uniql_set_path(path), "uniql_set_path")


def pack_u4(codes: torch.Tensor, packed: torch.Tensor, stream=None) -> None:
    N, K = codes.shape
    _check(_lib.uniql_pack_u4(_ptr(codes), N, K, _ptr(packed), _stream(stream)), "uniql_pack_u4")


def unpack_u4(packed: torch.Tensor, codes: torch.Tensor, stream=None) -> None:
    N, K = codes.shape
    _check(_lib.uniql_unpack_u4(_ptr(packed), N, K, _ptr(codes), _stream(stream)), "uniql_unpack_u4")


def dequant(packed: torch.Tensor, scales: torch.Tensor, zeros: torch.Tensor, w: torch.Tensor, stream=None) -> None:
    N, K = w.shape
    _check(_lib.uniql_dequant(_ptr(packed), _ptr(scales), _ptr(zeros), N, K, _dt(w), _ptr(w), _stream(stream)),
           "uniql_dequant")


def workspace_bytes(M: int, K: int, N_total: int) -> int:
    return int(_lib.uniql_workspace_bytes(M, K, N_total))


def workspace_init(ws: torch.Tensor, stream=None) -> None:
    _check(_lib.uniql_workspace_init(_ptr(ws), ws.numel() * ws.element_size(), _stream(stream)),
           "uniql_workspace_init")


def workspace_status(ws: Optional[torch.Tensor] = None) -> int:
    """Device status word of a workspace (None: the library's own); synchronises the device."""
    out = _i(0)
    _check(_lib.uniql_workspace_status(_ptr(ws), ctypes.byref(out)), "uniql_workspace_status")
    return int(out.value)


def qlinear(x, packed_w, scales, zeros, M, K, N, k_in, k_out, y, stream=None) -> None:
    _check(_lib.uniql_qlinear(_ptr(x), _ptr(packed_w), _ptr(scales), _ptr(zeros), M, K, N, k_in, k_out, _ptr(y),
                              _stream(stream)), "uniql_qlinear")


def qlinear_noalloc(x, packed_w, scales, zeros, M, K, N, k_in, k_out, y, stream=None) -> None:
    """uniql_qlinear for callers that must not allocate device memory: the kernel's scratch is a fixed
    array inside the library (decode sizes only, M <= 16)."""
    _check(_lib.uniql_qlinear_noalloc(_ptr(x), _ptr(packed_w), _ptr(scales), _ptr(zeros), M, K, N, k_in, k_out,
                                      _ptr(y), _stream(stream)), "uniql_qlinear_noalloc")


def noalloc_status() -> int:
    """Status word of the uniql_qlinear_noalloc calls made so far (synchronises the device; allocates nothing)."""
    v = ctypes.c_int(0)
    _check(_lib.uniql_noalloc_status(ctypes.byref(v)), "uniql_noalloc_status")
    return int(v.value)


def qlinear_ex(x, ldx, packed_w, scales, zeros, bias, M, K, N, in_map, k_in, out_map, k_out, y, ldy,
               workspace=None, stream=None) -> None:
    im, om = chanmap(in_map), chanmap(out_map)
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(_lib.uniql_qlinear_ex(_ptr(x), ldx, _dt(x), _ptr(packed_w), _ptr(scales), _ptr(zeros), _ptr(bias), M, K,
                                 N, _mapref(im), k_in, _mapref(om), k_out, _ptr(y), ldy, _ptr(workspace), ws_bytes,
                                 _stream(stream)), "uniql_qlinear_ex")


def qlinear_multi(x, ldx, M, K, in_map, k_in, jobs: List[dict], workspace=None, stream=None) -> None:
    """jobs: dicts with packed_w, scales, zeros, bias(None), N, k_out, out_map(None), y, ldy."""
    arr = (_Job * len(jobs))()
    keep = []
    for i, j in enumerate(jobs):
        om = chanmap(j.get("out_map"))
        keep.append(om)
        arr[i].packed_w = j["packed_w"].data_ptr()
        arr[i].scales = j["scales"].data_ptr()
        arr[i].zeros = j["zeros"].data_ptr()
        arr[i].bias = None if j.get("bias") is None else j["bias"].data_ptr()
        arr[i].N = j["N"]
        arr[i].k_out = j.get("k_out", 0)
        arr[i].out_map = ctypes.pointer(om) if om is not None else None
        arr[i].y = j["y"].data_ptr()
        arr[i].ldy = j["ldy"]
    im = chanmap(in_map)
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(_lib.uniql_qlinear_multi(_ptr(x), ldx, _dt(x), M, K, _mapref(im), k_in, len(jobs), arr, _ptr(workspace),
                                    ws_bytes, _stream(stream)), "uniql_qlinear_multi")


def qk_rope_proj(x, ldx, wq, sq, zq, wk, sk, zk, bq, bk, M, K, n_q_heads, n_kv_heads, head_dim, head_keep,
                 retained_idx, pos, theta, inv_freq, q_out, ldq, k_out, ldk, workspace=None, stream=None) -> None:
    f = None
    if inv_freq is not None:
        f = (ctypes.c_double * len(inv_freq))(*[float(v) for v in inv_freq])
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(_lib.uniql_qk_rope_proj(_ptr(x), ldx, _dt(x), _ptr(wq), _ptr(sq), _ptr(zq), _ptr(wk), _ptr(sk), _ptr(zk),
                                   _ptr(bq), _ptr(bk), M, K, n_q_heads, n_kv_heads, head_dim, head_keep,
                                   _ptr(retained_idx), _ptr(pos), float(theta), f, _ptr(q_out), ldq, _ptr(k_out),
                                   ldk, _ptr(workspace), ws_bytes, _stream(stream)), "uniql_qk_rope_proj")


def mlp_workspace_bytes(M: int, hidden: int, inter: int) -> int:
    return int(_lib.uniql_mlp_workspace_bytes(M, hidden, inter))


def mlp_swiglu_decode(x, ldx, wg, sg, zg, wu, su, zu, wd, sd, zd, M, hidden, inter, k_int, h, ldh, y, ldy,
                      fuse=-1, workspace=None, stream=None) -> None:
    if x.dtype != torch.float16 or h.dtype != torch.float16 or y.dtype != torch.float16:
        raise TypeError("uniql_mlp_swiglu_decode computes in fp16")
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(_lib.uniql_mlp_swiglu_decode(_ptr(x), ldx, _ptr(wg), _ptr(sg), _ptr(zg), _ptr(wu), _ptr(su), _ptr(zu),
                                        _ptr(wd), _ptr(sd), _ptr(zd), M, hidden, inter, k_int, _ptr(h), ldh,
                                        _ptr(y), ldy, int(fuse), _ptr(workspace), ws_bytes, _stream(stream)),
           "uniql_mlp_swiglu_decode")


def mlp_swiglu(x, ldx, wg, sg, zg, wu, su, zu, wd, sd, zd, M, hidden, inter, k_int, h, ldh, y, ldy,
               workspace=None, stream=None) -> None:
    """uniql_mlp_swiglu: the SwiGLU MLP block for fp16 or bf16 activations and any M (x, h, y of one type)."""
    if h.dtype != x.dtype or y.dtype != x.dtype:
        raise TypeError("x, h and y must have the same type")
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(_lib.uniql_mlp_swiglu(_ptr(x), ldx, _dt(x), _ptr(wg), _ptr(sg), _ptr(zg), _ptr(wu), _ptr(su), _ptr(zu),
                                 _ptr(wd), _ptr(sd), _ptr(zd), M, hidden, inter, k_int, _ptr(h), ldh, _ptr(y), ldy,
                                 _ptr(workspace), ws_bytes, _stream(stream)), "uniql_mlp_swiglu")


def qkv_rope_proj(x, ldx, wq, sq, zq, wk, sk, zk, wv, sv, zv, bq, bk, bv, M, K, n_q_heads, n_kv_heads, head_dim,
                  head_keep, v_keep, retained_idx, pos, theta, inv_freq, q_out, ldq, k_out, ldk, v_out, ldv,
                  workspace=None, stream=None) -> None:
    f = None
    if inv_freq is not None:
        f = (ctypes.c_double * len(inv_freq))(*[float(v) for v in inv_freq])
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(_lib.uniql_qkv_rope_proj(_ptr(x), ldx, _dt(x), _ptr(wq), _ptr(sq), _ptr(zq), _ptr(wk), _ptr(sk), _ptr(zk),
                                    _ptr(wv), _ptr(sv), _ptr(zv), _ptr(bq), _ptr(bk), _ptr(bv), M, K, n_q_heads,
                                    n_kv_heads, head_dim, head_keep, v_keep, _ptr(retained_idx), _ptr(pos),
                                    float(theta), f, _ptr(q_out), ldq, _ptr(k_out), ldk, _ptr(v_out), ldv,
                                    _ptr(workspace), ws_bytes, _stream(stream)), "uniql_qkv_rope_proj")


def embed_rows(packed, scales, zeros, ids, out, bad_id=None, stream=None) -> None:
    V, K = packed.shape[0], packed.shape[1] * 2
    _check(_lib.uniql_embed_rows(_ptr(packed), _ptr(scales), _ptr(zeros), V, K, _ptr(ids), ids.numel(), _dt(out),
                                 _ptr(out), out.stride(0), _ptr(bad_id), _stream(stream)), "uniql_embed_rows")
