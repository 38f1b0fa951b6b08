"""ctypes front end of the plain CPU oracle (``rudder_oracle.c``).

TEST INFRASTRUCTURE ONLY: imported by the tests, by the smoke check and by the benchmark's CPU
baseline leg.  The product package never imports this module, and this module never imports the
product package.  Arrays are numpy; bf16 / fp16 values travel as ``uint16`` bit patterns.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "rudder_oracle.c"
_HDR = _HERE / "rudder_oracle.h"
_LIB = _HERE / "_rudder_oracle.so"

RANGE_PER_TOKEN = 0
RANGE_STATIC = 1


def build(force: bool = False) -> Path:
    """Compile the oracle with gcc (fp32 operations individually rounded, OpenMP over rows)."""
    stale = (not _LIB.exists()) or _LIB.stat().st_mtime < max(_SRC.stat().st_mtime, _HDR.stat().st_mtime)
    if force or stale:
        tmp = _LIB.with_suffix(f".{os.getpid()}.tmp")
        cmd = ["gcc", "-std=c11", "-O2", "-ffp-contract=off", "-fno-fast-math", "-fopenmp", "-fPIC",
               "-shared", "-Wall", "-Wextra", "-o", str(tmp), str(_SRC), "-lm"]
        subprocess.run(cmd, check=True)
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(str(build()))
        _lib.orc_bf16_decode.restype = ctypes.c_float
        _lib.orc_fp16_decode.restype = ctypes.c_float
        _lib.orc_ue4m3_decode.restype = ctypes.c_float
        _lib.orc_e2m1_decode.restype = ctypes.c_float
        _lib.orc_bf16_encode.restype = ctypes.c_uint16
        _lib.orc_fp16_encode.restype = ctypes.c_uint16
        _lib.orc_ue4m3_encode.restype = ctypes.c_uint8
        _lib.orc_e2m1_encode.restype = ctypes.c_uint8
        for f in ("orc_bf16_encode", "orc_fp16_encode", "orc_ue4m3_encode", "orc_e2m1_encode"):
            getattr(_lib, f).argtypes = [ctypes.c_float]
        _lib.orc_bf16_decode.argtypes = [ctypes.c_uint16]
        _lib.orc_fp16_decode.argtypes = [ctypes.c_uint16]
        _lib.orc_ue4m3_decode.argtypes = [ctypes.c_uint8]
        _lib.orc_e2m1_decode.argtypes = [ctypes.c_uint8]
    return _lib


def num_threads() -> int:
    return int(lib().orc_num_threads())


def _p(a, dtype):
    """Pointer to a C-contiguous numpy array of the given dtype (None -> NULL)."""
    if a is None:
        return None
    assert isinstance(a, np.ndarray) and a.dtype == dtype and a.flags["C_CONTIGUOUS"], (a.dtype, dtype)
    return a.ctypes.data_as(ctypes.c_void_p)


def _c(a, dtype):
    return None if a is None else np.ascontiguousarray(a, dtype=dtype)


def _check(rc, name):
    if rc != 0:
        raise ValueError(f"{name}: invalid arguments (code {rc})")


# ---- scalar codecs -------------------------------------------------------------------------

def bf16_encode(x: float) -> int: return int(lib().orc_bf16_encode(float(x)))
def bf16_decode(h: int) -> float: return float(lib().orc_bf16_decode(int(h)))
def fp16_encode(x: float) -> int: return int(lib().orc_fp16_encode(float(x)))
def fp16_decode(h: int) -> float: return float(lib().orc_fp16_decode(int(h)))
def ue4m3_encode(x: float) -> int: return int(lib().orc_ue4m3_encode(float(x)))
def ue4m3_decode(b: int) -> float: return float(lib().orc_ue4m3_decode(int(b)))
def e2m1_encode(x: float) -> int: return int(lib().orc_e2m1_encode(float(x)))
def e2m1_decode(c: int) -> float: return float(lib().orc_e2m1_decode(int(c)))


# ---- offline pack --------------------------------------------------------------------------

def pack_int4(W, d, G):
    """Fold D into W and quantise to INT4 per (row, group of G).  Returns dict with
    qw int8 [N,K], packed uint8 [N,K/2], scales uint16(fp16) [N,K/G], dinv float32 [K]."""
    W = _c(W, np.float32)
    N, K = W.shape
    d = _c(d, np.float32)
    qw = np.empty((N, K), np.int8)
    packed = np.empty((N, K // 2), np.uint8)
    scales = np.empty((N, K // G), np.uint16)
    dinv = np.empty(K, np.float32)
    _check(lib().orc_pack_int4(_p(W, np.float32), _p(d, np.float32), N, K, G, _p(qw, np.int8),
                               _p(packed, np.uint8), _p(scales, np.uint16), _p(dinv, np.float32)),
           "orc_pack_int4")
    return dict(qw=qw, packed=packed, scales=scales, dinv=dinv, N=N, K=K, G=G)


def pack_nvfp4(W, d):
    """NVFP4 pack: e2m1 uint8 [N,K] (one code per byte), packed [N,K/2], sb uint8 [N,K/16],
    dinv [K], tensor_scale float."""
    W = _c(W, np.float32)
    N, K = W.shape
    d = _c(d, np.float32)
    e2m1 = np.empty((N, K), np.uint8)
    packed = np.empty((N, K // 2), np.uint8)
    sb = np.empty((N, K // 16), np.uint8)
    dinv = np.empty(K, np.float32)
    ts = ctypes.c_float(0.0)
    _check(lib().orc_pack_nvfp4(_p(W, np.float32), _p(d, np.float32), N, K, _p(e2m1, np.uint8),
                                _p(packed, np.uint8), _p(sb, np.uint8), _p(dinv, np.float32),
                                ctypes.byref(ts)), "orc_pack_nvfp4")
    return dict(e2m1=e2m1, packed=packed, sb=sb, dinv=dinv, tensor_scale=float(ts.value), N=N, K=K)


# ---- activation prologue -------------------------------------------------------------------

def _table_args(gamma, clip, seg_offsets, seg_stream):
    gamma = _c(gamma, np.float32)
    assert gamma.ndim == 2
    T, S = gamma.shape
    clip = _c(clip, np.float32)
    so = _c(seg_offsets, np.int32)
    ss = _c(seg_stream, np.int32)
    assert so.shape[0] == ss.shape[0] + 1
    return gamma, clip, T, S, so, ss, int(ss.shape[0])


def quantize_int(X, dinv, gamma, clip, step, mode, seg_offsets, seg_stream, qmax, rows=None):
    """X: uint16 (bf16 bits) [M,K].  Returns (codes int8 [R,K], r float32 [R])."""
    X = _c(X, np.uint16)
    M, K = X.shape
    dinv = _c(dinv, np.float32)
    gamma, clip, T, S, so, ss, n_seg = _table_args(gamma, clip, seg_offsets, seg_stream)
    rows = _c(rows, np.int32)
    R = M if rows is None else int(rows.shape[0])
    codes = np.empty((R, K), np.int8)
    r = np.empty(R, np.float32)
    _check(lib().orc_quantize_int(_p(X, np.uint16), ctypes.c_int64(K), M, K, _p(dinv, np.float32),
                                  _p(gamma, np.float32), _p(clip, np.float32), T, S, int(step), int(mode),
                                  _p(so, np.int32), _p(ss, np.int32), n_seg, int(qmax),
                                  _p(rows, np.int32), R, _p(codes, np.int8), _p(r, np.float32)),
           "orc_quantize_int")
    return codes, r


def quantize_nvfp4(X, dinv, gamma, clip, step, mode, seg_offsets, seg_stream, rows=None):
    """Returns (e2m1 uint8 [R,K] one code per byte, sb uint8 [R,K/16], r float32 [R])."""
    X = _c(X, np.uint16)
    M, K = X.shape
    dinv = _c(dinv, np.float32)
    gamma, clip, T, S, so, ss, n_seg = _table_args(gamma, clip, seg_offsets, seg_stream)
    rows = _c(rows, np.int32)
    R = M if rows is None else int(rows.shape[0])
    e2m1 = np.empty((R, K), np.uint8)
    sb = np.empty((R, K // 16), np.uint8)
    r = np.empty(R, np.float32)
    _check(lib().orc_quantize_nvfp4(_p(X, np.uint16), ctypes.c_int64(K), M, K, _p(dinv, np.float32),
                                    _p(gamma, np.float32), _p(clip, np.float32), T, S, int(step), int(mode),
                                    _p(so, np.int32), _p(ss, np.int32), n_seg,
                                    _p(rows, np.int32), R, _p(e2m1, np.uint8), _p(sb, np.uint8),
                                    _p(r, np.float32)), "orc_quantize_nvfp4")
    return e2m1, sb, r


# ---- contraction + epilogue ----------------------------------------------------------------

def accumulate_int(codes, qw, G):
    """Per-group INT32 accumulators, int32 [K/G, R, N]."""
    codes = _c(codes, np.int8)
    qw = _c(qw, np.int8)
    R, K = codes.shape
    N = qw.shape[0]
    acc = np.empty((K // G, R, N), np.int32)
    _check(lib().orc_accumulate_int(_p(codes, np.int8), R, _p(qw, np.int8), N, K, G, _p(acc, np.int32)),
           "orc_accumulate_int")
    return acc


def linear_int(codes, r, qw, scales, G, bias=None):
    """Returns (y uint16(bf16) [R,N], y64 float64 [R,N])."""
    codes = _c(codes, np.int8)
    qw = _c(qw, np.int8)
    scales = _c(scales, np.uint16)
    r = _c(r, np.float32)
    bias = _c(bias, np.float32)
    R, K = codes.shape
    N = qw.shape[0]
    y = np.empty((R, N), np.uint16)
    y64 = np.empty((R, N), np.float64)
    _check(lib().orc_linear_int(_p(codes, np.int8), _p(r, np.float32), R, _p(qw, np.int8),
                                _p(scales, np.uint16), N, K, G, _p(bias, np.float32),
                                _p(y, np.uint16), _p(y64, np.float64)), "orc_linear_int")
    return y, y64


def linear_nvfp4(a_e2m1, a_sb, r, w_e2m1, w_sb, tensor_scale, bias=None):
    a_e2m1 = _c(a_e2m1, np.uint8)
    a_sb = _c(a_sb, np.uint8)
    w_e2m1 = _c(w_e2m1, np.uint8)
    w_sb = _c(w_sb, np.uint8)
    r = _c(r, np.float32)
    bias = _c(bias, np.float32)
    R, K = a_e2m1.shape
    N = w_e2m1.shape[0]
    y = np.empty((R, N), np.uint16)
    y64 = np.empty((R, N), np.float64)
    _check(lib().orc_linear_nvfp4(_p(a_e2m1, np.uint8), _p(a_sb, np.uint8), _p(r, np.float32), R,
                                  _p(w_e2m1, np.uint8), _p(w_sb, np.uint8), ctypes.c_float(tensor_scale),
                                  N, K, _p(bias, np.float32), _p(y, np.uint16), _p(y64, np.float64)),
           "orc_linear_nvfp4")
    return y, y64


# ---- whole linear, as one call (steps in the paper's order) ---------------------------------

def rudder_linear(X, packed_w, gamma, clip, step, mode, seg_offsets, seg_stream, scheme, bias=None,
                  rows=None):
    """One quantized linear: prologue -> contraction -> epilogue.  ``packed_w`` is the dict from
    pack_int4 / pack_nvfp4; scheme in {"w4a8", "w4a4", "nvfp4"}.  Returns dict with the intermediate
    codes / row scales and y (bf16 bits), y64."""
    if scheme in ("w4a8", "w4a4"):
        qmax = 127 if scheme == "w4a8" else 7
        codes, r = quantize_int(X, packed_w["dinv"], gamma, clip, step, mode, seg_offsets, seg_stream,
                                qmax, rows)
        y, y64 = linear_int(codes, r, packed_w["qw"], packed_w["scales"], packed_w["G"], bias)
        return dict(codes=codes, r=r, y=y, y64=y64)
    if scheme == "nvfp4":
        e, sb, r = quantize_nvfp4(X, packed_w["dinv"], gamma, clip, step, mode, seg_offsets, seg_stream,
                                  rows)
        y, y64 = linear_nvfp4(e, sb, r, packed_w["e2m1"], packed_w["sb"], packed_w["tensor_scale"], bias)
        return dict(codes=e, sb=sb, r=r, y=y, y64=y64)
    raise ValueError(scheme)
