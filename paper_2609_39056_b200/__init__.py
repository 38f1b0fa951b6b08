"""Python binding of the Rudder C-ABI library (``include/rudder.h``): argument marshalling only.

Every step of the quantized linear runs in the CUDA kernels behind the C ABI; torch is used for
device memory and streams.  There is no CPU fallback: if ``librudder.so`` is missing or cannot be
loaded, every call raises.
"""
from __future__ import annotations

import ctypes
from pathlib import Path

import numpy as np
import torch

_HERE = Path(__file__).resolve().parent
LIB_PATH = _HERE / "librudder.so"

# enums of rudder.h
OK, ERR_ARG, ERR_SHAPE, ERR_ALIGN, ERR_UNSUPPORTED, ERR_WORKSPACE, ERR_CUDA, ERR_TIMEOUT = range(8)
W4A8_INT, W4A4_INT, W4A4_NVFP4 = 0, 1, 2
RANGE_PER_TOKEN, RANGE_STATIC = 0, 1
SCHEMES = {"w4a8": W4A8_INT, "w4a4": W4A4_INT, "nvfp4": W4A4_NVFP4}

EXPORTED = [
    "rudder_pack_weights", "rudder_weight_free", "rudder_weight_info", "rudder_weight_export", "rudder_weight_import",
    "rudder_linear_workspace_bytes", "rudder_linear", "rudder_block_workspace_bytes", "rudder_block",
    "rudder_linear_static_max_workspace_bytes", "rudder_linear_static",
    "rudder_block_profile", "rudder_block_host_staging_bytes", "rudder_block_host",
    "rudder_quantize_activations", "rudder_linear_dump_acc", "rudder_device_status", "rudder_status_string",
    "rudder_gelu", "rudder_selftest_wait_timeout", "rudder_rmsnorm", "rudder_add",
    "rudder_block_dit", "rudder_block_dit_workspace_bytes", "rudder_gelu_quantize_activations",
]


class RudderError(RuntimeError):
    def __init__(self, status: int, what: str):
        self.status = status
        super().__init__(f"{what}: {status_string(status)} (status {status})")


class _ScaleTable(ctypes.Structure):
    _fields_ = [("gamma", ctypes.c_void_p), ("clip", ctypes.c_void_p), ("T", ctypes.c_int), ("S", ctypes.c_int),
                ("mode", ctypes.c_int)]


class _Segments(ctypes.Structure):
    _fields_ = [("seg_offsets", ctypes.POINTER(ctypes.c_int32)), ("seg_stream", ctypes.POINTER(ctypes.c_int32)),
                ("n_seg", ctypes.c_int)]


class _BlockGlue(ctypes.Structure):
    _fields_ = [("norm1_weight", ctypes.c_void_p), ("norm2_weight", ctypes.c_void_p), ("eps", ctypes.c_float),
                ("out", ctypes.c_void_p), ("ldout", ctypes.c_int64)]


class _BlockArgs(ctypes.Structure):
    _fields_ = [("w", ctypes.c_void_p * 4), ("tab", ctypes.POINTER(_ScaleTable) * 4), ("bias", ctypes.c_void_p * 4),
                ("x", ctypes.c_void_p * 4), ("ldx", ctypes.c_int64 * 4), ("y", ctypes.c_void_p * 4),
                ("ldy", ctypes.c_int64 * 4)]


_lib = None


def lib() -> ctypes.CDLL:
    """The loaded C-ABI library.  Raises if it has not been built (``python -m paper_2609_39056_b200.build``)."""
    global _lib
    if _lib is None:
        if not LIB_PATH.exists():
            raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2609_39056_b200.build` "
                              "(there is no fallback path)")
        L = ctypes.CDLL(str(LIB_PATH))
        vp, i32, i64, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_int64, ctypes.c_size_t
        L.rudder_status_string.restype = ctypes.c_char_p
        L.rudder_status_string.argtypes = [i32]
        L.rudder_pack_weights.argtypes = [vp, vp, i32, i32, i32, i32, vp, ctypes.POINTER(vp)]
        L.rudder_weight_free.argtypes = [vp]
        L.rudder_weight_info.argtypes = [vp, ctypes.POINTER(i32), ctypes.POINTER(i32), ctypes.POINTER(i32),
                                         ctypes.POINTER(i32), ctypes.POINTER(sz)]
        L.rudder_weight_export.argtypes = [vp, vp, vp, vp, vp, vp]
        L.rudder_weight_import.argtypes = [vp, vp, vp, vp, i32, i32, i32, i32, vp, ctypes.POINTER(vp)]
        L.rudder_linear_workspace_bytes.restype = sz
        L.rudder_linear_workspace_bytes.argtypes = [vp, i32]
        L.rudder_linear.argtypes = [vp, vp, i64, i32, ctypes.POINTER(_Segments), i32, ctypes.POINTER(_ScaleTable),
                                    vp, vp, i64, vp, sz, vp]
        L.rudder_linear_static_max_workspace_bytes.restype = sz
        L.rudder_linear_static_max_workspace_bytes.argtypes = []
        L.rudder_linear_static.argtypes = [vp, vp, i64, i32, ctypes.POINTER(_Segments), i32, ctypes.POINTER(_ScaleTable),
                                           vp, vp, i64, vp]
        L.rudder_block_workspace_bytes.restype = sz
        L.rudder_block_workspace_bytes.argtypes = [ctypes.POINTER(_BlockArgs), i32]
        L.rudder_block.argtypes = [ctypes.POINTER(_BlockArgs), i32, ctypes.POINTER(_Segments), i32, vp, sz, vp]
        L.rudder_block_profile.argtypes = [ctypes.POINTER(_BlockArgs), i32, ctypes.POINTER(_Segments), i32, vp, sz, vp,
                                           ctypes.POINTER(ctypes.c_float)]
        L.rudder_block_host_staging_bytes.restype = sz
        L.rudder_block_host_staging_bytes.argtypes = [ctypes.POINTER(_BlockArgs), i32]
        L.rudder_block_host.argtypes = [ctypes.POINTER(_BlockArgs), i32, ctypes.POINTER(_Segments), i32, vp, sz, vp, sz, vp]
        L.rudder_quantize_activations.argtypes = [vp, vp, i64, i32, ctypes.POINTER(_Segments), i32,
                                                  ctypes.POINTER(_ScaleTable), vp, vp, vp, vp]
        L.rudder_gelu_quantize_activations.argtypes = [vp, vp, i64, i32, ctypes.POINTER(_Segments), i32,
                                                       ctypes.POINTER(_ScaleTable), vp, vp, vp]
        L.rudder_linear_dump_acc.argtypes = [vp, vp, i64, i32, ctypes.POINTER(_Segments), i32,
                                             ctypes.POINTER(_ScaleTable), vp, vp, i64, vp, sz, vp,
                                             i32, i32, i32, i32, vp]
        L.rudder_device_status.argtypes = [ctypes.POINTER(i32), ctypes.POINTER(i32)]
        L.rudder_gelu.argtypes = [vp, i64, i32, i32, vp, i64, vp]
        L.rudder_selftest_wait_timeout.argtypes = [ctypes.c_longlong, vp]
        L.rudder_rmsnorm.argtypes = [vp, i64, i32, i32, vp, ctypes.c_float, vp, i64, vp]
        L.rudder_add.argtypes = [vp, i64, vp, i64, i32, i32, vp, i64, vp]
        L.rudder_block_dit_workspace_bytes.restype = sz
        L.rudder_block_dit_workspace_bytes.argtypes = [ctypes.POINTER(_BlockArgs), i32]
        L.rudder_block_dit.argtypes = [ctypes.POINTER(_BlockArgs), ctypes.POINTER(_BlockGlue), i32, ctypes.POINTER(_Segments), i32, vp, sz, vp]
        _lib = L
    return _lib


def status_string(status: int) -> str:
    return lib().rudder_status_string(int(status)).decode()


def _check(status: int, what: str):
    if status != OK:
        raise RudderError(status, what)


def _ptr(t):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream(stream):
    s = torch.cuda.current_stream() if stream is None else stream
    return ctypes.c_void_p(s.cuda_stream)


class Weight:
    """Owner of a ``rudder_weight*``; frees it when collected."""

    def __init__(self, handle, N, K, group, scheme, device_bytes):
        self.handle, self.N, self.K, self.group, self.scheme, self.device_bytes = handle, N, K, group, scheme, device_bytes

    def free(self):
        if self.handle:
            lib().rudder_weight_free(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.free()
        except Exception:
            pass


class ScaleTable:
    """Layer-step lookup table: gamma [T,S] fp32 (device), clip [T] fp32 (device) or None."""

    def __init__(self, gamma: torch.Tensor, clip: torch.Tensor | None = None, mode: int = RANGE_PER_TOKEN):
        assert gamma.dtype == torch.float32 and gamma.dim() == 2 and gamma.is_contiguous()
        assert clip is None or (clip.dtype == torch.float32 and clip.is_contiguous())
        self.gamma, self.clip, self.mode = gamma, clip, mode
        self.c = _ScaleTable(gamma.data_ptr(), clip.data_ptr() if clip is not None else None,
                             gamma.shape[0], gamma.shape[1], mode)


class Segments:
    """Row -> stream map: host arrays seg_offsets [n_seg+1], seg_stream [n_seg]."""

    def __init__(self, seg_offsets, seg_stream):
        self.off = np.ascontiguousarray(seg_offsets, dtype=np.int32)
        self.st = np.ascontiguousarray(seg_stream, dtype=np.int32)
        self.c = _Segments(self.off.ctypes.data_as(ctypes.POINTER(ctypes.c_int32)),
                           self.st.ctypes.data_as(ctypes.POINTER(ctypes.c_int32)), int(self.st.shape[0]))


def rudder_pack_weights(W: torch.Tensor, d: torch.Tensor | None, scheme: int, group: int, stream=None) -> Weight:
    assert W.is_cuda and W.dtype == torch.float32 and W.dim() == 2 and W.is_contiguous()
    assert d is None or (d.is_cuda and d.dtype == torch.float32 and d.is_contiguous())
    N, K = W.shape
    out = ctypes.c_void_p()
    _check(lib().rudder_pack_weights(_ptr(W), _ptr(d), N, K, int(scheme), int(group), _stream(stream),
                                     ctypes.byref(out)), "rudder_pack_weights")
    n, k, g, s, b = ctypes.c_int(), ctypes.c_int(), ctypes.c_int(), ctypes.c_int(), ctypes.c_size_t()
    _check(lib().rudder_weight_info(out, ctypes.byref(n), ctypes.byref(k), ctypes.byref(g), ctypes.byref(s),
                                    ctypes.byref(b)), "rudder_weight_info")
    return Weight(out, n.value, k.value, g.value, s.value, b.value)


def rudder_weight_export(w: Weight, stream=None):
    """Canonical view: codes uint8 [N,K/2], scales (int16 view of fp16 [N,K/G] | uint8 [N,K/16]), dinv, tensor_scale."""
    dev = torch.device("cuda", torch.cuda.current_device())
    codes = torch.empty((w.N, w.K // 2), dtype=torch.uint8, device=dev)
    if w.scheme == W4A4_NVFP4:
        scales = torch.empty((w.N, w.K // 16), dtype=torch.uint8, device=dev)
    else:
        scales = torch.empty((w.N, w.K // w.group), dtype=torch.float16, device=dev)
    dinv = torch.empty(w.K, dtype=torch.float32, device=dev)
    ts = torch.empty(1, dtype=torch.float32, device=dev)
    _check(lib().rudder_weight_export(w.handle, _ptr(codes), _ptr(scales), _ptr(dinv), _ptr(ts), _stream(stream)),
           "rudder_weight_export")
    return dict(codes=codes, scales=scales, dinv=dinv, tensor_scale=ts)


def rudder_weight_import(ex: dict, N: int, K: int, scheme: int, group: int, stream=None) -> Weight:
    """Packed weight from its canonical view (the dict rudder_weight_export returns)."""
    out = ctypes.c_void_p()
    _check(lib().rudder_weight_import(_ptr(ex["codes"]), _ptr(ex["scales"]), _ptr(ex["dinv"]), _ptr(ex.get("tensor_scale")),
                                      int(N), int(K), int(scheme), int(group), _stream(stream), ctypes.byref(out)),
           "rudder_weight_import")
    n, k, g, s, b = ctypes.c_int(), ctypes.c_int(), ctypes.c_int(), ctypes.c_int(), ctypes.c_size_t()
    _check(lib().rudder_weight_info(out, ctypes.byref(n), ctypes.byref(k), ctypes.byref(g), ctypes.byref(s),
                                    ctypes.byref(b)), "rudder_weight_info")
    return Weight(out, n.value, k.value, g.value, s.value, b.value)


def rudder_linear_workspace_bytes(w: Weight, M: int) -> int:
    return int(lib().rudder_linear_workspace_bytes(w.handle, int(M)))


def _workspace(nbytes, device, stream=None):
    """Scratch the binding allocates for the caller.  It is dropped when the call returns, while the kernels
    may still be running: torch's caching allocator only hands a freed block to later work of the stream it
    was allocated on, so the block is allocated under the stream the kernels are launched on."""
    if stream is None:
        return torch.empty(nbytes + 256, dtype=torch.uint8, device=device)
    with torch.cuda.stream(stream):
        return torch.empty(nbytes + 256, dtype=torch.uint8, device=device)


def _aligned(ws: torch.Tensor):
    off = (-ws.data_ptr()) % 256
    return ctypes.c_void_p(ws.data_ptr() + off), ws.numel() - off


def rudder_linear(w: Weight, X: torch.Tensor, seg: Segments, step: int, tab: ScaleTable, bias=None, Y=None,
                  workspace=None, stream=None) -> torch.Tensor:
    assert X.is_cuda and X.dtype == torch.bfloat16 and X.dim() == 2 and X.stride(1) == 1
    M = X.shape[0]
    if Y is None:
        Y = torch.empty((M, w.N), dtype=torch.bfloat16, device=X.device)
    if workspace is None:
        workspace = _workspace(rudder_linear_workspace_bytes(w, M), X.device, stream)
    wp, wb = _aligned(workspace)
    _check(lib().rudder_linear(w.handle, _ptr(X), X.stride(0), M, ctypes.byref(seg.c), int(step), ctypes.byref(tab.c),
                               _ptr(bias), _ptr(Y), Y.stride(0), wp, wb, _stream(stream)), "rudder_linear")
    return Y


def rudder_linear_static_max_workspace_bytes() -> int:
    return int(lib().rudder_linear_static_max_workspace_bytes())


def rudder_linear_static(w: Weight, X: torch.Tensor, seg: Segments, step: int, tab: ScaleTable, bias=None, Y=None,
                         stream=None) -> torch.Tensor:
    """rudder_linear for callers that cannot allocate: the scratch between the two kernels is a fixed
    4 MiB array inside the library, so only inputs and the output are passed.  Raises
    RudderError(ERR_WORKSPACE) when the layer needs more scratch than the array holds.  Calls that may
    overlap on the GPU share the array and must be serialised by the caller."""
    assert X.is_cuda and X.dtype == torch.bfloat16 and X.dim() == 2 and X.stride(1) == 1
    M = X.shape[0]
    assert Y is not None, "the caller passes the output buffer: this entry point allocates nothing"
    _check(lib().rudder_linear_static(w.handle, _ptr(X), X.stride(0), M, ctypes.byref(seg.c), int(step),
                                      ctypes.byref(tab.c), _ptr(bias), _ptr(Y), Y.stride(0), _stream(stream)),
           "rudder_linear_static")
    return Y


def rudder_linear_dump_acc(w: Weight, X, seg, step, tab, bias=None, row0=0, rows=None, col0=0, cols=None, stream=None):
    """rudder_linear plus the INT32 group accumulators of a tile -> (Y, acc int32 [K/G, rows, cols])."""
    M = X.shape[0]
    rows = M - row0 if rows is None else rows
    cols = w.N - col0 if cols is None else cols
    Y = torch.empty((M, w.N), dtype=torch.bfloat16, device=X.device)
    acc = torch.full((w.K // w.group, rows, cols), -(2 ** 31), dtype=torch.int32, device=X.device)
    workspace = _workspace(rudder_linear_workspace_bytes(w, M), X.device, stream)
    wp, wb = _aligned(workspace)
    _check(lib().rudder_linear_dump_acc(w.handle, _ptr(X), X.stride(0), M, ctypes.byref(seg.c), int(step),
                                        ctypes.byref(tab.c), _ptr(bias), _ptr(Y), Y.stride(0), wp, wb, _stream(stream),
                                        int(row0), int(rows), int(col0), int(cols), _ptr(acc)),
           "rudder_linear_dump_acc")
    return Y, acc


def rudder_quantize_activations(w: Weight, X, seg, step, tab, stream=None):
    """First kernel alone -> (codes, block_scales | None, row_scale)."""
    M = X.shape[0]
    if w.scheme == W4A4_NVFP4:
        codes = torch.empty((M, w.K // 2), dtype=torch.uint8, device=X.device)
        sb = torch.empty((M, w.K // 16), dtype=torch.uint8, device=X.device)
    else:
        codes = torch.empty((M, w.K), dtype=torch.int8, device=X.device)
        sb = None
    r = torch.empty(M, dtype=torch.float32, device=X.device)
    _check(lib().rudder_quantize_activations(w.handle, _ptr(X), X.stride(0), M, ctypes.byref(seg.c), int(step),
                                             ctypes.byref(tab.c), _ptr(codes), _ptr(sb), _ptr(r), _stream(stream)),
           "rudder_quantize_activations")
    return codes, sb, r


class BlockArgs:
    """Arguments of rudder_block: 4 weights, tables, biases, replay inputs and outputs (QKV, O, up, down)."""

    def __init__(self, weights, tabs, biases, xs, ys):
        self.keep = (weights, tabs, biases, xs, ys)
        c = _BlockArgs()
        for l in range(4):
            c.w[l] = weights[l].handle
            c.tab[l] = ctypes.pointer(tabs[l].c)
            c.bias[l] = biases[l].data_ptr() if biases[l] is not None else None
            c.x[l] = xs[l].data_ptr() if xs[l] is not None else None        # None (l >= 1): chained to the previous output
            c.ldx[l] = xs[l].stride(0) if xs[l] is not None else 0
            c.y[l] = ys[l].data_ptr()
            c.ldy[l] = ys[l].stride(0)
        self.c = c


def rudder_gelu(X: torch.Tensor, Y: torch.Tensor | None = None, stream=None) -> torch.Tensor:
    """Y = bf16(gelu(X)), elementwise, in the bit-defined form the chained block uses."""
    assert X.is_cuda and X.dtype == torch.bfloat16 and X.dim() == 2 and X.stride(1) == 1
    M, N = X.shape
    if Y is None:
        Y = torch.empty((M, N), dtype=torch.bfloat16, device=X.device)
    _check(lib().rudder_gelu(_ptr(X), X.stride(0), int(M), int(N), _ptr(Y), Y.stride(0), _stream(stream)), "rudder_gelu")
    return Y


def rudder_block_workspace_bytes(args: BlockArgs, M: int) -> int:
    return int(lib().rudder_block_workspace_bytes(ctypes.byref(args.c), int(M)))


def rudder_block(args: BlockArgs, M: int, seg: Segments, step: int, workspace: torch.Tensor, stream=None):
    wp, wb = _aligned(workspace)
    _check(lib().rudder_block(ctypes.byref(args.c), int(M), ctypes.byref(seg.c), int(step), wp, wb, _stream(stream)),
           "rudder_block")


def rudder_block_profile(args: BlockArgs, M: int, seg: Segments, step: int, workspace: torch.Tensor, stream=None):
    """rudder_block with an event between kernels -> 8 device times in ms (prologue, GEMM) x (QKV, O, up, down)."""
    wp, wb = _aligned(workspace)
    ms = (ctypes.c_float * 8)()
    _check(lib().rudder_block_profile(ctypes.byref(args.c), int(M), ctypes.byref(seg.c), int(step), wp, wb,
                                      _stream(stream), ms), "rudder_block_profile")
    return [float(v) for v in ms]


def rudder_block_host_staging_bytes(args: BlockArgs, M: int) -> int:
    return int(lib().rudder_block_host_staging_bytes(ctypes.byref(args.c), int(M)))


def rudder_block_host(args: BlockArgs, M: int, seg: Segments, step: int, staging: torch.Tensor,
                      workspace: torch.Tensor, stream=None):
    """rudder_block whose x / y tensors in ``args`` are (pinned) HOST tensors."""
    sp, sb = _aligned(staging)
    wp, wb = _aligned(workspace)
    _check(lib().rudder_block_host(ctypes.byref(args.c), int(M), ctypes.byref(seg.c), int(step), sp, sb, wp, wb,
                                   _stream(stream)), "rudder_block_host")


def rudder_device_status():
    """(last status, code of the wait that gave up); clears the device word.  Synchronises."""
    last, where = ctypes.c_int(), ctypes.c_int()
    _check(lib().rudder_device_status(ctypes.byref(last), ctypes.byref(where)), "rudder_device_status")
    return last.value, where.value


def rudder_selftest_wait_timeout(limit_cycles: int = 1_000_000, stream=None):
    """One warp waits `limit_cycles` SM clocks on a barrier nobody signals, gives up and records the time-out."""
    _check(lib().rudder_selftest_wait_timeout(int(limit_cycles), _stream(stream)), "rudder_selftest_wait_timeout")


def rudder_rmsnorm(X: torch.Tensor, weight: torch.Tensor, eps: float, Y: torch.Tensor | None = None, stream=None) -> torch.Tensor:
    """Y = bf16((x / sqrt(mean(x^2) + eps)) * weight) per row, in the bit-defined form of the DiT block glue."""
    assert X.is_cuda and X.dtype == torch.bfloat16 and X.dim() == 2 and X.stride(1) == 1
    assert weight.is_cuda and weight.dtype == torch.float32 and weight.is_contiguous() and weight.numel() == X.shape[1]
    M, N = X.shape
    if Y is None:
        Y = torch.empty((M, N), dtype=torch.bfloat16, device=X.device)
    _check(lib().rudder_rmsnorm(_ptr(X), X.stride(0), int(M), int(N), _ptr(weight), ctypes.c_float(eps), _ptr(Y), Y.stride(0),
                                _stream(stream)), "rudder_rmsnorm")
    return Y


def rudder_add(A: torch.Tensor, B: torch.Tensor, Y: torch.Tensor | None = None, stream=None) -> torch.Tensor:
    """Y = bf16(A + B), elementwise (the residual addition of the DiT block glue)."""
    assert A.is_cuda and B.is_cuda and A.dtype == B.dtype == torch.bfloat16 and A.shape == B.shape and A.stride(1) == B.stride(1) == 1
    M, N = A.shape
    if Y is None:
        Y = torch.empty((M, N), dtype=torch.bfloat16, device=A.device)
    _check(lib().rudder_add(_ptr(A), A.stride(0), _ptr(B), B.stride(0), int(M), int(N), _ptr(Y), Y.stride(0), _stream(stream)), "rudder_add")
    return Y


def rudder_block_dit_workspace_bytes(args: BlockArgs, M: int) -> int:
    return int(lib().rudder_block_dit_workspace_bytes(ctypes.byref(args.c), int(M)))


def rudder_block_dit(args: BlockArgs, norm1_weight: torch.Tensor, norm2_weight: torch.Tensor, eps: float, out: torch.Tensor, M: int,
                     seg: Segments, step: int, workspace: torch.Tensor, stream=None):
    """One DiT block end to end from args.x[0]: norm -> QKV -> O (V third) -> + x -> norm -> up -> GELU -> down -> + h."""
    glue = _BlockGlue(norm1_weight.data_ptr(), norm2_weight.data_ptr(), float(eps), out.data_ptr(), out.stride(0))
    wp, wb = _aligned(workspace)
    _check(lib().rudder_block_dit(ctypes.byref(args.c), ctypes.byref(glue), int(M), ctypes.byref(seg.c), int(step), wp, wb,
                                  _stream(stream)), "rudder_block_dit")
    return out


def rudder_gelu_quantize_activations(w: Weight, X, seg, step, tab, stream=None):
    """The fused GELU + static-range prologue of a chained layer alone -> (codes int8 [M, K], row_scale)."""
    M = X.shape[0]
    codes = torch.empty((M, w.K), dtype=torch.int8, device=X.device)
    r = torch.empty(M, dtype=torch.float32, device=X.device)
    _check(lib().rudder_gelu_quantize_activations(w.handle, _ptr(X), X.stride(0), M, ctypes.byref(seg.c), int(step),
                                                  ctypes.byref(tab.c), _ptr(codes), _ptr(r), _stream(stream)),
           "rudder_gelu_quantize_activations")
    return codes, r
