"""Shared helpers of the GPU parity tests: run the same seeded inputs through the CPU oracle and the
CUDA library (through its C ABI) and compare."""
from __future__ import annotations

import numpy as np
import torch

import oracle
import workloads as wl

# Tolerance of the BF16 outputs against the oracle's fp64 evaluation (integer schemes):
# |y - y64| <= ABS + REL * |y64| elementwise.  NVFP4 uses REL_FP4.
ABS_TOL = 2e-2
REL_TOL = 1e-2
REL_TOL_FP4 = 2e-2


def dev():
    return torch.device("cuda", 0)


def to_dev_bf16(bits: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(bits.view(np.int16)).to(dev()).view(torch.bfloat16)


def bf16_to_np(t: torch.Tensor) -> np.ndarray:
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def static_clip(inp, dinv, q=99.9):
    X = wl.bf16_bits_to_f32(inp.X_bf16)
    row_stream = np.repeat(inp.seg_stream, np.diff(inp.seg_offsets))
    clip = np.empty(inp.T, np.float32)
    for t in range(inp.T):
        v = (X * dinv[None, :]) * inp.gamma[t, row_stream][:, None]
        clip[t] = np.percentile(np.abs(v), q)
    return clip


class GpuLinear:
    """One linear layer resident on the GPU, built from a LinearInputs."""

    def __init__(self, rd, inp, scheme: str, group: int, mode=0, clip=None):
        self.rd, self.inp, self.scheme, self.group, self.mode = rd, inp, scheme, group, mode
        d = dev()
        self.W = torch.from_numpy(inp.W).to(d)
        self.d = torch.from_numpy(inp.d).to(d)
        self.X = to_dev_bf16(inp.X_bf16)
        self.bias = torch.from_numpy(inp.bias).to(d)
        self.gamma = torch.from_numpy(inp.gamma).to(d)
        self.clip_np = clip
        self.clip = torch.from_numpy(clip).to(d) if clip is not None else None
        self.w = rd.rudder_pack_weights(self.W, self.d, rd.SCHEMES[scheme], group)
        self.tab = rd.ScaleTable(self.gamma, self.clip, mode)
        self.seg = rd.Segments(inp.seg_offsets, inp.seg_stream)


def oracle_pack(inp, scheme, group):
    return oracle.pack_nvfp4(inp.W, inp.d) if scheme == "nvfp4" else oracle.pack_int4(inp.W, inp.d, group)


# Tighter gate on top of the stated tolerance: the GPU result is the bf16 rounding (2^-9 relative) of an fp32
# evaluation whose summation order differs from the oracle's fp64 one by a few 2^-24 per term, so it must sit
# within one bf16 ulp (2^-8 relative, doubled for slack) of y64; the absolute term covers results that
# cancel against the bias.  A scale that is off by one ulp of fp16, or a partial sum added twice, fails this
# while passing the stated tolerance.
TIGHT_REL = 2.0 ** -7
TIGHT_ABS = 1e-3


def check_output(y_gpu_bits: np.ndarray, y64: np.ndarray, rel=REL_TOL, abs_=ABS_TOL, tight=True):
    """Elementwise: the stated tolerance |y - y64| <= abs_ + rel |y64|, and (tight) the one-ulp gate above."""
    y = wl.bf16_bits_to_f32(y_gpu_bits).astype(np.float64)
    err = np.abs(y - y64)
    bound = abs_ + rel * np.abs(y64)
    bad = err > bound
    assert not bad.any(), f"{bad.sum()} outputs outside tolerance; worst err {err.max():.4g} at |y64|={np.abs(y64).ravel()[err.argmax()]:.4g}"
    if tight:
        bad = err > TIGHT_ABS + TIGHT_REL * np.abs(y64)
        assert not bad.any(), f"{bad.sum()} outputs beyond one bf16 ulp of the fp64 result; worst err {err.max():.4g}"
    fro = np.linalg.norm(y - y64) / max(np.linalg.norm(y64), 1e-30)
    return fro, err.max()
