"""Toy calibrator of the per-stream gains and the shared threshold of one layer and one denoising
step (Stream-Specific Activation Modulation, Section 4.3, Eq. 9): the producer of one entry of the
layer-step lookup table that `rudder_linear` consumes.

    J(gamma, c) = sum_s omega_s / n_s * || Yhat_s(gamma_s, c) - Xtilde_s What ||_F^2
    s.t.  gamma_min <= gamma_s <= gamma_max,   sum_s n_s log gamma_s = 0

Yhat is the quantized layer itself -- `rudder_linear` in the static-range mode, one call per candidate,
so the search sees exactly the arithmetic of deployment -- and the unquantized reference Xtilde What
is one fp32 matrix product of the transformed activations with the dequantized 4-bit weights (an
offline step: a library GEMM, not part of the hot path).  omega (the map-derived stream weights) is
an input; the Action-Impact Stream Map that produces it is not built here, so the default is uniform.

The paper does not say how the arg-min is searched.  Reading taken: coordinate search over candidate
lists -- start at gamma = 1 with the best threshold of `c_candidates`; per sweep, for each stream in
turn try gamma_s * m for every m in `gamma_steps`, rescale the whole vector onto the constraint, skip
candidates outside the bounds, keep the best; then choose the threshold again.  Integer schemes only.
"""
from __future__ import annotations

import math

import torch

from . import (RANGE_STATIC, W4A4_NVFP4, ScaleTable, Segments, Weight, rudder_linear, rudder_linear_workspace_bytes,
               rudder_weight_export)


def dequantized_weights(w: Weight) -> torch.Tensor:
    """What [N, K] fp32 on the device: 4-bit codes (two's complement nibbles, low nibble = even channel)
    times the fp16 scale of their group."""
    if w.scheme == W4A4_NVFP4:
        raise NotImplementedError("the toy calibrator handles the integer schemes")
    ex = rudder_weight_export(w)
    codes = ex["codes"].to(torch.int16)                                  # [N, K/2]
    lo, hi = codes & 0xF, (codes >> 4) & 0xF
    q = torch.stack([lo, hi], dim=2).reshape(w.N, w.K)
    q = torch.where(q >= 8, q - 16, q).to(torch.float32)
    return q * ex["scales"].to(torch.float32).repeat_interleave(w.group, dim=1)


def _project(gamma: list[float], n: list[int]) -> list[float]:
    shift = sum(ns * math.log(g) for g, ns in zip(gamma, n)) / float(sum(n))
    return [g * math.exp(-shift) for g in gamma]


def calibrate_step(w: Weight, X: torch.Tensor, seg: Segments, n_streams: int, c_candidates, gamma_steps,
                   omega=None, gamma_bounds=(0.5, 2.0), sweeps: int = 2):
    """Returns dict(gamma=[S floats], clip=float, objective=float, evaluations=int).
    X bf16 [M, K] on the device; `seg` the row -> stream map of those rows."""
    S = int(n_streams)
    M = X.shape[0]
    dev = X.device
    omega = [1.0] * S if omega is None else [float(v) for v in omega]
    row_stream = torch.empty(M, dtype=torch.int64)
    for a, b, s in zip(seg.off[:-1], seg.off[1:], seg.st):
        row_stream[int(a):int(b)] = int(s)
    n = [int((row_stream == s).sum()) for s in range(S)]
    row_stream = row_stream.to(dev)
    # weight of each row's squared error: omega_s / n_s of its stream
    row_w = torch.tensor([omega[s] / n[s] if n[s] else 0.0 for s in range(S)], dtype=torch.float64, device=dev)[row_stream]

    ex = rudder_weight_export(w)
    y_ref = (X.to(torch.float32) * ex["dinv"][None, :]) @ dequantized_weights(w).t()
    Y = torch.empty((M, w.N), dtype=torch.bfloat16, device=dev)
    ws = torch.empty(rudder_linear_workspace_bytes(w, M) + 256, dtype=torch.uint8, device=dev)
    g_dev = torch.ones((1, S), dtype=torch.float32, device=dev)
    c_dev = torch.ones(1, dtype=torch.float32, device=dev)
    tab = ScaleTable(g_dev, c_dev, RANGE_STATIC)

    def J(gamma, c):
        g_dev.copy_(torch.tensor([gamma], dtype=torch.float32))
        c_dev.fill_(float(c))
        rudder_linear(w, X, seg, 0, tab, None, Y=Y, workspace=ws)
        err2 = ((Y.to(torch.float32) - y_ref).to(torch.float64) ** 2).sum(dim=1)
        return float((err2 * row_w).sum())

    gamma = [1.0] * S
    clip, best = None, math.inf
    for cc in c_candidates:
        v = J(gamma, cc)
        if v < best:
            clip, best = float(cc), v
    evals = len(c_candidates)
    for _ in range(sweeps):
        for s in range(S):
            if n[s] == 0:
                continue
            for m in gamma_steps:
                cand = list(gamma)
                cand[s] *= float(m)
                cand = _project(cand, n)
                if min(cand) < gamma_bounds[0] or max(cand) > gamma_bounds[1]:
                    continue
                v = J(cand, clip)
                evals += 1
                if v < best:
                    gamma, best = cand, v
        for cc in c_candidates:
            v = J(gamma, cc)
            evals += 1
            if v < best:
                clip, best = float(cc), v
    return dict(gamma=gamma, clip=clip, objective=best, evaluations=evals)
