"""Seeded synthetic inputs shaped like the workloads of the benchmark configurations.

This module holds NO arithmetic of the method (no quantisation, no scaling of activations by the
method's tables, no packing): it only draws random tensors with the stated distributions, so that
the CPU oracle and the CUDA library can be fed the same bytes.  It imports neither of them.

Recipe (numpy ``default_rng(seed)`` = PCG64, draws in this order, per linear):
  1. X = standard_normal(M, K) as float32
  2. outlier channels: idx = choice(K, max(1, round(p K)), replace=False); X[:, idx] *= f
  3. per segment, in order: m = choice([1.0, 0.5, 2.0]); X[segment] *= m; cast to bf16 (RN)
  4. W = standard_normal(N, K) * 0.02 as float32
  5. d = exp(uniform(ln 0.25, ln 4, K)) as float32          (shared channel scales D)
  6. gamma = exp(uniform(ln 0.5, ln 2, (T, S))) as float32   (per-step per-stream gains)
  7. bias = standard_normal(N) * 0.1 as float32
  8. (static-range tests only) clip[t] = 99.9th percentile of |v| at step t -- computed by the
     caller that needs it, from its own arithmetic, not here.
Stream ids: 0 = video, 1 = proprioceptive, 2 = action.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

VIDEO, PROPRIO, ACTION = 0, 1, 2


@dataclass
class LinearInputs:
    """One linear layer's synthetic inputs (host numpy arrays)."""
    M: int
    K: int
    N: int
    T: int
    S: int
    X_bf16: np.ndarray      # uint16 [M, K] bf16 bit patterns
    W: np.ndarray           # float32 [N, K]
    d: np.ndarray           # float32 [K]
    gamma: np.ndarray       # float32 [T, S]
    bias: np.ndarray        # float32 [N]
    seg_offsets: np.ndarray  # int32 [n_seg + 1]
    seg_stream: np.ndarray   # int32 [n_seg]


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even cast through torch (a library conversion, not the method)."""
    import torch
    t = torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32)).to(torch.bfloat16)
    return t.view(torch.int16).numpy().view(np.uint16).copy()


def bf16_bits_to_f32(h: np.ndarray) -> np.ndarray:
    return (h.astype(np.uint32) << 16).view(np.float32)


def segments(parts):
    """parts: list of (rows, stream id) -> (seg_offsets int32, seg_stream int32)."""
    off = [0]
    st = []
    for rows, s in parts:
        off.append(off[-1] + int(rows))
        st.append(int(s))
    return np.asarray(off, np.int32), np.asarray(st, np.int32)


def draw_linear(rng: np.random.Generator, M, K, N, T, S, seg_offsets, seg_stream,
                outlier_frac, outlier_gain) -> LinearInputs:
    X = rng.standard_normal((M, K)).astype(np.float32)
    n_out = max(1, int(round(outlier_frac * K)))
    idx = rng.choice(K, size=n_out, replace=False)
    X[:, idx] *= np.float32(outlier_gain)
    for s in range(len(seg_stream)):
        m = rng.choice([1.0, 0.5, 2.0])
        X[seg_offsets[s]:seg_offsets[s + 1]] *= np.float32(m)
    Xb = f32_to_bf16_bits(X)
    W = (rng.standard_normal((N, K)) * 0.02).astype(np.float32)
    d = np.exp(rng.uniform(np.log(0.25), np.log(4.0), K)).astype(np.float32)
    gamma = np.exp(rng.uniform(np.log(0.5), np.log(2.0), (T, S))).astype(np.float32)
    bias = (rng.standard_normal(N) * 0.1).astype(np.float32)
    return LinearInputs(M, K, N, T, S, Xb, W, d, gamma, bias,
                        np.asarray(seg_offsets, np.int32), np.asarray(seg_stream, np.int32))


@dataclass
class Config:
    name: str
    seed: int
    scheme: str                 # "w4a8" | "w4a4" | "nvfp4"
    group: int                  # weight group size for the integer schemes (ignored for nvfp4)
    T: int
    S: int
    parts: list                 # [(rows, stream)]
    linears: list               # [(name, K, N)]
    outlier_frac: float
    outlier_gain: float
    extra: dict = field(default_factory=dict)

    @property
    def M(self) -> int:
        return sum(r for r, _ in self.parts)

    def ops(self) -> float:
        return sum(2.0 * self.M * K * N for _, K, N in self.linears)

    def draw(self):
        """-> list of LinearInputs, one per linear, in order."""
        rng = np.random.default_rng(self.seed)
        so, ss = segments(self.parts)
        return [draw_linear(rng, self.M, K, N, self.T, self.S, so, ss,
                            self.outlier_frac, self.outlier_gain) for _, K, N in self.linears]


def _block(H, F):
    return [("qkv", H, 3 * H), ("o", H, H), ("up", H, F), ("down", F, H)]


def config(index: int, scheme: str | None = None, M: int | None = None, KN: int | None = None) -> Config:
    """The five benchmark configurations, and (5) the cross-attention key / value workload.  ``scheme`` selects the variant where a configuration
    names several; ``M`` / ``KN`` select the point of the small-M sweep (configuration 4)."""
    if index == 0:
        return Config("cfg0_w4a8_linear_256x1024x1024", 0, scheme or "w4a8", 64, 1, 3,
                      [(192, VIDEO), (16, PROPRIO), (48, ACTION)], [("linear", 1024, 1024)], 0.01, 30.0)
    if index == 1:
        return Config("cfg1_nvfp4_linear_1024x2048x2048", 1, scheme or "nvfp4", 64, 4, 3,
                      [(896, VIDEO), (32, PROPRIO), (96, ACTION)], [("linear", 2048, 2048)], 0.01, 30.0)
    if index == 2:
        return Config("cfg2_w4a8_block_h2048_f8192_m4416", 2, scheme or "w4a8", 64, 10, 3,
                      [(4096, VIDEO), (64, PROPRIO), (256, ACTION)], _block(2048, 8192), 0.005, 50.0)
    if index == 3:
        sch = scheme or "w4a4"
        return Config(f"cfg3_{sch}_block_h3072_f12288_m17536", 3, sch, 64, 10, 3,
                      [(8192, VIDEO), (64, PROPRIO), (512, ACTION)] * 2, _block(3072, 12288), 0.005, 50.0)
    if index == 4:
        m = M or 64
        kn = KN or 4096
        sch = scheme or "w4a8"
        return Config(f"cfg4_{sch}_smallM_m{m}_kn{kn}", 4, sch, 64, 20, 3,
                      [(m // 4, PROPRIO), (m - m // 4, ACTION)], [("linear", kn, kn)], 0.01, 30.0)
    if index == 5:
        # Cross-attention key / value projections: the text conditioning forms ONE global region per projection
        # (a single segment, a single stream), with its own per-step tables.  The paper gives neither the text
        # length nor the widths: 512 text tokens of width 1024 projected to the block width of configuration 2.
        sch = scheme or "w4a8"
        return Config(f"cfg5_{sch}_crossattn_kv_m512_k1024_n2048", 5, sch, 64, 10, 1,
                      [(M or 512, VIDEO)], [("k_proj", 1024, 2048), ("v_proj", 1024, 2048)], 0.01, 30.0)
    raise ValueError(index)


def tiny(seed=0, M=8, K=128, N=64, T=2, S=3, parts=None, outlier_frac=0.02, outlier_gain=30.0):
    """A small seeded case for brute-force checks."""
    rng = np.random.default_rng(seed)
    if parts is None:
        a = (M + 1) // 2
        b = (M - a + 1) // 2
        parts = [p for p in [(a, VIDEO), (b, PROPRIO), (M - a - b, ACTION)] if p[0] > 0]
    so, ss = segments(parts)
    return draw_linear(rng, M, K, N, T, S, so, ss, outlier_frac, outlier_gain)
