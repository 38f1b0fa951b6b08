"""GPU parity of the NVFP4 W4A4 path against the CPU oracle, through the C ABI: packed E2M1 codes,
UE4M3 block scales, tensor scale and row scales bit-exact; BF16 outputs within max relative error
2e-2 plus absolute error 2e-2 of the oracle's fp64 evaluation (the tensor core's fp32 accumulation
order is not specified, so the accumulators themselves are not compared)."""
import numpy as np
import pytest
import torch

import oracle
import workloads as wl
from helpers import ABS_TOL, REL_TOL_FP4, GpuLinear, bf16_to_np, check_output, static_clip

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def rd():
    import paper_2609_39056_b200 as rd
    rd.lib()
    return rd


def _assert_clean(rd):
    last, where = rd.rudder_device_status()
    assert last == 0, f"device status {last} (wait code {where})"


def _pack_codes(e2m1):
    return (e2m1[:, 0::2] | (e2m1[:, 1::2] << 4)).astype(np.uint8)


@pytest.mark.parametrize("N,K", [(64, 256), (128, 512), (320, 1024), (256, 2048)])
def test_pack_export_bit_exact(rd, N, K):
    inp = wl.tiny(seed=400 + N, M=4, K=K, N=N)
    ref = oracle.pack_nvfp4(inp.W, inp.d)
    g = GpuLinear(rd, inp, "nvfp4", 16)
    ex = rd.rudder_weight_export(g.w)
    assert np.array_equal(ex["codes"].cpu().numpy(), ref["packed"])
    assert np.array_equal(ex["scales"].cpu().numpy(), ref["sb"])
    assert np.array_equal(ex["dinv"].cpu().numpy().view(np.uint32), ref["dinv"].view(np.uint32))
    assert np.float32(ex["tensor_scale"].item()).view(np.uint32) == np.float32(ref["tensor_scale"]).view(np.uint32)
    _assert_clean(rd)


def test_pack_degenerate_weights(rd):
    """Zero row, zero block, a block of tiny negative weights whose scale rounds to zero, one dominant weight."""
    inp = wl.tiny(seed=431, M=4, K=512, N=64)
    inp.W[5, :] = 0.0
    inp.W[3, 16:32] = 0.0
    inp.W[7, 32:48] = -1e-9
    inp.W[9, 100] = 3.0
    ref = oracle.pack_nvfp4(inp.W, inp.d)
    g = GpuLinear(rd, inp, "nvfp4", 16)
    ex = rd.rudder_weight_export(g.w)
    assert np.array_equal(ex["scales"].cpu().numpy(), ref["sb"])
    assert np.array_equal(ex["codes"].cpu().numpy(), ref["packed"])
    _assert_clean(rd)


@pytest.mark.parametrize("mode", [0, 1])
@pytest.mark.parametrize("M,K", [(1, 256), (37, 512), (130, 1024), (64, 2048), (19, 4096), (9, 8192), (5, 12288),
                                 (300, 3072), (3, 16640)])   # many rows per CTA; rows too long to stage (warp-per-row kernel)
def test_activation_codes_bit_exact(rd, mode, M, K):
    inp = wl.tiny(seed=500 + M, M=M, K=K, N=64, T=3)
    ref_w = oracle.pack_nvfp4(inp.W, inp.d)
    clip = static_clip(inp, ref_w["dinv"]) if mode == 1 else None
    g = GpuLinear(rd, inp, "nvfp4", 16, mode, clip)
    for step in (0, 2):
        codes, sb, r = rd.rudder_quantize_activations(g.w, g.X, g.seg, step, g.tab)
        re, rsb, rr = oracle.quantize_nvfp4(inp.X_bf16, ref_w["dinv"], inp.gamma, clip, step, mode, inp.seg_offsets,
                                            inp.seg_stream)
        assert np.array_equal(sb.cpu().numpy(), rsb), "block scales differ"
        assert np.array_equal(codes.cpu().numpy(), _pack_codes(re)), "E2M1 codes differ"
        assert np.array_equal(r.cpu().numpy().view(np.uint32), rr.view(np.uint32))
    _assert_clean(rd)


@pytest.mark.parametrize("mode", [0, 1])
def test_activation_degenerate_rows(rd, mode):
    """Zero row, one non-zero element, an all-zero 16-channel block, one huge outlier among tiny values,
    values at the bottom of the bf16 range, equal magnitudes (every rounding tie the formats have)."""
    K = 512
    inp = wl.tiny(seed=577, M=8, K=K, N=64, T=2)
    X = wl.bf16_bits_to_f32(inp.X_bf16).copy()
    X[0, :] = 0.0
    X[1, :] = 0.0; X[1, 77] = -3.5
    X[2, 32:48] = 0.0
    X[3, :] *= 1e-3; X[3, 5] = 1.0e4
    X[4, :] *= 1e-30
    X[5, :] = np.where(np.arange(K) % 2 == 0, 1.0, -1.0)
    X[6, :] = np.tile(np.array([0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0, 6.0], np.float32), K // 8)   # E2M1 midpoints before scaling
    inp.X_bf16[:] = wl.f32_to_bf16_bits(X)
    ref_w = oracle.pack_nvfp4(inp.W, inp.d)
    clip = static_clip(inp, ref_w["dinv"]) if mode == 1 else None
    g = GpuLinear(rd, inp, "nvfp4", 16, mode, clip)
    for step in (0, 1):
        codes, sb, r = rd.rudder_quantize_activations(g.w, g.X, g.seg, step, g.tab)
        re, rsb, rr = oracle.quantize_nvfp4(inp.X_bf16, ref_w["dinv"], inp.gamma, clip, step, mode, inp.seg_offsets,
                                            inp.seg_stream)
        assert np.array_equal(sb.cpu().numpy(), rsb), "block scales differ"
        assert np.array_equal(codes.cpu().numpy(), _pack_codes(re)), "E2M1 codes differ"
        assert np.array_equal(r.cpu().numpy().view(np.uint32), rr.view(np.uint32))
    # and through the GEMM: the zero row gives the bias, nothing is NaN
    Y = rd.rudder_linear(g.w, g.X, g.seg, 0, g.tab, g.bias)
    out = oracle.rudder_linear(inp.X_bf16, ref_w, inp.gamma, clip, 0, mode, inp.seg_offsets, inp.seg_stream, "nvfp4", inp.bias)
    check_output(bf16_to_np(Y), out["y64"], rel=REL_TOL_FP4, abs_=ABS_TOL)
    _assert_clean(rd)


CASES = [
    # M, K, N
    (8, 256, 64),          # one stage, narrow channel tile
    (128, 512, 128),
    (130, 768, 256),       # ragged token tail, wide token tile, odd stage count
    (200, 1024, 320),      # ragged channel tile
    (300, 512, 128),       # last token tile owns a single 128-row scale atom
    (33, 2304, 256),       # 9 stages: the ring wraps
    (513, 1024, 256),
    # M >= 1024 with whole 256-channel tiles: the CTA-pair kernel
    (1024, 256, 256),      # one stage
    (1100, 768, 256),      # ragged token tail (last tile owns one scale atom), fewer stages than ring slots
    (1300, 2304, 512),     # two channel-pair tiles, the ring wraps
    (1030, 512, 320),      # 320 channels: not whole pair tiles -> single-CTA kernel at large M
]


@pytest.mark.parametrize("M,K,N", CASES)
@pytest.mark.parametrize("mode", [0, 1])
def test_linear_output(rd, M, K, N, mode):
    inp = wl.tiny(seed=600 + M + N, M=M, K=K, N=N, T=2)
    ref_w = oracle.pack_nvfp4(inp.W, inp.d)
    clip = static_clip(inp, ref_w["dinv"]) if mode == 1 else None
    g = GpuLinear(rd, inp, "nvfp4", 16, mode, clip)
    Y = rd.rudder_linear(g.w, g.X, g.seg, 1, g.tab, g.bias)
    out = oracle.rudder_linear(inp.X_bf16, ref_w, inp.gamma, clip, 1, mode, inp.seg_offsets, inp.seg_stream, "nvfp4",
                               inp.bias)
    check_output(bf16_to_np(Y), out["y64"], rel=REL_TOL_FP4, abs_=ABS_TOL)
    # tighter: fp32 accumulation of exactly representable products -> a few bf16 ulps at most
    y = wl.bf16_bits_to_f32(bf16_to_np(Y)).astype(np.float64)
    assert np.all(np.abs(y - out["y64"]) <= 2.0 ** -7 * np.abs(out["y64"]) + 1e-3)
    _assert_clean(rd)


def test_config1_all_steps(rd):
    """Configuration 1: M = 1024 (896 video / 32 proprio / 96 action), K = N = 2048, NVFP4, 4 steps."""
    cfg = wl.config(1)
    inp = cfg.draw()[0]
    ref_w = oracle.pack_nvfp4(inp.W, inp.d)
    g = GpuLinear(rd, inp, "nvfp4", 16)
    for step in range(cfg.T):
        Y = rd.rudder_linear(g.w, g.X, g.seg, step, g.tab, g.bias)
        out = oracle.rudder_linear(inp.X_bf16, ref_w, inp.gamma, None, step, 0, inp.seg_offsets, inp.seg_stream,
                                   "nvfp4", inp.bias)
        codes, sb, r = rd.rudder_quantize_activations(g.w, g.X, g.seg, step, g.tab)
        assert np.array_equal(codes.cpu().numpy(), _pack_codes(out["codes"]))
        assert np.array_equal(sb.cpu().numpy(), out["sb"])
        assert np.array_equal(r.cpu().numpy(), out["r"])
        fro, worst = check_output(bf16_to_np(Y), out["y64"], rel=REL_TOL_FP4, abs_=ABS_TOL)
        assert fro < 5e-3
    _assert_clean(rd)


def test_nvfp4_rejects_unsupported(rd):
    W = torch.randn(64, 384, device="cuda")
    with pytest.raises(rd.RudderError) as e:
        rd.rudder_pack_weights(W, None, rd.W4A4_NVFP4, 16)      # K % 256 != 0
    assert e.value.status == rd.ERR_SHAPE
