"""GPU parity of the integer schemes (W4A8, W4A4-INT) against the CPU oracle, through the C ABI:
pack export, activation codes, row scales and INT32 group accumulators bit-exact; BF16 outputs
within max relative error 1e-2 plus absolute error 2e-2 of the oracle's fp64 evaluation."""
import numpy as np
import pytest
import torch

import oracle
import workloads as wl
from helpers import GpuLinear, bf16_to_np, check_output, oracle_pack, static_clip, to_dev_bf16

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def rd():
    import paper_2609_39056_b200 as rd
    rd.lib()
    return rd


def _assert_clean(rd):
    last, where = rd.rudder_device_status()
    assert last == 0, f"device status {last} (wait code {where})"


@pytest.mark.parametrize("scheme", ["w4a8", "w4a4"])       # w4a4 with G <= 128 is stored in its own (sign-magnitude) layout
@pytest.mark.parametrize("N,K,G", [(64, 128, 64), (128, 256, 128), (256, 512, 512), (320, 1024, 64)])
def test_pack_export_bit_exact(rd, N, K, G, scheme):
    inp = wl.tiny(seed=100 + N, M=4, K=K, N=N)
    ref = oracle.pack_int4(inp.W, inp.d, G)
    g = GpuLinear(rd, inp, scheme, G)
    ex = rd.rudder_weight_export(g.w)
    assert np.array_equal(ex["codes"].cpu().numpy(), ref["packed"])
    assert np.array_equal(ex["scales"].view(torch.int16).cpu().numpy().view(np.uint16), ref["scales"])
    assert np.array_equal(ex["dinv"].cpu().numpy().view(np.uint32), ref["dinv"].view(np.uint32))
    _assert_clean(rd)


def test_pack_without_channel_scales(rd):
    inp = wl.tiny(seed=101, M=4, K=256, N=64)
    ref = oracle.pack_int4(inp.W, None, 64)
    W = torch.from_numpy(inp.W).cuda()
    w = rd.rudder_pack_weights(W, None, rd.W4A8_INT, 64)
    ex = rd.rudder_weight_export(w)
    assert np.array_equal(ex["codes"].cpu().numpy(), ref["packed"])
    assert np.array_equal(ex["dinv"].cpu().numpy(), np.ones(256, np.float32))


def test_pack_degenerate_weights(rd):
    """Zero row, zero group, a group of tiny negative weights (fp16 scale underflows), one dominant weight,
    weights exactly on rounding ties of the 4-bit grid."""
    inp = wl.tiny(seed=131, M=4, K=512, N=64)
    inp.W[5, :] = 0.0
    inp.W[3, 64:128] = 0.0
    inp.W[7, 128:192] = -1e-12
    inp.W[9, 100] = 3.0
    inp.W[11, 0:64] = np.tile(np.array([7.0, 3.5, 2.5, 1.5, 0.5, -0.5, -2.5, -6.5], np.float32), 8) * 0.01
    inp.d[:] = 1.0
    ref = oracle.pack_int4(inp.W, inp.d, 64)
    for scheme in ("w4a8", "w4a4"):
        g = GpuLinear(rd, inp, scheme, 64)
        ex = rd.rudder_weight_export(g.w)
        assert np.array_equal(ex["scales"].cpu().numpy().view(np.uint16), ref["scales"].view(np.uint16))
        assert np.array_equal(ex["codes"].cpu().numpy(), ref["packed"])
    _assert_clean(rd)


@pytest.mark.parametrize("scheme,qmax", [("w4a8", 127), ("w4a4", 7)])
@pytest.mark.parametrize("mode", [0, 1])
@pytest.mark.parametrize("M,K", [(1, 128), (37, 384), (130, 1024), (64, 2048), (19, 4096), (9, 8192), (5, 12288),
                                 (300, 2048), (3, 16512)])   # many rows per CTA; rows too long to stage (warp-per-row kernel)
def test_activation_codes_bit_exact(rd, scheme, qmax, mode, M, K):
    inp = wl.tiny(seed=200 + M, M=M, K=K, N=64, T=3)
    ref_w = oracle.pack_int4(inp.W, inp.d, 64)
    clip = static_clip(inp, ref_w["dinv"]) if mode == 1 else None
    g = GpuLinear(rd, inp, scheme, 64, mode, clip)
    for step in (0, 2):
        codes, _, r = rd.rudder_quantize_activations(g.w, g.X, g.seg, step, g.tab)
        rc, rr = oracle.quantize_int(inp.X_bf16, ref_w["dinv"], inp.gamma, clip, step, mode, inp.seg_offsets,
                                     inp.seg_stream, qmax)
        assert np.array_equal(codes.cpu().numpy(), rc)
        assert np.array_equal(r.cpu().numpy().view(np.uint32), rr.view(np.uint32))
    _assert_clean(rd)


def test_activation_zero_row_and_strided_input(rd):
    inp = wl.tiny(seed=201, M=12, K=256, N=64, T=1)
    inp.X_bf16[3] = 0
    ref_w = oracle.pack_int4(inp.W, inp.d, 64)
    g = GpuLinear(rd, inp, "w4a8", 64)
    wide = torch.zeros((12, 256 + 64), dtype=torch.bfloat16, device="cuda")
    wide[:, :256] = g.X
    codes, _, r = rd.rudder_quantize_activations(g.w, wide[:, :256], g.seg, 0, g.tab)
    rc, rr = oracle.quantize_int(inp.X_bf16, ref_w["dinv"], inp.gamma, None, 0, 0, inp.seg_offsets, inp.seg_stream, 127)
    assert np.array_equal(codes.cpu().numpy(), rc) and np.array_equal(r.cpu().numpy(), rr)
    assert r[3].item() == 0.0 and not codes[3].any().item()


CASES = [
    # M, K, N, G, scheme
    (8, 128, 64, 64, "w4a8"),          # one stage, two groups, narrow ragged N tile
    (128, 256, 128, 64, "w4a8"),
    (130, 384, 256, 64, "w4a8"),       # ragged M tail, wide tile
    (200, 512, 320, 128, "w4a8"),      # N = 320: 128-wide tiles with a ragged last tile
    (64, 512, 256, 512, "w4a8"),       # G = K: the paper's per-output-channel scales (Eq. 10 verbatim)
    (257, 1024, 512, 64, "w4a4"),
    (96, 256, 256, 128, "w4a4"),
    (33, 2304, 256, 64, "w4a8"),       # 18 stages: every ring wraps several times
    (20, 512, 320, 64, "w4a4"),        # W4A4 with group scales runs on the E4M3 tensor path: 32-token tiles, ragged N
    (200, 2304, 256, 128, "w4a4"),     # 64-token tiles, 18 stages
    (300, 640, 128, 64, "w4a4"),       # 256-token tiles with a ragged tail
    (64, 512, 256, 512, "w4a4"),       # G = K stays on the integer path
    # the register-level kernel for a few dozen to a few hundred rows (groups of 64, K a multiple of 256 up to 4096),
    # all four tile shapes
    (512, 256, 1536, 64, "w4a8"),      # 128 x 64 tiles
    (500, 512, 1536, 64, "w4a4"),      # the same with sign-magnitude weights and a ragged last token tile
    (250, 1280, 2048, 64, "w4a8"),     # 64 x 64 tiles, 5 stages
    (60, 512, 3072, 64, "w4a8"),       # 64 x 32 tiles
    (200, 768, 320, 64, "w4a8"),       # 64 x 16 tiles with four warps, ragged M
    (70, 2048, 192, 64, "w4a4"),       # the same, 8 stages: the copy ring wraps
]


@pytest.mark.parametrize("M,K,N,G,scheme", CASES)
@pytest.mark.parametrize("mode", [0, 1])
def test_linear_accumulators_and_output(rd, M, K, N, G, scheme, mode):
    qmax = 127 if scheme == "w4a8" else 7
    inp = wl.tiny(seed=300 + M + N, M=M, K=K, N=N, T=2)
    ref_w = oracle.pack_int4(inp.W, inp.d, G)
    clip = static_clip(inp, ref_w["dinv"]) if mode == 1 else None
    g = GpuLinear(rd, inp, scheme, G, mode, clip)
    step = 1
    Y, acc = rd.rudder_linear_dump_acc(g.w, g.X, g.seg, step, g.tab, g.bias)
    rc, rr = oracle.quantize_int(inp.X_bf16, ref_w["dinv"], inp.gamma, clip, step, mode, inp.seg_offsets,
                                 inp.seg_stream, qmax)
    racc = oracle.accumulate_int(rc, ref_w["qw"], G)
    assert np.array_equal(acc.cpu().numpy(), racc), "INT32 group accumulators differ"
    _, y64 = oracle.linear_int(rc, rr, ref_w["qw"], ref_w["scales"], G, inp.bias)
    check_output(bf16_to_np(Y), y64)
    # the production entry point (no dump; up to 256 rows it splits K, so its fp32 summation order differs
    # from the dump launch's): held to the same gates, and repeatable bit for bit
    Y2 = rd.rudder_linear(g.w, g.X, g.seg, step, g.tab, g.bias)
    check_output(bf16_to_np(Y2), y64)
    assert torch.equal(Y2, rd.rudder_linear(g.w, g.X, g.seg, step, g.tab, g.bias))
    if M > 256:
        assert torch.equal(Y, Y2)                      # same tiles, same order
    _assert_clean(rd)


@pytest.mark.parametrize("G", [64, 128])
@pytest.mark.parametrize("M", [40, 300])
def test_w4a4_extreme_sums_are_exact(rd, G, M):
    """Every code at +-7: the group sums reach +-49 G, the largest magnitude the E4M3 / FP32-accumulator
    path has to hold exactly.  Row 0 and channel 0 are all-positive (sum = 49 G), the rest random signs."""
    K, N = 512, 128
    inp = wl.tiny(seed=977 + G + M, M=M, K=K, N=N)
    rng = np.random.default_rng(5)
    sw = rng.choice(np.array([-1.0, 1.0], np.float32), size=(N, K)); sw[0, :] = 1.0
    sx = rng.choice(np.array([-1.0, 1.0], np.float32), size=(M, K)); sx[0, :] = 1.0; sx[1, :] = -1.0
    inp.W[:] = 0.03 * sw
    inp.d[:] = 1.0
    X = (2.0 * sx).astype(np.float32)
    inp.X_bf16[:] = (X.view(np.uint32) >> 16).astype(np.uint16)        # +-2.0 is exact in bf16
    ref_w = oracle.pack_int4(inp.W, inp.d, G)
    assert np.all(np.abs(ref_w["qw"]) == 7)
    g = GpuLinear(rd, inp, "w4a4", G)
    Y, acc = rd.rudder_linear_dump_acc(g.w, g.X, g.seg, 0, g.tab, g.bias)
    rc, rr = oracle.quantize_int(inp.X_bf16, ref_w["dinv"], inp.gamma, None, 0, 0, inp.seg_offsets, inp.seg_stream, 7)
    assert np.all(np.abs(rc) == 7)
    racc = oracle.accumulate_int(rc, ref_w["qw"], G)
    assert racc[0, 0, 0] == 49 * G and racc[0, 1, 0] == -49 * G
    assert np.array_equal(acc.cpu().numpy(), racc)
    _, y64 = oracle.linear_int(rc, rr, ref_w["qw"], ref_w["scales"], G, inp.bias)
    check_output(bf16_to_np(Y), y64)
    _assert_clean(rd)


@pytest.mark.parametrize("scheme,mode,G", [("w4a8", 0, 384), ("w4a8", 1, 384), ("w4a4", 0, 384), ("w4a8", 0, 128), ("w4a8", 1, 128)])
def test_many_tiles_persistent_form(rd, scheme, mode, G):
    """One scale per output channel (Eq. 10 as printed; G = K = 384) and groups of 128, over enough tiles
    (18 x 27) that the GEMM runs in its persistent form: every CTA walks several tiles, ragged last token
    tile and last channel tile included.  The oracle is evaluated on a seeded sample of rows that covers
    every token tile, first and last rows."""
    M, K, N = 4420, 384, 3392
    inp = wl.tiny(seed=4242, M=M, K=K, N=N, T=2)
    ref_w = oracle.pack_int4(inp.W, inp.d, G)
    clip = static_clip(inp, ref_w["dinv"]) if mode == 1 else None
    g = GpuLinear(rd, inp, scheme, G, mode, clip)
    Y = rd.rudder_linear(g.w, g.X, g.seg, 1, g.tab, g.bias)
    rng = np.random.default_rng(7)
    rows = np.unique(np.concatenate([[0, 1, 255, 256, 257, M - 2, M - 1], np.arange(0, M, 256) + 3,
                                     rng.choice(M, 160, replace=False)])).astype(np.int32)
    out = oracle.rudder_linear(inp.X_bf16, ref_w, inp.gamma, clip, 1, mode, inp.seg_offsets, inp.seg_stream, scheme,
                               inp.bias, rows=rows)
    check_output(bf16_to_np(Y)[rows], out["y64"])
    # deterministic: a second call gives the same bits
    assert torch.equal(Y, rd.rudder_linear(g.w, g.X, g.seg, 1, g.tab, g.bias))
    # every element: the accumulator-dump variant (one CTA per tile, whole-tile store) gives the same bits,
    # and its INT32 sums on the sampled rows are the oracle's
    Y2, acc = rd.rudder_linear_dump_acc(g.w, g.X, g.seg, 1, g.tab, g.bias)
    assert torch.equal(Y, Y2)
    racc = oracle.accumulate_int(out["codes"], ref_w["qw"], G)
    assert np.array_equal(acc.cpu().numpy()[:, rows, :], racc)
    _assert_clean(rd)


@pytest.mark.parametrize("scheme,G", [("w4a8", 64), ("w4a8", 512), ("w4a4", 128), ("w4a4", 512), ("nvfp4", 16)])
def test_weight_import_round_trip(rd, scheme, G):
    """export -> import gives a handle whose own export and whose outputs are the same bits."""
    inp = wl.tiny(seed=140, M=150, K=512, N=320, T=2)
    g = GpuLinear(rd, inp, scheme, G)
    ex = rd.rudder_weight_export(g.w)
    w2 = rd.rudder_weight_import(ex, inp.N, inp.K, rd.SCHEMES[scheme], G)
    assert (w2.N, w2.K, w2.group, w2.scheme, w2.device_bytes) == (g.w.N, g.w.K, g.w.group, g.w.scheme, g.w.device_bytes)
    ex2 = rd.rudder_weight_export(w2)
    for k in ("codes", "scales", "dinv", "tensor_scale"):
        assert torch.equal(ex[k].view(torch.uint8), ex2[k].view(torch.uint8)), k
    Y = rd.rudder_linear(g.w, g.X, g.seg, 1, g.tab, g.bias)
    assert torch.equal(Y, rd.rudder_linear(w2, g.X, g.seg, 1, g.tab, g.bias))
    _assert_clean(rd)


def test_linear_no_bias_and_padded_output(rd):
    inp = wl.tiny(seed=301, M=70, K=256, N=128, T=1)
    ref_w = oracle.pack_int4(inp.W, inp.d, 64)
    g = GpuLinear(rd, inp, "w4a8", 64)
    Ybuf = torch.full((70, 128 + 8), 7.0, dtype=torch.bfloat16, device="cuda")
    rd.rudder_linear(g.w, g.X, g.seg, 0, g.tab, None, Y=Ybuf[:, :128])
    out = oracle.rudder_linear(inp.X_bf16, ref_w, inp.gamma, None, 0, 0, inp.seg_offsets, inp.seg_stream, "w4a8", None)
    check_output(bf16_to_np(Ybuf[:, :128]), out["y64"])
    assert (Ybuf[:, 128:] == 7.0).all().item()          # nothing written past N
    _assert_clean(rd)


def test_config0_full(rd):
    """Configuration 0: M = 256 (192 video / 16 proprio / 48 action), K = N = 1024, W4A8, G = 64."""
    cfg = wl.config(0)
    inp = cfg.draw()[0]
    ref_w = oracle.pack_int4(inp.W, inp.d, cfg.group)
    g = GpuLinear(rd, inp, cfg.scheme, cfg.group)
    Y, acc = rd.rudder_linear_dump_acc(g.w, g.X, g.seg, 0, g.tab, g.bias)
    out = oracle.rudder_linear(inp.X_bf16, ref_w, inp.gamma, None, 0, 0, inp.seg_offsets, inp.seg_stream, "w4a8", inp.bias)
    assert np.array_equal(acc.cpu().numpy(), oracle.accumulate_int(out["codes"], ref_w["qw"], cfg.group))
    fro, worst = check_output(bf16_to_np(Y), out["y64"])
    assert fro < 4e-3
    _assert_clean(rd)


def test_row_independence_on_gpu(rd):
    """Rows 120..135 straddle a 128-row tile and a segment boundary; a sub-call on them alone gives
    the same bits as the full call."""
    inp = wl.tiny(seed=302, M=256, K=512, N=256, T=1, parts=[(126, 0), (6, 1), (124, 2)])
    g = GpuLinear(rd, inp, "w4a8", 64)
    Y = rd.rudder_linear(g.w, g.X, g.seg, 0, g.tab, g.bias)
    sub_seg = rd.Segments([0, 6, 12, 16], [0, 1, 2])
    Ys = rd.rudder_linear(g.w, g.X[120:136], sub_seg, 0, g.tab, g.bias)
    assert torch.equal(Y[120:136], Ys)
    _assert_clean(rd)


def test_block_matches_four_linears(rd):
    H, F, M = 256, 512, 150
    rng = np.random.default_rng(5)
    so, ss = wl.segments([(100, 0), (20, 1), (30, 2)])
    lins = [wl.draw_linear(rng, M, K, N, 2, 3, so, ss, 0.01, 30.0) for K, N in [(H, 3 * H), (H, H), (H, F), (F, H)]]
    gs = [GpuLinear(rd, l, "w4a8", 64) for l in lins]
    ys = [torch.empty((M, l.N), dtype=torch.bfloat16, device="cuda") for l in lins]
    args = rd.BlockArgs([g.w for g in gs], [g.tab for g in gs], [g.bias for g in gs], [g.X for g in gs], ys)
    ws = torch.empty(rd.rudder_block_workspace_bytes(args, M) + 256, dtype=torch.uint8, device="cuda")
    rd.rudder_block(args, M, gs[0].seg, 1, ws)
    for g, l, y in zip(gs, lins, ys):
        ref_w = oracle.pack_int4(l.W, l.d, 64)
        out = oracle.rudder_linear(l.X_bf16, ref_w, l.gamma, None, 1, 0, l.seg_offsets, l.seg_stream, "w4a8", l.bias)
        check_output(bf16_to_np(y), out["y64"])
        assert torch.equal(y, rd.rudder_linear(g.w, g.X, g.seg, 1, g.tab, g.bias))
    # the same block from pinned host buffers (uploads, kernels and downloads overlap on three streams),
    # twice in a row over the same staging area
    xh = [g.X.cpu().pin_memory() for g in gs]
    yh = [torch.zeros((M, l.N), dtype=torch.bfloat16).pin_memory() for l in lins]
    hargs = rd.BlockArgs([g.w for g in gs], [g.tab for g in gs], [g.bias for g in gs], xh, yh)
    staging = torch.empty(rd.rudder_block_host_staging_bytes(hargs, M) + 256, dtype=torch.uint8, device="cuda")
    for _ in range(2):
        for t in yh:
            t.zero_()
        rd.rudder_block_host(hargs, M, gs[0].seg, 1, staging, ws)
        torch.cuda.current_stream().synchronize()          # the stream waits for the last download
        for y, t in zip(ys, yh):
            assert torch.equal(y.cpu(), t)
    _assert_clean(rd)


def test_argument_errors_on_device_box(rd):
    inp = wl.tiny(seed=303, M=16, K=128, N=64, T=2)
    g = GpuLinear(rd, inp, "w4a8", 64)
    with pytest.raises(rd.RudderError) as e:
        rd.rudder_linear(g.w, g.X, g.seg, 2, g.tab, g.bias)            # step out of range
    assert e.value.status == rd.ERR_ARG
    with pytest.raises(rd.RudderError) as e:
        rd.rudder_linear(g.w, g.X, rd.Segments([0, 8], [0]), 0, g.tab)  # segments do not cover M
    assert e.value.status == rd.ERR_ARG
    with pytest.raises(rd.RudderError) as e:
        rd.rudder_linear(g.w, g.X, g.seg, 0, rd.ScaleTable(g.gamma, None, rd.RANGE_STATIC))   # static without clip
    assert e.value.status == rd.ERR_ARG
    with pytest.raises(rd.RudderError) as e:
        rd.rudder_linear(g.w, g.X, g.seg, 0, g.tab, workspace=torch.empty(512, dtype=torch.uint8, device="cuda"))
    assert e.value.status == rd.ERR_WORKSPACE
    _assert_clean(rd)


def test_bounded_wait_gives_up_and_context_survives(rd):
    """A wait that nothing satisfies runs into its limit: the kernel returns, the status word names the wait,
    reading it clears it, and the library goes on working."""
    _assert_clean(rd)
    rd.rudder_selftest_wait_timeout(1_000_000)               # about half a millisecond of SM clocks
    last, where = rd.rudder_device_status()
    assert (last, where) == (rd.ERR_TIMEOUT, 901)
    assert rd.rudder_device_status() == (0, 0)               # cleared by the read
    with pytest.raises(rd.RudderError) as e:
        rd.rudder_selftest_wait_timeout(10 ** 12)            # unreasonable limits are refused on the host
    assert e.value.status == rd.ERR_ARG
    inp = wl.tiny(seed=304, M=40, K=256, N=128, T=1)
    g = GpuLinear(rd, inp, "w4a8", 64)
    Y = rd.rudder_linear(g.w, g.X, g.seg, 0, g.tab, g.bias)
    out = oracle.rudder_linear(inp.X_bf16, oracle.pack_int4(inp.W, inp.d, 64), inp.gamma, None, 0, 0, inp.seg_offsets,
                               inp.seg_stream, "w4a8", inp.bias)
    check_output(bf16_to_np(Y), out["y64"])
    _assert_clean(rd)
