"""BF16 glue on the GPU: the GELU kernel against the oracle on every bf16 bit pattern, and the chained
block (x[1..3] = NULL) against the same four linears and the glue run one by one."""
import numpy as np
import pytest
import torch

import oracle
import workloads as wl
from helpers import GpuLinear, bf16_to_np, check_output, oracle_pack, to_dev_bf16
from oracle import glue

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def rd():
    import paper_2609_39056_b200 as rd
    rd.lib()
    return rd


def test_gelu_every_bf16_pattern(rd):
    bits = np.arange(65536, dtype=np.uint16).reshape(512, 128)
    X = to_dev_bf16(bits)
    Y = rd.rudder_gelu(X)
    got = bf16_to_np(Y)
    want = glue.gelu_bf16(bits)
    x = glue.bf16_to_f32(bits)
    finite = np.isfinite(x)
    assert np.array_equal(got[finite], want[finite])
    # infinities and NaN: same class of result (NaN payloads are not compared)
    g, w = glue.bf16_to_f32(got[~finite]), glue.bf16_to_f32(want[~finite])
    assert np.array_equal(np.isnan(g), np.isnan(w)) and np.array_equal(g[~np.isnan(g)], w[~np.isnan(w)])


def test_gelu_strided_and_errors(rd):
    X = torch.randn((37, 256), device="cuda").to(torch.bfloat16)
    Y = torch.full((37, 384), 7.0, dtype=torch.bfloat16, device="cuda")
    rd.rudder_gelu(X[:, 64:192], Y[:, 128:256])
    want = glue.gelu_bf16(bf16_to_np(X[:, 64:192].contiguous()))
    assert np.array_equal(bf16_to_np(Y[:, 128:256].contiguous()), want)
    assert torch.all(Y[:, :128] == 7.0) and torch.all(Y[:, 256:] == 7.0)
    with pytest.raises(rd.RudderError):
        rd.rudder_gelu(X[:, :100])              # N not a multiple of 8


@pytest.mark.parametrize("scheme,G", [("w4a8", 64), ("nvfp4", 16)])
def test_chained_block(rd, scheme, G):
    H, F, M = 256, 1024, 70
    shapes = [(H, 3 * H), (H, H), (H, F), (F, H)]
    layers = [GpuLinear(rd, wl.tiny(seed=700 + i, M=M, K=K, N=N, T=2), scheme, G) for i, (K, N) in enumerate(shapes)]
    seg, step = layers[0].seg, 1
    # one by one, with the same glue
    y0 = rd.rudder_linear(layers[0].w, layers[0].X, seg, step, layers[0].tab, layers[0].bias)
    y1 = rd.rudder_linear(layers[1].w, y0[:, 2 * H:3 * H], seg, step, layers[1].tab, layers[1].bias)
    y2 = rd.rudder_linear(layers[2].w, y1, seg, step, layers[2].tab, layers[2].bias)
    a2 = rd.rudder_gelu(y2)
    y3 = rd.rudder_linear(layers[3].w, a2, seg, step, layers[3].tab, layers[3].bias)
    # chained
    ys = [torch.full_like(y, float("nan")) for y in (y0, y1, y2, y3)]
    bargs = rd.BlockArgs([l.w for l in layers], [l.tab for l in layers], [l.bias for l in layers],
                         [layers[0].X, None, None, None], ys)
    ws = torch.empty(rd.rudder_block_workspace_bytes(bargs, M) + 256, dtype=torch.uint8, device="cuda")
    rd.rudder_block(bargs, M, seg, step, ws)
    torch.cuda.synchronize()
    for l, (a, b) in enumerate(zip(ys, (y0, y1, y2, y3))):
        assert torch.equal(a, b), f"layer {l}"
    # each layer against the oracle, fed the GPU's own input of that layer
    ins = [bf16_to_np(layers[0].X), bf16_to_np(y0[:, 2 * H:3 * H].contiguous()), bf16_to_np(y1), glue.gelu_bf16(bf16_to_np(y2))]
    assert np.array_equal(ins[3], bf16_to_np(a2))
    for l, g in enumerate(layers):
        ref_w = oracle_pack(g.inp, scheme, G)
        out = oracle.rudder_linear(ins[l], ref_w, g.inp.gamma, None, step, 0, layers[0].inp.seg_offsets, layers[0].inp.seg_stream,
                                   scheme, g.inp.bias)
        check_output(bf16_to_np(ys[l]), out["y64"], **({"rel": 2e-2} if scheme == "nvfp4" else {}))
    # a shape that does not chain is refused before anything is launched
    bad = rd.BlockArgs([layers[0].w, layers[2].w, layers[2].w, layers[3].w], [l.tab for l in layers], [None] * 4,
                       [layers[0].X, None, None, None], ys)
    with pytest.raises(rd.RudderError):
        rd.rudder_block(bad, M, seg, step, ws)
    last, where = rd.rudder_device_status()
    assert last == 0, (last, where)


@pytest.mark.parametrize("M,N", [(1, 8), (37, 264), (70, 2048), (5, 3072), (130, 12288)])
def test_rmsnorm_and_add_bit_exact(rd, M, N):
    rng = np.random.default_rng(900 + N)
    xb = glue.f32_to_bf16((rng.standard_normal((M, N)) * 3.0).astype(np.float32))
    yb = glue.f32_to_bf16((rng.standard_normal((M, N)) * 0.7).astype(np.float32))
    if M > 2:
        xb[1] = 0                                                  # an all-zero row
    w = (1.0 + 0.1 * rng.standard_normal(N)).astype(np.float32)
    X, Y2, W = to_dev_bf16(xb), to_dev_bf16(yb), torch.from_numpy(w).cuda()
    for eps in (1e-6, 0.0) if M > 2 else (1e-6,):
        got = bf16_to_np(rd.rudder_rmsnorm(X, W, eps))
        want = glue.rmsnorm_bf16(xb, w, eps)
        if eps == 0.0 and M > 2:                                   # 0 / 0 row: NaN on both sides
            assert np.isnan(glue.bf16_to_f32(got[1])).all() and np.isnan(glue.bf16_to_f32(want[1])).all()
            got, want = np.delete(got, 1, 0), np.delete(want, 1, 0)
        assert np.array_equal(got, want)
    assert np.array_equal(bf16_to_np(rd.rudder_add(X, Y2)), glue.add_bf16(xb, yb))
    # strided views
    wide = torch.zeros((M, N + 16), dtype=torch.bfloat16, device="cuda")
    wide[:, 8:N + 8] = X
    out = torch.full((M, N + 8), 5.0, dtype=torch.bfloat16, device="cuda")
    rd.rudder_rmsnorm(wide[:, 8:N + 8], W, 1e-6, Y=out[:, :N])
    assert np.array_equal(bf16_to_np(out[:, :N].contiguous()), glue.rmsnorm_bf16(xb, w, 1e-6)) and (out[:, N:] == 5.0).all().item()


@pytest.mark.parametrize("scheme,G", [("w4a8", 64), ("w4a8", 256), ("nvfp4", 16)])
def test_dit_block_with_bf16_glue(rd, scheme, G):
    """rudder_block_dit: every glue step is the oracle's bit for bit, every linear is within tolerance of the
    oracle fed the very input the GPU gave it."""
    H, F, M = 256, 1024, 70
    shapes = [(H, 3 * H), (H, H), (H, F), (F, H)]
    layers = [GpuLinear(rd, wl.tiny(seed=800 + i, M=M, K=K, N=N, T=2), scheme, G if G != 256 else K) for i, (K, N) in enumerate(shapes)]
    seg, step = layers[0].seg, 1
    rng = np.random.default_rng(77)
    w1 = (1.0 + 0.1 * rng.standard_normal(H)).astype(np.float32)
    w2 = (1.0 + 0.1 * rng.standard_normal(H)).astype(np.float32)
    W1, W2 = torch.from_numpy(w1).cuda(), torch.from_numpy(w2).cuda()
    eps = 1e-6
    ys = [torch.full((M, N), float("nan"), dtype=torch.bfloat16, device="cuda") for _, N in shapes]
    out = torch.full((M, H), float("nan"), dtype=torch.bfloat16, device="cuda")
    bargs = rd.BlockArgs([l.w for l in layers], [l.tab for l in layers], [l.bias for l in layers], [layers[0].X, None, None, None], ys)
    ws = torch.empty(rd.rudder_block_dit_workspace_bytes(bargs, M) + 256, dtype=torch.uint8, device="cuda")
    rd.rudder_block_dit(bargs, W1, W2, eps, out, M, seg, step, ws)
    torch.cuda.synchronize()
    x0 = bf16_to_np(layers[0].X)
    y = [bf16_to_np(t) for t in ys]
    # the glue, recomputed by the oracle from the GPU's own linear outputs
    n1 = glue.rmsnorm_bf16(x0, w1, eps)
    h1 = glue.add_bf16(x0, y[1])
    n2 = glue.rmsnorm_bf16(h1, w2, eps)
    ge = glue.gelu_bf16(y[2])
    assert np.array_equal(bf16_to_np(out), glue.add_bf16(h1, y[3]))
    ins = [n1, np.ascontiguousarray(y[0][:, 2 * H:3 * H]), n2, ge]
    for l, g in enumerate(layers):
        ref_w = oracle_pack(g.inp, scheme, g.group)
        o = oracle.rudder_linear(ins[l], ref_w, g.inp.gamma, None, step, 0, layers[0].inp.seg_offsets, layers[0].inp.seg_stream,
                                 scheme, g.inp.bias)
        check_output(y[l], o["y64"], **({"rel": 2e-2} if scheme == "nvfp4" else {}))
        # and the same layer through rudder_linear on the oracle's glue output gives the block's bits: the block
        # really fed that input
        assert torch.equal(ys[l], rd.rudder_linear(g.w, to_dev_bf16(ins[l]), seg, step, g.tab, g.bias)), f"layer {l}"
    # replay inputs are refused (the block runs from x[0] alone), and so are shapes that do not form a block
    bad = rd.BlockArgs([l.w for l in layers], [l.tab for l in layers], [l.bias for l in layers], [layers[0].X, layers[1].X, None, None], ys)
    with pytest.raises(rd.RudderError):
        rd.rudder_block_dit(bad, W1, W2, eps, out, M, seg, step, ws)
    bad2 = rd.BlockArgs([layers[0].w, layers[2].w, layers[2].w, layers[3].w], [l.tab for l in layers], [None] * 4, [layers[0].X, None, None, None], ys)
    with pytest.raises(rd.RudderError):
        rd.rudder_block_dit(bad2, W1, W2, eps, out, M, seg, step, ws)
    last, where = rd.rudder_device_status()
    assert last == 0, (last, where)


@pytest.mark.parametrize("scheme,G", [("w4a8", 0), ("w4a8", 64), ("w4a4", 64), ("w4a4", 0)])
@pytest.mark.parametrize("M", [20, 300])
def test_static_range_fuses_gelu_into_the_down_prologue(rd, scheme, G, M):
    """Chained block whose down projection has the paper's static threshold: the GELU runs inside that layer's
    prologue.  The codes and row scales of the fused pass are the oracle's (GELU, then static quantisation) bit
    for bit, and the block's outputs are the bits of the unfused sequence."""
    H, F = 256, 1024
    shapes = [(H, 3 * H), (H, H), (H, F), (F, H)]
    qmax = 127 if scheme == "w4a8" else 7
    inps = [wl.tiny(seed=860 + i, M=M, K=K, N=N, T=2) for i, (K, N) in enumerate(shapes)]
    step = 1
    # thresholds: for the down projection a value that clips some of the activated values
    clips = [np.array([3.0, 2.0], np.float32) for _ in shapes]
    clips[3] = np.array([0.8, 0.35], np.float32)
    layers = [GpuLinear(rd, inp, scheme, G or inp.K, 1, clips[i]) for i, inp in enumerate(inps)]
    seg = layers[0].seg
    ys = [torch.full((M, N), float("nan"), dtype=torch.bfloat16, device="cuda") for _, N in shapes]
    bargs = rd.BlockArgs([l.w for l in layers], [l.tab for l in layers], [l.bias for l in layers], [layers[0].X, None, None, None], ys)
    ws = torch.empty(rd.rudder_block_workspace_bytes(bargs, M) + 256, dtype=torch.uint8, device="cuda")
    rd.rudder_block(bargs, M, seg, step, ws)
    torch.cuda.synchronize()
    # the fused pass alone against the oracle
    y2 = bf16_to_np(ys[2])
    codes, r = rd.rudder_gelu_quantize_activations(layers[3].w, ys[2], seg, step, layers[3].tab)
    ref_w = oracle_pack(inps[3], scheme, G or inps[3].K)
    rc, rr = oracle.quantize_int(glue.gelu_bf16(y2), ref_w["dinv"], inps[3].gamma, clips[3], step, 1, inps[0].seg_offsets,
                                 inps[0].seg_stream, qmax)
    assert np.array_equal(codes.cpu().numpy(), rc)
    assert np.array_equal(r.cpu().numpy().view(np.uint32), rr.view(np.uint32))
    assert (np.abs(rc) == qmax).any()                              # the threshold does clip
    # the down output: the oracle on the GPU's own up output, and the unfused sequence bit for bit
    _, y64 = oracle.linear_int(rc, rr, ref_w["qw"], ref_w["scales"], G or inps[3].K, inps[3].bias)
    check_output(bf16_to_np(ys[3]), y64)
    a2 = rd.rudder_gelu(ys[2])
    assert torch.equal(ys[3], rd.rudder_linear(layers[3].w, a2, seg, step, layers[3].tab, layers[3].bias))
    # per-token tables are not fused: the hook says so
    pt = GpuLinear(rd, inps[3], scheme, G or inps[3].K)
    with pytest.raises(rd.RudderError) as e:
        rd.rudder_gelu_quantize_activations(pt.w, ys[2], seg, step, pt.tab)
    assert e.value.status == rd.ERR_UNSUPPORTED
    last, where = rd.rudder_device_status()
    assert last == 0, (last, where)
