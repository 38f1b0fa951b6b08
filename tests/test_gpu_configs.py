"""Parity at the benchmark configurations' full sizes, in the launch configuration bench.py times
(rudder_block / rudder_linear on the whole M), against the oracle on sampled rows.  Rows are
independent (pinned by the oracle's row-independence test), so a seeded row sample that includes
every segment's first and last row and rows around tile edges is computed by the oracle one row at a
time.  Activation codes and row scales of the sampled rows are compared bit for bit, outputs within
the stated tolerance."""
import numpy as np
import pytest
import torch

import oracle
import workloads as wl
from helpers import ABS_TOL, REL_TOL, REL_TOL_FP4, GpuLinear, bf16_to_np, check_output, oracle_pack

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def rd():
    import paper_2609_39056_b200 as rd
    rd.lib()
    return rd


def sample_rows(seg_offsets, M, n_random, seed):
    rows = set()
    for s in range(len(seg_offsets) - 1):
        lo, hi = int(seg_offsets[s]), int(seg_offsets[s + 1])
        if hi > lo:
            rows.update([lo, hi - 1])
    for edge in (127, 128, 255, 256, 511, 512, M - 129, M - 128, M - 1):
        if 0 <= edge < M:
            rows.add(edge)
    rng = np.random.default_rng(seed)
    rows.update(int(x) for x in rng.choice(M, size=min(n_random, M), replace=False))
    return np.array(sorted(rows), np.int32)


def check_linear_rows(rd, g, inp, ref_w, scheme, Y, step, rows):
    qmax = {"w4a8": 127, "w4a4": 7}.get(scheme)
    out = oracle.rudder_linear(inp.X_bf16, ref_w, inp.gamma, None, step, 0, inp.seg_offsets, inp.seg_stream, scheme,
                               inp.bias, rows=rows)
    codes, sb, r = rd.rudder_quantize_activations(g.w, g.X, g.seg, step, g.tab)
    idx = torch.from_numpy(rows.astype(np.int64)).cuda()
    if scheme == "nvfp4":
        packed = (out["codes"][:, 0::2] | (out["codes"][:, 1::2] << 4)).astype(np.uint8)
        assert np.array_equal(codes[idx].cpu().numpy(), packed)
        assert np.array_equal(sb[idx].cpu().numpy(), out["sb"])
    else:
        assert np.array_equal(codes[idx].cpu().numpy(), out["codes"])
    assert np.array_equal(r[idx].cpu().numpy().view(np.uint32), out["r"].view(np.uint32))
    rel = REL_TOL_FP4 if scheme == "nvfp4" else REL_TOL
    return check_output(bf16_to_np(Y[idx]), out["y64"], rel=rel, abs_=ABS_TOL)


def run_block_config(rd, cfg, steps, n_random):
    lins = cfg.draw()
    M = cfg.M
    gs = [GpuLinear(rd, l, cfg.scheme, cfg.group) for l in lins]
    refs = [oracle_pack(l, cfg.scheme, cfg.group) for l in lins]
    ys = [torch.empty((M, l.N), dtype=torch.bfloat16, device="cuda") for l in lins]
    args = rd.BlockArgs([g.w for g in gs], [g.tab for g in gs], [g.bias for g in gs], [g.X for g in gs], ys)
    ws = torch.empty(rd.rudder_block_workspace_bytes(args, M) + 256, dtype=torch.uint8, device="cuda")
    rows = sample_rows(lins[0].seg_offsets, M, n_random, cfg.seed)
    for step in steps:
        for y in ys:
            y.fill_(float("nan"))
        rd.rudder_block(args, M, gs[0].seg, step, ws)
        torch.cuda.synchronize()
        for g, l, ref, y in zip(gs, lins, refs, ys):
            assert not torch.isnan(y).any().item(), "rows left unwritten"
            check_linear_rows(rd, g, l, ref, cfg.scheme, y, step, rows)
    last, where = rd.rudder_device_status()
    assert last == 0, (last, where)


def test_config2_w4a8_block_full_size(rd):
    """Configuration 2: hidden 2048, MLP 8192, 4096 + 64 + 256 tokens, W4A8 group 64, steps 0, 4 and 9."""
    run_block_config(rd, wl.config(2), steps=(0, 4, 9), n_random=256)


@pytest.mark.parametrize("scheme", ["w4a4", "nvfp4"])
def test_config3_w4a4_block_full_size(rd, scheme):
    """Configuration 3: hidden 3072, MLP 12288, batch 2 x (8192 + 64 + 512) tokens; steps 0, 7 and 9 on
    256 seeded rows plus every segment's first and last row and the rows around tile edges."""
    run_block_config(rd, wl.config(3, scheme), steps=(0, 7, 9), n_random=256)


@pytest.mark.parametrize("scheme", ["w4a8", "w4a4"])
@pytest.mark.parametrize("M,KN", [(16, 2048), (64, 4096), (128, 2048), (256, 4096)])
def test_config4_small_m(rd, scheme, M, KN):
    """Configuration 4: action + proprio only, one packed weight reused across 20 steps of tables."""
    cfg = wl.config(4, scheme, M=M, KN=KN)
    inp = cfg.draw()[0]
    ref_w = oracle.pack_int4(inp.W, inp.d, cfg.group)
    g = GpuLinear(rd, inp, scheme, cfg.group)
    for step in (0, 11, 19):
        Y = rd.rudder_linear(g.w, g.X, g.seg, step, g.tab, g.bias)
        out = oracle.rudder_linear(inp.X_bf16, ref_w, inp.gamma, None, step, 0, inp.seg_offsets, inp.seg_stream, scheme,
                                   inp.bias)
        check_output(bf16_to_np(Y), out["y64"])
    last, where = rd.rudder_device_status()
    assert last == 0, (last, where)


@pytest.mark.parametrize("scheme,group", [("w4a8", 64), ("w4a8", 0), ("w4a4", 64), ("nvfp4", 16)])
def test_cross_attention_kv_projections(rd, scheme, group):
    """The cross-attention key and value projections: one global-text region each (a single segment of one
    stream), 512 x 1024 -> 2048, every row against the oracle at three steps."""
    cfg = wl.config(5, scheme)
    for inp in cfg.draw():
        G = group or inp.K
        g = GpuLinear(rd, inp, scheme, G)
        ref_w = oracle_pack(inp, scheme, G)
        assert len(inp.seg_stream) == 1 and inp.S == 1
        rows = np.arange(inp.M, dtype=np.int32)
        for step in (0, 5, 9):
            Y = rd.rudder_linear(g.w, g.X, g.seg, step, g.tab, g.bias)
            check_linear_rows(rd, g, inp, ref_w, scheme, Y, step, rows)
    last, where = rd.rudder_device_status()
    assert last == 0, (last, where)
