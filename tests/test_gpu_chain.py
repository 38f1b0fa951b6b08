"""Back-to-back linears on one stream that share one workspace.  The prologue kernel of a call may be
launched before the GEMM of the previous call has finished (programmatic dependent launch) and the
small-M GEMM before its own prologue has; both wait inside the kernel before they touch the shared
buffers.  The chain must therefore give, call by call, exactly the bits each call gives alone -- with
plain launches and replayed from a CUDA graph."""
import numpy as np
import pytest
import torch

import oracle
import workloads as wl
from helpers import ABS_TOL, REL_TOL, GpuLinear, bf16_to_np, check_output, oracle_pack

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def rd():
    import paper_2609_39056_b200 as rd
    rd.lib()
    return rd


def _layers(rd):
    return [
        GpuLinear(rd, wl.tiny(seed=901, M=16, K=2048, N=2048, T=2), "w4a8", 64),     # K split over several CTAs
        GpuLinear(rd, wl.tiny(seed=902, M=64, K=1024, N=512, T=2), "w4a4", 64),
        GpuLinear(rd, wl.tiny(seed=903, M=200, K=512, N=256, T=2), "nvfp4", 16),
        GpuLinear(rd, wl.tiny(seed=904, M=300, K=1024, N=384, T=2), "w4a8", 128),    # 256-token tiles, TMA store
        GpuLinear(rd, wl.tiny(seed=905, M=1030, K=512, N=256, T=2), "nvfp4", 16),    # CTA-pair kernel
        GpuLinear(rd, wl.tiny(seed=906, M=4420, K=256, N=3392, T=2), "w4a8", 256),   # 486 tiles, one scale per channel: persistent form
        GpuLinear(rd, wl.tiny(seed=907, M=4420, K=256, N=3392, T=2), "w4a8", 128),   # persistent form with two groups per tile
    ]


def test_chain_shares_workspace(rd):
    layers = _layers(rd)
    ws_bytes = max(rd.rudder_linear_workspace_bytes(g.w, g.X.shape[0]) for g in layers) + 256
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device="cuda")
    alone = []
    for g in layers:
        alone.append(rd.rudder_linear(g.w, g.X, g.seg, 1, g.tab, g.bias))
        torch.cuda.synchronize()
    # the first layer against the oracle, so that "alone" is anchored here too
    g = layers[0]
    ref_w = oracle_pack(g.inp, "w4a8", 64)
    out = oracle.rudder_linear(g.inp.X_bf16, ref_w, g.inp.gamma, None, 1, 0, g.inp.seg_offsets, g.inp.seg_stream, "w4a8",
                               g.inp.bias)
    check_output(bf16_to_np(alone[0]), out["y64"], rel=REL_TOL, abs_=ABS_TOL)

    order = [0, 1, 2, 3, 4, 0, 0, 2, 4, 4, 1, 3, 3, 1, 0, 2, 2, 4, 0, 5, 0, 6, 5, 5, 3, 6, 1]
    outs = [torch.full_like(alone[i], float("nan")) for i in order]
    for i, y in zip(order, outs):
        g = layers[i]
        rd.rudder_linear(g.w, g.X, g.seg, 1, g.tab, g.bias, Y=y, workspace=ws)
    torch.cuda.synchronize()
    for k, (i, y) in enumerate(zip(order, outs)):
        assert torch.equal(y, alone[i]), f"call {k} (layer {i}) differs from the same call alone"

    # the same chain captured once and replayed
    stream = torch.cuda.Stream()
    outs2 = [torch.full_like(alone[i], float("nan")) for i in order]
    with torch.cuda.stream(stream):
        g0 = layers[0]
        rd.rudder_linear(g0.w, g0.X, g0.seg, 1, g0.tab, g0.bias, Y=outs2[0], workspace=ws, stream=stream)   # one-time set-up outside capture
        stream.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            for i, y in zip(order, outs2):
                g = layers[i]
                rd.rudder_linear(g.w, g.X, g.seg, 1, g.tab, g.bias, Y=y, workspace=ws, stream=stream)
        for _ in range(3):
            for y in outs2:
                y.fill_(float("nan"))
            graph.replay()
            stream.synchronize()
            for k, (i, y) in enumerate(zip(order, outs2)):
                assert torch.equal(y, alone[i]), f"replayed call {k} (layer {i}) differs"
    last, where = rd.rudder_device_status()
    assert last == 0, (last, where)
