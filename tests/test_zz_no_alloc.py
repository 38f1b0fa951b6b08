"""rudder_linear_static: the entry point for callers that cannot allocate device memory (code inside
a captured or real-time region, plug-ins that only receive input and output buffers).  Its scratch
is a fixed array inside the library, so the test checks it against rudder_linear, whose scratch the
caller allocates (same kernels, so the outputs must agree within the suite's tolerance -- they are in
fact identical) and against the CPU oracle, on two calls in a row that reuse the array; an oversized
request is refused."""
import numpy as np
import pytest
import torch

import oracle
import workloads as wl
from helpers import ABS_TOL, REL_TOL, GpuLinear, bf16_to_np, check_output

pytestmark = pytest.mark.gpu


def _close(a: torch.Tensor, b: torch.Tensor):
    x = wl.bf16_bits_to_f32(bf16_to_np(a)).astype(np.float64)
    y = wl.bf16_bits_to_f32(bf16_to_np(b)).astype(np.float64)
    return bool(np.all(np.abs(x - y) <= ABS_TOL + REL_TOL * np.abs(y)))


def test_static_workspace_entry_point_matches_rudder_linear():
    import paper_2609_39056_b200 as rd
    rd.lib()
    assert rd.rudder_linear_static_max_workspace_bytes() == 4 << 20

    # first call: 256 x 1024 -> 1024 (the smallest benchmark configuration), second call: another
    # shape and scheme, so that the array still holds the first call's codes when it starts
    first = GpuLinear(rd, wl.config(0).draw()[0], "w4a8", 64)
    second = GpuLinear(rd, wl.tiny(seed=77, M=200, K=2048, N=320, T=2), "w4a4", 128)
    for g, step in ((first, 0), (second, 1)):
        want = rd.rudder_linear(g.w, g.X, g.seg, step, g.tab, g.bias)
        got = torch.full_like(want, float("nan"))
        rd.rudder_linear_static(g.w, g.X, g.seg, step, g.tab, g.bias, Y=got)
        torch.cuda.synchronize()
        assert _close(got, want)
        assert torch.equal(got, want)
        # and against the CPU oracle, like every other entry point
        inp = g.inp
        ref = oracle.rudder_linear(inp.X_bf16, oracle.pack_int4(inp.W, inp.d, g.group), inp.gamma, None, step,
                                   oracle.RANGE_PER_TOKEN, inp.seg_offsets, inp.seg_stream, g.scheme, inp.bias)
        check_output(bf16_to_np(got), ref["y64"])
    # and the first shape again, after the array was overwritten by the second
    want = rd.rudder_linear(first.w, first.X, first.seg, 0, first.tab, first.bias)
    got = torch.empty_like(want)
    rd.rudder_linear_static(first.w, first.X, first.seg, 0, first.tab, first.bias, Y=got)
    assert _close(got, want)

    # 4416 rows x 2048 channels of codes do not fit in 4 MiB: refused, nothing launched
    big = torch.zeros((4416, 2048), dtype=torch.bfloat16, device="cuda")
    wbig = rd.rudder_pack_weights(torch.randn(64, 2048, device="cuda"), None, rd.W4A8_INT, 64)
    out = torch.full((4416, 64), 3.0, dtype=torch.bfloat16, device="cuda")
    seg = rd.Segments([0, 4416], [0])
    tab = rd.ScaleTable(torch.ones((1, 1), device="cuda"))
    with pytest.raises(rd.RudderError) as e:
        rd.rudder_linear_static(wbig, big, seg, 0, tab, None, Y=out)
    assert e.value.status == rd.ERR_WORKSPACE
    torch.cuda.synchronize()
    assert (out == 3.0).all().item()
    last, where = rd.rudder_device_status()
    assert last == 0, (last, where)
