"""The GPU-side toy calibrator (Eq. 9) against the oracle's: the objective it evaluates through
`rudder_linear` agrees with the oracle's at fixed points, and the point it finds is as good as the
oracle's own when both are scored by the oracle's objective."""
import numpy as np
import pytest
import torch

import oracle
import workloads as wl
from helpers import GpuLinear
from oracle import calibrate as oc

pytestmark = pytest.mark.gpu

STEPS = [2 ** -0.5, 2 ** -0.25, 2 ** 0.25, 2 ** 0.5]


@pytest.fixture(scope="module")
def rd():
    import paper_2609_39056_b200 as rd
    rd.lib()
    return rd


def _case(scheme, G, seed=5, M=96, K=256, N=64):
    inp = wl.tiny(seed=seed, M=M, K=K, N=N, T=1)
    pw = oracle.pack_int4(inp.W, inp.d, G)
    X = wl.bf16_bits_to_f32(inp.X_bf16).astype(np.float64)
    v = np.abs(X * pw["dinv"][None, :].astype(np.float64))
    cs = [float(np.quantile(v, q)) for q in (0.99, 0.995, 0.999, 1.0)]
    return inp, pw, cs


@pytest.mark.parametrize("scheme,G", [("w4a8", 64), ("w4a4", 64), ("w4a8", 256)])
def test_calibrator_matches_oracle(rd, scheme, G):
    from paper_2609_39056_b200 import calibrate as gc
    inp, pw, cs = _case(scheme, G)
    g = GpuLinear(rd, inp, scheme, G)
    # dequantized weights and reference output
    What = gc.dequantized_weights(g.w).cpu().numpy().astype(np.float64)
    assert np.array_equal(What, oc.dequantized_weights(pw))
    y_ref = oc.reference_output(inp.X_bf16, pw)

    res = gc.calibrate_step(g.w, g.X, g.seg, 3, cs, STEPS)
    ref = oc.calibrate(inp.X_bf16, pw, inp.seg_offsets, inp.seg_stream, 3, scheme, cs, STEPS)
    _, n = oc.stream_rows(inp.seg_offsets, inp.seg_stream, 3)
    gam = np.array(res["gamma"])
    assert abs((n * np.log(gam)).sum()) < 1e-6 and gam.min() >= 0.5 and gam.max() <= 2.0 and res["clip"] in cs

    def J(gamma, c):
        return oc.objective(inp.X_bf16, pw, np.asarray(gamma), c, inp.seg_offsets, inp.seg_stream, scheme, np.ones(3), y_ref)

    # the value the GPU search reports is the oracle's objective at that point (fp32 reference product and
    # accumulation order aside)
    assert abs(res["objective"] - J(res["gamma"], res["clip"])) <= 1e-2 * res["objective"]
    # and its point is as good as the oracle's (equal unless two candidates tie within that noise)
    assert J(res["gamma"], res["clip"]) <= ref["objective"] * 1.02
    assert res["evaluations"] == ref["evaluations"] or abs(res["evaluations"] - ref["evaluations"]) <= len(STEPS) * 3 * 2
    last, where = rd.rudder_device_status()
    assert last == 0, (last, where)
