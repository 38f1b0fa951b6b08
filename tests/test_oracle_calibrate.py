"""Pins of the oracle's toy calibrator (Eq. 9): closed forms and invariants that do not pass through the
search itself, then the properties the search must have whatever it finds."""
import numpy as np

import oracle
import workloads as wl
from oracle import calibrate as oc


def _case(seed=5, M=96, K=256, N=64):
    inp = wl.tiny(seed=seed, M=M, K=K, N=N, T=1)
    pw = oracle.pack_int4(inp.W, inp.d, 64)
    X = wl.bf16_bits_to_f32(inp.X_bf16).astype(np.float64)
    v = np.abs(X * pw["dinv"][None, :].astype(np.float64))
    cs = [float(np.quantile(v, q)) for q in (0.99, 0.995, 0.999, 1.0)]
    return inp, pw, cs


def test_reference_output_is_the_dequantized_product():
    inp, pw, _ = _case()
    y_ref = oc.reference_output(inp.X_bf16, pw)
    # element (i, j) by hand: sum_k x_ik dinv_k q_jk scale_j,g(k)
    X = wl.bf16_bits_to_f32(inp.X_bf16).astype(np.float64)
    for i, j in [(0, 0), (17, 5), (95, 63)]:
        s = 0.0
        for k in range(256):
            s += X[i, k] * float(pw["dinv"][k]) * int(pw["qw"][j, k]) * oracle.fp16_decode(int(pw["scales"][j, k // 64]))
        assert abs(y_ref[i, j] - s) <= 1e-9 * max(1.0, abs(s))


def test_objective_with_a_huge_threshold_is_the_reference_energy():
    # c far above every |v|: all codes are 0, the layer outputs 0 (no bias), J = sum_s omega_s/n_s ||Yref_s||^2
    inp, pw, _ = _case()
    y_ref = oc.reference_output(inp.X_bf16, pw)
    row_stream, n = oc.stream_rows(inp.seg_offsets, inp.seg_stream, 3)
    omega = np.array([1.0, 2.0, 0.5])
    want = sum(omega[s] / n[s] * (y_ref[row_stream == s] ** 2).sum() for s in range(3))
    got = oc.objective(inp.X_bf16, pw, np.ones(3), 1e12, inp.seg_offsets, inp.seg_stream, "w4a8", omega, y_ref)
    assert abs(got - want) <= 1e-12 * want


def test_projection_meets_the_constraint_and_keeps_ratios():
    n = np.array([48.0, 24.0, 24.0])
    g = oc.project([1.7, 0.6, 1.1], n)
    assert abs((n * np.log(g)).sum()) < 1e-12
    assert np.allclose(g / g[0], np.array([1.7, 0.6, 1.1]) / 1.7)


def test_search_properties():
    inp, pw, cs = _case()
    steps = [2 ** -0.5, 2 ** -0.25, 2 ** 0.25, 2 ** 0.5]
    y_ref = oc.reference_output(inp.X_bf16, pw)
    start = min(oc.objective(inp.X_bf16, pw, np.ones(3), c, inp.seg_offsets, inp.seg_stream, "w4a8", np.ones(3), y_ref) for c in cs)
    r1 = oc.calibrate(inp.X_bf16, pw, inp.seg_offsets, inp.seg_stream, 3, "w4a8", cs, steps, sweeps=1)
    r2 = oc.calibrate(inp.X_bf16, pw, inp.seg_offsets, inp.seg_stream, 3, "w4a8", cs, steps, sweeps=2)
    _, n = oc.stream_rows(inp.seg_offsets, inp.seg_stream, 3)
    for r in (r1, r2):
        assert abs((n * np.log(r["gamma"])).sum()) < 1e-9
        assert r["gamma"].min() >= 0.5 and r["gamma"].max() <= 2.0
        assert r["clip"] in cs
        # the value it reports is the objective at the point it reports
        assert abs(r["objective"] - oc.objective(inp.X_bf16, pw, r["gamma"], r["clip"], inp.seg_offsets, inp.seg_stream,
                                                 "w4a8", np.ones(3), y_ref)) <= 1e-12 * r["objective"]
    assert r2["objective"] <= r1["objective"] <= start
    assert r1["objective"] < start        # on this case (streams scaled x1, x0.5, x2) gains do help


def test_stream_weights_steer_the_trade_off():
    # a large weight on one stream must not increase that stream's own error
    inp, pw, cs = _case(seed=9)
    steps = [2 ** -0.5, 2 ** -0.25, 2 ** 0.25, 2 ** 0.5]
    y_ref = oc.reference_output(inp.X_bf16, pw)
    row_stream, n = oc.stream_rows(inp.seg_offsets, inp.seg_stream, 3)

    def stream_err(r, s):
        one = np.zeros(3)
        one[s] = 1.0
        return oc.objective(inp.X_bf16, pw, r["gamma"], r["clip"], inp.seg_offsets, inp.seg_stream, "w4a8", one, y_ref)

    uni = oc.calibrate(inp.X_bf16, pw, inp.seg_offsets, inp.seg_stream, 3, "w4a8", cs, steps)
    for s in range(3):
        om = np.ones(3)
        om[s] = 100.0
        fav = oc.calibrate(inp.X_bf16, pw, inp.seg_offsets, inp.seg_stream, 3, "w4a8", cs, steps, omega=om)
        assert stream_err(fav, s) <= stream_err(uni, s) * (1 + 1e-9)
