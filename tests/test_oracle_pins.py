"""Pins for the oracle's method arithmetic.  The paper prints no numeric worked example of a
quantized linear, so the oracle is pinned to what the paper's equations and plain mathematics fix:

  P1  identity scales reduce it to a textbook per-token-absmax x per-group quantized matmul
      (written here independently, vectorised numpy) -- bit for bit on codes, accumulators, r
  P2  power-of-two scales commute exactly with quantisation (Eq. 6 cancellation; App. C.1)
  P3  tiny shapes: fp64 dequantise-then-matmul by triple loop, and Eq. 8's literal form
  P4  rounding-error bound of Eq. 1: |v - q Delta| <= Delta / 2 inside the clip range, q = +-q_max
      outside; effective clip c / gamma_s and step c / (q_max gamma_s) per stream (App. C.1)
  P5  rows are independent: permutations / subsets give identical bits
  P7  degenerate rows
  P8  Eq. 3 error falls with more bits; the equivalent transform cancels in full precision
"""
import numpy as np
import pytest

import oracle
import workloads as wl

PT, ST = oracle.RANGE_PER_TOKEN, oracle.RANGE_STATIC


def _f32(h):
    return wl.bf16_bits_to_f32(h)


def _fp16_to_f32(s):
    return s.view(np.float16).astype(np.float32)


def _static_clip(inp, dinv, q=99.9):
    """clip[t] = q-th percentile of |v| over all rows at step t (test-side arithmetic)."""
    X = _f32(inp.X_bf16)
    row_stream = np.repeat(inp.seg_stream, np.diff(inp.seg_offsets))
    clip = np.empty(inp.T, np.float32)
    for t in range(inp.T):
        v = (X * dinv[None, :]) * inp.gamma[t, row_stream][:, None]
        clip[t] = np.percentile(np.abs(v), q)
    return clip


# ------------------------------------------------------------------------------------------ P1
def _textbook_quantized_matmul(Xf, W, G, qmax):
    """Per-token absmax activations x per-(row, group) absmax INT4 weights, fp32 numpy."""
    N, K = W.shape
    Wg = W.reshape(N, K // G, G)
    dw = (np.abs(Wg).max(-1) / np.float32(7)).astype(np.float16).astype(np.float32)
    qw = np.clip(np.rint(Wg / dw[..., None]), -7, 7).astype(np.int32)
    a = np.abs(Xf).max(1)
    inv = np.float32(qmax) / a
    q = np.clip(np.rint(Xf * inv[:, None]), -qmax, qmax).astype(np.int32)
    r = a / np.float32(qmax)
    acc = np.einsum("mgk,ngk->gmn", q.reshape(-1, K // G, G), qw)
    y = (acc.astype(np.float64) * dw.T.astype(np.float64)[:, None, :]).sum(0) * r.astype(np.float64)[:, None]
    return q, r, qw.reshape(N, K), dw, acc, y


@pytest.mark.parametrize("scheme,qmax", [("w4a8", 127), ("w4a4", 7)])
@pytest.mark.parametrize("G", [64, 128, 256])
def test_p1_identity_scales_reduce_to_textbook(scheme, qmax, G):
    inp = wl.tiny(seed=11, M=24, K=256, N=96, T=1)
    ones_d = np.ones(inp.K, np.float32)
    ones_g = np.ones((1, inp.S), np.float32)
    pw = oracle.pack_int4(inp.W, ones_d, G)
    out = oracle.rudder_linear(inp.X_bf16, pw, ones_g, None, 0, PT, inp.seg_offsets, inp.seg_stream, scheme)
    q, r, qw, dw, acc, y = _textbook_quantized_matmul(_f32(inp.X_bf16), inp.W, G, qmax)
    assert np.array_equal(pw["qw"], qw)
    assert np.array_equal(_fp16_to_f32(pw["scales"]), dw)
    assert np.array_equal(out["codes"], q)
    assert np.array_equal(out["r"].view(np.uint32), r.astype(np.float32).view(np.uint32))
    assert np.array_equal(oracle.accumulate_int(out["codes"], pw["qw"], G), acc)
    np.testing.assert_allclose(out["y64"], y, rtol=1e-12, atol=1e-12)
    # canonical nibble packing: low nibble = even k, two's complement
    lo = (pw["packed"] & 0xF).astype(np.int8)
    hi = (pw["packed"] >> 4).astype(np.int8)
    lo = np.where(lo > 7, lo - 16, lo)
    hi = np.where(hi > 7, hi - 16, hi)
    assert np.array_equal(lo, qw[:, 0::2]) and np.array_equal(hi, qw[:, 1::2])


# ------------------------------------------------------------------------------------------ P2
def test_p2_uniform_power_of_two_channel_scale_commutes():
    inp = wl.tiny(seed=12, M=16, K=256, N=64, T=2)
    base = oracle.pack_int4(inp.W, np.ones(inp.K, np.float32), 64)
    y0 = oracle.rudder_linear(inp.X_bf16, base, inp.gamma, None, 1, PT, inp.seg_offsets, inp.seg_stream,
                              "w4a8", inp.bias)
    for p in (-3, 2, 5):
        pw = oracle.pack_int4(inp.W, np.full(inp.K, 2.0 ** p, np.float32), 64)
        assert np.array_equal(pw["qw"], base["qw"])
        assert np.array_equal(_fp16_to_f32(pw["scales"]), _fp16_to_f32(base["scales"]) * np.float32(2.0 ** p))
        y = oracle.rudder_linear(inp.X_bf16, pw, inp.gamma, None, 1, PT, inp.seg_offsets, inp.seg_stream,
                                 "w4a8", inp.bias)
        assert np.array_equal(y["codes"], y0["codes"])
        assert np.array_equal(y["y"], y0["y"])            # Eq. 6: D^-1 and D cancel exactly


@pytest.mark.parametrize("scheme", ["w4a8", "w4a4", "nvfp4"])
def test_p2_power_of_two_gains_per_token(scheme):
    inp = wl.tiny(seed=13, M=16, K=256, N=64, T=1)
    pw = oracle.pack_nvfp4(inp.W, inp.d) if scheme == "nvfp4" else oracle.pack_int4(inp.W, inp.d, 64)
    ones = np.ones((1, inp.S), np.float32)
    pow2 = np.array([[2.0, 0.25, 8.0]], np.float32)
    a = oracle.rudder_linear(inp.X_bf16, pw, ones, None, 0, PT, inp.seg_offsets, inp.seg_stream, scheme, inp.bias)
    b = oracle.rudder_linear(inp.X_bf16, pw, pow2, None, 0, PT, inp.seg_offsets, inp.seg_stream, scheme, inp.bias)
    assert np.array_equal(a["codes"], b["codes"])
    assert np.array_equal(a["r"], b["r"])                  # the inverse gain compensates exactly
    assert np.array_equal(a["y"], b["y"])


@pytest.mark.parametrize("scheme", ["w4a8", "w4a4"])
def test_p2_static_gain_equals_per_stream_clip(scheme):
    """App. C.1: with gain gamma_s stream s behaves as clip c / gamma_s.  For gamma_s = 2^p the rows
    of stream s are bit-identical to a one-segment call with gamma = 1 and clip c / gamma_s."""
    inp = wl.tiny(seed=14, M=24, K=256, N=64, T=1)
    pw = oracle.pack_int4(inp.W, inp.d, 64)
    pow2 = np.array([[4.0, 0.5, 2.0]], np.float32)
    c = np.array([3.0], np.float32)
    full = oracle.rudder_linear(inp.X_bf16, pw, pow2, c, 0, ST, inp.seg_offsets, inp.seg_stream, scheme, inp.bias)
    assert np.abs(full["codes"]).max() == (127 if scheme == "w4a8" else 7)      # clipping is active
    for s in range(len(inp.seg_stream)):
        lo, hi = inp.seg_offsets[s], inp.seg_offsets[s + 1]
        g = pow2[0, inp.seg_stream[s]]
        part = oracle.rudder_linear(inp.X_bf16[lo:hi], pw, np.ones((1, 1), np.float32), c / g, 0, ST,
                                    np.array([0, hi - lo], np.int32), np.array([0], np.int32), scheme, inp.bias)
        assert np.array_equal(part["codes"], full["codes"][lo:hi])
        assert np.array_equal(part["r"], full["r"][lo:hi])
        assert np.array_equal(part["y"], full["y"][lo:hi])


# ------------------------------------------------------------------------------------------ P3
@pytest.mark.parametrize("scheme,qmax", [("w4a8", 127), ("w4a4", 7)])
@pytest.mark.parametrize("mode", [PT, ST])
@pytest.mark.parametrize("K,G", [(128, 64), (256, 128), (128, 128)])
def test_p3_fp64_bruteforce_and_eq8(scheme, qmax, mode, K, G):
    inp = wl.tiny(seed=15 + K + G, M=6, K=K, N=64, T=3)
    pw = oracle.pack_int4(inp.W, inp.d, G)
    clip = _static_clip(inp, pw["dinv"]) if mode == ST else None
    step = 2
    out = oracle.rudder_linear(inp.X_bf16, pw, inp.gamma, clip, step, mode, inp.seg_offsets, inp.seg_stream,
                               scheme, inp.bias)
    dw = _fp16_to_f32(pw["scales"]).astype(np.float64)
    row_stream = np.repeat(inp.seg_stream, np.diff(inp.seg_offsets))
    Y = np.zeros((inp.M, inp.N))
    Y8 = np.zeros((inp.M, inp.N))
    X = _f32(inp.X_bf16)
    for i in range(inp.M):
        g = np.float32(inp.gamma[step, row_stream[i]])
        v = (X[i] * pw["dinv"]) * g
        a = np.float32(clip[step]) if mode == ST else np.abs(v).max()
        delta_x = a / np.float32(qmax)                       # Delta_X = c / q_max
        for j in range(inp.N):
            s = 0.0
            s8 = 0.0
            for k in range(K):
                xh = float(out["codes"][i, k]) * float(out["r"][i])        # dequantised activation
                wh = float(pw["qw"][j, k]) * dw[j, k // G]                 # dequantised weight
                s += xh * wh
                s8 += (float(delta_x) * float(out["codes"][i, k])) * wh    # Q(gamma X~; c) W^
            Y[i, j] = s + float(inp.bias[j])
            Y8[i, j] = s8 / float(g) + float(inp.bias[j])                  # gamma^-1 ( ... ), Eq. 8
    np.testing.assert_allclose(out["y64"], Y, rtol=1e-11, atol=1e-11)
    np.testing.assert_allclose(out["y64"], Y8, rtol=1e-6, atol=1e-7)       # r_i is an fp32 quotient
    # the bf16 output is the rounding of (nearly) the same number
    yb = _f32(out["y"]).astype(np.float64)
    assert np.all(np.abs(yb - out["y64"]) <= np.abs(out["y64"]) * 2.0 ** -8 + 1e-6)


def test_p3_nvfp4_bruteforce():
    inp = wl.tiny(seed=16, M=5, K=128, N=48, T=2)
    pw = oracle.pack_nvfp4(inp.W, inp.d)
    out = oracle.rudder_linear(inp.X_bf16, pw, inp.gamma, None, 1, PT, inp.seg_offsets, inp.seg_stream,
                               "nvfp4", inp.bias)
    vals = np.array([0, .5, 1, 1.5, 2, 3, 4, 6, -0.0, -.5, -1, -1.5, -2, -3, -4, -6])
    A = vals[out["codes"]] * np.repeat(np.array([[oracle.ue4m3_decode(int(b)) for b in row] for row in out["sb"]]), 16, 1)
    Wd = vals[pw["e2m1"]] * np.repeat(np.array([[oracle.ue4m3_decode(int(b)) for b in row] for row in pw["sb"]]), 16, 1)
    Y = np.zeros((inp.M, inp.N))
    for i in range(inp.M):
        for j in range(inp.N):
            s = 0.0
            for k in range(inp.K):
                s += A[i, k] * Wd[j, k]
            Y[i, j] = s * float(np.float32(out["r"][i]) * np.float32(pw["tensor_scale"])) + float(inp.bias[j])
    np.testing.assert_allclose(out["y64"], Y, rtol=1e-11, atol=1e-11)
    # and it approximates the full-precision layer (4-bit x 4-bit: coarse, but far from garbage)
    ref = _f32(inp.X_bf16).astype(np.float64) @ inp.W.astype(np.float64).T + inp.bias
    err = np.linalg.norm(out["y64"] - ref) / np.linalg.norm(ref)
    assert err < 0.25


# ------------------------------------------------------------------------------------------ P4
@pytest.mark.parametrize("qmax", [127, 7])
def test_p4_rounding_bound_per_token(qmax):
    inp = wl.tiny(seed=17, M=32, K=512, N=64, T=2)
    dinv = (np.float32(1) / inp.d).astype(np.float32)
    codes, r = oracle.quantize_int(inp.X_bf16, dinv, inp.gamma, None, 1, PT, inp.seg_offsets, inp.seg_stream, qmax)
    row_stream = np.repeat(inp.seg_stream, np.diff(inp.seg_offsets))
    g = inp.gamma[1, row_stream].astype(np.float64)
    v = (_f32(inp.X_bf16) * dinv[None, :]).astype(np.float64) * g[:, None]
    delta = r.astype(np.float64) * g                          # Delta_i = r_i gamma
    assert np.all(np.abs(v - codes * delta[:, None]) <= delta[:, None] / 2 * (1 + 2.0 ** -18))
    assert np.all(np.abs(codes).max(1) == qmax)               # absmax element hits the end code
    np.testing.assert_allclose(delta * qmax, np.abs(v).max(1), rtol=1e-6)


@pytest.mark.parametrize("qmax", [127, 7])
def test_p4_static_effective_range_per_stream(qmax):
    """App. C.1: after compensation stream s has clip c / gamma_s and step c / (q_max gamma_s)."""
    inp = wl.tiny(seed=18, M=48, K=512, N=64, T=2)
    dinv = (np.float32(1) / inp.d).astype(np.float32)
    clip = np.array([2.5, 1.75], np.float32)
    step = 1
    codes, r = oracle.quantize_int(inp.X_bf16, dinv, inp.gamma, clip, step, ST, inp.seg_offsets, inp.seg_stream, qmax)
    row_stream = np.repeat(inp.seg_stream, np.diff(inp.seg_offsets))
    xt = (_f32(inp.X_bf16) * dinv[None, :]).astype(np.float64)           # X~ = X D^-1
    for s in range(inp.S):
        rows = np.where(row_stream == s)[0]
        g = float(inp.gamma[step, s])
        c_eff = float(clip[step]) / g
        step_eff = c_eff / qmax
        np.testing.assert_allclose(r[rows], step_eff, rtol=1e-6)
        xh = codes[rows].astype(np.float64) * r[rows, None]              # compensated dequantised X~
        inside = np.abs(xt[rows]) <= c_eff * (1 - 1e-6)
        assert np.all(np.abs(xh - xt[rows])[inside] <= step_eff / 2 * (1 + 1e-5))
        outside = np.abs(xt[rows]) > c_eff * (1 + 1e-6)
        assert outside.any()
        assert np.all(codes[rows][outside] == np.sign(xt[rows][outside]) * qmax)


def test_p4_weight_rounding_bound():
    inp = wl.tiny(seed=19, M=4, K=512, N=128)
    for G in (64, 128, 512):
        pw = oracle.pack_int4(inp.W, inp.d, G)
        V = (inp.W * inp.d[None, :]).astype(np.float64)
        dw = np.repeat(_fp16_to_f32(pw["scales"]).astype(np.float64), G, 1)
        assert np.abs(pw["qw"]).max() == 7 and pw["qw"].min() >= -7
        err = np.abs(V - pw["qw"] * dw)
        unclipped = np.abs(V / dw) <= 7.0
        assert np.all(err[unclipped] <= dw[unclipped] / 2 * (1 + 1e-6))
        # fp16 rounding of the scale may push the absmax element just past 7 Delta: error stays < Delta
        assert np.all(err <= dw * (0.5 + 7 * 2.0 ** -11 + 1e-6))
        np.testing.assert_array_equal(pw["dinv"], (np.float32(1) / inp.d).astype(np.float32))


def test_p4_nvfp4_error_bound():
    inp = wl.tiny(seed=20, M=16, K=256, N=64, T=1)
    dinv = (np.float32(1) / inp.d).astype(np.float32)
    e, sb, r = oracle.quantize_nvfp4(inp.X_bf16, dinv, inp.gamma, None, 0, PT, inp.seg_offsets, inp.seg_stream)
    vals = np.array([0, .5, 1, 1.5, 2, 3, 4, 6, -0.0, -.5, -1, -1.5, -2, -3, -4, -6])
    sbd = np.array([[oracle.ue4m3_decode(int(b)) for b in row] for row in sb])
    xh = vals[e] * np.repeat(sbd, 16, 1) * r[:, None].astype(np.float64)
    xt = (_f32(inp.X_bf16) * dinv[None, :]).astype(np.float64)
    # per block: largest E2M1 spacing is 2 (between 4 and 6) -> error <= 1 block-scale unit, plus the
    # UE4M3 rounding of the block scale (relative 2^-4) on the block's absmax element.
    unit = np.repeat(sbd, 16, 1) * r[:, None].astype(np.float64)
    amax_b = np.repeat(np.abs(xt).reshape(16, -1, 16).max(-1), 16, 1)
    assert np.all(np.abs(xh - xt) <= unit * 1.0 + amax_b * 2.0 ** -4 + 1e-12)
    assert np.linalg.norm(xh - xt) / np.linalg.norm(xt) < 0.12
    assert sb.max() <= 0x7E and e.max() <= 15


# ------------------------------------------------------------------------------------------ P4 (NVFP4 recipe)
# The paper only names NVFP4, so the recipe is a reading; what the reading *means* is still fixed by
# mathematics: a block's scale is the block maximum divided by the largest E2M1 magnitude (6), rounded
# to UE4M3 (3 mantissa bits: relative error at most 2^-4), so the block's largest element lands in
# 6 x [1/(1+2^-4), 1/(1-2^-4)] = [5.65, 6.4] and must take the end code +-6; every other element is the
# nearest E2M1 value of (value / outer scale) / block scale; the outer scale maps the tensor's (row's)
# largest magnitude to 6 x 448 = 2688.  A wrong divisor, a dropped outer scale or a wrong table fails here.
_E2M1 = np.array([0, .5, 1, 1.5, 2, 3, 4, 6])


def _nvfp4_check(V, e, sb, outer_scale, what):
    """V fp64 [R, K] (the values that were quantised), e codes [R, K], sb UE4M3 bytes [R, K/16],
    outer_scale fp32 [R] (the fp32 scale of each row: tensor scale or row scale)."""
    R, K = V.shape
    sbd = np.array([oracle.ue4m3_decode(b) for b in range(127)])[sb]                 # decoded block scales
    amax_b = np.abs(V).reshape(R, K // 16, 16).max(-1)
    # (d) outer scale x 2688 = largest magnitude of the row / tensor, to fp32 rounding
    live = outer_scale > 0
    # (a) normal, unsaturated block scale -> the block's absmax element carries code 7 (+-6)
    normal = (sb >= 8) & (sb <= 0x7E)
    mag = (e & 7).reshape(R, K // 16, 16)
    arg = np.abs(V).reshape(R, K // 16, 16).argmax(-1)
    top_code = np.take_along_axis(mag, arg[..., None], -1)[..., 0]
    assert normal.sum() > 0.5 * normal.size, what
    assert np.all(top_code[normal] == 7), f"{what}: a block maximum is not encoded as +-6"
    # (b) the dequantised block maximum is the block's true maximum within the UE4M3 rounding (2^-4)
    deq_top = 6.0 * sbd * outer_scale[:, None].astype(np.float64)
    unsat = normal & (sb < 0x7E)
    assert np.all(np.abs(deq_top - amax_b)[unsat] <= amax_b[unsat] * (2.0 ** -4) * (1 + 1e-5)), what
    # (c) every code is the nearest E2M1 value of (V / outer) / block scale (near-ties left out: the oracle
    #     forms the quotient in fp32)
    with np.errstate(divide="ignore", invalid="ignore"):
        u = V / outer_scale[:, None].astype(np.float64) / np.repeat(sbd, 16, 1)
    ok = np.isfinite(u)
    au = np.minimum(np.abs(u), 6.0)
    nearest = np.abs(au[..., None] - _E2M1).argmin(-1)
    mids = np.array([.25, .75, 1.25, 1.75, 2.5, 3.5, 5.0])
    near_tie = (np.abs(au[..., None] - mids) <= 1e-5 * np.maximum(au[..., None], 1.0)).any(-1)
    sel = ok & ~near_tie
    assert sel.mean() > 0.9, what
    assert np.array_equal((e & 7)[sel], nearest[sel]), f"{what}: a code is not the nearest E2M1 value"
    sign_ok = ((e >> 3) == (V < 0))[sel & ((e & 7) != 0)]
    assert sign_ok.all(), what
    # zero block scale -> zero codes
    assert not (e.reshape(R, K // 16, 16)[sb == 0]).any(), what
    return live


def test_p4_nvfp4_weight_recipe():
    inp = wl.tiny(seed=31, M=4, K=512, N=96)
    pw = oracle.pack_nvfp4(inp.W, inp.d)
    V32 = inp.W * inp.d[None, :]                                   # fp32 product, as the fold defines it
    V = V32.astype(np.float64)
    ts = np.float32(pw["tensor_scale"])
    np.testing.assert_allclose(float(ts) * 2688.0, np.abs(V32).max(), rtol=2e-7)     # (d)
    _nvfp4_check(V, pw["e2m1"], pw["sb"], np.full(inp.N, ts, np.float32), "weights")
    # the block that holds the tensor's largest magnitude saturates the scale format: 448, code 0x7E
    j, k = np.unravel_index(np.abs(V32).argmax(), V32.shape)
    assert pw["sb"][j, k // 16] == 0x7E and (pw["e2m1"][j, k] & 7) == 7
    # canonical nibble packing: low nibble = even k
    assert np.array_equal(pw["packed"], (pw["e2m1"][:, 0::2] | (pw["e2m1"][:, 1::2] << 4)).astype(np.uint8))


@pytest.mark.parametrize("mode", [PT, ST])
def test_p4_nvfp4_activation_recipe(mode):
    inp = wl.tiny(seed=32, M=24, K=512, N=64, T=2)
    dinv = (np.float32(1) / inp.d).astype(np.float32)
    clip = _static_clip(inp, dinv) if mode == ST else None
    step = 1
    e, sb, r = oracle.quantize_nvfp4(inp.X_bf16, dinv, inp.gamma, clip, step, mode, inp.seg_offsets, inp.seg_stream)
    row_stream = np.repeat(inp.seg_stream, np.diff(inp.seg_offsets))
    g = inp.gamma[step, row_stream]
    v32 = (_f32(inp.X_bf16) * dinv[None, :]) * g[:, None]          # gamma X D^-1 in fp32, two rounded products
    a = np.full(inp.M, clip[step], np.float32) if mode == ST else np.abs(v32).max(1)
    s_row = (r.astype(np.float64) * g.astype(np.float64)).astype(np.float32)         # r_i = s_i / gamma
    np.testing.assert_allclose(s_row.astype(np.float64) * 2688.0, a, rtol=3e-7)      # (d)
    if mode == ST:
        # values beyond the threshold saturate: block scale 448 where the block maximum exceeds c, codes +-6
        v = v32.astype(np.float64)
        over = np.abs(v) > float(clip[step]) * (1 + 1e-6)
        assert over.any()
        assert np.all((e & 7)[over] == 7)
        assert np.all(sb[np.abs(v).reshape(inp.M, -1, 16).max(-1) > float(clip[step]) * (1 + 1e-6)] == 0x7E)
        keep = np.abs(v).reshape(inp.M, -1, 16).max(-1) <= float(clip[step])
        # check the recipe on the blocks that do not clip
        vv = np.where(np.repeat(keep, 16, 1), v, 0.0)
        ee = np.where(np.repeat(keep, 16, 1), e, 0)
        ss = np.where(keep, sb, 0)
        _nvfp4_check(vv, ee.astype(np.uint8), ss.astype(np.uint8), s_row, "activations (static)")
    else:
        _nvfp4_check(v32.astype(np.float64), e, sb, s_row, "activations (per token)")
        # the row's largest element: block scale 448, code +-6 -- it dequantises to a_i exactly
        top = np.abs(v32).argmax(1)
        assert np.all(sb[np.arange(inp.M), top // 16] == 0x7E)
        assert np.all((e[np.arange(inp.M), top] & 7) == 7)


# ------------------------------------------------------------------------------------------ P5
@pytest.mark.parametrize("scheme", ["w4a8", "w4a4", "nvfp4"])
@pytest.mark.parametrize("mode", [PT, ST])
def test_p5_rows_are_independent(scheme, mode):
    inp = wl.tiny(seed=21, M=40, K=256, N=64, T=2)
    pw = oracle.pack_nvfp4(inp.W, inp.d) if scheme == "nvfp4" else oracle.pack_int4(inp.W, inp.d, 64)
    clip = _static_clip(inp, pw["dinv"]) if mode == ST else None
    full = oracle.rudder_linear(inp.X_bf16, pw, inp.gamma, clip, 1, mode, inp.seg_offsets, inp.seg_stream,
                                scheme, inp.bias)
    rows = np.array([39, 0, 19, 20, 7, 29, 30], np.int32)
    sub = oracle.rudder_linear(inp.X_bf16, pw, inp.gamma, clip, 1, mode, inp.seg_offsets, inp.seg_stream,
                               scheme, inp.bias, rows=rows)
    for k in ("codes", "r", "y"):
        assert np.array_equal(sub[k], full[k][rows])
    # reversing the rows (and the segments with them) reverses the outputs bit for bit
    rev_off = np.concatenate([[0], np.cumsum(np.diff(inp.seg_offsets)[::-1])]).astype(np.int32)
    rev = oracle.rudder_linear(inp.X_bf16[::-1].copy(), pw, inp.gamma, clip, 1, mode, rev_off,
                               inp.seg_stream[::-1].copy(), scheme, inp.bias)
    for k in ("codes", "r", "y"):
        assert np.array_equal(rev[k], full[k][::-1])


# ------------------------------------------------------------------------------------------ P7
@pytest.mark.parametrize("scheme,qmax", [("w4a8", 127), ("w4a4", 7), ("nvfp4", None)])
def test_p7_degenerate_rows(scheme, qmax):
    inp = wl.tiny(seed=22, M=6, K=128, N=64, T=1)
    X = inp.X_bf16.copy()
    X[1] = 0                                                   # all-zero row
    X[4] = 0
    X[4, 37] = wl.f32_to_bf16_bits(np.array([-3.0], np.float32))[0]   # a single non-zero element
    pw = oracle.pack_nvfp4(inp.W, inp.d) if scheme == "nvfp4" else oracle.pack_int4(inp.W, inp.d, 64)
    out = oracle.rudder_linear(X, pw, inp.gamma, None, 0, PT, inp.seg_offsets, inp.seg_stream, scheme, inp.bias)
    assert not out["codes"][1].any() and out["r"][1] == 0.0
    assert np.array_equal(out["y"][1], wl.f32_to_bf16_bits(inp.bias))   # zero row -> bias
    nz = np.nonzero(out["codes"][4])[0]
    assert list(nz) == [37]
    if qmax:
        assert out["codes"][4, 37] == -qmax
    else:
        assert out["codes"][4, 37] == (8 | 7) and out["sb"][4, 37 // 16] == 0x7E   # -6 x 448 x s_i
    # zero weights -> zero scales, zero codes, output = bias
    Wz = inp.W.copy()
    Wz[3] = 0
    pz = oracle.pack_nvfp4(Wz, inp.d) if scheme == "nvfp4" else oracle.pack_int4(Wz, inp.d, 64)
    oz = oracle.rudder_linear(inp.X_bf16, pz, inp.gamma, None, 0, PT, inp.seg_offsets, inp.seg_stream, scheme, inp.bias)
    assert np.array_equal(oz["y"][:, 3], np.full(inp.M, wl.f32_to_bf16_bits(inp.bias[3:4])[0]))


# ------------------------------------------------------------------------------------------ P8
def test_p8_local_error_falls_with_bits_and_transform_cancels():
    """Eq. 3 error of the quantized layer against fp64 X W^T + b; Eq. 6: D only reshapes the error."""
    inp = wl.tiny(seed=23, M=64, K=512, N=128, T=1, outlier_frac=0.01)
    ref = _f32(inp.X_bf16).astype(np.float64) @ inp.W.astype(np.float64).T + inp.bias

    def eps(scheme, d):
        pw = oracle.pack_nvfp4(inp.W, d) if scheme == "nvfp4" else oracle.pack_int4(inp.W, d, 64)
        y = oracle.rudder_linear(inp.X_bf16, pw, inp.gamma, None, 0, PT, inp.seg_offsets, inp.seg_stream,
                                 scheme, inp.bias)["y64"]
        return np.linalg.norm(y - ref) / np.linalg.norm(ref)

    ones = np.ones(inp.K, np.float32)
    e8, e4, ef = eps("w4a8", ones), eps("w4a4", ones), eps("nvfp4", ones)
    assert e8 < 0.2 and e8 < e4 and ef < e4
    assert abs(eps("w4a8", ones * 4) - e8) < 1e-9              # power-of-two D: exactly the same error
    assert eps("w4a8", inp.d) < 1.0                            # random D: still a sane approximation


def test_argument_errors():
    inp = wl.tiny(seed=24, M=8, K=128, N=64, T=2)
    dinv = np.ones(inp.K, np.float32)
    with pytest.raises(ValueError):      # step out of range
        oracle.quantize_int(inp.X_bf16, dinv, inp.gamma, None, 2, PT, inp.seg_offsets, inp.seg_stream, 127)
    with pytest.raises(ValueError):      # static mode without clip
        oracle.quantize_int(inp.X_bf16, dinv, inp.gamma, None, 0, ST, inp.seg_offsets, inp.seg_stream, 127)
    with pytest.raises(ValueError):      # segments do not cover M
        oracle.quantize_int(inp.X_bf16, dinv, inp.gamma, None, 0, PT, inp.seg_offsets[:-1], inp.seg_stream[:-1], 127)
    with pytest.raises(ValueError):      # stream id out of range
        oracle.quantize_int(inp.X_bf16, dinv, inp.gamma, None, 0, PT, inp.seg_offsets, inp.seg_stream + 5, 127)
