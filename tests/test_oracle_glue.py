"""Pins of the oracle's GELU (the BF16 glue of a chained block) against the mathematics, over every finite
bf16 input: the tanh form it approximates, the erf form it stands for, exact special values, and the
approximant's own coefficients."""
import math

import numpy as np

from oracle import glue

ALL = np.arange(65536, dtype=np.uint16)
with np.errstate(invalid="ignore"):
    X = glue.bf16_to_f32(ALL).astype(np.float64)
FINITE = np.isfinite(X)


def _ulp_bf16(y):
    return np.maximum(np.abs(y), 2.0 ** -126) * 2.0 ** -8


def test_pade_coefficients_reproduce_tanh():
    u = np.linspace(-3.0, 3.0, 6001)
    assert np.abs(glue.pade_tanh(u) - np.tanh(u)).max() < 1e-6        # a wrong coefficient misses by orders of magnitude
    u = np.linspace(-5.0, 5.0, 10001)
    assert np.abs(glue.pade_tanh(u) - np.tanh(u)).max() < 1.1e-4


def test_gelu_tracks_the_tanh_form_on_every_bf16_input():
    x = X[FINITE]
    with np.errstate(over="ignore"):
        want = 0.5 * x * (1.0 + np.tanh(0.7978845608028654 * (x + 0.044715 * x ** 3)))
    got = glue.bf16_to_f32(glue.gelu_bf16(ALL[FINITE])).astype(np.float64)
    ok = np.abs(got - want) <= 2.5e-4 + _ulp_bf16(want)
    assert ok.all(), (x[~ok][:5], got[~ok][:5], want[~ok][:5])


def test_gelu_tracks_the_erf_form():
    x = X[FINITE & (np.abs(X) < 1e4)]
    want = np.array([0.5 * v * (1.0 + math.erf(v / math.sqrt(2.0))) for v in x])
    got = glue.bf16_to_f32(glue.gelu_bf16(ALL[FINITE & (np.abs(X) < 1e4)])).astype(np.float64)
    assert (np.abs(got - want) <= 7e-4 + _ulp_bf16(want)).all()


def test_special_values_and_shape():
    g = lambda v: float(glue.bf16_to_f32(glue.gelu_bf16(glue.f32_to_bf16(np.array([v], np.float32))))[0])
    assert g(0.0) == 0.0
    for v in (6.0, 17.5, 1024.0, 2.0 ** 100, 2.0 ** 127):     # bf16 values; x^3 overflows for the last two
        assert g(v) == v                         # tanh saturated: (x/2) * 2 is exact
    for v in (-6.0, -17.5, -1024.0):
        assert g(v) == 0.0                       # x/2 * (1 - 1)
    xs = glue.bf16_to_f32(ALL[(X >= 0) & FINITE])
    ys = glue.bf16_to_f32(glue.gelu_bf16(ALL[(X >= 0) & FINITE]))
    order = np.argsort(xs, kind="stable")
    assert (np.diff(ys[order]) >= 0).all()       # monotone on x >= 0
    assert math.isnan(g(float("nan")))


def test_bf16_rounding_is_nearest_even():
    # exactly half way between two bf16 values: ties go to the even mantissa
    lo, hi = 0x3F80, 0x3F81                      # 1.0 and the next bf16
    mid = np.array([0x3F808000], np.uint32).view(np.float32)
    assert int(glue.f32_to_bf16(mid)[0]) == lo   # tie -> even (0x3F80)
    mid2 = np.array([0x3F818000], np.uint32).view(np.float32)
    assert int(glue.f32_to_bf16(mid2)[0]) == 0x3F82
    assert int(glue.f32_to_bf16(np.array([0x3F808001], np.uint32).view(np.float32))[0]) == hi


# ---- RMS normalisation and residual addition ---------------------------------------------------------------
def _half_ulp(y):
    """Half the spacing of bf16 numbers at |y| (8 significant bits)."""
    e = np.floor(np.log2(np.maximum(np.abs(y), 2.0 ** -126)))
    return 2.0 ** (e - 8)


def _rand_bf16(rng, shape, scale=1.0):
    return glue.f32_to_bf16((rng.standard_normal(shape) * scale).astype(np.float32))


def test_rmsnorm_matches_fp64_definition():
    rng = np.random.default_rng(41)
    for N in (8, 64, 264, 2048, 3072):
        bits = _rand_bf16(rng, (9, N), 3.0)
        w = (1.0 + 0.1 * rng.standard_normal(N)).astype(np.float32)
        eps = 1e-6
        x = glue.bf16_to_f32(bits).astype(np.float64)
        want = x / np.sqrt((x * x).mean(1, keepdims=True) + eps) * w.astype(np.float64)
        got = glue.bf16_to_f32(glue.rmsnorm_bf16(bits, w, eps)).astype(np.float64)
        # fp32 evaluation (a few 2^-24) then one bf16 rounding: within just over half a bf16 ulp of the fp64 value
        assert (np.abs(got - want) <= 1.001 * _half_ulp(want) + 1e-30).all()


def test_rmsnorm_invariants():
    rng = np.random.default_rng(42)
    bits = _rand_bf16(rng, (5, 512))
    w = np.ones(512, np.float32)
    base = glue.rmsnorm_bf16(bits, w, 0.0)
    # a power-of-two factor on the input cancels exactly (eps = 0): every fp32 operation scales exactly
    x4 = glue.f32_to_bf16(glue.bf16_to_f32(bits) * np.float32(4.0))
    assert np.array_equal(glue.rmsnorm_bf16(x4, w, 0.0), base)
    # a power-of-two weight scales the output exactly
    assert np.array_equal(glue.bf16_to_f32(glue.rmsnorm_bf16(bits, w * np.float32(0.5), 0.0)), glue.bf16_to_f32(base) * np.float32(0.5))
    # the normalised row has unit mean square (up to the bf16 rounding of its entries)
    y = glue.bf16_to_f32(base).astype(np.float64)
    assert np.allclose((y * y).mean(1), 1.0, atol=2e-3)
    # a row of equal magnitudes normalises to +-1 exactly; an all-zero row with eps > 0 stays zero
    c = glue.f32_to_bf16(np.where(np.arange(64) % 2 == 0, 3.0, -3.0).astype(np.float32))[None, :]
    assert np.array_equal(glue.bf16_to_f32(glue.rmsnorm_bf16(c, np.ones(64, np.float32), 0.0)), np.sign(glue.bf16_to_f32(c)))
    z = np.zeros((1, 64), np.uint16)
    assert not glue.rmsnorm_bf16(z, np.ones(64, np.float32), 1e-6).any()
    # rows are independent
    both = glue.rmsnorm_bf16(bits, w, 1e-6)
    assert np.array_equal(glue.rmsnorm_bf16(bits[2:3], w, 1e-6), both[2:3])


def test_add_is_one_rounded_fp32_addition():
    rng = np.random.default_rng(43)
    a, b = _rand_bf16(rng, (7, 256), 2.0), _rand_bf16(rng, (7, 256), 50.0)
    got = glue.bf16_to_f32(glue.add_bf16(a, b)).astype(np.float64)
    want = glue.bf16_to_f32(a).astype(np.float64) + glue.bf16_to_f32(b).astype(np.float64)
    assert (np.abs(got - want) <= _half_ulp(want) * (1 + 2.0 ** -14) + 1e-30).all()      # fp32 then bf16: at most a whisker over half an ulp
    assert np.array_equal(glue.add_bf16(a, b), glue.add_bf16(b, a))
    assert np.array_equal(glue.add_bf16(a, np.zeros_like(a)), a)                       # x + 0 = x
    neg = (a ^ np.uint16(0x8000)).astype(np.uint16)
    assert not (glue.add_bf16(a, neg) & 0x7FFF).any()                                   # x + (-x) = 0
