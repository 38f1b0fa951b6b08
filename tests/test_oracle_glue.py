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
