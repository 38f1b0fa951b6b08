"""CPU oracle of the BF16 glue of a chained block: GELU, RMS normalisation, residual add (TEST INFRASTRUCTURE ONLY).

The paper keeps GELU in BF16 and does not say which GELU.  Reading: the tanh form
    gelu(x) = x/2 (1 + tanh(sqrt(2/pi) (x + 0.044715 x^3)))
with tanh u replaced, for |u| < 5, by its [7/6] Pade approximant
    u (135135 + 17325 u^2 + 378 u^4 + u^6) / (135135 + 62370 u^2 + 3150 u^4 + 28 u^6)
and by +-1 beyond.  So that a rounding decision (the bf16 result, and the integer code the next
layer makes of it) is taken in the same precision on both sides, the evaluation is fixed: fp32,
Horner's rule from the highest power, every add, multiply and the one divide rounded to nearest on
its own.  numpy's float32 array arithmetic does exactly that (no fused multiply-add).
"""
import numpy as np

F = np.float32


def bf16_to_f32(bits):
    return (np.asarray(bits, dtype=np.uint16).astype(np.uint32) << 16).view(np.float32)


def f32_to_bf16(x):
    """Round to nearest even on the bit pattern; NaN stays NaN (quiet)."""
    b = np.asarray(x, dtype=np.float32).view(np.uint32)
    r = ((b + np.uint32(0x7FFF) + ((b >> 16) & np.uint32(1))) >> 16).astype(np.uint16)
    nan = np.isnan(np.asarray(x, dtype=np.float32))
    return np.where(nan, np.uint16(0x7FC0) | (b >> 16).astype(np.uint16) & np.uint16(0x8000), r).astype(np.uint16)


def pade_tanh(u):
    """The approximant itself, in whatever precision `u` has (used by the pins in fp64 too)."""
    u2 = u * u
    n = u2 + 378
    n = n * u2 + 17325
    n = n * u2 + 135135
    n = n * u
    d = 28 * u2 + 3150
    d = d * u2 + 62370
    d = d * u2 + 135135
    return n / d


def gelu_f32(x):
    x = np.asarray(x, dtype=np.float32)
    with np.errstate(over="ignore", invalid="ignore"):
        x2 = x * x
        x3 = x2 * x
        inner = x + F(0.044715) * x3
        u = F(0.7978845608028654) * inner
        t = pade_tanh(np.where(np.abs(u) < F(5.0), u, F(0.0)).astype(np.float32))
        t = np.where(np.abs(u) < F(5.0), t, np.where(u < 0, F(-1.0), F(1.0))).astype(np.float32)
        t = np.where(np.isnan(u), u, t).astype(np.float32)
        return ((F(0.5) * x) * (F(1.0) + t)).astype(np.float32)


def gelu_bf16(bits):
    """bf16 bit patterns in -> bf16 bit patterns out."""
    return f32_to_bf16(gelu_f32(bf16_to_f32(bits)))


def rmsnorm_bf16(bits, weight, eps):
    """RMS normalisation of every row: y = bf16((x r) w), r = 1 / sqrt(mean(x^2) + eps), in the fixed fp32 order
    that makes the result (and the integer codes the next layer makes of it) a matter of definition, not of
    summation order: the row is cut into pieces of 8 values; partial sum l (of 32) adds x*x of pieces l, l + 32,
    ... in order, product and sum rounded separately; the partials are combined pairwise l ^ 16, 8, 4, 2, 1."""
    x = bf16_to_f32(bits)
    M, N = x.shape
    assert N % 8 == 0
    w = np.asarray(weight, dtype=np.float32)
    chunks = N // 8
    rounds = (chunks + 31) // 32
    xp = np.zeros((M, rounds * 32 * 8), np.float32)
    xp[:, :N] = x                                             # padding adds +0.0: no effect on any partial sum
    xp = xp.reshape(M, rounds, 32, 8)
    acc = np.zeros((M, 32), np.float32)
    for j in range(rounds):
        for e in range(8):
            v = xp[:, j, :, e]
            acc = (acc + (v * v).astype(np.float32)).astype(np.float32)
    for o in (16, 8, 4, 2, 1):
        acc = (acc + acc[:, np.arange(32) ^ o]).astype(np.float32)
    total = acc[:, 0]
    ms = (total / F(N)).astype(np.float32)
    with np.errstate(divide="ignore", invalid="ignore", over="ignore"):       # an all-zero row with eps = 0 is 0 / 0 = NaN, by definition
        r = (F(1.0) / np.sqrt((ms + F(eps)).astype(np.float32)).astype(np.float32)).astype(np.float32)
        y = ((x * r[:, None]).astype(np.float32) * w[None, :]).astype(np.float32)
    return f32_to_bf16(y)


def add_bf16(a_bits, b_bits):
    """Residual addition: bf16(a + b), one fp32 addition."""
    return f32_to_bf16((bf16_to_f32(a_bits) + bf16_to_f32(b_bits)).astype(np.float32))
