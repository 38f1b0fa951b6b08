"""Pins for the oracle's number-format codecs: exhaustive enumeration of every code point and every
midpoint, and agreement with library conversions (numpy float16, torch bfloat16 / float8_e4m3fn).
The formats themselves are fixed by IEEE 754 (binary16), by bfloat16 = upper half of binary32, and
by the OCP 8-bit / 4-bit float definitions (E4M3: bias 7, no inf, one NaN, max 448; E2M1: values
0, 0.5, 1, 1.5, 2, 3, 4, 6)."""
import numpy as np
import pytest
import torch

import oracle


def test_bf16_roundtrip_all_codes():
    for h in range(0x7F80):
        for s in (0, 0x8000):
            if h == 0 and s:
                continue
            assert oracle.bf16_encode(oracle.bf16_decode(h | s)) == (h | s)


def test_bf16_decode_matches_torch():
    codes = np.arange(0x7F80, dtype=np.uint16)
    ref = torch.from_numpy(codes.view(np.int16)).view(torch.bfloat16).float().numpy()
    got = np.array([oracle.bf16_decode(int(h)) for h in codes], np.float32)
    assert np.array_equal(ref, got)


def test_bf16_midpoints_tie_to_even():
    # The midpoint of two adjacent bf16 values is exactly representable in fp32.
    rng = np.random.default_rng(0)
    for h in rng.integers(0x0001, 0x7F7E, 4000):
        lo, hi = oracle.bf16_decode(int(h)), oracle.bf16_decode(int(h) + 1)
        mid = np.float32((np.float64(lo) + np.float64(hi)) / 2)
        assert np.float64(mid) * 2 == np.float64(lo) + np.float64(hi)
        want = int(h) if h % 2 == 0 else int(h) + 1
        assert oracle.bf16_encode(float(mid)) == want
        assert oracle.bf16_encode(float(np.nextafter(mid, np.float32(0)))) == int(h)
        assert oracle.bf16_encode(float(np.nextafter(mid, np.float32(np.inf)))) == int(h) + 1


def test_bf16_encode_matches_torch_random():
    rng = np.random.default_rng(1)
    x = np.concatenate([rng.standard_normal(20000) * 10.0 ** rng.integers(-30, 30, 20000),
                        [0.0, 1.0, -1.0, 3.3895314e38, 1e-45, -1e-40]]).astype(np.float32)
    ref = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    got = np.array([oracle.bf16_encode(float(v)) for v in x], np.uint16)
    assert np.array_equal(ref, got)


def test_fp16_all_codes_and_numpy():
    codes = np.arange(0x7C00, dtype=np.uint16)
    ref = codes.view(np.float16).astype(np.float32)
    for h in range(0x7C00):
        assert oracle.fp16_decode(h) == ref[h]
        assert oracle.fp16_encode(float(ref[h])) == h
    assert oracle.fp16_decode(0xBC00) == -1.0
    assert oracle.fp16_decode(0x7C00) == np.inf


def test_fp16_midpoints_and_numpy_random():
    for h in range(0x7BFF):
        lo, hi = oracle.fp16_decode(h), oracle.fp16_decode(h + 1)
        mid = (lo + hi) / 2           # exact in binary64, and in binary32
        want = h if h % 2 == 0 else h + 1
        assert oracle.fp16_encode(mid) == want
    rng = np.random.default_rng(2)
    x = (rng.standard_normal(50000) * 10.0 ** rng.integers(-9, 5, 50000)).astype(np.float32)
    x = x[np.abs(x) < 65504]
    ref = x.astype(np.float16).view(np.uint16)
    got = np.array([oracle.fp16_encode(float(v)) for v in x], np.uint16)
    assert np.array_equal(ref, got)
    assert oracle.fp16_encode(65519.0) == 0x7BFF and oracle.fp16_encode(65520.0) == 0x7C00


def test_ue4m3_all_codes_torch():
    codes = torch.arange(0x7F, dtype=torch.uint8)
    ref = codes.view(torch.float8_e4m3fn).float().numpy()
    for b in range(0x7F):
        assert oracle.ue4m3_decode(b) == ref[b]
        assert oracle.ue4m3_encode(float(ref[b])) == b
    assert oracle.ue4m3_decode(0x7E) == 448.0
    assert oracle.ue4m3_decode(0x01) == 2.0 ** -9
    assert np.isnan(oracle.ue4m3_decode(0x7F))


def test_ue4m3_midpoints_saturation_and_torch_random():
    for b in range(0x7E):
        lo, hi = oracle.ue4m3_decode(b), oracle.ue4m3_decode(b + 1)
        mid = (lo + hi) / 2
        assert oracle.ue4m3_encode(mid) == (b if b % 2 == 0 else b + 1)
        assert oracle.ue4m3_encode(float(np.nextafter(np.float32(mid), np.float32(0)))) == b
        assert oracle.ue4m3_encode(float(np.nextafter(np.float32(mid), np.float32(1e9)))) == b + 1
    for v in (448.0, 449.0, 463.9, 464.0, 480.0, 1e4, 3e38):
        assert oracle.ue4m3_encode(v) == 0x7E           # satfinite
    rng = np.random.default_rng(3)
    x = np.abs(rng.standard_normal(30000) * 10.0 ** rng.integers(-4, 3, 30000)).astype(np.float32)
    x = x[x <= 448.0]
    ref = torch.from_numpy(x).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    got = np.array([oracle.ue4m3_encode(float(v)) for v in x], np.uint8)
    assert np.array_equal(ref, got)


def test_e2m1_values_midpoints_saturation():
    vals = [0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0]
    for c, v in enumerate(vals):
        assert oracle.e2m1_decode(c) == v and oracle.e2m1_decode(c | 8) == -v
        assert oracle.e2m1_encode(v) == c
        if c:
            assert oracle.e2m1_encode(-v) == (c | 8)
    # midpoints: 0.25->0, 0.75->1.0, 1.25->1.0, 1.75->2.0, 2.5->2.0, 3.5->4.0, 5.0->4.0 (even codes)
    ties = {0.25: 0, 0.75: 2, 1.25: 2, 1.75: 4, 2.5: 4, 3.5: 6, 5.0: 6}
    for m, c in ties.items():
        assert oracle.e2m1_encode(m) == c and oracle.e2m1_encode(-m) == (c | 8 if c else 8)
        lo = float(np.nextafter(np.float32(m), np.float32(0)))
        hi = float(np.nextafter(np.float32(m), np.float32(10)))
        below = max(i for i, v in enumerate(vals) if v < m)
        assert oracle.e2m1_encode(lo) == below and oracle.e2m1_encode(hi) == below + 1
    for v in (6.0, 6.5, 7.0, 100.0, 3e38):
        assert oracle.e2m1_encode(v) == 7 and oracle.e2m1_encode(-v) == 15
    # brute force against "nearest value" on a fine grid (no ties on this grid)
    for x in np.arange(0.01, 6.0, 0.0173):
        want = int(np.argmin([abs(x - v) for v in vals]))
        assert oracle.e2m1_encode(float(x)) == want
