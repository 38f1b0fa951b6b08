"""Seeded random shapes, schemes, group sizes and range modes: the whole linear against the oracle
(BF16 output within tolerance) and the prologue's codes, block scales and row scales bit for bit.
The fixed cases elsewhere aim at known edges; this sweep looks for the ones nobody thought of."""
import numpy as np
import pytest

import oracle
import workloads as wl
from helpers import ABS_TOL, REL_TOL, REL_TOL_FP4, GpuLinear, bf16_to_np, oracle_pack, static_clip

pytestmark = pytest.mark.gpu

ROWS = [1, 2, 7, 16, 31, 33, 64, 65, 100, 128, 129, 200, 255, 256, 257, 300, 511, 513, 700, 1024, 1100, 1300]


def _draw_case(rng):
    scheme = str(rng.choice(["w4a8", "w4a4", "nvfp4"]))
    mode = int(rng.integers(0, 2))
    M = int(rng.choice(ROWS))
    N = int(rng.integers(1, 10)) * 64
    if scheme == "nvfp4":
        K, G = int(rng.integers(1, 13)) * 256, 16
        if M >= 1024 and rng.random() < 0.7:
            N = int(rng.integers(1, 4)) * 256          # whole 256-channel tiles: the CTA-pair kernel
    else:
        G = int(rng.choice([64, 128, 0]))
        K = int(rng.integers(1, 25)) * 128
        if G == 0:
            G = K                                       # one scale per output channel
        if K % G:
            K = (K // G + 1) * G
    return scheme, mode, M, K, N, G, int(rng.integers(0, 1 << 30))


@pytest.mark.parametrize("batch", range(4))
def test_random_cases(batch):
    import paper_2609_39056_b200 as rd
    rd.lib()
    rng = np.random.default_rng(9000 + batch)
    for _ in range(20):
        scheme, mode, M, K, N, G, seed = _draw_case(rng)
        tag = f"{scheme} mode={mode} M={M} K={K} N={N} G={G} seed={seed}"
        inp = wl.tiny(seed=seed, M=M, K=K, N=N, T=2)
        ref_w = oracle_pack(inp, scheme, G)
        clip = static_clip(inp, ref_w["dinv"]) if mode == 1 else None
        g = GpuLinear(rd, inp, scheme, G, mode, clip)
        Y = rd.rudder_linear(g.w, g.X, g.seg, 1, g.tab, g.bias)
        out = oracle.rudder_linear(inp.X_bf16, ref_w, inp.gamma, clip, 1, mode, inp.seg_offsets, inp.seg_stream, scheme,
                                   inp.bias)
        y = wl.bf16_bits_to_f32(bf16_to_np(Y)).astype(np.float64)
        rel = REL_TOL_FP4 if scheme == "nvfp4" else REL_TOL
        assert not np.isnan(y).any(), tag
        assert np.all(np.abs(y - out["y64"]) <= ABS_TOL + rel * np.abs(out["y64"])), tag
        res = rd.rudder_quantize_activations(g.w, g.X, g.seg, 1, g.tab)
        if scheme == "nvfp4":
            re, rsb, rr = oracle.quantize_nvfp4(inp.X_bf16, ref_w["dinv"], inp.gamma, clip, 1, mode, inp.seg_offsets,
                                                inp.seg_stream)
            assert np.array_equal(res[0].cpu().numpy(), (re[:, 0::2] | (re[:, 1::2] << 4)).astype(np.uint8)), tag
            assert np.array_equal(res[1].cpu().numpy(), rsb), tag
        else:
            rq, rr = oracle.quantize_int(inp.X_bf16, ref_w["dinv"], inp.gamma, clip, 1, mode, inp.seg_offsets,
                                         inp.seg_stream, 127 if scheme == "w4a8" else 7)
            assert np.array_equal(res[0].cpu().numpy(), rq), tag
        assert np.array_equal(res[2].cpu().numpy().view(np.uint32), rr.view(np.uint32)), tag
        last, where = rd.rudder_device_status()
        assert last == 0, (tag, last, where)
