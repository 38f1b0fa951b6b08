"""CPU oracle of the toy Stream-Specific Activation Modulation calibrator (Eq. 9; Section 4.3).

TEST INFRASTRUCTURE ONLY, like the rest of this package: plain numpy in fp64 around the oracle's
quantized linear.  For one layer and one denoising step it searches the per-stream gains gamma_s
and the shared threshold c that minimise

    J(gamma, c) = sum_s  omega_s / n_s  * || Yhat_s(gamma_s, c) - Xtilde_s What ||_F^2        (Eq. 9)

subject to  gamma_min <= gamma_s <= gamma_max  and  sum_s n_s log gamma_s = 0,  where Yhat is the
quantized layer's (bf16) output in the static-range mode, Xtilde = X D^-1 the transformed
activations, What the dequantized 4-bit weights, n_s the number of tokens of stream s and omega_s
the map-derived stream weights (uniform here: the map itself is out of scope).

The paper does not say how the arg-min is found; the reading taken is a coordinate search over
candidate lists (stated in the function below), the same reading as the GPU-side calibrator, written
independently of it.
"""
import numpy as np

from . import RANGE_STATIC, rudder_linear


def _bf16_to_f64(bits):
    return (np.asarray(bits, dtype=np.uint16).astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def dequantized_weights(packed_w):
    """What [N, K] in fp64 from the oracle's integer pack (codes x fp16 group scales)."""
    qw = packed_w["qw"].astype(np.float64)
    G = packed_w["G"]
    sc = np.ascontiguousarray(packed_w["scales"]).view(np.float16).astype(np.float64)       # fp16 bit patterns [N, K/G]
    return qw * np.repeat(sc, G, axis=1)


def reference_output(X_bf16, packed_w):
    """Xtilde What^T in fp64 (no activation quantization, no bias)."""
    xt = _bf16_to_f64(X_bf16) * packed_w["dinv"].astype(np.float64)[None, :]
    return xt @ dequantized_weights(packed_w).T


def stream_rows(seg_offsets, seg_stream, S):
    row_stream = np.repeat(np.asarray(seg_stream), np.diff(np.asarray(seg_offsets)))
    return row_stream, np.array([(row_stream == s).sum() for s in range(S)], dtype=np.float64)


def objective(X_bf16, packed_w, gamma, c, seg_offsets, seg_stream, scheme, omega, y_ref):
    """J(gamma, c) of Eq. 9 for one layer and step, from the oracle's static-mode quantized linear."""
    S = len(gamma)
    row_stream, n = stream_rows(seg_offsets, seg_stream, S)
    out = rudder_linear(X_bf16, packed_w, np.asarray(gamma, np.float32)[None, :], np.array([c], np.float32), 0,
                        RANGE_STATIC, seg_offsets, seg_stream, scheme, None)
    err2 = ((_bf16_to_f64(out["y"]) - y_ref) ** 2).sum(axis=1)
    return float(sum(omega[s] / n[s] * err2[row_stream == s].sum() for s in range(S) if n[s] > 0))


def project(gamma, n):
    """Rescale all gains by one factor so that sum_s n_s log gamma_s = 0."""
    g = np.asarray(gamma, dtype=np.float64)
    return g * np.exp(-(n * np.log(g)).sum() / n.sum())


def calibrate(X_bf16, packed_w, seg_offsets, seg_stream, S, scheme, c_candidates, gamma_steps, omega=None,
              gamma_bounds=(0.5, 2.0), sweeps=2):
    """Coordinate search.  Start at gamma = 1 with the best c of `c_candidates`.  One sweep: for each
    stream in order try gamma_s * m for every m in `gamma_steps` (the vector re-projected onto the
    constraint; candidates that leave the bounds are skipped) and keep the best; then choose c again.
    Ties keep the earlier candidate."""
    omega = np.ones(S) if omega is None else np.asarray(omega, np.float64)
    _, n = stream_rows(seg_offsets, seg_stream, S)
    y_ref = reference_output(X_bf16, packed_w)
    J = lambda g, c: objective(X_bf16, packed_w, g, c, seg_offsets, seg_stream, scheme, omega, y_ref)
    gamma = np.ones(S)
    c, best = None, np.inf
    for cc in c_candidates:
        v = J(gamma, cc)
        if v < best:
            c, best = cc, v
    evals = len(c_candidates)
    for _ in range(sweeps):
        for s in range(S):
            if n[s] == 0:
                continue
            for m in gamma_steps:
                cand = gamma.copy()
                cand[s] *= m
                cand = project(cand, n)
                if cand.min() < gamma_bounds[0] or cand.max() > gamma_bounds[1]:
                    continue
                v = J(cand, c)
                evals += 1
                if v < best:
                    gamma, best = cand, v
        for cc in c_candidates:
            v = J(gamma, cc)
            evals += 1
            if v < best:
                c, best = cc, v
    return dict(gamma=gamma, clip=float(c), objective=best, evaluations=evals)
