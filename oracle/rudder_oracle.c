/*
 * rudder_oracle.c -- plain CPU oracle of the SteerQuant / Rudder quantized linear layer.
 *
 * TEST INFRASTRUCTURE ONLY (see rudder_oracle.h).  Plain C, fp32 operations individually rounded
 * (build with -O2 -ffp-contract=off, never -ffast-math), OpenMP over rows, nothing clever.
 * Each function follows one passage of the paper, taken in the paper's order and notation:
 *
 *   Eq. 1   symmetric k-bit quantiser  Q = clip(round(x / Delta), -q_max, q_max), Delta = c/q_max,
 *           q_max = 2^(k-1) - 1
 *   Eq. 6   equivalent transform       Y(D) = Q(X D^-1) Q(D W)
 *   Sec 4.2 (last paragraph)           W^ = Q(D* W) stored as packed integers + scales
 *   Eq. 8   modulated output           Y^ = gamma^-1 Q(gamma X~ ; c) W^,  X~ = X D^-1
 *   Sec 4.4 first kernel               writes Q_X and r_i = Delta_X / gamma_{s(i)}
 *   Sec 4.4 second kernel, Eq. 10      C = Q_X Q_W (INT32);  Y_ij = cast[(FP32(C_ij) r_i) Delta_Wj + b_j]
 *
 * Readings taken where the paper is silent (each also listed in the design notes):
 *   round() is round-half-to-even; clip range is +-q_max (never -128 / -8);
 *   x/Delta is evaluated as x * (q_max / a) with one division per row;
 *   the channel scaling is applied before the gain: v = (x * dinv_k) * gamma;
 *   weight scales are per (output channel, group of G input channels), stored in fp16, and the
 *   weights are quantised against the fp16-rounded scale; G = K is the paper's per-channel case;
 *   a zero row / zero group / zero block gets scale 0 and codes 0;
 *   the NVFP4 variant (E2M1 codes, UE4M3 scale per 16 elements, one fp32 scale per weight tensor
 *   and per activation row) is specified here because the paper only names the format.
 */
#include "rudder_oracle.h"

#include <math.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* ------------------------------------------------------------------------------------------ */
/* Number formats.  Decoders are the formats' definitions.  Encoders search the table of all   */
/* non-negative finite values for the nearest one; a tie goes to the even code.                */
/* ------------------------------------------------------------------------------------------ */

float orc_bf16_decode(uint16_t h)
{
    uint32_t u = (uint32_t)h << 16;   /* bf16 is the upper half of an IEEE binary32 */
    float f;
    memcpy(&f, &u, sizeof f);
    return f;
}

float orc_fp16_decode(uint16_t h)
{
    int sign = (h >> 15) & 1;
    int e = (h >> 10) & 0x1F;
    int m = h & 0x3FF;
    double v;
    if (e == 0)        v = ldexp((double)m, -24);               /* subnormal: m * 2^-24 */
    else if (e == 31)  v = (m == 0) ? INFINITY : NAN;
    else               v = ldexp((double)(1024 + m), e - 25);   /* (1 + m/1024) * 2^(e-15) */
    return (float)(sign ? -v : v);
}

float orc_ue4m3_decode(uint8_t b)
{
    int e = (b >> 3) & 0xF;
    int m = b & 0x7;
    double v;
    if (e == 15 && m == 7) return NAN;                          /* the single NaN code of E4M3 */
    if (e == 0) v = ldexp((double)m, -9);                       /* subnormal: m/8 * 2^-6 */
    else        v = ldexp((double)(8 + m), e - 10);             /* (1 + m/8) * 2^(e-7) */
    return (float)v;
}

static const float E2M1_VALUES[8] = { 0.0f, 0.5f, 1.0f, 1.5f, 2.0f, 3.0f, 4.0f, 6.0f };

float orc_e2m1_decode(uint8_t c)
{
    float v = E2M1_VALUES[c & 7];
    return (c & 8) ? -v : v;
}

#define BF16_N   0x7F80    /* codes 0x0000 .. 0x7F7F are the non-negative finite bf16 values */
#define FP16_N   0x7C00
#define UE4M3_N  0x7F      /* codes 0x00 .. 0x7E, 0x7E = 448 */
static double bf16_tab[BF16_N];
static double fp16_tab[FP16_N];
static double ue4m3_tab[UE4M3_N];
static int tables_ready = 0;

static void build_tables(void)
{
    if (tables_ready) return;
#ifdef _OPENMP
#pragma omp critical(orc_tables)
#endif
    {
        if (!tables_ready) {
            for (int i = 0; i < BF16_N; ++i)  bf16_tab[i]  = (double)orc_bf16_decode((uint16_t)i);
            for (int i = 0; i < FP16_N; ++i)  fp16_tab[i]  = (double)orc_fp16_decode((uint16_t)i);
            for (int i = 0; i < UE4M3_N; ++i) ue4m3_tab[i] = (double)orc_ue4m3_decode((uint8_t)i);
            tables_ready = 1;
        }
    }
}

/* Index of the table entry nearest to ax >= 0 (table ascending, tab[0] = 0).  `beyond` is the value
 * the format would take one step above its largest finite one; returns n when ax rounds to it. */
static int nearest_code(const double* tab, int n, double beyond, double ax)
{
    int lo = 0, hi = n - 1;
    while (lo < hi) {                       /* largest lo with tab[lo] <= ax */
        int mid = (lo + hi + 1) / 2;
        if (tab[mid] <= ax) lo = mid; else hi = mid - 1;
    }
    double up = (lo + 1 < n) ? tab[lo + 1] : beyond;
    double dl = ax - tab[lo];
    double dh = up - ax;
    if (dl < dh) return lo;
    if (dl > dh) return lo + 1;
    return (lo % 2 == 0) ? lo : lo + 1;     /* tie: even code */
}

uint16_t orc_bf16_encode(float x)
{
    build_tables();
    uint16_t s = signbit(x) ? 0x8000 : 0;
    int c = nearest_code(bf16_tab, BF16_N, ldexp(1.0, 128), fabs((double)x));
    return (uint16_t)(s | c);               /* c == BF16_N is the inf pattern 0x7F80 */
}

uint16_t orc_fp16_encode(float x)
{
    build_tables();
    uint16_t s = signbit(x) ? 0x8000 : 0;
    int c = nearest_code(fp16_tab, FP16_N, 65536.0, fabs((double)x));
    return (uint16_t)(s | c);               /* c == FP16_N is the inf pattern 0x7C00 */
}

uint8_t orc_ue4m3_encode(float x)
{
    build_tables();
    double ax = fabs((double)x);
    if (ax >= 448.0) return 0x7E;           /* saturate to the largest finite value */
    return (uint8_t)nearest_code(ue4m3_tab, UE4M3_N, 512.0, ax);
}

uint8_t orc_e2m1_encode(float x)
{
    static const double tab[8] = { 0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0 };
    uint8_t s = signbit(x) ? 8 : 0;
    double ax = fabs((double)x);
    if (ax >= 6.0) return (uint8_t)(s | 7); /* saturate */
    return (uint8_t)(s | nearest_code(tab, 8, 8.0, ax));
}

/* ------------------------------------------------------------------------------------------ */
/* Offline: fold D into W, quantise, pack (Eq. 6; Section 4.2 last paragraph; Eq. 1, k = 4).   */
/* ------------------------------------------------------------------------------------------ */

static int clampi(int v, int lo, int hi) { return v < lo ? lo : (v > hi ? hi : v); }

static void pack_nibbles(const uint8_t* codes /* low 4 bits valid */, int K, uint8_t* out)
{
    for (int k = 0; k < K; k += 2)
        out[k / 2] = (uint8_t)((codes[k] & 0xF) | ((codes[k + 1] & 0xF) << 4));
}

int orc_pack_int4(const float* W, const float* d, int N, int K, int G,
                  int8_t* qw, uint8_t* packed, uint16_t* scales, float* dinv)
{
    if (!W || !qw || N < 1 || K < 2 || G < 1 || K % G != 0 || K % 2 != 0) return 1;
    build_tables();
    int n_groups = K / G;
    if (dinv) for (int k = 0; k < K; ++k) dinv[k] = 1.0f / (d ? d[k] : 1.0f);
#pragma omp parallel for schedule(static)
    for (int j = 0; j < N; ++j) {
        float* V = (float*)malloc(sizeof(float) * (size_t)K);
        uint8_t* nib = (uint8_t*)malloc((size_t)K);
        for (int k = 0; k < K; ++k) V[k] = W[(size_t)j * K + k] * (d ? d[k] : 1.0f);   /* D W */
        for (int g = 0; g < n_groups; ++g) {
            float amax = 0.0f;
            for (int k = g * G; k < (g + 1) * G; ++k) amax = fmaxf(amax, fabsf(V[k]));
            float delta_f = amax / 7.0f;                         /* Delta = c / q_max, c = amax */
            uint16_t delta_h = orc_fp16_encode(delta_f);
            float delta = orc_fp16_decode(delta_h);              /* quantise against the stored scale */
            if (scales) scales[(size_t)j * n_groups + g] = delta_h;
            for (int k = g * G; k < (g + 1) * G; ++k) {
                int q = 0;
                if (delta != 0.0f) q = clampi((int)rintf(V[k] / delta), -7, 7);
                qw[(size_t)j * K + k] = (int8_t)q;
                nib[k] = (uint8_t)(q & 0xF);
            }
        }
        if (packed) pack_nibbles(nib, K, packed + (size_t)j * (K / 2));
        free(V);
        free(nib);
    }
    return 0;
}

#define NVFP4_RANGE 2688.0f   /* 6 (largest E2M1) * 448 (largest UE4M3) */

int orc_pack_nvfp4(const float* W, const float* d, int N, int K,
                   uint8_t* e2m1, uint8_t* packed, uint8_t* sb, float* dinv, float* tensor_scale)
{
    if (!W || !e2m1 || !sb || N < 1 || K < 16 || K % 16 != 0) return 1;
    build_tables();
    if (dinv) for (int k = 0; k < K; ++k) dinv[k] = 1.0f / (d ? d[k] : 1.0f);
    float tmax = 0.0f;
    for (int j = 0; j < N; ++j)
        for (int k = 0; k < K; ++k)
            tmax = fmaxf(tmax, fabsf(W[(size_t)j * K + k] * (d ? d[k] : 1.0f)));
    if (tensor_scale) *tensor_scale = tmax / NVFP4_RANGE;
    float invW = (tmax != 0.0f) ? NVFP4_RANGE / tmax : 0.0f;
    int n_blocks = K / 16;
#pragma omp parallel for schedule(static)
    for (int j = 0; j < N; ++j) {
        for (int b = 0; b < n_blocks; ++b) {
            float V[16];
            float amax = 0.0f;
            for (int t = 0; t < 16; ++t) {
                int k = b * 16 + t;
                V[t] = W[(size_t)j * K + k] * (d ? d[k] : 1.0f);
                amax = fmaxf(amax, fabsf(V[t]));
            }
            float tt = (amax * invW) / 6.0f;
            uint8_t code = orc_ue4m3_encode(tt);
            float sbd = orc_ue4m3_decode(code);
            sb[(size_t)j * n_blocks + b] = code;
            float rb = (sbd != 0.0f) ? 1.0f / sbd : 0.0f;
            for (int t = 0; t < 16; ++t) {
                uint8_t e = 0;
                if (sbd != 0.0f) e = orc_e2m1_encode((V[t] * invW) * rb);
                e2m1[(size_t)j * K + b * 16 + t] = e;
            }
        }
        if (packed) pack_nibbles(e2m1 + (size_t)j * K, K, packed + (size_t)j * (K / 2));
    }
    return 0;
}

/* ------------------------------------------------------------------------------------------ */
/* Activation prologue (Section 4.4 first kernel; Eq. 8; Eq. 1).                               */
/* ------------------------------------------------------------------------------------------ */

static int stream_of_row(int i, const int32_t* seg_offsets, const int32_t* seg_stream, int n_seg)
{
    for (int s = 0; s < n_seg; ++s)
        if (i >= seg_offsets[s] && i < seg_offsets[s + 1]) return seg_stream[s];
    return -1;
}

static int check_table(const float* gamma, const float* clip, int T, int S, int step, int mode,
                       const int32_t* seg_offsets, const int32_t* seg_stream, int n_seg, int M)
{
    if (!gamma || T < 1 || S < 1 || step < 0 || step >= T) return 1;
    if (mode != 0 && mode != 1) return 1;
    if (mode == 1 && !clip) return 1;
    if (!seg_offsets || !seg_stream || n_seg < 1) return 1;
    if (seg_offsets[0] != 0 || seg_offsets[n_seg] != M) return 1;
    for (int s = 0; s < n_seg; ++s) {
        if (seg_offsets[s + 1] < seg_offsets[s]) return 1;
        if (seg_stream[s] < 0 || seg_stream[s] >= S) return 1;
    }
    return 0;
}

int orc_quantize_int(const uint16_t* X, int64_t ldx, int M, int K, const float* dinv,
                     const float* gamma, const float* clip, int T, int S, int step, int mode,
                     const int32_t* seg_offsets, const int32_t* seg_stream, int n_seg,
                     int qmax, const int32_t* rows, int n_rows,
                     int8_t* codes, float* r)
{
    if (!X || !dinv || !codes || !r || M < 1 || K < 1 || (qmax != 127 && qmax != 7)) return 1;
    if (check_table(gamma, clip, T, S, step, mode, seg_offsets, seg_stream, n_seg, M)) return 1;
    if (!rows) n_rows = M;
#pragma omp parallel for schedule(static)
    for (int t = 0; t < n_rows; ++t) {
        int i = rows ? rows[t] : t;
        int s = stream_of_row(i, seg_offsets, seg_stream, n_seg);
        float g = gamma[(size_t)step * S + s];                   /* gamma_{tau, s(i)} */
        float* v = (float*)malloc(sizeof(float) * (size_t)K);
        float a = 0.0f;
        for (int k = 0; k < K; ++k) {
            float x = orc_bf16_decode(X[(size_t)i * ldx + k]);
            float u = x * dinv[k];                               /* X D^-1 */
            v[k] = u * g;                                        /* gamma X~ */
            a = fmaxf(a, fabsf(v[k]));
        }
        if (mode == 1) a = clip[step];                           /* shared threshold c_tau */
        int8_t* q = codes + (size_t)t * K;
        if (a == 0.0f) {
            for (int k = 0; k < K; ++k) q[k] = 0;
            r[t] = 0.0f;
        } else {
            float inv = (float)qmax / a;                         /* 1 / Delta_X */
            for (int k = 0; k < K; ++k)
                q[k] = (int8_t)clampi((int)rintf(v[k] * inv), -qmax, qmax);
            float delta = a / (float)qmax;                       /* Delta_X = c / q_max */
            r[t] = delta / g;                                    /* r_i = Delta_X / gamma_{s(i)} */
        }
        free(v);
    }
    return 0;
}

int orc_quantize_nvfp4(const uint16_t* X, int64_t ldx, int M, int K, const float* dinv,
                       const float* gamma, const float* clip, int T, int S, int step, int mode,
                       const int32_t* seg_offsets, const int32_t* seg_stream, int n_seg,
                       const int32_t* rows, int n_rows,
                       uint8_t* e2m1, uint8_t* sb, float* r)
{
    if (!X || !dinv || !e2m1 || !sb || !r || M < 1 || K < 16 || K % 16 != 0) return 1;
    if (check_table(gamma, clip, T, S, step, mode, seg_offsets, seg_stream, n_seg, M)) return 1;
    build_tables();
    if (!rows) n_rows = M;
    int n_blocks = K / 16;
#pragma omp parallel for schedule(static)
    for (int t = 0; t < n_rows; ++t) {
        int i = rows ? rows[t] : t;
        int s = stream_of_row(i, seg_offsets, seg_stream, n_seg);
        float g = gamma[(size_t)step * S + s];
        float* v = (float*)malloc(sizeof(float) * (size_t)K);
        float a = 0.0f;
        for (int k = 0; k < K; ++k) {
            float x = orc_bf16_decode(X[(size_t)i * ldx + k]);
            float u = x * dinv[k];
            v[k] = u * g;
            a = fmaxf(a, fabsf(v[k]));
        }
        if (mode == 1) a = clip[step];
        uint8_t* e = e2m1 + (size_t)t * K;
        uint8_t* b8 = sb + (size_t)t * n_blocks;
        if (a == 0.0f) {
            for (int k = 0; k < K; ++k) e[k] = 0;
            for (int b = 0; b < n_blocks; ++b) b8[b] = 0;
            r[t] = 0.0f;
        } else {
            float s_row = a / NVFP4_RANGE;                       /* fp32 scale of the row */
            float inv = NVFP4_RANGE / a;
            for (int b = 0; b < n_blocks; ++b) {
                float amax = 0.0f;
                for (int u = 0; u < 16; ++u) amax = fmaxf(amax, fabsf(v[b * 16 + u]));
                float tt = (amax * inv) / 6.0f;
                uint8_t code = orc_ue4m3_encode(tt);             /* saturates at 448 */
                float sbd = orc_ue4m3_decode(code);
                b8[b] = code;
                float rb = (sbd != 0.0f) ? 1.0f / sbd : 0.0f;
                for (int u = 0; u < 16; ++u) {
                    uint8_t c = 0;
                    if (sbd != 0.0f) c = orc_e2m1_encode((v[b * 16 + u] * inv) * rb);
                    e[b * 16 + u] = c;
                }
            }
            r[t] = s_row / g;
        }
        free(v);
    }
    return 0;
}

/* ------------------------------------------------------------------------------------------ */
/* Integer contraction and epilogue (Section 4.4 second kernel; Eq. 10).                       */
/* ------------------------------------------------------------------------------------------ */

/* C^(g)_ij = sum over k in group g of q_ik * w_jk, in INT32. */
static int32_t group_dot(const int8_t* q_row, const int8_t* w_row, int g, int G)
{
    int32_t c = 0;
    for (int k = g * G; k < (g + 1) * G; ++k) c += (int32_t)q_row[k] * (int32_t)w_row[k];
    return c;
}

int orc_accumulate_int(const int8_t* codes, int n_rows, const int8_t* qw, int N, int K, int G,
                       int32_t* acc)
{
    if (!codes || !qw || !acc || n_rows < 1 || N < 1 || G < 1 || K % G != 0) return 1;
    int n_groups = K / G;
#pragma omp parallel for schedule(static)
    for (int t = 0; t < n_rows; ++t)
        for (int j = 0; j < N; ++j)
            for (int g = 0; g < n_groups; ++g)
                acc[((size_t)g * n_rows + t) * N + j] =
                    group_dot(codes + (size_t)t * K, qw + (size_t)j * K, g, G);
    return 0;
}

int orc_linear_int(const int8_t* codes, const float* r, int n_rows,
                   const int8_t* qw, const uint16_t* scales, int N, int K, int G,
                   const float* bias, uint16_t* y, double* y64)
{
    if (!codes || !r || !qw || !scales || n_rows < 1 || N < 1 || G < 1 || K % G != 0) return 1;
    build_tables();
    int n_groups = K / G;
#pragma omp parallel for schedule(static)
    for (int t = 0; t < n_rows; ++t) {
        for (int j = 0; j < N; ++j) {
            float b = bias ? bias[j] : 0.0f;
            float out32;
            double out64;
            if (n_groups == 1) {
                /* Eq. 10 verbatim: ((FP32(C_ij) * r_i) * Delta_Wj) + b_j */
                int32_t c = group_dot(codes + (size_t)t * K, qw + (size_t)j * K, 0, G);
                float dw = orc_fp16_decode(scales[j]);
                float p = (float)c * r[t];
                float q = p * dw;
                out32 = q + b;
                out64 = ((double)c * (double)r[t]) * (double)dw + (double)b;
            } else {
                /* Eq. 10 with one weight scale per group: the INT32 partial of each group is
                 * dequantised by its own Delta_W[j,g], the row scale and bias come last. */
                float acc32 = 0.0f;
                double acc64 = 0.0;
                for (int g = 0; g < n_groups; ++g) {
                    int32_t c = group_dot(codes + (size_t)t * K, qw + (size_t)j * K, g, G);
                    float dw = orc_fp16_decode(scales[(size_t)j * n_groups + g]);
                    float p = (float)c * dw;
                    acc32 = acc32 + p;
                    acc64 += (double)c * (double)dw;
                }
                float q = acc32 * r[t];
                out32 = q + b;
                out64 = acc64 * (double)r[t] + (double)b;
            }
            if (y)   y[(size_t)t * N + j] = orc_bf16_encode(out32);
            if (y64) y64[(size_t)t * N + j] = out64;
        }
    }
    return 0;
}

int orc_linear_nvfp4(const uint8_t* a_e2m1, const uint8_t* a_sb, const float* r, int n_rows,
                     const uint8_t* w_e2m1, const uint8_t* w_sb, float tensor_scale, int N, int K,
                     const float* bias, uint16_t* y, double* y64)
{
    if (!a_e2m1 || !a_sb || !r || !w_e2m1 || !w_sb || n_rows < 1 || N < 1 || K % 16 != 0) return 1;
    build_tables();
    int n_blocks = K / 16;
#pragma omp parallel for schedule(static)
    for (int t = 0; t < n_rows; ++t) {
        for (int j = 0; j < N; ++j) {
            double acc = 0.0;
            for (int b = 0; b < n_blocks; ++b) {
                double dot = 0.0;      /* products of E2M1 values are multiples of 1/4: exact */
                for (int u = 0; u < 16; ++u)
                    dot += (double)orc_e2m1_decode(a_e2m1[(size_t)t * K + b * 16 + u]) *
                           (double)orc_e2m1_decode(w_e2m1[(size_t)j * K + b * 16 + u]);
                acc += (double)orc_ue4m3_decode(a_sb[(size_t)t * n_blocks + b]) *
                       (double)orc_ue4m3_decode(w_sb[(size_t)j * n_blocks + b]) * dot;
            }
            float rs = r[t] * tensor_scale;                      /* row scale x weight tensor scale */
            double out64 = acc * (double)rs + (bias ? (double)bias[j] : 0.0);
            if (y)   y[(size_t)t * N + j] = orc_bf16_encode((float)out64);
            if (y64) y64[(size_t)t * N + j] = out64;
        }
    }
    return 0;
}

int orc_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
