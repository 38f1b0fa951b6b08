/*
 * rudder_oracle.h -- plain CPU oracle of the SteerQuant / Rudder quantized linear layer.
 *
 * TEST INFRASTRUCTURE ONLY.  This code exists so that the CUDA library can be checked against an
 * independent, slow, obviously-correct statement of the method.  It shares no code, header, table
 * or constant generator with the CUDA path, and nothing in the product may call it.
 *
 * Conventions (all pointers are HOST pointers):
 *   X      activations, bf16 bit patterns (uint16), row-major [M, ldx], K valid columns
 *   W      weights fp32 row-major [N, K]   (the paper writes Y = X W with W in R^{K x N}; we store
 *          its transpose so that K is contiguous; the diagonal D of Eq. 6 scales input channel k)
 *   d      shared channel scales D (Eq. 6), fp32 [K], positive
 *   gamma  per-step per-stream gains (Eq. 8), fp32 [T, S]
 *   clip   per-step clipping threshold c (Eq. 8 / Eq. 1), fp32 [T]  (static range mode only)
 *   rows   optional list of row indices to compute (NULL = all M rows, in order)
 *
 * Range modes: 0 = per-token absmax (range a_i = max_k |v_ik|), 1 = static (a_i = clip[step]),
 * the latter being exactly the paper's Delta_X = c / q_max with r_i = Delta_X / gamma_{s(i)}
 * (Section 4.4, first kernel).
 *
 * Parity status: every function below is pinned by tests/test_oracle_*.py against closed forms,
 * exhaustive codec enumeration, library conversions, brute force and invariants.  What stays
 * "parity unpinned" is only the *choice of conventions* where the paper is silent (tie rule,
 * group-wise weight scales, reciprocal-multiply quantisation, the whole NVFP4 recipe): the paper
 * prints no numeric worked example of a quantized linear to pin them to.
 */
#ifndef RUDDER_ORACLE_H
#define RUDDER_ORACLE_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* ---- number formats (encoders: round to nearest, ties to the even code; by table search) ---- */
uint16_t orc_bf16_encode(float x);      /* finite x; overflow -> inf pattern */
float    orc_bf16_decode(uint16_t h);
uint16_t orc_fp16_encode(float x);      /* finite x; overflow -> inf pattern */
float    orc_fp16_decode(uint16_t h);
uint8_t  orc_ue4m3_encode(float x);     /* x >= 0; saturates at 448 (code 0x7E) */
float    orc_ue4m3_decode(uint8_t b);   /* sign bit ignored */
uint8_t  orc_e2m1_encode(float x);      /* 4-bit code, bit 3 = sign; saturates at +-6 */
float    orc_e2m1_decode(uint8_t c);

/* ---- offline fold + quantise + pack (Eq. 6, Section 4.2 last paragraph, Eq. 1 with k = 4) ---- */
/* qw: one signed code per byte [N,K]; packed: [N,K/2], low nibble = even k, two's complement;
 * scales: fp16 bit patterns [N, K/G]; dinv: [K].  G in {64,128,...,K}, K % G == 0.  d may be NULL. */
int orc_pack_int4(const float* W, const float* d, int N, int K, int G,
                  int8_t* qw, uint8_t* packed, uint16_t* scales, float* dinv);
/* e2m1: one 4-bit code per byte [N,K]; packed as above; sb: UE4M3 bytes [N,K/16]. */
int orc_pack_nvfp4(const float* W, const float* d, int N, int K,
                   uint8_t* e2m1, uint8_t* packed, uint8_t* sb, float* dinv, float* tensor_scale);

/* ---- activation prologue (Section 4.4 first kernel; Eq. 8; Eq. 1) ---- */
/* codes: int8 [n_rows, K]; r: [n_rows].  qmax = 127 (A8) or 7 (A4). */
int orc_quantize_int(const uint16_t* X, int64_t ldx, int M, int K, const float* dinv,
                     const float* gamma, const float* clip, int T, int S, int step, int mode,
                     const int32_t* seg_offsets, const int32_t* seg_stream, int n_seg,
                     int qmax, const int32_t* rows, int n_rows,
                     int8_t* codes, float* r);
/* e2m1: one code per byte [n_rows,K]; sb: UE4M3 bytes [n_rows,K/16]; r: [n_rows]. */
int orc_quantize_nvfp4(const uint16_t* X, int64_t ldx, int M, int K, const float* dinv,
                       const float* gamma, const float* clip, int T, int S, int step, int mode,
                       const int32_t* seg_offsets, const int32_t* seg_stream, int n_seg,
                       const int32_t* rows, int n_rows,
                       uint8_t* e2m1, uint8_t* sb, float* r);

/* ---- integer contraction (Section 4.4 second kernel: C = Q_X Q_W in INT32), per group ---- */
/* acc: int32 [K/G][n_rows][N] */
int orc_accumulate_int(const int8_t* codes, int n_rows, const int8_t* qw, int N, int K, int G,
                       int32_t* acc);

/* ---- contraction + epilogue (Eq. 10, generalised to weight groups) ---- */
/* y: bf16 bit patterns [n_rows,N] from the fp32 evaluation order; y64: same value in double with
 * no final rounding (either may be NULL).  bias may be NULL. */
int orc_linear_int(const int8_t* codes, const float* r, int n_rows,
                   const int8_t* qw, const uint16_t* scales, int N, int K, int G,
                   const float* bias, uint16_t* y, double* y64);
int orc_linear_nvfp4(const uint8_t* a_e2m1, const uint8_t* a_sb, const float* r, int n_rows,
                     const uint8_t* w_e2m1, const uint8_t* w_sb, float tensor_scale, int N, int K,
                     const float* bias, uint16_t* y, double* y64);

int orc_num_threads(void);

#ifdef __cplusplus
}
#endif
#endif
