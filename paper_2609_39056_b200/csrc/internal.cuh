// Host-side declarations shared by the translation units of the library (not part of the C ABI).
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "../../include/rudder.h"

namespace rudder {

constexpr int kMaxSeg = 64;
constexpr int kMaxStreams = 16;

// Row -> stream map, passed by value in kernel parameters (no device allocation, graph-capturable).
struct SegParams {
    int n_seg;
    int offset[kMaxSeg + 1];
    int stream[kMaxSeg];
};

// What a packed weight holds on the device.  Layouts are private to the kernels:
//   codes     integer schemes: [N, K/2] bytes; inside every run of 32 input channels, byte b (0..15)
//             holds channel b in its low nibble and channel 16 + b in its high nibble (two's
//             complement), so that one 16-byte load expands into two 16-byte rows of int8 with two
//             logic operations per word.  NVFP4: [N, K/2] bytes, low nibble = even channel (E2M1).
//   scales_t  integer schemes: fp32 [K/G, N] = Delta_W[j,g] / 16 (the kernel feeds the tensor core
//             16 x the code: the nibble placed in the top half of the byte).
//   scales_c  integer schemes: fp16 [N, K/G] canonical copy.  NVFP4: UE4M3 [N, K/16] canonical copy.
//   sf_tiled  NVFP4: UE4M3 scale factors in the tensor core's tiled order:
//             [N/128][K/64][32 lanes][4 row-quarters][4 blocks] bytes.
//   dinv      fp32 [K]
}  // namespace rudder

struct rudder_weight {
    int N, K, G, scheme;
    int device;
    int f8;                   // W4A4 with groups up to 128: codes in the sign-magnitude layout, GEMM on the E4M3 tensor path
    uint8_t* codes;
    float* scales_t;
    void* scales_c;
    uint8_t* sf_tiled;
    float* dinv;
    float* tensor_scale;      // device [1]
    CUtensorMap* tm_codes;    // integer schemes: tensor map (in device memory) over the packed codes [N, K/2],
                              // box {64 bytes, 128 channels}: one pipeline stage of one channel tile
    size_t bytes;
};

namespace rudder {

struct ActqArgs {
    int* zero_ints;            // words the kernel clears for the GEMM that follows (tile counters), or nullptr
    int n_zero;
    const uint16_t* X;
    int64_t ldx;
    int M, K;
    const float* dinv;
    const float* gamma_step;   // gamma + step * S
    const float* clip_step;    // clip + step, or nullptr (per-token range)
    SegParams seg;
};

// SMs of the current device (cached per device).  The one number every tile / split / grid choice below is
// derived from, so that workspace sizing, tensor-map boxes and launches always see the same plan.
int device_sm_count();

// ---- launches (each returns cudaGetLastError of its launch) ----------------------------------
cudaError_t launch_pack_int4(const float* W, const float* d, int N, int K, int G, uint8_t* codes_il,
                             float* scales_t, uint16_t* scales_c, float* dinv, int8_t* tmp_codes, bool signmag,
                             cudaStream_t st);
cudaError_t launch_import_int4(const uint8_t* canonical, const uint16_t* scales_c, int N, int K, int G, uint8_t* codes_il,
                               float* scales_t, int8_t* tmp_codes, bool signmag, cudaStream_t st);
cudaError_t launch_import_nvfp4_scales(const uint8_t* sb_canonical, int N, int K, uint8_t* sf_tiled, size_t sf_tiled_bytes, cudaStream_t st);
cudaError_t launch_export_int4(const uint8_t* codes_il, int N, int K, uint8_t* canonical, bool signmag, cudaStream_t st);

cudaError_t launch_gelu(const uint16_t* X, int64_t ldx, uint16_t* Y, int64_t ldy, int M, int N, int sm_count, cudaStream_t st);
// GELU + static-range activation prologue in one elementwise pass (X is the tensor BEFORE the GELU; a.clip_step must be set)
cudaError_t launch_actq_gelu_static(const ActqArgs& a, int qmax, bool e4m3, int8_t* codes, int64_t ldc, float* r, int sm_count, cudaStream_t st);
cudaError_t launch_rmsnorm(const uint16_t* X, int64_t ldx, const float* w, float eps, uint16_t* Y, int64_t ldy, int M, int N, cudaStream_t st);
cudaError_t launch_add(const uint16_t* A, int64_t lda, const uint16_t* B, int64_t ldb, uint16_t* Y, int64_t ldy, int M, int N, int sm_count,
                       cudaStream_t st);
cudaError_t actq_init();
cudaError_t launch_wait_timeout_selftest(long long limit_cycles, cudaStream_t st);
// e4m3: the codes (integers in [-7, 7]) are written as E4M3 bytes for the FP8 tensor path instead of int8
cudaError_t launch_actq_int(const ActqArgs& a, int qmax, bool e4m3, int8_t* codes, int64_t ldc, float* r, cudaStream_t st);
cudaError_t launch_e4m3_to_int8(int8_t* codes, size_t n_bytes, cudaStream_t st);   // parity hook: E4M3 bytes -> the integers they hold, in place
cudaError_t launch_actq_nvfp4(const ActqArgs& a, uint8_t* codes, uint8_t* sf, bool sf_tiled, float* r, cudaStream_t st);
cudaError_t launch_pack_nvfp4(const float* W, const float* d, int N, int K, uint8_t* codes, uint8_t* sb_canonical,
                              uint8_t* sf_tiled, size_t sf_tiled_bytes, float* dinv, float* tensor_scale,
                              unsigned int* amax_bits, cudaStream_t st);

struct GemmFp4Args {
    CUtensorMap tm_x;           // activation codes, packed E2M1 bytes [M, K/2], box {128 bytes, token tile}, 128-byte swizzle
                                // (CTA-pair kernel: box of 128 tokens, one half of the pair's token tile)
    CUtensorMap tm_sfx;         // CTA-pair kernel only: activation block scales as [atoms][K/64][128 words], box {128, 4, 2}
    CUtensorMap tm_sfw;         // CTA-pair kernel only: weight block scales, same shape, box {128, 4, 1}
    CUtensorMap tm_w;           // weight codes, packed E2M1 bytes [N, K/2], box {128 bytes, 128 channels}, 128-byte swizzle
    CUtensorMap tm_y;           // output bf16 [M, N]
    const uint8_t* sf_x;        // activation block scales, tiled [ceil(M/128)][K/64][512]
    const uint8_t* sf_w;        // weight block scales, tiled [ceil(N/128)][K/64][512]
    int M, N, K;
    const float* row_scale;     // r [M]
    const float* tensor_scale;  // device [1]
    const float* bias;
    int sm_count;               // persistent grid size
};
int gemm_fp4_store_rows(int M, int N); // token rows of one TMA store box of the single-CTA kernel (a quarter of its token tile)
cudaError_t launch_gemm_fp4(const GemmFp4Args& a, cudaStream_t st);
cudaError_t gemm_fp4_init();
int gemm_fp4_token_tile(int M, int N);
bool gemm_fp4_use_pair(int M, int N, int K);   // two CTAs share a 256-channel x 256-token tile (cta_group::2)
cudaError_t gemm_fp4_pair_init();
cudaError_t launch_gemm_fp4_pair(const GemmFp4Args& a, cudaStream_t st);

struct GemmI8Args {
    CUtensorMap tm_x;           // activation codes int8 [M, K], box {128 bytes, token tile}, 128-byte swizzle
    CUtensorMap tm_y;           // output bf16 [M, N] (row pitch ldy), box {min(128, N) channels, token tile}
    uint16_t* y;                // the same output as a plain pointer (small tiles are stored without TMA)
    int64_t ldy;
    int sm_count;               // CTAs of the persistent form
    bool f8;                    // E4M3 operands (exact small integers), FP32 accumulators
    const CUtensorMap* tm_w;    // device-resident tensor map over the packed weights (256-token tiles stage them by TMA)
    const float* w_scales_t;    // [K/G][N]
    int M, N, K, G;
    const float* row_scale;     // r [M]
    const float* bias;          // [N] or nullptr
    // accumulator dump (parity hook); acc == nullptr in production
    int32_t* acc;
    int row0, rows, col0, cols;
    float* partials;            // split-K scratch (see gemm_i8_scratch_bytes) or nullptr
    int* counters;              // per-tile arrival counters, zeroed by the prologue kernel, or nullptr
};
struct GemmI8Plan {
    int token_tile;             // tokens per CTA tile: sizes the TMA boxes
    int splitk;                 // K splits
    bool pdl;                   // launched with programmatic dependent launch after the prologue kernel
    bool persist;               // persistent form (256-token tiles): one CTA per SM walks the tiles; output store boxes of 64 tokens
};
GemmI8Plan gemm_i8_plan(int M, int N, int K, int G, bool f8, bool dump);
size_t gemm_i8_scratch_bytes(int M, int N, int K, bool dump, size_t* counters_offset);
cudaError_t launch_gemm_i8(const GemmI8Args& a, cudaStream_t st);
cudaError_t gemm_i8_init();     // one-time function attributes (dynamic shared memory opt-in)

// Few rows (action / proprio-only passes): register-level GEMM after the prologue kernel, see gemm_i8_fewrows.cu.
struct GemmI8FewRowsArgs {
    const int8_t* codes; int64_t ldc;   // Q_X int8 [M, ldc]
    const float* row_scale;             // r [M]
    const uint8_t* wq;                  // packed weights
    bool signmag;                       // weights in the sign-magnitude layout (W4A4 with groups up to 128)
    const float* w_scales_t;
    const float* bias;
    uint16_t* Y; int64_t ldy;
    int M, N, K, G;
    int32_t* acc;                       // accumulator dump (parity hook) or nullptr
    int row0, rows, col0, cols;
};
bool gemm_i8_fewrows_applies(int M, int N, int K, int G);
cudaError_t launch_gemm_i8_fewrows(const GemmI8FewRowsArgs& a, cudaStream_t st);
// A few dozen to a few hundred rows: register-level GEMM with shared-memory operand staging, see gemm_i8_midrows.cu.
bool gemm_i8_midrows_applies(int M, int N, int K, int G, bool signmag);
cudaError_t launch_gemm_i8_midrows(const GemmI8FewRowsArgs& a, cudaStream_t st);
// Either of the two: the prologue then writes int8 codes whatever the weight layout.
inline bool gemm_i8_register_path(int M, int N, int K, int G, bool signmag) { return gemm_i8_fewrows_applies(M, N, K, G) || gemm_i8_midrows_applies(M, N, K, G, signmag); }

}  // namespace rudder
