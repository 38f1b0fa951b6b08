// Activation prologue (Section 4.4, first kernel; Eq. 8; Eq. 1): one pass over X that applies the
// inverse channel scaling D^-1 and the stream gain gamma_{tau,s(i)}, finds the row range, and writes
// only the integer codes Q_X and the row scale r_i = Delta_X / gamma_{s(i)}.
//
// HBM-bound: one warp owns one row; every lane moves 16 bytes (8 bf16) per step so that a warp reads
// 512 contiguous bytes and writes 256 contiguous bytes of codes.  The raw row stays in registers
// between the range pass and the rounding pass (rows up to 8192 channels; longer rows are read a
// second time, from L2).  All fp32 operations are individually rounded, in the order
// v = (x * dinv) * gamma, q = rint(v * (q_max / a)), r = (a / q_max) / gamma.
#include "internal.cuh"
#include "fp4.cuh"

namespace rudder {

__device__ __forceinline__ uint4 ld_nc_16(const uint4* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0, %1, %2, %3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

__device__ __forceinline__ int stream_of_row(const SegParams& seg, int row) {
    int s = 0;
    for (int i = 1; i < seg.n_seg; ++i)
        if (row >= seg.offset[i]) s = i;
    return seg.stream[s];
}

// 8 bf16 (one uint4) x 8 channel scales x gain -> 8 fp32
__device__ __forceinline__ void scale8(const uint4& x, const float4& d0, const float4& d1, float g, float (&v)[8]) {
    const uint32_t w[4] = {x.x, x.y, x.z, x.w};
    const float dd[8] = {d0.x, d0.y, d0.z, d0.w, d1.x, d1.y, d1.z, d1.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const float lo = __uint_as_float(w[i] << 16);
        const float hi = __uint_as_float(w[i] & 0xFFFF0000u);
        v[2 * i] = __fmul_rn(__fmul_rn(lo, dd[2 * i]), g);
        v[2 * i + 1] = __fmul_rn(__fmul_rn(hi, dd[2 * i + 1]), g);
    }
}

__device__ __forceinline__ uint2 round8(const float (&v)[8], float inv, int qmax) {
    uint32_t out[2] = {0u, 0u};
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        int q = __float2int_rn(__fmul_rn(v[i], inv));
        q = max(-qmax, min(qmax, q));
        out[i >> 2] |= (static_cast<uint32_t>(q) & 0xFFu) << (8 * (i & 3));
    }
    return make_uint2(out[0], out[1]);
}

// NIT = number of 256-channel steps whose raw data is kept in registers (0: re-read the row).
template <int NIT>
__global__ void __launch_bounds__(256) actq_int_kernel(ActqArgs a, int qmax, int8_t* __restrict__ codes, int64_t ldc,
                                                        float* __restrict__ r)
{
    const int row = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (row >= a.M) return;
    const float g = a.gamma_step[stream_of_row(a.seg, row)];
    const uint4* xrow = reinterpret_cast<const uint4*>(a.X + static_cast<size_t>(row) * a.ldx);
    const float4* dv = reinterpret_cast<const float4*>(a.dinv);
    const int n_chunks = a.K >> 3;                 // 16-byte chunks in the row
    const int n_it = (n_chunks + 31) >> 5;

    uint4 xr[NIT > 0 ? NIT : 1];
    float amax = 0.0f;
    if (a.clip_step == nullptr || NIT > 0) {
        if (NIT > 0) {
#pragma unroll
            for (int it = 0; it < NIT; ++it) {
                const int c = it * 32 + lane;
                if (c < n_chunks) xr[it] = ld_nc_16(xrow + c);
            }
        }
        if (a.clip_step == nullptr) {
            if (NIT > 0) {
#pragma unroll
                for (int it = 0; it < NIT; ++it) {
                    const int c = it * 32 + lane;
                    if (c < n_chunks) {
                        float v[8];
                        scale8(xr[it], __ldg(dv + 2 * c), __ldg(dv + 2 * c + 1), g, v);
#pragma unroll
                        for (int i = 0; i < 8; ++i) amax = fmaxf(amax, fabsf(v[i]));
                    }
                }
            } else {
                for (int it = 0; it < n_it; ++it) {
                    const int c = it * 32 + lane;
                    if (c < n_chunks) {
                        float v[8];
                        scale8(ld_nc_16(xrow + c), __ldg(dv + 2 * c), __ldg(dv + 2 * c + 1), g, v);
#pragma unroll
                        for (int i = 0; i < 8; ++i) amax = fmaxf(amax, fabsf(v[i]));
                    }
                }
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
        }
    }
    const float range = a.clip_step ? *a.clip_step : amax;     // a_i: shared threshold c_tau, or the row's absmax
    const float inv = (range != 0.0f) ? __fdiv_rn(static_cast<float>(qmax), range) : 0.0f;
    uint2* crow = reinterpret_cast<uint2*>(codes + static_cast<size_t>(row) * ldc);

    if (NIT > 0) {
#pragma unroll
        for (int it = 0; it < NIT; ++it) {
            const int c = it * 32 + lane;
            if (c < n_chunks) {
                float v[8];
                scale8(xr[it], __ldg(dv + 2 * c), __ldg(dv + 2 * c + 1), g, v);
                crow[c] = round8(v, inv, qmax);
            }
        }
    } else {
        for (int it = 0; it < n_it; ++it) {
            const int c = it * 32 + lane;
            if (c < n_chunks) {
                float v[8];
                scale8(ld_nc_16(xrow + c), __ldg(dv + 2 * c), __ldg(dv + 2 * c + 1), g, v);
                crow[c] = round8(v, inv, qmax);
            }
        }
    }
    if (lane == 0)
        r[row] = (range != 0.0f) ? __fdiv_rn(__fdiv_rn(range, static_cast<float>(qmax)), g) : 0.0f;
}

// ---- rows spread over TPR threads ---------------------------------------------------------------
// The warp-per-row kernels above keep a whole row in one warp's registers, which caps the occupancy
// (171 registers at K = 8192) and leaves the memory system idle while a warp computes.  Here a row is
// spread over TPR threads of a 256-thread CTA (256 / TPR rows per CTA), each thread holding at most
// NCH 16-byte pieces, so that registers stay low and many rows are in flight per SM.
// Range pass: max_k |x dinv| and one multiplication by gamma -- identical bits to max_k |(x dinv) gamma|
// because rounding is monotonic and gamma > 0.
template <int TPR>
__device__ __forceinline__ float row_max(float m, float* red /* [8] shared */, int row_in_cta, int tid_in_row) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    if (TPR == 32) return m;
    constexpr int WPR = TPR / 32;                  // warps per row
    const int w_in_row = tid_in_row >> 5;
    if ((tid_in_row & 31) == 0) red[row_in_cta * WPR + w_in_row] = m;
    __syncthreads();
    float r = red[row_in_cta * WPR];
#pragma unroll
    for (int i = 1; i < WPR; ++i) r = fmaxf(r, red[row_in_cta * WPR + i]);
    return r;
}

__device__ __forceinline__ void absmax8(const uint4& x, const float4& d0, const float4& d1, float& m) {
    const uint32_t w[4] = {x.x, x.y, x.z, x.w};
    const float dd[8] = {d0.x, d0.y, d0.z, d0.w, d1.x, d1.y, d1.z, d1.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        m = fmaxf(m, fabsf(__fmul_rn(__uint_as_float(w[i] << 16), dd[2 * i])));
        m = fmaxf(m, fabsf(__fmul_rn(__uint_as_float(w[i] & 0xFFFF0000u), dd[2 * i + 1])));
    }
}

// Eight scaled values -> eight int8 codes.  CLAMP: static range (values may exceed the range).
template <bool CLAMP>
__device__ __forceinline__ uint2 round8_fast(const float (&v)[8], float inv, float qmaxf) {
    int q[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        float t = __fmul_rn(v[i], inv);
        if (CLAMP) t = fminf(fmaxf(t, -qmaxf), qmaxf);
        q[i] = __float2int_rn(t);
    }
    uint32_t lo, hi, t0, t1;
    // cvt.pack: two s32 -> two saturated s8 in the low half, third operand supplies the upper half
    asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, 0;" : "=r"(t0) : "r"(q[3]), "r"(q[2]));
    asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(lo) : "r"(q[1]), "r"(q[0]), "r"(t0));
    asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, 0;" : "=r"(t1) : "r"(q[7]), "r"(q[6]));
    asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(hi) : "r"(q[5]), "r"(q[4]), "r"(t1));
    return make_uint2(lo, hi);
}

template <int TPR, int NCH>
__global__ void __launch_bounds__(256) actq_int_rows_kernel(ActqArgs a, int qmax, int8_t* __restrict__ codes, int64_t ldc,
                                                             float* __restrict__ r)
{
    __shared__ float red[8];
    constexpr int RPC = 256 / TPR;                 // rows per CTA
    const int row_in_cta = threadIdx.x / TPR;
    const int t = threadIdx.x % TPR;
    const int row = blockIdx.x * RPC + row_in_cta;
    const bool live = row < a.M;                   // whole rows are live or not: no divergence inside a row
    const int n_chunks = a.K >> 3;
    const float4* dv = reinterpret_cast<const float4*>(a.dinv);
    const uint4* xrow = reinterpret_cast<const uint4*>(a.X + static_cast<size_t>(live ? row : 0) * a.ldx);
    const float g = live ? a.gamma_step[stream_of_row(a.seg, row)] : 1.0f;

    uint4 xr[NCH];
#pragma unroll
    for (int i = 0; i < NCH; ++i) {
        const int c = i * TPR + t;
        xr[i] = (live && c < n_chunks) ? ld_nc_16(xrow + c) : make_uint4(0, 0, 0, 0);
    }
    float range;
    if (a.clip_step == nullptr) {
        float m = 0.0f;
#pragma unroll
        for (int i = 0; i < NCH; ++i) {
            const int c = i * TPR + t;
            if (c < n_chunks) absmax8(xr[i], __ldg(dv + 2 * c), __ldg(dv + 2 * c + 1), m);
        }
        range = __fmul_rn(row_max<TPR>(m, red, row_in_cta, t), g);
    } else {
        range = *a.clip_step;
    }
    if (!live) return;
    const float inv = (range != 0.0f) ? __fdiv_rn(static_cast<float>(qmax), range) : 0.0f;
    const float qmaxf = static_cast<float>(qmax);
    uint2* crow = reinterpret_cast<uint2*>(codes + static_cast<size_t>(row) * ldc);
#pragma unroll
    for (int i = 0; i < NCH; ++i) {
        const int c = i * TPR + t;
        if (c < n_chunks) {
            float v[8];
            scale8(xr[i], __ldg(dv + 2 * c), __ldg(dv + 2 * c + 1), g, v);
            crow[c] = (a.clip_step == nullptr) ? round8_fast<false>(v, inv, qmaxf) : round8_fast<true>(v, inv, qmaxf);
        }
    }
    if (t == 0) r[row] = (range != 0.0f) ? __fdiv_rn(__fdiv_rn(range, qmaxf), g) : 0.0f;
}


// ---- NVFP4 activations -------------------------------------------------------------------------
// One warp per row; a lane owns one block of 16 channels per step (two 16-byte loads), so a warp step
// covers 512 channels.  Writes packed E2M1 codes [M, K/2], one UE4M3 scale per block (in the tensor
// core's tiled order, or row-major for the parity hook) and the row scale r = (a / 2688) / gamma.
// Rows in [M, M_pad) only get zero scales, so that the GEMM never reads uninitialised scale bytes.
__device__ __forceinline__ void scale16(const uint4& x0, const uint4& x1, const float4* dv, float g, float (&v)[16]) {
    float a[8], b[8];
    scale8(x0, __ldg(dv), __ldg(dv + 1), g, a);
    scale8(x1, __ldg(dv + 2), __ldg(dv + 3), g, b);
#pragma unroll
    for (int i = 0; i < 8; ++i) { v[i] = a[i]; v[8 + i] = b[i]; }
}

template <int NIT>
__global__ void __launch_bounds__(256) actq_nvfp4_kernel(ActqArgs a, int M_pad, uint8_t* __restrict__ codes,
                                                          uint8_t* __restrict__ sf, int sf_tiled, float* __restrict__ r)
{
    const int row = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (row >= M_pad) return;
    const int n_blocks = a.K >> 4;                 // 16-channel blocks in the row
    const int n_it = (n_blocks + 31) >> 5;
    const int k64 = a.K >> 6;
    if (row >= a.M) {                              // padding row of the last 128-row scale atom
        for (int kb = lane; kb < n_blocks; kb += 32) sf[nvfp4_sf_offset(row, kb, k64)] = 0;
        return;
    }
    const float g = a.gamma_step[stream_of_row(a.seg, row)];
    const uint4* xrow = reinterpret_cast<const uint4*>(a.X + static_cast<size_t>(row) * a.ldx);
    const float4* dv = reinterpret_cast<const float4*>(a.dinv);

    uint4 xr[NIT > 0 ? 2 * NIT : 2];
    float amax = 0.0f;
    if (NIT > 0) {
#pragma unroll
        for (int it = 0; it < NIT; ++it) {
            const int kb = it * 32 + lane;
            if (kb < n_blocks) { xr[2 * it] = ld_nc_16(xrow + 2 * kb); xr[2 * it + 1] = ld_nc_16(xrow + 2 * kb + 1); }
        }
    }
    if (a.clip_step == nullptr) {
        if (NIT > 0) {
#pragma unroll
            for (int it = 0; it < NIT; ++it) {
                const int kb = it * 32 + lane;
                if (kb < n_blocks) {
                    float v[16];
                    scale16(xr[2 * it], xr[2 * it + 1], dv + 4 * kb, g, v);
#pragma unroll
                    for (int i = 0; i < 16; ++i) amax = fmaxf(amax, fabsf(v[i]));
                }
            }
        } else {
            for (int it = 0; it < n_it; ++it) {
                const int kb = it * 32 + lane;
                if (kb < n_blocks) {
                    float v[16];
                    scale16(ld_nc_16(xrow + 2 * kb), ld_nc_16(xrow + 2 * kb + 1), dv + 4 * kb, g, v);
#pragma unroll
                    for (int i = 0; i < 16; ++i) amax = fmaxf(amax, fabsf(v[i]));
                }
            }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
    }
    const float range = a.clip_step ? *a.clip_step : amax;
    const float inv = (range != 0.0f) ? __fdiv_rn(kNvfp4Range, range) : 0.0f;
    uint2* crow = reinterpret_cast<uint2*>(codes + static_cast<size_t>(row) * (a.K >> 1));

    auto emit = [&](int kb, const uint4& x0, const uint4& x1) {
        float v[16];
        scale16(x0, x1, dv + 4 * kb, g, v);
#pragma unroll
        for (int i = 0; i < 16; ++i) v[i] = __fmul_rn(v[i], inv);
        uint32_t lo, hi;
        const uint32_t sb = nvfp4_encode_block(v, lo, hi);
        crow[kb] = make_uint2(lo, hi);
        if (sf_tiled) sf[nvfp4_sf_offset(row, kb, k64)] = static_cast<uint8_t>(sb);
        else          sf[static_cast<size_t>(row) * n_blocks + kb] = static_cast<uint8_t>(sb);
    };
    if (NIT > 0) {
#pragma unroll
        for (int it = 0; it < NIT; ++it) {
            const int kb = it * 32 + lane;
            if (kb < n_blocks) emit(kb, xr[2 * it], xr[2 * it + 1]);
        }
    } else {
        for (int it = 0; it < n_it; ++it) {
            const int kb = it * 32 + lane;
            if (kb < n_blocks) emit(kb, ld_nc_16(xrow + 2 * kb), ld_nc_16(xrow + 2 * kb + 1));
        }
    }
    if (lane == 0)
        r[row] = (range != 0.0f) ? __fdiv_rn(__fdiv_rn(range, kNvfp4Range), g) : 0.0f;
}

template <int TPR, int NCH>
__global__ void __launch_bounds__(256) actq_nvfp4_rows_kernel(ActqArgs a, int M_pad, uint8_t* __restrict__ codes,
                                                               uint8_t* __restrict__ sf, int sf_tiled, float* __restrict__ r)
{
    __shared__ float red[8];
    constexpr int RPC = 256 / TPR;
    const int row_in_cta = threadIdx.x / TPR;
    const int t = threadIdx.x % TPR;
    const int row = blockIdx.x * RPC + row_in_cta;
    const int n_blocks = a.K >> 4;
    const int k64 = a.K >> 6;
    const bool live = row < a.M;
    if (!live && row < M_pad) {                    // padding row of the last 128-row scale atom
        for (int kb = t; kb < n_blocks; kb += TPR) sf[nvfp4_sf_offset(row, kb, k64)] = 0;
    }
    const float4* dv = reinterpret_cast<const float4*>(a.dinv);
    const uint4* xrow = reinterpret_cast<const uint4*>(a.X + static_cast<size_t>(live ? row : 0) * a.ldx);
    const float g = live ? a.gamma_step[stream_of_row(a.seg, row)] : 1.0f;

    uint4 xr[2 * NCH];
#pragma unroll
    for (int i = 0; i < NCH; ++i) {
        const int kb = i * TPR + t;
        const bool in = live && kb < n_blocks;
        xr[2 * i] = in ? ld_nc_16(xrow + 2 * kb) : make_uint4(0, 0, 0, 0);
        xr[2 * i + 1] = in ? ld_nc_16(xrow + 2 * kb + 1) : make_uint4(0, 0, 0, 0);
    }
    float range;
    if (a.clip_step == nullptr) {
        float m = 0.0f;
#pragma unroll
        for (int i = 0; i < NCH; ++i) {
            const int kb = i * TPR + t;
            if (kb < n_blocks) {
                absmax8(xr[2 * i], __ldg(dv + 4 * kb), __ldg(dv + 4 * kb + 1), m);
                absmax8(xr[2 * i + 1], __ldg(dv + 4 * kb + 2), __ldg(dv + 4 * kb + 3), m);
            }
        }
        range = __fmul_rn(row_max<TPR>(m, red, row_in_cta, t), g);
    } else {
        range = *a.clip_step;
    }
    if (!live) return;
    const float inv = (range != 0.0f) ? __fdiv_rn(kNvfp4Range, range) : 0.0f;
    uint2* crow = reinterpret_cast<uint2*>(codes + static_cast<size_t>(row) * (a.K >> 1));
#pragma unroll
    for (int i = 0; i < NCH; ++i) {
        const int kb = i * TPR + t;
        if (kb < n_blocks) {
            float v[16];
            scale16(xr[2 * i], xr[2 * i + 1], dv + 4 * kb, g, v);
#pragma unroll
            for (int j = 0; j < 16; ++j) v[j] = __fmul_rn(v[j], inv);
            uint32_t lo, hi;
            const uint32_t sb = nvfp4_encode_block(v, lo, hi);
            crow[kb] = make_uint2(lo, hi);
            if (sf_tiled) sf[nvfp4_sf_offset(row, kb, k64)] = static_cast<uint8_t>(sb);
            else          sf[static_cast<size_t>(row) * n_blocks + kb] = static_cast<uint8_t>(sb);
        }
    }
    if (t == 0) r[row] = (range != 0.0f) ? __fdiv_rn(__fdiv_rn(range, kNvfp4Range), g) : 0.0f;
}

cudaError_t launch_actq_nvfp4(const ActqArgs& a, uint8_t* codes, uint8_t* sf, bool sf_tiled, float* r, cudaStream_t st)
{
    const int M_pad = sf_tiled ? ((a.M + 127) / 128) * 128 : a.M;
    const int tiled = sf_tiled ? 1 : 0;
    const int n_blocks = a.K / 16;
#define RUDDER_FP4_ROWS(TPR, NCH)                                                                                  \
    actq_nvfp4_rows_kernel<TPR, NCH><<<(M_pad + 256 / TPR - 1) / (256 / TPR), 256, 0, st>>>(a, M_pad, codes, sf, tiled, r)
    if (n_blocks <= 32)        RUDDER_FP4_ROWS(32, 1);
    else if (n_blocks <= 64)   RUDDER_FP4_ROWS(64, 1);
    else if (n_blocks <= 128)  RUDDER_FP4_ROWS(128, 1);
    else if (n_blocks <= 256)  RUDDER_FP4_ROWS(256, 1);
    else if (n_blocks <= 512)  RUDDER_FP4_ROWS(256, 2);
    else if (n_blocks <= 768)  RUDDER_FP4_ROWS(256, 3);
    else if (n_blocks <= 1024) RUDDER_FP4_ROWS(256, 4);
    else {
        const int blocks = (M_pad * 32 + 255) / 256;      // very long rows: one warp per row, row read twice
        actq_nvfp4_kernel<0><<<blocks, 256, 0, st>>>(a, M_pad, codes, sf, tiled, r);
    }
#undef RUDDER_FP4_ROWS
    return cudaGetLastError();
}

cudaError_t launch_actq_int(const ActqArgs& a, int qmax, int8_t* codes, int64_t ldc, float* r, cudaStream_t st)
{
    const int n_chunks = a.K / 8;
#define RUDDER_INT_ROWS(TPR, NCH)                                                                                  \
    actq_int_rows_kernel<TPR, NCH><<<(a.M + 256 / TPR - 1) / (256 / TPR), 256, 0, st>>>(a, qmax, codes, ldc, r)
    if (n_chunks <= 32)        RUDDER_INT_ROWS(32, 1);
    else if (n_chunks <= 64)   RUDDER_INT_ROWS(64, 1);
    else if (n_chunks <= 128)  RUDDER_INT_ROWS(128, 1);
    else if (n_chunks <= 256)  RUDDER_INT_ROWS(256, 1);
    else if (n_chunks <= 512)  RUDDER_INT_ROWS(256, 2);
    else if (n_chunks <= 1024) RUDDER_INT_ROWS(256, 4);
    else if (n_chunks <= 1536) RUDDER_INT_ROWS(256, 6);
    else if (n_chunks <= 2048) RUDDER_INT_ROWS(256, 8);
    else {
        const int blocks = (a.M * 32 + 255) / 256;         // very long rows: one warp per row, row read twice
        actq_int_kernel<0><<<blocks, 256, 0, st>>>(a, qmax, codes, ldc, r);
    }
#undef RUDDER_INT_ROWS
    return cudaGetLastError();
}

}  // namespace rudder
