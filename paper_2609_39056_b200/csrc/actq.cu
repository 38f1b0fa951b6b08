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

// ---- one row per CTA step ------------------------------------------------------------------------
// The warp-per-row kernels above keep a whole row in one warp's registers, which caps the occupancy and
// leaves the memory system idle while a warp computes.  Here a row is spread over the T threads of a
// CTA (T = row pieces, up to 1024; NCH pieces per thread for longer rows).  The CTA is persistent: it
// walks rows blockIdx.x, blockIdx.x + gridDim.x, ..., so a thread always meets the same input channels
// and keeps their dinv in registers, and it issues the loads of its next row before working on the
// current one.  Range pass: max_k |x dinv| and one multiplication by gamma -- identical bits to
// max_k |(x dinv) gamma| because rounding is monotonic and gamma > 0.
__device__ __forceinline__ float block_max(float m, float* red /* [32] shared */) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    const int n_warps = (blockDim.x + 31) >> 5;
    if (n_warps == 1) return m;
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = m;
    __syncthreads();
    float r = (static_cast<int>(threadIdx.x & 31) < n_warps) ? red[threadIdx.x & 31] : 0.0f;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) r = fmaxf(r, __shfl_xor_sync(0xffffffffu, r, o));
    return r;
}

// x (8 bf16) * dinv -> 8 fp32 (the first of the two roundings of v = (x dinv) gamma)
__device__ __forceinline__ void mul_dinv8(const uint4& x, const float (&dd)[8], float (&u)[8]) {
    const uint32_t w[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        u[2 * i] = __fmul_rn(__uint_as_float(w[i] << 16), dd[2 * i]);
        u[2 * i + 1] = __fmul_rn(__uint_as_float(w[i] & 0xFFFF0000u), dd[2 * i + 1]);
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

template <int NCH>
__global__ void __launch_bounds__(1024) actq_int_row_kernel(ActqArgs a, int qmax, int8_t* __restrict__ codes, int64_t ldc,
                                                             float* __restrict__ r)
{
    __shared__ float red[2][32];
    const int t = threadIdx.x;
    const int T = blockDim.x;
    const int n_chunks = a.K >> 3;
    const float qmaxf = static_cast<float>(qmax);
    // Let a dependent GEMM launched with programmatic dependent launch start its own set-up now; it
    // still waits for this whole grid to finish before it reads anything written here.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (blockIdx.x == 0 && a.zero_ints != nullptr)
        for (int i = t; i < a.n_zero; i += T) a.zero_ints[i] = 0;

    float dd[NCH][8];
#pragma unroll
    for (int i = 0; i < NCH; ++i) {
        const int c = i * T + t;
        const float4 d0 = (c < n_chunks) ? __ldg(reinterpret_cast<const float4*>(a.dinv) + 2 * c) : make_float4(0, 0, 0, 0);
        const float4 d1 = (c < n_chunks) ? __ldg(reinterpret_cast<const float4*>(a.dinv) + 2 * c + 1) : make_float4(0, 0, 0, 0);
        dd[i][0] = d0.x; dd[i][1] = d0.y; dd[i][2] = d0.z; dd[i][3] = d0.w;
        dd[i][4] = d1.x; dd[i][5] = d1.y; dd[i][6] = d1.z; dd[i][7] = d1.w;
    }
    auto load_row = [&](int row, uint4 (&x)[NCH]) {
        const bool live = row < a.M;
        const uint4* xrow = reinterpret_cast<const uint4*>(a.X + static_cast<size_t>(live ? row : 0) * a.ldx);
#pragma unroll
        for (int i = 0; i < NCH; ++i) {
            const int c = i * T + t;
            x[i] = (live && c < n_chunks) ? ld_nc_16(xrow + c) : make_uint4(0, 0, 0, 0);
        }
    };

    uint4 nxt[NCH];
    load_row(blockIdx.x, nxt);
    int par = 0;
    for (int row = blockIdx.x; row < a.M; row += gridDim.x, par ^= 1) {
        float u[NCH][8];
        float m = 0.0f;
#pragma unroll
        for (int i = 0; i < NCH; ++i) {
            mul_dinv8(nxt[i], dd[i], u[i]);       // pieces past the row end are zero
#pragma unroll
            for (int j = 0; j < 8; ++j) m = fmaxf(m, fabsf(u[i][j]));
        }
        load_row(row + gridDim.x, nxt);            // prefetch the next row
        const float g = a.gamma_step[stream_of_row(a.seg, row)];
        float range;
        if (a.clip_step == nullptr) range = __fmul_rn(block_max(m, red[par]), g);
        else                        range = *a.clip_step;
        const float inv = (range != 0.0f) ? __fdiv_rn(qmaxf, range) : 0.0f;
        uint2* crow = reinterpret_cast<uint2*>(codes + static_cast<size_t>(row) * ldc);
#pragma unroll
        for (int i = 0; i < NCH; ++i) {
            const int c = i * T + t;
            if (c < n_chunks) {
                float v[8];
#pragma unroll
                for (int j = 0; j < 8; ++j) v[j] = __fmul_rn(u[i][j], g);
                crow[c] = (a.clip_step == nullptr) ? round8_fast<false>(v, inv, qmaxf) : round8_fast<true>(v, inv, qmaxf);
            }
        }
        if (t == 0) r[row] = (range != 0.0f) ? __fdiv_rn(__fdiv_rn(range, qmaxf), g) : 0.0f;
    }
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

template <int NCH>
__global__ void __launch_bounds__(1024) actq_nvfp4_row_kernel(ActqArgs a, int M_pad, uint8_t* __restrict__ codes,
                                                               uint8_t* __restrict__ sf, int sf_tiled, float* __restrict__ r)
{
    __shared__ float red[2][32];
    const int t = threadIdx.x;
    const int T = blockDim.x;
    const int lane = t & 31;
    const int n_blocks = a.K >> 4;
    const int k64 = a.K >> 6;

    float dd[NCH][16];
#pragma unroll
    for (int i = 0; i < NCH; ++i) {
        const int kb = i * T + t;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const float4 d4 = (kb < n_blocks) ? __ldg(reinterpret_cast<const float4*>(a.dinv) + 4 * kb + j) : make_float4(0, 0, 0, 0);
            dd[i][4 * j] = d4.x; dd[i][4 * j + 1] = d4.y; dd[i][4 * j + 2] = d4.z; dd[i][4 * j + 3] = d4.w;
        }
    }
    auto load_row = [&](int row, uint4 (&x)[2 * NCH]) {
        const bool live = row < a.M;
        const uint4* xrow = reinterpret_cast<const uint4*>(a.X + static_cast<size_t>(live ? row : 0) * a.ldx);
#pragma unroll
        for (int i = 0; i < NCH; ++i) {
            const int kb = i * T + t;
            const bool in = live && kb < n_blocks;
            x[2 * i] = in ? ld_nc_16(xrow + 2 * kb) : make_uint4(0, 0, 0, 0);
            x[2 * i + 1] = in ? ld_nc_16(xrow + 2 * kb + 1) : make_uint4(0, 0, 0, 0);
        }
    };
    // four neighbouring lanes own the four blocks of one 64-channel step: one 32-bit store for their scales
    auto store_sf = [&](int row, int kb, uint32_t sb) {
        uint32_t word = sb << (8 * (lane & 3));
        word |= __shfl_xor_sync(0xffffffffu, word, 1);
        word |= __shfl_xor_sync(0xffffffffu, word, 2);
        if ((lane & 3) == 0 && kb < n_blocks) {
            const size_t off = sf_tiled ? nvfp4_sf_offset(row, kb, k64) : static_cast<size_t>(row) * n_blocks + kb;
            *reinterpret_cast<uint32_t*>(sf + off) = word;
        }
    };

    uint4 nxt[2 * NCH];
    load_row(blockIdx.x, nxt);
    int par = 0;
    for (int row = blockIdx.x; row < M_pad; row += gridDim.x, par ^= 1) {
        if (row >= a.M) {                          // padding row of the last 128-row scale atom: zero scales
#pragma unroll
            for (int i = 0; i < NCH; ++i) store_sf(row, i * T + t, 0u);
            continue;
        }
        float u[NCH][16];
        float m = 0.0f;
#pragma unroll
        for (int i = 0; i < NCH; ++i) {
            float lo8[8], hi8[8];
            mul_dinv8(nxt[2 * i], *reinterpret_cast<const float(*)[8]>(&dd[i][0]), lo8);
            mul_dinv8(nxt[2 * i + 1], *reinterpret_cast<const float(*)[8]>(&dd[i][8]), hi8);
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                u[i][j] = lo8[j];
                u[i][8 + j] = hi8[j];
                m = fmaxf(m, fmaxf(fabsf(lo8[j]), fabsf(hi8[j])));
            }
        }
        load_row(row + gridDim.x, nxt);
        const float g = a.gamma_step[stream_of_row(a.seg, row)];
        float range;
        if (a.clip_step == nullptr) range = __fmul_rn(block_max(m, red[par]), g);
        else                        range = *a.clip_step;
        const float inv = (range != 0.0f) ? __fdiv_rn(kNvfp4Range, range) : 0.0f;
        uint2* crow = reinterpret_cast<uint2*>(codes + static_cast<size_t>(row) * (a.K >> 1));
#pragma unroll
        for (int i = 0; i < NCH; ++i) {
            const int kb = i * T + t;
            float v[16];
#pragma unroll
            for (int j = 0; j < 16; ++j) v[j] = __fmul_rn(__fmul_rn(u[i][j], g), inv);
            uint32_t lo, hi;
            const uint32_t sb = nvfp4_encode_block(v, lo, hi);
            if (kb < n_blocks) crow[kb] = make_uint2(lo, hi);
            store_sf(row, kb, sb);
        }
        if (t == 0) r[row] = (range != 0.0f) ? __fdiv_rn(__fdiv_rn(range, kNvfp4Range), g) : 0.0f;
    }
}

// Threads per CTA and pieces per thread for a row of n pieces.
static void row_launch_shape(int n, int& threads, int& nch) {
    nch = (n + 1023) / 1024;
    threads = ((n + nch - 1) / nch + 31) / 32 * 32;
}
static int row_grid(int rows, int threads) {
    const int per_sm = 2048 / threads > 0 ? 2048 / threads : 1;
    const int cap = 148 * (per_sm > 8 ? 8 : per_sm);
    return rows < cap ? rows : cap;
}

// The GEMMs that follow these kernels use ~200 KB of shared memory.  Asking for the same carve-out here
// keeps the SM's L1 / shared-memory split from being reconfigured at every kernel boundary.
cudaError_t actq_init()
{
    cudaError_t e;
#define RUDDER_CARVE(K)                                                                                         \
    e = cudaFuncSetAttribute(K, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared); \
    if (e != cudaSuccess) return e;
    RUDDER_CARVE(actq_int_row_kernel<1>) RUDDER_CARVE(actq_int_row_kernel<2>) RUDDER_CARVE(actq_int_row_kernel<4>)
    RUDDER_CARVE(actq_int_kernel<0>)
    RUDDER_CARVE(actq_nvfp4_row_kernel<1>) RUDDER_CARVE(actq_nvfp4_row_kernel<2>) RUDDER_CARVE(actq_nvfp4_kernel<0>)
#undef RUDDER_CARVE
    return cudaSuccess;
}

cudaError_t launch_actq_nvfp4(const ActqArgs& a, uint8_t* codes, uint8_t* sf, bool sf_tiled, float* r, cudaStream_t st)
{
    const int M_pad = sf_tiled ? ((a.M + 127) / 128) * 128 : a.M;
    const int tiled = sf_tiled ? 1 : 0;
    int threads, nch;
    row_launch_shape(a.K / 16, threads, nch);
    const int grid = row_grid(M_pad, threads);
    if (nch == 1)      actq_nvfp4_row_kernel<1><<<grid, threads, 0, st>>>(a, M_pad, codes, sf, tiled, r);
    else if (nch == 2) actq_nvfp4_row_kernel<2><<<grid, threads, 0, st>>>(a, M_pad, codes, sf, tiled, r);
    else {
        const int blocks = (M_pad * 32 + 255) / 256;      // very long rows: one warp per row, row read twice
        actq_nvfp4_kernel<0><<<blocks, 256, 0, st>>>(a, M_pad, codes, sf, tiled, r);
    }
    return cudaGetLastError();
}

cudaError_t launch_actq_int(const ActqArgs& a, int qmax, int8_t* codes, int64_t ldc, float* r, cudaStream_t st)
{
    int threads, nch;
    row_launch_shape(a.K / 8, threads, nch);
    const int grid = row_grid(a.M, threads);
    if (nch == 1)      actq_int_row_kernel<1><<<grid, threads, 0, st>>>(a, qmax, codes, ldc, r);
    else if (nch == 2) actq_int_row_kernel<2><<<grid, threads, 0, st>>>(a, qmax, codes, ldc, r);
    else if (nch <= 4) actq_int_row_kernel<4><<<grid, threads, 0, st>>>(a, qmax, codes, ldc, r);
    else {
        const int blocks = (a.M * 32 + 255) / 256;         // very long rows: one warp per row, row read twice
        actq_int_kernel<0><<<blocks, 256, 0, st>>>(a, qmax, codes, ldc, r);
    }
    return cudaGetLastError();
}

}  // namespace rudder
