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

#include <cuda_fp16.h>

constexpr int kRowNch = 2;          // blocks of 16 channels per thread of the row kernels

namespace rudder {

// ---- self-test of the bounded-wait path -------------------------------------------------------------
// One warp waits, with a short cycle limit, on a barrier that nobody signals (no copy, no tensor memory,
// nothing in flight), gives up, records the time-out in the device status word and returns.
constexpr int W_SELFTEST = 901;
__global__ void wait_timeout_selftest_kernel(long long limit_cycles)
{
    __shared__ __align__(8) uint64_t bar;
    __shared__ int abort_word;
    if (threadIdx.x == 0) {
        abort_word = 0;
        mbar_init(smem_u32(&bar), 1);
        fence_mbar_init();
    }
    __syncthreads();
    bool ok = mbar_wait<32>(smem_u32(&bar), 0, &abort_word, W_SELFTEST, limit_cycles);
    ok = __syncthreads_and(ok) != 0;          // the whole CTA leaves together
    (void)ok;
}
cudaError_t launch_wait_timeout_selftest(long long limit_cycles, cudaStream_t st)
{
    wait_timeout_selftest_kernel<<<1, 32, 0, st>>>(limit_cycles);
    return cudaGetLastError();
}

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

// Two integer-valued floats in [-7, 7] -> two E4M3 bytes (exact), lo in the low byte.
__device__ __forceinline__ uint32_t e4m3x2(float lo, float hi) {
    uint16_t h;
    asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(h) : "f"(hi), "f"(lo));
    return h;
}
__device__ __forceinline__ uint2 round8_e4m3(const float (&v)[8], float inv, int qmax) {
    const float qf = static_cast<float>(qmax);
    float q[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) q[i] = fminf(fmaxf(rintf(__fmul_rn(v[i], inv)), -qf), qf);
    return make_uint2(e4m3x2(q[0], q[1]) | (e4m3x2(q[2], q[3]) << 16), e4m3x2(q[4], q[5]) | (e4m3x2(q[6], q[7]) << 16));
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
__global__ void __launch_bounds__(256) actq_int_kernel(ActqArgs a, int qmax, int e4m3, int8_t* __restrict__ codes, int64_t ldc,
                                                        float* __restrict__ r)
{
    asm volatile("griddepcontrol.wait;" ::: "memory");     // may have been launched ahead of its stream predecessors
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
                crow[c] = e4m3 ? round8_e4m3(v, inv, qmax) : round8(v, inv, qmax);
            }
        }
    } else {
        for (int it = 0; it < n_it; ++it) {
            const int c = it * 32 + lane;
            if (c < n_chunks) {
                float v[8];
                scale8(ld_nc_16(xrow + c), __ldg(dv + 2 * c), __ldg(dv + 2 * c + 1), g, v);
                crow[c] = e4m3 ? round8_e4m3(v, inv, qmax) : round8(v, inv, qmax);
            }
        }
    }
    if (lane == 0)
        r[row] = (range != 0.0f) ? __fdiv_rn(__fdiv_rn(range, static_cast<float>(qmax)), g) : 0.0f;
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
    asm volatile("griddepcontrol.wait;" ::: "memory");     // may have been launched ahead of its stream predecessors
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

// ---- one row per CTA step ------------------------------------------------------------------------
// The warp-per-row kernels keep a whole row in one warp's registers, which caps the occupancy and
// leaves the memory system idle while a warp computes.  Here a row is spread over the T threads of a
// persistent CTA, NCH blocks of 16 channels per thread, and the CTA walks rows blockIdx.x,
// blockIdx.x + gridDim.x, ...: a thread always meets the same channels and keeps their dinv in
// registers.  Rows are staged in shared memory by bulk copies that run kRowSlots rows ahead of the
// arithmetic (one thread issues them), so the bytes in flight do not depend on registers or occupancy.
// Range pass: max_k |x dinv| and one multiplication by gamma -- identical bits to max_k |(x dinv) gamma|
// because rounding is monotonic and gamma > 0.  The kernel is bound by instruction issue before it is
// bound by HBM, so the arithmetic is kept to the fewest instructions that still round exactly like the
// scalar definition: packed two-lane fp32 multiplies (each lane rounded on its own), one warp-wide
// integer max instruction for the range (non-negative floats order like their bit patterns), a
// shared-memory atomic max across warps, and a table for the reciprocal of the block scale.
constexpr int kRowSlots = 4;
constexpr int kFewRows = 256;                      // up to this many rows the integer prologue runs one CTA per row
constexpr int W_ROW_FULL = 40;                     // wait identifier reported on a timeout

struct RowOut {
    void* codes;               // int8 [M, ldc] or packed E2M1 [M, K/2]
    int64_t ldc;               // bytes per code row
    uint8_t* sf;               // NVFP4 block scales
    int sf_tiled;              // tensor-core order (with zeroed padding rows up to M_pad) or row-major
    float* r;
    int M_pad;
    int qmax;
    int e4m3;                  // integer codes written as E4M3 bytes
};

typedef unsigned long long f32x2;                  // two fp32 lanes in one 64-bit register pair
__device__ __forceinline__ f32x2 pack2(float lo, float hi) {
    f32x2 p;
    asm("mov.b64 %0, {%1, %2};" : "=l"(p) : "f"(lo), "f"(hi));
    return p;
}
__device__ __forceinline__ void unpack2(f32x2 p, float& lo, float& hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(p));
}
// a *= b per lane, each product rounded to nearest on its own
__device__ __forceinline__ void mul2(f32x2& a, f32x2 b) {
    asm("mul.rn.f32x2 %0, %0, %1;" : "+l"(a) : "l"(b));
}
__device__ __forceinline__ uint4 lds128(uint32_t addr) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
}
__device__ __forceinline__ void bulk_row_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}

// Maximum over the CTA of a non-negative float.  `red` holds three slots that rotate from row to row:
// slot (i + 1) % 3 is cleared while row i is reduced; it was last read before the barrier of row i - 1,
// which thread 0 has already passed, and is next written after the barrier of row i.
// `ok` goes through the same barrier (AND over the CTA), so that every thread learns whether any thread
// gave up its wait for the row and all of them leave the row loop together.
__device__ __forceinline__ float cta_max_nonneg(float m, uint32_t* red, int& slot, bool& ok) {
    const uint32_t wm = __reduce_max_sync(0xffffffffu, __float_as_uint(m));
    const int nxt = (slot == 2) ? 0 : slot + 1;
    if ((threadIdx.x & 31) == 0) atomicMax(red + slot, wm);
    if (threadIdx.x == 0) red[nxt] = 0u;
    ok = __syncthreads_and(ok) != 0;
    const float r = __uint_as_float(*reinterpret_cast<volatile uint32_t*>(red + slot));
    slot = nxt;
    return r;
}

// 8 bf16 (one 16-byte word) times 8 channel scales -> 4 lane pairs; returns max |.| of the products
__device__ __forceinline__ float mul_dinv8(const uint4& x, const f32x2* dd, f32x2* u) {
    const uint32_t w[4] = {x.x, x.y, x.z, x.w};
    float lo[4], hi[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        u[i] = pack2(__uint_as_float(w[i] << 16), __uint_as_float(w[i] & 0xFFFF0000u));
        mul2(u[i], dd[i]);
        unpack2(u[i], lo[i], hi[i]);
    }
    float m = fmaxf(fabsf(lo[0]), fabsf(hi[0]));
#pragma unroll
    for (int i = 1; i < 4; ++i) m = fmaxf(fmaxf(m, fabsf(lo[i])), fabsf(hi[i]));
    return m;
}

// Correctly rounded a / 6 for a >= 0 (quotient, remainder by fma, one correction; checked against the
// IEEE division for every float whose quotient is a normal number -- smaller ones encode as zero).
__device__ __forceinline__ float div6(float a) {
    const float c = 1.0f / 6.0f;
    const float q0 = __fmul_rn(a, c);
    const float rem = __fmaf_rn(-6.0f, q0, a);
    return __fmaf_rn(rem, c, q0);
}

// Four lane pairs -> eight E2M1 codes in one word, element i in nibble i.
__device__ __forceinline__ uint32_t e2m1x8(const f32x2* v) {
    float f[8];
#pragma unroll
    for (int i = 0; i < 4; ++i) unpack2(v[i], f[2 * i], f[2 * i + 1]);
    return f32x8_to_e2m1(f);
}
// Four lane pairs -> eight int8 codes.  CLAMP: static range (values may exceed the range).
template <bool CLAMP>
__device__ __forceinline__ uint2 s8x8(const f32x2* v, float qmaxf) {
    int q[8];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        float lo, hi;
        unpack2(v[i], lo, hi);
        if (CLAMP) { lo = fminf(fmaxf(lo, -qmaxf), qmaxf); hi = fminf(fmaxf(hi, -qmaxf), qmaxf); }
        q[2 * i] = __float2int_rn(lo);
        q[2 * i + 1] = __float2int_rn(hi);
    }
    uint32_t lo, hi, t0, t1;
    // cvt.pack: two s32 -> two saturated s8 in the low half, third operand supplies the upper half
    asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, 0;" : "=r"(t0) : "r"(q[3]), "r"(q[2]));
    asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(lo) : "r"(q[1]), "r"(q[0]), "r"(t0));
    asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, 0;" : "=r"(t1) : "r"(q[7]), "r"(q[6]));
    asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(hi) : "r"(q[5]), "r"(q[4]), "r"(t1));
    return make_uint2(lo, hi);
}

// Four lane pairs -> eight E4M3 bytes holding the rounded integers (|.| <= qmaxf <= 7).
__device__ __forceinline__ uint2 e4m3x8(const f32x2* v, float qmaxf) {
    uint32_t h[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        float lo, hi;
        unpack2(v[i], lo, hi);
        lo = fminf(fmaxf(rintf(lo), -qmaxf), qmaxf);
        hi = fminf(fmaxf(rintf(hi), -qmaxf), qmaxf);
        h[i] = e4m3x2(lo, hi);
    }
    return make_uint2(h[0] | (h[1] << 16), h[2] | (h[3] << 16));
}

// ---- few rows (up to 256): one CTA per row ---------------------------------------------------------
// With a handful of rows the prologue is pure latency, so it is kept to one round trip: the 256 threads
// of a CTA load the whole row at once (NP 16-byte pieces each, rows up to 2048 NP channels), the range
// is reduced through shared memory with one barrier, the codes are rounded from the registers.  The
// arithmetic is the packed two-lane form of the row kernel (mul_dinv8, s8x8, e4m3x8): the very device
// functions the fused small-M GEMM quantises with, so this kernel doubles as its parity hook.
template <int NP>
__global__ void __launch_bounds__(256) actq_int_cta_row_kernel(ActqArgs a, int qmax, int e4m3, int8_t* __restrict__ codes, int64_t ldc,
                                                                float* __restrict__ r)
{
    __shared__ uint32_t wmax[8];
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // the GEMM behind this kernel may start its set-up
    asm volatile("griddepcontrol.wait;" ::: "memory");                // X may come from the kernel before this one
    const int row = blockIdx.x;
    const int t = threadIdx.x;
    if (row == 0 && a.zero_ints != nullptr)
        for (int i = t; i < a.n_zero; i += 256) a.zero_ints[i] = 0;
    const float g = a.gamma_step[stream_of_row(a.seg, row)];
    const uint4* xrow = reinterpret_cast<const uint4*>(a.X + static_cast<size_t>(row) * a.ldx);
    const float4* dv = reinterpret_cast<const float4*>(a.dinv);
    const int n_chunks = a.K >> 3;
    uint4 xr[NP];
    f32x2 dd[NP][4];
#pragma unroll
    for (int i = 0; i < NP; ++i) {
        const int c = t + i * 256;
        if (c < n_chunks) {
            xr[i] = ld_nc_16(xrow + c);
            const float4 d0 = __ldg(dv + 2 * c), d1 = __ldg(dv + 2 * c + 1);
            dd[i][0] = pack2(d0.x, d0.y); dd[i][1] = pack2(d0.z, d0.w); dd[i][2] = pack2(d1.x, d1.y); dd[i][3] = pack2(d1.z, d1.w);
        }
    }
    float range;
    if (a.clip_step == nullptr) {
        float amax = 0.0f;                         // max |x dinv|; the gain is applied to the maximum (monotonic rounding, gamma > 0)
#pragma unroll
        for (int i = 0; i < NP; ++i) {
            if (t + i * 256 < n_chunks) {
                f32x2 u[4];
                amax = fmaxf(amax, mul_dinv8(xr[i], dd[i], u));
            }
        }
        const uint32_t wm = __reduce_max_sync(0xffffffffu, __float_as_uint(amax));
        if ((t & 31) == 0) wmax[t >> 5] = wm;
        __syncthreads();
        uint32_t m = wmax[0];
#pragma unroll
        for (int i = 1; i < 8; ++i) m = max(m, wmax[i]);
        range = __fmul_rn(__uint_as_float(m), g);
    } else {
        range = *a.clip_step;
    }
    const float qmaxf = static_cast<float>(qmax);
    const float inv = (range != 0.0f) ? __fdiv_rn(qmaxf, range) : 0.0f;
    const f32x2 g2 = pack2(g, g), inv2 = pack2(inv, inv);
    const bool clamp = a.clip_step != nullptr;
    uint2* crow = reinterpret_cast<uint2*>(codes + static_cast<size_t>(row) * ldc);
#pragma unroll
    for (int i = 0; i < NP; ++i) {
        const int c = t + i * 256;
        if (c < n_chunks) {
            f32x2 u[4];
            mul_dinv8(xr[i], dd[i], u);
#pragma unroll
            for (int k = 0; k < 4; ++k) { mul2(u[k], g2); mul2(u[k], inv2); }
            crow[c] = e4m3 ? e4m3x8(u, qmaxf) : (clamp ? s8x8<true>(u, qmaxf) : s8x8<false>(u, qmaxf));
        }
    }
    if (t == 0) r[row] = (range != 0.0f) ? __fdiv_rn(__fdiv_rn(range, static_cast<float>(qmax)), g) : 0.0f;
}

template <bool FP4, int NCH>
__global__ void __launch_bounds__(NCH == 1 ? 1024 : (NCH == 2 ? 512 : 256)) actq_row_kernel(ActqArgs a, RowOut o)
{
    extern __shared__ __align__(128) uint8_t ring[];          // kRowSlots rows of K bf16
    __shared__ __align__(8) uint64_t full_bar[kRowSlots];
    __shared__ float g_slot[kRowSlots];                        // gain of the row staged in each slot
    __shared__ uint32_t red[3];
    __shared__ float rb_tab[128];                              // 1 / (decoded UE4M3 scale), 0 for a zero scale
    __shared__ int abort_word;

    const int t = threadIdx.x;
    const int T = blockDim.x;
    const int M = a.M;
    const int n_blocks = a.K >> 4;
    const uint32_t row_bytes = static_cast<uint32_t>(a.K) * 2u;
    const int first = blockIdx.x;
    const int stride = gridDim.x;
    const uint32_t ring_addr = smem_u32(ring);
    const uint32_t bar0 = smem_u32(full_bar);
    // Let a dependent GEMM launched with programmatic dependent launch start its own set-up now; it
    // still waits for this whole grid to finish before it reads anything written here.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (t == 0) {
        abort_word = 0;
        for (int i = 0; i < kRowSlots; ++i) mbar_init(bar0 + 8u * i, 1);
        fence_mbar_init();
    }
    if (t < 3) red[t] = 0u;
    if (FP4) {
        for (int i = t; i < 128; i += T) {
            const float sbd = ue4m3_to_f32(i);
            rb_tab[i] = (sbd != 0.0f && i < 127) ? __fdiv_rn(1.0f, sbd) : 0.0f;
        }
    }
    __syncthreads();

    // this CTA's rows: first + j * stride; j < n_live are rows of X, the rest (NVFP4, tiled scales) are
    // the padding rows of the last 128-row scale atom, which only get zero scales
    const int M_rows = FP4 ? o.M_pad : M;
    const int n_rows = first < M_rows ? (M_rows - 1 - first) / stride + 1 : 0;
    const int n_live = first < M ? (M - 1 - first) / stride + 1 : 0;
    f32x2 dd[NCH][8];
    uint32_t lds_off[NCH];                         // byte offset of the thread's blocks in a staged row
    size_t sf_col[NCH];                            // column part of the scale's address
#pragma unroll
    for (int i = 0; i < NCH; ++i) {
        const int kb = i * T + t;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const float4 d4 = (kb < n_blocks) ? __ldg(reinterpret_cast<const float4*>(a.dinv) + 4 * kb + j) : make_float4(0, 0, 0, 0);
            dd[i][2 * j] = pack2(d4.x, d4.y);
            dd[i][2 * j + 1] = pack2(d4.z, d4.w);
        }
        lds_off[i] = static_cast<uint32_t>(kb < n_blocks ? kb : n_blocks - 1) * 32u;   // spare threads re-read the last block (their dinv is 0)
        sf_col[i] = o.sf_tiled ? static_cast<size_t>(kb >> 2) * 512 + (kb & 3) : static_cast<size_t>(kb);
    }
    // This kernel may itself have been launched early (programmatic dependent launch): everything above
    // touches only what belongs to the weights or to this CTA.  From here on it reads X and writes the
    // workspace, which the kernels before it in the stream may still be producing or reading.
    asm volatile("griddepcontrol.wait;" ::: "memory");
    if (blockIdx.x == 0 && a.zero_ints != nullptr)
        for (int i = t; i < a.n_zero; i += T) a.zero_ints[i] = 0;
    auto issue = [&](int j) {                                  // thread 0: stage row j of this CTA
        const int slot = j & (kRowSlots - 1);
        const int row = first + j * stride;
        g_slot[slot] = __ldg(a.gamma_step + stream_of_row(a.seg, row));
        mbar_expect_tx(bar0 + 8u * slot, row_bytes);
        bulk_row_load(ring_addr + slot * row_bytes, a.X + static_cast<size_t>(row) * a.ldx, row_bytes, bar0 + 8u * slot);
    };
    if (t == 0)
        for (int j = 0; j < kRowSlots && j < n_live; ++j) issue(j);

    const bool per_token = a.clip_step == nullptr;
    const float clip = per_token ? 0.0f : __ldg(a.clip_step);
    const float range_max = FP4 ? kNvfp4Range : static_cast<float>(o.qmax);
    const int k64 = a.K >> 6;

    int slot3 = 0;
    for (int j = 0; j < n_rows; ++j) {
        const int row = first + j * stride;
        const size_t sf_row = !FP4 ? 0 : (o.sf_tiled ? static_cast<size_t>(row >> 7) * k64 * 512 + (row & 31) * 16 + ((row >> 5) & 3) * 4
                                                     : static_cast<size_t>(row) * n_blocks);
        if (j >= n_live) {                         // padding row: zero scales
            if (FP4) {
#pragma unroll
                for (int i = 0; i < NCH; ++i)
                    if (i * T + t < n_blocks) o.sf[sf_row + sf_col[i]] = 0;
            }
            continue;
        }
        const int slot = j & (kRowSlots - 1);
        // A thread whose wait gave up still walks to the row's barrier, where the outcome becomes common to
        // the CTA (what it computes from the unfinished row meanwhile is discarded).
        bool ok = mbar_wait<20>(bar0 + 8u * slot, (j / kRowSlots) & 1, &abort_word, W_ROW_FULL);
        const float g = g_slot[slot];
        const uint32_t src = ring_addr + slot * row_bytes;

        f32x2 u[NCH][8];
        float mb[NCH];                             // per block: max |x dinv|
        float m = 0.0f;
#pragma unroll
        for (int i = 0; i < NCH; ++i) {
            const uint4 x0 = lds128(src + lds_off[i]);
            const uint4 x1 = lds128(src + lds_off[i] + 16);
            const float m0 = mul_dinv8(x0, &dd[i][0], &u[i][0]);
            const float m1 = mul_dinv8(x1, &dd[i][4], &u[i][4]);
            mb[i] = fmaxf(m0, m1);
            m = fmaxf(m, mb[i]);
        }
        float range;
        if (per_token) range = __fmul_rn(cta_max_nonneg(m, red, slot3, ok), g);
        else { ok = __syncthreads_and(ok) != 0; range = clip; }
        if (!ok) {
            // let the copies already in flight land before the CTA's shared memory goes away (bounded)
            if (t == 0)
                for (int jj = j; jj < n_live && jj < j + kRowSlots; ++jj)
                    for (uint32_t it = 0; it < (1u << 16) && !mbar_try_wait(bar0 + 8u * (jj & (kRowSlots - 1)), (jj / kRowSlots) & 1); ++it) {}
            break;
        }
        // every thread has consumed the staged row: refill its slot
        if (t == 0 && j + kRowSlots < n_live) issue(j + kRowSlots);
        const float inv = (range != 0.0f) ? __fdiv_rn(range_max, range) : 0.0f;
        const f32x2 g2 = pack2(g, g), inv2 = pack2(inv, inv);
#pragma unroll
        for (int i = 0; i < NCH; ++i) {
            const int kb = i * T + t;
            if (FP4) {
                // The block's largest scaled magnitude is the scaled largest magnitude: both
                // multiplications are monotonic, so no second max pass over the 16 values is needed.
                const float vmax = __fmul_rn(__fmul_rn(mb[i], g), inv);
                const uint32_t sb = f32_to_ue4m3(div6(vmax));
                const float rb = rb_tab[sb];
                const f32x2 rb2 = pack2(rb, rb);
#pragma unroll
                for (int k = 0; k < 8; ++k) { mul2(u[i][k], g2); mul2(u[i][k], inv2); mul2(u[i][k], rb2); }
                uint32_t lo = e2m1x8(&u[i][0]);
                uint32_t hi = e2m1x8(&u[i][4]);
                if (sb == 0u) { lo = 0u; hi = 0u; }    // a block whose scale is zero holds +0 codes, not -0 for negative inputs
                if (kb < n_blocks) {
                    *reinterpret_cast<uint2*>(static_cast<uint8_t*>(o.codes) + static_cast<size_t>(row) * o.ldc + kb * 8) = make_uint2(lo, hi);
                    o.sf[sf_row + sf_col[i]] = static_cast<uint8_t>(sb);
                }
            } else {
#pragma unroll
                for (int k = 0; k < 8; ++k) { mul2(u[i][k], g2); mul2(u[i][k], inv2); }
                const float qmaxf = range_max;
                uint2 q0, q1;
                if (o.e4m3) {
                    q0 = e4m3x8(&u[i][0], qmaxf);
                    q1 = e4m3x8(&u[i][4], qmaxf);
                } else {
                    q0 = per_token ? s8x8<false>(&u[i][0], qmaxf) : s8x8<true>(&u[i][0], qmaxf);
                    q1 = per_token ? s8x8<false>(&u[i][4], qmaxf) : s8x8<true>(&u[i][4], qmaxf);
                }
                if (kb < n_blocks)
                    *reinterpret_cast<uint4*>(static_cast<uint8_t*>(o.codes) + static_cast<size_t>(row) * o.ldc + kb * 16) = make_uint4(q0.x, q0.y, q1.x, q1.y);
            }
        }
        if (t == 0) o.r[row] = (range != 0.0f) ? __fdiv_rn(__fdiv_rn(range, range_max), g) : 0.0f;
    }
}

// Launch that may start before the kernels ahead of it in the stream have finished (programmatic
// dependent launch); the kernel itself waits (griddepcontrol.wait) before it touches their data.
template <typename... KArgs, typename... Args>
static cudaError_t launch_early(void (*kernel)(KArgs...), int grid, int block, size_t smem, cudaStream_t st, Args... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid, 1, 1);
    cfg.blockDim = dim3(block, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, args...);
}

// Blocks of 16 channels per thread and threads per CTA for a row of n blocks.
static bool row_launch_shape(int n, int& threads, int& nch) {
    if (n > 1024) return false;
    nch = n > 512 ? 4 : kRowNch;             // long rows: fewer, fatter threads keep two CTAs per SM
    while (nch > 1 && n < 32 * nch) nch >>= 1;      // short rows: keep a full warp busy
    threads = ((n + nch - 1) / nch + 31) / 32 * 32;
    return true;
}
// Persistent grid: as many CTAs as fit on the device at once.
template <typename Kernel>
static int row_grid(Kernel kernel, int rows, int threads, size_t smem) {
    int dev = 0, sms = 148, per_sm = 1;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, threads, smem) != cudaSuccess || per_sm < 1) per_sm = 1;
    const int cap = sms * per_sm;
    return rows < cap ? rows : cap;
}

cudaError_t actq_init()
{
    cudaError_t e;
#define RUDDER_ROW_ATTR(K)                                                                      \
    e = cudaFuncSetAttribute(K, cudaFuncAttributeMaxDynamicSharedMemorySize, kRowSlots * 32768); \
    if (e != cudaSuccess) return e;
    RUDDER_ROW_ATTR((actq_row_kernel<true, 1>)) RUDDER_ROW_ATTR((actq_row_kernel<true, 2>)) RUDDER_ROW_ATTR((actq_row_kernel<true, 4>))
    RUDDER_ROW_ATTR((actq_row_kernel<false, 1>)) RUDDER_ROW_ATTR((actq_row_kernel<false, 2>)) RUDDER_ROW_ATTR((actq_row_kernel<false, 4>))
#undef RUDDER_ROW_ATTR
    return cudaSuccess;
}

// Rows can be staged by bulk copies when they start on 16-byte boundaries and are at most 16384 channels.
template <bool FP4>
static bool launch_row(const ActqArgs& a, const RowOut& o, int rows, cudaStream_t st, cudaError_t* err)
{
    int threads, nch;
    const bool aligned = (reinterpret_cast<uintptr_t>(a.X) % 16 == 0) && ((a.ldx * 2) % 16 == 0) &&
                         (reinterpret_cast<uintptr_t>(o.codes) % 16 == 0) && (o.ldc % 16 == 0) && (a.K % 16 == 0);
    if (!aligned || !row_launch_shape(a.K / 16, threads, nch)) return false;
    const size_t smem = static_cast<size_t>(kRowSlots) * a.K * 2;
    if (nch == 1)      *err = launch_early(actq_row_kernel<FP4, 1>, row_grid(actq_row_kernel<FP4, 1>, rows, threads, smem), threads, smem, st, a, o);
    else if (nch == 2) *err = launch_early(actq_row_kernel<FP4, 2>, row_grid(actq_row_kernel<FP4, 2>, rows, threads, smem), threads, smem, st, a, o);
    else               *err = launch_early(actq_row_kernel<FP4, 4>, row_grid(actq_row_kernel<FP4, 4>, rows, threads, smem), threads, smem, st, a, o);
    return true;
}

// Parity hook: E4M3 bytes (the form the E4M3 tensor path reads) -> the int8 codes they stand for, in place.
__global__ void e4m3_to_int8_kernel(uint32_t* __restrict__ codes, size_t n_words)
{
    for (size_t i = blockIdx.x * static_cast<size_t>(blockDim.x) + threadIdx.x; i < n_words; i += static_cast<size_t>(gridDim.x) * blockDim.x) {
        const uint32_t w = codes[i];
        uint32_t h01, h23;
        asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(h01) : "h"(static_cast<uint16_t>(w & 0xFFFFu)));
        asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(h23) : "h"(static_cast<uint16_t>(w >> 16)));
        const __half2 a = *reinterpret_cast<const __half2*>(&h01), b = *reinterpret_cast<const __half2*>(&h23);
        const int q0 = __half2int_rn(__low2half(a)), q1 = __half2int_rn(__high2half(a));
        const int q2 = __half2int_rn(__low2half(b)), q3 = __half2int_rn(__high2half(b));
        codes[i] = (q0 & 0xFF) | ((q1 & 0xFF) << 8) | ((q2 & 0xFF) << 16) | (static_cast<uint32_t>(q3 & 0xFF) << 24);
    }
}

cudaError_t launch_e4m3_to_int8(int8_t* codes, size_t n_bytes, cudaStream_t st)
{
    const size_t n_words = n_bytes / 4;
    const int blocks = static_cast<int>(n_words / 256 + 1 < 2048 ? n_words / 256 + 1 : 2048);
    e4m3_to_int8_kernel<<<blocks, 256, 0, st>>>(reinterpret_cast<uint32_t*>(codes), n_words);
    return cudaGetLastError();
}

cudaError_t launch_actq_nvfp4(const ActqArgs& a, uint8_t* codes, uint8_t* sf, bool sf_tiled, float* r, cudaStream_t st)
{
    const int M_pad = sf_tiled ? ((a.M + 127) / 128) * 128 : a.M;
    RowOut o;
    o.codes = codes; o.ldc = a.K / 2; o.sf = sf; o.sf_tiled = sf_tiled ? 1 : 0; o.r = r; o.M_pad = M_pad; o.qmax = 0; o.e4m3 = 0;
    cudaError_t err = cudaSuccess;
    if (!launch_row<true>(a, o, M_pad, st, &err)) {
        const int blocks = (M_pad * 32 + 255) / 256;      // unaligned or very long rows: one warp per row, row read twice
        err = launch_early(actq_nvfp4_kernel<0>, blocks, 256, 0, st, a, M_pad, codes, sf, o.sf_tiled, r);
    }
    return err != cudaSuccess ? err : cudaGetLastError();
}

cudaError_t launch_actq_int(const ActqArgs& a, int qmax, bool e4m3, int8_t* codes, int64_t ldc, float* r, cudaStream_t st)
{
    RowOut o;
    o.codes = codes; o.ldc = ldc; o.sf = nullptr; o.sf_tiled = 0; o.r = r; o.M_pad = a.M; o.qmax = qmax; o.e4m3 = e4m3 ? 1 : 0;
    cudaError_t err = cudaSuccess;
    const bool aligned16 = (reinterpret_cast<uintptr_t>(a.X) % 16 == 0) && ((a.ldx * 2) % 16 == 0) &&
                           (reinterpret_cast<uintptr_t>(codes) % 8 == 0) && (ldc % 8 == 0) && (a.K % 8 == 0);
    if (a.M <= kFewRows && a.K <= 8192 && aligned16) {
        // few rows: one CTA per row, one round trip
        if (a.K <= 2048)      err = launch_early(actq_int_cta_row_kernel<1>, a.M, 256, 0, st, a, qmax, e4m3 ? 1 : 0, codes, ldc, r);
        else if (a.K <= 4096) err = launch_early(actq_int_cta_row_kernel<2>, a.M, 256, 0, st, a, qmax, e4m3 ? 1 : 0, codes, ldc, r);
        else                  err = launch_early(actq_int_cta_row_kernel<4>, a.M, 256, 0, st, a, qmax, e4m3 ? 1 : 0, codes, ldc, r);
        return err != cudaSuccess ? err : cudaGetLastError();
    }
    if (!launch_row<false>(a, o, a.M, st, &err)) {
        const int blocks = (a.M * 32 + 255) / 256;         // unaligned or very long rows: one warp per row, row read twice
        if (a.zero_ints != nullptr && cudaMemsetAsync(a.zero_ints, 0, sizeof(int) * a.n_zero, st) != cudaSuccess) return cudaErrorUnknown;
        err = launch_early(actq_int_kernel<0>, blocks, 256, 0, st, a, qmax, e4m3 ? 1 : 0, codes, ldc, r);
    }
    return err != cudaSuccess ? err : cudaGetLastError();
}

}  // namespace rudder
