// Second kernel of the engine (Section 4.4; Eq. 10): C = Q_X Q_W on the tcgen05 integer tensor cores
// with INT32 accumulators in TMEM, and an epilogue that applies the weight scales, the row scale
// r_i (which already carries the inverse stream gain) and the bias, writing BF16.
//
// One CTA computes a 128 x NT output tile.  Warp roles (warpgroup-aligned):
//   warp 0        TMA producer: activation codes (int8, 128-byte swizzle), packed INT4 weights, scales
//   warp 1        allocates TMEM; one lane issues tcgen05.mma kind::i8 (M = 128, N = NT, K = 32)
//   warps 4-7     unpack INT4 -> int8 into the swizzled K-major layout the tensor core reads.  The
//                 nibble goes to the TOP half of the byte (value 16 q): two logic ops per 8 weights,
//                 no sign extension; the factor 16 is folded into the fp32 scales at pack time.
//   warps 8-15    epilogue: per weight group, drain the INT32 partial sums from TMEM, convert, and
//                 accumulate fp32(C) * Delta_W[j,g] in registers; finally * r_i + b_j -> bf16.
// The group partials alternate between two TMEM accumulator buffers so that the tensor core works on
// group g + 1 while group g is drained.
//
// Shared memory rings (stage = 128 input channels):
//   A   [SA ][128 rows][128 B]  int8, swizzled by TMA          full: TMA bytes      empty: umma commit
//   Bp  [SBP][NT rows][64 B]    packed nibbles, linear          full: TMA bytes      empty: 128 unpack threads
//   Bu  [SBU][NT rows][128 B]   int8 x16, swizzled by hand      full: 128 threads    empty: umma commit
//   SC  [SSC][NT] fp32          scales of one group             full: TMA bytes      empty: 8 epilogue warps
// TMEM: 2 x NT columns x 128 lanes of INT32.  acc_full[b]: umma commit; acc_empty[b]: 256 threads.
#include "internal.cuh"
#include "ptx.cuh"

#include <cuda_bf16.h>

namespace rudder {

namespace {

constexpr int BM = 128;          // rows per tile
constexpr int KSTAGE = 128;      // input channels (= bytes of int8 per row) per pipeline stage
constexpr int SA = 4;
constexpr int SBP = 4;
constexpr int SSC = 8;
constexpr int A_BYTES = BM * KSTAGE;
constexpr int NUM_THREADS = 512;
constexpr int UNPACK_THREADS = 128;
constexpr int EPI_THREADS = 256;

template <int NT> struct Tile {
    static constexpr int SBU = (NT == 256) ? 2 : 4;
    static constexpr int BP_BYTES = NT * 64;
    static constexpr int BU_BYTES = NT * 128;
    static constexpr int SC_BYTES = NT * 4;
    static constexpr int OFF_A = 0;
    static constexpr int OFF_BU = OFF_A + SA * A_BYTES;
    static constexpr int OFF_BP = OFF_BU + SBU * BU_BYTES;
    static constexpr int OFF_SC = OFF_BP + SBP * BP_BYTES;
    static constexpr int BYTES = OFF_SC + SSC * SC_BYTES;
    static constexpr int DYN_SMEM = BYTES + 1024;    // slack to align the base to 1024 bytes
    static constexpr int TMEM_COLS = 2 * NT;
    static constexpr int EC = NT / 2;                // columns per epilogue thread
};

struct Params {
    int M, N, K, G;
    const float* row_scale;
    const float* bias;
    uint16_t* Y;
    long long ldy;
    int32_t* acc;
    int row0, rows, col0, cols;
    uint32_t a_tx, b_tx, sc_tx;   // bytes one TMA box delivers (boxes are clamped to the tensor extent)
};

enum Where {   // codes recorded when a bounded wait gives up
    W_A_EMPTY = 101, W_BP_EMPTY = 102, W_SC_EMPTY = 103,
    W_BP_FULL = 201, W_BU_EMPTY = 202,
    W_A_FULL = 301, W_BU_FULL = 302, W_ACC_EMPTY = 303,
    W_SC_FULL = 401, W_ACC_FULL = 402
};

__device__ __forceinline__ uint4 lds128(uint32_t addr) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
}
__device__ __forceinline__ void sts128(uint32_t addr, const uint4& v) {
    asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}
__device__ __forceinline__ float4 lds_f4(uint32_t addr) {
    float4 v;
    asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr));
    return v;
}

__device__ __forceinline__ void tmem_ld_chunk(uint32_t taddr, uint32_t (&r)[32]) { tmem_ld_32x32b_x32(taddr, r); }
__device__ __forceinline__ void tmem_ld_chunk(uint32_t taddr, uint32_t (&r)[16]) { tmem_ld_32x32b_x16(taddr, r); }

template <int NT, bool DUMP>
__global__ void __launch_bounds__(NUM_THREADS, 1)
gemm_i8_w4_kernel(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_b,
                  const __grid_constant__ CUtensorMap tm_sc, const Params p)
{
    using T = Tile<NT>;
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t bars[2 * SA + 2 * SBP + 2 * T::SBU + 2 * SSC + 4];
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_word;

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const int m0 = blockIdx.y * BM;
    const int n0 = blockIdx.x * NT;
    const int n_stages = p.K / KSTAGE;
    const int n_groups = p.K / p.G;

    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t bar0 = smem_u32(bars);
    auto a_full = [&](int i) { return bar0 + 8u * i; };
    auto a_empty = [&](int i) { return bar0 + 8u * (SA + i); };
    auto bp_full = [&](int i) { return bar0 + 8u * (2 * SA + i); };
    auto bp_empty = [&](int i) { return bar0 + 8u * (2 * SA + SBP + i); };
    auto bu_full = [&](int i) { return bar0 + 8u * (2 * SA + 2 * SBP + i); };
    auto bu_empty = [&](int i) { return bar0 + 8u * (2 * SA + 2 * SBP + T::SBU + i); };
    auto sc_full = [&](int i) { return bar0 + 8u * (2 * SA + 2 * SBP + 2 * T::SBU + i); };
    auto sc_empty = [&](int i) { return bar0 + 8u * (2 * SA + 2 * SBP + 2 * T::SBU + SSC + i); };
    auto acc_full = [&](int i) { return bar0 + 8u * (2 * SA + 2 * SBP + 2 * T::SBU + 2 * SSC + i); };
    auto acc_empty = [&](int i) { return bar0 + 8u * (2 * SA + 2 * SBP + 2 * T::SBU + 2 * SSC + 2 + i); };

    if (threadIdx.x == 0) {
        abort_word = 0;
        for (int i = 0; i < SA; ++i) { mbar_init(a_full(i), 1); mbar_init(a_empty(i), 1); }
        for (int i = 0; i < SBP; ++i) { mbar_init(bp_full(i), 1); mbar_init(bp_empty(i), UNPACK_THREADS); }
        for (int i = 0; i < T::SBU; ++i) { mbar_init(bu_full(i), UNPACK_THREADS); mbar_init(bu_empty(i), 1); }
        for (int i = 0; i < SSC; ++i) { mbar_init(sc_full(i), 1); mbar_init(sc_empty(i), EPI_THREADS / 32); }
        for (int i = 0; i < 2; ++i) { mbar_init(acc_full(i), 1); mbar_init(acc_empty(i), EPI_THREADS); }
        fence_mbar_init();
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(&tmem_slot), T::TMEM_COLS);
        tmem_relinquish();
    }
    tcgen05_fence_before_sync();
    __syncthreads();
    tcgen05_fence_after_sync();
    const uint32_t tmem_base = tmem_slot;
    volatile int* abortp = &abort_word;

    // The epilogue warpgroups hold NT/2 fp32 accumulators per thread: hand them the registers the
    // producer / MMA / unpack warpgroups do not need.
    if (warp < 8) {
    if (NT == 256) reg_dec<56>();
    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            tma_prefetch_desc(&tm_a);
            tma_prefetch_desc(&tm_b);
            tma_prefetch_desc(&tm_sc);
            int sc_issued = 0;
            int a_issued = 0, bp_issued = 0;
            bool ok = true;
            for (int s = 0; s < n_stages && ok; ++s) {
                {
                    const int slot = s % SA, ph = (s / SA) & 1;
                    ok = mbar_wait(a_empty(slot), ph ^ 1, abortp, W_A_EMPTY);
                    if (!ok) break;
                    mbar_expect_tx(a_full(slot), p.a_tx);
                    tma_load_2d(smem_base + T::OFF_A + slot * A_BYTES, &tm_a, s * KSTAGE, m0, a_full(slot));
                    ++a_issued;
                }
                {
                    const int slot = s % SBP, ph = (s / SBP) & 1;
                    ok = mbar_wait(bp_empty(slot), ph ^ 1, abortp, W_BP_EMPTY);
                    if (!ok) break;
                    mbar_expect_tx(bp_full(slot), p.b_tx);
                    tma_load_2d(smem_base + T::OFF_BP + slot * T::BP_BYTES, &tm_b, s * (KSTAGE / 2), n0, bp_full(slot));
                    ++bp_issued;
                }
                while (sc_issued < n_groups && static_cast<long long>(sc_issued) * p.G < static_cast<long long>(s + 1) * KSTAGE) {
                    const int slot = sc_issued % SSC, ph = (sc_issued / SSC) & 1;
                    ok = mbar_wait(sc_empty(slot), ph ^ 1, abortp, W_SC_EMPTY);
                    if (!ok) break;
                    mbar_expect_tx(sc_full(slot), p.sc_tx);
                    tma_load_2d(smem_base + T::OFF_SC + slot * T::SC_BYTES, &tm_sc, n0, sc_issued, sc_full(slot));
                    ++sc_issued;
                }
            }
            if (!ok) {
                // Gave up: let the copies already in flight land before the CTA's shared memory goes away.
                for (int i = max(0, a_issued - SA); i < a_issued; ++i)
                    for (uint32_t it = 0; it < (1u << 16) && !mbar_try_wait(a_full(i % SA), (i / SA) & 1); ++it) {}
                for (int i = max(0, bp_issued - SBP); i < bp_issued; ++i)
                    for (uint32_t it = 0; it < (1u << 16) && !mbar_try_wait(bp_full(i % SBP), (i / SBP) & 1); ++it) {}
                for (int i = max(0, sc_issued - SSC); i < sc_issued; ++i)
                    for (uint32_t it = 0; it < (1u << 16) && !mbar_try_wait(sc_full(i % SSC), (i / SSC) & 1); ++it) {}
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            const uint32_t idesc = umma_idesc_i8(BM, NT);
            bool ok = true;
            for (int s = 0; s < n_stages && ok; ++s) {
                const int sa = s % SA, su = s % T::SBU;
                ok = mbar_wait(a_full(sa), (s / SA) & 1, abortp, W_A_FULL) &&
                     mbar_wait(bu_full(su), (s / T::SBU) & 1, abortp, W_BU_FULL);
                if (!ok) break;
                tcgen05_fence_after_sync();
                const uint64_t da = umma_desc_sw128(smem_base + T::OFF_A + sa * A_BYTES);
                const uint64_t db = umma_desc_sw128(smem_base + T::OFF_BU + su * T::BU_BYTES);
#pragma unroll
                for (int kk = 0; kk < KSTAGE / 32; ++kk) {
                    const int kpos = s * KSTAGE + kk * 32;
                    const int g = kpos / p.G;
                    const bool first = (kpos % p.G) == 0;
                    const bool last = ((kpos + 32) % p.G) == 0;
                    const int buf = g & 1;
                    if (first) {
                        ok = mbar_wait(acc_empty(buf), ((g >> 1) & 1) ^ 1, abortp, W_ACC_EMPTY);
                        if (!ok) break;
                        tcgen05_fence_after_sync();
                    }
                    umma_i8(tmem_base + buf * NT, da + 2u * kk, db + 2u * kk, idesc, first ? 0u : 1u);
                    if (last) umma_commit(acc_full(buf));
                }
                if (!ok) break;
                umma_commit(a_empty(sa));
                umma_commit(bu_empty(su));
            }
        }
    } else if (warp >= 4 && warp < 8) {
        // ------------------------------------------------------------------ INT4 -> int8 unpack
        const int tid = threadIdx.x - 128;
        for (int s = 0; s < n_stages; ++s) {
            const int sp = s % SBP, su = s % T::SBU;
            if (!mbar_wait(bp_full(sp), (s / SBP) & 1, abortp, W_BP_FULL)) break;
            if (!mbar_wait(bu_empty(su), ((s / T::SBU) & 1) ^ 1, abortp, W_BU_EMPTY)) break;
            const uint32_t src = smem_base + T::OFF_BP + sp * T::BP_BYTES;
            const uint32_t dst = smem_base + T::OFF_BU + su * T::BU_BYTES;
#pragma unroll 2
            for (int i = 0; i < NT * 4 / UNPACK_THREADS; ++i) {
                const int idx = i * UNPACK_THREADS + tid;
                const int row = idx >> 2, ch = idx & 3;
                const uint4 pk = lds128(src + idx * 16);
                uint4 lo, hi;
                lo.x = (pk.x << 4) & 0xF0F0F0F0u; hi.x = pk.x & 0xF0F0F0F0u;
                lo.y = (pk.y << 4) & 0xF0F0F0F0u; hi.y = pk.y & 0xF0F0F0F0u;
                lo.z = (pk.z << 4) & 0xF0F0F0F0u; hi.z = pk.z & 0xF0F0F0F0u;
                lo.w = (pk.w << 4) & 0xF0F0F0F0u; hi.w = pk.w & 0xF0F0F0F0u;
                const uint32_t drow = dst + (row >> 3) * 1024 + (row & 7) * 128;
                sts128(drow + (((2 * ch) ^ (row & 7)) << 4), lo);
                sts128(drow + (((2 * ch + 1) ^ (row & 7)) << 4), hi);
            }
            fence_proxy_async_smem();
            mbar_arrive(bu_full(su));
            mbar_arrive(bp_empty(sp));
        }
    }
    } else {
        // ------------------------------------------------------------------ epilogue
        if (NT == 256) reg_inc<200>();
        constexpr int EC = T::EC;
        constexpr int CH = (NT == 256) ? 16 : 32;    // columns per TMEM load (two loads in flight)
        constexpr int NCH = EC / CH;
        const int q = warp & 3;                  // TMEM lane quadrant this warp may read
        const int h = (warp - 8) >> 2;           // column half
        const int row = m0 + q * 32 + lane;
        float acc[EC];
#pragma unroll
        for (int j = 0; j < EC; ++j) acc[j] = 0.0f;
        bool ok = true;
        for (int g = 0; g < n_groups; ++g) {
            const int buf = g & 1;
            const int ss = g % SSC;
            ok = mbar_wait(sc_full(ss), (g / SSC) & 1, abortp, W_SC_FULL) &&
                 mbar_wait(acc_full(buf), (g >> 1) & 1, abortp, W_ACC_FULL);
            ok = __all_sync(0xffffffffu, ok);     // warp-uniform: the TMEM loads below are warp-collective
            if (!ok) break;
            tcgen05_fence_after_sync();
            const uint32_t taddr = tmem_base + (static_cast<uint32_t>(q * 32) << 16) + buf * NT + h * EC;
            const uint32_t sc = smem_base + T::OFF_SC + ss * T::SC_BYTES + h * EC * 4;
            uint32_t c0[CH], c1[CH];
            tmem_ld_chunk(taddr, c0);
#pragma unroll
            for (int ch = 0; ch < NCH; ++ch) {
                tmem_wait_ld();
                if (ch + 1 < NCH) {
                    if (ch & 1) tmem_ld_chunk(taddr + (ch + 1) * CH, c0);
                    else        tmem_ld_chunk(taddr + (ch + 1) * CH, c1);
                }
                const uint32_t (&cur)[CH] = (ch & 1) ? c1 : c0;
#pragma unroll
                for (int j4 = 0; j4 < CH / 4; ++j4) {
                    const float4 s4 = lds_f4(sc + (ch * CH + j4 * 4) * 4);
                    float* a4 = &acc[ch * CH + j4 * 4];
                    a4[0] = fmaf(__int2float_rn(static_cast<int>(cur[j4 * 4 + 0])), s4.x, a4[0]);
                    a4[1] = fmaf(__int2float_rn(static_cast<int>(cur[j4 * 4 + 1])), s4.y, a4[1]);
                    a4[2] = fmaf(__int2float_rn(static_cast<int>(cur[j4 * 4 + 2])), s4.z, a4[2]);
                    a4[3] = fmaf(__int2float_rn(static_cast<int>(cur[j4 * 4 + 3])), s4.w, a4[3]);
                }
                if (DUMP) {
                    const int rr = row - p.row0;
                    if (p.acc != nullptr && rr >= 0 && rr < p.rows && row < p.M) {
#pragma unroll
                        for (int j = 0; j < CH; ++j) {
                            const int col = n0 + h * EC + ch * CH + j;
                            const int cc = col - p.col0;
                            if (cc >= 0 && cc < p.cols && col < p.N)
                                p.acc[(static_cast<size_t>(g) * p.rows + rr) * p.cols + cc] = static_cast<int>(cur[j]) >> 4;
                        }
                    }
                }
            }
            tcgen05_fence_before_sync();
            mbar_arrive(acc_empty(buf));
            __syncwarp();
            if (lane == 0) mbar_arrive(sc_empty(ss));
        }
        if (ok && row < p.M) {
            const float rs = p.row_scale[row];
            uint16_t* yrow = p.Y + static_cast<size_t>(row) * p.ldy;
#pragma unroll
            for (int j = 0; j < EC; j += 8) {
                const int col = n0 + h * EC + j;
                if (col < p.N) {     // N % 64 == 0, so an 8-column run is all inside or all outside
                    float b[8] = {0, 0, 0, 0, 0, 0, 0, 0};
                    if (p.bias) {
                        const float4 b0 = __ldg(reinterpret_cast<const float4*>(p.bias + col));
                        const float4 b1 = __ldg(reinterpret_cast<const float4*>(p.bias + col + 4));
                        b[0] = b0.x; b[1] = b0.y; b[2] = b0.z; b[3] = b0.w;
                        b[4] = b1.x; b[5] = b1.y; b[6] = b1.z; b[7] = b1.w;
                    }
                    uint32_t o[4];
#pragma unroll
                    for (int t = 0; t < 4; ++t) {
                        const __nv_bfloat162 v = __floats2bfloat162_rn(fmaf(acc[j + 2 * t], rs, b[2 * t]),
                                                                       fmaf(acc[j + 2 * t + 1], rs, b[2 * t + 1]));
                        o[t] = *reinterpret_cast<const uint32_t*>(&v);
                    }
                    *reinterpret_cast<uint4*>(yrow + col) = make_uint4(o[0], o[1], o[2], o[3]);
                }
            }
        }
    }

    // ---------------------------------------------------------------------- teardown
    tcgen05_fence_before_sync();
    __syncthreads();
    if (warp == 1) {
        __syncwarp();
        tcgen05_fence_after_sync();
        tmem_dealloc(tmem_base, T::TMEM_COLS);
    }
}

}  // namespace

template <int NT, bool DUMP>
static cudaError_t launch_one(const GemmI8Args& a, cudaStream_t st)
{
    using T = Tile<NT>;
    const WeightTiles& wt = a.wt[NT == 256 ? 1 : 0];
    Params p;
    p.M = a.M; p.N = a.N; p.K = a.K; p.G = a.G;
    p.row_scale = a.row_scale; p.bias = a.bias; p.Y = a.Y; p.ldy = a.ldy;
    p.acc = a.acc; p.row0 = a.row0; p.rows = a.rows; p.col0 = a.col0; p.cols = a.cols;
    p.a_tx = static_cast<uint32_t>(min(BM, a.M)) * KSTAGE;
    p.b_tx = static_cast<uint32_t>(min(NT, a.N)) * (KSTAGE / 2);
    p.sc_tx = static_cast<uint32_t>(min(NT, a.N)) * 4;
    dim3 grid((a.N + NT - 1) / NT, (a.M + BM - 1) / BM);
    gemm_i8_w4_kernel<NT, DUMP><<<grid, NUM_THREADS, T::DYN_SMEM, st>>>(a.tm_a, wt.codes, wt.scales, p);
    return cudaGetLastError();
}

cudaError_t gemm_i8_init()
{
    cudaError_t e;
    e = cudaFuncSetAttribute(gemm_i8_w4_kernel<128, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, Tile<128>::DYN_SMEM);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(gemm_i8_w4_kernel<128, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, Tile<128>::DYN_SMEM);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(gemm_i8_w4_kernel<256, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, Tile<256>::DYN_SMEM);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(gemm_i8_w4_kernel<256, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, Tile<256>::DYN_SMEM);
    return e;
}

cudaError_t launch_gemm_i8(const GemmI8Args& a, cudaStream_t st)
{
    const bool wide = (a.N % 256 == 0);
    if (a.acc != nullptr) return wide ? launch_one<256, true>(a, st) : launch_one<128, true>(a, st);
    return wide ? launch_one<256, false>(a, st) : launch_one<128, false>(a, st);
}

}  // namespace rudder
