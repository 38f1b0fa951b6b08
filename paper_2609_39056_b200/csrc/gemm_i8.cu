// Second kernel of the engine (Section 4.4; Eq. 10): C = Q_X Q_W on the tcgen05 integer tensor cores
// with INT32 accumulators in TMEM, and an epilogue that applies the weight scales, the row scale
// r_i (which already carries the inverse stream gain) and the bias, writing BF16.
//
// Orientation: the WEIGHTS are the M-side operand of the MMA.  One CTA computes 128 output channels
// x TT tokens: D[channel][token] = sum_k W[channel][k] * Q_X[token][k].  A TMEM lane (= an epilogue
// thread) therefore owns one output channel, so the weight scale Delta_W[j,g] of a group is a single
// register per thread and the per-group drain is exactly one int->float conversion and one FMA per
// element.  That drain, not the tensor core, bounds the group-scaled path: the conversion pipe
// sustains about 64 elements per clock per SM against 128 for the MMA at G = 64.
//
// Warp roles (warpgroup-aligned so that registers can be moved between them):
//   warp 0        TMA producer: activation codes (int8 [TT tokens][128 B], 128-byte swizzle)
//   warp 1        allocates TMEM; one lane issues tcgen05.mma kind::i8 (M = 128, N = TT, K = 32)
//   warps 4-7     stream the packed INT4 weights from global memory (L2) into registers one stage
//                 ahead, expand them to int8 and store them in the swizzled K-major layout the tensor
//                 core reads.  The nibble goes to the TOP half of the byte (value 16 q): two logic ops
//                 per 8 weights, no sign extension; the factor 16 is folded into the fp32 scales.
//   warps 8-15    epilogue: per weight group, drain the INT32 partial sums from TMEM and accumulate
//                 fp32(C) * Delta_W[j,g] in registers; finally * r_i + b_j -> bf16, transposed through
//                 shared memory and written with one TMA store per tile.
// Group partials alternate between two TMEM buffers, so the tensor core runs group g + 1 while group
// g is drained.
//
// Shared memory rings (stage = 128 input channels):
//   X  [SX][TT tokens][128 B]     int8, swizzled by TMA       full: TMA bytes     empty: umma commit
//   W  [SW][128 channels][128 B]  int8 x16, swizzled by hand  full: 4 warps       empty: umma commit
// The output tile [TT tokens][128 channels] bf16 is staged over the X ring once the last MMA is done.
// TMEM: 2 x TT columns x 128 lanes of INT32.  acc_full[b]: umma commit; acc_empty[b]: 8 epilogue warps.
#include "internal.cuh"
#include "ptx.cuh"

#include <cuda_bf16.h>

namespace rudder {

namespace {

constexpr int BN = 128;          // output channels per tile (MMA M)
constexpr int KSTAGE = 128;      // input channels (= bytes of int8 per row) per pipeline stage
constexpr int SW = 4;            // unpacked-weight stages
constexpr int W_BYTES = BN * KSTAGE;
constexpr int NUM_THREADS = 512;
constexpr int UNPACK_THREADS = 128;
constexpr int EPI_THREADS = 256;

// Back-off (ns) between polls of a barrier, per role.
#ifndef RUDDER_REGS_LO
#define RUDDER_REGS_LO 72
#define RUDDER_REGS_HI 184
#endif
#ifndef RUDDER_REGS_LO128
#define RUDDER_REGS_LO128 88
#define RUDDER_REGS_HI128 168
#endif
#ifndef RUDDER_CH
#define RUDDER_CH 32
#endif
#ifndef RUDDER_EPI_BATCH
#define RUDDER_EPI_BATCH 1
#endif
#ifndef RUDDER_EPI_DB
#define RUDDER_EPI_DB 1
#endif
#ifndef RUDDER_SLEEP_PROD
#define RUDDER_SLEEP_PROD 64
#endif
#ifndef RUDDER_SLEEP_UNPACK
#define RUDDER_SLEEP_UNPACK 64
#endif
#ifndef RUDDER_SLEEP_MMA
#define RUDDER_SLEEP_MMA 0
#endif
#ifndef RUDDER_SLEEP_EPI
#define RUDDER_SLEEP_EPI 0
#endif

template <int TT> struct Tile {          // TT = tokens per tile (MMA N): 256 or 128
    static constexpr int SX = (TT == 256) ? 4 : 6;
    static constexpr int X_BYTES = TT * KSTAGE;
    static constexpr int OFF_X = 0;
    static constexpr int OFF_W = OFF_X + SX * X_BYTES;
    static constexpr int BYTES = OFF_W + SW * W_BYTES;
    static constexpr int DYN_SMEM = BYTES + 1024;    // slack to align the base to 1024 bytes
    static constexpr int TMEM_COLS = 2 * TT;
    static constexpr int EC = TT / 2;                // tokens per epilogue thread
    static_assert(SX * X_BYTES >= TT * BN * 2, "the output tile is staged over the X ring");
};

struct Params {
    int M, N, K, G;
    const uint8_t* codes;        // packed INT4 weights [N][K/2], 32-channel interleave
    const float* scales_t;       // [K/G][N] fp32 = Delta_W / 16
    const float* row_scale;      // r [M]
    const float* bias;           // [N] or nullptr
    int32_t* acc;                // accumulator dump [K/G][rows][cols] or nullptr
    int row0, rows, col0, cols;
    int m_tiles, n_tiles;        // token tiles, channel tiles (grid = m_tiles * n_tiles CTAs)
    uint32_t x_tx;               // bytes one activation TMA box delivers
    int out_pitch;               // channels per row of the staged output tile (= TMA store box width)
#ifdef RUDDER_ROLE_PROF
    long long* prof;             // [16] cycle counters of CTA (0,0): where each role waits (development aid)
#endif
};

#ifdef RUDDER_ROLE_PROF
#define PROF_DECL(n) long long prof_##n = 0
#define PROF_WAIT(n, expr) [&]() { const long long t_ = clock64(); const bool r_ = (expr); prof_##n += clock64() - t_; return r_; }()
#define PROF_PUT(i, n) do { if (blockIdx.x == 0 && p.prof) p.prof[i] = prof_##n; } while (0)
#else
#define PROF_DECL(n)
#define PROF_WAIT(n, expr) (expr)
#define PROF_PUT(i, n)
#endif

enum Where {   // codes recorded when a bounded wait gives up
    W_X_EMPTY = 101,
    W_W_EMPTY = 201,
    W_X_FULL = 301, W_W_FULL = 302, W_ACC_EMPTY = 303,
    W_ACC_FULL = 401, W_RS_FULL = 402
};

__device__ __forceinline__ void sts128(uint32_t addr, const uint4& v) {
    asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}
__device__ __forceinline__ void sts16(uint32_t addr, uint16_t v) {
    asm volatile("st.shared.u16 [%0], %1;" ::"r"(addr), "h"(v) : "memory");
}
__device__ __forceinline__ uint4 ldg_nc_16(const void* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0, %1, %2, %3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}
__device__ __forceinline__ float ldg_f32_volatile(const float* p) {
    float v;
    asm volatile("ld.global.nc.f32 %0, [%1];" : "=f"(v) : "l"(p));
    return v;
}
__device__ __forceinline__ void tmem_ld_chunk(uint32_t taddr, uint32_t (&r)[32]) { tmem_ld_32x32b_x32(taddr, r); }
__device__ __forceinline__ void tmem_ld_chunk(uint32_t taddr, uint32_t (&r)[16]) { tmem_ld_32x32b_x16(taddr, r); }

template <int TT, bool DUMP>
__global__ void __launch_bounds__(NUM_THREADS, 1)
gemm_i8_w4_kernel(const __grid_constant__ CUtensorMap tm_x, const __grid_constant__ CUtensorMap tm_y, const Params p)
{
    using T = Tile<TT>;
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t bars[2 * T::SX + 2 * SW + 5];
    __shared__ __align__(16) float rs_smem[TT];      // row scales r_i of the tile's tokens (0 past M)
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_word;

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    int tile_m, tile_n;
    tile_coords(blockIdx.x, p.m_tiles, p.n_tiles, 16, tile_m, tile_n);
    const int m0 = tile_m * TT;              // first token of the tile
    const int n0 = tile_n * BN;              // first output channel of the tile
    const int n_stages = p.K / KSTAGE;
    const int n_groups = p.K / p.G;

    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t bar0 = smem_u32(bars);
    auto x_full = [&](int i) { return bar0 + 8u * i; };
    auto x_empty = [&](int i) { return bar0 + 8u * (T::SX + i); };
    auto w_full = [&](int i) { return bar0 + 8u * (2 * T::SX + i); };
    auto w_empty = [&](int i) { return bar0 + 8u * (2 * T::SX + SW + i); };
    auto acc_full = [&](int i) { return bar0 + 8u * (2 * T::SX + 2 * SW + i); };
    auto acc_empty = [&](int i) { return bar0 + 8u * (2 * T::SX + 2 * SW + 2 + i); };
    const uint32_t rs_full = bar0 + 8u * (2 * T::SX + 2 * SW + 4);

    if (threadIdx.x == 0) {
        abort_word = 0;
        for (int i = 0; i < T::SX; ++i) { mbar_init(x_full(i), 1); mbar_init(x_empty(i), 1); }
        for (int i = 0; i < SW; ++i) { mbar_init(w_full(i), UNPACK_THREADS / 32); mbar_init(w_empty(i), 1); }
        for (int i = 0; i < 2; ++i) { mbar_init(acc_full(i), 1); mbar_init(acc_empty(i), EPI_THREADS / 32); }
        mbar_init(rs_full, 1);
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

    if (warp < 8) {
    // The epilogue warpgroups hold TT/2 fp32 accumulators per thread: hand them the registers the
    // producer / MMA / unpack warpgroups do not need.
    if (TT == 256) reg_dec<RUDDER_REGS_LO>(); else reg_dec<RUDDER_REGS_LO128>();
    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer (activations)
        if (lane == 0) {
            tma_prefetch_desc(&tm_x);
            tma_prefetch_desc(&tm_y);
            int issued = 0;
            bool ok = true;
            PROF_DECL(x_empty);
            int slot = 0;
            uint32_t ph = 0;
            for (int s = 0; s < n_stages; ++s) {
                ok = PROF_WAIT(x_empty, mbar_wait<RUDDER_SLEEP_PROD>(x_empty(slot), ph ^ 1u, abortp, W_X_EMPTY));
                if (!ok) break;
                mbar_expect_tx(x_full(slot), p.x_tx);
#ifndef RUDDER_DBG_NO_TMA
                tma_load_2d(smem_base + T::OFF_X + slot * T::X_BYTES, &tm_x, s * KSTAGE, m0, x_full(slot));
#else
                asm volatile("mbarrier.complete_tx.shared::cta.b64 [%0], %1;" ::"r"(x_full(slot)), "r"(p.x_tx) : "memory");
#endif
                ++issued;
                if (++slot == T::SX) { slot = 0; ph ^= 1u; }
            }
            PROF_PUT(0, x_empty);
            if (!ok) {
                // Gave up: let the copies already in flight land before the CTA's shared memory goes away.
                for (int i = max(0, issued - T::SX); i < issued; ++i)
                    for (uint32_t it = 0; it < (1u << 16) && !mbar_try_wait(x_full(i % T::SX), (i / T::SX) & 1); ++it) {}
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        // The whole warp walks the loop converged (so that addresses and descriptors stay in uniform
        // registers); one elected lane issues the MMAs and the commits.
        {
            const bool leader = elect_one();
            const uint32_t idesc = umma_idesc_i8(BN, TT);
            bool ok = true;
            PROF_DECL(x_full); PROF_DECL(w_full); PROF_DECL(acc_empty); PROF_DECL(mma_total);
#ifdef RUDDER_ROLE_PROF
            const long long mma_t0 = clock64();
#endif
            // No divisions in this loop: every instruction on this path is latency the tensor core may
            // end up waiting for.
            const int mma_per_group = p.G >> 5;        // MMAs (K = 32 each) per weight group
            int in_group = 0;                          // MMAs issued so far in the current group
            uint32_t g = 0;                            // current group
            int sx = 0, sw = 0;                        // ring slots
            uint32_t phx = 0, phw = 0;                 // ring phases
            for (int s = 0; s < n_stages && ok; ++s) {
                ok = PROF_WAIT(x_full, mbar_wait<RUDDER_SLEEP_MMA>(x_full(sx), phx, abortp, W_X_FULL)) &&
                     PROF_WAIT(w_full, mbar_wait<RUDDER_SLEEP_MMA>(w_full(sw), phw, abortp, W_W_FULL));
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                tcgen05_fence_after_sync();
                const uint64_t da = umma_desc_sw128(smem_base + T::OFF_W + sw * W_BYTES);        // weights: M side
                const uint64_t db = umma_desc_sw128(smem_base + T::OFF_X + sx * T::X_BYTES);     // tokens: N side
#pragma unroll
                for (int kk = 0; kk < KSTAGE / 32; ++kk) {
                    const uint32_t buf = g & 1u;
                    if (in_group == 0) {
                        ok = PROF_WAIT(acc_empty, mbar_wait<RUDDER_SLEEP_MMA>(acc_empty(buf), ((g >> 1) & 1u) ^ 1u, abortp, W_ACC_EMPTY));
                        ok = __all_sync(0xffffffffu, ok);
                        if (!ok) break;
                        tcgen05_fence_after_sync();
                    }
#ifndef RUDDER_DBG_NO_MMA
                    if (leader) umma_i8(tmem_base + buf * TT, da + 2u * kk, db + 2u * kk, idesc, in_group == 0 ? 0u : 1u);
#endif
                    if (++in_group == mma_per_group) {
                        if (leader) umma_commit(acc_full(buf));
                        in_group = 0;
                        ++g;
                    }
                }
                if (!ok) break;
                if (leader) {
                    umma_commit(x_empty(sx));
                    umma_commit(w_empty(sw));
                }
                __syncwarp();
                if (++sx == T::SX) { sx = 0; phx ^= 1u; }
                if (++sw == SW) { sw = 0; phw ^= 1u; }
            }
#ifdef RUDDER_ROLE_PROF
            prof_mma_total = clock64() - mma_t0;
#endif
            if (leader) { PROF_PUT(3, x_full); PROF_PUT(4, w_full); PROF_PUT(5, acc_empty); PROF_PUT(6, mma_total); }
        }
    } else if (warp == 2) {
        // ------------------------------------------------------------------ row scales of the tile -> shared
        for (int i = lane; i < TT; i += 32) rs_smem[i] = (m0 + i < p.M) ? __ldg(p.row_scale + m0 + i) : 0.0f;
        __syncwarp();
        if (lane == 0) mbar_arrive(rs_full);
    } else if (warp >= 4) {
        // ------------------------------------------------------------------ INT4 -> int8 unpack
        // 128 channels x 64 packed bytes per stage = 512 16-byte pieces, 4 per thread: piece idx covers
        // channel idx / 4, input channels [32 (idx % 4), 32 (idx % 4) + 32) of the stage.
        const int tid = threadIdx.x - 128;
        PROF_DECL(w_empty); PROF_DECL(unpack_total);
#ifdef RUDDER_ROLE_PROF
        const long long un_t0 = clock64();
#endif
        const size_t row_bytes = static_cast<size_t>(p.K / 2);
        const uint8_t* src[4];
        bool valid[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int idx = i * UNPACK_THREADS + tid;
            const int row = idx >> 2, ch = idx & 3;
            valid[i] = (n0 + row) < p.N;
            src[i] = p.codes + static_cast<size_t>(valid[i] ? n0 + row : 0) * row_bytes + ch * 16;
        }
        uint4 nxt[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) nxt[i] = valid[i] ? ldg_nc_16(src[i]) : make_uint4(0, 0, 0, 0);
        for (int s = 0; s < n_stages; ++s) {
            uint4 cur[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) cur[i] = nxt[i];
            if (s + 1 < n_stages) {
#pragma unroll
                for (int i = 0; i < 4; ++i)
                    nxt[i] = valid[i] ? ldg_nc_16(src[i] + static_cast<size_t>(s + 1) * (KSTAGE / 2)) : make_uint4(0, 0, 0, 0);
            }
            const int sw = s % SW;
            if (!PROF_WAIT(w_empty, mbar_wait<RUDDER_SLEEP_UNPACK>(w_empty(sw), ((s / SW) & 1) ^ 1, abortp, W_W_EMPTY))) break;
            const uint32_t dst = smem_base + T::OFF_W + sw * W_BYTES;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int idx = i * UNPACK_THREADS + tid;
                const int row = idx >> 2, ch = idx & 3;
                const uint4 pk = cur[i];
                uint4 lo, hi;
                lo.x = (pk.x << 4) & 0xF0F0F0F0u; hi.x = pk.x & 0xF0F0F0F0u;
                lo.y = (pk.y << 4) & 0xF0F0F0F0u; hi.y = pk.y & 0xF0F0F0F0u;
                lo.z = (pk.z << 4) & 0xF0F0F0F0u; hi.z = pk.z & 0xF0F0F0F0u;
                lo.w = (pk.w << 4) & 0xF0F0F0F0u; hi.w = pk.w & 0xF0F0F0F0u;
                const uint32_t drow = dst + (row >> 3) * 1024 + (row & 7) * 128;
#ifndef RUDDER_DBG_NO_STS
                sts128(drow + (((2 * ch) ^ (row & 7)) << 4), lo);
                sts128(drow + (((2 * ch + 1) ^ (row & 7)) << 4), hi);
#else
                if (lo.x == 0x12345678u && hi.y == 0x9abcdef0u) sts128(drow, lo);
#endif
            }
#ifndef RUDDER_DBG_NO_FENCE
            fence_proxy_async_smem();
#endif
            __syncwarp();
            if (lane == 0) mbar_arrive(w_full(sw));      // one arrival per warp: arrivals on one barrier serialise
        }
#ifdef RUDDER_ROLE_PROF
        prof_unpack_total = clock64() - un_t0;
        if (tid == 0) { PROF_PUT(8, w_empty); PROF_PUT(9, unpack_total); }
#endif
    }
    } else {
        // ------------------------------------------------------------------ epilogue
        if (TT == 256) reg_inc<RUDDER_REGS_HI>(); else reg_inc<RUDDER_REGS_HI128>();
        constexpr int EC = T::EC;
        constexpr int CH = (TT == 256) ? RUDDER_CH : 32;   // tokens per TMEM load
        constexpr int NCH = EC / CH;
        const int q = warp & 3;                  // TMEM lane quadrant this warp may read
        const int h = (warp - 8) >> 2;           // token half
        const int ch_local = q * 32 + lane;      // channel within the tile = TMEM lane
        const int n = n0 + ch_local;
        const bool n_ok = n < p.N;
        float acc[EC];
#pragma unroll
        for (int j = 0; j < EC; ++j) acc[j] = 0.0f;
        bool ok = true;
        PROF_DECL(acc_full); PROF_DECL(epi_total); PROF_DECL(epi_drain); PROF_DECL(epi_tail); PROF_DECL(epi_vote); PROF_DECL(epi_fence);
#ifdef RUDDER_ROLE_PROF
        const long long ep_t0 = clock64();
#endif
        // Scales are fetched two groups ahead with volatile loads: a plain load would be sunk next to
        // its use and expose the L2 latency once per group.
        const float* sc_ptr = p.scales_t + (n_ok ? n : 0);
        float sc_next = ldg_f32_volatile(sc_ptr);
        float sc_next2 = (n_groups > 1) ? ldg_f32_volatile(sc_ptr + p.N) : 0.0f;
        for (int g = 0; g < n_groups; ++g) {
            const int buf = g & 1;
#ifdef RUDDER_DBG_CONST_SC
            const float sc = 1.5f + threadIdx.x;
#else
            const float sc = n_ok ? sc_next : 0.0f;
            sc_next = sc_next2;
            if (g + 2 < n_groups) sc_next2 = ldg_f32_volatile(sc_ptr + static_cast<size_t>(g + 2) * p.N);
#endif
#ifndef RUDDER_DBG_EPI_FREE
            // lane 0 polls, the others wait at the shuffle: no 32-way spin, and the verdict is warp-uniform
            // (the TMEM loads below are warp-collective)
            if (lane == 0) ok = PROF_WAIT(acc_full, mbar_wait<RUDDER_SLEEP_EPI>(acc_full(buf), (g >> 1) & 1, abortp, W_ACC_FULL));
#ifdef RUDDER_ROLE_PROF
            const long long v_t0 = clock64();
#endif
            ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
            if (!ok) break;
#endif
#ifdef RUDDER_ROLE_PROF
            const long long f_t0 = clock64();
            prof_epi_vote += f_t0 - v_t0;
#endif
            tcgen05_fence_after_sync();
#ifdef RUDDER_ROLE_PROF
            prof_epi_fence += clock64() - f_t0;
#endif
#ifdef RUDDER_ROLE_PROF
            const long long dr_t0 = clock64();
#endif
            const uint32_t taddr = tmem_base + (static_cast<uint32_t>(q * 32) << 16) + buf * TT + h * EC;
            uint32_t c0[CH], c1[CH];
#if RUDDER_EPI_DB
            tmem_ld_chunk(taddr, c0);
#endif
#pragma unroll
            for (int ch = 0; ch < NCH; ++ch) {
#if RUDDER_EPI_DB
                tmem_wait_ld();
                if (ch + 1 < NCH) {
                    if (ch & 1) tmem_ld_chunk(taddr + (ch + 1) * CH, c0);
                    else        tmem_ld_chunk(taddr + (ch + 1) * CH, c1);
                }
                const uint32_t (&cur)[CH] = (ch & 1) ? c1 : c0;
#else
                tmem_ld_chunk(taddr + ch * CH, c0);
                tmem_wait_ld();
                const uint32_t (&cur)[CH] = c0;
                (void)c1;
#endif
#if RUDDER_EPI_BATCH
                // Convert the whole chunk first, then accumulate: every FMA then finds its operand ready
                // instead of waiting out the conversion latency element by element.
                float f[CH];
#pragma unroll
                for (int j = 0; j < CH; ++j) asm volatile("cvt.rn.f32.s32 %0, %1;" : "=f"(f[j]) : "r"(cur[j]));
#pragma unroll
                for (int j = 0; j < CH; ++j) asm volatile("fma.rn.f32 %0, %1, %2, %0;" : "+f"(acc[ch * CH + j]) : "f"(f[j]), "f"(sc));
#else
#pragma unroll
                for (int j = 0; j < CH; ++j)
                    acc[ch * CH + j] = fmaf(__int2float_rn(static_cast<int>(cur[j])), sc, acc[ch * CH + j]);
#endif
                if (DUMP) {
                    const int cc = n - p.col0;
                    if (p.acc != nullptr && n_ok && cc >= 0 && cc < p.cols) {
#pragma unroll
                        for (int j = 0; j < CH; ++j) {
                            const int tok = m0 + h * EC + ch * CH + j;
                            const int rr = tok - p.row0;
                            if (tok < p.M && rr >= 0 && rr < p.rows)
                                p.acc[(static_cast<size_t>(g) * p.rows + rr) * p.cols + cc] = static_cast<int>(cur[j]) >> 4;
                        }
                    }
                }
            }
            tcgen05_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(acc_empty(buf));  // one arrival per warp: arrivals on one barrier serialise
#ifdef RUDDER_ROLE_PROF
            prof_epi_drain += clock64() - dr_t0;
#endif
        }
#ifdef RUDDER_ROLE_PROF
        prof_epi_total = clock64() - ep_t0;
        const long long tail_t0 = clock64();
#endif
        // The last acc_full arrives after every MMA of the tile has completed, so the X ring is free:
        // stage the transposed bf16 tile there ([token][channel], `out_pitch` channels per row).
        if (ok) ok = mbar_wait<64>(rs_full, 0, abortp, W_RS_FULL);
        if (ok) {
            const float b = (p.bias != nullptr && n_ok) ? __ldg(p.bias + n) : 0.0f;
            const uint32_t stage0 = smem_base + T::OFF_X;
            const float4* rs4 = reinterpret_cast<const float4*>(rs_smem + h * EC);
            if (ch_local < p.out_pitch) {
                uint32_t dst = stage0 + static_cast<uint32_t>(h * EC * p.out_pitch + ch_local) * 2u;
                const uint32_t step = static_cast<uint32_t>(p.out_pitch) * 2u;
#pragma unroll
                for (int j = 0; j < EC; j += 4) {
                    const float4 rs = rs4[j >> 2];                   // broadcast read, zero past M
                    sts16(dst, __bfloat16_as_ushort(__float2bfloat16_rn(fmaf(acc[j + 0], rs.x, b)))); dst += step;
                    sts16(dst, __bfloat16_as_ushort(__float2bfloat16_rn(fmaf(acc[j + 1], rs.y, b)))); dst += step;
                    sts16(dst, __bfloat16_as_ushort(__float2bfloat16_rn(fmaf(acc[j + 2], rs.z, b)))); dst += step;
                    sts16(dst, __bfloat16_as_ushort(__float2bfloat16_rn(fmaf(acc[j + 3], rs.w, b)))); dst += step;
                }
            }
            fence_proxy_async_smem();                            // generic writes -> visible to the TMA store
        }
        asm volatile("bar.sync 1, %0;" ::"n"(EPI_THREADS) : "memory");
        if (ok && threadIdx.x == 256) {
            asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];"
                         ::"l"(reinterpret_cast<uint64_t>(&tm_y)), "r"(smem_base + T::OFF_X), "r"(n0), "r"(m0) : "memory");
            asm volatile("cp.async.bulk.commit_group;" ::: "memory");
            asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
        }
#ifdef RUDDER_ROLE_PROF
        prof_epi_tail = clock64() - tail_t0;
        if (threadIdx.x == 256) { PROF_PUT(10, epi_drain); PROF_PUT(11, acc_full); PROF_PUT(12, epi_total); PROF_PUT(13, epi_tail); PROF_PUT(14, epi_vote); PROF_PUT(15, epi_fence); }
#endif
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

template <int TT, bool DUMP>
static cudaError_t launch_one(const GemmI8Args& a, cudaStream_t st)
{
    using T = Tile<TT>;
    Params p;
    p.M = a.M; p.N = a.N; p.K = a.K; p.G = a.G;
    p.codes = a.w_codes; p.scales_t = a.w_scales_t;
    p.row_scale = a.row_scale; p.bias = a.bias;
    p.acc = a.acc; p.row0 = a.row0; p.rows = a.rows; p.col0 = a.col0; p.cols = a.cols;
    p.x_tx = static_cast<uint32_t>(min(TT, a.M)) * KSTAGE;
    p.out_pitch = min(BN, a.N);
#ifdef RUDDER_ROLE_PROF
    p.prof = reinterpret_cast<long long*>(a.acc);   // development build only: the dump pointer carries the counters
    p.acc = nullptr;
#endif
    p.m_tiles = (a.M + TT - 1) / TT;
    p.n_tiles = (a.N + BN - 1) / BN;
    gemm_i8_w4_kernel<TT, DUMP><<<p.m_tiles * p.n_tiles, NUM_THREADS, T::DYN_SMEM, st>>>(a.tm_x, a.tm_y, p);
    return cudaGetLastError();
}

int gemm_i8_token_tile(int M) { return M > 128 ? 256 : 128; }

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
    const bool wide = gemm_i8_token_tile(a.M) == 256;
#ifdef RUDDER_ROLE_PROF
    return wide ? launch_one<256, false>(a, st) : launch_one<128, false>(a, st);   // the dump pointer carries counters
#endif
    if (a.acc != nullptr) return wide ? launch_one<256, true>(a, st) : launch_one<128, true>(a, st);
    return wide ? launch_one<256, false>(a, st) : launch_one<128, false>(a, st);
}

}  // namespace rudder
