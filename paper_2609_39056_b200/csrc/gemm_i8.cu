// Second kernel of the engine (Section 4.4; Eq. 10): C = Q_X Q_W on the tcgen05 integer tensor cores
// with INT32 accumulators in TMEM, and an epilogue that applies the weight scales, the row scale
// r_i (which already carries the inverse stream gain) and the bias, writing BF16.
//
// Orientation: the WEIGHTS are the M-side operand of the MMA.  One CTA computes 128 output channels
// x TT tokens: D[channel][token] = sum_k W[channel][k] * Q_X[token][k].  A TMEM lane (= an epilogue
// thread) therefore owns one output channel, so the weight scale Delta_W[j,g] of a group is a single
// register per thread and the per-group drain is exactly one int->float conversion and one FMA per
// element.  That drain, not the tensor core, bounds the group-scaled path: the conversion pipe
// sustains about 64 elements per clock per SM against 128 for the MMA at G = 64, and every value
// drained costs register-file writes (TMEM load, conversion, FMA) on the same four sub-partitions.
//
// W4A4 with group scales (G <= 128) takes the E4M3 form of the same product: codes in [-7, 7] are
// exact in E4M3, |C^(g)| <= 128 * 49 is exact in the FP32 accumulators of kind::f8f6f4 (same tensor
// rate as kind::i8), so C^(g) arrives as fp32 and the drain is the FMA alone.  The activations come
// from the prologue as E4M3 bytes, the weights are stored sign-magnitude so that the unpack is two
// table look-ups (byte permutes) per eight weights.  The integers, and therefore the results, are
// the same bit for bit as on the INT32 path.
//
// Warp roles (warpgroup-aligned so that registers can be moved between them):
//   warp 0        TMA producer: activation codes (int8 [TT tokens][128 B], 128-byte swizzle)
//   warp 1        allocates TMEM; one lane issues tcgen05.mma kind::i8 (M = 128, N = TT, K = 32)
//   warp 3        TMA producer of the packed INT4 weights: a ring of raw stages [128 channels][64 B],
//                 several stages ahead of the unpack warps (the weights do not depend on the prologue
//                 kernel, so this stream starts while that kernel is still running)
//   warps 4-7     take the packed INT4 weights from the raw ring, expand them to int8 and store them in
//                 the swizzled K-major layout the tensor core reads.  The nibble goes to the TOP half of the byte (value 16 q): two logic ops
//                 per 8 weights, no sign extension; the factor 16 is folded into the fp32 scales.
//   warps 8-15    epilogue: per weight group, drain the INT32 partial sums from TMEM and accumulate
//                 fp32(C) * Delta_W[j,g] in registers; finally * r_i + b_j -> bf16, transposed through
//                 shared memory and written with one TMA store per tile.
// Group partials rotate through the TMEM buffers, so the tensor core runs ahead of the drain (by one
// group with 256-token tiles, by up to seven with small tiles, where the hand-shake latency per group
// would otherwise dominate).
//
// Shared memory rings (stage = 128 input channels):
//   X  [SX][TT tokens][128 B]     int8, swizzled by TMA       full: TMA bytes     empty: umma commit
//   W  [SW][128 channels][128 B]  int8 x16, swizzled by hand  full: 4 warps       empty: umma commit
//   RAW[SR][128 channels][64 B]   packed INT4, as in memory   full: TMA bytes     empty: 4 warps
// 256-token tiles: the output tile [256 tokens][128 channels] bf16 is staged over the X ring once the last
// MMA is done.
// Small M (up to 256 tokens: action / proprio-only passes): the token tile shrinks to 32 / 64 and the K
// dimension is split over blockIdx.y so that about one CTA per SM streams its own slice of the
// weights.  Each split writes its fp32 partial
// tile [token][channel]; the CTA that arrives last at the tile's counter adds the partials in split
// order (deterministic) and stores its bf16 results straight from registers.  The kernel is launched
// with programmatic dependent launch: everything that does not read the prologue's output (barrier
// set-up, TMEM allocation) overlaps the prologue kernel.
// Persistent form (256-token tiles, one scale per output channel or integer-path groups of 128, at least three tiles per SM): one CTA
// per SM walks tiles blockIdx.x, + gridDim.x, ...  With a single weight group per tile the drain warps
// are idle during the main loop, so the whole tail of a tile -- drain, scaling, staging, store -- runs
// under the next tile's MMAs (the two TMEM buffers alternate per tile).  The output leaves through a
// 32 KB slab of its own (two passes of 64 tokens from each token half, so that all drain warps stage at
// once; two TMA stores per pass, waited for only when the slab is needed again); the rings give up one stage each to pay for it; the row scales
// of the next tile are staged by the otherwise idle warp 2 through two shared-memory slots.
// TMEM: NBUF = 512 / TT (at most 8) buffers of TT columns x 128 lanes of INT32, one weight group each.
// acc_full[b]: umma commit; acc_empty[b]: 8 epilogue warps.
#include "internal.cuh"
#include "ptx.cuh"

#include <cuda_bf16.h>

namespace rudder {

namespace {

constexpr int BN = 128;          // output channels per tile (MMA M)
constexpr int KSTAGE = 128;      // input channels (= bytes of int8 per row) per pipeline stage
constexpr int kPersistStagesX = 3;   // persistent form: activation stages
constexpr int kPersistStagesW = 3;   // persistent form: unpacked-weight stages
constexpr int kPersistTilesPerSm = 3;   // fewest tiles per SM for which the persistent form is used
constexpr int W_BYTES = BN * KSTAGE;
constexpr int SR = 4;            // packed-weight stages (256-token tiles)
constexpr int RAW_BYTES = BN * KSTAGE / 2;
constexpr int NUM_THREADS = 512;
constexpr int UNPACK_THREADS = 128;
constexpr int EPI_THREADS = 256;

// Registers per thread after setmaxnreg (256-token tiles): the drain warps hold 128 accumulators each.
constexpr int RUDDER_REGS_LO = 72;
constexpr int RUDDER_REGS_HI = 184;
// (persistent form: the other roles carry their tile loops and measured 2-3 % faster with eight registers more)
constexpr int RUDDER_REGS_LO_PERSIST = 80;
constexpr int RUDDER_REGS_HI_PERSIST = 176;
// Back-off (ns) between polls of a barrier, per role: the roles that are rarely on the critical path
// sleep between polls so that they do not take issue slots from the warps that share their scheduler.
constexpr int RUDDER_SLEEP_PROD = 64;
constexpr int RUDDER_SLEEP_UNPACK = 64;
constexpr int RUDDER_SLEEP_MMA = 0;
constexpr int RUDDER_SLEEP_EPI = 0;

// TT = tokens per tile (MMA N): 256, 64 or 32.  PERSIST (256 only): the CTA walks several tiles; a slab
// of 128 tokens x 128 channels of bf16 output gets its own shared memory (the rings belong to the next
// tile by the time a tile is written), paid for with shallower rings.
template <int TT, bool PERSIST = false> struct Tile {
    static constexpr int SX = PERSIST ? kPersistStagesX : ((TT == 256) ? 4 : 8);
    static constexpr int SW = PERSIST ? kPersistStagesW : 4;  // unpacked-weight stages
    static constexpr int X_BYTES = TT * KSTAGE;
    static constexpr int OFF_X = 0;
    static constexpr int OFF_W = OFF_X + SX * X_BYTES;
    static constexpr int OFF_RAW = OFF_W + SW * W_BYTES;
    static constexpr int OFF_OUT = OFF_RAW + SR * RAW_BYTES;
    static constexpr int OUT_BYTES = 128 * BN * 2;   // persistent form: half a tile of bf16 results
    static constexpr int BYTES = OFF_OUT + (PERSIST ? OUT_BYTES : 0);
    static constexpr int DYN_SMEM = BYTES + 1024;    // slack to align the base to 1024 bytes
    static constexpr int NBUF = (512 / TT > 8) ? 8 : 512 / TT;   // TMEM accumulator buffers (one weight group each)
    static constexpr int TMEM_COLS = NBUF * TT;
    static constexpr int EC = TT / 2;                // tokens per epilogue thread
    static constexpr int CH = (EC < 32) ? EC : 32;   // tokens per TMEM load
    static_assert(PERSIST || SX * X_BYTES >= TT * BN * 2, "the output tile is staged over the X ring");
    static_assert(!PERSIST || TT == 256, "the persistent form is built for 256-token tiles");
};

struct Params {
    int M, N, K, G;
    const float* scales_t;       // [K/G][N] fp32 = Delta_W / 16
    const float* row_scale;      // r [M]
    const float* bias;           // [N] or nullptr
    // The parity hook's window and the plain output pointer share storage (a launch uses one of them):
    // kernel parameters beyond 376 bytes cost this kernel 7 % at large M, measured.
    union {
        struct { int32_t* acc; int row0, rows, col0, cols; } dump;    // accumulator dump [K/G][rows][cols]
        struct { uint16_t* y; int64_t ldy; } out;                     // output bf16 [M, ldy]: tiles of 32 / 64 tokens are stored without TMA
    } aux;
    int m_tiles, n_tiles;        // token tiles, channel tiles (grid.x = m_tiles * n_tiles)
    int splitk;                  // K splits (grid.y)
    int stages_per_split;        // 128-channel stages per split
    float* partials;             // tiles of 32 / 64 tokens: [splitk][m_tiles * TT][N] fp32 partial sums (splitk > 1)
    const CUtensorMap* tm_w;     // tensor map (device memory) over the packed weights, box {64 B, 128 channels}
    int* counters;               // [m_tiles * n_tiles] arrivals per tile, zeroed by the prologue kernel
    // (16-bit fields: the block must stay within the size above)
    uint16_t pdl;                // launched with programmatic dependent launch
    uint16_t x_rows;             // token rows one activation TMA box delivers (128 bytes each)
    uint16_t out_pitch;          // channels per row of the staged output tile (= TMA store box width)
    uint16_t w_rows;             // channel rows one packed-weight TMA box delivers (64 bytes each)
};
static_assert(sizeof(Params) <= 120, "kernel parameters beyond 376 bytes slow the 256-token kernel");

enum Where {   // codes recorded when a bounded wait gives up
    W_X_EMPTY = 101, W_RAW_EMPTY = 102,
    W_W_EMPTY = 201, W_RAW_FULL = 202,
    W_X_FULL = 301, W_W_FULL = 302, W_ACC_EMPTY = 303,
    W_ACC_FULL = 401, W_RS_FULL = 402
};

__device__ __forceinline__ void sts128(uint32_t addr, const uint4& v) {
    asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}
// No memory clobber: the compiler may move the loads of the token scales across these stores (with a
// clobber every store waits for the load before it); the fence and barrier that follow are volatile
// too and keep their place relative to the stores.
__device__ __forceinline__ void sts16(uint32_t addr, uint16_t v) {
    asm volatile("st.shared.u16 [%0], %1;" ::"r"(addr), "h"(v));
}
__device__ __forceinline__ uint4 lds128(uint32_t addr) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr) : "memory");
    return v;
}
__device__ __forceinline__ float ldg_f32_volatile(const float* p) {
    float v;
    asm volatile("ld.global.nc.f32 %0, [%1];" : "=f"(v) : "l"(p));
    return v;
}
__device__ __forceinline__ float ld_f32_volatile(const float* p) {
    float v;
    asm volatile("ld.global.f32 %0, [%1];" : "=f"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ float ld_f32_cg(const float* p) {     // from L2; no clobber, so that several can be in flight
    float v;
    asm volatile("ld.global.cg.f32 %0, [%1];" : "=f"(v) : "l"(p));
    return v;
}
__device__ __forceinline__ float4 ld_f32x4_volatile(const float* p) {
    float4 v;
    asm volatile("ld.global.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void griddep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void tmem_ld_chunk(uint32_t taddr, uint32_t (&r)[32]) { tmem_ld_32x32b_x32(taddr, r); }
__device__ __forceinline__ void tmem_ld_chunk(uint32_t taddr, uint32_t (&r)[16]) { tmem_ld_32x32b_x16(taddr, r); }

// Eight packed 4-bit weights -> two words of four operand bytes each.
// Integer path: two's complement nibbles moved to the top half of the byte (the value 16 q).
// E4M3 path: sign-magnitude words (see the offline pack); the magnitudes index a table of the E4M3
// encodings of 0..7 held in two registers (byte permute), the signs are moved to bit 7.
template <bool F8>
__device__ __forceinline__ void unpack8(uint32_t pk, uint32_t& lo, uint32_t& hi) {
    if (F8) {
        const uint32_t t_lo = 0x44403800u, t_hi = 0x4E4C4A48u;      // E4M3 of 0, 1, 2, 3 and of 4, 5, 6, 7
        uint32_t ma, mb;
        asm("prmt.b32 %0, %1, %2, %3;" : "=r"(ma) : "r"(t_lo), "r"(t_hi), "r"(pk & 0x7777u));
        asm("prmt.b32 %0, %1, %2, %3;" : "=r"(mb) : "r"(t_lo), "r"(t_hi), "r"((pk >> 16) & 0x7777u));
        lo = ma | ((pk << 4) & 0x80808080u);
        hi = mb | (pk & 0x80808080u);
    } else {
        lo = (pk << 4) & 0xF0F0F0F0u;
        hi = pk & 0xF0F0F0F0u;
    }
}
template <bool F8>
__device__ __forceinline__ void unpack32(const uint4& pk, uint4& lo, uint4& hi) {
    unpack8<F8>(pk.x, lo.x, hi.x);
    unpack8<F8>(pk.y, lo.y, hi.y);
    unpack8<F8>(pk.z, lo.z, hi.z);
    unpack8<F8>(pk.w, lo.w, hi.w);
}

template <int TT, bool DUMP, bool F8, bool PERSIST>
__global__ void __launch_bounds__(NUM_THREADS, 1)
gemm_i8_w4_kernel(const __grid_constant__ CUtensorMap tm_x, const __grid_constant__ CUtensorMap tm_y, const Params p)
{
    using T = Tile<TT, PERSIST>;
    constexpr int SW = T::SW;
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t bars[2 * T::SX + 2 * T::SW + 2 * T::NBUF + 1 + 2 * SR + 4];
    __shared__ __align__(16) float rs_smem[PERSIST ? 2 * TT : TT];   // row scales r_i of the tile's tokens (0 past M); persistent form: two tiles' worth
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_word;
    __shared__ int last_flag;

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    // PERSIST (256-token tiles, no K split): the CTA walks tiles blockIdx.x, + gridDim.x, ...; rings, TMEM
    // buffers and their phases simply carry on from one tile to the next, so the MMAs of the next tile
    // run while the drain warps scale, stage and store the current one.
    // Otherwise the grid has one CTA per tile and every tile loop below runs once.
    const int total_tiles = p.m_tiles * p.n_tiles;
    const int tile_step = PERSIST ? static_cast<int>(gridDim.x) : total_tiles;
    auto tile_origin = [&](int tile, int& m0, int& n0) {
        int tile_m, tile_n;
        tile_coords(tile, p.m_tiles, p.n_tiles, 16, tile_m, tile_n);
        m0 = tile_m * TT;                    // first token of the tile
        n0 = tile_n * BN;                    // first output channel of the tile
    };
    // this CTA's share of K: stages [s0, s0 + n_stages), weight groups [g0, g0 + n_groups)
    const int n_stages = p.stages_per_split;
    const int s0 = blockIdx.y * n_stages;
    const int k_split = n_stages * KSTAGE;
    const int g_len = p.G < k_split ? p.G : k_split;     // a group longer than the split is cut: its partial
    const int n_groups = k_split / g_len;                // integer sums are scaled and added per split
    const int g0 = (s0 * KSTAGE) / p.G;

    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t bar0 = smem_u32(bars);
    auto x_full = [&](int i) { return bar0 + 8u * i; };
    auto x_empty = [&](int i) { return bar0 + 8u * (T::SX + i); };
    auto w_full = [&](int i) { return bar0 + 8u * (2 * T::SX + i); };
    auto w_empty = [&](int i) { return bar0 + 8u * (2 * T::SX + SW + i); };
    auto acc_full = [&](int i) { return bar0 + 8u * (2 * T::SX + 2 * SW + i); };
    auto acc_empty = [&](int i) { return bar0 + 8u * (2 * T::SX + 2 * SW + T::NBUF + i); };
    const uint32_t rs_full = bar0 + 8u * (2 * T::SX + 2 * SW + 2 * T::NBUF);
    auto raw_full = [&](int i) { return rs_full + 8u * (1 + i); };
    auto raw_empty = [&](int i) { return rs_full + 8u * (1 + SR + i); };
    auto rsp_full = [&](int i) { return rs_full + 8u * (1 + 2 * SR + i); };        // persistent form: row-scale slots
    auto rsp_empty = [&](int i) { return rs_full + 8u * (1 + 2 * SR + 2 + i); };

    if (threadIdx.x == 0) {
        abort_word = 0;
        for (int i = 0; i < T::SX; ++i) { mbar_init(x_full(i), 1); mbar_init(x_empty(i), 1); }
        for (int i = 0; i < SW; ++i) { mbar_init(w_full(i), UNPACK_THREADS / 32); mbar_init(w_empty(i), 1); }
        for (int i = 0; i < T::NBUF; ++i) { mbar_init(acc_full(i), 1); mbar_init(acc_empty(i), EPI_THREADS / 32); }
        mbar_init(rs_full, 1);
        for (int i = 0; i < SR; ++i) { mbar_init(raw_full(i), 1); mbar_init(raw_empty(i), UNPACK_THREADS / 32); }
        if (PERSIST)
            for (int i = 0; i < 2; ++i) { mbar_init(rsp_full(i), 1); mbar_init(rsp_empty(i), EPI_THREADS / 32); }
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
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");     // the next prologue kernel may start its own set-up

    if (warp < 8) {
    // The epilogue warpgroups hold TT/2 fp32 accumulators per thread: hand them the registers the
    // producer / MMA / unpack warpgroups do not need.
    if (TT == 256) reg_dec<PERSIST ? RUDDER_REGS_LO_PERSIST : RUDDER_REGS_LO>();
    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer (activations)
        if (lane == 0) {
            tma_prefetch_desc(&tm_x);
            tma_prefetch_desc(&tm_y);
            if (p.pdl) griddep_wait();                 // the activation codes come from the prologue kernel
            int issued = 0;
            bool ok = true;
            int slot = 0;
            uint32_t ph = 0;
            for (int tile = blockIdx.x; tile < total_tiles && ok; tile += tile_step) {
                int m0, n0;
                tile_origin(tile, m0, n0);
                for (int s = 0; s < n_stages; ++s) {
                    ok = mbar_wait<RUDDER_SLEEP_PROD>(x_empty(slot), ph ^ 1u, abortp, W_X_EMPTY);
                    if (!ok) break;
                    mbar_expect_tx(x_full(slot), static_cast<uint32_t>(p.x_rows) * KSTAGE);
                    tma_load_2d(smem_base + T::OFF_X + slot * T::X_BYTES, &tm_x, (s0 + s) * KSTAGE, m0, x_full(slot));
                    ++issued;
                    if (++slot == T::SX) { slot = 0; ph ^= 1u; }
                }
            }
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
            const uint32_t idesc = F8 ? umma_idesc_e4m3(BN, TT) : umma_idesc_i8(BN, TT);
            bool ok = true;
            // No divisions in this loop: every instruction on this path is latency the tensor core may
            // end up waiting for.
            const int mma_per_group = g_len >> 5;      // MMAs (K = 32 each) per weight group
            int in_group = 0;                          // MMAs issued so far in the current group
            uint32_t buf = 0, phb = 0;                 // accumulator buffer of the current group, its phase
            int g_issued = 0;                          // groups started so far
            int sx = 0, sw = 0;                        // ring slots
            uint32_t phx = 0, phw = 0;                 // ring phases
            for (int tile = blockIdx.x; tile < total_tiles && ok; tile += tile_step)
            for (int s = 0; s < n_stages && ok; ++s) {
                ok = mbar_wait<RUDDER_SLEEP_MMA>(x_full(sx), phx, abortp, W_X_FULL) &&
                     mbar_wait<RUDDER_SLEEP_MMA>(w_full(sw), phw, abortp, W_W_FULL);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                tcgen05_fence_after_sync();
                const uint64_t da = umma_desc_sw128(smem_base + T::OFF_W + sw * W_BYTES);        // weights: M side
                const uint64_t db = umma_desc_sw128(smem_base + T::OFF_X + sx * T::X_BYTES);     // tokens: N side
#pragma unroll
                for (int kk = 0; kk < KSTAGE / 32; ++kk) {
                    if (in_group == 0 && g_issued >= T::NBUF) {     // a buffer's first use needs no wait
                        ok = mbar_wait<RUDDER_SLEEP_MMA>(acc_empty(buf), phb ^ 1u, abortp, W_ACC_EMPTY);
                        ok = __all_sync(0xffffffffu, ok);
                        if (!ok) break;
                        tcgen05_fence_after_sync();
                    }
                    if (leader) {
                        if (F8) umma_e4m3(tmem_base + buf * TT, da + 2u * kk, db + 2u * kk, idesc, in_group == 0 ? 0u : 1u);
                        else    umma_i8(tmem_base + buf * TT, da + 2u * kk, db + 2u * kk, idesc, in_group == 0 ? 0u : 1u);
                    }
                    if (++in_group == mma_per_group) {
                        if (leader) umma_commit(acc_full(buf));
                        in_group = 0;
                        ++g_issued;
                        if (++buf == T::NBUF) { buf = 0; phb ^= 1u; }
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
        }
    } else if (warp == 2) {
        // ------------------------------------------------------------------ row scales of the tile -> shared
        if (PERSIST) {
            // one tile ahead of the drain warps, two slots
            bool ok = true;
            int it = 0;
            for (int tile = blockIdx.x; tile < total_tiles && ok; tile += tile_step, ++it) {
                int m0, n0;
                tile_origin(tile, m0, n0);
                const int slot = it & 1;
                ok = mbar_wait<RUDDER_SLEEP_PROD>(rsp_empty(slot), ((it >> 1) & 1) ^ 1u, abortp, W_RS_FULL);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                for (int i = lane; i < TT; i += 32) rs_smem[slot * TT + i] = (m0 + i < p.M) ? ld_f32_volatile(p.row_scale + m0 + i) : 0.0f;
                __syncwarp();
                if (lane == 0) mbar_arrive(rsp_full(slot));
            }
        }
        if (!PERSIST) {
            int m0, n0;
            tile_origin(blockIdx.x, m0, n0);
            if (p.pdl) griddep_wait();                 // so do the row scales
            for (int i = lane; i < TT; i += 32) rs_smem[i] = (m0 + i < p.M) ? ld_f32_volatile(p.row_scale + m0 + i) : 0.0f;
            __syncwarp();
            if (lane == 0) mbar_arrive(rs_full);
        }
    } else if (warp == 3) {
        // ------------------------------------------------------------------ TMA producer (packed weights)
        // The weights do not depend on the prologue kernel: this stream starts at once.  Channels past N
        // are zero-filled by the copy.
        if (lane == 0) {
            tma_prefetch_desc(p.tm_w);
            int issued = 0;
            bool ok = true;
            int slot = 0;
            uint32_t ph = 0;
            for (int tile = blockIdx.x; tile < total_tiles && ok; tile += tile_step) {
                int m0, n0;
                tile_origin(tile, m0, n0);
                for (int s = 0; s < n_stages; ++s) {
                    ok = mbar_wait<RUDDER_SLEEP_PROD>(raw_empty(slot), ph ^ 1u, abortp, W_RAW_EMPTY);
                    if (!ok) break;
                    mbar_expect_tx(raw_full(slot), static_cast<uint32_t>(p.w_rows) * (KSTAGE / 2));
                    tma_load_2d(smem_base + T::OFF_RAW + slot * RAW_BYTES, p.tm_w, (s0 + s) * (KSTAGE / 2), n0, raw_full(slot));
                    ++issued;
                    if (++slot == SR) { slot = 0; ph ^= 1u; }
                }
            }
            if (!ok) {
                for (int i = max(0, issued - SR); i < issued; ++i)
                    for (uint32_t it = 0; it < (1u << 16) && !mbar_try_wait(raw_full(i % SR), (i / SR) & 1); ++it) {}
            }
        }
    } else if (warp >= 4) {
        // ------------------------------------------------------------------ INT4 -> int8 unpack
        // 128 channels x 64 packed bytes per stage = 512 16-byte pieces, 4 per thread: piece idx covers
        // channel idx / 4, input channels [32 (idx % 4), 32 (idx % 4) + 32) of the stage.
        const int tid = threadIdx.x - 128;
        {
            bool ok = true;
            int sw = 0, sr = 0;
            uint32_t phw = 0, phr = 0;
            for (int tile = blockIdx.x; tile < total_tiles && ok; tile += tile_step) {
            int m0, n0;
            tile_origin(tile, m0, n0);
            bool valid[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) valid[i] = (n0 + ((i * UNPACK_THREADS + tid) >> 2)) < p.N;
            for (int s = 0; s < n_stages && ok; ++s) {
                ok = mbar_wait<RUDDER_SLEEP_UNPACK>(raw_full(sr), phr, abortp, W_RAW_FULL);
                if (!ok) break;
                uint4 cur[4];
                const uint32_t rsrc = smem_base + T::OFF_RAW + sr * RAW_BYTES;
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    cur[i] = lds128(rsrc + (i * UNPACK_THREADS + tid) * 16);
                    if (!valid[i]) cur[i] = make_uint4(0, 0, 0, 0);
                }
                ok = mbar_wait<RUDDER_SLEEP_UNPACK>(w_empty(sw), phw ^ 1u, abortp, W_W_EMPTY);
                if (!ok) break;
                const uint32_t dst = smem_base + T::OFF_W + sw * W_BYTES;
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int idx = i * UNPACK_THREADS + tid;
                    const int row = idx >> 2, ch = idx & 3;
                    const uint4 pk = cur[i];
                    uint4 lo, hi;
                    unpack32<F8>(pk, lo, hi);
                    const uint32_t drow = dst + (row >> 3) * 1024 + (row & 7) * 128;
                    sts128(drow + (((2 * ch) ^ (row & 7)) << 4), lo);
                    sts128(drow + (((2 * ch + 1) ^ (row & 7)) << 4), hi);
                }
                fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) { mbar_arrive(w_full(sw)); mbar_arrive(raw_empty(sr)); }
                if (++sw == SW) { sw = 0; phw ^= 1u; }
                if (++sr == SR) { sr = 0; phr ^= 1u; }
            }
            }
        }
    }
    } else {
        // ------------------------------------------------------------------ epilogue
        if (TT == 256) reg_inc<PERSIST ? RUDDER_REGS_HI_PERSIST : RUDDER_REGS_HI>();
        constexpr int EC = T::EC;
        constexpr int CH = T::CH;                // tokens per TMEM load
        constexpr int NCH = EC / CH;
        const int q = warp & 3;                  // TMEM lane quadrant this warp may read
        const int h = (warp - 8) >> 2;           // token half
        const int ch_local = q * 32 + lane;      // channel within the tile = TMEM lane
        int buf = 0;                             // TMEM buffer of the next group and its phase: carried across tiles
        uint32_t phb = 0;
        bool ok = true;
        int tile_it = 0;
        for (int tile = blockIdx.x; tile < total_tiles && ok; tile += tile_step, ++tile_it) {
        int m0, n0;
        tile_origin(tile, m0, n0);
        const int n = n0 + ch_local;
        const bool n_ok = n < p.N;
        float acc[EC];
#pragma unroll
        for (int j = 0; j < EC; ++j) acc[j] = 0.0f;
        // E4M3 path: the operands are the integers themselves (no factor 16 to undo) and the accumulators
        // arrive as fp32 holding exact integers, so a group costs one FMA per element and no conversion.
        // (Packed two-lane FMAs measured the same: the drain is bound by the FMA pipe and the register
        // file's write port, which the TMEM loads share, not by issue slots.)
        const float sc_mul = F8 ? 16.0f : 1.0f;
        // Scales are fetched two groups ahead with volatile loads: a plain load would be sunk next to
        // its use and expose the L2 latency once per group.
        const float* sc_ptr = p.scales_t + static_cast<size_t>(g0) * p.N + (n_ok ? n : 0);
        float sc_next = ldg_f32_volatile(sc_ptr);
        float sc_next2 = (n_groups > 1) ? ldg_f32_volatile(sc_ptr + p.N) : 0.0f;
        int g = 0;
        if (NCH == 1 && !DUMP) {
            // Small tiles: a group is one TMEM load per thread, so the fixed cost of a hand-shake (barrier
            // poll, vote, fences) dominates.  Take up to four groups per round: poll their barriers, issue
            // all the loads, wait once, then scale and accumulate.
            constexpr int GU = (T::NBUF >= 4) ? 4 : T::NBUF;
            for (; g + GU <= n_groups && ok; g += GU) {
                float scu[GU];
#pragma unroll
                for (int u = 0; u < GU; ++u) scu[u] = n_ok ? ldg_f32_volatile(sc_ptr + static_cast<size_t>(g + u) * p.N) : 0.0f;
#pragma unroll
                for (int u = 0; u < GU; ++u)
                    ok = ok && mbar_wait<RUDDER_SLEEP_EPI>(acc_full(buf + u), phb, abortp, W_ACC_FULL);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                tcgen05_fence_after_sync();
                uint32_t c[GU][CH];
#pragma unroll
                for (int u = 0; u < GU; ++u)
                    tmem_ld_chunk(tmem_base + (static_cast<uint32_t>(q * 32) << 16) + (buf + u) * TT + h * EC, c[u]);
                tmem_wait_ld();
#pragma unroll
                for (int u = 0; u < GU; ++u) {
                    if (F8) {
                        const float s16 = scu[u] * sc_mul;
#pragma unroll
                        for (int j = 0; j < CH; ++j) asm volatile("fma.rn.f32 %0, %1, %2, %0;" : "+f"(acc[j]) : "f"(__uint_as_float(c[u][j])), "f"(s16));
                    } else {
                        float f[CH];
#pragma unroll
                        for (int j = 0; j < CH; ++j) asm volatile("cvt.rn.f32.s32 %0, %1;" : "=f"(f[j]) : "r"(c[u][j]));
#pragma unroll
                        for (int j = 0; j < CH; ++j) asm volatile("fma.rn.f32 %0, %1, %2, %0;" : "+f"(acc[j]) : "f"(f[j]), "f"(scu[u]));
                    }
                }
                tcgen05_fence_before_sync();
                __syncwarp();
                if (lane == 0) {
#pragma unroll
                    for (int u = 0; u < GU; ++u) mbar_arrive(acc_empty(buf + u));
                }
                buf += GU;                               // NBUF is a multiple of GU: no wrap inside a round
                if (buf == T::NBUF) { buf = 0; phb ^= 1u; }
            }
            if (g < n_groups) {                          // the scale prefetch of the one-group loop starts here
                sc_next = ldg_f32_volatile(sc_ptr + static_cast<size_t>(g) * p.N);
                sc_next2 = (g + 1 < n_groups) ? ldg_f32_volatile(sc_ptr + static_cast<size_t>(g + 1) * p.N) : 0.0f;
            }
        }
        for (; g < n_groups && ok; ++g) {
            const float sc = n_ok ? sc_next * sc_mul : 0.0f;
            sc_next = sc_next2;
            if (g + 2 < n_groups) sc_next2 = ldg_f32_volatile(sc_ptr + static_cast<size_t>(g + 2) * p.N);
            // the outcome is made warp-uniform (the TMEM loads below are warp-collective)
            // every lane polls: a single polling lane followed by a shuffle measured 10 % slower per group
            ok = mbar_wait<RUDDER_SLEEP_EPI>(acc_full(buf), phb, abortp, W_ACC_FULL);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tcgen05_fence_after_sync();
            const uint32_t taddr = tmem_base + (static_cast<uint32_t>(q * 32) << 16) + buf * TT + h * EC;
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
                // Convert the whole chunk first, then accumulate: every FMA then finds its operand ready
                // instead of waiting out the conversion latency element by element.
                if (F8) {
#pragma unroll
                    for (int j = 0; j < CH; ++j) asm volatile("fma.rn.f32 %0, %1, %2, %0;" : "+f"(acc[ch * CH + j]) : "f"(__uint_as_float(cur[j])), "f"(sc));
                } else {
                    float f[CH];
#pragma unroll
                    for (int j = 0; j < CH; ++j) asm volatile("cvt.rn.f32.s32 %0, %1;" : "=f"(f[j]) : "r"(cur[j]));
#pragma unroll
                    for (int j = 0; j < CH; ++j) asm volatile("fma.rn.f32 %0, %1, %2, %0;" : "+f"(acc[ch * CH + j]) : "f"(f[j]), "f"(sc));
                }
                if (DUMP) {
                    const int cc = n - p.aux.dump.col0;
                    if (p.aux.dump.acc != nullptr && n_ok && cc >= 0 && cc < p.aux.dump.cols) {
#pragma unroll
                        for (int j = 0; j < CH; ++j) {
                            const int tok = m0 + h * EC + ch * CH + j;
                            const int rr = tok - p.aux.dump.row0;
                            if (tok < p.M && rr >= 0 && rr < p.aux.dump.rows)
                                p.aux.dump.acc[(static_cast<size_t>(g0 + g) * p.aux.dump.rows + rr) * p.aux.dump.cols + cc] = F8 ? static_cast<int>(__uint_as_float(cur[j])) : static_cast<int>(cur[j]) >> 4;
                        }
                    }
                }
            }
            tcgen05_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(acc_empty(buf));  // one arrival per warp: arrivals on one barrier serialise
            if (++buf == T::NBUF) { buf = 0; phb ^= 1u; }
        }
        if (PERSIST) {
            // The tile leaves through one slab of 32 KB in two passes: pass p holds tokens [64 p, 64 p + 64) of
            // both token halves (two boxes of 64 tokens x 128 channels, one TMA store each), so that all eight
            // drain warps stage at once.  A pass is staged once the stores that last used the slab have
            // read it; the wait for the second pass's stores is left to the next tile, whose MMAs are
            // running all the while.
            const float b = (p.bias != nullptr && n_ok) ? __ldg(p.bias + n) : 0.0f;
            const uint32_t slab = smem_base + T::OFF_OUT;
            const int rs_slot = tile_it & 1;
            if (ok) ok = mbar_wait<32>(rsp_full(rs_slot), (tile_it >> 1) & 1, abortp, W_RS_FULL);
            const float4* rs4 = reinterpret_cast<const float4*>(rs_smem + rs_slot * TT + h * EC);
#pragma unroll
            for (int pass = 0; pass < 2; ++pass) {
                if (threadIdx.x == 256) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
                // the barrier also makes the outcome common to all drain threads: they leave the tile loop together
                ok = bar_sync_and(1, EPI_THREADS, ok);
                if (ok) {
                    if (ch_local < p.out_pitch) {
                        const uint32_t step = static_cast<uint32_t>(p.out_pitch) * 2u;
                        uint32_t dst = slab + static_cast<uint32_t>(h) * (T::OUT_BYTES / 2) + static_cast<uint32_t>(ch_local) * 2u;
#pragma unroll
                        for (int jj = 0; jj < EC / 2; jj += 4) {
                            const int j = pass * (EC / 2) + jj;
                            const float4 rs = rs4[j >> 2];                   // broadcast read, zero past M
                            sts16(dst, __bfloat16_as_ushort(__float2bfloat16_rn(fmaf(acc[j + 0], rs.x, b)))); dst += step;
                            sts16(dst, __bfloat16_as_ushort(__float2bfloat16_rn(fmaf(acc[j + 1], rs.y, b)))); dst += step;
                            sts16(dst, __bfloat16_as_ushort(__float2bfloat16_rn(fmaf(acc[j + 2], rs.z, b)))); dst += step;
                            sts16(dst, __bfloat16_as_ushort(__float2bfloat16_rn(fmaf(acc[j + 3], rs.w, b)))); dst += step;
                        }
                    }
                    fence_proxy_async_smem();                    // generic writes -> visible to the TMA store
                }
                asm volatile("bar.sync 1, %0;" ::"n"(EPI_THREADS) : "memory");
                if (threadIdx.x == 256) {
#pragma unroll
                    for (int hh = 0; hh < 2; ++hh) {
                        const int t0 = m0 + hh * EC + pass * (EC / 2);
                        if (ok && t0 < p.M)
                            asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];"
                                         ::"l"(reinterpret_cast<uint64_t>(&tm_y)), "r"(slab + static_cast<uint32_t>(hh) * (T::OUT_BYTES / 2)),
                                           "r"(n0), "r"(t0) : "memory");
                    }
                    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(rsp_empty(rs_slot));      // this warp has read its row scales
            continue;
        }
        // Split K: publish this split's partial sums; the CTA that arrives last at the tile's counter adds
        // the splits in order and goes on to write the tile, the others are done.
        bool writer = true;
        if (TT <= 64 && p.splitk > 1) {            // only launches with tiles of 32 / 64 tokens split K
            const int m_pad = p.m_tiles * TT;
            // partials[split][token][channel]: a warp (32 consecutive channels) writes and reads whole
            // 128-byte lines.  (With the channel outermost every lane touched its own line, and the
            // reduction spent its time in the L1 tag stage: 32 lines per load instruction.)
            float* mine = p.partials + (static_cast<size_t>(blockIdx.y) * m_pad + m0 + h * EC) * p.N + (n_ok ? n : 0);
            if (ok && n_ok) {
#pragma unroll
                for (int j = 0; j < EC; ++j) mine[static_cast<size_t>(j) * p.N] = acc[j];
            }
            // The barrier orders every drain thread's stores before thread 256's release; its acquire on
            // the other side, again followed by a barrier, orders them before the readers' loads (which
            // go to L2).  One round trip instead of a fence per thread plus an atomic.
            asm volatile("bar.sync 1, %0;" ::"n"(EPI_THREADS) : "memory");
            if (threadIdx.x == 256) {
                int old;
                asm volatile("atom.add.acq_rel.gpu.global.s32 %0, [%1], 1;" : "=r"(old) : "l"(p.counters + blockIdx.x) : "memory");
                last_flag = (old == p.splitk - 1) ? 1 : 0;
            }
            asm volatile("bar.sync 1, %0;" ::"n"(EPI_THREADS) : "memory");
            writer = last_flag != 0;
            if (writer && ok) {
#pragma unroll
                for (int j = 0; j < EC; ++j) acc[j] = 0.0f;
                if (n_ok) {
                    // ZB splits are requested together (the loads of one split alone would expose one L2
                    // round trip per split) and added in split order.
                    constexpr int ZB = (EC >= 64) ? 1 : 64 / EC;
                    for (int z0 = 0; z0 < p.splitk; z0 += ZB) {
                        float v[ZB][EC];
#pragma unroll
                        for (int zz = 0; zz < ZB; ++zz) {
                            const int z = (z0 + zz < p.splitk) ? z0 + zz : p.splitk - 1;
                            const float* src = p.partials + (static_cast<size_t>(z) * m_pad + m0 + h * EC) * p.N + n;
#pragma unroll
                            for (int j = 0; j < EC; ++j) v[zz][j] = ld_f32_cg(src + static_cast<size_t>(j) * p.N);
                        }
#pragma unroll
                        for (int zz = 0; zz < ZB; ++zz) {
                            if (z0 + zz < p.splitk) {
#pragma unroll
                                for (int j = 0; j < EC; ++j) acc[j] += v[zz][j];
                            }
                        }
                    }
                }
            }
        }
        // The last acc_full arrives after every MMA of the tile has completed, so the X ring is free:
        // stage the transposed bf16 tile there ([token][channel], `out_pitch` channels per row).
        ok = ok && writer;
        if (ok) ok = mbar_wait<64>(rs_full, 0, abortp, W_RS_FULL);
        if (TT <= 64 && !DUMP) {
            // Small tiles: 16 or 32 results per thread go straight to global memory (a warp writes 64
            // contiguous bytes per token); nothing to stage, no store to wait for.
            if (ok && n_ok) {
                const float b = (p.bias != nullptr) ? __ldg(p.bias + n) : 0.0f;
                uint16_t* yp = p.aux.out.y + static_cast<size_t>(m0 + h * EC) * p.aux.out.ldy + n;
#pragma unroll
                for (int j = 0; j < EC; ++j) {
                    if (m0 + h * EC + j < p.M)
                        yp[static_cast<size_t>(j) * p.aux.out.ldy] = __bfloat16_as_ushort(__float2bfloat16_rn(fmaf(acc[j], rs_smem[h * EC + j], b)));
                }
            }
            ok = false;                                          // nothing left for the staged path below
        }
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
        }   // tile loop (one pass unless PERSIST)
        if (PERSIST && threadIdx.x == 256) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
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

template <int TT, bool DUMP, bool F8, bool PERSIST>
static cudaError_t launch_one(const GemmI8Args& a, const GemmI8Plan& plan, cudaStream_t st)
{
    using T = Tile<TT, PERSIST>;
    Params p;
    p.M = a.M; p.N = a.N; p.K = a.K; p.G = a.G;
    p.scales_t = a.w_scales_t;
    p.row_scale = a.row_scale; p.bias = a.bias;
    if (DUMP) { p.aux.dump.acc = a.acc; p.aux.dump.row0 = a.row0; p.aux.dump.rows = a.rows; p.aux.dump.col0 = a.col0; p.aux.dump.cols = a.cols; }
    else      { p.aux.out.y = a.y; p.aux.out.ldy = a.ldy; }
    p.x_rows = static_cast<uint16_t>(min(TT, a.M));
    p.out_pitch = static_cast<uint16_t>(min(BN, a.N));
    p.w_rows = static_cast<uint16_t>(min(BN, a.N));
    p.m_tiles = (a.M + TT - 1) / TT;
    p.n_tiles = (a.N + BN - 1) / BN;
    p.splitk = plan.splitk;
    p.stages_per_split = a.K / KSTAGE / plan.splitk;
    p.tm_w = a.tm_w;
    p.partials = a.partials;
    p.counters = a.counters;
    p.pdl = plan.pdl ? 1 : 0;

    cudaLaunchConfig_t cfg = {};
    const int tiles = p.m_tiles * p.n_tiles;
    cfg.gridDim = dim3(PERSIST ? min(tiles, max(1, a.sm_count)) : tiles, plan.splitk, 1);
    cfg.blockDim = dim3(NUM_THREADS, 1, 1);
    cfg.dynamicSmemBytes = T::DYN_SMEM;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = plan.pdl ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, gemm_i8_w4_kernel<TT, DUMP, F8, PERSIST>, a.tm_x, a.tm_y, p);
}

// Tile and split choice.  Large M: 256-token tiles, no split.  M <= 256: the smallest tile that holds
// the rows, and K split so that about one CTA per SM streams weights, as long as every split keeps at
// least two stages and the fp32 partials stay small (they must also fit the fixed scratch of
// rudder_linear_static).
GemmI8Plan gemm_i8_plan(int M, int N, int K, int G, bool f8, bool dump)
{
    GemmI8Plan plan;
    const int sm_count = device_sm_count();
    // The persistent form pays where the drain warps have slack during the main loop and a CTA gets
    // several tiles: one scale per output channel (a single group per tile, drain warps idle: 20 % faster)
    // and groups of 128 on the integer path (6 %); level at groups of 64, 10 % slower on the E4M3 path.
    {
        const long long tiles = static_cast<long long>((M + 255) / 256) * ((N + BN - 1) / BN);
        const bool shape_ok = G >= K || (G >= 128 && !f8);
        plan.persist = !dump && M > 256 && shape_ok && tiles >= static_cast<long long>(kPersistTilesPerSm) * sm_count;
    }
    // Small tiles (eight TMEM buffers) and split K wherever 256-token tiles would leave more than half of
    // the SMs without one: up to 256 rows always, above that while the 64-token tiles still fit one wave.
    const int n_tiles = (N + BN - 1) / BN;
    const long long tiles256 = static_cast<long long>((M + 255) / 256) * n_tiles;
    const long long tiles64 = static_cast<long long>((M + 63) / 64) * n_tiles;
    const bool small = M <= 256 || (tiles256 * 2 <= sm_count && tiles64 <= sm_count + sm_count / 12);
    plan.token_tile = !small ? 256 : (M > 32 ? 64 : 32);
    plan.splitk = 1;
    plan.pdl = false;
    if (dump || !small) return plan;
    const int m_tiles = (M + plan.token_tile - 1) / plan.token_tile;
    const int base = m_tiles * n_tiles;
    const size_t m_pad = static_cast<size_t>(m_tiles) * plan.token_tile;
    // Split K until about one CTA per SM, but leave every CTA at least four stages (deeper splits cost
    // more in the reduction than they gain) and keep the fp32 partial sums within 4 MiB.
    int sk = 1;
    while (sk < 16 && base * (sk * 2) <= sm_count + sm_count / 12 && (K / KSTAGE) % (sk * 2) == 0 && K / (sk * 2) >= 4 * KSTAGE &&
           static_cast<size_t>(sk * 2) * N * m_pad * sizeof(float) <= (size_t(4) << 20))
        sk *= 2;
    plan.splitk = sk;
    plan.pdl = true;
    return plan;
}

size_t gemm_i8_scratch_bytes(int M, int N, int K, bool dump, size_t* counters_offset)
{
    const GemmI8Plan plan = gemm_i8_plan(M, N, K, 0, false, dump);
    const int n_tiles = (N + BN - 1) / BN;
    const int m_tiles = (M + plan.token_tile - 1) / plan.token_tile;
    size_t partial = 0;
    if (plan.splitk > 1) partial = static_cast<size_t>(plan.splitk) * N * m_tiles * plan.token_tile * sizeof(float);
    partial = (partial + 255) / 256 * 256;
    if (counters_offset) *counters_offset = partial;
    const size_t counters = plan.splitk > 1 ? (static_cast<size_t>(m_tiles) * n_tiles * sizeof(int) + 255) / 256 * 256 : 0;
    return partial + counters;
}

cudaError_t gemm_i8_init()
{
    cudaError_t e;
#define RUDDER_I8_ATTR1(TT, D, F, P)                                                                                                  \
    e = cudaFuncSetAttribute(gemm_i8_w4_kernel<TT, D, F, P>, cudaFuncAttributeMaxDynamicSharedMemorySize, Tile<TT, P>::DYN_SMEM); \
    if (e != cudaSuccess) return e;
#define RUDDER_I8_ATTR(TT, D) RUDDER_I8_ATTR1(TT, D, false, false) RUDDER_I8_ATTR1(TT, D, true, false)
    RUDDER_I8_ATTR(32, false) RUDDER_I8_ATTR(64, false) RUDDER_I8_ATTR(256, false)
    RUDDER_I8_ATTR(32, true) RUDDER_I8_ATTR(64, true) RUDDER_I8_ATTR(256, true)
    RUDDER_I8_ATTR1(256, false, false, true) RUDDER_I8_ATTR1(256, false, true, true)
#undef RUDDER_I8_ATTR
#undef RUDDER_I8_ATTR1
    return cudaSuccess;
}

cudaError_t launch_gemm_i8(const GemmI8Args& a, cudaStream_t st)
{
    const GemmI8Plan plan = gemm_i8_plan(a.M, a.N, a.K, a.G, a.f8, a.acc != nullptr);
    const bool dump = a.acc != nullptr;
    if (plan.persist)
        return a.f8 ? launch_one<256, false, true, true>(a, plan, st) : launch_one<256, false, false, true>(a, plan, st);
#define RUDDER_I8_LAUNCH(TT)                                                                                     \
    return a.f8 ? (dump ? launch_one<TT, true, true, false>(a, plan, st) : launch_one<TT, false, true, false>(a, plan, st))   \
                : (dump ? launch_one<TT, true, false, false>(a, plan, st) : launch_one<TT, false, false, false>(a, plan, st));
    switch (plan.token_tile) {
        case 32:  RUDDER_I8_LAUNCH(32)
        case 64:  RUDDER_I8_LAUNCH(64)
        default:  RUDDER_I8_LAUNCH(256)
    }
#undef RUDDER_I8_LAUNCH
}

}  // namespace rudder
