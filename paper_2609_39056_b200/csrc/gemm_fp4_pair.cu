// NVFP4 W4A4 second kernel (Section 4.4; Eq. 10 with block-scaled operands) on CTA pairs.
//
// The single-CTA kernel of gemm_fp4.cu is bound by the shared-memory fill rate: a 128-channel x
// 256-token tile needs 128 + 256 operand rows per K step.  Here two CTAs of a cluster (two SMs) share
// one 256-channel x 256-token tile with tcgen05.mma.cta_group::2: each CTA stages its own 128 weight
// rows and HALF of the token rows (the tensor cores of the pair read each other's half), so a CTA
// moves 128 + 128 rows for the same 128 x 256 outputs, a third less.
//   both CTAs   warp 0: TMA producer for this CTA's operand rows and scale factors; every copy counts
//               its bytes on the full barrier of the pair's first CTA (the leader)
//               warps 4-11: epilogue of this CTA's 128 channels, as in the single-CTA kernel
//   leader      warp 1: scale copies smem -> TMEM and MMAs for the pair (both with cta_group::2);
//               tcgen05.commit signals the empty / accumulator-full barriers of both CTAs
// The epilogue warps of both CTAs report "accumulator drained" to the leader's barrier.
// All waits are bounded; a CTA leaves only through the cluster barrier at the end, so no barrier of a
// CTA that has already exited is ever signalled.
#include "internal.cuh"
#include "ptx.cuh"

#include <cuda_bf16.h>

namespace rudder {

namespace fp4 {

constexpr int PAIR_TT = 256;                         // tokens per pair tile (MMA N)
constexpr int PAIR_S = 4;                            // pipeline stages
constexpr int PAIR_X_BYTES = 128 * KSTAGE_BYTES;     // this CTA's half of the token rows
constexpr int PAIR_W_BYTES = BN * KSTAGE_BYTES;
constexpr int PAIR_SFW_BYTES = KSTEPS * SF_CHUNK;
constexpr int PAIR_SFX_BYTES = 2 * KSTEPS * SF_CHUNK;    // all 256 tokens: every CTA needs the scales of the whole N side
constexpr int PAIR_STAGE_BYTES = PAIR_X_BYTES + PAIR_W_BYTES + PAIR_SFW_BYTES + PAIR_SFX_BYTES;
constexpr int PAIR_EC = PAIR_TT / 2;
constexpr int PAIR_SLAB_TOK = PAIR_EC / 2;
constexpr int PAIR_SLAB_BYTES = PAIR_SLAB_TOK * BN * 2;
constexpr int PAIR_OFF_X = 0;
constexpr int PAIR_OFF_W = PAIR_OFF_X + PAIR_S * PAIR_X_BYTES;
constexpr int PAIR_OFF_SFW = PAIR_OFF_W + PAIR_S * PAIR_W_BYTES;
constexpr int PAIR_OFF_SFX = PAIR_OFF_SFW + PAIR_S * PAIR_SFW_BYTES;
constexpr int PAIR_OFF_OUT = PAIR_OFF_SFX + PAIR_S * PAIR_SFX_BYTES;
constexpr int PAIR_DYN_SMEM = PAIR_OFF_OUT + 4 * PAIR_SLAB_BYTES + 1024;   // four output slabs: two per epilogue phase
constexpr int PAIR_SF_COLS = KSTEPS * 4 * 3;         // scale columns per region: weights 4, tokens 8 per MMA
constexpr int PAIR_TMEM_COLS = 512;

struct PairParams {
    int M, N, K;
    const float* row_scale;
    const float* tensor_scale;
    const float* bias;
    int m_tiles, n_tiles;        // token tiles (256), channel-pair tiles (256)
};

enum PairWhere { WP_EMPTY = 611, WP_FULL = 711, WP_ACC_EMPTY = 712, WP_ACC_FULL = 811 };

// Shared-memory store that the compiler may move loads across (the fences and barriers that follow
// are volatile and keep it in place relative to them).
__device__ __forceinline__ void sts16_free(uint32_t addr, uint16_t v) {
    asm volatile("st.shared.u16 [%0], %1;" ::"r"(addr), "h"(v));
}
__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
// Address of the same shared-memory offset in the CTA of rank `rank` of this cluster.
__device__ __forceinline__ uint32_t map_to_rank(uint32_t addr, uint32_t rank) {
    uint32_t out;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(out) : "r"(addr), "r"(rank));
    return out;
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
    asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// Tiled loads whose completion bytes are counted on a barrier that may live in the peer CTA.
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* tm, int x, int y, uint32_t bar_cluster) {
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(tm)), "r"(bar_cluster), "r"(x), "r"(y)
        : "memory");
}
__device__ __forceinline__ void tma_load_3d_pair(uint32_t dst, const CUtensorMap* tm, int x, int y, int z, uint32_t bar_cluster) {
    asm volatile(
        "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(tm)), "r"(bar_cluster), "r"(x), "r"(y), "r"(z)
        : "memory");
}
__device__ __forceinline__ void tmem_alloc_pair(uint32_t smem_dst, uint32_t ncols) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_dst), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish_pair() {
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t taddr, uint32_t ncols) {
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
// Scale chunk smem -> TMEM in both CTAs of the pair, each from its own shared memory.
__device__ __forceinline__ void tmem_cp_sf_pair(uint32_t taddr, uint64_t desc) {
    asm volatile("tcgen05.cp.cta_group::2.32x128b.warpx4 [%0], %1;" ::"r"(taddr), "l"(desc) : "memory");
}
__device__ __forceinline__ void umma_nvfp4_pair(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b, uint32_t idesc,
                                                uint32_t tmem_sfa, uint32_t tmem_sfb, uint32_t accumulate) {
    asm volatile(
        "{\n\t"
        ".reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::mxf4nvf4.block_scale.block16 [%0], %1, %2, %3, [%5], [%6], p;\n\t"
        "}\n"
        ::"r"(tmem_d), "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(accumulate), "r"(tmem_sfa), "r"(tmem_sfb)
        : "memory");
}
// All MMAs issued so far by this thread: when they are done, arrive on the barrier at this offset in
// both CTAs of the pair.
__device__ __forceinline__ void umma_commit_pair(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(bar), "h"(static_cast<uint16_t>(3)) : "memory");
}

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(NUM_THREADS, 1)
gemm_nvfp4_pair_kernel(const __grid_constant__ CUtensorMap tm_x, const __grid_constant__ CUtensorMap tm_w,
                       const __grid_constant__ CUtensorMap tm_sfx, const __grid_constant__ CUtensorMap tm_sfw,
                       const __grid_constant__ CUtensorMap tm_y, const PairParams p)
{
    constexpr int S = PAIR_S;
    constexpr int TT = PAIR_TT;
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t bars[2 * S + 2];
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_word;
    __shared__ __align__(16) float rs_smem[PAIR_TT];               // r_i * s_W of the tile's tokens

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();
    const int pair = blockIdx.x >> 1;
    const int n_pairs = gridDim.x >> 1;
    const int n_stages = p.K / 256;
    const int total_tiles = p.m_tiles * p.n_tiles;

    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t bar0 = smem_u32(bars);
    auto full = [&](int i) { return bar0 + 8u * i; };              // used in the leader only
    auto empty = [&](int i) { return bar0 + 8u * (S + i); };
    const uint32_t acc_full = bar0 + 8u * (2 * S);
    const uint32_t acc_empty = bar0 + 8u * (2 * S + 1);            // used in the leader only

    if (threadIdx.x == 0) {
        abort_word = 0;
        for (int i = 0; i < S; ++i) { mbar_init(full(i), 1); mbar_init(empty(i), 1); }
        mbar_init(acc_full, 1);
        mbar_init(acc_empty, 2 * (EPI_THREADS / 32));              // the epilogue warps of both CTAs
        fence_mbar_init();
    }
    if (warp == 1) {
        tmem_alloc_pair(smem_u32(&tmem_slot), PAIR_TMEM_COLS);
        tmem_relinquish_pair();
    }
    tcgen05_fence_before_sync();
    cluster_sync_all();                       // barriers and TMEM of both CTAs exist from here on
    tcgen05_fence_after_sync();
    const uint32_t tmem_base = tmem_slot;
    volatile int* abortp = &abort_word;
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");     // the next prologue kernel may start its own set-up
    // Launched ahead of the prologue kernel's end: everything above is this CTA's own set-up; the codes,
    // scales and token scales that the roles below read are the prologue's output.
    asm volatile("griddepcontrol.wait;" ::: "memory");

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer (both CTAs)
        if (lane == 0) {
            tma_prefetch_desc(&tm_x);
            tma_prefetch_desc(&tm_w);
            tma_prefetch_desc(&tm_sfx);
            tma_prefetch_desc(&tm_sfw);
            tma_prefetch_desc(&tm_y);
            int issued = 0, slot = 0;
            uint32_t ph = 0;
            bool ok = true;
            for (int tile = pair; tile < total_tiles && ok; tile += n_pairs) {
                int tm, tn;
                tile_coords(tile, p.m_tiles, p.n_tiles, kGroupM, tm, tn);
                const int m0 = tm * TT;
                const int n0 = tn * 2 * BN + static_cast<int>(rank) * BN;
                for (int s = 0; s < n_stages; ++s) {
                    ok = mbar_wait<32>(empty(slot), ph ^ 1u, abortp, WP_EMPTY);
                    if (!ok) break;
                    const uint32_t fb = map_to_rank(full(slot), 0);
                    if (rank == 0) mbar_expect_tx(full(slot), 2u * PAIR_STAGE_BYTES);
                    tma_load_2d_pair(smem_base + PAIR_OFF_X + slot * PAIR_X_BYTES, &tm_x, s * KSTAGE_BYTES,
                                     m0 + static_cast<int>(rank) * 128, fb);
                    tma_load_2d_pair(smem_base + PAIR_OFF_W + slot * PAIR_W_BYTES, &tm_w, s * KSTAGE_BYTES, n0, fb);
                    tma_load_3d_pair(smem_base + PAIR_OFF_SFW + slot * PAIR_SFW_BYTES, &tm_sfw, 0, s * KSTEPS, n0 >> 7, fb);
                    tma_load_3d_pair(smem_base + PAIR_OFF_SFX + slot * PAIR_SFX_BYTES, &tm_sfx, 0, s * KSTEPS, m0 >> 7, fb);
                    ++issued;
                    if (++slot == S) { slot = 0; ph ^= 1u; }
                }
            }
            if (!ok && rank == 0) {           // give copies in flight a bounded time to land
                for (int i = max(0, issued - S); i < issued; ++i)
                    for (uint32_t it = 0; it < (1u << 16) && !mbar_try_wait(full(i % S), (i / S) & 1); ++it) {}
            }
        }
    } else if (warp == 1 && rank == 0) {
        // ------------------------------------------------------------------ scale copies + MMA issue (leader)
        const bool leader = elect_one();
        const uint32_t idesc = idesc_nvfp4(2 * BN, TT);
        bool ok = true;
        int slot = 0;
        uint32_t ph = 0, region = 0, tile_ph = 0;
        for (int tile = pair; tile < total_tiles && ok; tile += n_pairs) {
            ok = mbar_wait(acc_empty, tile_ph ^ 1u, abortp, WP_ACC_EMPTY);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tcgen05_fence_after_sync();
            for (int s = 0; s < n_stages; ++s) {
                ok = mbar_wait(full(slot), ph, abortp, WP_FULL);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                tcgen05_fence_after_sync();
                if (leader) {
                    const uint32_t sf_cols = tmem_base + TT + region * PAIR_SF_COLS;
                    const uint32_t sfw_smem = smem_base + PAIR_OFF_SFW + slot * PAIR_SFW_BYTES;
                    const uint32_t sfx_smem = smem_base + PAIR_OFF_SFX + slot * PAIR_SFX_BYTES;
                    const uint64_t da = umma_desc_sw128(smem_base + PAIR_OFF_W + slot * PAIR_W_BYTES);
                    const uint64_t db = umma_desc_sw128(smem_base + PAIR_OFF_X + slot * PAIR_X_BYTES);
#pragma unroll
                    for (int j = 0; j < KSTEPS; ++j) {
                        const uint32_t t_sfw = sf_cols + j * 4;
                        const uint32_t t_sfx = sf_cols + KSTEPS * 4 + j * 8;
                        tmem_cp_sf_pair(t_sfw, sf_desc(sfw_smem + j * SF_CHUNK));
                        tmem_cp_sf_pair(t_sfx, sf_desc(sfx_smem + j * SF_CHUNK));
                        tmem_cp_sf_pair(t_sfx + 4, sf_desc(sfx_smem + (KSTEPS + j) * SF_CHUNK));
                        umma_nvfp4_pair(tmem_base, da + 2u * j, db + 2u * j, idesc, t_sfw, t_sfx, (s > 0 || j > 0) ? 1u : 0u);
                    }
                    umma_commit_pair(empty(slot));
                    if (s == n_stages - 1) umma_commit_pair(acc_full);
                }
                __syncwarp();
                region ^= 1u;
                if (++slot == S) { slot = 0; ph ^= 1u; }
            }
            tile_ph ^= 1u;
        }
    } else if (warp >= 4) {
        // ------------------------------------------------------------------ epilogue (both CTAs)
        constexpr int EC = PAIR_EC;
        constexpr int SLAB = PAIR_SLAB_TOK;
        const int q = warp & 3;
        const int h = (warp - 4) >> 2;
        const int ch_local = q * 32 + lane;
        const float sw = __ldg(p.tensor_scale);
        const uint32_t out_base = smem_base + PAIR_OFF_OUT + h * PAIR_SLAB_BYTES;   // this thread's slab of phase 0
        const uint32_t acc_empty_leader = map_to_rank(acc_empty, 0);
        bool ok = true;
        uint32_t tile_ph = 0;
        for (int tile = pair; tile < total_tiles; tile += n_pairs) {
            int tm, tn;
            tile_coords(tile, p.m_tiles, p.n_tiles, kGroupM, tm, tn);
            const int m0 = tm * TT;
            const int n0 = tn * 2 * BN + static_cast<int>(rank) * BN;
            const int n = n0 + ch_local;
            const float b = (p.bias != nullptr) ? __ldg(p.bias + n) : 0.0f;
            {   // token scales of this tile; read after the next epilogue barrier.  The previous tile's
                // reads all came before its last barrier, which this thread has passed.
                const int tok = m0 + static_cast<int>(threadIdx.x) - 128;
                rs_smem[threadIdx.x - 128] = tok < p.M ? __fmul_rn(__ldg(p.row_scale + tok), sw) : 0.0f;
            }
            ok = mbar_wait(acc_full, tile_ph, abortp, WP_ACC_FULL);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tile_ph ^= 1u;
            tcgen05_fence_after_sync();
            // Pull the thread's whole share of the accumulator into registers, then hand TMEM back: the
            // next tile's MMAs run while this tile is scaled, converted and stored.
            uint32_t v[EC];
            const uint32_t taddr = tmem_base + (static_cast<uint32_t>(q * 32) << 16) + h * EC;
#pragma unroll
            for (int c = 0; c < EC / 32; ++c) tmem_ld_32x32b_x32(taddr + c * 32, *reinterpret_cast<uint32_t(*)[32]>(&v[c * 32]));
            tmem_wait_ld();
            tcgen05_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(acc_empty_leader);
#pragma unroll
            for (int phase = 0; phase < 2; ++phase) {
                // tokens [h EC + phase SLAB, + SLAB) of the tile go to slab 2 phase + h.  The stores of a
                // phase are not waited for until its slabs are needed again, one tile later.
                const uint32_t out0 = out_base + phase * 2 * PAIR_SLAB_BYTES;
                if (threadIdx.x == 128) asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
                asm volatile("bar.sync 1, %0;" ::"n"(EPI_THREADS) : "memory");
#pragma unroll
                for (int j = 0; j < SLAB; j += 4) {
                    const float4 rr4 = *reinterpret_cast<const float4*>(&rs_smem[h * EC + phase * SLAB + j]);
                    const float rr[4] = {rr4.x, rr4.y, rr4.z, rr4.w};
#pragma unroll
                    for (int t = 0; t < 4; ++t) {
                        const __nv_bfloat16 y = __float2bfloat16_rn(fmaf(__uint_as_float(v[phase * SLAB + j + t]), rr[t], b));
                        sts16_free(out0 + static_cast<uint32_t>((j + t) * BN + ch_local) * 2u, __bfloat16_as_ushort(y));
                    }
                }
                fence_proxy_async_smem();
                asm volatile("bar.sync 1, %0;" ::"n"(EPI_THREADS) : "memory");
                if (threadIdx.x == 128) {
#pragma unroll
                    for (int hh = 0; hh < 2; ++hh) {
                        const int tok0 = m0 + hh * EC + phase * SLAB;
                        if (tok0 < p.M)
                            asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];"
                                         ::"l"(reinterpret_cast<uint64_t>(&tm_y)),
                                           "r"(smem_base + PAIR_OFF_OUT + (2 * phase + hh) * PAIR_SLAB_BYTES), "r"(n0), "r"(tok0) : "memory");
                    }
                    asm volatile("cp.async.bulk.commit_group;" ::: "memory");    // one group per phase, even when empty
                }
            }
        }
        (void)ok;
        if (threadIdx.x == 128) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
    }

    __syncwarp();
    tcgen05_fence_before_sync();
    cluster_sync_all();                       // nobody signals a barrier of, or reads operands from, a CTA that has left
    if (warp == 1) {
        tcgen05_fence_after_sync();
        tmem_dealloc_pair(tmem_base, PAIR_TMEM_COLS);
    }
}

}  // namespace fp4

// The pair kernel needs whole 256-channel tiles and is worth its fixed cost only with many tokens.
bool gemm_fp4_use_pair(int M, int N, int K)
{
    return M >= 1024 && N % 256 == 0 && K % 256 == 0;
}

static int g_pair_clusters[64] = {0};

cudaError_t gemm_fp4_pair_init()
{
    cudaError_t e = cudaFuncSetAttribute(fp4::gemm_nvfp4_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, fp4::PAIR_DYN_SMEM);
    if (e != cudaSuccess) return e;
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev >= 0 && dev < 64) {
        // how many CTA pairs the device runs at once
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(2 * device_sm_count(), 1, 1);
        cfg.blockDim = dim3(fp4::NUM_THREADS, 1, 1);
        cfg.dynamicSmemBytes = fp4::PAIR_DYN_SMEM;
        int n = 0;
        if (cudaOccupancyMaxActiveClusters(&n, fp4::gemm_nvfp4_pair_kernel, &cfg) != cudaSuccess || n < 1) n = 0;
        g_pair_clusters[dev] = n;
    }
    return cudaSuccess;
}

cudaError_t launch_gemm_fp4_pair(const GemmFp4Args& a, cudaStream_t st)
{
    fp4::PairParams p;
    p.M = a.M; p.N = a.N; p.K = a.K;
    p.row_scale = a.row_scale; p.tensor_scale = a.tensor_scale; p.bias = a.bias;
    p.m_tiles = (a.M + fp4::PAIR_TT - 1) / fp4::PAIR_TT;
    p.n_tiles = a.N / (2 * fp4::BN);
    int dev = 0;
    cudaGetDevice(&dev);
    int clusters = (dev >= 0 && dev < 64) ? g_pair_clusters[dev] : 0;
    if (clusters < 1) clusters = a.sm_count / 2;
    const int tiles = p.m_tiles * p.n_tiles;
    const int pairs = tiles < clusters ? tiles : clusters;
    return launch_early(fp4::gemm_nvfp4_pair_kernel, 2 * pairs, fp4::NUM_THREADS, fp4::PAIR_DYN_SMEM, st, a.tm_x, a.tm_w, a.tm_sfx,
                        a.tm_sfw, a.tm_y, p);
}

}  // namespace rudder
