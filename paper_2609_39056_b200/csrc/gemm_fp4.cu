// NVFP4 W4A4 variant of the second kernel (Section 4.4; Eq. 10 with block-scaled operands): E2M1
// codes x E2M1 codes with one UE4M3 scale per 16 input channels on either side, multiplied and
// accumulated in fp32 by the block-scaled tensor-core instruction (tcgen05.mma kind::mxf4nvf4), so
// the only work left for the epilogue is acc * (r_i * s_W) + b_j -> bf16, once per tile.
//
// Orientation as in the integer kernel: 128 output channels on the MMA M side (TMEM lanes), TT tokens
// on the N side.  Stage = 256 input channels = 128 bytes of packed codes per row = 4 MMAs of K = 64.
//   warp 0       TMA producer: activation codes, weight codes (128-byte swizzle), and the block scales
//                of both sides (plain bulk copies of 512-byte chunks laid out in the tensor core's order)
//   warp 1       allocates TMEM; converged loop, one elected lane copies the scales smem -> TMEM
//                (tcgen05.cp) and issues the MMAs
//   warps 4-11   epilogue: TMEM -> registers (then TMEM is handed back at once) -> * (r_i s_W) + b_j
//                -> bf16 -> shared, in two slabs per phase -> TMA stores
// Persistent: one CTA per SM walks its tiles, so the epilogue of a tile overlaps the main loop of the
// next one and TMEM / barriers are set up once.
// TMEM: TT columns of fp32 accumulators, then two alternating regions of scale columns (4 columns per
// 128 rows per MMA).
#include "internal.cuh"
#include "ptx.cuh"

#include <cuda_bf16.h>

namespace rudder {

constexpr int BN_FP4 = 128;        // output channels per single-CTA tile

namespace fp4 {

constexpr int BN = 128;            // output channels per tile (MMA M)
constexpr int KSTAGE_BYTES = 128;  // packed bytes per row per stage (256 input channels)
constexpr int KSTEPS = 4;          // MMAs (K = 64) per stage
constexpr int SF_CHUNK = 512;      // scale bytes of 128 rows x 64 input channels
constexpr int NUM_THREADS = 384;
constexpr int EPI_THREADS = 256;
constexpr int kGroupM = 16;        // token tiles per rasterisation group (their activation rows stay in L2)

template <int TT> struct Tile {
    static constexpr int S = (TT == 256) ? 3 : 5;                 // pipeline stages
    static constexpr int ATOMS = TT / 128;                        // 128-token scale atoms per tile
    static constexpr int X_BYTES = TT * KSTAGE_BYTES;
    static constexpr int W_BYTES = BN * KSTAGE_BYTES;
    static constexpr int SFW_BYTES = KSTEPS * SF_CHUNK;
    static constexpr int SFX_BYTES = ATOMS * KSTEPS * SF_CHUNK;
    static constexpr int EC = TT / 2;                             // tokens per epilogue thread
    static constexpr int SLAB_TOK = EC / 2;                       // tokens per staged slab (= TMA store box rows)
    static constexpr int SLAB_BYTES = SLAB_TOK * BN * 2;
    static constexpr int OFF_X = 0;
    static constexpr int OFF_W = OFF_X + S * X_BYTES;
    static constexpr int OFF_SFW = OFF_W + S * W_BYTES;
    static constexpr int OFF_SFX = OFF_SFW + S * SFW_BYTES;
    static constexpr int OFF_OUT = OFF_SFX + S * SFX_BYTES;       // two slabs of the bf16 output tile
    static constexpr int BYTES = OFF_OUT + 2 * SLAB_BYTES;
    static constexpr int DYN_SMEM = BYTES + 1024;
    static constexpr int SF_COLS = KSTEPS * 4 * (1 + ATOMS);      // scale columns per region
    static constexpr int TMEM_COLS = (TT + 2 * SF_COLS > 256) ? 512 : 256;
};

struct Params {
    int M, N, K;
    const uint8_t* sf_x;
    const uint8_t* sf_w;
    const float* row_scale;
    const float* tensor_scale;
    const float* bias;
    uint32_t x_tx, w_tx;
    int out_pitch;
    int m_atoms;                 // 128-row scale atoms that exist on the activation side
    int m_tiles, n_tiles;        // token tiles, channel tiles
};

enum Where { W_EMPTY = 601, W_FULL = 701, W_ACC_EMPTY = 702, W_ACC_FULL = 801 };

// No memory clobber: the loads of the token scales may move across these stores; the fence and
// barrier that follow are volatile too and keep their place relative to the stores.
__device__ __forceinline__ void sts16(uint32_t addr, uint16_t v) {
    asm volatile("st.shared.u16 [%0], %1;" ::"r"(addr), "h"(v));
}
// 1D bulk copy global -> shared, completion counted on an mbarrier (addresses and size multiples of 16).
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
// Shared-memory descriptor of one 512-byte scale chunk: 32 rows x 16 bytes, no swizzle, 8-row groups 128 B apart.
__device__ __forceinline__ uint64_t sf_desc(uint32_t smem_addr) {
    uint64_t d = 0;
    d |= static_cast<uint64_t>((smem_addr & 0x3FFFFu) >> 4);
    d |= static_cast<uint64_t>(1) << 16;
    d |= static_cast<uint64_t>(128 >> 4) << 32;
    d |= static_cast<uint64_t>(1) << 46;
    return d;
}
// 32 lanes x 128 bits from shared memory into 4 TMEM columns, replicated to the four lane quadrants.
__device__ __forceinline__ void tmem_cp_sf(uint32_t taddr, uint64_t desc) {
    asm volatile("tcgen05.cp.cta_group::1.32x128b.warpx4 [%0], %1;" ::"r"(taddr), "l"(desc) : "memory");
}
// Instruction descriptor for kind::mxf4nvf4: E2M1 x E2M1, UE4M3 scales, both operands K-major, K = 64.
__device__ __forceinline__ uint32_t idesc_nvfp4(int m, int n) {
    uint32_t d = 0;
    d |= 1u << 7;                 // A format: E2M1
    d |= 1u << 10;                // B format: E2M1
    d |= static_cast<uint32_t>(n >> 3) << 17;
    d |= static_cast<uint32_t>(m >> 4) << 24;     // bit 23 = 0: UE4M3 scales
    return d;
}
__device__ __forceinline__ void umma_nvfp4(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b, uint32_t idesc,
                                           uint32_t tmem_sfa, uint32_t tmem_sfb, uint32_t accumulate) {
    asm volatile(
        "{\n\t"
        ".reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::mxf4nvf4.block_scale.block16 [%0], %1, %2, %3, [%5], [%6], p;\n\t"
        "}\n"
        ::"r"(tmem_d), "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(accumulate), "r"(tmem_sfa), "r"(tmem_sfb)
        : "memory");
}

// Persistent kernel: CTA b works on tiles b, b + gridDim.x, ... in the grouped order of tile_coords.
template <int TT>
__global__ void __launch_bounds__(NUM_THREADS, 1)
gemm_nvfp4_kernel(const __grid_constant__ CUtensorMap tm_x, const __grid_constant__ CUtensorMap tm_w,
                  const __grid_constant__ CUtensorMap tm_y, const Params p)
{
    using T = Tile<TT>;
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t bars[2 * T::S + 2];
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_word;

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const int n_stages = p.K / 256;
    const int k64 = p.K / 64;
    const int total_tiles = p.m_tiles * p.n_tiles;

    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t bar0 = smem_u32(bars);
    auto full = [&](int i) { return bar0 + 8u * i; };
    auto empty = [&](int i) { return bar0 + 8u * (T::S + i); };
    const uint32_t acc_full = bar0 + 8u * (2 * T::S);
    const uint32_t acc_empty = bar0 + 8u * (2 * T::S + 1);

    if (threadIdx.x == 0) {
        abort_word = 0;
        for (int i = 0; i < T::S; ++i) { mbar_init(full(i), 1); mbar_init(empty(i), 1); }
        mbar_init(acc_full, 1);
        mbar_init(acc_empty, EPI_THREADS / 32);
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
    // Launched ahead of the prologue kernel's end: everything above is this CTA's own set-up; the codes,
    // scales and token scales that the roles below read are the prologue's output.
    asm volatile("griddepcontrol.wait;" ::: "memory");

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            tma_prefetch_desc(&tm_x);
            tma_prefetch_desc(&tm_w);
            tma_prefetch_desc(&tm_y);
            int issued = 0, slot = 0;
            uint32_t ph = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x) {
                int tm, tn;
                tile_coords(tile, p.m_tiles, p.n_tiles, kGroupM, tm, tn);
                const int m0 = tm * TT;
                const int n0 = tn * BN;
                // scale atoms of this tile that exist (the last token tile may own fewer)
                int atoms = p.m_atoms - (m0 >> 7);
                atoms = atoms > T::ATOMS ? T::ATOMS : atoms;
                const uint32_t tx = p.x_tx + p.w_tx + T::SFW_BYTES + static_cast<uint32_t>(atoms) * KSTEPS * SF_CHUNK;
                const uint8_t* sfw_src = p.sf_w + static_cast<size_t>(n0 >> 7) * k64 * SF_CHUNK;
                for (int s = 0; s < n_stages; ++s) {
                    ok = mbar_wait<32>(empty(slot), ph ^ 1u, abortp, W_EMPTY);
                    if (!ok) break;
                    mbar_expect_tx(full(slot), tx);
                    tma_load_2d(smem_base + T::OFF_X + slot * T::X_BYTES, &tm_x, s * KSTAGE_BYTES, m0, full(slot));
                    tma_load_2d(smem_base + T::OFF_W + slot * T::W_BYTES, &tm_w, s * KSTAGE_BYTES, n0, full(slot));
                    bulk_load(smem_base + T::OFF_SFW + slot * T::SFW_BYTES, sfw_src + static_cast<size_t>(s) * T::SFW_BYTES,
                              T::SFW_BYTES, full(slot));
                    for (int a = 0; a < atoms; ++a)
                        bulk_load(smem_base + T::OFF_SFX + slot * T::SFX_BYTES + a * KSTEPS * SF_CHUNK,
                                  p.sf_x + (static_cast<size_t>((m0 >> 7) + a) * k64 + static_cast<size_t>(s) * KSTEPS) * SF_CHUNK,
                                  KSTEPS * SF_CHUNK, full(slot));
                    ++issued;
                    if (++slot == T::S) { slot = 0; ph ^= 1u; }
                }
            }
            if (!ok) {
                for (int i = max(0, issued - T::S); i < issued; ++i)
                    for (uint32_t it = 0; it < (1u << 16) && !mbar_try_wait(full(i % T::S), (i / T::S) & 1); ++it) {}
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ scale copies + MMA issue
        const bool leader = elect_one();
        const uint32_t idesc = idesc_nvfp4(BN, TT);
        bool ok = true;
        int slot = 0;
        uint32_t ph = 0, region = 0, tile_ph = 0;
        for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x) {
            // the accumulator is free once the epilogue has pulled the previous tile into registers
            ok = mbar_wait(acc_empty, tile_ph ^ 1u, abortp, W_ACC_EMPTY);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tcgen05_fence_after_sync();
            for (int s = 0; s < n_stages; ++s) {
                ok = mbar_wait(full(slot), ph, abortp, W_FULL);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                tcgen05_fence_after_sync();
                if (leader) {
                    const uint32_t sf_cols = tmem_base + TT + region * T::SF_COLS;
                    const uint32_t sfw_smem = smem_base + T::OFF_SFW + slot * T::SFW_BYTES;
                    const uint32_t sfx_smem = smem_base + T::OFF_SFX + slot * T::SFX_BYTES;
                    const uint64_t da = umma_desc_sw128(smem_base + T::OFF_W + slot * T::W_BYTES);
                    const uint64_t db = umma_desc_sw128(smem_base + T::OFF_X + slot * T::X_BYTES);
#pragma unroll
                    for (int j = 0; j < KSTEPS; ++j) {
                        const uint32_t t_sfw = sf_cols + j * 4;
                        const uint32_t t_sfx = sf_cols + KSTEPS * 4 + j * 4 * T::ATOMS;
                        tmem_cp_sf(t_sfw, sf_desc(sfw_smem + j * SF_CHUNK));
#pragma unroll
                        for (int a = 0; a < T::ATOMS; ++a)
                            tmem_cp_sf(t_sfx + a * 4, sf_desc(sfx_smem + (a * KSTEPS + j) * SF_CHUNK));
                        umma_nvfp4(tmem_base, da + 2u * j, db + 2u * j, idesc, t_sfw, t_sfx, (s > 0 || j > 0) ? 1u : 0u);
                    }
                    umma_commit(empty(slot));
                    if (s == n_stages - 1) umma_commit(acc_full);
                }
                __syncwarp();
                region ^= 1u;
                if (++slot == T::S) { slot = 0; ph ^= 1u; }
            }
            tile_ph ^= 1u;
        }
    } else if (warp >= 4) {
        // ------------------------------------------------------------------ epilogue
        constexpr int EC = T::EC;
        constexpr int SLAB = T::SLAB_TOK;
        const int q = warp & 3;
        const int h = (warp - 4) >> 2;
        const int ch_local = q * 32 + lane;
        const float sw = __ldg(p.tensor_scale);
        const uint32_t out0 = smem_base + T::OFF_OUT + h * T::SLAB_BYTES;    // this thread's slab
        bool ok = true;
        uint32_t tile_ph = 0;
        for (int tile = blockIdx.x; tile < total_tiles; tile += gridDim.x) {
            int tm, tn;
            tile_coords(tile, p.m_tiles, p.n_tiles, kGroupM, tm, tn);
            const int m0 = tm * TT;
            const int n0 = tn * BN;
            const int n = n0 + ch_local;
            const bool n_ok = n < p.N;
            const float b = (p.bias != nullptr && n_ok) ? __ldg(p.bias + n) : 0.0f;
            ok = mbar_wait<64>(acc_full, tile_ph, abortp, W_ACC_FULL);
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
            if (lane == 0) mbar_arrive(acc_empty);
#pragma unroll
            for (int phase = 0; phase < 2; ++phase) {
                // tokens [h EC + phase SLAB, + SLAB) of the tile go to slab h
#pragma unroll
                for (int j = 0; j < SLAB; j += 4) {
                    const int tok = h * EC + phase * SLAB + j;
                    float4 rs = make_float4(0.f, 0.f, 0.f, 0.f);
                    if (m0 + tok + 3 < p.M) {
                        rs = __ldg(reinterpret_cast<const float4*>(p.row_scale + m0 + tok));
                    } else {
                        if (m0 + tok + 0 < p.M) rs.x = __ldg(p.row_scale + m0 + tok + 0);
                        if (m0 + tok + 1 < p.M) rs.y = __ldg(p.row_scale + m0 + tok + 1);
                        if (m0 + tok + 2 < p.M) rs.z = __ldg(p.row_scale + m0 + tok + 2);
                    }
                    const float rr[4] = {__fmul_rn(rs.x, sw), __fmul_rn(rs.y, sw), __fmul_rn(rs.z, sw), __fmul_rn(rs.w, sw)};
                    if (ch_local < p.out_pitch) {
#pragma unroll
                        for (int t = 0; t < 4; ++t) {
                            const float acc = n_ok ? __uint_as_float(v[phase * SLAB + j + t]) : 0.0f;
                            const __nv_bfloat16 y = __float2bfloat16_rn(fmaf(acc, rr[t], b));
                            sts16(out0 + static_cast<uint32_t>((j + t) * p.out_pitch + ch_local) * 2u, __bfloat16_as_ushort(y));
                        }
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
                                         ::"l"(reinterpret_cast<uint64_t>(&tm_y)), "r"(smem_base + T::OFF_OUT + hh * T::SLAB_BYTES),
                                           "r"(n0), "r"(tok0) : "memory");
                    }
                    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                    asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");     // slabs may be overwritten again
                }
                asm volatile("bar.sync 1, %0;" ::"n"(EPI_THREADS) : "memory");
            }
        }
        (void)ok;
    }

    tcgen05_fence_before_sync();
    __syncthreads();
    if (warp == 1) {
        __syncwarp();
        tcgen05_fence_after_sync();
        tmem_dealloc(tmem_base, T::TMEM_COLS);
    }
}

}  // namespace fp4

template <int TT>
static cudaError_t launch_fp4_one(const GemmFp4Args& a, cudaStream_t st)
{
    using T = fp4::Tile<TT>;
    fp4::Params p;
    p.M = a.M; p.N = a.N; p.K = a.K;
    p.sf_x = a.sf_x; p.sf_w = a.sf_w;
    p.row_scale = a.row_scale; p.tensor_scale = a.tensor_scale; p.bias = a.bias;
    p.x_tx = static_cast<uint32_t>(min(TT, a.M)) * fp4::KSTAGE_BYTES;
    p.w_tx = static_cast<uint32_t>(min(fp4::BN, a.N)) * fp4::KSTAGE_BYTES;
    p.out_pitch = min(fp4::BN, a.N);
    p.m_atoms = (a.M + 127) / 128;
    p.m_tiles = (a.M + TT - 1) / TT;
    p.n_tiles = (a.N + fp4::BN - 1) / fp4::BN;
    const int tiles = p.m_tiles * p.n_tiles;
    const int grid = tiles < a.sm_count ? tiles : a.sm_count;
    return launch_early(fp4::gemm_nvfp4_kernel<TT>, grid, fp4::NUM_THREADS, T::DYN_SMEM, st, a.tm_x, a.tm_w, a.tm_y, p);
}

// 256-token tiles once they fill the device; smaller problems get twice the CTAs from 128-token tiles.
int gemm_fp4_token_tile(int M, int N)
{
    if (M <= 128) return 128;
    const long long tiles256 = static_cast<long long>((M + 255) / 256) * ((N + BN_FP4 - 1) / BN_FP4);
    return tiles256 >= device_sm_count() ? 256 : 128;
}
int gemm_fp4_store_rows(int M, int N) { return gemm_fp4_token_tile(M, N) / 4; }

cudaError_t gemm_fp4_init()
{
    cudaError_t e = cudaFuncSetAttribute(fp4::gemm_nvfp4_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, fp4::Tile<128>::DYN_SMEM);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(fp4::gemm_nvfp4_kernel<256>, cudaFuncAttributeMaxDynamicSharedMemorySize, fp4::Tile<256>::DYN_SMEM);
    if (e != cudaSuccess) return e;
    return gemm_fp4_pair_init();
}

cudaError_t launch_gemm_fp4(const GemmFp4Args& a, cudaStream_t st)
{
    if (gemm_fp4_use_pair(a.M, a.N, a.K)) return launch_gemm_fp4_pair(a, st);
    return gemm_fp4_token_tile(a.M, a.N) == 256 ? launch_fp4_one<256>(a, st) : launch_fp4_one<128>(a, st);
}

}  // namespace rudder
