// Second kernel of the engine (Section 4.4; Eq. 10) for a handful of tokens (action / proprio-only passes).
//
// With at most a few dozen tokens the layer is a stream of packed weights and what it costs is latency, not
// tensor throughput.  tcgen05.mma is the wrong tool here: its smallest tile has 64 / 128 operand rows on the
// M side, and the tensor core walks those rows at one row per clock whatever the other side holds, so a CTA
// with 16 tokens spends 4 clocks per input channel per 128 output channels (2.2 us for a 1024-channel slice,
// measured) on a product of 2 million multiply-adds; on top come TMEM allocation, shared-memory operand
// staging, an unpack stage and a split-K exchange between CTAs.  This kernel keeps everything in registers:
//
//   * a CTA owns 8 T output channels (T = 1, 2 or 4, so that the grid is about one CTA per SM) over ALL of K;
//     its 8 warps take 1/8 of K each (blocks of 64 input channels), so the only reduction is across the warps
//     of one CTA, through shared memory: no split-K scratch, no counters, no cluster.
//   * weights: each lane loads its 8 bytes (16 four-bit codes) per block and channel tile straight from the
//     packed array into registers -- BEFORE waiting for the prologue kernel (programmatic dependent launch):
//     the weight stream overlaps the kernel that quantises the activations.  The packed layout (byte b of a
//     16-byte run = channels b and 16 + b of a 32-channel run) is exactly the B fragment of
//     mma.sync.m16n8k32.s8: one shift and two masks per 8 weights, the nibble in the top half of the byte
//     (16 q; the factor is folded into the fp32 scales).  The sign-magnitude layout of the W4A4 group path is
//     turned into two's complement bytes with two byte permutes and a per-byte negate.
//   * activations: the int8 codes Q_X of the prologue kernel, 16 tokens x 64 channels per block, loaded as A
//     fragments straight from global memory (L2), all blocks of a chunk in flight at once.
//   * C^(g) = sum over the group of Q_X Q_W in INT32 in the MMA's accumulator registers (two MMAs per 64
//     channels); at the end of each weight group: fp32(C) * Delta_W[j,g] added into fp32 registers (Eq. 10
//     with group scales); then the warps' partial sums are added in warp order (deterministic), * r_i + b_j,
//     bf16.
// Tokens beyond 16 are taken in further passes of 16 over the same weight registers.
#include "internal.cuh"

#include <cuda_bf16.h>

namespace rudder {

namespace {

constexpr int FR_THREADS = 256;
constexpr int FR_WARPS = 8;
constexpr int FR_CHUNK = 8;            // 64-channel blocks whose weights and codes a warp holds in registers at once
constexpr int FR_MAX_M = 32;           // rows up to which this kernel is used (every further 16 rows are another pass: about 3 us)

struct FewRowsParams {
    const int8_t* codes; int64_t ldc;  // Q_X int8 [M, ldc]
    const float* row_scale;            // r [M]
    const uint8_t* wq;                 // packed weights [N, K/2]
    const float* scales_t;             // [K/G][N] fp32 = Delta_W / 16
    const float* bias;                 // [N] or nullptr
    uint16_t* Y; int64_t ldy;          // bf16 [M, ldy]
    int32_t* dump;                     // parity hook: INT32 group sums [K/G][rows][cols] (zeroed by the host), or nullptr
    int row0, rows, col0, cols;
    int M, N, K, G;
};

__device__ __forceinline__ void mma_s8(int (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k32.row.col.s32.s8.s8.s32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
                 : "+r"(c[0]), "+r"(c[1]), "+r"(c[2]), "+r"(c[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint2 ldg_nc_8(const void* p) {
    uint2 v;
    asm volatile("ld.global.nc.L1::no_allocate.v2.u32 {%0, %1}, [%2];" : "=r"(v.x), "=r"(v.y) : "l"(p));
    return v;
}
__device__ __forceinline__ uint2 ldg_cg_8(const void* p) {        // written by the kernel before this one: not through the read-only path
    uint2 v;
    asm volatile("ld.global.cg.v2.u32 {%0, %1}, [%2];" : "=r"(v.x), "=r"(v.y) : "l"(p));
    return v;
}
// One packed word (8 weights) -> the two B-fragment registers of one MMA step.
template <bool SIGNMAG>
__device__ __forceinline__ void b_frag(uint32_t pk, uint32_t& b0, uint32_t& b1) {
    if (SIGNMAG) {
        // magnitudes index a table of the bytes 0..7, the sign bits are spread to whole bytes and the byte is
        // negated where set (a negative code has magnitude >= 1, so the + 1 never carries into the next byte)
        const uint32_t t_lo = 0x03020100u, t_hi = 0x07060504u;
        uint32_t ma, mb;
        asm("prmt.b32 %0, %1, %2, %3;" : "=r"(ma) : "r"(t_lo), "r"(t_hi), "r"(pk & 0x7777u));
        asm("prmt.b32 %0, %1, %2, %3;" : "=r"(mb) : "r"(t_lo), "r"(t_hi), "r"((pk >> 16) & 0x7777u));
        const uint32_t sa = ((pk << 4) & 0x80808080u) >> 7, sb = (pk & 0x80808080u) >> 7;
        b0 = (ma ^ (sa * 0xFFu)) + sa;
        b1 = (mb ^ (sb * 0xFFu)) + sb;
    } else {
        b0 = (pk << 4) & 0xF0F0F0F0u;
        b1 = pk & 0xF0F0F0F0u;
    }
}

// T = channel tiles of 8 per warp (the CTA owns 8 T channels).
// G64: weight groups of 64 (every block ends a group: the block loop is branch-free and the compiler interleaves blocks).
template <int T, bool SIGNMAG, bool DUMP, bool G64>
__global__ void __launch_bounds__(FR_THREADS, 1)
gemm_i8_w4_fewrows_kernel(const FewRowsParams p)
{
    extern __shared__ float scales_s[];                    // [K/G][8 T] group scales of the CTA's channels
    __shared__ float red[FR_WARPS][16][8 * T + 2];         // the warps' partial sums of one pass of 16 tokens

    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const int tid = threadIdx.x;
    const int warp = tid >> 5, lane = tid & 31;
    const int g = lane >> 2, q = lane & 3;                 // fragment coordinates
    constexpr int NC = 8 * T;
    const int n0 = blockIdx.x * NC;
    const int n_groups_all = p.K / p.G;
    const int nblk = p.K >> 6;
    const int per = (nblk + FR_WARPS - 1) / FR_WARPS;
    const int b_begin = min(nblk, warp * per), b_end = min(nblk, b_begin + per);
    const int blk_per_group = G64 ? 1 : (p.G >> 6);
    const float sc_mul = SIGNMAG ? 16.0f : 1.0f;           // sign-magnitude weights are the integers themselves, not 16 x

    // ---- everything that belongs to the weights: before waiting for the prologue kernel
    for (int i = tid; i < n_groups_all * NC; i += FR_THREADS) {
        const int gg = i / NC, c = i - gg * NC;
        scales_s[i] = __ldg(p.scales_t + static_cast<size_t>(gg) * p.N + n0 + c) * sc_mul;
    }
    // byte offset of this lane's 8 weight bytes inside a 64-channel block of a channel row: run (q >> 1), words 2 (q & 1), + 1
    const uint32_t lane_off = 16u * (q >> 1) + 8u * (q & 1);
    const uint8_t* wrow[T];
#pragma unroll
    for (int t = 0; t < T; ++t) wrow[t] = p.wq + static_cast<size_t>(n0 + 8 * t + g) * (p.K >> 1) + lane_off;
    uint2 wreg[FR_CHUNK][T];
#pragma unroll
    for (int i = 0; i < FR_CHUNK; ++i) {
        const int blk = b_begin + i;
#pragma unroll
        for (int t = 0; t < T; ++t) wreg[i][t] = (blk < b_end) ? ldg_nc_8(wrow[t] + 32 * blk) : make_uint2(0, 0);
    }
    // this thread's output column in the reduction below (256 is a multiple of 8 T): its bias, requested now
    const int out_col = tid % NC, out_row0 = tid / NC;
    constexpr int OUT_ROWS_STEP = FR_THREADS / NC;          // rows out_row0, + step, ... < 16
    const float out_bias = (p.bias != nullptr) ? __ldg(p.bias + n0 + out_col) : 0.0f;
    asm volatile("griddepcontrol.wait;" ::: "memory");       // the codes and row scales come from the kernel before this one
    __syncthreads();                                        // scales_s

    const int n_pass = (p.M + 15) >> 4;
    for (int pass = 0; pass < n_pass; ++pass) {
        const int r0 = min(p.M - 1, pass * 16 + g), r1 = min(p.M - 1, pass * 16 + g + 8);     // rows past M repeat the last row (never stored)
        // this lane's 8 + 8 code bytes per row inside a block: bytes 32 (q >> 1) + 8 (q & 1) .. + 7 and the same + 16
        const int8_t* c0 = p.codes + static_cast<size_t>(r0) * p.ldc + 32 * (q >> 1) + 8 * (q & 1);
        const int8_t* c1 = p.codes + static_cast<size_t>(r1) * p.ldc + 32 * (q >> 1) + 8 * (q & 1);
        constexpr int N_OUT = (16 + OUT_ROWS_STEP - 1) / OUT_ROWS_STEP;
        float out_rs[N_OUT];                                // row scales of this thread's outputs, requested ahead of the MMAs
#pragma unroll
        for (int i = 0; i < N_OUT; ++i) {
            const int tok = pass * 16 + out_row0 + i * OUT_ROWS_STEP;
            out_rs[i] = (out_row0 + i * OUT_ROWS_STEP < 16 && tok < p.M) ? __ldcg(p.row_scale + tok) : 0.0f;
        }
        float acc[T][4];
#pragma unroll
        for (int t = 0; t < T; ++t) { acc[t][0] = acc[t][1] = acc[t][2] = acc[t][3] = 0.0f; }
        int C[T][4];
#pragma unroll
        for (int t = 0; t < T; ++t) { C[t][0] = C[t][1] = C[t][2] = C[t][3] = 0; }

        for (int cb = b_begin; cb < b_end; cb += FR_CHUNK) {
            if (cb != b_begin || pass != 0) {
                // weights of this chunk (the first chunk of the first pass is already in registers; K up to 4096 needs no other)
                if (cb != b_begin || b_end - b_begin > FR_CHUNK) {
#pragma unroll
                    for (int i = 0; i < FR_CHUNK; ++i) {
                        const int blk = cb + i;
#pragma unroll
                        for (int t = 0; t < T; ++t) wreg[i][t] = (blk < b_end) ? ldg_nc_8(wrow[t] + 32 * blk) : make_uint2(0, 0);
                    }
                }
            }
            uint2 a00[FR_CHUNK], a01[FR_CHUNK], a10[FR_CHUNK], a11[FR_CHUNK];     // [row half][k half]
#pragma unroll
            for (int i = 0; i < FR_CHUNK; ++i) {
                const int blk = min(cb + i, b_end - 1);
                a00[i] = ldg_cg_8(c0 + 64 * blk);
                a01[i] = ldg_cg_8(c0 + 64 * blk + 16);
                a10[i] = ldg_cg_8(c1 + 64 * blk);
                a11[i] = ldg_cg_8(c1 + 64 * blk + 16);
            }
#pragma unroll
            for (int i = 0; i < FR_CHUNK; ++i) {
                const int blk = cb + i;
                // (G64: a block past the end has zero weights and adds nothing; its group index is clamped)
                if (G64 || blk < b_end) {
#pragma unroll
                    for (int t = 0; t < T; ++t) {
                        uint32_t b0, b1;
                        b_frag<SIGNMAG>(wreg[i][t].x, b0, b1);
                        mma_s8(C[t], a00[i].x, a10[i].x, a01[i].x, a11[i].x, b0, b1);
                        b_frag<SIGNMAG>(wreg[i][t].y, b0, b1);
                        mma_s8(C[t], a00[i].y, a10[i].y, a01[i].y, a11[i].y, b0, b1);
                    }
                    // end of a weight group (or of this warp's share of it): Eq. 10's dequantisation of the group
                    if (G64 || (blk + 1) % blk_per_group == 0 || blk + 1 == b_end) {
                        const int grp = G64 ? min(blk, nblk - 1) : blk / blk_per_group;
                        const float* sc = scales_s + grp * NC + 2 * q;
#pragma unroll
                        for (int t = 0; t < T; ++t) {
                            const float s0 = sc[8 * t], s1 = sc[8 * t + 1];
                            acc[t][0] = fmaf(static_cast<float>(C[t][0]), s0, acc[t][0]);
                            acc[t][1] = fmaf(static_cast<float>(C[t][1]), s1, acc[t][1]);
                            acc[t][2] = fmaf(static_cast<float>(C[t][2]), s0, acc[t][2]);
                            acc[t][3] = fmaf(static_cast<float>(C[t][3]), s1, acc[t][3]);
                            if (DUMP && p.dump != nullptr) {
                                // (a group shared by several warps arrives in parts: integer adds, exact in any order)
#pragma unroll
                                for (int e = 0; e < 4; ++e) {
                                    const int tok = pass * 16 + g + ((e >> 1) << 3);
                                    const int rr = tok - p.row0, cc = n0 + 8 * t + 2 * q + (e & 1) - p.col0;
                                    if (blk < b_end && tok < p.M && rr >= 0 && rr < p.rows && cc >= 0 && cc < p.cols)
                                        atomicAdd(p.dump + (static_cast<size_t>(grp) * p.rows + rr) * p.cols + cc, SIGNMAG ? C[t][e] : (C[t][e] >> 4));
                                }
                            }
                            C[t][0] = C[t][1] = C[t][2] = C[t][3] = 0;
                        }
                    }
                }
            }
        }
        // ---- the warps' partial sums, added in warp order; row scale and bias (Eq. 10); bf16
#pragma unroll
        for (int t = 0; t < T; ++t) {
            *reinterpret_cast<float2*>(&red[warp][g][8 * t + 2 * q]) = make_float2(acc[t][0], acc[t][1]);
            *reinterpret_cast<float2*>(&red[warp][g + 8][8 * t + 2 * q]) = make_float2(acc[t][2], acc[t][3]);
        }
        __syncthreads();
#pragma unroll
        for (int i = 0; i < N_OUT; ++i) {
            const int row = out_row0 + i * OUT_ROWS_STEP;
            const int tok = pass * 16 + row;
            if (row < 16 && tok < p.M) {
                float sum = 0.0f;
#pragma unroll
                for (int w = 0; w < FR_WARPS; ++w) sum += red[w][row][out_col];
                p.Y[static_cast<size_t>(tok) * p.ldy + n0 + out_col] = __bfloat16_as_ushort(__float2bfloat16_rn(fmaf(sum, out_rs[i], out_bias)));
            }
        }
        __syncthreads();
    }
}

// Channel tiles per warp: the largest of 4, 2, 1 that still gives about one CTA per SM.
int fewrows_tiles(int N)
{
    const int sms = device_sm_count();
    int t = 4;
    while (t > 1 && N / (8 * t) < sms / 2) t >>= 1;
    return t;
}

}  // namespace

bool gemm_i8_fewrows_applies(int M, int N, int K, int G)
{
    return M >= 1 && M <= FR_MAX_M && K % 64 == 0 && N % 32 == 0 && G % 64 == 0 &&
           static_cast<size_t>(K / G) * 32 * sizeof(float) <= 96 * 1024;
}

template <int T, bool SIGNMAG, bool DUMP, bool G64>
static cudaError_t launch_fewrows(const GemmI8FewRowsArgs& a, cudaStream_t st)
{
    FewRowsParams p;
    p.codes = a.codes; p.ldc = a.ldc; p.row_scale = a.row_scale; p.wq = a.wq; p.scales_t = a.w_scales_t; p.bias = a.bias;
    p.Y = a.Y; p.ldy = a.ldy; p.dump = a.acc; p.row0 = a.row0; p.rows = a.rows; p.col0 = a.col0; p.cols = a.cols;
    p.M = a.M; p.N = a.N; p.K = a.K; p.G = a.G;
    const size_t smem = static_cast<size_t>(a.K / a.G) * 8 * T * sizeof(float);
    if (smem > 40 * 1024) {
        cudaError_t e = cudaFuncSetAttribute(gemm_i8_w4_fewrows_kernel<T, SIGNMAG, DUMP, G64>, cudaFuncAttributeMaxDynamicSharedMemorySize, 96 * 1024);
        if (e != cudaSuccess) return e;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(a.N / (8 * T), 1, 1);
    cfg.blockDim = dim3(FR_THREADS, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, gemm_i8_w4_fewrows_kernel<T, SIGNMAG, DUMP, G64>, p);
}

cudaError_t launch_gemm_i8_fewrows(const GemmI8FewRowsArgs& a, cudaStream_t st)
{
    const bool dump = a.acc != nullptr;
    if (dump) {
        // groups shared by several warps are added into the window by parts: it starts from zero
        cudaError_t e = cudaMemsetAsync(a.acc, 0, static_cast<size_t>(a.K / a.G) * a.rows * a.cols * sizeof(int32_t), st);
        if (e != cudaSuccess) return e;
    }
    const int t = fewrows_tiles(a.N);
#define RUDDER_FR_LAUNCH2(T, G64)                                                                                                 \
    return a.signmag ? (dump ? launch_fewrows<T, true, true, G64>(a, st) : launch_fewrows<T, true, false, G64>(a, st))            \
                     : (dump ? launch_fewrows<T, false, true, G64>(a, st) : launch_fewrows<T, false, false, G64>(a, st));
#define RUDDER_FR_LAUNCH(T) if (a.G == 64) { RUDDER_FR_LAUNCH2(T, true) } else { RUDDER_FR_LAUNCH2(T, false) }
    if (t == 4) { RUDDER_FR_LAUNCH(4) }
    if (t == 2) { RUDDER_FR_LAUNCH(2) }
    RUDDER_FR_LAUNCH(1)
#undef RUDDER_FR_LAUNCH2
#undef RUDDER_FR_LAUNCH
}

}  // namespace rudder
