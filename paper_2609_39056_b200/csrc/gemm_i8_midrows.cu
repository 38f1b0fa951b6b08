// Second kernel of the engine (Section 4.4; Eq. 10) for a few dozen to a few hundred tokens.
//
// Between the few-rows kernel (everything in one warp's registers) and the tcgen05 kernel (256-token
// tiles, accumulators in tensor memory) lies a range where neither fits: a tcgen05.mma with 128 weight
// rows on its M side costs about the same issue time whatever the token count, so 64-token tiles leave
// the kernel bound by MMA issue (measured: about 110 clocks per instruction that holds 32 clocks of
// math), while wider tiles move the bound to the per-group drain of tensor memory.  Here the per-group
// INT32 sums stay in registers, as Eq. 10 with group scales wants them:
//
//   * a CTA of 8 (or 4) warps owns BM tokens x BN output channels over all of K; a warp owns 32 tokens x
//     8 NT channels (two m16 tiles x NT n8 tiles of mma.sync.m16n8k32.s8);
//   * codes Q_X (int8, from the prologue kernel) and packed 4-bit weights are staged through a ring of
//     shared-memory stages of 256 input channels by 16-byte cp.async copies; the weight copies of the
//     first stages and the group scales of the CTA's channels are requested BEFORE waiting for the
//     prologue kernel (programmatic dependent launch);
//   * fragments are 8-byte shared-memory loads in the layout the few-rows kernel uses (the packed weight
//     word is the B fragment: one shift and two masks; sign-magnitude layout: two byte permutes and a
//     per-byte negate); both tiles are stored with their 16-byte pieces permuted by row so that the loads
//     of a half warp fall into 16 different bank pairs;
//   * at the end of each weight group (64 channels): fp32(C) * Delta_W[j,g] added into fp32 registers; the
//     next group starts from a zero accumulator in a second set of registers, so that the conversions of one
//     group run under the MMAs of the next; at the end of K: * r_i + b_j, bf16.  No tensor memory, no split K,
//     no scratch.
#include "internal.cuh"

#include <cuda_bf16.h>

namespace rudder {

namespace {

constexpr int MR_KS = 256;             // input channels per stage (128 measured 5-9 % slower: twice the barriers)
// Stages in the ring: what is in flight per SM has to cover an L2 round trip per stage, so as many as fit.
__host__ __device__ constexpr int mr_stages(int wm) { return wm == 4 ? 4 : 6; }
constexpr int MR_MAX_M = 512;          // rows up to which this kernel is considered
constexpr int MR_MAX_K = 4096;         // and row length

struct MidRowsParams {
    const int8_t* codes; int64_t ldc;  // Q_X int8 [M, ldc]
    const float* row_scale;            // r [M]
    const uint8_t* wq;                 // packed weights [N, K/2]
    const float* scales_t;             // [K/G][N] fp32 = Delta_W / 16
    const float* bias;                 // [N] or nullptr
    uint16_t* Y; int64_t ldy;          // bf16 [M, ldy]
    int32_t* dump;                     // parity hook: INT32 group sums [K/G][rows][cols], or nullptr
    int row0, rows, col0, cols;
    int M, N, K, G;
};

__device__ __forceinline__ void mr_mma_s8(int (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
    asm("mma.sync.aligned.m16n8k32.row.col.s32.s8.s8.s32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
        : "+r"(c[0]), "+r"(c[1]), "+r"(c[2]), "+r"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
// the first MMA of a weight group starts from zero: no registers to clear
__device__ __forceinline__ void mr_mma_s8_first(int (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
    asm("mma.sync.aligned.m16n8k32.row.col.s32.s8.s8.s32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%10, %10, %10, %10};"
        : "=r"(c[0]), "=r"(c[1]), "=r"(c[2]), "=r"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1), "r"(0));
}
__device__ __forceinline__ void mr_cp16(uint32_t dst, const void* src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void mr_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void mr_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ uint2 mr_lds8(uint32_t addr) {
    uint2 v;
    asm volatile("ld.shared.v2.u32 {%0, %1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"(addr));
    return v;
}
// One packed word (8 weights) -> the two B-fragment registers of one MMA step (see the few-rows kernel).
template <bool SIGNMAG>
__device__ __forceinline__ void mr_b_frag(uint32_t pk, uint32_t& b0, uint32_t& b1) {
    if (SIGNMAG) {
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
// Permutation of the 16-byte pieces of a code row (16 pieces per stage; bits 0 and 2 of the piece index) and of
// a weight row (8 pieces per stage), each a function of the row so that the fragment loads of a half warp (four
// rows x four lanes, 8 bytes each) cover 16 different bank pairs.
__device__ __forceinline__ uint32_t mr_swz_a(uint32_t row) { return (row & 1u) | ((row & 2u) << 1); }
__device__ __forceinline__ uint32_t mr_swz_b(uint32_t row) { return (row & 3u) << 1; }

// WM = warps along the tokens (32 each), NW / WM warps along the channels, NT = n8 tiles per warp:
// the CTA owns BM = 32 WM tokens x BN = 8 NT (NW / WM) channels.  Weight groups of 64 only: every 64-channel
// block is a group.  (A second set of 8 warps per CTA that takes every other stage -- the loop is bound by
// latency, and the small shapes have the registers -- measured 10 % slower: the barrier per stage grows.)
template <int WM, int NT, int NW, bool SIGNMAG, bool DUMP>
__global__ void __launch_bounds__(32 * NW, 1)
gemm_i8_w4_midrows_kernel(const MidRowsParams p)
{
    constexpr int NTHR = 32 * NW;
    constexpr int WNW = NW / WM;
    constexpr int BM = 32 * WM;
    constexpr int BN = 8 * NT * WNW;
    constexpr int A_BYTES = BM * MR_KS;            // codes of one stage
    constexpr int B_BYTES = BN * MR_KS / 2;        // packed weights of one stage
    constexpr int A_PIECES = BM * (MR_KS / 16) / NTHR;        // 16-byte pieces per thread and stage
    constexpr int B_ALL = BN * (MR_KS / 32);       // 16-byte weight pieces per stage
    constexpr int B_PIECES = (B_ALL + NTHR - 1) / NTHR;
    constexpr int MR_NST = mr_stages(WM);
    static_assert(A_PIECES >= 1, "copy assignment");
    extern __shared__ __align__(128) uint8_t mr_smem[];

    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const int tid = threadIdx.x;
    const int warp = tid >> 5, lane = tid & 31;
    const int g = lane >> 2, q = lane & 3;
    const int wm = warp % WM, wn = warp / WM;
    const int n0 = blockIdx.x * BN;
    const int m0 = blockIdx.y * BM;
    const int n_stages = p.K / MR_KS;
    const int n_groups = p.K >> 6;
    const uint32_t smem0 = smem_u32(mr_smem);
    const uint32_t a_base = smem0;
    const uint32_t b_base = smem0 + MR_NST * A_BYTES;
    float* scales_s = reinterpret_cast<float*>(mr_smem + MR_NST * (A_BYTES + B_BYTES));     // [K/64][BN]
    const float sc_mul = SIGNMAG ? 16.0f : 1.0f;   // sign-magnitude weights are the integers themselves, not 16 x

    // ---- what belongs to the weights: before waiting for the prologue kernel
    constexpr int BPR = MR_KS / 32;                // weight pieces per channel row
    const uint8_t* b_src[B_PIECES];
    uint32_t b_dst[B_PIECES];
    bool b_on[B_PIECES];
#pragma unroll
    for (int i = 0; i < B_PIECES; ++i) {
        const int id = i * NTHR + tid;
        b_on[i] = id < B_ALL;
        const int row = b_on[i] ? id / BPR : 0, c = id % BPR;
        b_src[i] = p.wq + static_cast<size_t>(n0 + row) * (p.K >> 1) + c * 16;
        b_dst[i] = static_cast<uint32_t>(row) * (MR_KS / 2) + ((static_cast<uint32_t>(c) ^ mr_swz_b(row)) << 4);
    }
    auto load_b = [&](int ks) {
#pragma unroll
        for (int i = 0; i < B_PIECES; ++i)
            if (b_on[i]) mr_cp16(b_base + (ks % MR_NST) * B_BYTES + b_dst[i], b_src[i] + static_cast<size_t>(ks) * (MR_KS / 2));
    };
    for (int ks = 0; ks < MR_NST - 1 && ks < n_stages; ++ks) load_b(ks);
    for (int i = tid; i < n_groups * BN; i += NTHR) {
        const int gg = i / BN, c = i - gg * BN;
        scales_s[i] = __ldg(p.scales_t + static_cast<size_t>(gg) * p.N + n0 + c) * sc_mul;
    }
    const int8_t* a_src[A_PIECES];
    uint32_t a_dst[A_PIECES];
#pragma unroll
    for (int i = 0; i < A_PIECES; ++i) {
        const int id = i * NTHR + tid;
        const int row = id / (MR_KS / 16), c = id % (MR_KS / 16);
        const int tok = min(m0 + row, p.M - 1);    // rows past M repeat the last row (never stored)
        a_src[i] = p.codes + static_cast<size_t>(tok) * p.ldc + c * 16;
        a_dst[i] = static_cast<uint32_t>(row) * MR_KS + ((static_cast<uint32_t>(c) ^ mr_swz_a(row)) << 4);
    }
    auto load_a = [&](int ks) {
#pragma unroll
        for (int i = 0; i < A_PIECES; ++i) mr_cp16(a_base + (ks % MR_NST) * A_BYTES + a_dst[i], a_src[i] + static_cast<size_t>(ks) * MR_KS);
    };
    asm volatile("griddepcontrol.wait;" ::: "memory");       // the codes and row scales come from the kernel before this one
    for (int ks = 0; ks < MR_NST - 1; ++ks) {
        if (ks < n_stages) load_a(ks);
        mr_commit();                                         // one group per stage, empty ones included
    }

    // fragment addresses inside a stage (without the 64-channel block's piece offset, which is XORed in below)
    const uint32_t swa = mr_swz_a(g), swb = mr_swz_b(g);
    const uint32_t a_row0 = static_cast<uint32_t>(wm * 32 + g) * MR_KS + 8u * (q & 1);
    const uint32_t b_row0 = static_cast<uint32_t>(wn * 8 * NT + g) * (MR_KS / 2) + 8u * (q & 1);
    // Two sets of INT32 sums alternate between the two blocks of a stage, and a group is dequantised after
    // the MMAs of the NEXT block have been issued: its own MMAs have long finished by then, so neither the
    // conversions wait for the tensor pipe nor the next MMAs for the conversions.
    // With fewer than four channel tiles per warp the two MMA steps of a block get accumulators of their own
    // (added at the group's end): otherwise the second step would wait out the first one's latency every time.
    constexpr int NS = (NT < 4) ? 2 : 1;
    int C[2][NS][2][NT][4];
    float acc[2][NT][4];
#pragma unroll
    for (int mt = 0; mt < 2; ++mt)
#pragma unroll
        for (int t = 0; t < NT; ++t)
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                acc[mt][t][e] = 0.0f;
#pragma unroll
                for (int cs = 0; cs < 2; ++cs)
#pragma unroll
                    for (int st = 0; st < NS; ++st) C[cs][st][mt][t][e] = 0;
            }
    auto dequant = [&](int (&Cs)[NS][2][NT][4], int grp) {       // Eq. 10's dequantisation of one weight group
        const float* sc = scales_s + grp * BN + wn * 8 * NT + 2 * q;
#pragma unroll
        for (int t = 0; t < NT; ++t) {
            const float2 s = *reinterpret_cast<const float2*>(sc + 8 * t);
#pragma unroll
            for (int mt = 0; mt < 2; ++mt) {
                int cv[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) cv[e] = (NS == 2) ? Cs[0][mt][t][e] + Cs[NS - 1][mt][t][e] : Cs[0][mt][t][e];
                acc[mt][t][0] = fmaf(static_cast<float>(cv[0]), s.x, acc[mt][t][0]);
                acc[mt][t][1] = fmaf(static_cast<float>(cv[1]), s.y, acc[mt][t][1]);
                acc[mt][t][2] = fmaf(static_cast<float>(cv[2]), s.x, acc[mt][t][2]);
                acc[mt][t][3] = fmaf(static_cast<float>(cv[3]), s.y, acc[mt][t][3]);
                if (DUMP && p.dump != nullptr) {
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const int tok = m0 + wm * 32 + mt * 16 + g + ((e >> 1) << 3);
                        const int rr = tok - p.row0, cc = n0 + wn * 8 * NT + 8 * t + 2 * q + (e & 1) - p.col0;
                        if (tok < p.M && rr >= 0 && rr < p.rows && cc >= 0 && cc < p.cols)
                            p.dump[(static_cast<size_t>(grp) * p.rows + rr) * p.cols + cc] = SIGNMAG ? cv[e] : (cv[e] >> 4);
                    }
                }
            }
        }
    };
    // the MMAs of one 64-channel block (= one weight group) of the stage at (a_st, b_st) into Cs, starting from zero
    auto block_mmas = [&](uint32_t a_st, uint32_t b_st, int blk, int (&Cs)[NS][2][NT][4]) {
        const uint32_t ca = static_cast<uint32_t>(blk * 4 + 2 * (q >> 1));       // 16-byte piece of the low half of this lane's codes
        const uint32_t cb = static_cast<uint32_t>(blk * 2 + (q >> 1));
        uint2 a00[2], a01[2], a10[2], a11[2];
#pragma unroll
        for (int mt = 0; mt < 2; ++mt) {
            const uint32_t r = a_st + mt * 16 * MR_KS;
            a00[mt] = mr_lds8(r + ((ca ^ swa) << 4));
            a01[mt] = mr_lds8(r + (((ca + 1) ^ swa) << 4));
            a10[mt] = mr_lds8(r + 8 * MR_KS + ((ca ^ swa) << 4));
            a11[mt] = mr_lds8(r + 8 * MR_KS + (((ca + 1) ^ swa) << 4));
        }
        uint2 w[NT];
#pragma unroll
        for (int t = 0; t < NT; ++t) w[t] = mr_lds8(b_st + t * 8 * (MR_KS / 2) + ((cb ^ swb) << 4));
        // first MMA step of every tile, then the second: consecutive MMAs never share an accumulator
#pragma unroll
        for (int t = 0; t < NT; ++t) {
            uint32_t b0, b1;
            mr_b_frag<SIGNMAG>(w[t].x, b0, b1);
#pragma unroll
            for (int mt = 0; mt < 2; ++mt) mr_mma_s8_first(Cs[0][mt][t], a00[mt].x, a10[mt].x, a01[mt].x, a11[mt].x, b0, b1);
        }
#pragma unroll
        for (int t = 0; t < NT; ++t) {
            uint32_t b0, b1;
            mr_b_frag<SIGNMAG>(w[t].y, b0, b1);
#pragma unroll
            for (int mt = 0; mt < 2; ++mt) {
                if (NS == 2) mr_mma_s8_first(Cs[NS - 1][mt][t], a00[mt].y, a10[mt].y, a01[mt].y, a11[mt].y, b0, b1);
                else         mr_mma_s8(Cs[NS - 1][mt][t], a00[mt].y, a10[mt].y, a01[mt].y, a11[mt].y, b0, b1);
            }
        }
    };

    for (int ks = 0; ks < n_stages; ++ks) {
        mr_wait<MR_NST - 2>();                               // this thread's copies of stage ks have landed
        __syncthreads();                                     // everybody's have; everybody is done with stage ks - 1
        if (ks + MR_NST - 1 < n_stages) { load_a(ks + MR_NST - 1); load_b(ks + MR_NST - 1); }
        mr_commit();
        const uint32_t a_st = a_base + (ks % MR_NST) * A_BYTES + a_row0;
        const uint32_t b_st = b_base + (ks % MR_NST) * B_BYTES + b_row0;
        constexpr int BPS = MR_KS / 64;                      // blocks (= weight groups) per stage
#pragma unroll
        for (int blk = 0; blk < BPS; ++blk) {
            block_mmas(a_st, b_st, blk, C[blk & 1]);
            if (ks > 0 || blk > 0) dequant(C[(blk & 1) ^ 1], ks * BPS + blk - 1);
        }
    }
    dequant(C[1], n_groups - 1);
    mr_wait<0>();
    // ---- row scale and bias (Eq. 10), bf16: a lane holds two adjacent channels of rows g and g + 8 per tile
    const bool pair_ok = ((p.ldy & 1) == 0) && ((reinterpret_cast<uintptr_t>(p.Y) & 3u) == 0);      // both channels in one 4-byte store
#pragma unroll
    for (int mt = 0; mt < 2; ++mt) {
        const int tok0 = m0 + wm * 32 + mt * 16 + g, tok1 = tok0 + 8;
        const float rs0 = tok0 < p.M ? __ldcg(p.row_scale + tok0) : 0.0f;
        const float rs1 = tok1 < p.M ? __ldcg(p.row_scale + tok1) : 0.0f;
#pragma unroll
        for (int t = 0; t < NT; ++t) {
            const int col = n0 + wn * 8 * NT + 8 * t + 2 * q;
            const float bx = p.bias != nullptr ? __ldg(p.bias + col) : 0.0f;
            const float by = p.bias != nullptr ? __ldg(p.bias + col + 1) : 0.0f;
#pragma unroll
            for (int hh = 0; hh < 2; ++hh) {
                const int tok = hh ? tok1 : tok0;
                if (tok >= p.M) continue;
                const float rs = hh ? rs1 : rs0;
                const __nv_bfloat16 y0 = __float2bfloat16_rn(fmaf(acc[mt][t][2 * hh], rs, bx));
                const __nv_bfloat16 y1 = __float2bfloat16_rn(fmaf(acc[mt][t][2 * hh + 1], rs, by));
                uint16_t* dst = p.Y + static_cast<size_t>(tok) * p.ldy + col;
                if (pair_ok) *reinterpret_cast<uint32_t*>(dst) = static_cast<uint32_t>(__bfloat16_as_ushort(y0)) | (static_cast<uint32_t>(__bfloat16_as_ushort(y1)) << 16);
                else { dst[0] = __bfloat16_as_ushort(y0); dst[1] = __bfloat16_as_ushort(y1); }
            }
        }
    }
}

}  // namespace

// Tile shapes, largest first: {warps along the tokens, n8 tiles per warp, warps} -> BM = 32 WM,
// BN = 8 NT (warps / WM).  The largest shape that still gives at least 0.6 CTAs per SM; failing that the one
// with the most CTAs (the last one, 64 x 16 with four warps, is there for the smallest layers).  Returns the
// number of CTAs.
constexpr int kMidShapes[4][3] = {{4, 4, 8}, {2, 2, 8}, {2, 1, 8}, {2, 1, 4}};
static long long midrows_shape(int M, int N, int& idx)
{
    const int sms = device_sm_count();
    long long best = -1;
    idx = 3;
    for (int i = 0; i < 4; ++i) {
        const int bm = 32 * kMidShapes[i][0], bn = 8 * kMidShapes[i][1] * (kMidShapes[i][2] / kMidShapes[i][0]);
        if (N % bn != 0 || (i == 0 && M <= 64)) continue;
        const long long ctas = static_cast<long long>((M + bm - 1) / bm) * (N / bn);
        if (ctas > sms) continue;
        if (ctas * 10 >= 6LL * sms) { idx = i; return ctas; }
        if (ctas > best) { best = ctas; idx = i; }
    }
    return best;
}
static size_t midrows_smem(int wm, int nt, int nw, int K)
{
    const int bm = 32 * wm, bn = 8 * nt * (nw / wm);
    return static_cast<size_t>(mr_stages(wm)) * (bm * MR_KS + bn * MR_KS / 2) + static_cast<size_t>(K / 64) * bn * sizeof(float);
}

// Where this kernel is the faster one (measured against the tcgen05 kernel with 64-token tiles and split K):
// weight groups of 64, rows of up to 4096 channels (8192: slower), one wave of CTAs, and little work in all --
// its MMAs run at the legacy rate, so beyond about 2 GOP (1.2 with the costlier sign-magnitude fragments) the
// tensor-memory kernel wins again (level at 4 GOP).
bool gemm_i8_midrows_applies(int M, int N, int K, int G, bool signmag)
{
    if (!(M > 32 && M <= MR_MAX_M && K % MR_KS == 0 && N % 64 == 0 && G == 64 && K <= MR_MAX_K)) return false;
    if (2.0 * M * N * K > (signmag ? 1.2e9 : 2.2e9)) return false;
    int idx;
    const long long ctas = midrows_shape(M, N, idx);
    return ctas > 0 && midrows_smem(kMidShapes[idx][0], kMidShapes[idx][1], kMidShapes[idx][2], K) <= 220 * 1024;
}

template <int WM, int NT, int NW, bool SIGNMAG, bool DUMP>
static cudaError_t launch_midrows(const GemmI8FewRowsArgs& a, cudaStream_t st)
{
    MidRowsParams p;
    p.codes = a.codes; p.ldc = a.ldc; p.row_scale = a.row_scale; p.wq = a.wq; p.scales_t = a.w_scales_t; p.bias = a.bias;
    p.Y = a.Y; p.ldy = a.ldy; p.dump = a.acc; p.row0 = a.row0; p.rows = a.rows; p.col0 = a.col0; p.cols = a.cols;
    p.M = a.M; p.N = a.N; p.K = a.K; p.G = a.G;
    constexpr int BM = 32 * WM, BN = 8 * NT * (NW / WM);
    const size_t smem = midrows_smem(WM, NT, NW, a.K);
    cudaError_t e = cudaFuncSetAttribute(gemm_i8_w4_midrows_kernel<WM, NT, NW, SIGNMAG, DUMP>, cudaFuncAttributeMaxDynamicSharedMemorySize, 220 * 1024);
    if (e != cudaSuccess) return e;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(a.N / BN, (a.M + BM - 1) / BM, 1);
    cfg.blockDim = dim3(32 * NW, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, gemm_i8_w4_midrows_kernel<WM, NT, NW, SIGNMAG, DUMP>, p);
}

cudaError_t launch_gemm_i8_midrows(const GemmI8FewRowsArgs& a, cudaStream_t st)
{
    const bool dump = a.acc != nullptr;
    int idx;
    midrows_shape(a.M, a.N, idx);
#define RUDDER_MR_LAUNCH(WM, NT, NW)                                                                                              \
    return a.signmag ? (dump ? launch_midrows<WM, NT, NW, true, true>(a, st) : launch_midrows<WM, NT, NW, true, false>(a, st))    \
                     : (dump ? launch_midrows<WM, NT, NW, false, true>(a, st) : launch_midrows<WM, NT, NW, false, false>(a, st));
    if (idx == 0) { RUDDER_MR_LAUNCH(4, 4, 8) }
    if (idx == 1) { RUDDER_MR_LAUNCH(2, 2, 8) }
    if (idx == 2) { RUDDER_MR_LAUNCH(2, 1, 8) }
    RUDDER_MR_LAUNCH(2, 1, 4)
#undef RUDDER_MR_LAUNCH
}

}  // namespace rudder
