// Offline weight preparation: fold the shared channel scaling D into W, quantise to INT4 per
// (output channel, group) and lay the codes out for the GEMM's unpack warps (Eq. 6; Section 4.2,
// last paragraph; Eq. 1 with k = 4).  Not on the hot path: clarity over speed.
#include "internal.cuh"

#include <cuda_fp16.h>

namespace rudder {

// One warp per (row j, group g).  V = W * d; Delta = fp16(amax / 7); q = clip(rint(V / Delta), +-7).
__global__ void pack_int4_quantize_kernel(const float* __restrict__ W, const float* __restrict__ d, int N, int K,
                                          int G, int8_t* __restrict__ q_out, float* __restrict__ scales_t,
                                          uint16_t* __restrict__ scales_c)
{
    const int n_groups = K / G;
    const long long warp = (static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (warp >= static_cast<long long>(N) * n_groups) return;
    const int j = static_cast<int>(warp / n_groups);
    const int g = static_cast<int>(warp % n_groups);
    const float* w = W + static_cast<size_t>(j) * K + static_cast<size_t>(g) * G;
    const float* dd = d ? d + static_cast<size_t>(g) * G : nullptr;

    float amax = 0.0f;
    for (int k = lane; k < G; k += 32) {
        const float v = __fmul_rn(w[k], dd ? dd[k] : 1.0f);
        amax = fmaxf(amax, fabsf(v));
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));

    const __half delta_h = __float2half_rn(__fdiv_rn(amax, 7.0f));
    const float delta = __half2float(delta_h);
    if (lane == 0) {
        scales_c[static_cast<size_t>(j) * n_groups + g] = __half_as_ushort(delta_h);
        scales_t[static_cast<size_t>(g) * N + j] = delta * 0.0625f;   // exact: power of two
    }
    int8_t* q = q_out + static_cast<size_t>(j) * K + static_cast<size_t>(g) * G;
    for (int k = lane; k < G; k += 32) {
        int c = 0;
        if (delta != 0.0f) {
            const float v = __fmul_rn(w[k], dd ? dd[k] : 1.0f);
            c = __float2int_rn(__fdiv_rn(v, delta));
            c = max(-7, min(7, c));
        }
        q[k] = static_cast<int8_t>(c);
    }
}

// codes_il[n][16 c + b] = nibble(q[n][32 c + b]) | nibble(q[n][32 c + 16 + b]) << 4
__global__ void pack_int4_interleave_kernel(const int8_t* __restrict__ q, int N, int K, uint8_t* __restrict__ codes_il)
{
    const size_t idx = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    const size_t total = static_cast<size_t>(N) * (K / 2);
    if (idx >= total) return;
    const size_t n = idx / (K / 2);
    const int byte = static_cast<int>(idx % (K / 2));
    const int c = byte >> 4, b = byte & 15;
    const int8_t lo = q[n * K + 32 * c + b];
    const int8_t hi = q[n * K + 32 * c + 16 + b];
    codes_il[idx] = static_cast<uint8_t>((lo & 0xF) | ((hi & 0xF) << 4));
}

// Layout for the FP8 tensor path (W4A4 with group scales): sign and magnitude apart, arranged so that the
// GEMM's unpack turns one 32-bit word into eight E4M3 bytes with two byte-permute look-ups.  Word j of
// the 16-byte piece c covers channels A_i = 32 c + 4 j + i and B_i = 32 c + 16 + 4 j + i (i = 0..3):
//   bits [4i, 4i+3)       |A_i|        bits [16+4i, 16+4i+3)   |B_i|
//   bit 3 + 8i            sign of A_i  bit 7 + 8i              sign of B_i
// (every sign sits in bit 3 of some nibble, which the look-up's selector masks away).
__device__ __forceinline__ uint32_t sm_word(const int8_t* qa, const int8_t* qb)
{
    uint32_t w = 0;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int a = qa[i], b = qb[i];
        w |= static_cast<uint32_t>(a < 0 ? -a : a) << (4 * i);
        w |= static_cast<uint32_t>(b < 0 ? -b : b) << (16 + 4 * i);
        w |= static_cast<uint32_t>(a < 0) << (3 + 8 * i);
        w |= static_cast<uint32_t>(b < 0) << (7 + 8 * i);
    }
    return w;
}
__global__ void pack_int4_signmag_kernel(const int8_t* __restrict__ q, int N, int K, uint32_t* __restrict__ codes_sm)
{
    const size_t idx = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x;      // one 32-bit word
    const size_t total = static_cast<size_t>(N) * (K / 8);
    if (idx >= total) return;
    const size_t n = idx / (K / 8);
    const int word = static_cast<int>(idx % (K / 8));
    const int c = word >> 2, j = word & 3;
    const int8_t* base = q + n * K + 32 * c + 4 * j;
    codes_sm[idx] = sm_word(base, base + 16);
}
__global__ void export_int4_signmag_kernel(const uint32_t* __restrict__ codes_sm, int N, int K, uint8_t* __restrict__ out)
{
    const size_t idx = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    const size_t total = static_cast<size_t>(N) * (K / 2);
    if (idx >= total) return;
    const size_t n = idx / (K / 2);
    const int k0 = static_cast<int>(idx % (K / 2)) * 2;
    uint8_t nib[2];
#pragma unroll
    for (int t = 0; t < 2; ++t) {
        const int k = k0 + t;
        const int c = k >> 5, p = k & 31;
        const int is_b = p >> 4, j = (p & 15) >> 2, i = p & 3;
        const uint32_t w = codes_sm[n * (K / 8) + 4 * c + j];
        const int mag = static_cast<int>((w >> (16 * is_b + 4 * i)) & 7u);
        const int neg = static_cast<int>((w >> ((is_b ? 7 : 3) + 8 * i)) & 1u);
        nib[t] = static_cast<uint8_t>((neg ? -mag : mag) & 0xF);
    }
    out[idx] = static_cast<uint8_t>(nib[0] | (nib[1] << 4));
}

__global__ void dinv_kernel(const float* __restrict__ d, int K, float* __restrict__ dinv)
{
    const int k = blockIdx.x * blockDim.x + threadIdx.x;
    if (k < K) dinv[k] = __fdiv_rn(1.0f, d ? d[k] : 1.0f);
}

// canonical[n][k/2] = nibble(q[n][k]) | nibble(q[n][k+1]) << 4   (k even), read back from codes_il
__global__ void export_int4_kernel(const uint8_t* __restrict__ codes_il, int N, int K, uint8_t* __restrict__ out)
{
    const size_t idx = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    const size_t total = static_cast<size_t>(N) * (K / 2);
    if (idx >= total) return;
    const size_t n = idx / (K / 2);
    const int k0 = static_cast<int>(idx % (K / 2)) * 2;
    uint8_t nib[2];
#pragma unroll
    for (int t = 0; t < 2; ++t) {
        const int k = k0 + t;
        const int c = k >> 5, p = k & 31;
        const uint8_t byte = codes_il[n * (K / 2) + 16 * c + (p & 15)];
        nib[t] = (p < 16) ? (byte & 0xF) : (byte >> 4);
    }
    out[idx] = static_cast<uint8_t>(nib[0] | (nib[1] << 4));
}

cudaError_t launch_pack_int4(const float* W, const float* d, int N, int K, int G, uint8_t* codes_il,
                             float* scales_t, uint16_t* scales_c, float* dinv, int8_t* tmp_codes, bool signmag,
                             cudaStream_t st)
{
    const long long warps = static_cast<long long>(N) * (K / G);
    const int threads = 256;
    const long long blocks = (warps * 32 + threads - 1) / threads;
    pack_int4_quantize_kernel<<<static_cast<unsigned>(blocks), threads, 0, st>>>(W, d, N, K, G, tmp_codes, scales_t, scales_c);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    const size_t total = static_cast<size_t>(N) * (K / 2);
    if (signmag)
        pack_int4_signmag_kernel<<<static_cast<unsigned>((total / 4 + 255) / 256), 256, 0, st>>>(tmp_codes, N, K, reinterpret_cast<uint32_t*>(codes_il));
    else
        pack_int4_interleave_kernel<<<static_cast<unsigned>((total + 255) / 256), 256, 0, st>>>(tmp_codes, N, K, codes_il);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    dinv_kernel<<<(K + 255) / 256, 256, 0, st>>>(d, K, dinv);
    return cudaGetLastError();
}

// ---- import of a canonical packed weight (the layout rudder_weight_export writes) -------------------
// canonical nibbles [N, K/2] (low nibble = even k, two's complement) -> one int8 code per byte [N, K]
__global__ void import_int4_expand_kernel(const uint8_t* __restrict__ canonical, size_t total, int8_t* __restrict__ q)
{
    const size_t idx = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (idx >= total) return;
    const uint8_t b = canonical[idx];
    const int lo = b & 0xF, hi = b >> 4;
    q[2 * idx] = static_cast<int8_t>(lo > 7 ? lo - 16 : lo);
    q[2 * idx + 1] = static_cast<int8_t>(hi > 7 ? hi - 16 : hi);
}
// fp16 scales [N, K/G] -> the GEMM's fp32 [K/G, N] = Delta_W / 16
__global__ void import_scales_kernel(const uint16_t* __restrict__ scales_c, int N, int n_groups, float* __restrict__ scales_t)
{
    const size_t idx = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (idx >= static_cast<size_t>(N) * n_groups) return;
    const int j = static_cast<int>(idx / n_groups), g = static_cast<int>(idx % n_groups);
    scales_t[static_cast<size_t>(g) * N + j] = __half2float(__ushort_as_half(scales_c[idx])) * 0.0625f;
}

cudaError_t launch_import_int4(const uint8_t* canonical, const uint16_t* scales_c, int N, int K, int G, uint8_t* codes_il,
                               float* scales_t, int8_t* tmp_codes, bool signmag, cudaStream_t st)
{
    const size_t total = static_cast<size_t>(N) * (K / 2);
    import_int4_expand_kernel<<<static_cast<unsigned>((total + 255) / 256), 256, 0, st>>>(canonical, total, tmp_codes);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    if (signmag)
        pack_int4_signmag_kernel<<<static_cast<unsigned>((total / 4 + 255) / 256), 256, 0, st>>>(tmp_codes, N, K, reinterpret_cast<uint32_t*>(codes_il));
    else
        pack_int4_interleave_kernel<<<static_cast<unsigned>((total + 255) / 256), 256, 0, st>>>(tmp_codes, N, K, codes_il);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    const size_t ns = static_cast<size_t>(N) * (K / G);
    import_scales_kernel<<<static_cast<unsigned>((ns + 255) / 256), 256, 0, st>>>(scales_c, N, K / G, scales_t);
    return cudaGetLastError();
}

cudaError_t launch_export_int4(const uint8_t* codes_il, int N, int K, uint8_t* canonical, bool signmag, cudaStream_t st)
{
    const size_t total = static_cast<size_t>(N) * (K / 2);
    if (signmag)
        export_int4_signmag_kernel<<<static_cast<unsigned>((total + 255) / 256), 256, 0, st>>>(reinterpret_cast<const uint32_t*>(codes_il), N, K, canonical);
    else
    export_int4_kernel<<<static_cast<unsigned>((total + 255) / 256), 256, 0, st>>>(codes_il, N, K, canonical);
    return cudaGetLastError();
}

}  // namespace rudder
