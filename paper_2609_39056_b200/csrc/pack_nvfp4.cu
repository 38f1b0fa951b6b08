// Offline weight preparation, NVFP4 variant: V = W diag(d); one fp32 scale for the tensor
// (max|V| / 2688), one UE4M3 scale per 16 input channels, E2M1 codes.  The paper only names the
// format; the recipe is the one stated in the design notes.  Not on the hot path.
#include "internal.cuh"
#include "fp4.cuh"

namespace rudder {

__global__ void nvfp4_absmax_kernel(const float* __restrict__ W, const float* __restrict__ d, int N, int K,
                                    unsigned int* __restrict__ amax_bits)
{
    const size_t total = static_cast<size_t>(N) * K;
    float m = 0.0f;
    for (size_t i = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x; i < total; i += static_cast<size_t>(gridDim.x) * blockDim.x)
        m = fmaxf(m, fabsf(__fmul_rn(W[i], d ? d[i % K] : 1.0f)));
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    if ((threadIdx.x & 31) == 0) atomicMax(amax_bits, __float_as_uint(m));   // non-negative floats order like their bits
}

// One thread per (row, block of 16).
__global__ void nvfp4_quantize_kernel(const float* __restrict__ W, const float* __restrict__ d, int N, int K,
                                      const unsigned int* __restrict__ amax_bits, uint8_t* __restrict__ codes,
                                      uint8_t* __restrict__ sb_canonical, uint8_t* __restrict__ sf_tiled,
                                      float* __restrict__ tensor_scale)
{
    const int n_blocks = K / 16;
    const size_t idx = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    const float tmax = __uint_as_float(*amax_bits);
    if (idx == 0) *tensor_scale = __fdiv_rn(tmax, kNvfp4Range);
    if (idx >= static_cast<size_t>(N) * n_blocks) return;
    const int j = static_cast<int>(idx / n_blocks), b = static_cast<int>(idx % n_blocks);
    const float inv = (tmax != 0.0f) ? __fdiv_rn(kNvfp4Range, tmax) : 0.0f;
    float u[16];
#pragma unroll
    for (int t = 0; t < 16; ++t) {
        const int k = b * 16 + t;
        u[t] = __fmul_rn(__fmul_rn(W[static_cast<size_t>(j) * K + k], d ? d[k] : 1.0f), inv);
    }
    uint32_t lo, hi;
    const uint32_t sb = nvfp4_encode_block(u, lo, hi);
    *reinterpret_cast<uint2*>(codes + static_cast<size_t>(j) * (K / 2) + b * 8) = make_uint2(lo, hi);
    sb_canonical[static_cast<size_t>(j) * n_blocks + b] = static_cast<uint8_t>(sb);
    sf_tiled[nvfp4_sf_offset(j, b, K / 64)] = static_cast<uint8_t>(sb);
}

// Import: row-major UE4M3 block scales [N, K/16] -> the tensor core's tiled order (padding rows stay zero).
__global__ void nvfp4_tile_scales_kernel(const uint8_t* __restrict__ sb_canonical, int N, int K, uint8_t* __restrict__ sf_tiled)
{
    const int n_blocks = K / 16;
    const size_t idx = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (idx >= static_cast<size_t>(N) * n_blocks) return;
    const int j = static_cast<int>(idx / n_blocks), b = static_cast<int>(idx % n_blocks);
    sf_tiled[nvfp4_sf_offset(j, b, K / 64)] = sb_canonical[idx];
}

cudaError_t launch_import_nvfp4_scales(const uint8_t* sb_canonical, int N, int K, uint8_t* sf_tiled, size_t sf_tiled_bytes, cudaStream_t st)
{
    cudaError_t e = cudaMemsetAsync(sf_tiled, 0, sf_tiled_bytes, st);
    if (e != cudaSuccess) return e;
    const size_t total = static_cast<size_t>(N) * (K / 16);
    nvfp4_tile_scales_kernel<<<static_cast<unsigned>((total + 255) / 256), 256, 0, st>>>(sb_canonical, N, K, sf_tiled);
    return cudaGetLastError();
}

cudaError_t launch_pack_nvfp4(const float* W, const float* d, int N, int K, uint8_t* codes, uint8_t* sb_canonical,
                              uint8_t* sf_tiled, size_t sf_tiled_bytes, float* dinv, float* tensor_scale,
                              unsigned int* amax_bits, cudaStream_t st)
{
    cudaError_t e = cudaMemsetAsync(amax_bits, 0, sizeof(unsigned int), st);
    if (e != cudaSuccess) return e;
    e = cudaMemsetAsync(sf_tiled, 0, sf_tiled_bytes, st);      // rows past N (padding of the last 128-row atom)
    if (e != cudaSuccess) return e;
    nvfp4_absmax_kernel<<<592, 256, 0, st>>>(W, d, N, K, amax_bits);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    const size_t total = static_cast<size_t>(N) * (K / 16);
    nvfp4_quantize_kernel<<<static_cast<unsigned>((total + 255) / 256), 256, 0, st>>>(W, d, N, K, amax_bits, codes, sb_canonical,
                                                                                      sf_tiled, tensor_scale);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    dinv_kernel<<<(K + 255) / 256, 256, 0, st>>>(d, K, dinv);
    return cudaGetLastError();
}

}  // namespace rudder
