// BF16 glue between the quantized linears of a chained DiT block (the paper keeps GELU in BF16,
// outside the quantized path, like normalisation and residual additions: Appendix "Quantization").  What a
// chain of rudder_linear calls needs to run back to back on the device: GELU, RMS normalisation, residual add.
//
// GELU is taken in its tanh form, g(x) = x/2 (1 + tanh(sqrt(2/pi) (x + 0.044715 x^3))), with tanh
// replaced by its [7/6] Pade approximant
//     tanh u ~ u (135135 + 17325 u^2 + 378 u^4 + u^6) / (135135 + 62370 u^2 + 3150 u^4 + 28 u^6)
// for |u| < 5 and by +-1 beyond (error below 2e-4 of the tanh form, under the bf16 step of the
// result).  Every operation is a single correctly rounded fp32 add, multiply or divide in the order
// written below -- no fused multiply-add, no approximate instruction -- so that the result is
// defined bit for bit and a plain CPU program can repeat it.
#include "internal.cuh"

#include <cuda_bf16.h>

namespace rudder {

namespace {

__device__ __forceinline__ float gelu_f32(float x) {
    const float x2 = __fmul_rn(x, x);
    const float x3 = __fmul_rn(x2, x);
    const float inner = __fadd_rn(x, __fmul_rn(0.044715f, x3));
    const float u = __fmul_rn(0.7978845608028654f, inner);
    float t;
    if (!(fabsf(u) < 5.0f)) {
        t = (u < 0.0f) ? -1.0f : 1.0f;              // also +-infinity; NaN propagates through the product below
        if (u != u) t = u;
    } else {
        const float u2 = __fmul_rn(u, u);
        float n = __fadd_rn(u2, 378.0f);
        n = __fadd_rn(__fmul_rn(n, u2), 17325.0f);
        n = __fadd_rn(__fmul_rn(n, u2), 135135.0f);
        n = __fmul_rn(n, u);
        float d = __fadd_rn(__fmul_rn(28.0f, u2), 3150.0f);
        d = __fadd_rn(__fmul_rn(d, u2), 62370.0f);
        d = __fadd_rn(__fmul_rn(d, u2), 135135.0f);
        t = __fdiv_rn(n, d);
    }
    return __fmul_rn(__fmul_rn(0.5f, x), __fadd_rn(1.0f, t));
}

__device__ __forceinline__ uint32_t gelu_pair(uint32_t w) {
    const float lo = gelu_f32(__uint_as_float(w << 16));
    const float hi = gelu_f32(__uint_as_float(w & 0xFFFF0000u));
    return static_cast<uint32_t>(__bfloat16_as_ushort(__float2bfloat16_rn(lo))) |
           (static_cast<uint32_t>(__bfloat16_as_ushort(__float2bfloat16_rn(hi))) << 16);
}

// One 16-byte chunk (8 values) per thread step; rows of N values (N % 8 == 0), leading dimensions in elements.
__global__ void __launch_bounds__(256) gelu_bf16_kernel(const uint16_t* __restrict__ X, int64_t ldx, uint16_t* __restrict__ Y, int64_t ldy,
                                                        int M, int N)
{
    const int chunks = N >> 3;
    const long long total = static_cast<long long>(M) * chunks;
    for (long long i = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x; i < total;
         i += static_cast<long long>(gridDim.x) * blockDim.x) {
        const int row = static_cast<int>(i / chunks);
        const int c = static_cast<int>(i - static_cast<long long>(row) * chunks);
        const uint4 v = *reinterpret_cast<const uint4*>(X + static_cast<size_t>(row) * ldx + 8 * c);
        uint4 o;
        o.x = gelu_pair(v.x); o.y = gelu_pair(v.y); o.z = gelu_pair(v.z); o.w = gelu_pair(v.w);
        *reinterpret_cast<uint4*>(Y + static_cast<size_t>(row) * ldy + 8 * c) = o;
    }
}

// RMS normalisation of the rows of X with a weight per channel: y = bf16(((x * r) * w)), r = 1 / sqrt(mean(x^2) + eps).
// (The paper keeps normalisation in BF16 and does not say which; reading: RMSNorm with a learned weight.)
// Bit-defined like the GELU: one warp per row; lane l takes the 8-value pieces l, l + 32, ... in order and adds
// x * x (product and sum rounded separately) into one fp32 partial; the 32 partials are combined by the
// butterfly l ^ 16, 8, 4, 2, 1 (every lane ends with the same bits); mean = sum / N, r = 1 / sqrt(mean + eps) with
// IEEE division and square root.
__global__ void __launch_bounds__(256) rmsnorm_bf16_kernel(const uint16_t* __restrict__ X, int64_t ldx, const float* __restrict__ w,
                                                           float eps, uint16_t* __restrict__ Y, int64_t ldy, int M, int N)
{
    const int row = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (row >= M) return;
    const int chunks = N >> 3;
    const uint4* xr = reinterpret_cast<const uint4*>(X + static_cast<size_t>(row) * ldx);
    float s = 0.0f;
    for (int c = lane; c < chunks; c += 32) {
        const uint4 v = xr[c];
        const uint32_t wds[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float lo = __uint_as_float(wds[i] << 16), hi = __uint_as_float(wds[i] & 0xFFFF0000u);
            s = __fadd_rn(s, __fmul_rn(lo, lo));
            s = __fadd_rn(s, __fmul_rn(hi, hi));
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s = __fadd_rn(s, __shfl_xor_sync(0xffffffffu, s, o));
    const float r = __fdiv_rn(1.0f, __fsqrt_rn(__fadd_rn(__fdiv_rn(s, static_cast<float>(N)), eps)));
    uint4* yr = reinterpret_cast<uint4*>(Y + static_cast<size_t>(row) * ldy);
    for (int c = lane; c < chunks; c += 32) {
        const uint4 v = xr[c];
        const float4 w0 = __ldg(reinterpret_cast<const float4*>(w) + 2 * c), w1 = __ldg(reinterpret_cast<const float4*>(w) + 2 * c + 1);
        const float ww[8] = {w0.x, w0.y, w0.z, w0.w, w1.x, w1.y, w1.z, w1.w};
        const uint32_t wds[4] = {v.x, v.y, v.z, v.w};
        uint32_t o[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float lo = __uint_as_float(wds[i] << 16), hi = __uint_as_float(wds[i] & 0xFFFF0000u);
            const float a = __fmul_rn(__fmul_rn(lo, r), ww[2 * i]), b = __fmul_rn(__fmul_rn(hi, r), ww[2 * i + 1]);
            o[i] = static_cast<uint32_t>(__bfloat16_as_ushort(__float2bfloat16_rn(a))) |
                   (static_cast<uint32_t>(__bfloat16_as_ushort(__float2bfloat16_rn(b))) << 16);
        }
        yr[c] = make_uint4(o[0], o[1], o[2], o[3]);
    }
}

// Residual addition, elementwise: y = bf16(a + b), one fp32 addition.
__global__ void __launch_bounds__(256) add_bf16_kernel(const uint16_t* __restrict__ A, int64_t lda, const uint16_t* __restrict__ B, int64_t ldb,
                                                       uint16_t* __restrict__ Y, int64_t ldy, int M, int N)
{
    const int chunks = N >> 3;
    const long long total = static_cast<long long>(M) * chunks;
    for (long long i = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x; i < total;
         i += static_cast<long long>(gridDim.x) * blockDim.x) {
        const int row = static_cast<int>(i / chunks);
        const int c = static_cast<int>(i - static_cast<long long>(row) * chunks);
        const uint4 a = *reinterpret_cast<const uint4*>(A + static_cast<size_t>(row) * lda + 8 * c);
        const uint4 b = *reinterpret_cast<const uint4*>(B + static_cast<size_t>(row) * ldb + 8 * c);
        const uint32_t aw[4] = {a.x, a.y, a.z, a.w}, bw[4] = {b.x, b.y, b.z, b.w};
        uint32_t o[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const float lo = __fadd_rn(__uint_as_float(aw[j] << 16), __uint_as_float(bw[j] << 16));
            const float hi = __fadd_rn(__uint_as_float(aw[j] & 0xFFFF0000u), __uint_as_float(bw[j] & 0xFFFF0000u));
            o[j] = static_cast<uint32_t>(__bfloat16_as_ushort(__float2bfloat16_rn(lo))) |
                   (static_cast<uint32_t>(__bfloat16_as_ushort(__float2bfloat16_rn(hi))) << 16);
        }
        *reinterpret_cast<uint4*>(Y + static_cast<size_t>(row) * ldy + 8 * c) = make_uint4(o[0], o[1], o[2], o[3]);
    }
}

// ---- GELU fused into the activation prologue of the layer behind it (static range) ----------------------
// With the paper's static threshold c_tau (Section 4.3; Appendix "Quantization": one calibrated base scale
// shared by all streams) the prologue of the down projection needs no row reduction: a_i = c_tau for every
// row.  Requantising the up projection's output is then purely elementwise, so the GELU between the two
// layers moves into the same pass: read the up output once, bf16(gelu(.)), v = (g * dinv_k) * gamma_s(i),
// code = clip(round(v * q_max / c)), and r_i = (c / q_max) / gamma_s(i).  The activated tensor is never
// written, the prologue never reads it back, and one launch goes away.  The arithmetic per element is
// gelu_f32 above followed by scale8 / round8 of the prologue: the same bits as the two separate passes.
__global__ void __launch_bounds__(256) actq_gelu_static_kernel(ActqArgs a, int qmax, int e4m3, int8_t* __restrict__ codes, int64_t ldc,
                                                                float* __restrict__ r)
{
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    if (blockIdx.x == 0 && a.zero_ints != nullptr)
        for (int i = threadIdx.x; i < a.n_zero; i += blockDim.x) a.zero_ints[i] = 0;
    const int chunks = a.K >> 3;
    const long long total = static_cast<long long>(a.M) * chunks;
    const float range = *a.clip_step;
    const float qf = static_cast<float>(qmax);
    const float inv = (range != 0.0f) ? __fdiv_rn(qf, range) : 0.0f;
    const float4* dv = reinterpret_cast<const float4*>(a.dinv);
    for (long long i = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x; i < total;
         i += static_cast<long long>(gridDim.x) * blockDim.x) {
        const int row = static_cast<int>(i / chunks);
        const int c = static_cast<int>(i - static_cast<long long>(row) * chunks);
        const float g = a.gamma_step[stream_of_row(a.seg, row)];
        const uint4 x = *reinterpret_cast<const uint4*>(a.X + static_cast<size_t>(row) * a.ldx + 8 * c);
        uint4 act;
        act.x = gelu_pair(x.x); act.y = gelu_pair(x.y); act.z = gelu_pair(x.z); act.w = gelu_pair(x.w);
        float v[8];
        scale8(act, __ldg(dv + 2 * c), __ldg(dv + 2 * c + 1), g, v);
        *reinterpret_cast<uint2*>(codes + static_cast<size_t>(row) * ldc + 8 * c) = e4m3 ? round8_e4m3(v, inv, qmax) : round8(v, inv, qmax);
        if (c == 0) r[row] = (range != 0.0f) ? __fdiv_rn(__fdiv_rn(range, qf), g) : 0.0f;
    }
}

}  // namespace

cudaError_t launch_actq_gelu_static(const ActqArgs& a, int qmax, bool e4m3, int8_t* codes, int64_t ldc, float* r, int sm_count, cudaStream_t st)
{
    const long long total = static_cast<long long>(a.M) * (a.K >> 3);
    long long blocks = (total + 255) / 256;
    const long long cap = static_cast<long long>(sm_count > 0 ? sm_count : 148) * 8;
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(blocks), 1, 1);
    cfg.blockDim = dim3(256, 1, 1);
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaError_t e = cudaLaunchKernelEx(&cfg, actq_gelu_static_kernel, a, qmax, e4m3 ? 1 : 0, codes, ldc, r);
    return e != cudaSuccess ? e : cudaGetLastError();
}

cudaError_t launch_rmsnorm(const uint16_t* X, int64_t ldx, const float* w, float eps, uint16_t* Y, int64_t ldy, int M, int N, cudaStream_t st)
{
    const int blocks = (M * 32 + 255) / 256;
    rmsnorm_bf16_kernel<<<blocks, 256, 0, st>>>(X, ldx, w, eps, Y, ldy, M, N);
    return cudaGetLastError();
}

cudaError_t launch_add(const uint16_t* A, int64_t lda, const uint16_t* B, int64_t ldb, uint16_t* Y, int64_t ldy, int M, int N, int sm_count,
                       cudaStream_t st)
{
    const long long total = static_cast<long long>(M) * (N >> 3);
    long long blocks = (total + 255) / 256;
    const long long cap = static_cast<long long>(sm_count > 0 ? sm_count : 148) * 8;
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    add_bf16_kernel<<<static_cast<unsigned>(blocks), 256, 0, st>>>(A, lda, B, ldb, Y, ldy, M, N);
    return cudaGetLastError();
}

cudaError_t launch_gelu(const uint16_t* X, int64_t ldx, uint16_t* Y, int64_t ldy, int M, int N, int sm_count, cudaStream_t st)
{
    const long long total = static_cast<long long>(M) * (N >> 3);
    long long blocks = (total + 255) / 256;
    const long long cap = static_cast<long long>(sm_count > 0 ? sm_count : 148) * 8;
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    gelu_bf16_kernel<<<static_cast<unsigned>(blocks), 256, 0, st>>>(X, ldx, Y, ldy, M, N);
    return cudaGetLastError();
}

}  // namespace rudder
