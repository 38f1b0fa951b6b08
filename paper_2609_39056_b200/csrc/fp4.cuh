// NVFP4 number formats on the device: E2M1 codes (4 bit) and UE4M3 block scales (8 bit), converted
// with the hardware's round-to-nearest-even, saturating instructions.
#pragma once

#include <cuda_fp16.h>
#include <stdint.h>

namespace rudder {

constexpr float kNvfp4Range = 2688.0f;   // 6 (largest E2M1) x 448 (largest UE4M3)

// UE4M3 byte of a non-negative float (round to nearest even, saturate at 448).
__device__ __forceinline__ uint32_t f32_to_ue4m3(float x) {
    uint16_t h;
    asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(h) : "f"(0.0f), "f"(x));
    return h & 0xFFu;
}
__device__ __forceinline__ float ue4m3_to_f32(uint32_t b) {
    uint32_t h2;
    asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(h2) : "h"(static_cast<uint16_t>(b & 0xFFu)));
    return __half2float(__ushort_as_half(static_cast<unsigned short>(h2 & 0xFFFFu)));
}
// Eight floats -> eight E2M1 codes in one word, element i in nibble i.
__device__ __forceinline__ uint32_t f32x8_to_e2m1(const float (&v)[8]) {
    uint32_t out;
    asm("{\n\t"
        ".reg .b8 b0, b1, b2, b3;\n\t"
        "cvt.rn.satfinite.e2m1x2.f32 b0, %2, %1;\n\t"
        "cvt.rn.satfinite.e2m1x2.f32 b1, %4, %3;\n\t"
        "cvt.rn.satfinite.e2m1x2.f32 b2, %6, %5;\n\t"
        "cvt.rn.satfinite.e2m1x2.f32 b3, %8, %7;\n\t"
        "mov.b32 %0, {b0, b1, b2, b3};\n\t"
        "}\n"
        : "=r"(out)
        : "f"(v[0]), "f"(v[1]), "f"(v[2]), "f"(v[3]), "f"(v[4]), "f"(v[5]), "f"(v[6]), "f"(v[7]));
    return out;
}

// One block of 16 values that are already multiplied by the outer reciprocal scale (`inv`):
// UE4M3 block scale = rn(amax / 6), codes = rn(value / decoded scale).  Returns the scale byte.
__device__ __forceinline__ uint32_t nvfp4_encode_block(const float (&u)[16], uint32_t& lo, uint32_t& hi) {
    float amax = 0.0f;
#pragma unroll
    for (int i = 0; i < 16; ++i) amax = fmaxf(amax, fabsf(u[i]));
    const uint32_t sb = f32_to_ue4m3(__fdiv_rn(amax, 6.0f));
    const float sbd = ue4m3_to_f32(sb);
    const float rb = (sbd != 0.0f) ? __fdiv_rn(1.0f, sbd) : 0.0f;
    float a[8], b[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        a[i] = __fmul_rn(u[i], rb);
        b[i] = __fmul_rn(u[8 + i], rb);
    }
    lo = f32x8_to_e2m1(a);
    hi = f32x8_to_e2m1(b);
    if (sb == 0u) { lo = 0u; hi = 0u; }        // a block whose scale is zero holds +0 codes, not -0 for negative inputs
    return sb;
}

// Byte offset of the scale of (row, 16-element block kb) in the tensor core's tiled order:
// [row / 128][kb / 4][row % 32][(row / 32) % 4][kb % 4], K/64 chunks of 512 bytes per 128 rows.
__device__ __host__ __forceinline__ size_t nvfp4_sf_offset(int row, int kb, int k64) {
    return (static_cast<size_t>(row >> 7) * k64 + (kb >> 2)) * 512 + (row & 31) * 16 + ((row >> 5) & 3) * 4 + (kb & 3);
}

}  // namespace rudder
