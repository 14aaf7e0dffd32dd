// Device helpers shared by the kernels that quantise activations (Sec. 3.4) and by the two forms of the
// SiLU(gate) * up step that follows the fused gate+up projection (Sec. 3.5, "Kernel Fusion"): every kernel that
// produces a code or an h value goes through these, so that the forms agree bit for bit.
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <stdint.h>

namespace w4a8 {

// s_a = fp16_rne(min(amax / 127, 65504)) from the largest magnitude of a row, given as bf16 bits (15-bit pattern)
__device__ __forceinline__ __half row_scale_from_amax_bits(uint32_t amax_bf16_bits) {
    const float amax = __uint_as_float(amax_bf16_bits << 16);
    return __float2half_rn(fminf(__fdiv_rn(amax, 127.0f), 65504.0f));
}

// one code: rne(x / s) by IEEE division, clamped to [-127, 127]; x given as bf16 bits in the upper half of a word
__device__ __forceinline__ int quant1(uint32_t bf16_hi_bits, float s) {
    float q = __fdiv_rn(__uint_as_float(bf16_hi_bits), s);
    int r;
    asm("cvt.rni.sat.s8.f32 %0, %1;" : "=r"(r) : "f"(q));   // ties to even, saturates to [-128,127]
    return max(r, -127);
}

// h = bf16_rne(SiLU(g) * u) in fp32, g and u bf16 values: g / (1 + e^-g) * u with the fast exponential and
// division (a few fp32 ulps from the exact value: the rounded h equals the exactly computed one or its bf16
// neighbour; far out on the negative side, where e^-g overflows, the result is a signed zero like the limit).
__device__ __forceinline__ uint32_t silu_mul_bf16_bits(float g, float u) {
    const float h = __fmul_rn(__fdividef(g, 1.0f + __expf(-g)), u);
    return (uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(h));
}

// two h values from packed pairs of bf16 (low half = even element), result packed the same way
__device__ __forceinline__ uint32_t silu_mul_bf16x2(uint32_t g2, uint32_t u2) {
    const uint32_t lo = silu_mul_bf16_bits(__uint_as_float(g2 << 16), __uint_as_float(u2 << 16));
    const uint32_t hi = silu_mul_bf16_bits(__uint_as_float(g2 & 0xFFFF0000u), __uint_as_float(u2 & 0xFFFF0000u));
    return lo | (hi << 16);
}

}  // namespace w4a8
