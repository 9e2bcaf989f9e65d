// Register-level unpack of packed weights to exact fp16 integers (device only).
//
// One routine per bit width, shared by the decode kernel, the prefill kernel and the debug unpack
// kernel, so that "the integers the device sees" means the same thing everywhere.  The conversions
// are exact: an integer u in [0, 1023] placed in the mantissa of fp16 1024.0 (0x6400) is the value
// 1024 + u, and subtracting the offset gives q without rounding.  The scale is never folded into the
// offset subtraction (that would round the offset); it is applied afterwards, once.
#pragma once
#include <cuda_fp16.h>
#include <stdint.h>

#include "../../include/qlinear.h"

namespace ql {

// Activation of the gate branch in the fused gating epilogue (paper Section 3.6), fp32, with the hardware
// exponential and reciprocal (a few ulp, far inside the tolerance of the product).
// tanh(t) = 1 - 2 / (exp(2t) + 1), so 0.5 * g * (1 + tanh(t)) = g * (1 - 1 / (exp(2t) + 1)) = g / (1 + exp(-2t)).
__device__ __forceinline__ float gate_activation(float g, int act)
{
    if (act == QL_ACT_IDENTITY) return g;
    const float t = act == QL_ACT_SILU ? g : 1.5957691216057308f * (g + 0.044715f * g * g * g);
    return __fdividef(g, 1.f + __expf(-t));
}

// mma.m16n8k16 (fp16 in, fp32 accumulate), not `volatile`: the compiler may interleave independent MMA chains.
__device__ __forceinline__ void mma_16816_pure(float d[4], const uint32_t a[4], uint32_t b0, uint32_t b1)
{
    asm("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// D = A.B with a zero accumulator input (no register has to be cleared first).
__device__ __forceinline__ void mma_16816_zero(float d[4], const uint32_t a[4], uint32_t b0, uint32_t b1)
{
    asm("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%10,%10,%10};"
        : "=f"(d[0]), "=f"(d[1]), "=f"(d[2]), "=f"(d[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1), "f"(0.f));
}

__device__ __forceinline__ uint32_t lop3_and_or(uint32_t a, uint32_t mask, uint32_t orv)
{
    uint32_t r;
    asm("lop3.b32 %0, %1, %2, %3, 0xEA;" : "=r"(r) : "r"(a), "r"(mask), "r"(orv));   // (a & mask) | orv
    return r;
}

__device__ __forceinline__ uint32_t h2_sub(uint32_t a, uint32_t b)
{
    uint32_t r;
    asm("sub.f16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
    return r;
}

__device__ __forceinline__ uint32_t h2_fma(uint32_t a, uint32_t b, uint32_t c)
{
    uint32_t r;
    asm("fma.rn.f16x2 %0, %1, %2, %3;" : "=r"(r) : "r"(a), "r"(b), "r"(c));
    return r;
}

__device__ __forceinline__ uint32_t h2_mul(uint32_t a, uint32_t b)
{
    uint32_t r;
    asm("mul.f16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
    return r;
}

// One int4 word (8 nibbles, stored as q + 8) -> four fp16x2 registers holding q exactly:
//   a[0] = (row g;   slots j0, j1)     a[1] = (row g+8; slots j0, j1)
//   a[2] = (row g;   slots j2, j3)     a[3] = (row g+8; slots j2, j3)
// which is the A fragment of mma.m16n8k16 for this lane.
__device__ __forceinline__ void unpack_int4_word(uint32_t w, uint32_t a[4])
{
    constexpr uint32_t kMagic = 0x64006400u;      // {1024, 1024}
    constexpr uint32_t kLoMask = 0x000F000Fu, kHiMask = 0x00F000F0u;
    constexpr uint32_t k1032 = 0x64086408u;       // {1032, 1032}: 1024 + the +8 storage offset
    constexpr uint32_t kSixteenth = 0x2C002C00u;  // {1/16, 1/16}
    constexpr uint32_t kNeg72 = 0xD480D480u;      // {-72, -72}: -(1024/16 + 8)
    const uint32_t w8 = w >> 8;
    a[0] = h2_sub(lop3_and_or(w, kLoMask, kMagic), k1032);
    a[1] = h2_fma(lop3_and_or(w, kHiMask, kMagic), kSixteenth, kNeg72);
    a[2] = h2_sub(lop3_and_or(w8, kLoMask, kMagic), k1032);
    a[3] = h2_fma(lop3_and_or(w8, kHiMask, kMagic), kSixteenth, kNeg72);
}

// Two int8 words (bytes stored as q + 128) -> the same four registers:
//   w0 = (g,j0) (g,j1) (g+8,j0) (g+8,j1)      w1 = (g,j2) (g,j3) (g+8,j2) (g+8,j3)
__device__ __forceinline__ void unpack_int8_words(uint32_t w0, uint32_t w1, uint32_t a[4])
{
    constexpr uint32_t kHi = 0x64646464u;
    constexpr uint32_t k1152 = 0x64806480u;       // {1152, 1152}: 1024 + the +128 storage offset
    a[0] = h2_sub(__byte_perm(w0, kHi, 0x4140), k1152);
    a[1] = h2_sub(__byte_perm(w0, kHi, 0x4342), k1152);
    a[2] = h2_sub(__byte_perm(w1, kHi, 0x4140), k1152);
    a[3] = h2_sub(__byte_perm(w1, kHi, 0x4342), k1152);
}

}  // namespace ql
