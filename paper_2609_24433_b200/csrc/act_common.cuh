// Device helpers shared by the two prologue kernels.
#pragma once

#include <stdint.h>

namespace fq {

// Round-to-nearest-even code extraction: bits(t + 1.5*2^23) = 0x4B400000 + rint(t) for |t| < 2^22.
constexpr uint32_t kMagicBits = 0x4B400000u;

// Pack 8 four-bit (or 4 eight-bit) two's-complement codes from the raw bit patterns
// b[i] = kMagicBits + code_i (element 0 in the lowest field) with one shift-add per code:
// the Horner sum of the raw patterns equals the Horner sum of the codes plus a constant;
// adding half the field range to every field removes the borrows between fields, and
// flipping each field's top bit afterwards turns offset binary into two's complement.
template <int FMT>
__device__ __forceinline__ uint32_t pack_word(const uint32_t* b) {
    if (FMT == 0) {
        uint32_t w = b[7];
#pragma unroll
        for (int i = 6; i >= 0; --i) w = (w << 4) + b[i];
        return (w + (0x88888888u - kMagicBits * 0x11111111u)) ^ 0x88888888u;
    } else {
        // 8-bit codes: the low byte of every raw pattern already is the two's-complement code
        // (0x4B400000 + code has the code's low 8 bits in its lowest byte), so three byte permutes
        // gather the four bytes.
        uint32_t lo, hi, w;
        asm("prmt.b32 %0, %1, %2, 0x0040;" : "=r"(lo) : "r"(b[0]), "r"(b[1]));
        asm("prmt.b32 %0, %1, %2, 0x0040;" : "=r"(hi) : "r"(b[2]), "r"(b[3]));
        asm("prmt.b32 %0, %1, %2, 0x5410;" : "=r"(w) : "r"(lo), "r"(hi));
        return w;
    }
}

// Warp maximum of a non-negative float (an absolute-value maximum): non-negative IEEE values order
// like their bit patterns, so one integer warp reduction replaces five shuffle + max steps.
__device__ __forceinline__ float warp_max_nonneg(float m) {
    return __uint_as_float(__reduce_max_sync(0xffffffffu, __float_as_uint(m)));
}

// Channel (within a thread's run) that field i of 32-bit word j holds, per store format.
template <int FMT>
__device__ __forceinline__ constexpr int code_index(int j, int i) {
    return FMT == 0 ? 8 * j + i : (FMT == 1 ? 4 * j + i : 8 * (j / 2) + 2 * i + (j & 1));
}

// Packed binary32 arithmetic (two independent IEEE operations per instruction).  Written as PTX
// with an explicit rounding modifier: such instructions are never contracted into fused
// multiply-adds by the optimizer, which the bit-exact contract of the prologue depends on.
__device__ __forceinline__ float2 f2_mul(float2 a, float2 b) {
    float2 d;
    asm("mul.rn.f32x2 %0, %1, %2;"
        : "=l"(*reinterpret_cast<uint64_t*>(&d))
        : "l"(*reinterpret_cast<const uint64_t*>(&a)), "l"(*reinterpret_cast<const uint64_t*>(&b)));
    return d;
}
__device__ __forceinline__ float2 f2_add(float2 a, float2 b) {
    float2 d;
    asm("add.rn.f32x2 %0, %1, %2;"
        : "=l"(*reinterpret_cast<uint64_t*>(&d))
        : "l"(*reinterpret_cast<const uint64_t*>(&a)), "l"(*reinterpret_cast<const uint64_t*>(&b)));
    return d;
}
__device__ __forceinline__ float2 f2_fma(float2 a, float2 b, float2 c) {
    float2 d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;"
        : "=l"(*reinterpret_cast<uint64_t*>(&d))
        : "l"(*reinterpret_cast<const uint64_t*>(&a)), "l"(*reinterpret_cast<const uint64_t*>(&b)),
          "l"(*reinterpret_cast<const uint64_t*>(&c)));
    return d;
}

}  // namespace fq
