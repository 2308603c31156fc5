// Device helpers shared by the kernels that rebuild scaled weights from plane bits: power-of-two
// scalings that keep fp16 operands in range, and the byte-wise lookup table of the 2^q levels
// sum_i +-alpha_i of one (row, group) that PRMT indexes.
#pragma once
#include <cuda_fp16.h>
#include <stdint.h>

namespace bcq {

__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t c) {
    uint32_t d;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
    return d;
}

__device__ __forceinline__ uint32_t pack_half2(float lo, float hi) {
    __half2 h = __floats2half2_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&h);
}

// 2^e as a float, e clamped to the normal range.
__device__ __forceinline__ float pow2f(int e) {
    e = max(-126, min(127, e));
    return __uint_as_float((uint32_t)(e + 127) << 23);
}

// Exponent of a positive finite float given by its bits (0 for zero / subnormal input).
__device__ __forceinline__ int exponent_of_bits(uint32_t fbits) {
    const int be = (int)((fbits >> 23) & 0xFFu);
    return be == 0 ? -127 : be - 127;
}

// Power of two that brings a magnitude with exponent `e` to [2^target, 2^(target+1)).
__device__ __forceinline__ int shift_for(int e, int target) {
    if (e <= -127 || e >= 128) return 0;  // zero, subnormal, inf or nan: leave alone
    return max(-100, min(100, target - e));
}

// Byte-wise lookup table of eight fp16 levels: tl* low bytes, th* high bytes; *0 = levels 0..3.
struct Lut {
    uint32_t tl0, tl1, th0, th1;
};

// Level s (bit i of s set <=> plane i is +1) = base + sum_{i<3} (+-a_i).
__device__ __forceinline__ Lut build_lut(float a0, float a1, float a2, float base) {
    const float t0 = base - a0, t1 = base + a0;
    const float u0 = t0 - a1, u1 = t1 - a1, u2 = t0 + a1, u3 = t1 + a1;
    const uint32_t p0 = pack_half2(u0 - a2, u1 - a2);
    const uint32_t p1 = pack_half2(u2 - a2, u3 - a2);
    const uint32_t p2 = pack_half2(u0 + a2, u1 + a2);
    const uint32_t p3 = pack_half2(u2 + a2, u3 + a2);
    Lut t;
    t.tl0 = prmt(p0, p1, 0x6420u);
    t.th0 = prmt(p0, p1, 0x7531u);
    t.tl1 = prmt(p2, p3, 0x6420u);
    t.th1 = prmt(p2, p3, 0x7531u);
    return t;
}

}  // namespace bcq
