// Device helpers shared by the kernels that rebuild scaled weights from plane bits: power-of-two
// scalings that keep fp16 operands in range, and the byte-wise lookup table of the 2^q levels
// sum_i +-alpha_i of one (row, group) that PRMT indexes.
#pragma once
#include <cuda_fp16.h>
#include <stdint.h>

#include "ptx.cuh"

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

// ------------------------------------------------------------------------------------------
// Selector codes.  The planes of a frozen matrix can be rewritten once so that the level index of
// every weight is already the 4-bit selector nibble PRMT wants: selector word r of a block of 32
// weights holds, in nibble e, the index of weight 8r + e (bit i <=> b_{i+1} = +1; for q = 4 the
// index of b_1..b_3, mirrored when b_4 = -1, with bit 3 set in that case: the level is then the
// negative of the mirrored one).  Stored per 32 weights in Q words (the same q bits per weight):
//   Q = 4   the four selector words;
//   Q = 3   selector words 0..2, with selector word 3 spread over bit 3 of their nibbles;
//   Q = 2   two words, each holding two selector words two bits apart;
//   Q = 1   one word holding the four selector words one bit apart.
// ------------------------------------------------------------------------------------------

// Host/device: the Q stored words from the four selector words.
template <int Q>
__host__ __device__ inline void pack_selectors(const uint32_t (&S)[4], uint32_t* dst) {
    if (Q == 4) {
        for (int r = 0; r < 4; ++r) dst[r] = S[r];
    } else if (Q == 3) {
        for (int v = 0; v < 3; ++v) dst[v] = S[v] | (((S[3] >> v) & 0x11111111u) << 3);
    } else if (Q == 2) {
        dst[0] = S[0] | (S[1] << 2);
        dst[1] = S[2] | (S[3] << 2);
    } else {
        dst[0] = S[0] | (S[1] << 1) | (S[2] << 2) | (S[3] << 3);
    }
}

// The four selector words of the 32 weights whose plane words are w[0..q-1] (canonical bit order).
__host__ __device__ inline void selectors_from_planes(const uint32_t (&w)[4], int q, uint32_t (&S)[4]) {
    for (int r = 0; r < 4; ++r) S[r] = 0u;
    for (int e = 0; e < 32; ++e) {
        uint32_t code = 0u;
        for (int i = 0; i < 3 && i < q; ++i) code |= ((w[i] >> e) & 1u) << i;
        if (q == 4 && !((w[3] >> e) & 1u)) code = (~code & 7u) | 8u;
        S[e >> 3] |= code << (4 * (e & 7));
    }
}

template <int Q>
__device__ __forceinline__ void load_codes(uint32_t addr, uint32_t (&v)[Q]) {
    if constexpr (Q == 4) {
        asm volatile("ld.shared.v4.b32 {%0,%1,%2,%3}, [%4];" : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3])
                     : "r"(addr) : "memory");
    } else if constexpr (Q == 2) {
        asm volatile("ld.shared.v2.b32 {%0,%1}, [%2];" : "=r"(v[0]), "=r"(v[1]) : "r"(addr) : "memory");
    } else {
#pragma unroll
        for (int i = 0; i < Q; ++i) v[i] = ptx::ld_shared_u32(addr + 4 * i);
    }
}

// The four selector words of 32 weights from the q stored words (see pack_codes_kernel).
template <int Q>
__device__ __forceinline__ void selectors(const uint32_t (&v)[Q], uint32_t (&S)[4]) {
    constexpr uint32_t M = 0x11111111u;
    if constexpr (Q == 4) {
#pragma unroll
        for (int r = 0; r < 4; ++r) S[r] = v[r];
    } else if constexpr (Q == 3) {
#pragma unroll
        for (int r = 0; r < 3; ++r) S[r] = v[r] & 0x77777777u;
        S[3] = (__umulhi(v[0], 1u << 29) & M) | (__umulhi(v[1], 1u << 30) & (M << 1)) | (__umulhi(v[2], 1u << 31) & (M << 2));
    } else if constexpr (Q == 2) {
        S[0] = v[0] & 0x33333333u;
        S[1] = (v[0] >> 2) & 0x33333333u;
        S[2] = v[1] & 0x33333333u;
        S[3] = (v[1] >> 2) & 0x33333333u;
    } else {
#pragma unroll
        for (int r = 0; r < 4; ++r) S[r] = (v[0] >> r) & M;
    }
}

// 32 weights of one row: selector word r gives the eight fp16 values of 16-byte chunk chunk0 + r
// of the row's 128-byte line (swizzle key lx), in natural k order.  `line` is 128-byte aligned, so
// the swizzled chunk address is line ^ (lx << 4) ^ (chunk << 4): one XOR per store.
template <int Q>
__device__ __forceinline__ void expand32_codes(const uint32_t (&S)[4], const Lut& t, uint32_t line, uint32_t lx,
                                               uint32_t chunk0) {
    const uint32_t linex = line ^ (lx << 4);
#pragma unroll
    for (int r = 0; r < 4; ++r) {
        // (shifts written as multiplications run on the multiply-add pipe; the logic pipe, which does
        // the PRMTs, is the one that paces this loop)
        const uint32_t s = (Q == 4) ? (S[r] & 0x77777777u) : S[r];
        const uint32_t sh = __umulhi(s, 1u << 16);
        const uint32_t lbl = prmt(t.tl0, t.tl1, s), lbh = prmt(t.tl0, t.tl1, sh);
        uint32_t hbl = prmt(t.th0, t.th1, s), hbh = prmt(t.th0, t.th1, sh);
        if (Q == 4) {
            // bit 3 of nibble e = "negate": replicate it over byte e (PRMT's sign mode reads the most
            // significant bit of a byte; shifting by 4 brings the even nibbles' flags there)
            const uint32_t fa = S[r] * 16u;
            hbl ^= prmt(fa, S[r], 0xD9C8u) & 0x80808080u;
            hbh ^= prmt(fa, S[r], 0xFBEAu) & 0x80808080u;
        }
        ptx::st_shared_v4(linex ^ ((chunk0 + r) << 4), prmt(lbl, hbl, 0x5140u), prmt(lbl, hbl, 0x7362u),
                          prmt(lbh, hbh, 0x5140u), prmt(lbh, hbh, 0x7362u));
    }
}

}  // namespace bcq
