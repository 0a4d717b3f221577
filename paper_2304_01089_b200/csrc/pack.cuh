// Device-side writer of the packed code formats (format version 2, described in rptq.h):
// 32 consecutive codes, one per register, become BITS 32-bit words.
#pragma once
#include <stdint.h>

namespace rptq {

// The quantiser decision of the GEMM's re-quantising epilogue (Eq. 1 with codes re-based to
// [0, 2^bits - 1]): t = y * inv_s rounded ONCE to an integer, half to even (the fused multiply-add
// forms the product exactly; adding 1.5 * 2^23 leaves the rounded integer in the low mantissa bits
// for |t| < 2^22; larger t keep their order, and everything below -2^22, the negative sums whose bit
// patterns would wrap included, is raised to 2^23, i.e. to an integer far below any zero point),
// then + z_c and clamp. zc = z_c - 0x4B400000 (the bit pattern of 1.5 * 2^23); |z_c| < 2^21.
__device__ __forceinline__ uint32_t quant_code(float y, float inv_s, int zc, int qmax)
{
    const float v = fmaxf(__fmaf_rn(y, inv_s, 12582912.0f), 8388608.0f);
    const int q = __float_as_int(v) + zc;
    return (uint32_t)min(max(q, 0), qmax);
}

__device__ __forceinline__ uint32_t nibble_word(const uint32_t* q)   // 8 codes -> one 4-bit-layout word
{
    uint32_t w = 0;
#pragma unroll
    for (int t = 0; t < 8; ++t) w |= q[t] << (8 * (t & 3) + 4 * (t >> 2));
    return w;
}

template <int BITS>
__device__ __forceinline__ void pack32(const uint32_t (&q)[32], uint32_t (&w)[BITS])
{
    if constexpr (BITS == 8) {
#pragma unroll
        for (int i = 0; i < 8; ++i) w[i] = q[4 * i] | (q[4 * i + 1] << 8) | (q[4 * i + 2] << 16) | (q[4 * i + 3] << 24);
    } else if constexpr (BITS == 4) {
#pragma unroll
        for (int i = 0; i < 4; ++i) w[i] = nibble_word(q + 8 * i);
    } else {
        const uint32_t tail = nibble_word(q + 24);
#pragma unroll
        for (int j = 0; j < 3; ++j) w[j] = nibble_word(q + 8 * j) | (((tail >> j) & 0x11111111u) << 3);
    }
}

// The same words from UNCLAMPED integers: the saturating pack instruction clamps to [0, 15] (or
// [0, 255]) and appends two codes per instruction, d = (c << 8) | (sat(a) << 4) | sat(b) for 4-bit
// fields and d = (c << 16) | (sat(a) << 8) | sat(b) for bytes; 3-bit codes are clamped to 7 afterwards.
// `flip` (zero or all ones) then replaces every code q by 2^BITS - 1 - q.
__device__ __forceinline__ uint32_t sat_pack_u4(int a, int b, uint32_t c)
{
    uint32_t d;
    asm("cvt.pack.sat.u4.s32.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
    return d;
}
__device__ __forceinline__ uint32_t sat_pack_u8(int a, int b, uint32_t c)
{
    uint32_t d;
    asm("cvt.pack.sat.u8.s32.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
    return d;
}
__device__ __forceinline__ uint32_t sat_nibble_word(const int* v)     // 8 integers -> one 4-bit-layout word
{
    uint32_t d = sat_pack_u4(v[7], v[3], 0u);
    d = sat_pack_u4(v[6], v[2], d);
    d = sat_pack_u4(v[5], v[1], d);
    return sat_pack_u4(v[4], v[0], d);
}
template <int BITS>
__device__ __forceinline__ void pack32_sat(const int (&v)[32], uint32_t (&w)[BITS], uint32_t flip = 0u)
{
    if constexpr (BITS == 8) {
#pragma unroll
        for (int i = 0; i < 8; ++i) w[i] = sat_pack_u8(v[4 * i + 1], v[4 * i], sat_pack_u8(v[4 * i + 3], v[4 * i + 2], 0u)) ^ flip;
    } else if constexpr (BITS == 4) {
#pragma unroll
        for (int i = 0; i < 4; ++i) w[i] = sat_nibble_word(v + 8 * i) ^ flip;
    } else {
        // the pack instruction clamps to [0, 15]; nibbles above 7 (bit 3 set) become 7, eight at a time
        const uint32_t f7 = flip & 0x77777777u;
        auto clamp7 = [f7](uint32_t x) { return ((x | (((x >> 3) & 0x11111111u) * 7u)) & 0x77777777u) ^ f7; };
        const uint32_t tail = clamp7(sat_nibble_word(v + 24));
#pragma unroll
        for (int j = 0; j < 3; ++j) w[j] = clamp7(sat_nibble_word(v + 8 * j)) | (((tail >> j) & 0x11111111u) << 3);
    }
}

}  // namespace rptq
