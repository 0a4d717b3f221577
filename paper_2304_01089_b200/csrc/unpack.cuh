// Device-side readers of the packed code formats (format version 2, described in rptq.h).
// 32 consecutive codes (one contraction step) become eight 32-bit words of four 8-bit operands
// each, in K order: out[2i] holds codes 8i..8i+3, out[2i+1] codes 8i+4..8i+7.
#pragma once
#include <stdint.h>

namespace rptq {

// Activation codes, unsigned. `p` holds the step's packed words: BITS words.
template <int BITS>
__device__ __forceinline__ void unpack_act32(const uint32_t (&p)[BITS], uint32_t (&out)[8])
{
    if constexpr (BITS == 8) {
#pragma unroll
        for (int i = 0; i < 8; ++i) out[i] = p[i];
    } else if constexpr (BITS == 4) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            out[2 * i] = p[i] & 0x0F0F0F0Fu;
            out[2 * i + 1] = (p[i] >> 4) & 0x0F0F0F0Fu;
        }
    } else {
        uint32_t tail = 0;
#pragma unroll
        for (int j = 0; j < 3; ++j) {
            out[2 * j] = p[j] & 0x07070707u;
            out[2 * j + 1] = (p[j] >> 4) & 0x07070707u;
            tail |= ((p[j] >> 3) & 0x11111111u) << j;
        }
        out[6] = tail & 0x07070707u;
        out[7] = (tail >> 4) & 0x07070707u;
    }
}

// Signed 4-bit weight codes, four packed words per step. Each nibble is moved to the top of its
// byte, so the 8-bit operand equals 16 * w (two's complement) and integer products come out
// exactly 16 times too large; the caller shifts or scales that factor away.
__device__ __forceinline__ void unpack_w32_x16(const uint32_t (&p)[4], uint32_t (&out)[8])
{
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        out[2 * i] = (p[i] << 4) & 0xF0F0F0F0u;
        out[2 * i + 1] = p[i] & 0xF0F0F0F0u;
    }
}

}  // namespace rptq
