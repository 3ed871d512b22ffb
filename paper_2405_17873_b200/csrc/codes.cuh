// Reading single codes out of the packed weight layouts (both the canonical and the device layout): the slow,
// general decoder behind the unpack hook, the code sums and the one-off expansion of a layer's weights.
#pragma once

#include "common.cuh"

namespace mixdq {

#ifdef __CUDACC__
// Code k of a packed row.
__device__ __forceinline__ int decode_code(const uint8_t* __restrict__ row, int64_t k, int bits, int is_signed,
                                           int layout)
{
    int c;
    if (bits == 8) {
        c = is_signed ? static_cast<int>(static_cast<int8_t>(row[k])) : static_cast<int>(row[k]);
    } else if (bits == 4) {
        int nib;
        if (layout == MIXDQ_LAYOUT_CANONICAL) {
            nib = (k & 1) ? (row[k >> 1] >> 4) : (row[k >> 1] & 0xf);
        } else {
            const int64_t g = k >> 3;
            const int j = static_cast<int>(k & 7);
            const uint8_t b = row[4 * g + (j & 3)];
            nib = (j >= 4) ? (b >> 4) : (b & 0xf);
        }
        c = (is_signed && nib >= 8) ? nib - 16 : nib;
    } else {
        c = 0;
        for (int p = 0; p < bits; ++p) {
            int64_t byte;
            int bit;
            if (layout == MIXDQ_LAYOUT_CANONICAL) {
                byte = (k / 32) * 4 * bits + p * 4 + ((k % 32) >> 3);
                bit = static_cast<int>(k & 7);
            } else {
                const int64_t blk = k / 128;
                const int r = static_cast<int>(k % 128);
                const int t = r >> 5, sft = (r & 31) >> 3, j = r & 7;
                const int f = (j < 4) ? 2 * j : 2 * (j - 4) + 1;
                const int pos = 4 * f + sft;
                byte = blk * 16 * bits + p * 16 + t * 4 + (pos >> 3);
                bit = pos & 7;
            }
            c |= ((row[byte] >> bit) & 1) << p;
        }
    }
    return c;
}

// Eight consecutive codes k0 .. k0 + 7 (k0 a multiple of 8) of a row in the device layout, as integers.
// 8 bits: eight bytes.  4 bits: one 32-bit word, byte j = code j (low nibble) | code j + 4 (high nibble).
// 2 / 3 bits: blocks of 128 codes, one 16-byte plane per bit; the eight codes' bits sit in ONE 32-bit word of
// each plane, code j at bit ((k0 % 32) / 8) + {0, 8, 16, 24, 4, 12, 20, 28}[j] (the interleave that lets the
// register decode of the few-token kernel rebuild 4-bit fields with shifts).
template <int BITS, bool SIGNED>
__device__ __forceinline__ void codes8(const uint8_t* __restrict__ row, int k0, int (&c)[8])
{
    if (BITS == 8) {
        const uint2 v = *reinterpret_cast<const uint2*>(row + k0);
        const uint32_t w[2] = {v.x, v.y};
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const uint32_t byte = (w[j >> 2] >> (8 * (j & 3))) & 0xffu;
            c[j] = SIGNED ? static_cast<int>(static_cast<int8_t>(byte)) : static_cast<int>(byte);
        }
    } else if (BITS == 4) {
        const uint32_t w = *reinterpret_cast<const uint32_t*>(row + (k0 >> 1));
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const int nib = static_cast<int>((w >> (8 * (j & 3) + (j >= 4 ? 4 : 0))) & 0xfu);
            c[j] = (SIGNED && nib >= 8) ? nib - 16 : nib;
        }
    } else {
        const int blk = k0 >> 7, r = k0 & 127;
        const int t = r >> 5, sft = (r & 31) >> 3;
        const uint8_t* base = row + blk * 16 * BITS + t * 4;
        uint32_t w[BITS];
#pragma unroll
        for (int p = 0; p < BITS; ++p) w[p] = *reinterpret_cast<const uint32_t*>(base + p * 16) >> sft;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const int pos = (j < 4) ? 8 * j : 8 * (j - 4) + 4;
            int v = 0;
#pragma unroll
            for (int p = 0; p < BITS; ++p) v |= static_cast<int>((w[p] >> pos) & 1u) << p;
            c[j] = v;
        }
    }
}

#endif  // __CUDACC__

}  // namespace mixdq
