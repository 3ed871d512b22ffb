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

#endif  // __CUDACC__

}  // namespace mixdq
