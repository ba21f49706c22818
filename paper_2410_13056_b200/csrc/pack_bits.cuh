// Bit-level packing of byte codes shared by the packing kernel and the last assignment of the K-means
// (packed layout: a channel's codes form an LSB-first bit stream of C bits each, cut into 32-bit words).
#pragma once

#include <stdint.h>

namespace cmpq {

// Four codes held one per byte -> one 4C-bit field (C bits each, first code lowest).
template <int C>
__device__ __forceinline__ uint32_t squeeze4(uint32_t x) {
    constexpr uint32_t m1 = ((1u << (2 * C)) - 1u) * 0x00010001u;
    constexpr uint32_t m2 = (C == 4) ? 0xffffu : ((1u << (4 * C)) - 1u);
    x &= ((1u << C) - 1u) * 0x01010101u;  // ignore anything above the channel's width
    uint32_t t = (x | (x >> (8 - C))) & m1;
    return (t | (t >> (16 - 2 * C))) & m2;
}

template <int C>
__device__ __forceinline__ void pack32(const uint32_t (&b)[8], uint32_t (&w)[4]) {
    uint32_t r[8];
#pragma unroll
    for (int q = 0; q < 8; ++q) r[q] = squeeze4<C>(b[q]);
    if (C == 2) {
        w[0] = r[0] | (r[1] << 8) | (r[2] << 16) | (r[3] << 24);
        w[1] = r[4] | (r[5] << 8) | (r[6] << 16) | (r[7] << 24);
        w[2] = w[3] = 0;
    } else if (C == 3) {
        w[0] = r[0] | (r[1] << 12) | (r[2] << 24);
        w[1] = (r[2] >> 8) | (r[3] << 4) | (r[4] << 16) | (r[5] << 28);
        w[2] = (r[5] >> 4) | (r[6] << 8) | (r[7] << 20);
        w[3] = 0;
    } else {
        w[0] = r[0] | (r[1] << 16);
        w[1] = r[2] | (r[3] << 16);
        w[2] = r[4] | (r[5] << 16);
        w[3] = r[6] | (r[7] << 16);
    }
}

}  // namespace cmpq
