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

// One block (any multiple of 32 threads, called by all of them): segment sizes, perm, row_off (segment order) and word_off (by channel id).
// Thread t owns the consecutive channels [t R, t R + R); the three per-width counts travel through
// one block-wide scan packed into a 64-bit integer (21 bits each, d_in <= 2^18).
__device__ __forceinline__ void pack_layout_block(const uint8_t* __restrict__ bits, int64_t d_in, int64_t d_out,
                                                  int64_t* __restrict__ row_off, int32_t* __restrict__ perm,
                                                  int64_t* __restrict__ seg_rows, int64_t* __restrict__ word_off,
                                                  unsigned long long* warp_tot /* 32 words of shared memory */) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nwarps = blockDim.x >> 5;
    const int64_t R = (d_in + blockDim.x - 1) / blockDim.x;
    const int64_t i0 = (int64_t)tid * R;
    const int64_t i1 = i0 + R < d_in ? i0 + R : d_in;
    unsigned long long mine = 0;
    for (int64_t i = i0; i < i1; ++i) {
        int c = bits[i];
        if (c >= 2 && c <= 4) mine += 1ull << (21 * (c - 2));
    }
    unsigned long long incl = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        unsigned long long up = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += up;
    }
    if (lane == 31) warp_tot[warp] = incl;
    __syncthreads();
    // lane w holds the total of warp w: the three 21-bit fields are summed separately, over the warps below
    // this one and over all of them
    const unsigned long long wt = lane < nwarps ? warp_tot[lane] : 0ull;
    const unsigned long long own = incl - mine;
    long long seen[3], count[3], words[3], seg_base[3], seg_word_base[3];
    long long rb = 0, wb = 0;
#pragma unroll
    for (int sgm = 0; sgm < 3; ++sgm) {
        const unsigned f = (unsigned)((wt >> (21 * sgm)) & 0x1fffffull);
        seen[sgm] = (long long)(__reduce_add_sync(0xffffffffu, lane < warp ? f : 0u) +
                                (unsigned)((own >> (21 * sgm)) & 0x1fffffull));
        count[sgm] = (long long)__reduce_add_sync(0xffffffffu, f);
        words[sgm] = (d_out * (sgm + 2) + 31) / 32;
        seg_base[sgm] = rb;
        seg_word_base[sgm] = wb;
        rb += count[sgm];
        wb += count[sgm] * words[sgm];
    }
    if (tid < 3) seg_rows[tid] = count[tid];
    if (tid == 0) row_off[d_in] = wb;
    for (int64_t i = i0; i < i1; ++i) {
        int c = bits[i];
        if (c < 2 || c > 4) continue;
        int sgm = c - 2;
        long long pos = seen[sgm]++;
        long long r = seg_base[sgm] + pos;
        long long off = seg_word_base[sgm] + pos * words[sgm];
        perm[r] = (int32_t)i;
        row_off[r] = off;
        word_off[i] = off;
    }
}

}  // namespace cmpq
