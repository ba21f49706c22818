// Pieces of the exact top-n_q selection (Section 3.2.2: the entries with the largest error are
// kept) shared by the kernels that read materialised errors and those that work on value tables.
#pragma once

#include "common.cuh"

namespace cmpq {

constexpr int kSelBins = 4096;
constexpr int kSelThreads = 256;

struct SelectState {
    uint32_t prefix;        // bits of tau fixed so far
    uint32_t mask;          // which bits are fixed
    long long remaining;    // entries still to take among those matching prefix
    uint32_t tau;           // final threshold pattern
    long long take_equal;   // entries equal to tau that belong to the set
};

__device__ __forceinline__ int block_exclusive_scan(int v, int* warp_totals, int& total) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    int incl = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        int up = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += up;
    }
    __syncthreads();  // warp_totals may still be read from a previous call
    if (lane == 31) warp_totals[warp] = incl;
    __syncthreads();
    int base = 0, all = 0;
    for (int w = 0; w < nwarps; ++w) {
        int t = warp_totals[w];
        if (w < warp) base += t;
        all += t;
    }
    total = all;
    return base + incl - v;
}

constexpr int kEmitListCap = 1024;  // candidates of a row ordered in shared memory; more: scan-based compaction

}  // namespace cmpq
