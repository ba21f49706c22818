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
    unsigned int done;      // blocks of the running histogram kernel that have added their counts
    uint32_t lower;         // an error pattern known not to exceed tau (0: nothing known)
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
    const int t = lane < nwarps ? warp_totals[lane] : 0;  // at most 32 warps: one total per lane
    total = __reduce_add_sync(0xffffffffu, t);
    return __reduce_add_sync(0xffffffffu, lane < warp ? t : 0) + incl - v;
}

// One block: walks the histogram from the largest digit down to the one that holds the
// remaining-th largest entry, fixes that digit in the prefix and clears the histogram for the next
// pass.  THREADS = blockDim.x; the histogram is read past the L1 cache (other blocks wrote it).
template <int THREADS>
__device__ __forceinline__ void select_digit_block(unsigned int* hist, int shift, int bins, SelectState* st,
                                                   int final_pass, int* warp_totals, int* found_digit,
                                                   long long* found_above) {
    constexpr int per = kSelBins / THREADS;  // bins per thread, descending digit order
    const long long remaining = st->remaining;
    int v[per], s = 0;
#pragma unroll
    for (int t = 0; t < per; ++t) {
        const int d = bins - 1 - (threadIdx.x * per + t);
        v[t] = d >= 0 ? (int)__ldcg(hist + d) : 0;
        s += v[t];
    }
    if (threadIdx.x == 0) *found_digit = -1;
    int total;
    long long above = block_exclusive_scan(s, warp_totals, total);  // entries with a larger digit
    if (remaining > 0 && above < remaining && remaining <= above + s) {
#pragma unroll
        for (int t = 0; t < per; ++t) {
            if (above < remaining && remaining <= above + v[t]) {
                *found_digit = bins - 1 - (threadIdx.x * per + t);
                *found_above = above;
            }
            above += v[t];
        }
    }
    __syncthreads();
    if (threadIdx.x == 0 && *found_digit >= 0) {
        st->prefix |= (uint32_t)*found_digit << shift;
        st->mask |= (uint32_t)(bins - 1) << shift;
        st->remaining = remaining - *found_above;
        if (final_pass) { st->tau = st->prefix; st->take_equal = st->remaining; }
    }
    for (int b = threadIdx.x; b < bins; b += THREADS) hist[b] = 0;
}

constexpr int kEmitListCap = 1024;  // candidates of a row ordered in shared memory; more: scan-based compaction

}  // namespace cmpq
