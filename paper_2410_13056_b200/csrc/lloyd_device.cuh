// Device helpers shared by the channel K-means kernels (Section 3.2.1; quantizer of Section 3):
// the order-preserving 16-bit key of a weight, warp scans, the nearest-centroid rule and the load
// of one channel with its exactness diagnostics.
#pragma once

#include "lloyd.cuh"

namespace cmpq {

constexpr int kMaxK = 16;

template <int DT>
__device__ __forceinline__ uint32_t sort_key16(float x) {
    uint32_t h;
    if (DT == CMPQ_BF16) h = __float_as_uint(x) >> 16;
    else h = __half_as_ushort(__float2half_rn(x));
    return (h & 0x8000u) ? (~h & 0xffffu) : (h | 0x8000u);
}

template <int DT>
__device__ __forceinline__ float value_of_key16(uint32_t key) {
    uint32_t h = (key & 0x8000u) ? (key & 0x7fffu) : (~key & 0xffffu);
    return widen16<DT>((uint16_t)h);
}

__device__ __forceinline__ int warp_sum(int v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// exclusive prefix of 256 counters by one warp (8 per lane, in place allowed); returns the total
__device__ __forceinline__ int warp_scan256(const int* in, int* out_excl) {
    const int lane = threadIdx.x & 31;
    int v[8], s = 0;
#pragma unroll
    for (int t = 0; t < 8; ++t) { v[t] = in[lane * 8 + t]; s += v[t]; }
    int incl = s;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        int up = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += up;
    }
    int run = incl - s;
    __syncwarp();
#pragma unroll
    for (int t = 0; t < 8; ++t) { out_excl[lane * 8 + t] = run; run += v[t]; }
    return __shfl_sync(0xffffffffu, incl, 31);
}

// Code of one weight by the defining scan: first k minimising |x - c_k|.
template <int K>
__device__ __forceinline__ int nearest_scan(float x, const float (&c)[K]) {
    float best = fabsf(x - c[0]);
    int bk = 0;
#pragma unroll
    for (int k = 1; k < K; ++k) {
        float d = fabsf(x - c[k]);
        if (d < best) { best = d; bk = k; }
    }
    return bk;
}

// Whether the counting sweep is valid for the centroids (lane k holds c_k): strictly increasing
// with every gap above 2^-22 of the channel's value range.  Same answer in every lane.
template <int K>
__device__ __forceinline__ bool counting_sweep_valid(float ck_lane, double need) {
    const int lane = threadIdx.x & 31;
    float ck = __shfl_sync(0xffffffffu, ck_lane, lane < K ? lane : K - 1);
    float cp = __shfl_up_sync(0xffffffffu, ck, 1);
    bool ok = (lane == 0 || lane >= K) ? true : ((double)ck - (double)cp > need);
    return __all_sync(0xffffffffu, ok);
}

// Reads channel `row` (all threads of the block), sets the removed positions to +0 and returns the
// weights as sort keys: key[e] belongs to column ((e >> 2) * nthr + tid) * 4 + (e & 3), the first
// nval_cols of a thread's keys are real.  `removed` is shared scratch of at least d_out bits, free
// again when the function returns.  Also leaves the channel's value range in sh.vmin / sh.vmax
// (written by thread 0 after the function's last barrier: published by the caller's next one) and
// counts the channel in a.inexact_rows when its dynamic range is too wide for exact fp64 sums.
// Sh needs the members vmin, vmax, wlo, whi, wtop, wulp.
template <int DT, int E, class Sh>
__device__ __forceinline__ void load_channel_keys(const LloydArgs& a, int64_t row, Sh& sh, uint32_t* removed,
                                                  uint32_t (&key)[E], int& nval_cols) {
    const int N = (int)a.d_out;
    const int tid = threadIdx.x, nthr = blockDim.x, lane = tid & 31, warp = tid >> 5;
    const int nwarps = nthr >> 5;
    // removed positions (outliers of this row) are marked in a bitmap over the columns
    int64_t p0 = 0, p1 = 0;
    if (a.row_ptr) { p0 = a.row_ptr[row]; p1 = a.row_ptr[row + 1]; }
    const bool has_removed = p1 > p0;
    if (has_removed) {
        for (int w = tid; w < (N + 31) / 32; w += nthr) removed[w] = 0;
        __syncthreads();
        for (int64_t p = p0 + tid; p < p1; p += nthr) {
            int col = a.cols[p];
            atomicOr(&removed[col >> 5], 1u << (col & 31));
        }
        __syncthreads();
    }

    // column layout for the load: thread owns columns (g * nthr + tid) * 4 + u
    const uint16_t* w = a.W + row * a.ldw;
    const bool vec = ((a.ldw & 3) == 0) && ((reinterpret_cast<uintptr_t>(a.W) & 7) == 0);
    nval_cols = 0;
    {
        float lo = __int_as_float(0x7f800000), hi = __int_as_float(0xff800000);
        uint32_t amax = 0u, amin1 = 0xffffffffu;  // largest |x| pattern; smallest non-zero |x| pattern minus 1
#pragma unroll
        for (int g = 0; g < E / 4; ++g) {
            const int j0 = (g * nthr + tid) * 4;
            uint16_t h[4] = {0, 0, 0, 0};
            if (j0 + 3 < N && vec) {
                uint2 v = *reinterpret_cast<const uint2*>(w + j0);
                h[0] = (uint16_t)(v.x & 0xffff); h[1] = (uint16_t)(v.x >> 16);
                h[2] = (uint16_t)(v.y & 0xffff); h[3] = (uint16_t)(v.y >> 16);
            } else {
#pragma unroll
                for (int u = 0; u < 4; ++u)
                    if (j0 + u < N) h[u] = w[j0 + u];
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int j = j0 + u;
                float v = widen16<DT>(h[u]);
                if (j < N) {
                    ++nval_cols;
                    if (has_removed && ((removed[j >> 5] >> (j & 31)) & 1)) v = 0.f;
                    v = (v == 0.f) ? 0.f : v;  // -0 and +0 are the same point
                    lo = fminf(lo, v);
                    hi = fmaxf(hi, v);
                    const uint32_t ub = __float_as_uint(v) & 0x7fffffffu;
                    amax = max(amax, ub);
                    amin1 = min(amin1, ub - 1u);  // zero wraps to the largest value
                }
                key[4 * g + u] = sort_key16<DT>(v);
            }
        }
        // value range (for the gap test) and the magnitude range (for the exactness test)
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            lo = fminf(lo, __shfl_xor_sync(0xffffffffu, lo, o));
            hi = fmaxf(hi, __shfl_xor_sync(0xffffffffu, hi, o));
            amax = max(amax, __shfl_xor_sync(0xffffffffu, amax, o));
            amin1 = min(amin1, __shfl_xor_sync(0xffffffffu, amin1, o));
        }
        if (lane == 0) { sh.wlo[warp] = lo; sh.whi[warp] = hi; sh.wtop[warp] = (int)amax; sh.wulp[warp] = (int)amin1; }
        __syncthreads();  // also: every thread is done with the removed-column bitmap
        // every warp reduces the per-warp values again, so the decision below is the same in all threads
        amax = lane < nwarps ? (uint32_t)sh.wtop[lane] : 0u;
        amin1 = lane < nwarps ? (uint32_t)sh.wulp[lane] : 0xffffffffu;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            amax = max(amax, __shfl_xor_sync(0xffffffffu, amax, o));
            amin1 = min(amin1, __shfl_xor_sync(0xffffffffu, amin1, o));
        }
        if (tid == 0) {
            for (int wv = 1; wv < nwarps; ++wv) {
                lo = fminf(lo, sh.wlo[wv]);
                hi = fmaxf(hi, sh.whi[wv]);
            }
            sh.vmin = lo;
            sh.vmax = hi;
        }
        // Sums and differences of up to 2N weights stay exact in fp64 while 2 N 2^(top+1) / 2^q <= 2^53,
        // top = exponent of the largest magnitude, 2^q = smallest unit in the last place of a non-zero
        // weight.  First with a lower bound of q from the smallest magnitude's exponent and the trailing
        // zero bits every widened 16-bit value has; only a channel that fails this is examined bit by bit.
        if (a.nonfinite && tid == 0 && amax >= 0x7f800000u) atomicOr(a.nonfinite, 2);  // a NaN or an infinity
        if (a.inexact_rows && amax != 0u) {
            const int log2n = 32 - __clz(N - 1 > 0 ? N - 1 : 1);
            const int ex_max = (int)(amax >> 23), ex_min = (int)((amin1 + 1u) >> 23);
            const int top = ex_max ? ex_max - 127 : (31 - __clz(amax)) - 149;
            const int q_low = (ex_min ? ex_min - 150 : -149) + (DT == CMPQ_BF16 ? 16 : 13);
            if (log2n + 1 + (top + 1 - q_low) > 53) {  // same value in every thread of the block
                int q = 100000;
#pragma unroll
                for (int e = 0; e < E; ++e) {
                    const uint32_t ub = __float_as_uint(value_of_key16<DT>(key[e])) & 0x7fffffffu;
                    if (e < nval_cols && ub) {
                        const int ex = (int)(ub >> 23);
                        const uint32_t m = ub & 0x7fffffu;
                        q = min(q, ex ? ex - 150 + (__ffs(m | 0x800000u) - 1) : (__ffs(m) - 1) - 149);
                    }
                }
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) q = min(q, __shfl_xor_sync(0xffffffffu, q, o));
                __syncthreads();  // every warp has read wtop / wulp
                if (lane == 0) sh.wulp[warp] = q;
                __syncthreads();
                if (tid == 0) {
                    for (int wv = 1; wv < nwarps; ++wv) q = min(q, sh.wulp[wv]);
                    if (log2n + 1 + (top + 1 - q) > 53) atomicAdd(a.inexact_rows, 1);
                }
            }
        }
    }
}

}  // namespace cmpq
