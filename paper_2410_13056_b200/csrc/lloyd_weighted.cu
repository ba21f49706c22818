// Channel-wise K-means with per-weight sensitivities (the weighted form of the quantizer of Section 3:
// the centroid update becomes the weighted mean  c_k = sum s_i x_i / sum s_i  over the cluster's members,
// the assignment stays the nearest centroid).  Start, tie and rounding rules are those of the unweighted fit:
// start at K evenly spaced order statistics of the channel, first minimum of fabsf(x - c_k) in fp32, sums in
// fp64, one fp64 divide, one rounding to fp32, an empty cluster keeps its centroid.
//
// One block per channel, the channel resident in shared memory as fp32 for all iterations (HBM traffic: the
// weights and their sensitivities once per iteration from L2, codes once).  The products s_i x_i are not
// exact in fp64, so cluster sums depend on the order of summation: the order here is fixed (thread-strided
// partial sums, a fixed tree inside each warp, the warps in order), which makes the result deterministic, but it is not the index order of a
// sequential sum -- results agree with such a sum to rounding, not bit for bit.
#include "common.cuh"
#include "lloyd.cuh"

namespace cmpq {

constexpr int kWThreads = 256;
constexpr int kWWarps = kWThreads / 32;

// Order-preserving 16-bit key of a finite fp16/bf16 pattern (ascending key = ascending value); -0 maps to +0's key.
__device__ __forceinline__ uint32_t ordered_key(uint16_t h) {
    if (h == 0x8000u) h = 0;
    return (h & 0x8000u) ? (uint32_t)(uint16_t)~h : (uint32_t)(h | 0x8000u);
}
__device__ __forceinline__ uint16_t key_pattern(uint32_t key) {
    return (key & 0x8000u) ? (uint16_t)(key & 0x7fffu) : (uint16_t)~key;
}

// Nearest centroid of every weight of the channel (first minimum of fabsf(x - c_k), k ascending), the K
// centroids held in registers.
template <int K>
__device__ __forceinline__ void assign_codes(const float* __restrict__ x, const float* c, int N, uint8_t* out) {
    float cr[K];
#pragma unroll
    for (int k = 0; k < K; ++k) cr[k] = c[k];
    for (int j = threadIdx.x; j < N; j += kWThreads) {
        const float v = x[j];
        int best = 0;
        float bd = fabsf(v - cr[0]);
#pragma unroll
        for (int k = 1; k < K; ++k) {
            const float d = fabsf(v - cr[k]);
            if (d < bd) {
                bd = d;
                best = k;
            }
        }
        out[j] = (uint8_t)best;
    }
}

__device__ __forceinline__ void assign_codes(int K, const float* __restrict__ x, const float* c, int N, uint8_t* out) {
    if (K == 4) assign_codes<4>(x, c, N, out);
    else if (K == 8) assign_codes<8>(x, c, N, out);
    else assign_codes<16>(x, c, N, out);
}

template <int DT>
__global__ void __launch_bounds__(kWThreads)
lloyd_weighted_kernel(const uint16_t* __restrict__ W, int64_t d_out, int64_t ldw, const uint8_t* __restrict__ bits,
                      const int64_t* __restrict__ row_ptr, const int32_t* __restrict__ cols,
                      const float* __restrict__ sens, int iters, float* __restrict__ lut,
                      uint8_t* __restrict__ codes, unsigned long long* __restrict__ sweeps,
                      const uint8_t* __restrict__ skip_row) {
    extern __shared__ __align__(16) unsigned char smem[];
    if (skip_row != nullptr && skip_row[blockIdx.x]) return;  // fitted elsewhere (the whole block leaves)
    float* x = reinterpret_cast<float*>(smem);                       // [d_out]
    uint8_t* code = reinterpret_cast<uint8_t*>(x + d_out);           // [d_out]
    __shared__ int hist_hi[256];
    __shared__ int hist_lo[16][256];
    __shared__ int bin_of[16], rank_in_bin[16];
    __shared__ float c[16];
    __shared__ double warp_sums[16][kWWarps][2];  // per cluster and warp: sum of s*x, sum of s
    __shared__ int changed;
    const int64_t i = blockIdx.x;
    const int tid = threadIdx.x;
    const int width = bits[i];
    const int K = 1 << (width < 2 ? 2 : (width > 4 ? 4 : width));
    const uint16_t* w = W + i * ldw;
    const float* s = sens + i * d_out;
    const int N = (int)d_out;

    // ordered keys of W'' (listed positions are +0) for the start; they share the slots of the fp32 values,
    // which replace them once the start is known
    uint32_t* xkey = reinterpret_cast<uint32_t*>(x);
    for (int j = tid; j < N; j += kWThreads) xkey[j] = ordered_key(w[j]);
    for (int j = tid; j < 256; j += kWThreads) hist_hi[j] = 0;
    for (int j = tid; j < 16 * 256; j += kWThreads) (&hist_lo[0][0])[j] = 0;
    __syncthreads();
    if (row_ptr != nullptr)
        for (int64_t p = row_ptr[i] + tid; p < row_ptr[i + 1]; p += kWThreads) xkey[cols[p]] = ordered_key(0);
    __syncthreads();
    // start: the ((2k+1) N) / (2K)-th smallest value, by a two-level count over the 16-bit keys
    for (int j = tid; j < N; j += kWThreads) atomicAdd(&hist_hi[xkey[j] >> 8], 1);
    __syncthreads();
    if (tid < K) {
        const int target = (int)(((int64_t)(2 * tid + 1) * N) / (2 * (int64_t)K));
        int cum = 0, b = 0;
        for (; b < 256; ++b) {
            if (target < cum + hist_hi[b]) break;
            cum += hist_hi[b];
        }
        bin_of[tid] = b;
        rank_in_bin[tid] = target - cum;
    }
    __syncthreads();
    for (int j = tid; j < N; j += kWThreads) {
        const uint32_t key = xkey[j];
        for (int k = 0; k < K; ++k)
            if ((int)(key >> 8) == bin_of[k]) atomicAdd(&hist_lo[k][key & 255u], 1);
    }
    __syncthreads();
    if (tid < K) {
        int cum = 0, b = 0;
        for (; b < 256; ++b) {
            if (rank_in_bin[tid] < cum + hist_lo[tid][b]) break;
            cum += hist_lo[tid][b];
        }
        c[tid] = widen16<DT>(key_pattern(((uint32_t)bin_of[tid] << 8) | (uint32_t)b)) + 0.0f;
    }
    __syncthreads();
    // keys -> values (x_i + 0.0f canonicalises -0)
    for (int j = tid; j < N; j += kWThreads) x[j] = widen16<DT>(key_pattern(xkey[j])) + 0.0f;  // own slot only
    __syncthreads();

    int done = 0;
    for (int it = 0; it < iters; ++it) {
        if (tid == 0) changed = 0;  // ordered before the updates by the barrier after the assignment
        assign_codes(K, x, c, N, code);
        __syncthreads();
        // update: weighted mean of each cluster's members.  Every thread sums its own weights of cluster k,
        // a warp adds its lanes in a fixed tree, and after ONE barrier thread k adds the warps in order.
        for (int k = 0; k < K; ++k) {
            double S = 0.0, n = 0.0;
            for (int j = tid; j < N; j += kWThreads)
                if (code[j] == k) {
                    const double sj = (double)s[j];
                    S += sj * (double)x[j];
                    n += sj;
                }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                S += __shfl_down_sync(0xffffffffu, S, o);
                n += __shfl_down_sync(0xffffffffu, n, o);
            }
            if ((tid & 31) == 0) {
                warp_sums[k][tid >> 5][0] = S;
                warp_sums[k][tid >> 5][1] = n;
            }
        }
        __syncthreads();
        if (tid < K) {
            double S = 0.0, n = 0.0;
#pragma unroll
            for (int wq = 0; wq < kWWarps; ++wq) {
                S += warp_sums[tid][wq][0];
                n += warp_sums[tid][wq][1];
            }
            if (n > 0.0) {
                const float nc = (float)(S / n);
                if (__float_as_uint(nc) != __float_as_uint(c[tid])) changed = 1;
                c[tid] = nc;
            }
        }
        __syncthreads();
        ++done;
        const int moved = changed;
        __syncthreads();           // everyone has read the flag before the next iteration clears it
        if (!moved) break;         // every later iteration would repeat this one
    }
    // last assignment and outputs
    assign_codes(K, x, c, N, codes + i * d_out);
    if (tid < CMPQ_LUT_STRIDE) lut[i * CMPQ_LUT_STRIDE + tid] = tid < K ? c[tid] : 0.0f;
    if (sweeps != nullptr && tid == 0) atomicAdd(sweeps, (unsigned long long)(done + 1) * (unsigned long long)N * K);
}

cmpq_status launch_lloyd_weighted(const LloydArgs& a, cmpq_dtype dt, const float* sens, cudaStream_t st) {
    const size_t smem = (size_t)a.d_out * 5 + 16;
    static bool raised[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return CMPQ_ERR_CUDA;
    if (dev < 0 || dev >= 64 || !raised[dev]) {
        const int limit = CMPQ_MAX_D_OUT * 5 + 16;
        if (cudaFuncSetAttribute(lloyd_weighted_kernel<CMPQ_F16>, cudaFuncAttributeMaxDynamicSharedMemorySize, limit) != cudaSuccess ||
            cudaFuncSetAttribute(lloyd_weighted_kernel<CMPQ_BF16>, cudaFuncAttributeMaxDynamicSharedMemorySize, limit) != cudaSuccess)
            return CMPQ_ERR_CUDA;
        if (dev >= 0 && dev < 64) raised[dev] = true;
    }
    if (dt == CMPQ_F16)
        lloyd_weighted_kernel<CMPQ_F16><<<(unsigned)a.d_in, kWThreads, smem, st>>>(
            a.W, a.d_out, a.ldw, a.bits, a.row_ptr, a.cols, sens, a.iters, a.lut, a.codes, a.sweeps, a.skip_row);
    else
        lloyd_weighted_kernel<CMPQ_BF16><<<(unsigned)a.d_in, kWThreads, smem, st>>>(
            a.W, a.d_out, a.ldw, a.bits, a.row_ptr, a.cols, sens, a.iters, a.lut, a.codes, a.sweeps, a.skip_row);
    return launch_status();
}

}  // namespace cmpq
