// Channel-wise precision allocation of CMPQ (Algorithm 1).
//
// The allocation only needs the rank of every channel in the ascending order of (a, id).
// d_in is at most a few tens of thousands, so the rank is counted directly: channel i's rank
// is the number of channels that sort before it.  The count is exact, needs no sort network
// and is spread over (channel tile) x (candidate slice) blocks that add integer partial counts.
#include "common.cuh"

namespace cmpq {

constexpr int kRankThreads = 256;
constexpr int kRankSlice = 256;   // candidates one block compares against

size_t alloc_ws_bytes(int64_t d_in) {
    return 2 * round_up((size_t)d_in * sizeof(int32_t), 256);
}

// rank[i] += #{ j in slice : (a_j, j) < (a_i, i) }
__global__ void __launch_bounds__(kRankThreads)
rank_count_kernel(const float* __restrict__ a, int64_t d_in, int32_t* __restrict__ rank) {
    __shared__ float tile[kRankThreads];
    const int64_t i = (int64_t)blockIdx.x * kRankThreads + threadIdx.x;
    const float ai = i < d_in ? a[i] : 0.f;
    const int64_t j0 = (int64_t)blockIdx.y * kRankSlice;
    int64_t j1 = j0 + kRankSlice;
    if (j1 > d_in) j1 = d_in;
    int count = 0;
    for (int64_t base = j0; base < j1; base += kRankThreads) {
        int64_t j = base + threadIdx.x;
        __syncthreads();
        tile[threadIdx.x] = j < j1 ? a[j] : 0.f;
        __syncthreads();
        int lim = (int)min((int64_t)kRankThreads, j1 - base);
        for (int t = 0; t < lim; ++t) {
            float aj = tile[t];
            count += (aj < ai || (aj == ai && base + t < i)) ? 1 : 0;
        }
    }
    if (i < d_in && count) atomicAdd(&rank[i], count);
}

__global__ void rank_scatter_kernel(const int32_t* __restrict__ rank, int64_t d_in, int64_t n2,
                                    int64_t n4, uint8_t* __restrict__ bits,
                                    int32_t* __restrict__ order) {
    int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= d_in) return;
    int64_t r = rank[i];
    if (order) order[r] = (int32_t)i;
    if (bits) bits[i] = r < n2 ? 2 : (r >= d_in - n4 ? 4 : 3);
}

__device__ double interp_quantile(const float* a, const int32_t* order, int64_t d_in, double q) {
    double pos = q * (double)(d_in - 1);
    if (pos < 0.0) pos = 0.0;
    if (pos > (double)(d_in - 1)) pos = (double)(d_in - 1);
    int64_t lo = (int64_t)floor(pos);
    int64_t hi = lo + 1 < d_in ? lo + 1 : lo;
    double frac = pos - (double)lo;
    double vlo = (double)a[order[lo]], vhi = (double)a[order[hi]];
    return __dadd_rn(vlo, __dmul_rn(vhi - vlo, frac));
}

// Algorithm 1 as printed: thresholds from interpolated quantiles, strict comparisons.
__global__ void quantile_bits_kernel(const float* __restrict__ a, const int32_t* __restrict__ order,
                                     int64_t d_in, double avg_bits, uint8_t* __restrict__ bits) {
    __shared__ double thr[2];
    if (threadIdx.x == 0) {
        if (avg_bits > 3.0) {
            thr[1] = interp_quantile(a, order, d_in, 1.0 - (avg_bits - 3.0));
        } else if (avg_bits < 3.0) {
            thr[0] = interp_quantile(a, order, d_in, 3.0 - avg_bits);
        } else {
            thr[0] = interp_quantile(a, order, d_in, 0.01);
            thr[1] = interp_quantile(a, order, d_in, 0.99);
        }
    }
    __syncthreads();
    int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= d_in) return;
    double v = (double)a[i];
    uint8_t c = 3;
    if (avg_bits <= 3.0 && v < thr[0]) c = 2;
    if (avg_bits >= 3.0 && v > thr[1]) c = 4;
    bits[i] = c;
}

// rank[i] = position of channel i in the ascending order of (a, id).  rank must hold d_in ints.
cmpq_status launch_rank(const float* a, int64_t d_in, int32_t* rank, cudaStream_t st) {
    if (cudaMemsetAsync(rank, 0, (size_t)d_in * sizeof(int32_t), st) != cudaSuccess) return CMPQ_ERR_CUDA;
    dim3 grid((unsigned)((d_in + kRankThreads - 1) / kRankThreads), (unsigned)((d_in + kRankSlice - 1) / kRankSlice));
    rank_count_kernel<<<grid, kRankThreads, 0, st>>>(a, d_in, rank);
    return launch_status();
}

}  // namespace cmpq

using namespace cmpq;

extern "C" void cmpq_alloc_counts(int64_t d_in, double avg_bits, int64_t* n2, int64_t* n4) {
    int64_t two = 0, four = 0;
    if (avg_bits == 3.0) {
        two = four = (int64_t)floor(0.01 * (double)d_in + 0.5);
    } else {
        int64_t n = (int64_t)floor(fabs(avg_bits - 3.0) * (double)d_in + 0.5);
        if (n > d_in) n = d_in;
        if (avg_bits > 3.0) four = n; else two = n;
    }
    if (n2) *n2 = two;
    if (n4) *n4 = four;
}

extern "C" cmpq_status cmpq_allocate_bits(const float* a, int64_t d_in, double avg_bits,
                                          cmpq_alloc_mode mode, uint8_t* bits, int32_t* order,
                                          void* ws, size_t ws_bytes, void* stream) {
    if (!a || !bits || d_in < 1 || d_in > CMPQ_MAX_D_IN) return CMPQ_ERR_INVALID_ARG;
    if (!(avg_bits >= 2.0 && avg_bits <= 4.0)) return CMPQ_ERR_INVALID_ARG;
    if (mode != CMPQ_ALLOC_RANK && mode != CMPQ_ALLOC_QUANTILE) return CMPQ_ERR_INVALID_ARG;
    if (!ws || !aligned_to(ws, 256) || ws_bytes < alloc_ws_bytes(d_in)) return CMPQ_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    Workspace w(ws, ws_bytes);
    int32_t* rank = w.take<int32_t>(d_in);
    int32_t* order_ws = w.take<int32_t>(d_in);
    cmpq_status s = launch_rank(a, d_in, rank, st);
    if (s != CMPQ_OK) return s;
    int64_t n2 = 0, n4 = 0;
    cmpq_alloc_counts(d_in, avg_bits, &n2, &n4);
    const unsigned blocks = (unsigned)((d_in + 255) / 256);
    if (mode == CMPQ_ALLOC_RANK) {
        rank_scatter_kernel<<<blocks, 256, 0, st>>>(rank, d_in, n2, n4, bits, order);
    } else {
        int32_t* ord = order ? order : order_ws;
        rank_scatter_kernel<<<blocks, 256, 0, st>>>(rank, d_in, 0, 0, nullptr, ord);
        quantile_bits_kernel<<<blocks, 256, 0, st>>>(a, ord, d_in, avg_bits, bits);
    }
    return launch_status();
}
