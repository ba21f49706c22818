// Channel-wise precision allocation of CMPQ (Algorithm 1).
//
// The allocation only needs the rank of every channel in the ascending order of (a, id).
// d_in is at most a few tens of thousands, so the rank is counted directly: channel i's rank
// is the number of channels that sort before it.  The count is exact, needs no sort network
// and is spread over (channel tile) x (candidate slice) blocks that add integer partial counts.
#include "common.cuh"
#include "pack_bits.cuh"
#include "select.cuh"

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

// ------------------------------------------------------------------------------------------------
// Classification without a full rank.  Algorithm 1 in rank form and the choice of the O_act channels
// (Section 3.2.2) only ask on which side of one or two rank cuts a channel lies.  One block finds, for
// each cut k, the element of rank k in the ascending order of (a, id) by an exact radix select over the
// order-preserving bit pattern of a (8-bit digits, both cuts at once), then every channel is
// compared with the cut elements; equal statistics are ordered by channel id through a prefix count.
constexpr int kCutThreads = 1024;
constexpr int kCutRegKeys = 8;  // statistics per thread held in registers

__device__ __forceinline__ uint32_t ordered_bits(float v) {
    const uint32_t u = __float_as_uint(v + 0.0f);  // -0 and +0 are the same value
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// Small per-layer steps that ride along with a rank-cut launch (a second block, nothing else running yet):
// the layout of the packed segments from the widths, and the start state of the radix select.
struct CutExtras {
    const uint8_t* bits;     // pack layout wanted: widths, and its five outputs
    int64_t d_out;
    int64_t* row_off;
    int32_t* perm;
    int64_t* seg_rows;
    int64_t* word_off;
    SelectState* select;     // select start state wanted: entries to take, histogram to clear
    long long n_q;
    unsigned int* hist;
};

// out[i] = base + #{ t in {0,1} : channel i has rank >= k_t }.  k_t >= d_in: no channel reaches cut t.
__global__ void __launch_bounds__(kCutThreads)
rank_cut_kernel(const float* __restrict__ a, int64_t d_in, long long k0, long long k1, int base,
                uint8_t* __restrict__ out, const CutExtras x) {
    __shared__ unsigned int hist[2][256];
    __shared__ uint32_t prefix[2];
    __shared__ long long remaining[2];  // rank of the cut element among the elements matching the prefix
    __shared__ unsigned long long warp_tot[32];
    __shared__ uint32_t warp_min[32], warp_max[32];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (blockIdx.x == 1) {  // the steps that ride along need nothing from the cut: a block of their own
        if (x.select) {
            if (tid == 0) {
                SelectState* st = x.select;
                st->prefix = 0; st->mask = 0; st->remaining = x.n_q; st->tau = 0xffffffffu; st->take_equal = 0; st->done = 0; st->lower = 0;
            }
            for (int b = tid; b < kSelBins; b += kCutThreads) x.hist[b] = 0u;
        }
        if (x.bits) pack_layout_block(x.bits, d_in, x.d_out, x.row_off, x.perm, x.seg_rows, x.word_off, warp_tot);
        return;
    }
    const long long k[2] = {k0, k1};
    const bool live[2] = {k0 < d_in, k1 < d_in};
    if (tid < 2) { prefix[tid] = 0u; remaining[tid] = k[tid] < 0 ? 0 : k[tid]; }
    // Up to kCutRegKeys patterns per thread stay in registers (channel u * kCutThreads + tid in slot u); a
    // longer statistic is read again in every pass.
    const bool in_regs = d_in <= (int64_t)kCutRegKeys * kCutThreads;
    const int n = (int)d_in;  // d_in <= CMPQ_MAX_D_IN fits
    uint32_t rk[kCutRegKeys];
    uint32_t kmin = 0xffffffffu, kmax = 0u;
    if (in_regs) {
#pragma unroll
        for (int u = 0; u < kCutRegKeys; ++u) {
            const int i = u * kCutThreads + tid;
            rk[u] = i < n ? ordered_bits(a[i]) : 0u;
            if (i < n) { kmin = min(kmin, rk[u]); kmax = max(kmax, rk[u]); }
        }
    } else {
        for (int i = tid; i < n; i += kCutThreads) {
            const uint32_t key = ordered_bits(a[i]);
            kmin = min(kmin, key);
            kmax = max(kmax, key);
        }
    }
    // The statistics of a layer share their leading bits.  The digits are therefore taken from the distance
    // to the smallest pattern, and only as many 8-bit digits as the largest distance has: the counters of a
    // pass are then hit evenly and a layer needs three passes rather than four.
    kmin = __reduce_min_sync(0xffffffffu, kmin);
    kmax = __reduce_max_sync(0xffffffffu, kmax);
    if (lane == 0) { warp_min[warp] = kmin; warp_max[warp] = kmax; }
    __syncthreads();
    kmin = __reduce_min_sync(0xffffffffu, warp_min[lane]);  // kCutThreads / 32 = 32 warps: one value per lane
    kmax = __reduce_max_sync(0xffffffffu, warp_max[lane]);
    if (in_regs) {
#pragma unroll
        for (int u = 0; u < kCutRegKeys; ++u) rk[u] -= kmin;
    }
    const int nbits = 32 - __clz(kmax - kmin);  // 0: all statistics are equal
    for (int pass = (nbits + 7) / 8 - 1; pass >= 0; --pass) {
        const int shift = 8 * pass;
        const uint32_t mask = shift + 8 >= 32 ? 0u : (0xffffffffu << (shift + 8));
        if (tid < 512) (&hist[0][0])[tid] = 0u;
        __syncthreads();
        const uint32_t p0 = prefix[0], p1 = prefix[1];
        auto count = [&](uint32_t key) {
            const uint32_t d = (key >> shift) & 255u;
            if (live[0] && (key & mask) == p0) atomicAdd(&hist[0][d], 1u);
            if (live[1] && (key & mask) == p1) atomicAdd(&hist[1][d], 1u);
        };
        if (in_regs) {
#pragma unroll
            for (int u = 0; u < kCutRegKeys; ++u)
                if (u * kCutThreads + tid < n) count(rk[u]);
        } else {
            for (int i = tid; i < n; i += kCutThreads) count(ordered_bits(a[i]) - kmin);
        }
        __syncthreads();
        if (warp < 2 && live[warp]) {  // warp t walks the histogram of cut t upwards
            unsigned int v[8], sum = 0;
#pragma unroll
            for (int u = 0; u < 8; ++u) { v[u] = hist[warp][lane * 8 + u]; sum += v[u]; }
            unsigned int incl = sum;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const unsigned int up = __shfl_up_sync(0xffffffffu, incl, o);
                if (lane >= o) incl += up;
            }
            const long long rem = remaining[warp];
            long long below = (long long)(incl - sum);
            if (below <= rem && rem < (long long)incl) {  // exactly one lane
#pragma unroll
                for (int u = 0; u < 8; ++u) {
                    if (below <= rem && rem < below + (long long)v[u]) {
                        prefix[warp] |= (uint32_t)(lane * 8 + u) << shift;
                        remaining[warp] = rem - below;
                        below = rem + 1;  // stop
                    } else {
                        below += v[u];
                    }
                }
            }
        }
        __syncthreads();
    }
    const uint32_t v0 = prefix[0], v1 = prefix[1];  // the cut elements, as distances to the smallest pattern
    const long long r0 = remaining[0], r1 = remaining[1];
    if ((!live[0] || r0 == 0) && (!live[1] || r1 == 0)) {
        // The cut element is the first of those equal to it in channel order (always so without ties): every
        // channel at or above the cut value is at or above the cut.
        auto classify = [&](int i, uint32_t key) {
            out[i] = (uint8_t)(base + ((live[0] && key >= v0) ? 1 : 0) + ((live[1] && key >= v1) ? 1 : 0));
        };
        if (in_regs) {
#pragma unroll
            for (int u = 0; u < kCutRegKeys; ++u)
                if (u * kCutThreads + tid < n) classify(u * kCutThreads + tid, rk[u]);
        } else {
            for (int i = tid; i < n; i += kCutThreads) classify(i, ordered_bits(a[i]) - kmin);
        }
    } else {
        // every thread owns a contiguous range of channels: how many statistics equal to a cut value precede it
        const int64_t per = (d_in + kCutThreads - 1) / kCutThreads;
        const int64_t c0 = (int64_t)tid * per;
        const int64_t c1 = c0 + per < d_in ? c0 + per : d_in;
        unsigned long long mine = 0;  // two counts of 32 bits
        for (int64_t i = c0; i < c1; ++i) {
            const uint32_t key = ordered_bits(a[i]) - kmin;
            mine += (key == v0 ? 1ull : 0ull) + (key == v1 ? (1ull << 32) : 0ull);
        }
        unsigned long long incl = mine;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const unsigned long long up = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += up;
        }
        if (lane == 31) warp_tot[warp] = incl;
        __syncthreads();
        unsigned long long before = incl - mine;
        for (int w = 0; w < warp; ++w) before += warp_tot[w];
        long long eq0 = (long long)(before & 0xffffffffull), eq1 = (long long)(before >> 32);
        for (int64_t i = c0; i < c1; ++i) {
            const uint32_t key = ordered_bits(a[i]) - kmin;
            int cls = base;
            if (live[0] && (key > v0 || (key == v0 && eq0 >= r0))) ++cls;
            if (live[1] && (key > v1 || (key == v1 && eq1 >= r1))) ++cls;
            eq0 += key == v0 ? 1 : 0;
            eq1 += key == v1 ? 1 : 0;
            out[i] = (uint8_t)cls;
        }
    }
}

cmpq_status launch_rank_cut(const float* a, int64_t d_in, int64_t k0, int64_t k1, int base, uint8_t* out,
                            cudaStream_t st) {
    rank_cut_kernel<<<1, kCutThreads, 0, st>>>(a, d_in, (long long)k0, (long long)k1, base, out, CutExtras{});
    return launch_status();
}

// The O_act cut of the outlier step with what else one block can prepare for it: the start state of the
// select (state / hist / n_q) and, when bits is given, the layout of the packed segments.
cmpq_status launch_act_cut(const float* a, int64_t d_in, int64_t n_act, uint8_t* is_act, void* select_state,
                           long long n_q, unsigned int* hist, const uint8_t* bits, int64_t d_out, int64_t* row_off,
                           int32_t* perm, int64_t* seg_rows, int64_t* word_off, cudaStream_t st) {
    CutExtras x{};
    x.select = static_cast<SelectState*>(select_state);
    x.n_q = n_q;
    x.hist = hist;
    x.bits = bits;
    x.d_out = d_out;
    x.row_off = row_off;
    x.perm = perm;
    x.seg_rows = seg_rows;
    x.word_off = word_off;
    rank_cut_kernel<<<2, kCutThreads, 0, st>>>(a, d_in, (long long)(d_in - n_act), (long long)d_in, 0, is_act, x);
    return launch_status();
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
    int64_t n2 = 0, n4 = 0;
    cmpq_alloc_counts(d_in, avg_bits, &n2, &n4);
    // without the order only two rank cuts matter: 2 bits below rank n2, 4 bits from rank d_in - n4
    if (mode == CMPQ_ALLOC_RANK && !order) return launch_rank_cut(a, d_in, n2, d_in - n4, 2, bits, st);
    cmpq_status s = launch_rank(a, d_in, rank, st);
    if (s != CMPQ_OK) return s;
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
