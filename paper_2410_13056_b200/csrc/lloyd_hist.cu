// Channel-wise K-means of CMPQ (Section 3.2.1: K-means per channel W_{i,:} with K = 2^bits;
// Section 3: each weight is replaced by its nearest centroid) -- the ordered formulation.
//
// A channel of 16-bit weights is fully described by how often each 16-bit value occurs.  Three
// kernels use that:
//
//   lloyd_table_kernel    one block per channel: reads the row from HBM once, sets the removed
//                         positions to +0, counts the values with a two-level histogram in shared
//                         memory (high byte, then low byte inside the non-empty high-byte buckets)
//                         and writes the DISTINCT values in ascending order with, for each, the
//                         number of smaller weights (exclusive prefix of the counts).
//   lloyd_iterate_kernel  one WARP per channel, all iterations.  While the centroids are strictly
//                         increasing with gaps above 2^-22 of the value range, the predicate
//                         fabsf(x - c_k) < fabsf(x - c_{k-1}) is false on a prefix of the ascending
//                         values and true on the rest, and the first k minimising fabsf(x - c_k) is
//                         the number of k >= 1 for which it is true.  Cluster k is then a run of the
//                         table: lane k finds the first entry where predicate k holds (galloping
//                         from the previous boundary, then bisection), and the cluster's count and
//                         sum are differences of
//                         prefix counts and prefix sums at two such entries (the warp builds the
//                         prefix sums once, at every eighth entry; table and sums stay in shared
//                         memory when they fit).  Centroids that fail the test are handled
//                         by the plain first-minimum scan over the distinct values.  The sums are
//                         count x value products added in fp64: exact for 16-bit weights of bounded
//                         dynamic range, hence equal to the sums taken weight by weight.
//   lloyd_assign_kernel   streams the row once more and applies the defining rule (first k
//                         minimising fabsf(x - c_k), fp32) to every weight with the final centroids:
//                         codes or errors leave in column order, no staging.
//
// Nothing here is a dense contraction, so no tensor cores are used.
#include "lloyd.cuh"
#include "lloyd_device.cuh"
#include "pack_bits.cuh"
#include "select.cuh"

#include <cuda_bf16.h>

#include <mutex>

namespace cmpq {

constexpr int kSlots = 32;       // high-byte buckets refined per pass of the second histogram level
constexpr int kSlotWords = 128;  // 256 low-byte counters of 16 bits, two per word
static_assert(CMPQ_MAX_D_OUT < 65536, "second-level counters and count prefixes are 16 bits wide");

struct ChannelHeader {
    int M;        // distinct values of the channel
    int suspect;  // 1 if the magnitude range alone does not prove the fp64 sums exact
};

// Per channel: `stride` entries (M used, entry M is a sentinel holding the totals).
struct Tables {
    int64_t stride;
    ChannelHeader* hdr;  // [d_in]
    uint16_t* keys;      // [d_in][stride] sort keys of the distinct values, ascending
    uint16_t* cum;       // [d_in][stride] number of weights below the entry's value
    double* sum;         // [d_in][stride] scratch of the iterate kernel for tables too large for shared memory
    float* lut;          // [d_in][16] centroids for the assign kernel when the caller wants no lut
    float* thr;          // [d_in][16] value thresholds of the last assignment ([0]: 1 if valid)
};

static int64_t table_stride(int64_t d_out) { return (d_out + 1 + 7) / 8 * 8; }

static Tables carve_tables(Workspace& w, int64_t d_in, int64_t d_out) {
    Tables t;
    t.stride = table_stride(d_out);
    t.hdr = w.take<ChannelHeader>(d_in);
    t.keys = w.take<uint16_t>((size_t)d_in * t.stride);
    t.cum = w.take<uint16_t>((size_t)d_in * t.stride);
    t.sum = w.take<double>((size_t)d_in * t.stride);
    t.lut = w.take<float>((size_t)d_in * CMPQ_LUT_STRIDE);
    t.thr = w.take<float>((size_t)d_in * CMPQ_LUT_STRIDE);
    return t;
}

size_t lloyd_tables_bytes(int64_t d_in, int64_t d_out) {
    Workspace w(nullptr, 0);
    carve_tables(w, d_in, d_out);
    return w.used;
}

// ------------------------------------------------------------------------------------------------
// value table of one channel

constexpr int kShortList = 16;  // removed positions of a row kept as a list up to this many, else as a bitmap

struct alignas(16) TableShared {
    int hist1[256];        // 1 where the high byte occurs
    int bucket_rank[256];  // rank of a high-byte bucket among the non-empty ones, or -1
    int slot_hi[256];      // the inverse: high byte of the r-th non-empty bucket
    int n_nonempty;
    int wtop[32], wulp[32];   // per-warp magnitude range (largest pattern, smallest non-zero pattern - 1)
    int w_nz[32], w_cnt[32];  // per-warp totals of the block scan
    int base_nz, base_cnt;    // entries / weights emitted by the previous passes
    int rem_list[kShortList];
};
// dynamic shared memory after TableShared: kSlots * kSlotWords words of second-level counters, then
// a bitmap of d_out bits for rows with many removed positions

template <int DT, int E, int MAXT, int MINB>
__global__ void __launch_bounds__(MAXT, MINB)
lloyd_table_kernel(const LloydArgs a, const Tables t) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const int64_t row = blockIdx.x;
    if (a.skip_row && a.skip_row[row]) return;
    TableShared& sh = *reinterpret_cast<TableShared*>(smem_raw);
    uint32_t* h2 = reinterpret_cast<uint32_t*>(smem_raw + sizeof(TableShared));
    uint32_t* bitmap = h2 + kSlots * kSlotWords;
    const int tid = threadIdx.x, nthr = blockDim.x, lane = tid & 31, warp = tid >> 5;
    const int nwarps = nthr >> 5;
    const int N = (int)a.d_out;

    // The weights are requested first (the order of the columns does not matter for a histogram:
    // a thread takes VEC consecutive ones per load), then the row's metadata.
    constexpr int VEC = E >= 8 ? 8 : 4;
    constexpr int G = E / VEC;
    const uint16_t* w = a.W + row * a.ldw;
    const bool vec = ((a.ldw & (VEC - 1)) == 0) && ((reinterpret_cast<uintptr_t>(a.W) & (2 * VEC - 1)) == 0);
    uint32_t raw[E / 2];  // two weights per word
#pragma unroll
    for (int g = 0; g < G; ++g) {
        const int j0 = (g * nthr + tid) * VEC;
        if (j0 + VEC - 1 < N && vec) {
            if (VEC == 8) {
                const uint4 v = __ldcs(reinterpret_cast<const uint4*>(w + j0));
                raw[4 * g] = v.x; raw[4 * g + 1] = v.y; raw[4 * g + 2] = v.z; raw[4 * g + 3] = v.w;
            } else {
                const uint2 v = __ldcs(reinterpret_cast<const uint2*>(w + j0));
                raw[2 * g] = v.x; raw[2 * g + 1] = v.y;
            }
        } else {
#pragma unroll
            for (int u = 0; u < VEC; u += 2) {
                const uint32_t a0 = j0 + u < N ? w[j0 + u] : 0u, a1 = j0 + u + 1 < N ? w[j0 + u + 1] : 0u;
                raw[(g * VEC + u) / 2] = a0 | (a1 << 16);
            }
        }
    }
    int64_t p0 = 0, p1 = 0;
    if (a.row_ptr) { p0 = a.row_ptr[row]; p1 = a.row_ptr[row + 1]; }
    const int nrem = (int)(p1 - p0);
    for (int b = tid; b < 256; b += nthr) sh.hist1[b] = 0;
    for (int i = tid; i < kSlots * kSlotWords / 4; i += nthr) reinterpret_cast<uint4*>(h2)[i] = make_uint4(0u, 0u, 0u, 0u);
    if (nrem > kShortList) {
        for (int i = tid; i < (N + 31) / 32; i += nthr) bitmap[i] = 0;
        __syncthreads();
        for (int64_t p = p0 + tid; p < p1; p += nthr) {
            const int col = a.cols[p];
            atomicOr(&bitmap[col >> 5], 1u << (col & 31));
        }
    } else if (tid < nrem) {
        sh.rem_list[tid] = a.cols[p0 + tid];
    }
    __syncthreads();

    // keys (removed positions and -0 become +0), which high bytes occur, range of the magnitudes
    uint32_t key[E];
    uint32_t valid = 0;  // bit e: key[e] is a weight of the row
    uint32_t amax = 0u, amin1 = 0xffffffffu;
#pragma unroll
    for (int g = 0; g < G; ++g) {
        const int j0 = (g * nthr + tid) * VEC;
        uint32_t rm = 0;  // removed positions among the VEC
        if (nrem > kShortList) {
            rm = j0 < N ? (bitmap[j0 >> 5] >> (j0 & 31)) & ((1u << VEC) - 1u) : 0u;  // j0 is a multiple of VEC
        } else {
            for (int i = 0; i < nrem; ++i) {
                const unsigned d = (unsigned)(sh.rem_list[i] - j0);
                if (d < (unsigned)VEC) rm |= 1u << d;
            }
        }
#pragma unroll
        for (int u = 0; u < VEC; ++u) {
            const int e = g * VEC + u;
            uint32_t h = (raw[e >> 1] >> (16 * (e & 1))) & 0xffffu;
            if ((rm >> u) & 1u) h = 0u;
            if (h == 0x8000u) h = 0u;  // -0 and +0 are the same point
            const uint32_t ub = h & 0x7fffu;
            key[e] = (h & 0x8000u) ? (~h & 0xffffu) : (h | 0x8000u);
            if (j0 + u < N) {
                valid |= 1u << e;
                amax = max(amax, ub);
                amin1 = min(amin1, ub - 1u);  // zero wraps to the largest value
                sh.hist1[key[e] >> 8] = 1;
            }
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        amax = max(amax, __shfl_xor_sync(0xffffffffu, amax, o));
        amin1 = min(amin1, __shfl_xor_sync(0xffffffffu, amin1, o));
    }
    if (lane == 0) { sh.wtop[warp] = (int)amax; sh.wulp[warp] = (int)amin1; }
    __syncthreads();
    if (warp == 0) {
        int flag[8], sum = 0;
#pragma unroll
        for (int u = 0; u < 8; ++u) { flag[u] = sh.hist1[lane * 8 + u]; sum += flag[u]; }
        int incl = sum;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            int up = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += up;
        }
        int run = incl - sum;
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            sh.bucket_rank[lane * 8 + u] = flag[u] ? run : -1;
            if (flag[u]) sh.slot_hi[run] = lane * 8 + u;
            run += flag[u];
        }
        if (lane == 31) { sh.n_nonempty = incl; sh.base_nz = 0; sh.base_cnt = 0; }
    }
    // Exactness of fp64 sums (see load_channel_keys): first from the magnitude range alone, bit by bit
    // only for a channel that fails that.  Every warp reduces the per-warp ranges, so the decision is
    // the same in all threads.
    bool suspect = false;  // kept in the header: a later fit of a subset of these weights can skip the test
    {
        amax = lane < nwarps ? (uint32_t)sh.wtop[lane] : 0u;
        amin1 = lane < nwarps ? (uint32_t)sh.wulp[lane] : 0xffffffffu;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            amax = max(amax, __shfl_xor_sync(0xffffffffu, amax, o));
            amin1 = min(amin1, __shfl_xor_sync(0xffffffffu, amin1, o));
        }
        if (amax != 0u) {
            const uint32_t fmax = __float_as_uint(widen16<DT>((uint16_t)amax));
            const uint32_t fmin = __float_as_uint(widen16<DT>((uint16_t)(amin1 + 1u)));
            const int log2n = 32 - __clz(N - 1 > 0 ? N - 1 : 1);
            const int ex_max = (int)(fmax >> 23), ex_min = (int)(fmin >> 23);
            const int top = ex_max ? ex_max - 127 : (31 - __clz(fmax)) - 149;
            const int q_low = (ex_min ? ex_min - 150 : -149) + (DT == CMPQ_BF16 ? 16 : 13);
            suspect = log2n + 1 + (top + 1 - q_low) > 53;
            if (suspect && a.inexact_rows) {
                int q = 100000;
#pragma unroll
                for (int e = 0; e < E; ++e) {
                    const uint32_t ub = __float_as_uint(value_of_key16<DT>(key[e])) & 0x7fffffffu;
                    if (((valid >> e) & 1u) && ub) {
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
    __syncthreads();

    uint16_t* keys = t.keys + row * t.stride;
    uint16_t* cum = t.cum + row * t.stride;
    const int n_nonempty = sh.n_nonempty;
    int run_nz = 0, run_cnt = 0;
    for (int g0 = 0; g0 < n_nonempty; g0 += kSlots) {
        const int nslots = n_nonempty - g0 < kSlots ? n_nonempty - g0 : kSlots;
        const int words_total = nslots * kSlotWords;
        // Second level: the low byte inside the buckets g0 .. g0 + nslots.  Two 16-bit counters share a
        // word (a channel has fewer than 2^16 weights, so the halves never carry into each other).
        if (g0 > 0) {  // the counters of the first pass were cleared at the start
            for (int w = tid; w < words_total / 4; w += nthr) reinterpret_cast<uint4*>(h2)[w] = make_uint4(0u, 0u, 0u, 0u);
            __syncthreads();  // also: the previous pass has published its bases
        }
#pragma unroll
        for (int e = 0; e < E; ++e) {
            if ((valid >> e) & 1u) {
                const int r = sh.bucket_rank[key[e] >> 8] - g0;
                const uint32_t lo = key[e] & 0xffu;
                if (r >= 0 && r < kSlots) atomicAdd(&h2[r * kSlotWords + (lo >> 1)], 1u << (16 * (lo & 1u)));
            }
        }
        __syncthreads();
        // Every thread owns a contiguous range of counters: totals first, a block scan, then the entries.
        const int w0 = (int)((long long)tid * words_total / nthr);
        const int w1 = (int)((long long)(tid + 1) * words_total / nthr);
        int nz = 0, cnt = 0;
        for (int w = w0; w < w1; ++w) {
            const uint32_t word = h2[w];
            const int c0 = (int)(word & 0xffffu), c1 = (int)(word >> 16);
            nz += (c0 ? 1 : 0) + (c1 ? 1 : 0);
            cnt += c0 + c1;
        }
        int inz = nz, icnt = cnt;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int unz = __shfl_up_sync(0xffffffffu, inz, o);
            const int ucnt = __shfl_up_sync(0xffffffffu, icnt, o);
            if (lane >= o) { inz += unz; icnt += ucnt; }
        }
        if (lane == 31) { sh.w_nz[warp] = inz; sh.w_cnt[warp] = icnt; }
        __syncthreads();
        run_nz = sh.base_nz + inz - nz;
        run_cnt = sh.base_cnt + icnt - cnt;
        for (int wv = 0; wv < warp; ++wv) { run_nz += sh.w_nz[wv]; run_cnt += sh.w_cnt[wv]; }
        for (int w = w0; w < w1; ++w) {
            const uint32_t word = h2[w];
            if (word) {
                const uint32_t kb = ((uint32_t)sh.slot_hi[g0 + (w >> 7)] << 8) | ((uint32_t)(w & 127) << 1);
                const int c0 = (int)(word & 0xffffu), c1 = (int)(word >> 16);
                if (c0) { keys[run_nz] = (uint16_t)kb; cum[run_nz] = (uint16_t)run_cnt; ++run_nz; run_cnt += c0; }
                if (c1) { keys[run_nz] = (uint16_t)(kb | 1u); cum[run_nz] = (uint16_t)run_cnt; ++run_nz; run_cnt += c1; }
            }
        }
        __syncthreads();  // every thread has read the bases and the counters of this pass
        if (tid == nthr - 1) { sh.base_nz = run_nz; sh.base_cnt = run_cnt; }
    }
    if (tid == nthr - 1) {
        // the last thread's running values are the totals: sentinel entry and header
        keys[run_nz] = 0xffffu;
        cum[run_nz] = (uint16_t)run_cnt;
        ChannelHeader h;
        h.M = run_nz;
        h.suspect = suspect ? 1 : 0;
        t.hdr[row] = h;
    }
}

// ------------------------------------------------------------------------------------------------
// iterations: one warp per channel

// fits kept between calls (see lloyd.cuh): slot (bits - 2) * d_in + row
struct FitCacheHeader {
    int iters;  // the iteration count the cached fits were made with
};
struct FitCache {
    FitCacheHeader* hdr;  // NULL: no cache
    uint8_t* valid;
    float* lut;
    float* thr;
};

static FitCache carve_fit_cache(void* p, int64_t d_in) {
    FitCache c{};
    if (!p) return c;
    Workspace w(p, ~(size_t)0);
    c.hdr = w.take<FitCacheHeader>(1);
    c.valid = w.take<uint8_t>(3 * (size_t)d_in);
    c.lut = w.take<float>(3 * (size_t)d_in * CMPQ_LUT_STRIDE);
    c.thr = w.take<float>(3 * (size_t)d_in * CMPQ_LUT_STRIDE);
    return c;
}

size_t lloyd_fit_cache_bytes(int64_t d_in) {
    return 256 + round_up(3 * (size_t)d_in, 256) + 2 * round_up(3 * (size_t)d_in * CMPQ_LUT_STRIDE * sizeof(float), 256);
}

__global__ void fit_cache_clear_kernel(FitCache c, int64_t n, int iters) {
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) c.valid[i] = 0;
    if (i == 0) c.hdr->iters = iters;
}

cmpq_status launch_fit_cache_clear(void* fit_cache, int64_t d_in, int iters, cudaStream_t st) {
    const FitCache c = carve_fit_cache(fit_cache, d_in);
    const int64_t n = 3 * d_in;
    fit_cache_clear_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(c, n, iters);
    return launch_status();
}

struct IterArgs {
    Tables t;
    FitCache fc;
    const uint8_t* bits;
    const uint8_t* skip_row;
    int64_t d_in, d_out;
    int iters;
    int cap;     // table entries a warp can stage in shared memory (multiple of 8)
    float* lut;  // [d_in][16]
    unsigned long long* sweeps;
};

// Lane k (1..K-1) receives e_k = the number of table entries for whose value the predicate
// fabsf(x - c_k) < fabsf(x - c_{k-1}) is false (a prefix of the table); lane 0 receives 0, lane K
// receives M.  Every lane searches its own boundary: the warp's instruction stream then serves all
// K-1 boundaries at once, which matters because the kernel is bound by instruction issue.  e_prev
// (the lane's result of the previous iteration, or -1) starts a galloping search next to the old
// boundary -- boundaries move by a few entries per iteration -- followed by bisection.
template <int DT, int K>
__device__ __forceinline__ int search_entries(const uint16_t* keys, int M, float ck_lane, int e_prev) {
    const int lane = threadIdx.x & 31;
    const float cm = __shfl_up_sync(0xffffffffu, ck_lane, 1);  // c_{k-1}
    const float ck = ck_lane;
    int lo = 0, hi = 0;  // the predicate is false for entries < lo and true for entries >= hi
    if (lane > 0 && lane < K) {
        hi = M;
        auto pred = [&](int i) {
            const float v = value_of_key16<DT>(keys[i]);
            return fabsf(v - ck) < fabsf(v - cm);
        };
        if (e_prev >= 0) {
            // gallop away from the old boundary p, downwards if the predicate holds at p and upwards if
            // not, in one loop for both directions (lanes of both kinds then share the instructions)
            const int p = e_prev < M ? e_prev : M;
            const bool down = p >= M || pred(p);
            if (down) hi = p; else lo = p + 1;
            bool open = true;
            for (int step = 1; open; step <<= 1) {
                const int q = down ? hi - step : lo - 1 + step;
                if (q < 0 || q >= M) break;  // ran off the table: the bracket is [0, hi] or [lo, M]
                const bool t = pred(q);
                if (t) hi = q; else lo = q + 1;
                open = (t == down);          // closed by the first false (down) or the first true (up)
            }
        }
        while (lo < hi) {
            const int mid = (lo + hi) >> 1;
            if (pred(mid)) hi = mid; else lo = mid + 1;
        }
    }
    __syncwarp();
    return lane == K ? M : lo;
}

constexpr int kIterWarps = 4;

// Shared memory of one warp of the iterate kernel: the channel's table when it has at most `cap`
// distinct values (cap is a multiple of 8, chosen by the host from d_out).
__host__ __device__ inline size_t iter_warp_bytes(int cap) {
    return (size_t)cap * 2 + (size_t)(cap + 8) * 2 + (size_t)(cap / 8 + 1) * 8 + 8;  // keys, cum, coarse sums
}

// Eight consecutive 16-bit table entries starting at a multiple of 8 (16-byte aligned), one load.
struct Eight {
    uint32_t w[4];
    __device__ __forceinline__ uint32_t at(int u) const { return (w[u >> 1] >> (16 * (u & 1))) & 0xffffu; }
};
__device__ __forceinline__ Eight load_eight(const uint16_t* p) {
    const uint4 v = *reinterpret_cast<const uint4*>(p);
    Eight r;
    r.w[0] = v.x; r.w[1] = v.y; r.w[2] = v.z; r.w[3] = v.w;
    return r;
}

// fp64 sum of all weights below entry e (0 <= e <= M): the prefix stored for entry 8 (e / 8)
// plus at most seven count x value products.
template <int DT>
__device__ __forceinline__ double prefix_sum_at(const uint16_t* keys, const uint16_t* cum, const double* coarse,
                                                int e) {
    const int j0 = e & ~7, r = e & 7;
    double P = coarse[e >> 3];
    const Eight k8 = load_eight(keys + j0), c8 = load_eight(cum + j0);
#pragma unroll
    for (int u = 0; u < 7; ++u) {
        if (u < r) {
            const int cnt = (int)c8.at(u + 1) - (int)c8.at(u);
            P += (double)cnt * (double)value_of_key16<DT>(k8.at(u));
        }
    }
    return P;
}

template <int DT, int K>
__device__ void iterate_channel(const IterArgs& a, int64_t row, unsigned char* warp_smem) {
    const int lane = threadIdx.x & 31;
    const ChannelHeader h = a.t.hdr[row];
    const int N = (int)a.d_out, T = a.iters;
    const int M = h.M < 1 ? 1 : (h.M > N ? N : h.M);  // 1 <= M <= N by construction
    const uint16_t* keys = a.t.keys + row * a.t.stride;
    const uint16_t* cum = a.t.cum + row * a.t.stride;
    double* coarse = a.t.sum + row * a.t.stride;  // global scratch, used when the table is too large
    if (M <= a.cap) {  // the rows are 16-byte aligned and padded to a multiple of 8 entries
        double* s_coarse = reinterpret_cast<double*>(warp_smem);
        uint16_t* s_keys = reinterpret_cast<uint16_t*>(s_coarse + a.cap / 8 + 1 + 1);
        uint16_t* s_cum = s_keys + a.cap;
        for (int i = lane; i < (M + 7) / 8; i += 32)
            reinterpret_cast<uint4*>(s_keys)[i] = __ldg(reinterpret_cast<const uint4*>(keys) + i);
        for (int i = lane; i < (M + 1 + 7) / 8; i += 32)  // with the sentinel cum[M] = d_out
            reinterpret_cast<uint4*>(s_cum)[i] = __ldg(reinterpret_cast<const uint4*>(cum) + i);
        keys = s_keys;
        cum = s_cum;
        coarse = s_coarse;
    }
    __syncwarp();
    // prefix sums at every eighth entry: each lane sums a contiguous range of groups of eight entries,
    // the lane totals are scanned, then every group receives its base
    {
        const int groups = (M >> 3) + 1;  // coarse[g] for g = 0 .. M / 8
        const int per_lane = (groups + 31) / 32;
        const int g_begin = lane * per_lane;
        double local = 0.0;
        for (int g = g_begin; g < g_begin + per_lane && g < groups; ++g) {
            coarse[g] = local;
            const Eight k8 = load_eight(keys + g * 8), c8 = load_eight(cum + g * 8);
            const int c_end = g * 8 + 8 <= M ? (int)cum[g * 8 + 8] : 0;
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                if (g * 8 + u < M) {
                    const int c_next = u < 7 ? (int)c8.at(u + 1) : c_end;
                    local += (double)(c_next - (int)c8.at(u)) * (double)value_of_key16<DT>(k8.at(u));
                }
            }
        }
        double incl = local;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const double up = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += up;
        }
        double base = __shfl_up_sync(0xffffffffu, incl, 1);
        if (lane == 0) base = 0.0;
        for (int g = g_begin; g < g_begin + per_lane && g < groups; ++g) coarse[g] += base;
        __threadfence_block();  // the sums may live in global memory: make them visible to the other lanes
        __syncwarp();
    }
    // range * 2^-22, the range being last minus first value of the table
    const double need = ((double)value_of_key16<DT>(keys[M - 1]) - (double)value_of_key16<DT>(keys[0])) * (1.0 / 4194304.0);

    // start: K evenly spaced order statistics; the weight at sorted position pos has the value of the
    // entry e with cum[e] <= pos < cum[e + 1]
    float ck = 0.f;
    if (lane < K) {
        const int pos = (int)(((long long)(2 * lane + 1) * N) / (2 * K));
        int lo = 0, hi = M;  // cum[lo] <= pos < cum[hi]   (cum[0] = 0, cum[M] = N)
        while (hi - lo > 1) {
            const int mid = (lo + hi) >> 1;
            if ((int)cum[mid] <= pos) lo = mid; else hi = mid;
        }
        ck = value_of_key16<DT>(keys[lo]);
    }
    __syncwarp();

    int updates = 0;
    int e_prev = -1;  // this lane's boundary of the previous ordered search
    while (updates < T) {
        float cn = ck;
        if (counting_sweep_valid<K>(ck, need)) {
            const int e = search_entries<DT, K>(keys, M, ck, e_prev);
            e_prev = e;
            int B = 0;
            double P = 0.0;
            if (lane <= K) { B = (int)cum[e]; P = prefix_sum_at<DT>(keys, cum, coarse, e); }
            const int Bn = __shfl_down_sync(0xffffffffu, B, 1);
            const double Pn = __shfl_down_sync(0xffffffffu, P, 1);
            if (lane < K) {
                const int cnt = Bn - B;
                if (cnt > 0) cn = __double2float_rn(__ddiv_rn(Pn - P, (double)cnt));
            }
        } else {
            // plain rule on every distinct value; cluster sums as count x value in fp64
            float c[K];
#pragma unroll
            for (int k = 0; k < K; ++k) c[k] = __shfl_sync(0xffffffffu, ck, k);
            double s[K];
            int n[K];
#pragma unroll
            for (int k = 0; k < K; ++k) { s[k] = 0.0; n[k] = 0; }
            for (int j = lane; j < M; j += 32) {
                const float v = value_of_key16<DT>(keys[j]);
                const int cnt = (int)cum[j + 1] - (int)cum[j];
                const int code = nearest_scan<K>(v, c);
                const double prod = (double)cnt * (double)v;
#pragma unroll
                for (int k = 0; k < K; ++k)
                    if (code == k) { s[k] += prod; n[k] += cnt; }
            }
#pragma unroll
            for (int k = 0; k < K; ++k) {
                const double sk = warp_sum(s[k]);
                const int nk = warp_sum(n[k]);
                if (lane == k && nk > 0) cn = __double2float_rn(__ddiv_rn(sk, (double)nk));
            }
        }
        ++updates;
        const bool same = __all_sync(0xffffffffu, lane >= K || __float_as_uint(cn) == __float_as_uint(ck));
        ck = cn;
        if (same) break;  // identical centroids: every later iteration repeats this one
    }
    if (lane < CMPQ_LUT_STRIDE) a.lut[row * CMPQ_LUT_STRIDE + lane] = lane < K ? ck : 0.f;
    // Last assignment: when the final centroids pass the test, predicate k holds exactly for the values
    // from the first entry where it is true, so the assign kernel only compares with K-1 thresholds.
    {
        const bool ok = counting_sweep_valid<K>(ck, need);
        float thr = ok ? 1.f : 0.f;
        if (ok) {
            const int e = search_entries<DT, K>(keys, M, ck, e_prev);
            if (lane > 0 && lane < K) thr = e < M ? value_of_key16<DT>(keys[e]) : __int_as_float(0x7f800000);
        }
        if (lane < CMPQ_LUT_STRIDE) a.t.thr[row * CMPQ_LUT_STRIDE + lane] = lane < K ? thr : 0.f;
    }
    // assignments made: one per update, and the last one by the assign kernel
    if (a.sweeps && lane == 0)
        atomicAdd(a.sweeps, (unsigned long long)(updates + 1) * (unsigned long long)N * (unsigned long long)K);
}

template <int DT>
__global__ void __launch_bounds__(kIterWarps * 32, 7)
lloyd_iterate_kernel(const IterArgs a) {
    extern __shared__ __align__(16) unsigned char iter_smem[];
    const int warp = threadIdx.x >> 5;
    unsigned char* warp_smem = iter_smem + (size_t)warp * iter_warp_bytes(a.cap);
    const int64_t row = (int64_t)blockIdx.x * kIterWarps + warp;
    if (row >= a.d_in) return;
    if (a.skip_row && a.skip_row[row]) return;
    const int bits = a.bits[row];
    const int lane = threadIdx.x & 31;
    // a fit of this channel at this width kept from an earlier call on the same weights: copy it
    const bool cached_ok = a.fc.hdr && a.fc.hdr->iters == a.iters;
    const int64_t slot = (int64_t)(bits == 2 ? 0 : (bits == 3 ? 1 : 2)) * a.d_in + row;
    if (cached_ok && a.fc.valid[slot]) {
        if (lane < CMPQ_LUT_STRIDE) {
            a.lut[row * CMPQ_LUT_STRIDE + lane] = a.fc.lut[slot * CMPQ_LUT_STRIDE + lane];
            a.t.thr[row * CMPQ_LUT_STRIDE + lane] = a.fc.thr[slot * CMPQ_LUT_STRIDE + lane];
        }
        return;
    }
    if (bits == 2) iterate_channel<DT, 4>(a, row, warp_smem);
    else if (bits == 3) iterate_channel<DT, 8>(a, row, warp_smem);
    else iterate_channel<DT, 16>(a, row, warp_smem);
    if (cached_ok) {  // lane l wrote entry l of both rows above and reads its own writes back
        if (lane < CMPQ_LUT_STRIDE) {
            a.fc.lut[slot * CMPQ_LUT_STRIDE + lane] = a.lut[row * CMPQ_LUT_STRIDE + lane];
            a.fc.thr[slot * CMPQ_LUT_STRIDE + lane] = a.t.thr[row * CMPQ_LUT_STRIDE + lane];
        }
        __syncwarp();
        if (lane == 0) {
            __threadfence();
            a.fc.valid[slot] = 1;
        }
    }
}

// ------------------------------------------------------------------------------------------------
// last assignment

constexpr int kAssignThreads = 256;

// Two weights at once in their 16-bit storage type: acc += (x >= t) per half, as 1.0 or 0.0.
template <int DT>
__device__ __forceinline__ uint32_t add_ge_x2(uint32_t acc, uint32_t x2, uint32_t t2) {
    if (DT == CMPQ_BF16) {
        const __nv_bfloat162 r = __hadd2(*reinterpret_cast<const __nv_bfloat162*>(&acc),
                                         __hge2(*reinterpret_cast<const __nv_bfloat162*>(&x2),
                                                *reinterpret_cast<const __nv_bfloat162*>(&t2)));
        return *reinterpret_cast<const uint32_t*>(&r);
    } else {
        const __half2 r = __hadd2(*reinterpret_cast<const __half2*>(&acc),
                                  __hge2(*reinterpret_cast<const __half2*>(&x2), *reinterpret_cast<const __half2*>(&t2)));
        return *reinterpret_cast<const uint32_t*>(&r);
    }
}

// A threshold (a value of the channel or +infinity, so exact in the storage type) in both halves.
template <int DT>
__device__ __forceinline__ uint32_t threshold_x2(float t) {
    uint32_t h;
    if (DT == CMPQ_BF16) h = __float_as_uint(t) >> 16;
    else h = __half_as_ushort(__float2half_rn(t));
    return h | (h << 16);
}

// Code (and distance) of one weight.  by_threshold: the code is the number of k >= 1 with
// x >= t[k] (thresholds from lloyd_iterate_kernel); otherwise the defining scan.
template <int K, bool ERR>
__device__ __forceinline__ void assign_one(float x, const float (&c)[K], const float (&t)[K], bool by_threshold,
                                           uint32_t& code, float& dist) {
    if (by_threshold) {
        uint32_t bk = 0;
        float cc = c[0];
#pragma unroll
        for (int k = 1; k < K; ++k) {
            const bool ge = x >= t[k];
            if (!ERR) bk += ge ? 1u : 0u;   // the provisional fit (ERR) asks for distances only
            if (ERR) cc = ge ? c[k] : cc;  // thresholds ascend: the last one reached is the code's
        }
        code = bk;
        dist = ERR ? fabsf(x - cc) : 0.f;
    } else {
        float best = fabsf(x - c[0]);
        uint32_t bk = 0;
#pragma unroll
        for (int k = 1; k < K; ++k) {
            const float d = fabsf(x - c[k]);
            if (d < best) { best = d; bk = k; }
        }
        code = bk;
        dist = best;
    }
}

// One row, 8 weights per thread and step (one 128-bit load when the layout allows).
// removed positions of the row: a bitmap over the columns (nrem > kShortList) or a short list
struct RemovedCols {
    const uint32_t* bitmap;
    const int* list;
    int nrem;
};
template <int DT, int K, bool ERR>
__device__ void assign_row(const LloydArgs& a, int64_t row, const float* __restrict__ lut,
                           const float* __restrict__ thr, const RemovedCols& rem, uint4 first) {
    constexpr int C = K == 4 ? 2 : (K == 8 ? 3 : 4);
    const int N = (int)a.d_out;
    const int tid = threadIdx.x, nthr = blockDim.x, lane = tid & 31;
    float c[K], t[K];
#pragma unroll
    for (int k = 0; k < K; ++k) {
        c[k] = __ldg(lut + row * CMPQ_LUT_STRIDE + k);
        t[k] = __ldg(thr + row * CMPQ_LUT_STRIDE + k);
    }
    const bool by_threshold = t[0] != 0.f;
    // codes only, by thresholds: two weights per compare in the storage type.  A count c sits in
    // the low mantissa bits of 128 + c (bf16) or 1024 + c (fp16).
    uint32_t t2[K];
#pragma unroll
    for (int k = 0; k < K; ++k) t2[k] = threshold_x2<DT>(t[k]);
    const uint32_t acc0 = DT == CMPQ_BF16 ? 0x43004300u : 0x64006400u;
    const uint16_t* w = a.W + row * a.ldw;
    const bool vec_in = ((a.ldw & 7) == 0) && ((reinterpret_cast<uintptr_t>(a.W) & 15) == 0);
    const bool vec_out = (N & 7) == 0;
    uint8_t* codes = a.codes ? a.codes + row * a.d_out : nullptr;
    float* err = a.err ? a.err + row * a.d_out : nullptr;
    // packed output: the eight codes of a thread become a field of 8 C bits, four neighbouring threads
    // hold 32 consecutive codes = C words
    uint32_t* packed = (!ERR && a.packed) ? a.packed + a.word_off[row] : nullptr;
    const int words_per_row = (N * C + 31) / 32;
#pragma unroll 1
    for (int base = 0; base < N; base += nthr * 8) {  // the same trip count in every thread of the block
        const int j0 = base + tid * 8;
        uint2 o = make_uint2(0u, 0u);  // eight codes, one per byte; zero beyond the end of the row
        if (j0 < N) {
            uint32_t pk[4] = {0u, 0u, 0u, 0u};  // 8 weights, two per word
            if (j0 + 7 < N && vec_in) {
                // the first step's weights were requested before anything else in the kernel
                const uint4 v = base == 0 ? first : __ldcs(reinterpret_cast<const uint4*>(w + j0));
                pk[0] = v.x; pk[1] = v.y; pk[2] = v.z; pk[3] = v.w;
            } else {
#pragma unroll
                for (int u = 0; u < 8; ++u)
                    if (j0 + u < N) pk[u >> 1] |= (uint32_t)w[j0 + u] << (16 * (u & 1));
            }
            uint32_t mask = 0;  // removed positions among the 8
            if (rem.nrem > kShortList) {
                mask = (rem.bitmap[j0 >> 5] >> (j0 & 31)) & 0xffu;  // j0 is a multiple of 8
            } else {
                for (int i = 0; i < rem.nrem; ++i) {
                    const unsigned d = (unsigned)(rem.list[i] - j0);
                    if (d < 8u) mask |= 1u << d;
                }
            }
            if (!ERR && by_threshold && j0 + 7 < N) {
                uint32_t r[4];
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    uint32_t x2 = pk[q];
                    if ((mask >> (2 * q)) & 1u) x2 &= 0xffff0000u;      // removed positions become +0
                    if ((mask >> (2 * q + 1)) & 1u) x2 &= 0x0000ffffu;
                    uint32_t acc = acc0;
#pragma unroll
                    for (int k = 1; k < K; ++k) acc = add_ge_x2<DT>(acc, x2, t2[k]);
                    r[q] = acc & 0x000f000fu;
                }
                o.x = __byte_perm(r[0], r[1], 0x6420);
                o.y = __byte_perm(r[2], r[3], 0x6420);
                if (codes) {
                    if (vec_out) {
                        *reinterpret_cast<uint2*>(codes + j0) = o;
                    } else {
#pragma unroll
                        for (int u = 0; u < 8; ++u) codes[j0 + u] = (uint8_t)(((u < 4 ? o.x : o.y) >> (8 * (u & 3))) & 0xffu);
                    }
                }
            } else {
                uint32_t code[8];
                float dist[8];
#pragma unroll
                for (int u = 0; u < 8; ++u) {
                    float x = widen16<DT>((uint16_t)(pk[u >> 1] >> (16 * (u & 1))));
                    if ((mask >> u) & 1u) x = 0.f;
                    x = (x == 0.f) ? 0.f : x;  // -0 and +0 are the same point
                    assign_one<K, ERR>(x, c, t, by_threshold, code[u], dist[u]);
                    if (j0 + u >= N) code[u] = 0u;
                }
                o.x = code[0] | (code[1] << 8) | (code[2] << 16) | (code[3] << 24);
                o.y = code[4] | (code[5] << 8) | (code[6] << 16) | (code[7] << 24);
                if (j0 + 7 < N && vec_out) {
                    if (codes) *reinterpret_cast<uint2*>(codes + j0) = o;
                    if (ERR && err) {
                        *reinterpret_cast<float4*>(err + j0) = make_float4(dist[0], dist[1], dist[2], dist[3]);
                        *reinterpret_cast<float4*>(err + j0 + 4) = make_float4(dist[4], dist[5], dist[6], dist[7]);
                    }
                } else {
#pragma unroll
                    for (int u = 0; u < 8; ++u) {
                        if (j0 + u < N) {
                            if (codes) codes[j0 + u] = (uint8_t)code[u];
                            if (ERR && err) err[j0 + u] = dist[u];
                        }
                    }
                }
            }
        }
        if (!ERR && packed) {
            const uint32_t field = squeeze4<C>(o.x) | (squeeze4<C>(o.y) << (4 * C));
            const uint32_t next = __shfl_down_sync(0xffffffffu, field, 1);  // the following eight codes
            const int q = lane & 3;    // position in the group of 32 codes
            const int g = j0 >> 5;
            uint32_t word;
            int widx;
            bool mine;
            if (C == 4) { word = field; widx = g * 4 + q; mine = true; }
            else if (C == 2) { word = field | (next << 16); widx = g * 2 + (q >> 1); mine = (q & 1) == 0; }
            else { word = (field >> (8 * q)) | (next << (24 - 8 * q)); widx = g * 3 + q; mine = q < 3; }
            if (mine && widx < words_per_row) packed[widx] = word;
        }
    }
}

template <int DT, bool ERR>
__global__ void __launch_bounds__(kAssignThreads, ERR ? 4 : 6)
lloyd_assign_kernel(const LloydArgs a, const float* __restrict__ lut, const float* __restrict__ thr) {
    __shared__ uint32_t bitmap[CMPQ_MAX_D_OUT / 32];
    __shared__ int list[kShortList];
    const int64_t row = blockIdx.x;
    const int N = (int)a.d_out;
    const int tid = threadIdx.x, nthr = blockDim.x;
    // request this thread's first 8 weights before the row's metadata: the loads overlap
    uint4 first = make_uint4(0u, 0u, 0u, 0u);
    if (tid * 8 + 7 < N && ((a.ldw & 7) == 0) && ((reinterpret_cast<uintptr_t>(a.W) & 15) == 0))
        first = __ldcs(reinterpret_cast<const uint4*>(a.W + row * a.ldw + tid * 8));
    if (a.skip_row && a.skip_row[row]) return;
    int64_t p0 = 0, p1 = 0;
    if (a.row_ptr) { p0 = a.row_ptr[row]; p1 = a.row_ptr[row + 1]; }
    RemovedCols rem;
    rem.bitmap = bitmap;
    rem.list = list;
    rem.nrem = (int)(p1 - p0);
    if (rem.nrem > kShortList) {
        for (int w = tid; w < (N + 31) / 32; w += nthr) bitmap[w] = 0;
        __syncthreads();
        for (int64_t p = p0 + tid; p < p1; p += nthr) {
            const int col = a.cols[p];
            atomicOr(&bitmap[col >> 5], 1u << (col & 31));
        }
        __syncthreads();
    } else if (rem.nrem > 0) {
        if (tid < rem.nrem) list[tid] = a.cols[p0 + tid];
        __syncthreads();
    }
    const int bits = a.bits[row];
    if (bits == 2) assign_row<DT, 4, ERR>(a, row, lut, thr, rem, first);
    else if (bits == 3) assign_row<DT, 8, ERR>(a, row, lut, thr, rem, first);
    else assign_row<DT, 16, ERR>(a, row, lut, thr, rem, first);
}

// ------------------------------------------------------------------------------------------------
// Selection of the worst-fitted entries (Section 3.2.2) on the value tables.  The error of a
// weight depends only on its value, so the radix select and the per-row counts weigh the error of
// every DISTINCT value with its count instead of reading one error per weight, and the errors are
// never written to memory; the emit kernel recomputes them for the rows that keep entries.

// Centroids and thresholds of a row of the provisional fit, and the error of a value under them.
template <int K>
struct RowFit {
    float c[K], t[K];
    bool by_threshold;
    __device__ __forceinline__ void load(const float* __restrict__ lut, const float* __restrict__ thr, int64_t row) {
#pragma unroll
        for (int k = 0; k < K; ++k) {
            c[k] = __ldg(lut + row * CMPQ_LUT_STRIDE + k);
            t[k] = __ldg(thr + row * CMPQ_LUT_STRIDE + k);
        }
        by_threshold = t[0] != 0.f;
    }
    __device__ __forceinline__ uint32_t err_bits(float x) const {
        uint32_t code;
        float dist;
        assign_one<K, true>(x, c, t, by_threshold, code, dist);
        return __float_as_uint(dist);
    }
};

constexpr int kTableSelWarps = 8;

template <int DT, int K>
__device__ __forceinline__ void table_hist_row(const Tables& t, int64_t row, uint32_t prefix, uint32_t mask, int shift,
                                               int bins, unsigned int* local) {
    const int lane = threadIdx.x & 31;
    RowFit<K> fit;
    fit.load(t.lut, t.thr, row);
    const int M = t.hdr[row].M;
    const uint16_t* keys = t.keys + row * t.stride;
    const uint16_t* cum = t.cum + row * t.stride;
    // eight entries per lane and step: two 128-bit loads, the eight errors are independent
    for (int j0 = lane * 8; j0 < M; j0 += 256) {
        const Eight k8 = load_eight(keys + j0), c8 = load_eight(cum + j0);
        const uint32_t c_end = j0 + 8 <= M ? cum[j0 + 8] : 0u;
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            if (j0 + u < M) {
                const uint32_t e = fit.err_bits(value_of_key16<DT>(k8.at(u)));
                const uint32_t cnt = (u < 7 ? c8.at(u + 1) : c_end) - c8.at(u);
                if ((e & mask) == prefix) atomicAdd(&local[(e >> shift) & (bins - 1)], cnt);
            }
        }
    }
}

// hist[d] += number of weights in non-act rows whose error has the fixed bits of the prefix and the
// digit d at `shift`.  One warp per row, block-local histogram first.
template <int DT>
__global__ void __launch_bounds__(kTableSelWarps * 32)
table_select_hist_kernel(const Tables t, const uint8_t* __restrict__ bits, const uint8_t* __restrict__ is_act,
                         int64_t d_in, SelectState* st, int shift, int bins, int final_pass, unsigned int* hist) {
    __shared__ unsigned int local[kSelBins];
    __shared__ int warp_totals[32];
    __shared__ int found_digit, is_last;
    __shared__ long long found_above;
    for (int b = threadIdx.x; b < bins; b += blockDim.x) local[b] = 0;
    __syncthreads();
    const uint32_t prefix = st->prefix, mask = st->mask;
    const int warp = threadIdx.x >> 5;
    for (int64_t row = (int64_t)blockIdx.x * kTableSelWarps + warp; row < d_in; row += (int64_t)gridDim.x * kTableSelWarps) {
        if (is_act[row]) continue;
        const int b = bits[row];
        if (b == 2) table_hist_row<DT, 4>(t, row, prefix, mask, shift, bins, local);
        else if (b == 3) table_hist_row<DT, 8>(t, row, prefix, mask, shift, bins, local);
        else table_hist_row<DT, 16>(t, row, prefix, mask, shift, bins, local);
    }
    __syncthreads();
    for (int b = threadIdx.x; b < bins; b += blockDim.x)
        if (local[b]) atomicAdd(&hist[b], local[b]);
    // The block that finishes last fixes the digit (no block waits for another: a counter tells which
    // one is last) and leaves the histogram and the counter cleared for the next pass.
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) is_last = atomicAdd(&st->done, 1u) == gridDim.x - 1 ? 1 : 0;
    __syncthreads();
    if (is_last) {
        __threadfence();
        select_digit_block<kTableSelWarps * 32>(hist, shift, bins, st, final_pass, warp_totals, &found_digit, &found_above);
        if (threadIdx.x == 0) st->done = 0;
    }
}

template <int DT, int K>
__device__ __forceinline__ void table_count_row(const Tables& t, int64_t row, uint32_t tau, int& g, int& q) {
    const int lane = threadIdx.x & 31;
    RowFit<K> fit;
    fit.load(t.lut, t.thr, row);
    const int M = t.hdr[row].M;
    const uint16_t* keys = t.keys + row * t.stride;
    const uint16_t* cum = t.cum + row * t.stride;
    for (int j0 = lane * 8; j0 < M; j0 += 256) {
        const Eight k8 = load_eight(keys + j0), c8 = load_eight(cum + j0);
        const uint32_t c_end = j0 + 8 <= M ? cum[j0 + 8] : 0u;
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            if (j0 + u < M) {
                const uint32_t e = fit.err_bits(value_of_key16<DT>(k8.at(u)));
                const int cnt = (int)((u < 7 ? c8.at(u + 1) : c_end) - c8.at(u));
                g += e > tau ? cnt : 0;
                q += e == tau ? cnt : 0;
            }
        }
    }
}

// Per row: how many errors exceed tau and how many equal it.  One warp per row.
template <int DT>
__global__ void __launch_bounds__(kTableSelWarps * 32)
table_row_count_kernel(const Tables t, const uint8_t* __restrict__ bits, const uint8_t* __restrict__ is_act,
                       int64_t d_in, const SelectState* __restrict__ st, int32_t* __restrict__ gt,
                       int32_t* __restrict__ eq) {
    const int64_t row = (int64_t)blockIdx.x * kTableSelWarps + (threadIdx.x >> 5);
    if (row >= d_in) return;
    int g = 0, q = 0;
    if (!is_act[row]) {
        const uint32_t tau = st->tau;
        const int b = bits[row];
        if (b == 2) table_count_row<DT, 4>(t, row, tau, g, q);
        else if (b == 3) table_count_row<DT, 8>(t, row, tau, g, q);
        else table_count_row<DT, 16>(t, row, tau, g, q);
    }
    g = warp_sum(g);
    q = warp_sum(q);
    if ((threadIdx.x & 31) == 0) { gt[row] = g; eq[row] = q; }
}

// Kept entries of one non-act row in column order; errors recomputed from the weights.  Same
// procedure as the emit kernel that reads materialised errors: candidates (error >= tau) go to a
// short list that is ordered by counting; a row with more candidates uses scan-based compaction.
template <int DT, int K>
__device__ void table_emit_row(const uint16_t* __restrict__ w, int64_t d_out, const Tables& t, int64_t row,
                               uint32_t tau, int te, int ncand, int64_t out0, int32_t* __restrict__ rows,
                               int32_t* __restrict__ cols, uint16_t* __restrict__ vals, int* warp_totals,
                               int* list_col, unsigned char* list_eq, int* list_n) {
    RowFit<K> fit;
    fit.load(t.lut, t.thr, row);
    auto err_at = [&](int64_t j) {
        float x = widen16<DT>(w[j]);
        x = (x == 0.f) ? 0.f : x;  // -0 and +0 are the same point
        return fit.err_bits(x);
    };
    if (ncand <= kEmitListCap) {
        if (threadIdx.x == 0) *list_n = 0;
        __syncthreads();
        const bool vec = ((reinterpret_cast<uintptr_t>(w) & 15) == 0);
        for (int64_t j0 = (int64_t)threadIdx.x * 8; j0 < d_out; j0 += (int64_t)blockDim.x * 8) {
            uint32_t pk[4] = {0u, 0u, 0u, 0u};
            if (j0 + 7 < d_out && vec) {
                const uint4 v = __ldg(reinterpret_cast<const uint4*>(w + j0));
                pk[0] = v.x; pk[1] = v.y; pk[2] = v.z; pk[3] = v.w;
            } else {
#pragma unroll
                for (int u = 0; u < 8; ++u)
                    if (j0 + u < d_out) pk[u >> 1] |= (uint32_t)w[j0 + u] << (16 * (u & 1));
            }
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                float x = widen16<DT>((uint16_t)(pk[u >> 1] >> (16 * (u & 1))));
                x = (x == 0.f) ? 0.f : x;  // -0 and +0 are the same point
                const uint32_t e = fit.err_bits(x);
                if (j0 + u < d_out && e >= tau) {
                    const int p = atomicAdd(list_n, 1);
                    if (p < kEmitListCap) {
                        list_col[p] = (int)(j0 + u);
                        list_eq[p] = e == tau ? 1 : 0;
                    }
                }
            }
        }
        __syncthreads();
        const int n = *list_n < kEmitListCap ? *list_n : kEmitListCap;
        for (int i = threadIdx.x; i < n; i += blockDim.x) {
            const int c = list_col[i];
            const int is_eq = list_eq[i];
            int before = 0, eq_before = 0;  // candidates / tau-candidates in lower columns
            for (int u = 0; u < n; ++u) {
                const int lower = list_col[u] < c ? 1 : 0;
                before += lower;
                eq_before += lower & list_eq[u];
            }
            const bool keep = !is_eq || eq_before < te;
            if (keep) {
                // dropped tau-candidates are exactly those of tau-rank >= te, all after the kept ones
                const int dropped_before = eq_before > te ? eq_before - te : 0;
                const int64_t pos = out0 + before - dropped_before;
                rows[pos] = (int32_t)row;
                cols[pos] = c;
                vals[pos] = w[c];
            }
        }
        return;
    }
    int eq_seen = 0, written = 0;
    for (int64_t base = 0; base < d_out; base += blockDim.x) {
        const int64_t j = base + threadIdx.x;
        const bool in = j < d_out;
        const uint32_t u = in ? err_at(j) : 0u;
        const int is_eq = (in && u == tau) ? 1 : 0;
        int tot_eq;
        const int eq_rank = eq_seen + block_exclusive_scan(is_eq, warp_totals, tot_eq);
        const int keep = in && (u > tau || (is_eq && eq_rank < te)) ? 1 : 0;
        int tot_keep;
        const int pos = written + block_exclusive_scan(keep, warp_totals, tot_keep);
        if (keep) {
            rows[out0 + pos] = (int32_t)row;
            cols[out0 + pos] = (int32_t)j;
            vals[out0 + pos] = w[j];
        }
        eq_seen += tot_eq;
        written += tot_keep;
    }
}

template <int DT>
__global__ void __launch_bounds__(kSelThreads)
table_emit_kernel(const uint16_t* __restrict__ W, int64_t ldw, const Tables t, const uint8_t* __restrict__ bits,
                  const uint8_t* __restrict__ is_act, int64_t d_out, const SelectState* __restrict__ st,
                  const int32_t* __restrict__ gt, const int32_t* __restrict__ eq,
                  const int32_t* __restrict__ take_eq, const int64_t* __restrict__ row_start,
                  int32_t* __restrict__ rows, int32_t* __restrict__ cols, uint16_t* __restrict__ vals) {
    __shared__ int warp_totals[32];
    __shared__ int list_col[kEmitListCap];
    __shared__ unsigned char list_eq[kEmitListCap];
    __shared__ int list_n;
    const int64_t row = blockIdx.x;
    const int64_t out0 = row_start[row];
    if (row_start[row + 1] == out0) return;
    const uint16_t* w = W + row * ldw;
    if (is_act[row]) {
        for (int64_t j = threadIdx.x; j < d_out; j += blockDim.x) {
            rows[out0 + j] = (int32_t)row;
            cols[out0 + j] = (int32_t)j;
            vals[out0 + j] = w[j];
        }
        return;
    }
    const uint32_t tau = st->tau;
    const int te = take_eq[row];
    const int ncand = gt[row] + eq[row];
    const int b = bits[row];
    if (b == 2) table_emit_row<DT, 4>(w, d_out, t, row, tau, te, ncand, out0, rows, cols, vals, warp_totals, list_col, list_eq, &list_n);
    else if (b == 3) table_emit_row<DT, 8>(w, d_out, t, row, tau, te, ncand, out0, rows, cols, vals, warp_totals, list_col, list_eq, &list_n);
    else table_emit_row<DT, 16>(w, d_out, t, row, tau, te, ncand, out0, rows, cols, vals, warp_totals, list_col, list_eq, &list_n);
}

static Tables tables_at(void* tables, size_t tables_bytes, int64_t d_in, int64_t d_out) {
    Workspace w(tables, tables_bytes);
    return carve_tables(w, d_in, d_out);
}

cmpq_status launch_table_select_hist(void* tables, size_t tables_bytes, cmpq_dtype dt, const uint8_t* bits,
                                     const uint8_t* is_act, int64_t d_in, int64_t d_out, void* state,
                                     int shift, int bins, int final_pass, unsigned int* hist, cudaStream_t st) {
    const Tables t = tables_at(tables, tables_bytes, d_in, d_out);
    const int sms = sm_count();
    if (sms <= 0) return CMPQ_ERR_CUDA;
    int64_t blocks = (d_in + kTableSelWarps - 1) / kTableSelWarps;
    if (blocks > (int64_t)sms * 4) blocks = (int64_t)sms * 4;
    SelectState* ss = static_cast<SelectState*>(state);
    if (dt == CMPQ_F16)
        table_select_hist_kernel<CMPQ_F16><<<(unsigned)blocks, kTableSelWarps * 32, 0, st>>>(t, bits, is_act, d_in, ss, shift, bins, final_pass, hist);
    else
        table_select_hist_kernel<CMPQ_BF16><<<(unsigned)blocks, kTableSelWarps * 32, 0, st>>>(t, bits, is_act, d_in, ss, shift, bins, final_pass, hist);
    return launch_status();
}

cmpq_status launch_table_row_count(void* tables, size_t tables_bytes, cmpq_dtype dt, const uint8_t* bits,
                                   const uint8_t* is_act, int64_t d_in, int64_t d_out, const void* state,
                                   int32_t* gt, int32_t* eq, cudaStream_t st) {
    const Tables t = tables_at(tables, tables_bytes, d_in, d_out);
    const unsigned blocks = (unsigned)((d_in + kTableSelWarps - 1) / kTableSelWarps);
    const SelectState* ss = static_cast<const SelectState*>(state);
    if (dt == CMPQ_F16)
        table_row_count_kernel<CMPQ_F16><<<blocks, kTableSelWarps * 32, 0, st>>>(t, bits, is_act, d_in, ss, gt, eq);
    else
        table_row_count_kernel<CMPQ_BF16><<<blocks, kTableSelWarps * 32, 0, st>>>(t, bits, is_act, d_in, ss, gt, eq);
    return launch_status();
}

cmpq_status launch_table_emit(void* tables, size_t tables_bytes, cmpq_dtype dt, const uint16_t* W, int64_t ldw,
                              const uint8_t* bits, const uint8_t* is_act, int64_t d_in, int64_t d_out,
                              const void* state, const int32_t* gt, const int32_t* eq, const int32_t* take_eq,
                              const int64_t* row_start, int32_t* rows, int32_t* cols, uint16_t* vals,
                              cudaStream_t st) {
    const Tables t = tables_at(tables, tables_bytes, d_in, d_out);
    const SelectState* ss = static_cast<const SelectState*>(state);
    if (dt == CMPQ_F16)
        table_emit_kernel<CMPQ_F16><<<(unsigned)d_in, kSelThreads, 0, st>>>(W, ldw, t, bits, is_act, d_out, ss, gt, eq, take_eq, row_start, rows, cols, vals);
    else
        table_emit_kernel<CMPQ_BF16><<<(unsigned)d_in, kSelThreads, 0, st>>>(W, ldw, t, bits, is_act, d_out, ss, gt, eq, take_eq, row_start, rows, cols, vals);
    return launch_status();
}

// ------------------------------------------------------------------------------------------------
// host side

template <int DT, int E, int MAXT, int MINB>
static cmpq_status launch_table(const LloydArgs& args, const Tables& t, int threads, cudaStream_t st) {
    const size_t smem = sizeof(TableShared) + (size_t)kSlots * kSlotWords * sizeof(uint32_t) +
                        (((size_t)args.d_out + 31) / 32) * sizeof(uint32_t);
    auto kern = lloyd_table_kernel<DT, E, MAXT, MINB>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
        return CMPQ_ERR_CUDA;
    kern<<<(unsigned)args.d_in, threads, smem, st>>>(args, t);
    return launch_status();
}

// Optional timing of the three kernels: events supplied by cmpq_lloyd_phase_events are recorded
// around them by the next ordered launch, once.
static std::mutex g_phase_mutex;
static cudaEvent_t g_phase_events[4] = {nullptr, nullptr, nullptr, nullptr};

void set_lloyd_phase_events(void* const* events) {
    std::lock_guard<std::mutex> lock(g_phase_mutex);
    for (int i = 0; i < 4; ++i) g_phase_events[i] = events ? static_cast<cudaEvent_t>(events[i]) : nullptr;
}

static void take_phase_events(cudaEvent_t (&ev)[4]) {
    std::lock_guard<std::mutex> lock(g_phase_mutex);
    for (int i = 0; i < 4; ++i) { ev[i] = g_phase_events[i]; g_phase_events[i] = nullptr; }
}

template <int DT>
static cmpq_status launch_table_dt(const LloydArgs& args, const Tables& t, cudaStream_t st) {
    const int64_t N = args.d_out;
    auto threads_for = [N](int e) {
        int64_t th = (N + e - 1) / e;
        th = (th + 31) / 32 * 32;
        return (int)(th < 32 ? 32 : th);
    };
    if (N <= 2048) return launch_table<DT, 4, 512, 2>(args, t, threads_for(4), st);
    if (N <= 4096) return launch_table<DT, 16, 256, 4>(args, t, threads_for(16), st);
    if (N <= 8192) return launch_table<DT, 16, 512, 2>(args, t, threads_for(16), st);
    if (N <= 16384) return launch_table<DT, 16, 1024, 1>(args, t, threads_for(16), st);
    return launch_table<DT, 32, 1024, 1>(args, t, threads_for(32), st);
}

const void* lloyd_table_kernel_address() {
    return reinterpret_cast<const void*>(&lloyd_table_kernel<CMPQ_BF16, 16, 256, 4>);
}

// tables_ready: the value tables of every row to be fitted are in place already (skip the table kernel)
template <int DT>
static cmpq_status launch_ordered_dt(const LloydArgs& args, const Tables& t, bool tables_ready, cudaStream_t st) {
    tables_ready = tables_ready || args.tables_ready;
    if (args.err && args.codes) return CMPQ_ERR_INTERNAL;  // the assign kernel writes one or the other
    cudaEvent_t ev[4];
    take_phase_events(ev);
    if (ev[0]) cudaEventRecord(ev[0], st);
    const int64_t N = args.d_out;
    cmpq_status s = CMPQ_OK;
    if (!tables_ready) s = launch_table_dt<DT>(args, t, st);
    if (s != CMPQ_OK) return s;
    if (ev[1]) cudaEventRecord(ev[1], st);

    IterArgs ia{};
    ia.t = t;
    ia.fc = carve_fit_cache(args.fit_cache, args.d_in);
    ia.bits = args.bits;
    ia.skip_row = args.skip_row;
    ia.d_in = args.d_in;
    ia.d_out = args.d_out;
    ia.iters = args.iters;
    ia.lut = args.lut ? args.lut : t.lut;
    ia.sweeps = args.sweeps;
    // distinct 16-bit values grow slowly with the channel length (about 1400 at 4096 weights, 2300 at
    // 28672 for Gaussian-like bf16 weights); longer tables are read from global memory
    ia.cap = N <= 4096 ? 1536 : (N <= 12288 ? 2048 : 3072);
    const size_t iter_smem = (size_t)kIterWarps * iter_warp_bytes(ia.cap);
    if (cudaFuncSetAttribute(lloyd_iterate_kernel<DT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)iter_smem) !=
        cudaSuccess)
        return CMPQ_ERR_CUDA;
    const unsigned iter_blocks = (unsigned)((args.d_in + kIterWarps - 1) / kIterWarps);
    lloyd_iterate_kernel<DT><<<iter_blocks, kIterWarps * 32, iter_smem, st>>>(ia);
    s = launch_status();
    if (s != CMPQ_OK) return s;
    if (ev[2]) cudaEventRecord(ev[2], st);

    // neither codes nor errors wanted: the fit alone (centroids and thresholds stay in the tables)
    if (args.err) lloyd_assign_kernel<DT, true><<<(unsigned)args.d_in, kAssignThreads, 0, st>>>(args, ia.lut, t.thr);
    else if (args.codes || args.packed) lloyd_assign_kernel<DT, false><<<(unsigned)args.d_in, kAssignThreads, 0, st>>>(args, ia.lut, t.thr);
    s = launch_status();
    if (ev[3]) cudaEventRecord(ev[3], st);
    return s;
}

cmpq_status launch_lloyd_tables(const LloydArgs& args, cmpq_dtype dt, void* tables, size_t tables_bytes,
                                cudaStream_t st) {
    if (!tables || tables_bytes < lloyd_tables_bytes(args.d_in, args.d_out)) return CMPQ_ERR_WORKSPACE;
    const Tables t = tables_at(tables, tables_bytes, args.d_in, args.d_out);
    return dt == CMPQ_F16 ? launch_table_dt<CMPQ_F16>(args, t, st) : launch_table_dt<CMPQ_BF16>(args, t, st);
}

cmpq_status launch_lloyd_ordered(const LloydArgs& args, cmpq_dtype dt, void* tables, size_t tables_bytes,
                                 cudaStream_t st) {
    if (!tables || tables_bytes < lloyd_tables_bytes(args.d_in, args.d_out)) return CMPQ_ERR_WORKSPACE;
    Workspace w(tables, tables_bytes);
    const Tables t = carve_tables(w, args.d_in, args.d_out);
    return dt == CMPQ_F16 ? launch_ordered_dt<CMPQ_F16>(args, t, false, st) : launch_ordered_dt<CMPQ_BF16>(args, t, false, st);
}

// ------------------------------------------------------------------------------------------------
// Final fit from the tables of the provisional fit.  W'' differs from W' only at the positions of
// O_q (and the O_act rows are all zero in both), so the table of a row of W'' is the table of the
// same row of W' with the counts of the removed values moved to the value +0.  One warp per row
// does that for rows with at most kPatchCap removed positions; a row whose every position is
// removed gets the one-entry table of an all-zero channel; the few other rows are flagged and
// rebuilt from the weights by the table kernel.

constexpr int kPatchCap = 64;
constexpr int kPatchWarps = 4;

template <int DT>
__global__ void __launch_bounds__(kPatchWarps * 32)
lloyd_patch_tables_kernel(const uint16_t* __restrict__ W, int64_t ldw, const Tables src, const Tables dst,
                          const int64_t* __restrict__ row_ptr, const int32_t* __restrict__ cols, int64_t d_in,
                          int64_t d_out, int32_t* inexact_rows, uint8_t* __restrict__ skip_rebuild, int cap) {
    extern __shared__ __align__(16) unsigned char patch_smem[];  // per warp: cap keys, cap + 8 count prefixes
    __shared__ uint32_t removed_keys[kPatchWarps][kPatchCap];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t row = (int64_t)blockIdx.x * kPatchWarps + warp;
    if (row >= d_in) return;
    const int N = (int)d_out;
    const int64_t p0 = row_ptr[row];
    const int64_t nrem64 = row_ptr[row + 1] - p0;
    uint16_t* dkeys = dst.keys + row * dst.stride;
    uint16_t* dcum = dst.cum + row * dst.stride;
    const uint32_t kZeroKey = 0x8000u;  // sort key of +0
    if (nrem64 >= N) {  // an all-zero channel
        if (lane == 0) {
            dkeys[0] = (uint16_t)kZeroKey; dcum[0] = 0;
            dkeys[1] = 0xffffu; dcum[1] = (uint16_t)N;
            ChannelHeader h; h.M = 1; h.suspect = 0; dst.hdr[row] = h;
            skip_rebuild[row] = 1;
        }
        return;
    }
    if (nrem64 > kPatchCap) {
        if (lane == 0) skip_rebuild[row] = 0;
        return;
    }
    if (lane == 0) skip_rebuild[row] = 1;
    const int nrem = (int)nrem64;
    uint32_t* rk = removed_keys[warp];
    for (int i = lane; i < nrem; i += 32) {
        uint32_t h = W[row * ldw + cols[p0 + i]];
        if (h == 0x8000u) h = 0u;  // -0 and +0 are the same point
        rk[i] = (h & 0x8000u) ? (~h & 0xffffu) : (h | 0x8000u);
    }
    __syncwarp();
    const int M = src.hdr[row].M;
    const uint16_t* skeys = src.keys + row * src.stride;
    const uint16_t* scum = src.cum + row * src.stride;
    if (M <= cap) {  // stage the old table in shared memory: all its loads are in flight at once
        uint16_t* s_keys = reinterpret_cast<uint16_t*>(patch_smem + (size_t)warp * (4 * (size_t)cap + 16));
        uint16_t* s_cum = s_keys + cap;
        for (int i = lane; i < (M + 7) / 8; i += 32)
            reinterpret_cast<uint4*>(s_keys)[i] = __ldg(reinterpret_cast<const uint4*>(skeys) + i);
        for (int i = lane; i < (M + 1 + 7) / 8; i += 32)
            reinterpret_cast<uint4*>(s_cum)[i] = __ldg(reinterpret_cast<const uint4*>(scum) + i);
        __syncwarp();
        skeys = s_keys;
        scum = s_cum;
    }
    // where +0 sits in the old table, or would sit
    int lo = 0, hi = M;
    while (lo < hi) {
        const int mid = (lo + hi) >> 1;
        if ((uint32_t)skeys[mid] >= kZeroKey) hi = mid; else lo = mid + 1;
    }
    const int pos0 = lo;
    const bool present = pos0 < M && (uint32_t)skeys[pos0] == kZeroKey;
    const int ins = (nrem > 0 && !present) ? 1 : 0;  // +0 becomes a new entry
    const int Mm = M + ins;
    // The magnitude range of the old table proved its sums exact: so are those of any subset with zeros
    // added, and the bit-by-bit test is skipped.
    const bool test = inexact_rows && src.hdr[row].suspect;
    int deleted = 0;  // entries dropped so far (their count fell to zero)
    uint32_t amax = 0u;
    int q = 100000;
    for (int base = 0; base < Mm; base += 32) {
        const int i = base + lane;
        const bool valid = i < Mm;
        uint32_t key = kZeroKey;
        int cnt = 0, below = 0;  // weights with this value / with a smaller value in the old table
        if (valid) {
            if (ins && i == pos0) {
                below = (int)scum[pos0];
            } else {
                const int j = (ins && i > pos0) ? i - 1 : i;
                key = skeys[j];
                below = (int)scum[j];
                cnt = (int)scum[j + 1] - below;
            }
            int eq = 0, lt = 0;
            for (int r = 0; r < nrem; ++r) {
                const uint32_t k = rk[r];
                eq += k == key ? 1 : 0;
                lt += k < key ? 1 : 0;
            }
            cnt -= eq;
            below -= lt;
            if (key == kZeroKey) cnt += nrem;      // the removed weights are zeros now
            if (key > kZeroKey) below += nrem;
        }
        const bool keep = cnt > 0;
        const uint32_t gone = __ballot_sync(0xffffffffu, valid && !keep);
        if (keep) {
            const int o = i - deleted - __popc(gone & ((1u << lane) - 1u));
            dkeys[o] = (uint16_t)key;
            dcum[o] = (uint16_t)below;
            if (test) {
                const uint32_t ub = __float_as_uint(value_of_key16<DT>(key)) & 0x7fffffffu;
                if (ub) {
                    amax = max(amax, ub);
                    const int ex = (int)(ub >> 23);
                    const uint32_t m = ub & 0x7fffffu;
                    q = min(q, ex ? ex - 150 + (__ffs(m | 0x800000u) - 1) : (__ffs(m) - 1) - 149);
                }
            }
        }
        deleted += __popc(gone);
    }
    if (lane == 0) {
        const int out = Mm - deleted;
        dkeys[out] = 0xffffu;
        dcum[out] = (uint16_t)N;
        ChannelHeader h; h.M = out; h.suspect = src.hdr[row].suspect; dst.hdr[row] = h;
    }
    if (test) {  // the exactness test of the table kernel, on the new table
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            amax = max(amax, __shfl_xor_sync(0xffffffffu, amax, o));
            q = min(q, __shfl_xor_sync(0xffffffffu, q, o));
        }
        if (lane == 0 && amax != 0u) {
            const int log2n = 32 - __clz(N - 1 > 0 ? N - 1 : 1);
            const int ex_max = (int)(amax >> 23);
            const int top = ex_max ? ex_max - 127 : (31 - __clz(amax)) - 149;
            if (log2n + 1 + (top + 1 - q) > 53) atomicAdd(inexact_rows, 1);
        }
    }
}

// args: the final fit (row_ptr / cols = the removed positions, skip_row unused).  prov_tables: the
// tables the provisional fit left; tables: scratch of the final fit; skip_rebuild: d_in bytes.
cmpq_status launch_lloyd_ordered_patched(const LloydArgs& args, cmpq_dtype dt, void* prov_tables, void* tables,
                                         size_t tables_bytes, uint8_t* skip_rebuild, cudaStream_t st) {
    if (!prov_tables || !tables || tables_bytes < lloyd_tables_bytes(args.d_in, args.d_out)) return CMPQ_ERR_WORKSPACE;
    const Tables src = tables_at(prov_tables, tables_bytes, args.d_in, args.d_out);
    const Tables dst = tables_at(tables, tables_bytes, args.d_in, args.d_out);
    const unsigned blocks = (unsigned)((args.d_in + kPatchWarps - 1) / kPatchWarps);
    const int cap = args.d_out <= 4096 ? 1536 : (args.d_out <= 12288 ? 2048 : 3072);  // as in the iterate kernel
    const size_t smem = (size_t)kPatchWarps * (4 * (size_t)cap + 16);
    if (cudaFuncSetAttribute(lloyd_patch_tables_kernel<CMPQ_F16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess ||
        cudaFuncSetAttribute(lloyd_patch_tables_kernel<CMPQ_BF16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
        return CMPQ_ERR_CUDA;
    if (dt == CMPQ_F16)
        lloyd_patch_tables_kernel<CMPQ_F16><<<blocks, kPatchWarps * 32, smem, st>>>(args.W, args.ldw, src, dst, args.row_ptr, args.cols, args.d_in, args.d_out, args.inexact_rows, skip_rebuild, cap);
    else
        lloyd_patch_tables_kernel<CMPQ_BF16><<<blocks, kPatchWarps * 32, smem, st>>>(args.W, args.ldw, src, dst, args.row_ptr, args.cols, args.d_in, args.d_out, args.inexact_rows, skip_rebuild, cap);
    cmpq_status s = launch_status();
    if (s != CMPQ_OK) return s;
    LloydArgs rebuild = args;  // rows with too many removed positions for the patch: from the weights
    rebuild.skip_row = skip_rebuild;
    s = dt == CMPQ_F16 ? launch_table_dt<CMPQ_F16>(rebuild, dst, st) : launch_table_dt<CMPQ_BF16>(rebuild, dst, st);
    if (s != CMPQ_OK) return s;
    return dt == CMPQ_F16 ? launch_ordered_dt<CMPQ_F16>(args, dst, true, st) : launch_ordered_dt<CMPQ_BF16>(args, dst, true, st);
}

}  // namespace cmpq
