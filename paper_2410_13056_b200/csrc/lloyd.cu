// Channel-wise K-means of CMPQ (Section 3.2.1: K-means per channel W_{i,:} with K = 2^bits;
// Section 3: each weight is replaced by its nearest centroid).
//
// One thread block fits one channel.  Nothing here is a dense contraction: the work is K
// subtract / compare steps per weight per sweep on the fp32 pipes, so no tensor cores are used.
//
//   load        the channel is read from HBM once, removed positions are zeroed, and the weights
//               are SORTED by value inside the block with a two-level counting sort on their
//               16-bit keys (high byte, then low byte inside each high-byte bucket).  Thread t
//               then keeps the E consecutive order statistics [E t, E t + E) in REGISTERS for all
//               iterations, so an iteration moves no HBM bytes.
//   start       the K order statistics xs[((2k+1) N)/(2K)] are read straight from the sorted array
//   sweep       defined as: the first k minimising fabsf(x - c_k) (fp32, strict '<' scan), for
//               every weight and every centroid.  When the centroids are strictly increasing and
//               every gap exceeds 2^-22 times the channel's value range, x - c_k and x - c_{k-1}
//               can never round to the same float, and then that first minimum equals the number
//               of k >= 1 with fabsf(x - c_k) < fabsf(x - c_{k-1}); the sweep counts those with one
//               subtract, one compare and one predicated add per (weight, centroid) and the codes
//               are non-decreasing along the sorted order.  Otherwise it runs the plain scan.
//   update      with non-decreasing codes a cluster is a run [B_k, B_{k+1}) of the sorted order:
//               its count is B_{k+1} - B_k and its sum a difference of fp64 prefix sums (per-thread
//               totals scanned once at load, plus at most E-1 weights of the thread that holds the
//               boundary).  The boundaries come from K-1 warp votes.  16-bit weights of bounded
//               dynamic range make these fp64 sums exact, so they equal the sums taken in any
//               other order.  Without the ordering guarantee the sums are rebuilt by plain
//               per-cluster accumulation.
//   stop        a sweep that moves no boundary (changes no code) ends the loop early: later
//               iterations would repeat it exactly
//   output      codes / errors are put back into column order through shared memory and stored
//               with coalesced writes
#include "lloyd.cuh"
#include "lloyd_device.cuh"

#include <atomic>

namespace cmpq {

constexpr int kMaxWarps = 32;
constexpr int kSortSlots = 32;  // high-byte buckets refined per pass of the sort's second level
static_assert(CMPQ_MAX_D_OUT < 65536, "the sort's second-level counters are 16 bits wide");

struct alignas(16) LloydShared {
    double* pt4;                       // [nthr E / 4 + 1] fp64 sum of the first 4 i sorted weights
    double (*wsum)[kMaxK];             // [nwarps][K] per-warp cluster sums (rebuild path)
    int (*wcnt)[kMaxK];                // [nwarps][K] per-warp counts (rebuild) / threads below boundary k
    int hist1[256];
    int excl1[257];
    int bucket_rank[256];              // rank of a high-byte bucket among the non-empty ones, or -1
    float c[kMaxK];                    // centroids for the next sweep, written by warp 0
    int below_total[kMaxK];            // ordered path: threads of the block entirely below boundary k
    int flag_fast, flag_moved;         // warp 0's decisions: counting sweep valid / a boundary moved
    int n_nonempty;
    float vmin, vmax;                  // value range of the channel
    float wlo[kMaxWarps], whi[kMaxWarps];
    int wtop[kMaxWarps], wulp[kMaxWarps];
};
// dynamic shared memory after LloydShared:
//   scratch (lloyd_scratch_bytes): removed-column bitmap during the load, second-level histogram
//                                  during the sort, then the threads' packed codes
//   sorted  (4 bytes per weight):  key << 16 | column, ascending; reused for the output staging

__host__ __device__ inline size_t lloyd_pt_bytes(int nthr, int E) { return (((size_t)nthr * E / 4 + 1) * sizeof(double) + 15) & ~(size_t)15; }

__host__ __device__ inline size_t lloyd_codes_bytes(int nthr, int E) { return (size_t)nthr * ((E + 7) / 8) * 4; }
__host__ __device__ inline size_t lloyd_tail_bytes(int nthr, int E) {
    return lloyd_pt_bytes(nthr, E) + (size_t)(nthr / 32) * 16 * (sizeof(double) + sizeof(int));
}
__host__ __device__ inline bool lloyd_tail_fits_scratch(int nthr, int E) {
    return lloyd_codes_bytes(nthr, E) + lloyd_tail_bytes(nthr, E) <= (size_t)16 * 256 * sizeof(int);
}

__host__ __device__ inline int lloyd_scratch_bytes(int /*N*/) {
    // 16 KiB = kSortSlots x 256 16-bit counters >= 16 bytes x 1024 threads >= 32768 bits
    return kSortSlots * 128 * (int)sizeof(uint32_t);
}

// In-place exclusive prefix of 256 16-bit counters packed two per word (128 words, 16-byte
// aligned), by one warp: 4 words per lane.
__device__ __forceinline__ void warp_scan256_packed(uint32_t* h) {
    const int lane = threadIdx.x & 31;
    uint4 v = reinterpret_cast<uint4*>(h)[lane];
    uint32_t w[4] = {v.x, v.y, v.z, v.w};
    uint32_t s = 0;
#pragma unroll
    for (int t = 0; t < 4; ++t) s += (w[t] & 0xffffu) + (w[t] >> 16);
    uint32_t incl = s;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        uint32_t up = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += up;
    }
    uint32_t run = incl - s;
#pragma unroll
    for (int t = 0; t < 4; ++t) {
        uint32_t lo = run;
        run += w[t] & 0xffffu;
        uint32_t hi = run;
        run += w[t] >> 16;
        w[t] = lo | (hi << 16);
    }
    reinterpret_cast<uint4*>(h)[lane] = make_uint4(w[0], w[1], w[2], w[3]);
}

// Sorts the block's weights by 16-bit key into `sorted` (key << 16 | column).  key[e] belongs to
// column ((e >> 2) * nthr + tid) * 4 + (e & 3); the first nval of a thread's keys are real.
template <int E>
__device__ void sort_channel(const uint32_t (&key)[E], int nval, LloydShared& sh, int* hist2,
                             uint32_t* sorted) {
    const int tid = threadIdx.x, nthr = blockDim.x, lane = tid & 31, warp = tid >> 5;
    const int nwarps = nthr >> 5;
    for (int b = tid; b < 256; b += nthr) sh.hist1[b] = 0;
    __syncthreads();
#pragma unroll
    for (int e = 0; e < E; ++e)
        if (e < nval) atomicAdd(&sh.hist1[key[e] >> 8], 1);
    __syncthreads();
    if (warp == 0) {
        int total = warp_scan256(sh.hist1, sh.excl1);
        if (lane == 0) sh.excl1[256] = total;
        // rank of every non-empty bucket among the non-empty ones
        int flag[8], s = 0;
#pragma unroll
        for (int t = 0; t < 8; ++t) { flag[t] = sh.hist1[lane * 8 + t] > 0; s += flag[t]; }
        int incl = s;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            int up = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += up;
        }
        int run = incl - s;
#pragma unroll
        for (int t = 0; t < 8; ++t) { sh.bucket_rank[lane * 8 + t] = flag[t] ? run : -1; run += flag[t]; }
        if (lane == 31) sh.n_nonempty = incl;
    }
    __syncthreads();
    // Second level: the low byte inside each non-empty high-byte bucket, kSortSlots buckets at a
    // time.  Two 16-bit counters share a word (a channel has at most 32768 weights, so neither a
    // count nor a prefix inside one bucket reaches 2^16 and the halves never carry into each other).
    uint32_t* h2 = reinterpret_cast<uint32_t*>(hist2);
    const int ngroups = (sh.n_nonempty + kSortSlots - 1) / kSortSlots;
    for (int grp = 0; grp < ngroups; ++grp) {
        for (int b = tid; b < kSortSlots * 32; b += nthr) reinterpret_cast<uint4*>(h2)[b] = make_uint4(0u, 0u, 0u, 0u);
        __syncthreads();
#pragma unroll
        for (int e = 0; e < E; ++e) {
            if (e < nval) {
                int r = sh.bucket_rank[key[e] >> 8];
                uint32_t lo = key[e] & 0xffu;
                if ((r >> 5) == grp) atomicAdd(&h2[(r & 31) * 128 + (lo >> 1)], 1u << (16 * (lo & 1u)));
            }
        }
        __syncthreads();
        for (int s = warp; s < kSortSlots; s += nwarps) warp_scan256_packed(h2 + s * 128);
        __syncthreads();
#pragma unroll
        for (int e = 0; e < E; ++e) {
            if (e < nval) {
                int r = sh.bucket_rank[key[e] >> 8];
                uint32_t lo = key[e] & 0xffu;
                if ((r >> 5) == grp) {
                    uint32_t sh16 = 16 * (lo & 1u);
                    uint32_t old = atomicAdd(&h2[(r & 31) * 128 + (lo >> 1)], 1u << sh16);
                    int pos = sh.excl1[key[e] >> 8] + (int)((old >> sh16) & 0xffffu);
                    uint32_t col = (uint32_t)(((e >> 2) * nthr + tid) * 4 + (e & 3));
                    sorted[pos] = (key[e] << 16) | col;
                }
            }
        }
        __syncthreads();
    }
}

// Per-warp cluster sums and counts of all weights, from the codes in registers (any order).
template <int K, int E>
__device__ void rebuild_partials(const float (&x)[E], const uint32_t (&cw)[(E + 7) / 8], int nval,
                                 LloydShared& sh) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    int code[E];
#pragma unroll
    for (int e = 0; e < E; ++e) code[e] = (e < nval) ? (int)((cw[e >> 3] >> (4 * (e & 7))) & 15u) : -1;
#pragma unroll 1
    for (int k = 0; k < K; ++k) {
        double s = 0.0;
        int cnt = 0;
#pragma unroll
        for (int e = 0; e < E; ++e) {
            bool mine = code[e] == k;
            s += mine ? (double)x[e] : 0.0;
            cnt += mine ? 1 : 0;
        }
        s = warp_sum(s);
        cnt = warp_sum(cnt);
        if (lane == 0) { sh.wsum[warp][k] = s; sh.wcnt[warp][k] = cnt; }
    }
}

// Rebuild path, warp 0: lane k combines the per-warp partials of cluster k and moves
// the centroid to the mean if the cluster has members.
template <int K>
__device__ __forceinline__ float centroid_from_partials(const LloydShared& sh, float ck, int nwarps) {
    const int lane = threadIdx.x & 31;
    if (lane < K) {
        double s = 0.0;
        int cnt = 0;
        for (int w = 0; w < nwarps; ++w) { s += sh.wsum[w][lane]; cnt += sh.wcnt[w][lane]; }
        if (cnt > 0) ck = __double2float_rn(__ddiv_rn(s, (double)cnt));
    }
    return ck;
}

// Number of the E packed 4-bit codes that are below k (byte-wise SWAR compare of the even and the
// odd nibbles: n + 128 - k has bit 7 set exactly when n >= k).
template <int E>
struct PackedCodes { uint32_t w[(E + 7) / 8]; };

template <int E>
__device__ __forceinline__ int count_below(const PackedCodes<E>& pc, int k) {
    constexpr int WORDS = (E + 7) / 8;
    const uint32_t (&cw)[WORDS] = pc.w;
    const uint32_t kk = (uint32_t)k * 0x01010101u;
    int ge = 0;
#pragma unroll
    for (int w = 0; w < WORDS; ++w) {
        uint32_t ev = cw[w] & 0x0f0f0f0fu, od = (cw[w] >> 4) & 0x0f0f0f0fu;
        ge += __popc(((ev | 0x80808080u) - kk) & 0x80808080u) + __popc(((od | 0x80808080u) - kk) & 0x80808080u);
    }
    // a word holding fewer than 8 codes has zero padding nibbles: they compare as "below"
    return 8 * WORDS - ge - (8 * WORDS - E);
}

// Warp 0, lane k (0..K) holds B_k = number of weights (in sorted order) before cluster k, B_0 = 0
// and B_K = N: cluster k is the run [B_k, B_{k+1}) of the sorted order.  Its fp64 sum is a
// difference of prefix sums P_k (table at every fourth weight plus at most three weights read from
// the sorted array).  Returns the new centroid of cluster `lane` (the old one if the run is empty).
template <int DT, int K>
__device__ __forceinline__ float centroid_from_runs(const LloydShared& sh, const uint32_t* sorted, int N,
                                                    float ck, int B) {
    const int lane = threadIdx.x & 31;
    double P = 0.0;
    if (lane <= K) {
        const int q = B >> 2, r = B & 3;
        double tail[3];  // the three loads are independent of r, so they overlap
#pragma unroll
        for (int e = 0; e < 3; ++e) {
            const int idx = 4 * q + e < N ? 4 * q + e : N - 1;
            tail[e] = (double)value_of_key16<DT>(sorted[idx] >> 16);
        }
        P = sh.pt4[q];
#pragma unroll
        for (int e = 0; e < 3; ++e)
            if (e < r) P += tail[e];
    }
    const int Bn = __shfl_down_sync(0xffffffffu, B, 1);
    const double Pn = __shfl_down_sync(0xffffffffu, P, 1);
    if (lane < K) {
        const int cnt = Bn - B;
        if (cnt > 0) ck = __double2float_rn(__ddiv_rn(Pn - P, (double)cnt));
    }
    return ck;
}

// All-pairs path, warp 0: lane k (0..K) evaluates B_k = number of weights with a code below k from
//   sh.below_total[k] = threads whose last code is < k  (k = 1..K-1); read and cleared here
//   codes_s[t]        = packed codes of thread t
// and returns the new centroid of cluster `lane`; B_out = B_lane.
template <int DT, int K, int E>
__device__ __forceinline__ float centroid_from_boundaries(LloydShared& sh, const uint32_t* codes_s,
                                                          const uint32_t* sorted, int N, float ck, int& B_out) {
    constexpr int WORDS = (E + 7) / 8;
    const int lane = threadIdx.x & 31, nthr = blockDim.x;
    int B = 0;
    if (lane == K) {
        B = N;
    } else if (lane > 0 && lane < K) {
        const int t = sh.below_total[lane];
        sh.below_total[lane] = 0;
        B = t * E;
        if (t < nthr) {  // thread t is the first whose last code reaches k: its weights below k
            PackedCodes<E> pc;
#pragma unroll
            for (int w = 0; w < WORDS; ++w) pc.w[w] = codes_s[t * WORDS + w];
            B += count_below<E>(pc, lane);
        }
        if (B > N) B = N;
    }
    B_out = B;
    return centroid_from_runs<DT, K>(sh, sorted, N, ck, B);
}

// One sweep over a thread's E weights: their codes for the centroids c, packed 8 per word.
template <int K, int E>
__device__ __forceinline__ void sweep_codes(const float (&x)[E], const float (&c)[K], bool fast,
                                            uint32_t (&nw)[(E + 7) / 8]) {
    constexpr int G = E / 4, WORDS = (E + 7) / 8;
    uint32_t half[G];  // 16 bits: the codes of weights 4g..4g+3
    if (fast) {
#pragma unroll
        for (int g = 0; g < G; ++g) {
            // 2^23 + sum code_u 16^u is exact in fp32, so the low mantissa bits are the codes
            float acc = 8388608.f;
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const float xv = x[4 * g + u];
                const float inc = (float)(1 << (4 * u));
                float dp = fabsf(xv - c[0]);
#pragma unroll
                for (int k = 1; k < K; ++k) {
                    float d = fabsf(xv - c[k]);
                    if (d < dp) acc += inc;
                    dp = d;
                }
            }
            half[g] = __float_as_uint(acc);
        }
    } else {
#pragma unroll
        for (int g = 0; g < G; ++g) {
            uint32_t p = 0;
#pragma unroll
            for (int u = 0; u < 4; ++u) p |= (uint32_t)nearest_scan<K>(x[4 * g + u], c) << (4 * u);
            half[g] = p;
        }
    }
#pragma unroll
    for (int w = 0; w < WORDS; ++w)
        nw[w] = (2 * w + 1 < G) ? __byte_perm(half[2 * w], half[2 * w + 1], 0x5410) : (half[2 * w] & 0xffffu);
}

// Outputs of one channel, staged through shared memory back into column order.  Called by every
// thread of the block after a barrier that follows the last read of keys from `sorted`; sh.c holds
// the final centroids.
template <int E>
__device__ void write_outputs(const LloydArgs& a, int64_t row, int K, const LloydShared& sh, uint32_t* sorted,
                              const float (&x)[E], const uint32_t (&cw)[(E + 7) / 8], int nval,
                              int sweeps_done) {
    const int tid = threadIdx.x, nthr = blockDim.x;
    const int N = (int)a.d_out;
    if (a.lut && tid < CMPQ_LUT_STRIDE) a.lut[row * CMPQ_LUT_STRIDE + tid] = tid < K ? sh.c[tid] : 0.f;
    uint32_t colv[E];
#pragma unroll
    for (int e = 0; e < E; ++e) colv[e] = (e < nval) ? (sorted[tid * E + e] & 0xffffu) : 0u;
    __syncthreads();  // every thread has its columns: `sorted` may be overwritten
    if (a.codes) {
        uint8_t* stage = reinterpret_cast<uint8_t*>(sorted);
#pragma unroll
        for (int e = 0; e < E; ++e)
            if (e < nval) stage[colv[e]] = (uint8_t)((cw[e >> 3] >> (4 * (e & 7))) & 15u);
        __syncthreads();
        uint8_t* out = a.codes + row * a.d_out;
        if ((a.d_out & 3) == 0) {
            const uint32_t* s4 = reinterpret_cast<const uint32_t*>(stage);
            uint32_t* o4 = reinterpret_cast<uint32_t*>(out);
            for (int j = tid; j < (N >> 2); j += nthr) o4[j] = s4[j];
        } else {
            for (int j = tid; j < N; j += nthr) out[j] = stage[j];
        }
    }
    if (a.err) {
        float* stage = reinterpret_cast<float*>(sorted);
#pragma unroll
        for (int e = 0; e < E; ++e)
            if (e < nval) stage[colv[e]] = fabsf(x[e] - sh.c[(cw[e >> 3] >> (4 * (e & 7))) & 15u]);
        __syncthreads();
        float* out = a.err + row * a.d_out;
        for (int j = tid; j < N; j += nthr) out[j] = stage[j];
    }
    if (a.sweeps && tid == 0)
        atomicAdd(a.sweeps, (unsigned long long)sweeps_done * (unsigned long long)N * (unsigned long long)K);
}

template <int DT, int K, int E>
__device__ void fit_channel(const LloydArgs& a, int64_t row, const float (&x)[E], int nval,
                            LloydShared& sh, uint32_t* codes_s, uint32_t* sorted) {
    constexpr int WORDS = (E + 7) / 8;  // packed codes: 8 weights per 32-bit word
    const int tid = threadIdx.x, nthr = blockDim.x, lane = tid & 31, warp = tid >> 5;
    const int N = (int)a.d_out;
    const int T = a.iters;
    const double need = ((double)sh.vmax - (double)sh.vmin) * (1.0 / 4194304.0);  // range * 2^-22

    // Warp 0 owns the centroids (lane k holds c_k) and publishes them, with the mode of the next
    // sweep, in shared memory; a sweep costs two barriers and the update is computed once.
    float ck_lane = 0.f;
    int B_prev = -1;  // warp 0, lane k: B_k of the previous ordered sweep (-1: none)
    if (warp == 0) {
        if (lane < K) {
            int pos = (int)(((long long)(2 * lane + 1) * N) / (2 * K));  // K evenly spaced order statistics
            ck_lane = value_of_key16<DT>(sorted[pos] >> 16);
            sh.c[lane] = ck_lane;
        }
        const bool f = counting_sweep_valid<K>(ck_lane, need);
        if (lane == 0) { sh.flag_fast = f ? 1 : 0; sh.flag_moved = 1; }
        if (lane < kMaxK) sh.below_total[lane] = 0;
    }
    __syncthreads();

    uint32_t cw[WORDS];
#pragma unroll
    for (int w = 0; w < WORDS; ++w) cw[w] = 0xffffffffu;
    float c[K];
    int sweeps_done = 0;
    for (int it = 0; it <= T; ++it) {
#pragma unroll
        for (int k = 0; k < K; ++k) c[k] = sh.c[k];
        const bool fast = sh.flag_fast != 0;
        const bool last = (it == T);

        uint32_t nw[WORDS];
        sweep_codes<K, E>(x, c, fast, nw);
        ++sweeps_done;
        uint32_t any = 0;
#pragma unroll
        for (int w = 0; w < WORDS; ++w) { any |= nw[w] ^ cw[w]; cw[w] = nw[w]; }
        if (last) break;

        if (fast) {
            // codes are non-decreasing along the sorted order: publish them and add, per warp, how many of
            // its threads lie entirely below each boundary to the block's totals.  The threads' last codes are non-decreasing
            // along the lanes: a boundary at or below the first lane's code adds nothing, one above the last
            // lane's code adds 32, and a lane whose successor has a larger code owns those in between.
#pragma unroll
            for (int w = 0; w < WORDS; ++w) codes_s[tid * WORDS + w] = cw[w];
            const int c_last = (int)((cw[WORDS - 1] >> (4 * ((E - 1) & 7))) & 15u);
            const int c31 = __shfl_sync(0xffffffffu, c_last, 31);
            const int c_next = __shfl_down_sync(0xffffffffu, c_last, 1);
            if (lane > 0 && lane < K && lane > c31) atomicAdd(&sh.below_total[lane], 32);
            if (lane < 31 && c_next > c_last)
                for (int k = c_last + 1; k <= c_next; ++k) atomicAdd(&sh.below_total[k], lane + 1);
            __syncthreads();
            if (warp == 0) {
                int B;
                ck_lane = centroid_from_boundaries<DT, K, E>(sh, codes_s, sorted, N, ck_lane, B);
                const bool moved = __any_sync(0xffffffffu, lane < K && B != B_prev);
                B_prev = B;
                const bool f = counting_sweep_valid<K>(ck_lane, need);
                if (lane < K) sh.c[lane] = ck_lane;
                if (lane == 0) { sh.flag_fast = f ? 1 : 0; sh.flag_moved = moved ? 1 : 0; }
            }
            __syncthreads();
            if (!sh.flag_moved) break;  // no boundary moved: later sweeps would repeat this one
        } else {
            const int changed = __syncthreads_or(any != 0);
            if (!changed) break;
            rebuild_partials<K, E>(x, cw, nval, sh);
            __syncthreads();
            if (warp == 0) {
                ck_lane = centroid_from_partials<K>(sh, ck_lane, nthr >> 5);
                const bool f = counting_sweep_valid<K>(ck_lane, need);
                if (lane < K) sh.c[lane] = ck_lane;
                if (lane == 0) sh.flag_fast = f ? 1 : 0;
                B_prev = -1;
            }
            __syncthreads();
        }
    }
    __syncthreads();  // sh.c holds the final centroids; no thread reads keys from `sorted` after this point
    write_outputs<E>(a, row, K, sh, sorted, x, cw, nval, sweeps_done);
}

// One-time work for a channel, by every thread of the block: read the row, zero the removed
// positions, note the value range and the exactness diagnostics, sort it into `sorted`, load this
// thread's run of E order statistics into x and build the fp64 prefix table sh.pt4.
template <int DT, int E>
__device__ void prepare_channel(const LloydArgs& a, int64_t row, LloydShared& sh, unsigned char* scratch,
                                uint32_t* sorted, float (&x)[E], int& nval_out) {
    const int N = (int)a.d_out;
    const int tid = threadIdx.x, nthr = blockDim.x, lane = tid & 31, warp = tid >> 5;
    uint32_t key[E];
    int nval_cols = 0;
    load_channel_keys<DT, E>(a, row, sh, reinterpret_cast<uint32_t*>(scratch), key, nval_cols);

    sort_channel<E>(key, nval_cols, sh, reinterpret_cast<int*>(scratch), sorted);

    // sorted layout: thread t keeps order statistics [E t, E t + E); padding repeats the maximum
    int nval = N - tid * E;
    nval = nval < 0 ? 0 : (nval > E ? E : nval);
    {
        const float vlast = value_of_key16<DT>(sorted[N - 1] >> 16);
        double tot = 0.0;
#pragma unroll
        for (int e = 0; e < E; ++e) {
            if (e < nval) {
                x[e] = value_of_key16<DT>(sorted[tid * E + e] >> 16);
                tot += (double)x[e];
            } else {
                x[e] = vlast;
            }
        }
        // exclusive scan of the thread totals over the block, then the table at every fourth weight
        double incl = tot;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            double up = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += up;
        }
        if (lane == 31) sh.wsum[warp][0] = incl;
        __syncthreads();
        double run = incl - tot;
        for (int wv = 0; wv < warp; ++wv) run += sh.wsum[wv][0];
#pragma unroll
        for (int g = 0; g < E / 4; ++g) {
            sh.pt4[tid * (E / 4) + g] = run;
#pragma unroll
            for (int u = 0; u < 4; ++u)
                if (4 * g + u < nval) run += (double)x[4 * g + u];
        }
        if (tid == nthr - 1) sh.pt4[nthr * (E / 4)] = run;
        __syncthreads();
    }

    nval_out = nval;
}

template <int DT, int E, int MAXT, int MINB>
__global__ void __launch_bounds__(MAXT, MINB)
lloyd_kernel(const LloydArgs a) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const int64_t row = blockIdx.x;
    if (a.skip_row && a.skip_row[row]) return;
    const int N = (int)a.d_out;
    LloydShared& sh = *reinterpret_cast<LloydShared*>(smem_raw);
    const int tid = threadIdx.x, nthr = blockDim.x;
    const int nwarps = nthr >> 5;
    unsigned char* scratch = smem_raw + sizeof(LloydShared);
    uint32_t* sorted = reinterpret_cast<uint32_t*>(scratch + lloyd_scratch_bytes(N));
    // prefix table and per-warp exchange arrays: inside the scratch region (behind the packed codes)
    // when they fit there -- they are first written after the sort is done with it -- else behind `sorted`
    unsigned char* tail = lloyd_tail_fits_scratch(nthr, E)
                              ? scratch + lloyd_codes_bytes(nthr, E)
                              : reinterpret_cast<unsigned char*>(sorted) + (((size_t)N + 3) & ~(size_t)3) * 4;
    if (tid == 0) {  // published by the first barrier below, long before anyone uses them
        sh.pt4 = reinterpret_cast<double*>(tail);
        sh.wsum = reinterpret_cast<double (*)[kMaxK]>(tail + lloyd_pt_bytes(nthr, E));
        sh.wcnt = reinterpret_cast<int (*)[kMaxK]>(tail + lloyd_pt_bytes(nthr, E) + (size_t)nwarps * kMaxK * sizeof(double));
    }

    float x[E];
    int nval;
    prepare_channel<DT, E>(a, row, sh, scratch, sorted, x, nval);

    uint32_t* codes_s = reinterpret_cast<uint32_t*>(scratch);  // [nthr][WORDS], at most 16 KiB
    const int bits = a.bits[row];
    if (bits == 2) fit_channel<DT, 4, E>(a, row, x, nval, sh, codes_s, sorted);
    else if (bits == 3) fit_channel<DT, 8, E>(a, row, x, nval, sh, codes_s, sorted);
    else fit_channel<DT, 16, E>(a, row, x, nval, sh, codes_s, sorted);
}

static size_t lloyd_smem_bytes(int64_t d_out, int threads, int E) {
    size_t bytes = sizeof(LloydShared) + (size_t)lloyd_scratch_bytes((int)d_out) + (((size_t)d_out + 3) & ~(size_t)3) * 4;
    if (!lloyd_tail_fits_scratch(threads, E)) bytes += lloyd_tail_bytes(threads, E);
    return bytes;
}

template <int DT, int E, int MAXT, int MINB>
static cmpq_status launch_variant(const LloydArgs& args, int threads, cudaStream_t st) {
    const size_t smem = lloyd_smem_bytes(args.d_out, threads, E);
    auto kern = lloyd_kernel<DT, E, MAXT, MINB>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
        return CMPQ_ERR_CUDA;
    kern<<<(unsigned)args.d_in, threads, smem, st>>>(args);
    return launch_status();
}

template <int DT>
static cmpq_status launch_dt(const LloydArgs& args, cudaStream_t st) {
    const int64_t N = args.d_out;
    auto threads_for = [N](int e) {
        int64_t t = (N + e - 1) / e;
        t = (t + 31) / 32 * 32;
        return (int)(t < 32 ? 32 : t);
    };
    if (N <= 2048) return launch_variant<DT, 4, 512, 1>(args, threads_for(4), st);
    if (N <= 4096) return launch_variant<DT, 16, 256, 4>(args, threads_for(16), st);
    if (N <= 8192) return launch_variant<DT, 16, 512, 2>(args, threads_for(16), st);
    if (N <= 12288) return launch_variant<DT, 32, 384, 2>(args, threads_for(32), st);
    if (N <= 16384) return launch_variant<DT, 16, 1024, 1>(args, threads_for(16), st);
    return launch_variant<DT, 32, 1024, 1>(args, threads_for(32), st);
}

static std::atomic<int> g_assignment{CMPQ_ASSIGN_ORDERED};

cmpq_lloyd_assignment lloyd_assignment() { return (cmpq_lloyd_assignment)g_assignment.load(); }

cmpq_status launch_lloyd(const LloydArgs& args, cmpq_dtype dt, cudaStream_t st) {
    return dt == CMPQ_F16 ? launch_dt<CMPQ_F16>(args, st) : launch_dt<CMPQ_BF16>(args, st);
}

// row_ptr[r] = first position p with rows[p] >= r; every thread owns one position and fills the
// row numbers between its predecessor's row and its own.
__global__ void row_ptr_kernel(const int32_t* __restrict__ rows, int64_t nnz, int64_t d_in,
                               int64_t* __restrict__ row_ptr) {
    int64_t p = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (p > nnz) return;
    int64_t prev = p == 0 ? -1 : (int64_t)rows[p - 1];
    int64_t cur = p == nnz ? d_in : (int64_t)rows[p];
    for (int64_t r = prev + 1; r <= cur; ++r) row_ptr[r] = p;
}

cmpq_status launch_row_ptr(const int32_t* rows, int64_t nnz, int64_t d_in, int64_t* row_ptr,
                           cudaStream_t st) {
    if (nnz == 0) {
        if (cudaMemsetAsync(row_ptr, 0, (size_t)(d_in + 1) * sizeof(int64_t), st) != cudaSuccess) return CMPQ_ERR_CUDA;
        return CMPQ_OK;
    }
    row_ptr_kernel<<<(unsigned)((nnz + 1 + 255) / 256), 256, 0, st>>>(rows, nnz, d_in, row_ptr);
    return launch_status();
}

static size_t row_ptr_bytes(int64_t d_in) { return round_up((size_t)(d_in + 1) * sizeof(int64_t), 256); }

size_t quantize_ws_bytes(int64_t d_in, int64_t d_out) {
    return row_ptr_bytes(d_in) + lloyd_tables_bytes(d_in, d_out);
}

}  // namespace cmpq

using namespace cmpq;

extern "C" cmpq_status cmpq_set_lloyd_assignment(cmpq_lloyd_assignment mode) {
    if (mode != CMPQ_ASSIGN_ORDERED && mode != CMPQ_ASSIGN_ALL_PAIRS) return CMPQ_ERR_INVALID_ARG;
    g_assignment.store((int)mode);
    return CMPQ_OK;
}

extern "C" cmpq_lloyd_assignment cmpq_get_lloyd_assignment(void) { return lloyd_assignment(); }

extern "C" cmpq_status cmpq_lloyd_phase_events(void* before_table, void* after_table, void* after_iterate,
                                               void* after_assign) {
    if (!before_table && !after_table && !after_iterate && !after_assign) {
        set_lloyd_phase_events(nullptr);
        return CMPQ_OK;
    }
    if (!before_table || !after_table || !after_iterate || !after_assign) return CMPQ_ERR_INVALID_ARG;
    void* ev[4] = {before_table, after_table, after_iterate, after_assign};
    set_lloyd_phase_events(ev);
    return CMPQ_OK;
}

namespace cmpq {
cmpq_status launch_pack_layout(const uint8_t* bits, int64_t d_in, int64_t d_out, int64_t* row_off, int32_t* perm,
                               int64_t* seg_rows, int64_t* word_off, cudaStream_t st);
cmpq_status launch_pack_codes(const uint8_t* codes, const uint8_t* bits, int64_t d_in, int64_t d_out,
                              const int64_t* word_off, uint32_t* packed, cudaStream_t st);

size_t quantize_packed_ws_bytes(int64_t d_in, int64_t d_out) {
    return quantize_ws_bytes(d_in, d_out) + pack_ws_bytes(d_in, d_out);
}

// The final fit; with `packed` also the packing, fused into the last assignment where the formulation allows.
static cmpq_status quantize_impl(const void* W, cmpq_dtype dt, int64_t d_in, int64_t d_out, int64_t ldw,
                                 const uint8_t* bits, const int32_t* rows, const int32_t* cols, int64_t nnz,
                                 int lloyd_iters, const float* sens, float* lut, uint8_t* codes, uint32_t* packed,
                                 int64_t* row_off, int32_t* perm, int64_t* seg_rows, int32_t* inexact_rows,
                                 unsigned long long* sweeps, int32_t* nonfinite, void* ws, size_t ws_bytes,
                                 void* stream) {
    if (!W || !bits || !lut) return CMPQ_ERR_INVALID_ARG;
    if (!codes && !packed) return CMPQ_ERR_INVALID_ARG;
    if (dt != CMPQ_F16 && dt != CMPQ_BF16) return CMPQ_ERR_INVALID_ARG;
    if (d_in < 1 || d_in > CMPQ_MAX_D_IN || d_out < 1 || d_out > CMPQ_MAX_D_OUT || ldw < d_out)
        return CMPQ_ERR_INVALID_ARG;
    if (nnz < 0 || nnz > d_in * d_out || (nnz > 0 && (!rows || !cols))) return CMPQ_ERR_INVALID_ARG;
    if (lloyd_iters < 0 || lloyd_iters > CMPQ_MAX_LLOYD_ITERS) return CMPQ_ERR_INVALID_ARG;
    if (!aligned_to(W, 2) || !aligned_to(lut, 4)) return CMPQ_ERR_INVALID_ARG;
    if (codes && !aligned_to(codes, 8)) return CMPQ_ERR_INVALID_ARG;  // eight codes leave in one store
    if (sens && !aligned_to(sens, 4)) return CMPQ_ERR_INVALID_ARG;
    if (!aligned_to(nonfinite, 4)) return CMPQ_ERR_INVALID_ARG;
    if (packed && (!row_off || !perm || !seg_rows || !aligned_to(packed, 4) || !aligned_to(row_off, 8) ||
                   !aligned_to(perm, 4) || !aligned_to(seg_rows, 8)))
        return CMPQ_ERR_INVALID_ARG;
    const bool fused_pack_ok = !sens && lloyd_assignment() != CMPQ_ASSIGN_ALL_PAIRS;
    if (packed && !codes && !fused_pack_ok) return CMPQ_ERR_UNSUPPORTED;  // those kernels write byte codes
    const size_t need = packed ? quantize_packed_ws_bytes(d_in, d_out) : quantize_ws_bytes(d_in, d_out);
    if (!ws || !aligned_to(ws, 256) || ws_bytes < need) return CMPQ_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int64_t* row_ptr = static_cast<int64_t*>(ws);
    int64_t* word_off = reinterpret_cast<int64_t*>(static_cast<char*>(ws) + quantize_ws_bytes(d_in, d_out));
    cmpq_status s = launch_row_ptr(rows, nnz, d_in, row_ptr, st);
    if (s != CMPQ_OK) return s;
    if (packed) {
        s = launch_pack_layout(bits, d_in, d_out, row_off, perm, seg_rows, word_off, st);
        if (s != CMPQ_OK) return s;
    }
    LloydArgs a{};
    a.W = static_cast<const uint16_t*>(W);
    a.d_in = d_in; a.d_out = d_out; a.ldw = ldw;
    a.bits = bits;
    a.iters = lloyd_iters;
    a.row_ptr = row_ptr;
    a.cols = cols;
    a.lut = lut;
    a.codes = codes;
    a.inexact_rows = inexact_rows;
    a.sweeps = sweeps;
    a.nonfinite = nonfinite;
    if (!fused_pack_ok) {
        if (sens && lloyd_assignment() != CMPQ_ASSIGN_ALL_PAIRS)
            s = launch_lloyd_weighted_tables(a, dt, sens, static_cast<char*>(ws) + row_ptr_bytes(d_in),
                                             lloyd_tables_bytes(d_in, d_out), st);
        else
            s = sens ? launch_lloyd_weighted(a, dt, sens, st) : launch_lloyd(a, dt, st);
        if (s != CMPQ_OK || !packed) return s;
        return launch_pack_codes(codes, bits, d_in, d_out, word_off, packed, st);
    }
    a.packed = packed;
    a.word_off = word_off;
    return launch_lloyd_ordered(a, dt, static_cast<char*>(ws) + row_ptr_bytes(d_in), lloyd_tables_bytes(d_in, d_out), st);
}

}  // namespace cmpq

extern "C" cmpq_status cmpq_quantize_layer(const void* W, cmpq_dtype dt, int64_t d_in, int64_t d_out,
                                           int64_t ldw, const uint8_t* bits, const int32_t* rows,
                                           const int32_t* cols, int64_t nnz, int lloyd_iters,
                                           const float* sens, float* lut, uint8_t* codes,
                                           int32_t* inexact_rows, unsigned long long* sweeps,
                                           int32_t* nonfinite, void* ws, size_t ws_bytes, void* stream) {
    if (!codes) return CMPQ_ERR_INVALID_ARG;
    return quantize_impl(W, dt, d_in, d_out, ldw, bits, rows, cols, nnz, lloyd_iters, sens, lut, codes, nullptr,
                         nullptr, nullptr, nullptr, inexact_rows, sweeps, nonfinite, ws, ws_bytes, stream);
}

extern "C" cmpq_status cmpq_quantize_layer_packed(const void* W, cmpq_dtype dt, int64_t d_in, int64_t d_out,
                                                  int64_t ldw, const uint8_t* bits, const int32_t* rows,
                                                  const int32_t* cols, int64_t nnz, int lloyd_iters,
                                                  const float* sens, float* lut, uint8_t* codes, uint32_t* packed,
                                                  int64_t* row_off, int32_t* perm, int64_t* seg_rows,
                                                  int32_t* inexact_rows, unsigned long long* sweeps,
                                                  int32_t* nonfinite, void* ws, size_t ws_bytes, void* stream) {
    if (!packed) return CMPQ_ERR_INVALID_ARG;
    return quantize_impl(W, dt, d_in, d_out, ldw, bits, rows, cols, nnz, lloyd_iters, sens, lut, codes, packed,
                         row_off, perm, seg_rows, inexact_rows, sweeps, nonfinite, ws, ws_bytes, stream);
}
