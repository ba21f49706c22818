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

constexpr int kSlotWords = 128;  // 256 low-byte counters of 16 bits, two per word
constexpr uint32_t kZeroKeyOfTable = 0x8000u;  // sort key of +0
constexpr int kStageCap = 4096;  // table entries of one pass gathered in shared memory before they are stored
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
    int64_t sum_stride;  // doubles per channel in `sum`
    double* sum;         // [d_in][sum_stride] prefix sums at every eighth entry, for tables too large for shared memory
    float* lut;          // [d_in][16] centroids for the assign kernel when the caller wants no lut
    float* thr;          // [d_in][16] value thresholds of the last assignment ([0]: 1 if valid)
    uint16_t* bnd;       // [d_in][32] provisional fit with valid thresholds: [2k] first entry of cluster k,
                         // [2k+1] its first entry whose value is >= c_k (the cluster ends where the next begins)
    uint32_t* kept;      // [d_in][32] after the selection: [0] = n, then the n keys of the row's values that keep
                         // entries (bit 16: only some of their entries, error equal to the threshold);
                         // n = kKeptUnknown: not listed
};

// d_out + 1 entries and the sentinel, plus one entry of slack while a table is patched in place
static int64_t table_stride(int64_t d_out) { return (d_out + 2 + 7) / 8 * 8; }

static Tables carve_tables(Workspace& w, int64_t d_in, int64_t d_out) {
    Tables t;
    t.stride = table_stride(d_out);
    t.hdr = w.take<ChannelHeader>(d_in);
    t.keys = w.take<uint16_t>((size_t)d_in * t.stride);
    t.cum = w.take<uint16_t>((size_t)d_in * t.stride);
    t.sum_stride = t.stride / 8 + 2;
    t.sum = w.take<double>((size_t)d_in * t.sum_stride);
    t.lut = w.take<float>((size_t)d_in * CMPQ_LUT_STRIDE);
    t.thr = w.take<float>((size_t)d_in * CMPQ_LUT_STRIDE);
    t.bnd = w.take<uint16_t>((size_t)d_in * 32);
    t.kept = w.take<uint32_t>((size_t)d_in * 32);
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
constexpr int kScanWords = 16;  // counter words a thread owns at most on the register path of the scan

struct alignas(16) TableShared {
    unsigned char hist1[256];  // 1 where the high byte occurs
    int bucket_rank[256];      // rank of a high-byte bucket among the non-empty ones, or -1
    int slot_hi[256];          // the inverse: high byte of the r-th non-empty bucket
    int n_nonempty;
    int wtop[32], wulp[32];  // per-warp magnitude range (largest pattern, smallest non-zero pattern - 1)
    uint32_t w_scan[32];     // per-warp totals of the block scan: entries << 16 | weights
    int base_nz, base_cnt;   // entries / weights emitted by the previous passes
    int rem_list[kShortList];
};
// dynamic shared memory after TableShared: SLOTS * kSlotWords words of second-level counters, then a bitmap of
// d_out bits for rows with many removed positions, then the staging area of one pass (key | prefix << 16)

// Sort keys of two 16-bit patterns at once (neither half is -0): a positive pattern gets its top bit set,
// a negative one is complemented.
__device__ __forceinline__ uint32_t keys_of_patterns_x2(uint32_t w) {
    const uint32_t s = w & 0x80008000u;
    return w ^ (0x80008000u | (s - (s >> 15)));
}

// E weights per thread, at most MAXT threads; SLOTS high-byte buckets are refined per pass.
template <int DT, int E, int MAXT, int MINB, int SLOTS>
__global__ void __launch_bounds__(MAXT, MINB)
lloyd_table_kernel(const LloydArgs a, const Tables t) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const int64_t row = blockIdx.x;
    if (a.skip_row && a.skip_row[row]) return;
    TableShared& sh = *reinterpret_cast<TableShared*>(smem_raw);
    uint32_t* h2 = reinterpret_cast<uint32_t*>(smem_raw + sizeof(TableShared));
    uint32_t* bitmap = h2 + SLOTS * kSlotWords;
    uint32_t* stage = bitmap + (a.d_out + 31) / 32;  // entries of one pass, gathered
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
    for (int i = tid; i < 64; i += nthr) reinterpret_cast<uint32_t*>(sh.hist1)[i] = 0u;
    for (int i = tid; i < SLOTS * kSlotWords / 4; i += nthr) reinterpret_cast<uint4*>(h2)[i] = make_uint4(0u, 0u, 0u, 0u);
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

    // keys (removed positions and -0 become +0), which high bytes occur, range of the magnitudes.  A group of
    // VEC weights that lies inside the row, has no removed position and no zero is handled two weights at a
    // time; everything else weight by weight.
    uint32_t kw[E / 2];  // two keys per word
    uint32_t valid = 0;  // bit e: key e is a weight of the row
    uint32_t amax = 0u, amin1 = 0xffffffffu;
    uint32_t amax2 = 0u, amin2 = 0xffffffffu;  // the same for the pairs: one magnitude per half
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
        uint32_t has_zero = 0u;  // non-zero if some magnitude of the group is zero (may also be set without one)
#pragma unroll
        for (int u = 0; u < VEC / 2; ++u) {
            const uint32_t m = raw[g * (VEC / 2) + u] & 0x7fff7fffu;
            has_zero |= (m - 0x00010001u) & ~m & 0x80008000u;
        }
        if (j0 + VEC - 1 < N && rm == 0u && has_zero == 0u) {
            valid |= ((1u << VEC) - 1u) << (g * VEC);
#pragma unroll
            for (int u = 0; u < VEC / 2; ++u) {
                const uint32_t word = raw[g * (VEC / 2) + u];
                const uint32_t m = word & 0x7fff7fffu;
                const uint32_t k2 = keys_of_patterns_x2(word);
                kw[g * (VEC / 2) + u] = k2;
                amax2 = __vmaxu2(amax2, m);
                amin2 = __vminu2(amin2, m - 0x00010001u);  // no half is zero: no borrow
                sh.hist1[(k2 >> 8) & 0xffu] = 1;
                sh.hist1[k2 >> 24] = 1;
            }
        } else {
#pragma unroll
            for (int u = 0; u < VEC; ++u) {
                const int e = g * VEC + u;
                uint32_t h = (raw[e >> 1] >> (16 * (e & 1))) & 0xffffu;
                if ((rm >> u) & 1u) h = 0u;
                if (h == 0x8000u) h = 0u;  // -0 and +0 are the same point
                const uint32_t ub = h & 0x7fffu;
                const uint32_t key = (h & 0x8000u) ? (~h & 0xffffu) : (h | 0x8000u);
                if (e & 1) kw[e >> 1] |= key << 16;
                else kw[e >> 1] = key;
                if (j0 + u < N) {
                    valid |= 1u << e;
                    amax = max(amax, ub);
                    amin1 = min(amin1, ub - 1u);  // zero wraps to the largest value
                    sh.hist1[key >> 8] = 1;
                }
            }
        }
    }
    amax = max(amax, max(amax2 & 0xffffu, amax2 >> 16));
    amin1 = min(amin1, min(amin2 & 0xffffu, amin2 >> 16));  // untouched halves read 0xffff: above every pattern - 1
    amax = __reduce_max_sync(0xffffffffu, amax);
    amin1 = __reduce_min_sync(0xffffffffu, amin1);
    if (lane == 0) { sh.wtop[warp] = (int)amax; sh.wulp[warp] = (int)amin1; }
    // Every table holds an entry for +0, with count 0 if no weight is zero: a later fit of the same weights
    // with some positions removed (set to +0) then only changes counts, never the list of entries.
    if (tid == 0) sh.hist1[kZeroKeyOfTable >> 8] = 1;
    __syncthreads();
    if (warp == 0) {
        const uint2 eight = reinterpret_cast<const uint2*>(sh.hist1)[lane];
        int flag[8], sum = 0;
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            flag[u] = (int)(((u < 4 ? eight.x : eight.y) >> (8 * (u & 3))) & 1u);
            sum += flag[u];
        }
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
        amax = __reduce_max_sync(0xffffffffu, lane < nwarps ? (uint32_t)sh.wtop[lane] : 0u);
        amin1 = __reduce_min_sync(0xffffffffu, lane < nwarps ? (uint32_t)sh.wulp[lane] : 0xffffffffu);
        // the largest magnitude pattern of the row tells whether any weight is a NaN or an infinity
        if (a.nonfinite && tid == 0 && amax >= (DT == CMPQ_BF16 ? 0x7f80u : 0x7c00u)) atomicOr(a.nonfinite, 2);
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
                    const uint32_t key = (kw[e >> 1] >> (16 * (e & 1))) & 0xffffu;
                    const uint32_t ub = __float_as_uint(value_of_key16<DT>(key)) & 0x7fffffffu;
                    if (((valid >> e) & 1u) && ub) {
                        const int ex = (int)(ub >> 23);
                        const uint32_t m = ub & 0x7fffffu;
                        q = min(q, ex ? ex - 150 + (__ffs(m | 0x800000u) - 1) : (__ffs(m) - 1) - 149);
                    }
                }
                q = __reduce_min_sync(0xffffffffu, q);
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
    constexpr uint32_t kAllValid = E == 32 ? 0xffffffffu : (1u << E) - 1u;
    int run_nz = 0, run_cnt = 0;
    for (int g0 = 0; g0 < n_nonempty; g0 += SLOTS) {
        const int nslots = n_nonempty - g0 < SLOTS ? n_nonempty - g0 : SLOTS;
        const int words_total = nslots * kSlotWords;
        // Second level: the low byte inside the buckets g0 .. g0 + nslots.  Two 16-bit counters share a
        // word (a channel has fewer than 2^16 weights, so the halves never carry into each other).
        if (g0 > 0) {  // the counters of the first pass were cleared at the start
            for (int w = tid; w < words_total / 4; w += nthr) reinterpret_cast<uint4*>(h2)[w] = make_uint4(0u, 0u, 0u, 0u);
            __syncthreads();  // also: the previous pass has published its bases
        }
#pragma unroll
        for (int e = 0; e < E; ++e) {
            if (valid == kAllValid || ((valid >> e) & 1u)) {
                const uint32_t key = (kw[e >> 1] >> (16 * (e & 1))) & 0xffffu;
                const int r = sh.bucket_rank[key >> 8] - g0;
                if ((unsigned)r < (unsigned)SLOTS) atomicAdd(&h2[r * kSlotWords + ((key & 0xffu) >> 1)], (key & 1u) ? 0x10000u : 1u);
            }
        }
        __syncthreads();
        // Every thread owns a contiguous range of counters: totals first, a block scan, then the entries.
        // With at most kScanWords words per thread (a power of two, so a range stays inside one bucket) the
        // counters of a thread are held in registers between the two steps.
        int wpt = 4;
        while (wpt * nthr < words_total) wpt *= 2;
        const bool in_regs = wpt <= kScanWords;
        const int w0 = in_regs ? min(tid * wpt, words_total) : (int)((unsigned)tid * (unsigned)words_total / (unsigned)nthr);
        const int w1 = in_regs ? min(w0 + wpt, words_total) : (int)((unsigned)(tid + 1) * (unsigned)words_total / (unsigned)nthr);
        const int r_zero = sh.bucket_rank[kZeroKeyOfTable >> 8] - g0;  // the counter of +0 always makes an entry
        const int w_zero = (r_zero >= 0 && r_zero < nslots) ? r_zero * kSlotWords : -1;
        uint32_t occupied = 0;  // bit 2 (w - w0) + half: that counter makes an entry (register path)
        int nz = 0, cnt = 0;
        if (in_regs) {
            uint32_t total = 0;
#pragma unroll
            for (int q = 0; q < kScanWords / 4; ++q) {
                uint4 v = make_uint4(0u, 0u, 0u, 0u);
                if (w0 + 4 * q < w1) v = *reinterpret_cast<const uint4*>(h2 + w0 + 4 * q);
                const uint32_t wd[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    total = __dp2a_lo(wd[i], 0x0101u, total);  // both halves added
                    occupied |= ((wd[i] & 0xffffu) ? 1u : 0u) << (2 * (4 * q + i));
                    occupied |= ((wd[i] >> 16) ? 1u : 0u) << (2 * (4 * q + i) + 1);
                }
            }
            if (w_zero >= w0 && w_zero < w1) occupied |= 1u << (2 * (w_zero - w0));
            nz = __popc(occupied);
            cnt = (int)total;
        } else {
            for (int w = w0; w < w1; ++w) {
                const uint32_t word = h2[w];
                const int c0 = (int)(word & 0xffffu), c1 = (int)(word >> 16);
                nz += ((c0 != 0 || w == w_zero) ? 1 : 0) + (c1 != 0 ? 1 : 0);
                cnt += c0 + c1;
            }
        }
        // block scan of (entries, weights) in one word: neither total reaches 2^16
        const uint32_t mine = ((uint32_t)nz << 16) | (uint32_t)cnt;
        uint32_t incl = mine;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const uint32_t up = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += up;
        }
        if (lane == 31) sh.w_scan[warp] = incl;
        __syncthreads();
        const uint32_t wv = lane < nwarps ? sh.w_scan[lane] : 0u;
        const uint32_t before = __reduce_add_sync(0xffffffffu, lane < warp ? wv : 0u) + incl - mine;
        const int pass_nz = (int)(__reduce_add_sync(0xffffffffu, wv) >> 16);  // entries of this pass (all warps)
        run_nz = sh.base_nz + (int)(before >> 16);
        run_cnt = sh.base_cnt + (int)(before & 0xffffu);
        // The entries of a pass are gathered in shared memory when they fit and leave in order with
        // coalesced stores.
        const bool staged = pass_nz <= kStageCap;
        const int stage_base = sh.base_nz;
        auto emit_range = [&](auto&& put) {
            if (in_regs) {  // a thread walks the set bits of its range instead of every counter
                const uint32_t kb0 = w0 < words_total
                    ? ((uint32_t)sh.slot_hi[g0 + (w0 >> 7)] << 8) | ((uint32_t)(w0 & 127) << 1) : 0u;
                while (occupied) {
                    const int b = __ffs(occupied) - 1;
                    occupied &= occupied - 1u;
                    const uint32_t word = h2[w0 + (b >> 1)];
                    put(kb0 + (uint32_t)b, (int)((b & 1) ? word >> 16 : word & 0xffffu));
                }
            } else {
                for (int w = w0; w < w1; ++w) {
                    const uint32_t word = h2[w];
                    if (word || w == w_zero) {
                        const uint32_t kb = ((uint32_t)sh.slot_hi[g0 + (w >> 7)] << 8) | ((uint32_t)(w & 127) << 1);
                        const int c0 = (int)(word & 0xffffu), c1 = (int)(word >> 16);
                        if (c0 || w == w_zero) put(kb, c0);
                        if (c1) put(kb | 1u, c1);
                    }
                }
            }
        };
        if (staged) {
            uint32_t* out = stage - stage_base;
            emit_range([&](uint32_t k, int c) {
                out[run_nz] = k | ((uint32_t)run_cnt << 16);
                ++run_nz;
                run_cnt += c;
            });
        } else {
            emit_range([&](uint32_t k, int c) {
                keys[run_nz] = (uint16_t)k;
                cum[run_nz] = (uint16_t)run_cnt;
                ++run_nz;
                run_cnt += c;
            });
        }
        __syncthreads();  // every thread has read the bases and the counters of this pass
        if (staged) {
            for (int i = tid; i < pass_nz; i += nthr) {
                const uint32_t en = stage[i];
                keys[stage_base + i] = (uint16_t)en;
                cum[stage_base + i] = (uint16_t)(en >> 16);
            }
        }
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
// fits kept between calls

// fits kept between calls (see lloyd.cuh): slot (bits - 2) * d_in + row
struct FitCacheHeader {
    int iters;  // the iteration count the cached fits were made with
};
struct FitCache {
    FitCacheHeader* hdr;  // NULL: no cache
    uint8_t* valid;
    float* lut;
    float* thr;
    uint16_t* bnd;
};

static FitCache carve_fit_cache(void* p, int64_t d_in) {
    FitCache c{};
    if (!p) return c;
    Workspace w(p, ~(size_t)0);
    c.hdr = w.take<FitCacheHeader>(1);
    c.valid = w.take<uint8_t>(3 * (size_t)d_in);
    c.lut = w.take<float>(3 * (size_t)d_in * CMPQ_LUT_STRIDE);
    c.thr = w.take<float>(3 * (size_t)d_in * CMPQ_LUT_STRIDE);
    c.bnd = w.take<uint16_t>(3 * (size_t)d_in * 32);
    return c;
}

size_t lloyd_fit_cache_bytes(int64_t d_in) {
    return 256 + round_up(3 * (size_t)d_in, 256) + 2 * round_up(3 * (size_t)d_in * CMPQ_LUT_STRIDE * sizeof(float), 256) +
           round_up(3 * (size_t)d_in * 32 * sizeof(uint16_t), 256);
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
    int cap;     // table entries a channel can stage in shared memory (multiple of 16)
    float* lut;  // [d_in][16]
    unsigned long long* sweeps;
    // Final fit derived from the tables an earlier fit of the same weights left in `src`: this launch's
    // table of a channel is src's with the positions row_ptr / cols removed (set to +0), built by the
    // channel's lanes in shared memory (or in t, for tables too large to stage).  src.hdr == NULL: the
    // tables in t are complete already.
    Tables src;
    const uint16_t* W;
    int64_t ldw;
    const int64_t* row_ptr;
    const int32_t* cols;
    int32_t* inexact_rows;
    const int32_t* nonfinite;  // optional flag word of the call: once it is set the iterations are skipped
    unsigned int* side_hist;   // provisional fit of the outlier step (see LloydArgs), else NULL
};

// ------------------------------------------------------------------------------------------------
// iterations: one half-warp per channel, two channels per warp
//
// While the centroids are strictly increasing with safe gaps, cluster k of a channel is the run of
// table entries between two boundaries, and the boundary between clusters k-1 and k is a 16-bit KEY:
// the first key b (in sort-key order) whose value is closer to c_k than to c_{k-1} under the defining
// fp32 rule.  Between the two centroids fl(c_k - v) falls and fl(v - c_{k-1}) rises with v whatever the
// rounding does, so the rule is monotone there and b is well defined; it lies next to the midpoint, so
// b is found with two evaluations of the rule on register operands (no table access) in all but rare
// cases, which fall back to bisection over keys.  The boundary as a table index -- how many table keys
// lie below b -- is then read off the sixteen keys around the lane's previous boundary (boundaries move
// by a few entries per iteration), with bisection over the rest of the table when it moved further.
// The kernel is bound by the latency of this dependent chain (every channel of a layer is resident at
// once), so the chain is kept short: no fp64 on the way to the boundary, the partial sums below a
// boundary as a tree of independent products, one vote per iteration.

constexpr int kGroup = 16;     // lanes that share one channel
constexpr int kIterWarps = 2;  // warps per block: four channels
constexpr int kKeyPad = 16;    // staged keys are followed by this many 0xffff entries

// Shared memory of one channel: prefix sums at every eighth entry, keys (padded), count prefixes (table
// of at most `cap` entries, cap a multiple of 16).
constexpr int kPatchChunk = 64;  // removed positions of a channel handled per pass over its table (their keys
                                 // borrow the space of the prefix sums, which are built afterwards)
constexpr int kMinIterCap = 1536;  // smallest table capacity the host ever chooses
static_assert(kPatchChunk * 4 <= (kMinIterCap / 8 + 2) * 8, "the prefix-sum area holds a chunk of removed keys");
__host__ __device__ inline size_t iter_channel_bytes(int cap) {
    const size_t b = (size_t)(cap / 8 + 2) * 8 + (size_t)(cap + kKeyPad) * 2 + (size_t)(cap + 8) * 2;
    return (b + 15) / 16 * 16;
}

__device__ __forceinline__ unsigned group_mask() { return 0xffffu << (threadIdx.x & 16); }

// Largest 16-bit storage value <= f / smallest >= f, as sort keys (f finite).
__device__ __forceinline__ uint32_t key_of_pattern(uint32_t h) {
    if ((h & 0x7fffu) == 0u) h = 0u;  // -0 and +0 are the same point
    return (h & 0x8000u) ? (~h & 0xffffu) : (h | 0x8000u);
}
template <int DT>
__device__ __forceinline__ uint32_t key_floor(float f) {
    uint32_t h;
    if (DT == CMPQ_BF16) {
        const uint32_t u = __float_as_uint(f);
        h = (u & 0x80000000u) ? ((u + 0xffffu) >> 16) : (u >> 16);  // negative: the magnitude rounds up
    } else {
        h = __half_as_ushort(__float2half_rd(f));
    }
    return key_of_pattern(h);
}
template <int DT>
__device__ __forceinline__ uint32_t key_ceil(float f) {
    uint32_t h;
    if (DT == CMPQ_BF16) {
        const uint32_t u = __float_as_uint(f);
        h = (u & 0x80000000u) ? (u >> 16) : ((u + 0xffffu) >> 16);
    } else {
        h = __half_as_ushort(__float2half_ru(f));
    }
    return key_of_pattern(h);
}

// The defining rule on one storage value given as a key: closer to ck than to cm (cm < ck)?
template <int DT>
__device__ __forceinline__ bool nearer_upper(uint32_t key, float cm, float ck) {
    const float v = value_of_key16<DT>(key);
    return fabsf(v - ck) < fabsf(v - cm);
}

// First key in [kfirst, kend] for which the rule holds, kend (one past the table's last key) counting as
// true: every table key below the result goes to cluster k-1 or lower, every other one to k or higher.
template <int DT>
__device__ __forceinline__ uint32_t boundary_key(float cm, float ck, uint32_t kfirst, uint32_t kend) {
    // candidate: the first storage value at or above the midpoint (fp32 is enough for a candidate)
    uint32_t kc = key_ceil<DT>(0.5f * cm + 0.5f * ck);
    kc = kc < kfirst ? kfirst : (kc > kend ? kend : kc);
    const bool at = kc >= kend ? true : nearer_upper<DT>(kc, cm, ck);
    const bool before = kc <= kfirst ? false : nearer_upper<DT>(kc - 1u, cm, ck);
    if (at && !before) return kc;  // inside [cm, ck] the rule is monotone: this is the only change
    // values <= cm are never nearer to ck; values >= ck inside the table's range always are
    uint32_t lo = key_floor<DT>(cm) + 1u;
    if (lo < kfirst) lo = kfirst;
    uint32_t hi = key_ceil<DT>(ck);
    if (hi > kend) hi = kend;
    if (lo >= hi) return lo < kend ? lo : kend;
    if (kc >= lo && kc <= hi) {  // use what the two evaluations told (kc - 1 holds the rule when kc does)
        if (!at) lo = kc + 1u; else hi = kc - 1u;
    }
    while (lo < hi) {  // hi always names a key for which the rule holds
        const uint32_t mid = (lo + hi) >> 1;
        if (nearer_upper<DT>(mid, cm, ck)) hi = mid; else lo = mid + 1u;
    }
    return lo;
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

// Number of table entries whose key is below b.  hint >= 0 (staged tables only: the keys are followed by
// kKeyPad entries of 0xffff): the sixteen keys around entry `hint` are examined first.
__device__ __forceinline__ int rank_of_key(const uint16_t* keys, int M, uint32_t b, int hint) {
    int lo = 0, hi = M;
    if (hint >= 0) {
        int j0 = (hint & ~7) - 8;
        if (j0 < 0) j0 = 0;
        const Eight a8 = load_eight(keys + j0), b8 = load_eight(keys + j0 + 8);
        // the sixteen keys ascend: bisection on registers (a word holds two keys, the lower one in its low half)
        const bool hi8 = b8.at(0) < b;  // at least eight keys below b?
        const uint32_t w0 = hi8 ? b8.w[0] : a8.w[0], w1 = hi8 ? b8.w[1] : a8.w[1];
        const uint32_t w2 = hi8 ? b8.w[2] : a8.w[2], w3 = hi8 ? b8.w[3] : a8.w[3];
        const bool hi4 = (w2 & 0xffffu) < b;  // key 4 of those eight
        const uint32_t v0 = hi4 ? w2 : w0, v1 = hi4 ? w3 : w1;
        const bool hi2 = (v1 & 0xffffu) < b;  // key 2 of those four
        const uint32_t u0 = hi2 ? v1 : v0;
        const bool hi1 = (u0 >> 16) < b;      // key 1 of those two
        const uint32_t last = hi1 ? (u0 >> 16) : (u0 & 0xffffu);
        const int below = (hi8 ? 8 : 0) + (hi4 ? 4 : 0) + (hi2 ? 2 : 0) + (hi1 ? 1 : 0) + (last < b ? 1 : 0);
        if (below == 0 && j0 > 0) hi = j0;                    // the boundary moved below the window
        else if (below == 16 && j0 + 16 < M) lo = j0 + 16;    // ... or above it
        else return j0 + below;                               // (entries past the table are 0xffff: never below)
    }
    while (lo < hi) {
        const int mid = (lo + hi) >> 1;
        if ((uint32_t)keys[mid] < b) lo = mid + 1; else hi = mid;
    }
    return lo;
}

// fp64 sum of count x value over the first r (0..7) of eight entries: independent products, added as a tree.
template <int DT>
__device__ __forceinline__ double partial_sum8(const Eight& k8, const Eight& c8, int r) {
    double t[8];
#pragma unroll
    for (int u = 0; u < 7; ++u) {
        const int cnt = (int)c8.at(u + 1) - (int)c8.at(u);
        const double prod = (double)cnt * (double)value_of_key16<DT>(k8.at(u));
        t[u] = u < r ? prod : 0.0;  // entries past the table may hold anything, NaN patterns included
    }
    return ((t[0] + t[1]) + (t[2] + t[3])) + ((t[4] + t[5]) + t[6]);
}

// fp64 sum of all weights below entry e (0 <= e <= M): the prefix stored for entry 8 (e / 8)
// plus at most seven count x value products.
template <int DT>
__device__ __forceinline__ double prefix_sum_at(const uint16_t* keys, const uint16_t* cum, const double* coarse,
                                                int e) {
    const int j0 = e & ~7;
    const double P = coarse[e >> 3];
    const Eight k8 = load_eight(keys + j0), c8 = load_eight(cum + j0);
    return P + partial_sum8<DT>(k8, c8, e & 7);
}

// Lane gl holds c_gl: is every centroid above its lower neighbour by more than `need`?  (per lane)
__device__ __forceinline__ bool gap_ok(unsigned gmask, int gl, int K, float ck, double need) {
    const float cp = __shfl_up_sync(gmask, ck, 1, kGroup);
    return (gl == 0 || gl >= K) ? true : ((double)ck - (double)cp > need);
}

__device__ __forceinline__ double group_sum(unsigned gmask, double v) {
#pragma unroll
    for (int o = kGroup / 2; o > 0; o >>= 1) v += __shfl_xor_sync(gmask, v, o, kGroup);
    return v;
}
__device__ __forceinline__ int group_sum(unsigned gmask, int v) {
#pragma unroll
    for (int o = kGroup / 2; o > 0; o >>= 1) v += __shfl_xor_sync(gmask, v, o, kGroup);
    return v;
}

// W'' differs from W' only at the removed positions (the entries kept as outliers): the table of a row of
// W'' is the table of the same row of W' with the counts of the removed values moved to the value +0.
// Every table has an entry for +0 and entries may have count 0, so the list of keys does not change: only
// the count prefixes do, and the prefix of an entry with key k becomes
//     cum(k) - #{removed weights with key < k} + (k > key of +0 ? number of removed weights : 0) ,
// which is applied while the table is copied.  Copies keys[0..M) and cum[0..M] (eight entries per lane and
// step), adjusting for the `nr` removed keys in rk.
__device__ __forceinline__ void copy_table_removing(uint16_t* w_keys, uint16_t* w_cum, const uint16_t* g_keys,
                                                    const uint16_t* g_cum, int M, const uint32_t* rk, int nr) {
    const int gl = threadIdx.x & 15;
    const int steps = (M + 1 + 7) / 8;  // with the sentinel (key 0xffff, cum[M] = d_out)
    constexpr int kAhead = 4;           // groups of eight a lane requests before it stores any (the loads are L2 latency)
    for (int i0 = gl; i0 < steps; i0 += kGroup * kAhead) {
        // plain loads: after the first pass over a row the source is the copy itself, which may be shared memory
        uint4 kv[kAhead], cv[kAhead];
#pragma unroll
        for (int q = 0; q < kAhead; ++q) {
            const int i = i0 + q * kGroup;
            if (i < steps) {
                kv[q] = reinterpret_cast<const uint4*>(g_keys)[i];
                cv[q] = reinterpret_cast<const uint4*>(g_cum)[i];
            }
        }
#pragma unroll
        for (int q = 0; q < kAhead; ++q) {
            const int i = i0 + q * kGroup;
            if (i >= steps) continue;
            if (nr > 0) {
                const uint32_t kw[4] = {kv[q].x, kv[q].y, kv[q].z, kv[q].w};
                uint32_t cw[4] = {cv[q].x, cv[q].y, cv[q].z, cv[q].w};
                // Both parts of the shift are monotone in the key, so if the first and the last of the eight
                // ascending keys get the same parts, all eight get the same shift (nearly every group does).
                const uint32_t k_lo = kw[0] & 0xffffu, k_hi = kw[3] >> 16;
                int below_lo = 0, below_hi = 0;
                for (int r = 0; r < nr; ++r) {
                    const uint32_t k = rk[r];
                    below_lo += k < k_lo ? 1 : 0;
                    below_hi += k < k_hi ? 1 : 0;
                }
                // (a group that reaches past the sentinel holds unordered left-overs: entry by entry)
                if (8 * i + 7 <= M && below_lo == below_hi && (k_lo > kZeroKeyOfTable) == (k_hi > kZeroKeyOfTable)) {
                    const uint32_t d = (uint32_t)((k_lo > kZeroKeyOfTable ? nr : 0) - below_lo);
#pragma unroll
                    for (int h = 0; h < 4; ++h)
                        cw[h] = ((cw[h] + d) & 0xffffu) | ((((cw[h] >> 16) + d) & 0xffffu) << 16);
                } else {
#pragma unroll
                    for (int h = 0; h < 4; ++h) {
                        const uint32_t k0 = kw[h] & 0xffffu, k1 = kw[h] >> 16;
                        int d0 = k0 > kZeroKeyOfTable ? nr : 0, d1 = k1 > kZeroKeyOfTable ? nr : 0;
                        for (int r = 0; r < nr; ++r) {
                            const uint32_t k = rk[r];
                            d0 -= k < k0 ? 1 : 0;
                            d1 -= k < k1 ? 1 : 0;
                        }
                        cw[h] = ((cw[h] + (uint32_t)d0) & 0xffffu) | ((((cw[h] >> 16) + (uint32_t)d1) & 0xffffu) << 16);
                    }
                }
                cv[q] = make_uint4(cw[0], cw[1], cw[2], cw[3]);
            }
            reinterpret_cast<uint4*>(w_keys)[i] = kv[q];
            reinterpret_cast<uint4*>(w_cum)[i] = cv[q];
        }
    }
}

// The exactness test of the table kernel (see load_channel_keys) on a finished table.
template <int DT>
__device__ void count_if_inexact(const uint16_t* keys, const uint16_t* cum, int M, int N, int32_t* inexact_rows) {
    const unsigned gmask = group_mask();
    const int gl = threadIdx.x & 15;
    uint32_t amax = 0u;
    int q = 100000;
    for (int i = gl; i < M; i += kGroup) {
        const uint32_t ub = __float_as_uint(value_of_key16<DT>(keys[i])) & 0x7fffffffu;
        if (ub && cum[i + 1] != cum[i]) {  // values that still occur
            amax = max(amax, ub);
            const int ex = (int)(ub >> 23);
            const uint32_t m = ub & 0x7fffffu;
            q = min(q, ex ? ex - 150 + (__ffs(m | 0x800000u) - 1) : (__ffs(m) - 1) - 149);
        }
    }
#pragma unroll
    for (int o = kGroup / 2; o > 0; o >>= 1) {
        amax = max(amax, __shfl_xor_sync(gmask, amax, o, kGroup));
        q = min(q, __shfl_xor_sync(gmask, q, o, kGroup));
    }
    if (gl == 0 && amax != 0u) {
        const int log2n = 32 - __clz(N - 1 > 0 ? N - 1 : 1);
        const int ex_max = (int)(amax >> 23);
        const int top = ex_max ? ex_max - 127 : (31 - __clz(amax)) - 149;
        if (log2n + 1 + (top + 1 - q) > 53) atomicAdd(inexact_rows, 1);
    }
}

// K = 2^bits of the channel is a run-time value on purpose: the two channels of a warp may differ in
// width and still share one instruction stream (lanes >= K of a group idle).
template <int DT>
__device__ void iterate_channel(const IterArgs& a, int64_t row, const int K, unsigned char* smem) {
    const unsigned gmask = group_mask();
    const int gl = threadIdx.x & 15;
    const int N = (int)a.d_out, T = a.iters;
    double* s_coarse = reinterpret_cast<double*>(smem);
    uint16_t* s_keys = reinterpret_cast<uint16_t*>(s_coarse + a.cap / 8 + 2);
    uint16_t* s_cum = s_keys + a.cap + kKeyPad;
    uint32_t* s_removed = reinterpret_cast<uint32_t*>(s_coarse);  // keys of removed weights: used before the sums exist
    const bool patch = a.src.hdr != nullptr;
    const Tables& from = patch ? a.src : a.t;
    int64_t p0 = 0, nrem = 0;
    const ChannelHeader h = from.hdr[row];  // requested together with the row's list limits
    if (patch) { p0 = a.row_ptr[row]; nrem = a.row_ptr[row + 1] - p0; }
    int M = 1;
    const uint16_t* keys = s_keys;
    const uint16_t* cum = s_cum;
    double* coarse = s_coarse;
    bool staged = true;
    if (patch && nrem >= N) {  // every position removed: an all-zero channel
        if (gl == 0) { s_keys[0] = (uint16_t)kZeroKeyOfTable; s_cum[0] = 0; s_cum[1] = (uint16_t)N; }
    } else {
        M = h.M < 1 ? 1 : (h.M > N + 1 ? N + 1 : h.M);  // 1 <= M <= N + 1 by construction (the entry of +0 may be empty)
        const uint16_t* g_keys = from.keys + row * from.stride;  // rows are 16-byte aligned, padded to 8 entries
        const uint16_t* g_cum = from.cum + row * from.stride;
        staged = M <= a.cap;
        uint16_t* w_keys = staged ? s_keys : a.t.keys + row * a.t.stride;
        uint16_t* w_cum = staged ? s_cum : a.t.cum + row * a.t.stride;
        if (staged || patch) {  // copy: into shared memory, or into this launch's own table when patching
            int done = 0;
            do {  // removed weights are taken kPatchChunk at a time (one pass in all but pathological rows)
                const int nr = (int)(nrem - done < kPatchChunk ? nrem - done : kPatchChunk);
                for (int i = gl; i < nr; i += kGroup) {
                    uint32_t hh = a.W[row * a.ldw + a.cols[p0 + done + i]];
                    if (hh == 0x8000u) hh = 0u;  // -0 and +0 are the same point
                    s_removed[i] = (hh & 0x8000u) ? (~hh & 0xffffu) : (hh | 0x8000u);
                }
                __syncwarp(gmask);
                copy_table_removing(w_keys, w_cum, done == 0 ? g_keys : w_keys, done == 0 ? g_cum : w_cum, M, s_removed, nr);
                __syncwarp(gmask);
                done += nr;
            } while (done < nrem);
            if (patch && a.inexact_rows && h.suspect) count_if_inexact<DT>(w_keys, w_cum, M, N, a.inexact_rows);
            keys = w_keys;
            cum = w_cum;
        } else {
            keys = g_keys;
            cum = g_cum;
        }
        if (!staged) coarse = a.t.sum + row * a.t.sum_stride;  // global scratch for tables too large to stage
    }
    __syncwarp(gmask);
    if (staged)  // nothing past the table
        for (int i = M + gl; i < ((M + 7) & ~7) + kKeyPad; i += kGroup) s_keys[i] = 0xffffu;
    __syncwarp(gmask);
    // prefix sums at every eighth entry: each lane owns a contiguous range of groups of eight entries,
    // sums each group (independent products), the lane totals are scanned, every group receives its base
    {
        const int groups = (M >> 3) + 1;  // coarse[g] for g = 0 .. M / 8
        const int per_lane = (groups + kGroup - 1) / kGroup;
        const int g_begin = gl * per_lane;
        double local = 0.0;
        for (int g = g_begin; g < g_begin + per_lane && g < groups; ++g) {
            const Eight k8 = load_eight(keys + g * 8), c8 = load_eight(cum + g * 8);
            const int left = M - g * 8;  // entries of this group that exist (may exceed 8)
            double s7 = partial_sum8<DT>(k8, c8, left < 7 ? left : 7);
            if (left >= 8) s7 += (double)((int)cum[g * 8 + 8] - (int)c8.at(7)) * (double)value_of_key16<DT>(k8.at(7));
            coarse[g] = local;
            local += s7;
        }
        double incl = local;
#pragma unroll
        for (int o = 1; o < kGroup; o <<= 1) {
            const double up = __shfl_up_sync(gmask, incl, o, kGroup);
            if (gl >= o) incl += up;
        }
        double base = __shfl_up_sync(gmask, incl, 1, kGroup);
        if (gl == 0) base = 0.0;
        for (int g = g_begin; g < g_begin + per_lane && g < groups; ++g) coarse[g] += base;
        __threadfence_block();  // the sums may live in global memory: make them visible to the other lanes
        __syncwarp(gmask);
    }
    const uint32_t kfirst = keys[0], kend = (uint32_t)keys[M - 1] + 1u;
    // range * 2^-22, the range being last minus first value of the table
    const double need = ((double)value_of_key16<DT>(kend - 1u) - (double)value_of_key16<DT>(kfirst)) * (1.0 / 4194304.0);
    const double p_total = prefix_sum_at<DT>(keys, cum, coarse, M);  // sum of all weights of the channel

    // start: K evenly spaced order statistics; the weight at sorted position pos has the value of the
    // entry e with cum[e] <= pos < cum[e + 1]
    float ck = 0.f;
    if (gl < K) {
        const int pos = (int)(((long long)(2 * gl + 1) * N) / (2 * K));
        int lo = 0, hi = M;  // cum[lo] <= pos < cum[hi]   (cum[0] = 0, cum[M] = N)
        while (hi - lo > 1) {
            const int mid = (lo + hi) >> 1;
            if ((int)cum[mid] <= pos) lo = mid; else hi = mid;
        }
        ck = value_of_key16<DT>(keys[lo]);
    }
    __syncwarp(gmask);

    // the boundary formulation needs strictly increasing centroids with gaps above `need`
    bool ordered = __all_sync(gmask, gap_ok(gmask, gl, K, ck, need)) != 0;
    int updates = 0;
    int e_hint = -1;       // this lane's boundary of the previous ordered iteration (staged tables)
    uint32_t b_last = 0;   // ... and its key
    while (updates < T) {
        float cn = ck;
        if (ordered) {
            const float cm = __shfl_up_sync(gmask, ck, 1, kGroup);  // c_{k-1}
            int e = 0;  // first table entry of this lane's cluster
            if (gl > 0 && gl < K) {
                b_last = boundary_key<DT>(cm, ck, kfirst, kend);
                e = b_last >= kend ? M : rank_of_key(keys, M, b_last, staged ? e_hint : -1);
                e_hint = e;
            }
            int B = 0;
            double P = 0.0;
            if (gl < K) { B = (int)cum[e]; P = prefix_sum_at<DT>(keys, cum, coarse, e); }
            int Bn = __shfl_down_sync(gmask, B, 1, kGroup);
            double Pn = __shfl_down_sync(gmask, P, 1, kGroup);
            if (gl == K - 1) { Bn = N; Pn = p_total; }  // the last cluster ends with the table
            if (gl < K) {
                const int cnt = Bn - B;
                if (cnt > 0) cn = __double2float_rn(__ddiv_rn(Pn - P, (double)cnt));
            }
        } else {
            e_hint = -1;
            // plain rule on every distinct value; cluster sums as count x value in fp64
            float c[kMaxK];
#pragma unroll
            for (int k = 0; k < kMaxK; ++k) c[k] = __shfl_sync(gmask, ck, k, kGroup);
            double s[kMaxK];
            int n[kMaxK];
#pragma unroll
            for (int k = 0; k < kMaxK; ++k) { s[k] = 0.0; n[k] = 0; }
            for (int j = gl; j < M; j += kGroup) {
                const float v = value_of_key16<DT>(keys[j]);
                const int cnt = (int)cum[j + 1] - (int)cum[j];
                float best = fabsf(v - c[0]);
                int code = 0;  // first k < K minimising |v - c_k|
#pragma unroll
                for (int k = 1; k < kMaxK; ++k) {
                    const float d = fabsf(v - c[k]);
                    if (k < K && d < best) { best = d; code = k; }
                }
                const double prod = (double)cnt * (double)v;
#pragma unroll
                for (int k = 0; k < kMaxK; ++k)
                    if (code == k) { s[k] += prod; n[k] += cnt; }
            }
#pragma unroll
            for (int k = 0; k < kMaxK; ++k) {
                if (k < K) {  // K is the same in every lane of the group
                    const double sk = group_sum(gmask, s[k]);
                    const int nk = group_sum(gmask, n[k]);
                    if (gl == k && nk > 0) cn = __double2float_rn(__ddiv_rn(sk, (double)nk));
                }
            }
        }
        ++updates;
        // one round of votes answers both questions about the new centroids
        const bool ok = gap_ok(gmask, gl, K, cn, need);
        const bool same_here = gl >= K || __float_as_uint(cn) == __float_as_uint(ck);
        const unsigned full = gmask;
        const bool same = __ballot_sync(gmask, same_here) == full;
        const bool was_ordered = ordered;
        ordered = __ballot_sync(gmask, ok) == full;
        ck = cn;
        if (same) {  // identical centroids: every later iteration repeats this one
            if (!was_ordered) e_hint = -1;
            break;
        }
    }
    a.lut[row * CMPQ_LUT_STRIDE + gl] = gl < K ? ck : 0.f;
    // Last assignment: when the final centroids pass the test, a weight's code is the number of k >= 1
    // whose boundary value it reaches, so the assign kernel only compares with K-1 thresholds.
    {
        const float cm = __shfl_up_sync(gmask, ck, 1, kGroup);
        float thr = ordered ? 1.f : 0.f;
        uint32_t b = kfirst;
        if (ordered && gl > 0 && gl < K) {
            b = boundary_key<DT>(cm, ck, kfirst, kend);
            thr = b < kend ? value_of_key16<DT>(b) : __int_as_float(0x7f800000);
        }
        a.t.thr[row * CMPQ_LUT_STRIDE + gl] = gl < K ? thr : 0.f;
        // For the selection of the worst-fitted entries: cluster k is the run [first, next first) of the table;
        // on each side of c_k the error grows towards the end of the run, so the largest error of a side sits
        // at its outer end.  Those maxima (of entries that hold at least one weight) go into the histogram.
        if (a.side_hist && ordered) {
            int first = 0, mid = 0;
            if (gl < K) {
                if (gl > 0) first = b < kend ? rank_of_key(keys, M, b, staged ? e_hint : -1) : M;
                const uint32_t kc = key_ceil<DT>(ck);  // the first storage value not below c_k
                mid = kc >= kend ? M : (kc <= kfirst ? 0 : rank_of_key(keys, M, kc, staged ? first : -1));
            }
            int next = __shfl_down_sync(gmask, first, 1, kGroup);
            if (gl == K - 1) next = M;
            if (gl < K) {
                mid = mid < first ? first : (mid > next ? next : mid);
                uint16_t* bnd = a.t.bnd + row * 32;
                bnd[2 * gl] = (uint16_t)first;
                bnd[2 * gl + 1] = (uint16_t)mid;
                int j = first;  // left side: [first, mid), largest error at its first entry that is not empty
                if (j < mid && cum[j + 1] == cum[j]) ++j;
                if (j < mid) atomicAdd(&a.side_hist[__float_as_uint(fabsf(value_of_key16<DT>(keys[j]) - ck)) >> 20], 1u);
                j = next - 1;   // right side: [mid, next), largest error at its last entry that is not empty
                if (j >= mid && cum[j + 1] == cum[j]) --j;
                if (j >= mid) atomicAdd(&a.side_hist[__float_as_uint(fabsf(value_of_key16<DT>(keys[j]) - ck)) >> 20], 1u);
            }
        }
    }
    // assignments made: one per update, and the last one by the assign kernel
    if (a.sweeps && gl == 0)
        atomicAdd(a.sweeps, (unsigned long long)(updates + 1) * (unsigned long long)N * (unsigned long long)K);
}

template <int DT>
__global__ void __launch_bounds__(kIterWarps * 32)
lloyd_iterate_kernel(const IterArgs a) {
    extern __shared__ __align__(16) unsigned char iter_smem[];
    const int group = threadIdx.x >> 4;  // channel of the block
    unsigned char* smem = iter_smem + (size_t)group * iter_channel_bytes(a.cap);
    const int64_t row = (int64_t)blockIdx.x * (kIterWarps * 2) + group;
    if (row >= a.d_in) return;
    // the per-row words are all requested before any of them is looked at (each is a round trip to L2)
    const int skip = a.skip_row ? (int)a.skip_row[row] : 0;
    const int bad = a.nonfinite ? *a.nonfinite : 0;
    const int bits = a.bits[row];
    const int cache_iters = a.fc.hdr ? a.fc.hdr->iters : -1;
    if (skip) return;
    // Non-finite inputs were found by an earlier kernel of the call: its outputs are unspecified anyway, and
    // although every loop below is bounded whatever the values (bisections halve an interval, the update
    // loop counts to the iteration limit), there is nothing worth computing.
    if (bad) return;
    const unsigned gmask = group_mask();
    const int gl = threadIdx.x & 15;
    // a fit of this channel at this width kept from an earlier call on the same weights: copy it
    const bool cached_ok = a.fc.hdr && cache_iters == a.iters;
    const int64_t slot = (int64_t)(bits == 2 ? 0 : (bits == 3 ? 1 : 2)) * a.d_in + row;
    if (cached_ok && a.fc.valid[slot]) {
        const float ck = a.fc.lut[slot * CMPQ_LUT_STRIDE + gl];
        const float thr0 = a.fc.thr[slot * CMPQ_LUT_STRIDE];
        const uint32_t limits = reinterpret_cast<const uint32_t*>(a.fc.bnd + slot * 32)[gl];  // first | mid << 16
        a.lut[row * CMPQ_LUT_STRIDE + gl] = ck;
        a.t.thr[row * CMPQ_LUT_STRIDE + gl] = a.fc.thr[slot * CMPQ_LUT_STRIDE + gl];
        reinterpret_cast<uint32_t*>(a.t.bnd + row * 32)[gl] = limits;
        // the selection's lower bound counts the largest error of every cluster side (see iterate_channel):
        // a copied fit contributes them too, read off the table at the copied cluster limits
        if (a.side_hist && thr0 != 0.f) {
            const int K = bits == 2 ? 4 : (bits == 3 ? 8 : 16);
            const int M = a.t.hdr[row].M;
            const int first = (int)(limits & 0xffffu), mid = (int)(limits >> 16);
            int next = (int)(__shfl_down_sync(gmask, limits, 1, kGroup) & 0xffffu);
            if (gl == K - 1) next = M;
            if (gl < K) {
                const uint16_t* keys = a.t.keys + row * a.t.stride;
                const uint16_t* cum = a.t.cum + row * a.t.stride;
                int j = first;
                if (j < mid && cum[j + 1] == cum[j]) ++j;
                if (j < mid) atomicAdd(&a.side_hist[__float_as_uint(fabsf(value_of_key16<DT>(keys[j]) - ck)) >> 20], 1u);
                j = next - 1;
                if (j >= mid && cum[j + 1] == cum[j]) --j;
                if (j >= mid) atomicAdd(&a.side_hist[__float_as_uint(fabsf(value_of_key16<DT>(keys[j]) - ck)) >> 20], 1u);
            }
        }
        return;
    }
    iterate_channel<DT>(a, row, bits == 2 ? 4 : (bits == 3 ? 8 : 16), smem);
    if (cached_ok) {  // lane l wrote entry l of both rows above and reads its own writes back
        a.fc.lut[slot * CMPQ_LUT_STRIDE + gl] = a.lut[row * CMPQ_LUT_STRIDE + gl];
        a.fc.thr[slot * CMPQ_LUT_STRIDE + gl] = a.t.thr[row * CMPQ_LUT_STRIDE + gl];
        __syncwarp(gmask);  // lanes below K wrote the cluster limits (two 16-bit values each) just before
        reinterpret_cast<uint32_t*>(a.fc.bnd + slot * 32)[gl] = reinterpret_cast<const uint32_t*>(a.t.bnd + row * 32)[gl];
        __syncwarp(gmask);
        if (gl == 0) {
            __threadfence();
            a.fc.valid[slot] = 1;
        }
    }
}

// ------------------------------------------------------------------------------------------------
// sensitivity-weighted fit on the value tables
//
// With sensitivities the update is the weighted mean  c_k = sum s x / sum s  over a cluster's members.
// Members with the same value contribute  value * (sum of their s), so the table of a channel carries the
// weighted fit as well once every entry knows the sum S of its members' sensitivities: cluster sums are again
// differences of prefix sums over the ascending entries, and the boundaries are found exactly as in the
// unweighted iterations.  S is accumulated in 64-bit fixed point (scale: a power of two chosen from the
// channel's largest sensitivity so that the total stays below 2^52), which makes the sums independent of the
// order in which the threads add them: the same inputs give the same bytes.  A sensitivity smaller than
// 2^-(52 - log2 d_out) of the channel's largest loses its low bits; nothing else is rounded before the fp64
// prefix sums.
//
// One block per channel: table and prefix sums in shared memory, the block accumulates S (one search in the
// table per weight), then a half-warp iterates.  The kernel is launched twice: with a capacity that fits the
// tables of nearly all channels and lets several blocks share an SM, then, for the channels that exceeded it,
// with the largest capacity shared memory allows.  Channels beyond that are left to the kernel that scans
// every weight (flags tell which).
constexpr int kWtThreads = 128;

__host__ __device__ inline size_t weighted_table_smem(int cap, int64_t d_out) {
    return (size_t)(cap + 1) * 16 + (size_t)(cap + kKeyPad + 8) * 2 + (size_t)(cap + 8) * 2 + ((size_t)d_out + 31) / 32 * 4 + 16;
}

template <int DT>
__global__ void __launch_bounds__(kWtThreads, 8)
lloyd_weighted_table_kernel(const LloydArgs a, const Tables t, const float* __restrict__ sens, int cap, int second_try,
                            uint8_t* fitted, uint8_t* not_fitted) {
    extern __shared__ __align__(16) unsigned char wt_smem[];
    __shared__ unsigned long long warp_s[kWtThreads / 32];
    __shared__ double warp_sx[kWtThreads / 32];
    __shared__ uint32_t warp_max[kWtThreads / 32];
    double* s_ps = reinterpret_cast<double*>(wt_smem);  // [cap + 1] fixed-point sums first, then their prefix
    double* s_psx = s_ps + cap + 1;                     // [cap + 1] prefix of value * S
    uint16_t* s_keys = reinterpret_cast<uint16_t*>(s_psx + cap + 1);  // [cap + kKeyPad + 8]
    uint16_t* s_cum = s_keys + cap + kKeyPad + 8;                     // [cap + 8]
    uint32_t* bitmap = reinterpret_cast<uint32_t*>(s_cum + cap + 8);  // removed columns of the row
    unsigned long long* s_fix = reinterpret_cast<unsigned long long*>(s_ps);
    const int64_t row = blockIdx.x;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int N = (int)a.d_out, T = a.iters;
    if (second_try && fitted[row]) return;  // the launch with the small capacity did this channel
    const ChannelHeader h = t.hdr[row];
    const int M = h.M < 1 ? 1 : (h.M > N + 1 ? N + 1 : h.M);
    if (M > cap) {
        if (tid == 0) { fitted[row] = 0; not_fitted[row] = 1; }
        return;
    }
    const uint16_t* g_keys = t.keys + row * t.stride;
    const uint16_t* g_cum = t.cum + row * t.stride;
    for (int i = tid; i <= M; i += kWtThreads) { s_keys[i] = g_keys[i]; s_cum[i] = g_cum[i]; s_fix[i] = 0ull; }
    for (int i = M + 1 + tid; i < ((M + 8) & ~7) + kKeyPad; i += kWtThreads) s_keys[i] = 0xffffu;
    int64_t p0 = 0, p1 = 0;
    if (a.row_ptr) { p0 = a.row_ptr[row]; p1 = a.row_ptr[row + 1]; }
    if (p1 > p0) for (int i = tid; i < (N + 31) / 32; i += kWtThreads) bitmap[i] = 0u;
    // largest sensitivity of the channel (s >= 0: the bit patterns order like the values)
    const float* s_row = sens + row * a.d_out;
    uint32_t smax = 0u;
    for (int j = tid; j < N; j += kWtThreads) smax = max(smax, __float_as_uint(s_row[j]));
    smax = __reduce_max_sync(0xffffffffu, smax);
    if (lane == 0) warp_max[warp] = smax;
    __syncthreads();
    if (p1 > p0)
        for (int64_t p = p0 + tid; p < p1; p += kWtThreads) {
            const int col = a.cols[p];
            atomicOr(&bitmap[col >> 5], 1u << (col & 31));
        }
    smax = __reduce_max_sync(0xffffffffu, lane < kWtThreads / 32 ? warp_max[lane] : 0u);
    double scale = 0.0;  // all sensitivities zero: every sum stays zero and the centroids stay at the start
    if (smax != 0u) {
        int ex;
        frexpf(__uint_as_float(smax), &ex);  // largest sensitivity < 2^ex
        const int log2n = 32 - __clz(N - 1 > 0 ? N - 1 : 1);
        scale = ldexp(1.0, 52 - ex - log2n);
    }
    __syncthreads();
    // S of every entry: the entry of a weight is found by bisection (its key is in the table).  The number of
    // steps depends on the table alone, so four searches run side by side.
    const uint16_t* w = a.W + row * a.ldw;
    constexpr int kSide = 4;
    for (int j0 = tid; j0 < N; j0 += kWtThreads * kSide) {
        uint32_t key[kSide];
        int base[kSide];
#pragma unroll
        for (int u = 0; u < kSide; ++u) {
            const int j = j0 + u * kWtThreads;
            uint32_t hh = j < N ? w[j] : 0u;
            if (j < N && p1 > p0 && ((bitmap[j >> 5] >> (j & 31)) & 1u)) hh = 0u;
            if (hh == 0x8000u) hh = 0u;  // -0 and +0 are the same point
            key[u] = (hh & 0x8000u) ? (~hh & 0xffffu) : (hh | 0x8000u);
            base[u] = 0;
        }
        for (int n = M; n > 1;) {  // first entry whose key is not below the weight's
            const int half = n >> 1;
#pragma unroll
            for (int u = 0; u < kSide; ++u) base[u] = (uint32_t)s_keys[base[u] + half - 1] < key[u] ? base[u] + half : base[u];
            n -= half;
        }
#pragma unroll
        for (int u = 0; u < kSide; ++u) {
            const int j = j0 + u * kWtThreads;
            if (j < N) {
                const unsigned long long fx = __double2ull_rn((double)s_row[j] * scale);
                if (fx) atomicAdd(&s_fix[base[u]], fx);
            }
        }
    }
    __syncthreads();
    // prefix sums over the entries, every thread a contiguous range, always in the same order
    {
        const int chunk = (M + kWtThreads - 1) / kWtThreads;
        const int e0 = min(tid * chunk, M), e1 = min(e0 + chunk, M);
        unsigned long long ls = 0ull;
        double lsx = 0.0;
        for (int e = e0; e < e1; ++e) {
            const unsigned long long S = s_fix[e];
            ls += S;
            lsx += (double)S * (double)value_of_key16<DT>(s_keys[e]);
        }
        unsigned long long is = ls;
        double isx = lsx;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const unsigned long long us = __shfl_up_sync(0xffffffffu, is, o);
            const double ux = __shfl_up_sync(0xffffffffu, isx, o);
            if (lane >= o) { is += us; isx += ux; }
        }
        if (lane == 31) { warp_s[warp] = is; warp_sx[warp] = isx; }
        __syncthreads();
        unsigned long long run_s = is - ls;
        double run_sx = 0.0, tot_sx = 0.0;
        unsigned long long tot_s = 0ull;
        for (int wv = 0; wv < kWtThreads / 32; ++wv) {  // the warps in order
            if (wv < warp) { run_s += warp_s[wv]; run_sx += warp_sx[wv]; }
            tot_s += warp_s[wv];
            tot_sx += warp_sx[wv];
        }
        run_sx += isx - lsx;
        for (int e = e0; e < e1; ++e) {
            const unsigned long long S = s_fix[e];
            s_ps[e] = (double)run_s;  // below 2^52: exact
            s_psx[e] = run_sx;
            run_s += S;
            run_sx += (double)S * (double)value_of_key16<DT>(s_keys[e]);
        }
        __syncthreads();  // every range is written before the totals replace the sentinel's slot
        if (tid == 0) { s_ps[M] = (double)tot_s; s_psx[M] = tot_sx; }
    }
    __syncthreads();
    if (tid >= kGroup) return;

    // iterations: lane k of the half-warp owns centroid k (as in iterate_channel, sums from the prefixes above)
    const unsigned gmask = 0xffffu;
    const int gl = tid;
    const int width = a.bits[row];
    const int K = width == 2 ? 4 : (width == 3 ? 8 : 16);
    const uint32_t kfirst = s_keys[0], kend = (uint32_t)s_keys[M - 1] + 1u;
    const double need = ((double)value_of_key16<DT>(kend - 1u) - (double)value_of_key16<DT>(kfirst)) * (1.0 / 4194304.0);
    float ck = 0.f;
    if (gl < K) {
        const int pos = (int)(((long long)(2 * gl + 1) * N) / (2 * K));
        int lo = 0, hi = M;  // cum[lo] <= pos < cum[hi]
        while (hi - lo > 1) {
            const int mid = (lo + hi) >> 1;
            if ((int)s_cum[mid] <= pos) lo = mid; else hi = mid;
        }
        ck = value_of_key16<DT>(s_keys[lo]);
    }
    bool ordered = __all_sync(gmask, gap_ok(gmask, gl, K, ck, need)) != 0;
    int updates = 0, e_hint = -1;
    while (updates < T) {
        float cn = ck;
        if (ordered) {
            const float cm = __shfl_up_sync(gmask, ck, 1, kGroup);
            int e = 0;
            if (gl > 0 && gl < K) {
                const uint32_t b = boundary_key<DT>(cm, ck, kfirst, kend);
                e = b >= kend ? M : rank_of_key(s_keys, M, b, e_hint);
                e_hint = e;
            }
            double P = 0.0, Q = 0.0;
            if (gl < K) { P = s_ps[e]; Q = s_psx[e]; }
            double Pn = __shfl_down_sync(gmask, P, 1, kGroup);
            double Qn = __shfl_down_sync(gmask, Q, 1, kGroup);
            if (gl == K - 1) { Pn = s_ps[M]; Qn = s_psx[M]; }
            if (gl < K && Pn - P > 0.0) cn = __double2float_rn(__ddiv_rn(Qn - Q, Pn - P));
        } else {
            e_hint = -1;
            float c[kMaxK];
#pragma unroll
            for (int k = 0; k < kMaxK; ++k) c[k] = __shfl_sync(gmask, ck, k, kGroup);
            double s[kMaxK], n[kMaxK];
#pragma unroll
            for (int k = 0; k < kMaxK; ++k) { s[k] = 0.0; n[k] = 0.0; }
            for (int j = gl; j < M; j += kGroup) {
                const float v = value_of_key16<DT>(s_keys[j]);
                const double S = s_ps[j + 1] - s_ps[j];  // integers below 2^52: exact
                float best = fabsf(v - c[0]);
                int code = 0;
#pragma unroll
                for (int k = 1; k < kMaxK; ++k) {
                    const float d = fabsf(v - c[k]);
                    if (k < K && d < best) { best = d; code = k; }
                }
#pragma unroll
                for (int k = 0; k < kMaxK; ++k)
                    if (code == k) { s[k] += S * (double)v; n[k] += S; }
            }
#pragma unroll
            for (int k = 0; k < kMaxK; ++k) {
                if (k < K) {
                    const double sk = group_sum(gmask, s[k]);
                    const double nk = group_sum(gmask, n[k]);
                    if (gl == k && nk > 0.0) cn = __double2float_rn(__ddiv_rn(sk, nk));
                }
            }
        }
        ++updates;
        const bool ok = gap_ok(gmask, gl, K, cn, need);
        const bool same_here = gl >= K || __float_as_uint(cn) == __float_as_uint(ck);
        const bool same = __ballot_sync(gmask, same_here) == gmask;
        const bool was_ordered = ordered;
        ordered = __ballot_sync(gmask, ok) == gmask;
        ck = cn;
        if (same) {
            if (!was_ordered) e_hint = -1;
            break;
        }
    }
    a.lut[row * CMPQ_LUT_STRIDE + gl] = gl < K ? ck : 0.f;
    {
        const float cm = __shfl_up_sync(gmask, ck, 1, kGroup);
        float thr = ordered ? 1.f : 0.f;
        if (ordered && gl > 0 && gl < K) {
            const uint32_t b = boundary_key<DT>(cm, ck, kfirst, kend);
            thr = b < kend ? value_of_key16<DT>(b) : __int_as_float(0x7f800000);
        }
        t.thr[row * CMPQ_LUT_STRIDE + gl] = gl < K ? thr : 0.f;
    }
    if (gl == 0) {
        fitted[row] = 1;
        not_fitted[row] = 0;
        if (a.sweeps) atomicAdd(a.sweeps, (unsigned long long)(updates + 1) * (unsigned long long)N * (unsigned long long)K);
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
    for (int k = 0; k < K; ++k) t[k] = __ldg(thr + row * CMPQ_LUT_STRIDE + k);
    const bool by_threshold = t[0] != 0.f;
    if (ERR || !by_threshold) {  // codes by thresholds never look at the centroids
#pragma unroll
        for (int k = 0; k < K; ++k) c[k] = __ldg(lut + row * CMPQ_LUT_STRIDE + k);
    } else {
#pragma unroll
        for (int k = 0; k < K; ++k) c[k] = 0.f;
    }
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
                if (mask) {  // rare: removed positions become +0
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        if ((mask >> (2 * q)) & 1u) pk[q] &= 0xffff0000u;
                        if ((mask >> (2 * q + 1)) & 1u) pk[q] &= 0x0000ffffu;
                    }
                }
                uint32_t r[4];
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const uint32_t x2 = pk[q];
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
constexpr int kKeptCap = 31;                  // values of a row listed for the emit step
constexpr uint32_t kKeptUnknown = 0xffffffffu;

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

// A row fitted with valid thresholds: lane 2k takes the left side of cluster k (entries below c_k), lane
// 2k + 1 the right side.  Towards the centroid the error |v - c_k| (fp32, the rounding is monotone) never
// grows, so the entries of a side with error >= lo are the ones at its outer end.  A lane reads its side
// eight table entries at a time (two 128-bit loads), starting at the outer end, and stops after the first
// group that holds a smaller error: visit(error pattern, count, key) sees exactly the non-empty entries of
// the row with error >= lo, each once.
template <int DT, class Visit>
__device__ __forceinline__ void walk_row_sides(const Tables& t, int64_t row, int K, uint32_t lo, Visit&& visit) {
    const int lane = threadIdx.x & 31;
    if (lane >= 2 * K) return;
    const int k = lane >> 1;
    const bool left = (lane & 1) == 0;
    const uint16_t* bnd = t.bnd + row * 32;
    const int M = t.hdr[row].M;
    const int first = bnd[2 * k], mid = bnd[2 * k + 1], next = k + 1 < K ? (int)bnd[2 * k + 2] : M;
    const int j_lo = left ? first : mid, j_hi = left ? mid : next;  // the side: entries [j_lo, j_hi)
    if (j_lo >= j_hi) return;
    const float c = t.lut[row * CMPQ_LUT_STRIDE + k];
    const uint16_t* keys = t.keys + row * t.stride;
    const uint16_t* cum = t.cum + row * t.stride;
    int g = (left ? j_lo : j_hi - 1) & ~7;
    for (;;) {
        const Eight k8 = load_eight(keys + g), c8 = load_eight(cum + g);
        const uint32_t c_end = g + 8 <= M ? cum[g + 8] : 0u;
        bool below = false;  // an entry of the side with error < lo: everything further in is smaller still
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const uint32_t cnt = (u < 7 ? c8.at(u + 1) : c_end) - c8.at(u);
            if (g + u >= j_lo && g + u < j_hi && cnt != 0u) {
                const uint32_t e = __float_as_uint(fabsf(value_of_key16<DT>(k8.at(u)) - c));
                if (e >= lo) visit(e, cnt, k8.at(u));
                else below = true;
            }
        }
        if (below) break;
        g += left ? 8 : -8;
        if (left ? g >= j_hi : g + 8 <= j_lo) break;
    }
}

// hist[d] += number of weights in non-act rows whose error has the fixed bits of the prefix and the
// digit d at `shift`.  One warp per row, block-local histogram first.  Errors below st->lower (a bound
// known not to exceed the threshold sought) are left out wherever the row's fit allows the walk above.
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
    const uint32_t lo = st->lower > prefix ? st->lower : prefix;  // a matching error is at least the prefix
    const int warp = threadIdx.x >> 5;
    for (int64_t row = (int64_t)blockIdx.x * kTableSelWarps + warp; row < d_in; row += (int64_t)gridDim.x * kTableSelWarps) {
        if (is_act[row]) continue;
        const int b = bits[row];
        if (t.thr[row * CMPQ_LUT_STRIDE] != 0.f) {
            walk_row_sides<DT>(t, row, 1 << b, lo, [&](uint32_t e, uint32_t cnt, uint32_t) {
                if ((e & mask) == prefix) atomicAdd(&local[(e >> shift) & (bins - 1)], cnt);
            });
        } else if (b == 2) table_hist_row<DT, 4>(t, row, prefix, mask, shift, bins, local);
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

// The histogram holds, by the top 12 bits of the error pattern, the largest error of every cluster side of
// every fitted row: distinct entries that each stand for at least one weight.  If n_q or more of them lie in
// bin d or above, so do n_q or more errors of the layer: the n_q-th largest error is at least the lower edge
// of the bin in which the n_q-th largest of the maxima lies.  Clears the histogram for the select passes.
__global__ void __launch_bounds__(1024)
select_lower_kernel(unsigned int* hist, SelectState* st) {
    __shared__ int warp_totals[32];
    __shared__ uint32_t found;
    constexpr int per = kSelBins / 1024;  // bins per thread, descending
    const long long want = st->remaining;
    int v[per], sum = 0;
#pragma unroll
    for (int u = 0; u < per; ++u) {
        v[u] = (int)hist[kSelBins - 1 - (threadIdx.x * per + u)];
        sum += v[u];
    }
    if (threadIdx.x == 0) found = 0u;
    int total;
    long long above = block_exclusive_scan(sum, warp_totals, total);  // maxima in higher bins (publishes `found`)
    if (want > 0 && above < want && want <= above + sum) {  // at most one thread
#pragma unroll
        for (int u = 0; u < per; ++u) {
            if (above < want && want <= above + v[u]) found = (uint32_t)(kSelBins - 1 - (threadIdx.x * per + u)) << 20;
            above += v[u];
        }
    }
    __syncthreads();
    if (threadIdx.x == 0) st->lower = found;
#pragma unroll
    for (int u = 0; u < per; ++u) hist[threadIdx.x * per + u] = 0u;
}

cmpq_status launch_select_lower(void* state, unsigned int* hist, cudaStream_t st) {
    select_lower_kernel<<<1, 1024, 0, st>>>(hist, static_cast<SelectState*>(state));
    return launch_status();
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
        uint32_t* kept = t.kept + row * 32;
        if (t.thr[row * CMPQ_LUT_STRIDE] != 0.f) {
            int mine = 0;  // values this lane's walk finds at or above the threshold
            walk_row_sides<DT>(t, row, 1 << b, tau, [&](uint32_t e, uint32_t cnt, uint32_t) {
                g += e > tau ? (int)cnt : 0;
                q += e == tau ? (int)cnt : 0;
                ++mine;
            });
            // the emit step only needs to know WHICH values keep entries: list them (second, identical walk)
            const int lane = threadIdx.x & 31;
            int incl = mine;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int up = __shfl_up_sync(0xffffffffu, incl, o);
                if (lane >= o) incl += up;
            }
            const int total = __shfl_sync(0xffffffffu, incl, 31);
            if (total <= kKeptCap) {
                int at = 1 + incl - mine;
                walk_row_sides<DT>(t, row, 1 << b, tau, [&](uint32_t e, uint32_t, uint32_t key) {
                    kept[at++] = key | (e == tau ? 0x10000u : 0u);
                });
            }
            if (lane == 0) kept[0] = total <= kKeptCap ? (uint32_t)total : kKeptUnknown;
        } else {
            if ((threadIdx.x & 31) == 0) kept[0] = kKeptUnknown;
            if (b == 2) table_count_row<DT, 4>(t, row, tau, g, q);
            else if (b == 3) table_count_row<DT, 8>(t, row, tau, g, q);
            else table_count_row<DT, 16>(t, row, tau, g, q);
        }
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

// Kept entries of a row whose entry-keeping values were listed by the count step: a weight is a candidate
// exactly when its key is in the list, so no error is evaluated here.  Ordering as in table_emit_row.
__device__ void table_emit_row_by_keys(const uint16_t* __restrict__ w, int64_t d_out, const uint32_t my_kept /* list slot threadIdx.x */,
                                       int nkept, int64_t row, int te, int64_t out0, int32_t* __restrict__ rows,
                                       int32_t* __restrict__ cols, uint16_t* __restrict__ vals, int* list_col,
                                       unsigned char* list_eq, int* list_n, uint32_t* s_kept, const uint4 first, const uint4 second) {
    if (threadIdx.x == 0) *list_n = 0;
    // Almost no weight is a candidate, and candidates lie far from their centroids: a weight whose magnitude
    // is below the smallest magnitude among the listed values cannot be one.
    if (threadIdx.x < 32) {  // at most kKeptCap = 31 listed values: the last slot carries that magnitude
        uint32_t mag = 0x7fffu;
        if ((int)threadIdx.x < nkept) {
            const uint32_t kk = my_kept;
            s_kept[threadIdx.x] = kk;
            mag = (kk & 0xffffu) >= 0x8000u ? kk & 0x7fffu : 0x7fffu - (kk & 0xffffu);
        }
        mag = __reduce_min_sync(0xffffffffu, mag);
        if (threadIdx.x == 31) s_kept[31] = mag;
    }
    __syncthreads();
    const uint32_t mag_bias = (0x8000u - s_kept[31]) * 0x00010001u;
    const bool vec = ((reinterpret_cast<uintptr_t>(w) & 15) == 0);
    for (int64_t j0 = (int64_t)threadIdx.x * 8; j0 < d_out; j0 += (int64_t)blockDim.x * 8) {
        uint32_t pk[4] = {0u, 0u, 0u, 0u};
        if (j0 + 7 < d_out && vec) {
            // the first two groups of eight of a thread were requested when the kernel started
            const uint4 v = j0 == (int64_t)threadIdx.x * 8 ? first
                          : (j0 == (int64_t)(blockDim.x + threadIdx.x) * 8 ? second : __ldg(reinterpret_cast<const uint4*>(w + j0)));
            pk[0] = v.x; pk[1] = v.y; pk[2] = v.z; pk[3] = v.w;
        } else {
#pragma unroll
            for (int u = 0; u < 8; ++u)
                if (j0 + u < d_out) pk[u >> 1] |= (uint32_t)w[j0 + u] << (16 * (u & 1));
        }
        // two magnitudes per word against the smallest listed one: bit 15 of a half survives the addition
        // exactly when that weight is at least as large (no carry between the halves: both terms < 2^15 + 1)
        uint32_t large = 0u;
#pragma unroll
        for (int q = 0; q < 4; ++q) large |= ((pk[q] & 0x7fff7fffu) + mag_bias) & 0x80008000u;
        if (!large) continue;
        uint32_t key[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            uint32_t h = (pk[u >> 1] >> (16 * (u & 1))) & 0xffffu;
            if (h == 0x8000u) h = 0u;  // -0 and +0 are the same point
            key[u] = (h & 0x8000u) ? (~h & 0xffffu) : (h | 0x8000u);
        }
        for (int i = 0; i < nkept; ++i) {
            const uint32_t kk = s_kept[i];
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                if (key[u] == (kk & 0xffffu) && j0 + u < d_out) {
                    const int p = atomicAdd(list_n, 1);
                    if (p < kEmitListCap) {
                        list_col[p] = (int)(j0 + u);
                        list_eq[p] = (unsigned char)(kk >> 16);
                    }
                }
            }
        }
    }
    __syncthreads();
    const int n = *list_n < kEmitListCap ? *list_n : kEmitListCap;
    for (int i = threadIdx.x; i < n; i += blockDim.x) {
        const int c = list_col[i];
        const int is_eq = list_eq[i];
        int before = 0, eq_before = 0;  // candidates / threshold-candidates in lower columns
        for (int u = 0; u < n; ++u) {
            const int lower = list_col[u] < c ? 1 : 0;
            before += lower;
            eq_before += lower & list_eq[u];
        }
        const bool keep = !is_eq || eq_before < te;
        if (keep) {
            const int dropped_before = eq_before > te ? eq_before - te : 0;
            const int64_t pos = out0 + before - dropped_before;
            rows[pos] = (int32_t)row;
            cols[pos] = c;
            vals[pos] = w[c];
        }
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
    __shared__ uint32_t s_kept[32];
    const int64_t row = blockIdx.x;
    const uint16_t* w = W + row * ldw;
    // nearly every row keeps something: its weights are requested before anything else is looked at
    uint4 first = make_uint4(0u, 0u, 0u, 0u), second = make_uint4(0u, 0u, 0u, 0u);
    if ((reinterpret_cast<uintptr_t>(w) & 15) == 0) {
        if ((int64_t)threadIdx.x * 8 + 7 < d_out) first = __ldg(reinterpret_cast<const uint4*>(w + (int64_t)threadIdx.x * 8));
        if ((int64_t)(blockDim.x + threadIdx.x) * 8 + 7 < d_out)
            second = __ldg(reinterpret_cast<const uint4*>(w + (int64_t)(blockDim.x + threadIdx.x) * 8));
    }
    // ... and so are the row's few words (each a round trip to L2 when asked for one after the other)
    const int64_t out0 = row_start[row], out1 = row_start[row + 1];
    const int act = is_act[row];
    const int te = take_eq[row];
    const int ncand = gt[row] + eq[row];
    const uint32_t nkept = t.kept[row * 32];
    const uint32_t my_kept = threadIdx.x < (unsigned)kKeptCap ? t.kept[row * 32 + 1 + threadIdx.x] : 0u;  // slot of the list, if used
    if (out1 == out0) return;
    if (act) {
        for (int64_t j = threadIdx.x; j < d_out; j += blockDim.x) {
            rows[out0 + j] = (int32_t)row;
            cols[out0 + j] = (int32_t)j;
            vals[out0 + j] = w[j];
        }
        return;
    }
    if (nkept != kKeptUnknown && ncand <= kEmitListCap) {
        table_emit_row_by_keys(w, d_out, my_kept, (int)nkept, row, te, out0, rows, cols, vals, list_col, list_eq,
                               &list_n, s_kept, first, second);
        return;
    }
    const uint32_t tau = st->tau;
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

template <int DT, int E, int MAXT, int MINB, int SLOTS>
static cmpq_status launch_table(const LloydArgs& args, const Tables& t, int threads, cudaStream_t st) {
    const size_t smem = sizeof(TableShared) + (size_t)SLOTS * kSlotWords * sizeof(uint32_t) +
                        (((size_t)args.d_out + 31) / 32) * sizeof(uint32_t) + (size_t)kStageCap * sizeof(uint32_t);
    auto kern = lloyd_table_kernel<DT, E, MAXT, MINB, SLOTS>;
    static bool raised[64] = {};  // per instance of this template, hence per kernel
    const size_t smem_limit = sizeof(TableShared) + (size_t)SLOTS * kSlotWords * sizeof(uint32_t) +
                              (((size_t)CMPQ_MAX_D_OUT + 31) / 32) * sizeof(uint32_t) + (size_t)kStageCap * sizeof(uint32_t);
    if (!raise_smem_limit_once(kern, smem_limit, raised)) return CMPQ_ERR_CUDA;
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
    // 32 high-byte buckets per pass cover a zero-centred channel of a few thousand weights in one pass; longer
    // rows reach further into the small magnitudes and get 64
    if (N <= 2048) return launch_table<DT, 4, 512, 2, 32>(args, t, threads_for(4), st);
    if (N <= 4096) return launch_table<DT, 16, 256, 4, 32>(args, t, threads_for(16), st);
    if (N <= 8192) return launch_table<DT, 16, 512, 2, 32>(args, t, threads_for(16), st);
    if (N <= 16384) return launch_table<DT, 16, 1024, 1, 64>(args, t, threads_for(16), st);
    return launch_table<DT, 32, 1024, 1, 64>(args, t, threads_for(32), st);
}

const void* lloyd_table_kernel_address() {
    return reinterpret_cast<const void*>(&lloyd_table_kernel<CMPQ_BF16, 16, 256, 4, 32>);
}

// Sensitivity-weighted fit (see lloyd_weighted_table_kernel): value tables, the weighted iterations on them,
// the all-weights kernel for channels whose tables are too long for shared memory, then the last assignment
// of the channels fitted on tables.  The two flag arrays live in the tables' list area, unused here.
cmpq_status launch_lloyd_weighted_tables(const LloydArgs& args, cmpq_dtype dt, const float* sens, void* tables,
                                         size_t tables_bytes, cudaStream_t st) {
    const Tables t = tables_at(tables, tables_bytes, args.d_in, args.d_out);
    const int64_t N = args.d_out;
    LloydArgs ta = args;
    ta.inexact_rows = nullptr;  // the exactness diagnostic belongs to the unweighted sums
    cmpq_status s = dt == CMPQ_F16 ? launch_table_dt<CMPQ_F16>(ta, t, st) : launch_table_dt<CMPQ_BF16>(ta, t, st);
    if (s != CMPQ_OK) return s;
    const int fit = (int)((N + 2 + 15) / 16 * 16);  // a table has at most d_out + 1 entries
    int caps[2] = {N <= 4096 ? 1536 : (N <= 12288 ? 2560 : 3584), fit < 11264 ? fit : 11264};
    if (caps[0] > fit) caps[0] = fit;
    uint8_t* fitted = reinterpret_cast<uint8_t*>(t.kept);
    uint8_t* not_fitted = fitted + args.d_in;
    const size_t smem_max = weighted_table_smem(caps[1], N);
    static bool raised_f16[64] = {}, raised_bf16[64] = {};
    const size_t smem_limit = weighted_table_smem(11264, CMPQ_MAX_D_OUT);
    if (smem_max > smem_limit) return CMPQ_ERR_INTERNAL;
    if (!raise_smem_limit_once(lloyd_weighted_table_kernel<CMPQ_F16>, smem_limit, raised_f16) ||
        !raise_smem_limit_once(lloyd_weighted_table_kernel<CMPQ_BF16>, smem_limit, raised_bf16))
        return CMPQ_ERR_CUDA;
    for (int pass = 0; pass < 2; ++pass) {
        if (pass == 1 && caps[1] <= caps[0]) break;
        const size_t smem = weighted_table_smem(caps[pass], N);
        if (dt == CMPQ_F16)
            lloyd_weighted_table_kernel<CMPQ_F16><<<(unsigned)args.d_in, kWtThreads, smem, st>>>(ta, t, sens, caps[pass], pass, fitted, not_fitted);
        else
            lloyd_weighted_table_kernel<CMPQ_BF16><<<(unsigned)args.d_in, kWtThreads, smem, st>>>(ta, t, sens, caps[pass], pass, fitted, not_fitted);
        s = launch_status();
        if (s != CMPQ_OK) return s;
    }
    LloydArgs oa = args;
    oa.skip_row = fitted;
    s = launch_lloyd_weighted(oa, dt, sens, st);
    if (s != CMPQ_OK) return s;
    LloydArgs aa = args;
    aa.skip_row = not_fitted;
    aa.packed = nullptr;
    const int assign_threads = N <= 4096 ? kAssignThreads / 2 : kAssignThreads;
    if (dt == CMPQ_F16) lloyd_assign_kernel<CMPQ_F16, false><<<(unsigned)args.d_in, assign_threads, 0, st>>>(aa, args.lut, t.thr);
    else lloyd_assign_kernel<CMPQ_BF16, false><<<(unsigned)args.d_in, assign_threads, 0, st>>>(aa, args.lut, t.thr);
    return launch_status();
}

// tables_ready: the value tables of every row to be fitted are in place already (skip the table kernel)
template <int DT>
static cmpq_status launch_ordered_dt(const LloydArgs& args, const Tables& t, bool tables_ready, cudaStream_t st,
                                     const Tables* patch_from = nullptr) {
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
    ia.nonfinite = args.nonfinite;
    ia.side_hist = args.side_hist;
    if (patch_from) {
        ia.src = *patch_from;
        ia.W = args.W;
        ia.ldw = args.ldw;
        ia.row_ptr = args.row_ptr;
        ia.cols = args.cols;
        ia.inexact_rows = args.inexact_rows;
    }
    // distinct 16-bit values grow slowly with the channel length (about 1400 at 4096 weights, 2300 at
    // 28672 for Gaussian-like bf16 weights); longer tables are read from global memory
    ia.cap = N <= 4096 ? kMinIterCap : (N <= 12288 ? 2048 : 3072);
    const size_t iter_smem = (size_t)kIterWarps * 2 * iter_channel_bytes(ia.cap);
    static bool raised[64] = {};  // per instance of this template, hence per kernel
    if (!raise_smem_limit_once(lloyd_iterate_kernel<DT>, (size_t)kIterWarps * 2 * iter_channel_bytes(3072), raised))
        return CMPQ_ERR_CUDA;
    const unsigned iter_blocks = (unsigned)((args.d_in + kIterWarps * 2 - 1) / (kIterWarps * 2));
    lloyd_iterate_kernel<DT><<<iter_blocks, kIterWarps * 32, iter_smem, st>>>(ia);
    s = launch_status();
    if (s != CMPQ_OK) return s;
    if (ev[2]) cudaEventRecord(ev[2], st);

    // neither codes nor errors wanted: the fit alone (centroids and thresholds stay in the tables)
    // a short row keeps fewer threads busy for longer: the per-row set-up (centroids, thresholds, removed
    // columns) is paid once per thread
    const int assign_threads = N <= 4096 ? kAssignThreads / 2 : kAssignThreads;
    if (args.err) lloyd_assign_kernel<DT, true><<<(unsigned)args.d_in, assign_threads, 0, st>>>(args, ia.lut, t.thr);
    else if (args.codes || args.packed) lloyd_assign_kernel<DT, false><<<(unsigned)args.d_in, assign_threads, 0, st>>>(args, ia.lut, t.thr);
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
// Final fit from the tables of the provisional fit: the iterate kernel builds every channel's table
// from the provisional one (see patch_table), so nothing is read from the weights and counted again.

// args: the final fit (row_ptr / cols = the removed positions, skip_row unused).  prov_tables: the
// tables the provisional fit left; tables: scratch of the final fit for the channels whose table does not
// fit in shared memory.  tables == prov_tables is allowed: those channels are then patched in place (the
// update is element-wise), which destroys the provisional tables.
cmpq_status launch_lloyd_ordered_patched(const LloydArgs& args, cmpq_dtype dt, void* prov_tables, void* tables,
                                         size_t tables_bytes, cudaStream_t st) {
    if (!prov_tables || !tables || tables_bytes < lloyd_tables_bytes(args.d_in, args.d_out)) return CMPQ_ERR_WORKSPACE;
    if (!args.row_ptr) return CMPQ_ERR_INTERNAL;
    const Tables src = tables_at(prov_tables, tables_bytes, args.d_in, args.d_out);
    const Tables dst = tables_at(tables, tables_bytes, args.d_in, args.d_out);
    return dt == CMPQ_F16 ? launch_ordered_dt<CMPQ_F16>(args, dst, true, st, &src)
                          : launch_ordered_dt<CMPQ_BF16>(args, dst, true, st, &src);
}

}  // namespace cmpq
