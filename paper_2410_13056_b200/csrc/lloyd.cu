// Channel-wise K-means of CMPQ (Section 3.2.1: K-means per channel W_{i,:} with K = 2^bits;
// Section 3: each weight is replaced by its nearest centroid).
//
// One thread block fits one channel.  The channel is read from HBM once, widened to fp32 and
// kept in REGISTERS (E weights per thread) for all iterations together with its codes, so an
// iteration moves no HBM bytes and no shared-memory bytes either.  Nothing here is a dense
// contraction: the work is K subtract / compare steps per weight per sweep on the fp32 pipes, so
// no tensor cores are used.
//
//   start       K order statistics of the channel, found by a two-level counting select on the
//               16-bit keys (256 buckets by high byte, then 256 by low byte inside the buckets
//               that hold a target) -- no sort
//   sweep       defined as: the first k minimising fabsf(x - c_k) (fp32, strict '<' scan).
//               When the centroids are strictly increasing and every gap exceeds 2^-22 times the
//               channel's value range, two values x - c_k and x - c_{k-1} can never round to the
//               same float, and then that first minimum equals the number of k >= 1 with
//               fabsf(x - c_k) < fabsf(x - c_{k-1}); the sweep counts those with one subtract, one
//               compare and one predicated add per (weight, centroid).  Otherwise it runs the
//               plain scan.  Codes of four weights are accumulated in one float (base 16), so
//               an unchanged group costs one compare.
//   update      cluster sums are kept in fp64 and counts in int32.  The first sweep rebuilds them
//               from scratch (per-warp partials added in warp order); later sweeps list the
//               weights whose code changed and move only those between clusters (
//               per-warp partial changes, no atomics on the sums); a sweep that changes more than
//               1/8 of the weights rebuilds instead.
//               16-bit weights of bounded dynamic range make every such sum exact in fp64, so
//               the order of the additions cannot change the result
//   stop        a sweep that changes no code ends the loop early: later iterations would
//               repeat it exactly
#include "lloyd.cuh"

namespace cmpq {

constexpr int kMaxK = 16;
constexpr int kMaxWarps = 32;

struct alignas(16) LloydShared {
    double wsum[kMaxWarps][kMaxK];  // per-warp cluster sums of a rebuild
    int wcnt[kMaxWarps][kMaxK];
    int hist1[256];
    int excl1[257];
    double S[kMaxK];
    int n[kMaxK];
    float c[kMaxK];
    int tgt_bucket[kMaxK];
    int tgt_resid[kMaxK];
    int tgt_slot[kMaxK];
    unsigned char slot_of_bucket[256];
    int changed[2];     // weights whose code changed in the current sweep (by sweep parity)
    int list_count[2];  // entries appended to the change list (may exceed its capacity)
    int fast;         // centroids strictly increasing with safe gaps
    float vmin, vmax; // value range of the channel
    float wlo[kMaxWarps], whi[kMaxWarps];  // per-warp value range, largest exponent, smallest ulp
    int wtop[kMaxWarps], wulp[kMaxWarps];
};
// dynamic shared memory after LloydShared: scratch region (lloyd_scratch_bytes), then float xs[N]

// Bytes of the multi-purpose scratch region: second-level histogram (start), change list (N/8
// entries), removed-column bitmap (load).
__host__ __device__ inline int lloyd_scratch_bytes(int N) {
    int hist2 = kMaxK * 256 * (int)sizeof(int);
    int list = (N >> 3) * 4;
    int bitmap = ((N + 31) / 32) * 4;
    int m = hist2 > list ? hist2 : list;
    m = m > bitmap ? m : bitmap;
    return (m + 15) & ~15;
}

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

// The K starting centroids: the ((2k+1) N)/(2K)-th smallest values of the channel.
template <int DT, int K, int E>
__device__ void select_start(const float (&x)[E], int nval, int N, LloydShared& sh, int* hist2) {
    const int tid = threadIdx.x, nthr = blockDim.x, lane = tid & 31, warp = tid >> 5;
    const int nwarps = nthr >> 5;
    for (int b = tid; b < 256; b += nthr) { sh.hist1[b] = 0; sh.slot_of_bucket[b] = 0xff; }
    for (int b = tid; b < K * 256; b += nthr) hist2[b] = 0;
    __syncthreads();
#pragma unroll
    for (int e = 0; e < E; ++e)
        if (e < nval) atomicAdd(&sh.hist1[sort_key16<DT>(x[e]) >> 8], 1);
    __syncthreads();
    if (warp == 0) {  // exclusive prefix of the 256 bucket counts
        int v[8], s = 0;
#pragma unroll
        for (int t = 0; t < 8; ++t) { v[t] = sh.hist1[lane * 8 + t]; s += v[t]; }
        int incl = s;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            int up = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += up;
        }
        int run = incl - s;
#pragma unroll
        for (int t = 0; t < 8; ++t) { sh.excl1[lane * 8 + t] = run; run += v[t]; }
        if (lane == 31) sh.excl1[256] = run;
    }
    __syncthreads();
    if (tid < K) {
        int pos = (int)(((long long)(2 * tid + 1) * N) / (2 * K));
        int lo = 0, hi = 256;  // last bucket b with excl1[b] <= pos
        while (hi - lo > 1) {
            int mid = (lo + hi) >> 1;
            if (sh.excl1[mid] <= pos) lo = mid; else hi = mid;
        }
        sh.tgt_bucket[tid] = lo;
        sh.tgt_resid[tid] = pos - sh.excl1[lo];
    }
    __syncthreads();
    if (tid == 0) {
        int slots = 0;
        for (int k = 0; k < K; ++k) {
            int b = sh.tgt_bucket[k];
            if (k == 0 || b != sh.tgt_bucket[k - 1]) sh.slot_of_bucket[b] = (unsigned char)slots++;
            sh.tgt_slot[k] = sh.slot_of_bucket[b];
        }
    }
    __syncthreads();
#pragma unroll
    for (int e = 0; e < E; ++e) {
        if (e < nval) {
            uint32_t key = sort_key16<DT>(x[e]);
            int slot = sh.slot_of_bucket[key >> 8];
            if (slot != 0xff) atomicAdd(&hist2[slot * 256 + (key & 0xff)], 1);
        }
    }
    __syncthreads();
    for (int k = warp; k < K; k += nwarps) {  // one warp resolves one target inside its bucket
        const int* h = hist2 + sh.tgt_slot[k] * 256;
        const int resid = sh.tgt_resid[k];
        int v[8], s = 0;
#pragma unroll
        for (int t = 0; t < 8; ++t) { v[t] = h[lane * 8 + t]; s += v[t]; }
        int incl = s;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            int up = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += up;
        }
        int run = incl - s;
        if (resid >= run && resid < incl) {
            int t = 0;
            while (resid >= run + v[t]) { run += v[t]; ++t; }
            sh.c[k] = value_of_key16<DT>((uint32_t)(sh.tgt_bucket[k] << 8) | (uint32_t)(lane * 8 + t));
        }
    }
    __syncthreads();
}

// Warp 0 decides whether the counting sweep is valid for the centroids now in sh.c.
template <int K>
__device__ __forceinline__ void decide_fast(LloydShared& sh) {
    if (threadIdx.x < 32) {
        const int lane = threadIdx.x;
        float ck = sh.c[lane < K ? lane : K - 1];
        float cp = __shfl_up_sync(0xffffffffu, ck, 1);
        double need = ((double)sh.vmax - (double)sh.vmin) * (1.0 / 4194304.0);  // range * 2^-22
        bool ok = (lane == 0 || lane >= K) ? true : ((double)ck - (double)cp > need);
        ok = __all_sync(0xffffffffu, ok);
        if (lane == 0) sh.fast = ok ? 1 : 0;
    }
}

// Per-warp cluster sums and counts of all weights, from the codes in registers.
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

// Per-warp changes of the cluster sums and counts caused by the listed weights.  Thread t looks
// after cluster t mod K and every (nthr/K)-th list entry; lanes with the same cluster are combined
// with shuffles, so no two threads ever add to the same address.
template <int K>
__device__ void list_partials(const uint32_t* list, int L, const float* xs, LloydShared& sh) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int k = tid & (K - 1), seg = tid / K, nseg = blockDim.x / K;
    double ds = 0.0;
    int dn = 0;
    for (int t = seg; t < L; t += nseg) {
        const uint32_t en = list[t];  // column | old code << 16 | new code << 20
        const int o = (en >> 16) & 15, nw = (en >> 20) & 15;
        const double xv = (double)xs[en & 0xffffu];
        if (nw == k) { ds += xv; ++dn; }
        if (o == k) { ds -= xv; --dn; }
    }
#pragma unroll
    for (int o = K; o < 32; o <<= 1) {
        ds += __shfl_xor_sync(0xffffffffu, ds, o);
        dn += __shfl_xor_sync(0xffffffffu, dn, o);
    }
    if (lane < K) { sh.wsum[warp][lane] = ds; sh.wcnt[warp][lane] = dn; }
}

// Warp 0: combine the per-warp partials into S and n (absolute after a rebuild, as a change after
// a list pass), move every non-empty cluster's centroid to its mean and decide whether the counting
// sweep is valid for the new centroids.
template <int K>
__device__ __forceinline__ void update_centroids(LloydShared& sh, bool absolute) {
    if (threadIdx.x < 32) {
        const int lane = threadIdx.x, nwarps = blockDim.x >> 5;
        float ck = 0.f;
        if (lane < K) {
            double s = 0.0;
            int cnt = 0;
            for (int w = 0; w < nwarps; ++w) { s += sh.wsum[w][lane]; cnt += sh.wcnt[w][lane]; }
            if (!absolute) { s += sh.S[lane]; cnt += sh.n[lane]; }
            sh.S[lane] = s;
            sh.n[lane] = cnt;
            ck = sh.c[lane];
            if (cnt > 0) { ck = __double2float_rn(__ddiv_rn(s, (double)cnt)); sh.c[lane] = ck; }
        }
        ck = __shfl_sync(0xffffffffu, ck, lane < K ? lane : K - 1);
        float cp = __shfl_up_sync(0xffffffffu, ck, 1);
        double need = ((double)sh.vmax - (double)sh.vmin) * (1.0 / 4194304.0);  // range * 2^-22
        bool ok = (lane == 0 || lane >= K) ? true : ((double)ck - (double)cp > need);
        ok = __all_sync(0xffffffffu, ok);
        if (lane == 0) sh.fast = ok ? 1 : 0;
    }
}

template <int DT, int K, int E>
__device__ void fit_channel(const LloydArgs& a, int64_t row, float (&x)[E], int nval, LloydShared& sh,
                            unsigned char* dyn, const float* xs) {
    constexpr int G = E / 4;          // float accumulators: codes of 4 weights each, base 16
    constexpr int WORDS = (E + 7) / 8;  // packed codes: 8 weights per 32-bit word
    const int tid = threadIdx.x, nthr = blockDim.x, lane = tid & 31;
    const int N = (int)a.d_out;
    const int T = a.iters;
    uint32_t* list = reinterpret_cast<uint32_t*>(dyn);
    const int list_cap = N >> 3;

    select_start<DT, K, E>(x, nval, N, sh, reinterpret_cast<int*>(dyn));
    if (tid < 2) { sh.changed[tid] = 0; sh.list_count[tid] = 0; }
    decide_fast<K>(sh);
    __syncthreads();

    uint32_t cw[WORDS];
#pragma unroll
    for (int w = 0; w < WORDS; ++w) cw[w] = 0;
    float c[K];
    int sweeps_done = 0;
    int prev_changed = N;
    for (int it = 0; it <= T; ++it) {
#pragma unroll
        for (int k = 0; k < K; ++k) c[k] = sh.c[k];
        const bool fast = sh.fast != 0;
        const bool last = (it == T), first = (it == 0);
        const bool use_list = !first && !last && prev_changed <= list_cap;
        const int par = it & 1;

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
        uint32_t nw[WORDS];
#pragma unroll
        for (int w = 0; w < WORDS; ++w)
            nw[w] = (2 * w + 1 < G) ? __byte_perm(half[2 * w], half[2 * w + 1], 0x5410) : (half[2 * w] & 0xffffu);
        ++sweeps_done;

        // weights whose code changed (few once the fit settles)
        uint32_t any = 0;
#pragma unroll
        for (int w = 0; w < WORDS; ++w) any |= nw[w] ^ cw[w];
        int nch = 0;
        if (first) {
            nch = nval;
        } else if (any) {
            uint32_t m[WORDS];  // bit 4i set: weight i of the word changed
#pragma unroll
            for (int w = 0; w < WORDS; ++w) {
                uint32_t xr = nw[w] ^ cw[w];
                m[w] = (xr | (xr >> 1) | (xr >> 2) | (xr >> 3)) & 0x11111111u;
                nch += __popc(m[w]);
            }
            if (use_list) {
                int pos = atomicAdd(&sh.list_count[par], nch);
#pragma unroll
                for (int w = 0; w < WORDS; ++w) {
                    uint32_t mm = m[w];
                    while (mm) {
                        const int b = __ffs(mm) - 1;
                        mm &= mm - 1;
                        const int e = 8 * w + (b >> 2);
                        const uint32_t j = (uint32_t)(((e >> 2) * nthr + tid) * 4 + (e & 3));
                        if (pos < list_cap)
                            list[pos] = j | (((cw[w] >> b) & 15u) << 16) | (((nw[w] >> b) & 15u) << 20);
                        ++pos;
                    }
                }
            }
        }
#pragma unroll
        for (int w = 0; w < WORDS; ++w) cw[w] = nw[w];
        nch = warp_sum(nch);
        if (lane == 0 && nch) atomicAdd(&sh.changed[par], nch);
        __syncthreads();
        const int total_changed = sh.changed[par];
        const int L = sh.list_count[par];
        if (tid == 0) { sh.changed[par ^ 1] = 0; sh.list_count[par ^ 1] = 0; }
        prev_changed = total_changed;
        if (last || total_changed == 0) break;  // uniform: every thread reads the same value
        const bool by_list = use_list && L <= list_cap;
        if (by_list) list_partials<K>(list, L, xs, sh);
        else rebuild_partials<K, E>(x, cw, nval, sh);
        __syncthreads();
        update_centroids<K>(sh, !by_list);
        __syncthreads();
    }

    // outputs: thread owns weights j = (g * nthr + tid) * 4 + u
    if (a.lut && tid < CMPQ_LUT_STRIDE) a.lut[row * CMPQ_LUT_STRIDE + tid] = tid < K ? sh.c[tid] : 0.f;
    const bool vec4 = (a.d_out & 3) == 0;
#pragma unroll
    for (int g = 0; g < G; ++g) {
        const int j0 = (g * nthr + tid) * 4;
        if (j0 >= N) continue;
        const uint32_t p = (cw[g >> 1] >> (16 * (g & 1))) & 0xffffu;
        if (a.codes) {
            uint8_t* out = a.codes + row * a.d_out + j0;
            if (vec4) {
                uint32_t w = (p & 15u) | (((p >> 4) & 15u) << 8) | (((p >> 8) & 15u) << 16) | (((p >> 12) & 15u) << 24);
                *reinterpret_cast<uint32_t*>(out) = w;
            } else {
#pragma unroll
                for (int u = 0; u < 4; ++u)
                    if (j0 + u < N) out[u] = (uint8_t)((p >> (4 * u)) & 15u);
            }
        }
        if (a.err) {
            float* out = a.err + row * a.d_out + j0;
            float ev[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) ev[u] = fabsf(x[4 * g + u] - sh.c[(p >> (4 * u)) & 15u]);
            if (vec4) {
                *reinterpret_cast<float4*>(out) = make_float4(ev[0], ev[1], ev[2], ev[3]);
            } else {
#pragma unroll
                for (int u = 0; u < 4; ++u)
                    if (j0 + u < N) out[u] = ev[u];
            }
        }
    }
    if (a.sweeps && tid == 0)
        atomicAdd(a.sweeps, (unsigned long long)sweeps_done * (unsigned long long)N * (unsigned long long)K);
}

template <int DT, int E, int MAXT>
__global__ void __launch_bounds__(MAXT)
lloyd_kernel(const LloydArgs a) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const int64_t row = blockIdx.x;
    if (a.skip_row && a.skip_row[row]) return;
    const int N = (int)a.d_out;
    LloydShared& sh = *reinterpret_cast<LloydShared*>(smem_raw);
    unsigned char* dyn = smem_raw + sizeof(LloydShared);          // hist2 / change list / bitmap
    float* xs = reinterpret_cast<float*>(dyn + lloyd_scratch_bytes(N));  // fp32 copy of the channel
    const int tid = threadIdx.x, nthr = blockDim.x, lane = tid & 31;

    // removed positions (outliers of this row) are marked in a bitmap over the columns
    uint32_t* removed = reinterpret_cast<uint32_t*>(dyn);
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
    }
    __syncthreads();

    // thread owns weights j = (g * nthr + tid) * 4 + u, u = 0..3; valid ones form a prefix
    const uint16_t* w = a.W + row * a.ldw;
    const bool vec = ((a.ldw & 3) == 0) && ((reinterpret_cast<uintptr_t>(a.W) & 7) == 0);
    float x[E];
    int nval = 0;
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
            float v = widen16<DT>(h[u]);
            const int j = j0 + u;
            if (j < N) {
                ++nval;
                if (has_removed && ((removed[j >> 5] >> (j & 31)) & 1)) v = 0.f;
                v = (v == 0.f) ? 0.f : v;  // -0 and +0 are the same point
                xs[j] = v;
            } else {
                v = __int_as_float(0x7f800000);  // padding: +inf always gets code 0 and never changes
            }
            x[4 * g + u] = v;
        }
    }
    // value range (for the gap test) and exactness diagnostics
    {
        float lo = __int_as_float(0x7f800000), hi = __int_as_float(0xff800000);
        int top = -100000, ulp = 100000;
#pragma unroll
        for (int e = 0; e < E; ++e) {
            if (e < nval) {
                lo = fminf(lo, x[e]);
                hi = fmaxf(hi, x[e]);
                uint32_t u = __float_as_uint(x[e]) & 0x7fffffffu;
                if (u) {
                    int ex = (int)(u >> 23);
                    uint32_t m = u & 0x7fffffu;
                    int t, q;
                    if (ex) { t = ex - 127; q = ex - 150 + (__ffs(m | 0x800000u) - 1); }
                    else    { t = (31 - __clz(m)) - 149; q = (__ffs(m) - 1) - 149; }
                    top = max(top, t);
                    ulp = min(ulp, q);
                }
            }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            lo = fminf(lo, __shfl_xor_sync(0xffffffffu, lo, o));
            hi = fmaxf(hi, __shfl_xor_sync(0xffffffffu, hi, o));
            top = max(top, __shfl_xor_sync(0xffffffffu, top, o));
            ulp = min(ulp, __shfl_xor_sync(0xffffffffu, ulp, o));
        }
        const int warp = tid >> 5, nwarps = nthr >> 5;
        if (lane == 0) { sh.wlo[warp] = lo; sh.whi[warp] = hi; sh.wtop[warp] = top; sh.wulp[warp] = ulp; }
        __syncthreads();  // also: every thread is done with the removed-column bitmap
        if (tid == 0) {
            for (int wv = 1; wv < nwarps; ++wv) {
                lo = fminf(lo, sh.wlo[wv]);
                hi = fmaxf(hi, sh.whi[wv]);
                top = max(top, sh.wtop[wv]);
                ulp = min(ulp, sh.wulp[wv]);
            }
            sh.vmin = lo;
            sh.vmax = hi;
            if (a.inexact_rows && top > -100000) {
                // sums and differences of up to 2N weights stay exact in fp64 while
                // 2 N 2^(top+1) / 2^ulp <= 2^53
                int log2n = 32 - __clz(N - 1 > 0 ? N - 1 : 1);
                if (log2n + 1 + (top + 1 - ulp) > 53) atomicAdd(a.inexact_rows, 1);
            }
        }
        __syncthreads();
    }
    const int bits = a.bits[row];
    if (bits == 2) fit_channel<DT, 4, E>(a, row, x, nval, sh, dyn, xs);
    else if (bits == 3) fit_channel<DT, 8, E>(a, row, x, nval, sh, dyn, xs);
    else fit_channel<DT, 16, E>(a, row, x, nval, sh, dyn, xs);
}

static size_t lloyd_smem_bytes(int64_t d_out) {
    return sizeof(LloydShared) + (size_t)lloyd_scratch_bytes((int)d_out) + (((size_t)d_out + 3) & ~(size_t)3) * sizeof(float);
}

template <int DT, int E, int MAXT>
static cmpq_status launch_variant(const LloydArgs& args, int threads, cudaStream_t st) {
    const size_t smem = lloyd_smem_bytes(args.d_out);
    auto kern = lloyd_kernel<DT, E, MAXT>;
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
    if (N <= 2048) return launch_variant<DT, 4, 512>(args, threads_for(4), st);
    if (N <= 16384) return launch_variant<DT, 16, 1024>(args, threads_for(16), st);
    return launch_variant<DT, 32, 1024>(args, threads_for(32), st);
}

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

size_t quantize_ws_bytes(int64_t d_in, int64_t) {
    return round_up((size_t)(d_in + 1) * sizeof(int64_t), 256);
}

}  // namespace cmpq

using namespace cmpq;

extern "C" cmpq_status cmpq_quantize_layer(const void* W, cmpq_dtype dt, int64_t d_in, int64_t d_out,
                                           int64_t ldw, const uint8_t* bits, const int32_t* rows,
                                           const int32_t* cols, int64_t nnz, int lloyd_iters,
                                           const float* sens, float* lut, uint8_t* codes,
                                           int32_t* inexact_rows, unsigned long long* sweeps,
                                           void* ws, size_t ws_bytes, void* stream) {
    if (!W || !bits || !lut || !codes) return CMPQ_ERR_INVALID_ARG;
    if (dt != CMPQ_F16 && dt != CMPQ_BF16) return CMPQ_ERR_INVALID_ARG;
    if (d_in < 1 || d_in > CMPQ_MAX_D_IN || d_out < 1 || d_out > CMPQ_MAX_D_OUT || ldw < d_out)
        return CMPQ_ERR_INVALID_ARG;
    if (nnz < 0 || nnz > d_in * d_out || (nnz > 0 && (!rows || !cols))) return CMPQ_ERR_INVALID_ARG;
    if (lloyd_iters < 0 || lloyd_iters > CMPQ_MAX_LLOYD_ITERS) return CMPQ_ERR_INVALID_ARG;
    if (!aligned_to(W, 2) || !aligned_to(lut, 4)) return CMPQ_ERR_INVALID_ARG;
    if (sens) return CMPQ_ERR_UNSUPPORTED;
    if (!ws || !aligned_to(ws, 256) || ws_bytes < quantize_ws_bytes(d_in, d_out)) return CMPQ_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int64_t* row_ptr = static_cast<int64_t*>(ws);
    cmpq_status s = launch_row_ptr(rows, nnz, d_in, row_ptr, st);
    if (s != CMPQ_OK) return s;
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
    return launch_lloyd(a, dt, st);
}
