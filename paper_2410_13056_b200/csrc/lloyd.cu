// Channel-wise K-means of CMPQ (Section 3.2.1: K-means per channel W_{i,:} with K = 2^bits;
// Section 3: each weight is replaced by its nearest centroid).
//
// One thread block fits one channel.  The channel is read from HBM once, widened to fp32 and
// kept in shared memory for all iterations together with its current codes, so an iteration
// moves no HBM bytes.  Nothing here is a dense contraction: the work is K subtract / compare
// steps per weight per sweep on the fp32 pipes, so no tensor cores are used.
//
//   start       K order statistics of the channel, found by a two-level counting select on the
//               16-bit keys (256 buckets by high byte, then 256 by low byte inside the buckets
//               that hold a target) -- no sort
//   sweep       every thread assigns its weights to the first nearest centroid (centroids in
//               registers, fp32 |x - c_k|, strict '<' scan)
//   update      cluster sums are kept in fp64 and counts in int32.  The first sweep, and any
//               sweep after one that moved more than 1/8 of the weights, rebuilds them from
//               scratch (per-warp partials added in warp order); otherwise only the weights
//               whose code changed are moved between clusters with shared-memory atomics.
//               16-bit weights of bounded dynamic range make every such sum exact in fp64, so
//               the order of the additions cannot change the result
//   stop        a sweep that changes no code ends the loop early: later iterations would
//               repeat it exactly
#include "lloyd.cuh"

namespace cmpq {

constexpr int kMaxK = 16;
constexpr int kMaxWarps = 32;

struct alignas(16) LloydShared {
    union {
        int hist2[kMaxK][256];  // second-level counts, one row per distinct target bucket
        struct {
            double wsum[kMaxWarps][kMaxK];  // per-warp cluster sums of a rebuild
            int wcnt[kMaxWarps][kMaxK];
        } acc;
    } u;
    int hist1[256];
    int excl1[257];
    double S[kMaxK];
    int n[kMaxK];
    float c[kMaxK];
    int tgt_bucket[kMaxK];
    int tgt_resid[kMaxK];
    int tgt_slot[kMaxK];
    unsigned char slot_of_bucket[256];
    int changed;
    int max_top;   // largest exponent of a non-zero weight
    int min_ulp;   // exponent of the smallest unit in the last place among non-zero weights
};

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

template <int K>
__device__ __forceinline__ int nearest(float x, const float (&c)[K]) {
    float best = fabsf(x - c[0]);
    int bk = 0;
#pragma unroll
    for (int k = 1; k < K; ++k) {
        float d = fabsf(x - c[k]);
        if (d < best) { best = d; bk = k; }
    }
    return bk;
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

// The K starting centroids: the ((2k+1) N)/(2K)-th smallest values of the channel.
template <int DT, int K>
__device__ void select_start(const float* xs, int N, LloydShared& sh) {
    const int tid = threadIdx.x, nthr = blockDim.x, lane = tid & 31, warp = tid >> 5;
    const int nwarps = nthr >> 5;
    for (int b = tid; b < 256; b += nthr) { sh.hist1[b] = 0; sh.slot_of_bucket[b] = 0xff; }
    for (int b = tid; b < K * 256; b += nthr) (&sh.u.hist2[0][0])[b] = 0;
    __syncthreads();
    for (int j = tid; j < N; j += nthr) atomicAdd(&sh.hist1[sort_key16<DT>(xs[j]) >> 8], 1);
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
    for (int j = tid; j < N; j += nthr) {
        uint32_t key = sort_key16<DT>(xs[j]);
        int slot = sh.slot_of_bucket[key >> 8];
        if (slot != 0xff) atomicAdd(&sh.u.hist2[slot][key & 0xff], 1);
    }
    __syncthreads();
    for (int k = warp; k < K; k += nwarps) {  // one warp resolves one target inside its bucket
        const int* h = sh.u.hist2[sh.tgt_slot[k]];
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

// Rebuilds S and n from the codes in shared memory (per-warp partials, added in warp order).
template <int K>
__device__ void rebuild_sums(const float* xs, const unsigned char* code, int N, LloydShared& sh) {
    const int tid = threadIdx.x, nthr = blockDim.x, lane = tid & 31, warp = tid >> 5;
    const int nwarps = nthr >> 5;
    for (int k = 0; k < K; ++k) {
        double s = 0.0;
        int cnt = 0;
        for (int j = tid; j < N; j += nthr) {
            bool mine = code[j] == k;
            s += mine ? (double)xs[j] : 0.0;
            cnt += mine ? 1 : 0;
        }
        s = warp_sum(s);
        cnt = warp_sum(cnt);
        if (lane == 0) { sh.u.acc.wsum[warp][k] = s; sh.u.acc.wcnt[warp][k] = cnt; }
    }
    __syncthreads();
    if (tid < K) {
        double s = 0.0;
        int cnt = 0;
        for (int w = 0; w < nwarps; ++w) { s += sh.u.acc.wsum[w][tid]; cnt += sh.u.acc.wcnt[w][tid]; }
        sh.S[tid] = s;
        sh.n[tid] = cnt;
    }
    __syncthreads();
}

template <int DT, int K>
__device__ void fit_channel(const LloydArgs& a, int64_t row, float* xs, unsigned char* code,
                            LloydShared& sh) {
    const int tid = threadIdx.x, nthr = blockDim.x, lane = tid & 31;
    const int N = (int)a.d_out;
    const int T = a.iters;

    select_start<DT, K>(xs, N, sh);

    float c[K];
    bool rebuild = true;  // the first sweep has no previous codes
    int sweeps_done = 0;
    for (int it = 0; it <= T; ++it) {
#pragma unroll
        for (int k = 0; k < K; ++k) c[k] = sh.c[k];
        if (tid == 0) sh.changed = 0;
        __syncthreads();
        const bool last = (it == T);
        const bool first = (it == 0);
        int changed = 0;
        for (int j = tid; j < N; j += nthr) {
            float x = xs[j];
            int nk = nearest<K>(x, c);
            int ok = first ? -1 : (int)code[j];
            if (nk != ok) {
                ++changed;
                code[j] = (unsigned char)nk;
                if (!rebuild && !last) {
                    atomicAdd(&sh.S[nk], (double)x);
                    atomicAdd(&sh.S[ok], -(double)x);
                    atomicAdd(&sh.n[nk], 1);
                    atomicAdd(&sh.n[ok], -1);
                }
            }
        }
        ++sweeps_done;
        changed = warp_sum(changed);
        if (lane == 0 && changed) atomicAdd(&sh.changed, changed);
        __syncthreads();
        const int total_changed = sh.changed;
        if (last || total_changed == 0) break;  // uniform: every thread reads the same value
        if (rebuild) rebuild_sums<K>(xs, code, N, sh);
        if (tid < K && sh.n[tid] > 0)
            sh.c[tid] = __double2float_rn(__ddiv_rn(sh.S[tid], (double)sh.n[tid]));
        rebuild = total_changed > (N >> 3);
        __syncthreads();
    }

    // outputs
#pragma unroll
    for (int k = 0; k < K; ++k) c[k] = sh.c[k];
    if (a.lut && tid < CMPQ_LUT_STRIDE) a.lut[row * CMPQ_LUT_STRIDE + tid] = tid < K ? sh.c[tid] : 0.f;
    if (a.codes) {
        uint8_t* out = a.codes + row * a.d_out;
        if ((a.d_out & 3) == 0) {
            const uint32_t* src = reinterpret_cast<const uint32_t*>(code);
            uint32_t* dst = reinterpret_cast<uint32_t*>(out);
            for (int j = tid; j < (N >> 2); j += nthr) dst[j] = src[j];
        } else {
            for (int j = tid; j < N; j += nthr) out[j] = code[j];
        }
    }
    if (a.err) {
        float* out = a.err + row * a.d_out;
        for (int j = tid; j < N; j += nthr) out[j] = fabsf(xs[j] - sh.c[code[j]]);
    }
    if (a.sweeps && tid == 0)
        atomicAdd(a.sweeps, (unsigned long long)sweeps_done * (unsigned long long)N * (unsigned long long)K);
}

template <int DT>
__global__ void __launch_bounds__(1024)
lloyd_kernel(const LloydArgs a) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const int64_t row = blockIdx.x;
    if (a.skip_row && a.skip_row[row]) return;
    const int N = (int)a.d_out;
    const int npad = (N + 15) & ~15;
    LloydShared& sh = *reinterpret_cast<LloydShared*>(smem_raw);
    float* xs = reinterpret_cast<float*>(smem_raw + sizeof(LloydShared));
    unsigned char* code = reinterpret_cast<unsigned char*>(xs + npad);
    const int tid = threadIdx.x, nthr = blockDim.x, lane = tid & 31;

    if (tid == 0) { sh.max_top = -100000; sh.min_ulp = 100000; }
    const uint16_t* w = a.W + row * a.ldw;
    for (int j = tid; j < N; j += nthr) {
        float x = widen16<DT>(w[j]);
        xs[j] = (x == 0.f) ? 0.f : x;  // -0 and +0 are the same point
    }
    __syncthreads();
    if (a.row_ptr) {
        const int64_t p0 = a.row_ptr[row], p1 = a.row_ptr[row + 1];
        for (int64_t p = p0 + tid; p < p1; p += nthr) xs[a.cols[p]] = 0.f;
        __syncthreads();
    }
    if (a.inexact_rows) {
        int top = -100000, ulp = 100000;
        for (int j = tid; j < N; j += nthr) {
            uint32_t u = __float_as_uint(xs[j]) & 0x7fffffffu;
            if (u) {
                int e = (int)(u >> 23);
                uint32_t m = u & 0x7fffffu;
                int t, q;
                if (e) { t = e - 127; q = e - 150 + (__ffs(m | 0x800000u) - 1); }
                else   { t = (31 - __clz(m)) - 149; q = (__ffs(m) - 1) - 149; }
                top = max(top, t);
                ulp = min(ulp, q);
            }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            top = max(top, __shfl_xor_sync(0xffffffffu, top, o));
            ulp = min(ulp, __shfl_xor_sync(0xffffffffu, ulp, o));
        }
        if (lane == 0) { atomicMax(&sh.max_top, top); atomicMin(&sh.min_ulp, ulp); }
        __syncthreads();
        if (tid == 0 && sh.max_top > -100000) {
            // sums and differences of up to 2N weights stay exact in fp64 while
            // 2 N 2^(top+1) / 2^ulp <= 2^53
            int log2n = 32 - __clz(N - 1 > 0 ? N - 1 : 1);
            if (log2n + 1 + (sh.max_top + 1 - sh.min_ulp) > 53) atomicAdd(a.inexact_rows, 1);
        }
    }
    const int bits = a.bits[row];
    if (bits == 2) fit_channel<DT, 4>(a, row, xs, code, sh);
    else if (bits == 3) fit_channel<DT, 8>(a, row, xs, code, sh);
    else fit_channel<DT, 16>(a, row, xs, code, sh);
}

static size_t lloyd_smem_bytes(int64_t d_out) {
    size_t npad = ((size_t)d_out + 15) & ~(size_t)15;
    return sizeof(LloydShared) + npad * 5;
}

static int lloyd_threads(int64_t d_out) {
    int64_t t = (d_out + 15) / 16;
    t = (t + 31) / 32 * 32;
    if (t < 64) t = 64;
    if (t > 1024) t = 1024;
    return (int)t;
}

cmpq_status launch_lloyd(const LloydArgs& args, cmpq_dtype dt, cudaStream_t st) {
    const size_t smem = lloyd_smem_bytes(args.d_out);
    auto kern = dt == CMPQ_F16 ? lloyd_kernel<CMPQ_F16> : lloyd_kernel<CMPQ_BF16>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
        return CMPQ_ERR_CUDA;
    kern<<<(unsigned)args.d_in, lloyd_threads(args.d_out), smem, st>>>(args);
    return launch_status();
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
