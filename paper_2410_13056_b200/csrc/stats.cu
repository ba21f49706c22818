// Activation statistic of CMPQ (Section 3.2.1): per input channel j the sum over the
// calibration tokens of X[t,j]^2, whose square root is the channel's L2 norm a_j.
//
// HBM-bound column reduction.  A warp reads 512 contiguous bytes of a row with one 128-bit
// load per lane (8 adjacent columns per thread), eight warps of a block take eight rows at a
// time, four rows are in flight per thread.  Squares are exact in fp32; a thread keeps fp32
// partial sums for at most kFlushRows of its rows and folds them into fp64.  The blocks of
// one column tile write fp64 partials to the work space; a second kernel adds them in a fixed
// order, so the result does not depend on scheduling.
#include "common.cuh"

#include <atomic>

namespace cmpq {

constexpr int kStatsThreads = 256;
constexpr int kStatsWarps = kStatsThreads / 32;
constexpr int kTileCols = 256;       // columns per block: 32 lanes x 8 columns
constexpr int kFlushRows = 32;       // rows a thread sums in fp32 before folding into fp64
constexpr int kMaxRowBlocks = 2048;  // upper bound used to size the work space
constexpr int kCtasPerSm = 5;       // resident blocks per SM of the vector kernel (48 registers)

int sm_count() {
    constexpr int kMaxDevices = 64;
    static std::atomic<int> cached[kMaxDevices];  // zero-initialised: 0 = not asked yet
    int dev = 0, n = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 0;
    const bool slot = dev >= 0 && dev < kMaxDevices;
    if (slot && (n = cached[dev].load(std::memory_order_relaxed)) > 0) return n;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 0;
    if (slot) cached[dev].store(n, std::memory_order_relaxed);
    return n;
}

static int64_t col_tiles(int64_t d_in) { return (d_in + kTileCols - 1) / kTileCols; }

// Row blocks per column tile for a device with `sms` SMs: as many blocks as are resident at once
// (one full wave, no tail), never more than kMaxRowBlocks / col_tiles (work-space bound).
static int64_t row_blocks_for(int64_t d_in, int64_t n_tokens, int sms) {
    int64_t ct = col_tiles(d_in);
    int64_t want = ((int64_t)sms * kCtasPerSm) / ct;
    int64_t cap = kMaxRowBlocks / ct;
    if (cap < 1) cap = 1;
    if (want > cap) want = cap;
    int64_t by_rows = (n_tokens + kStatsWarps - 1) / kStatsWarps;  // at least one row per warp
    if (want > by_rows) want = by_rows;
    if (want < 1) want = 1;
    return want;
}

size_t stats_ws_bytes(int64_t d_in) {
    int64_t ct = col_tiles(d_in);
    int64_t rb = kMaxRowBlocks / ct;
    if (rb < 1) rb = 1;
    return round_up((size_t)rb * (size_t)ct * kTileCols * sizeof(double), 256);
}

// One activation folded into a running fp32 value: x^2 added (l2, the paper's default), |x| added (l1) or
// the larger of the two magnitudes (l_inf); the latter two are the criteria of the norm-ablation table.
template <int NORM>
__device__ __forceinline__ float fold(float x, float acc) {
    if (NORM == CMPQ_NORM_L2) return fmaf(x, x, acc);
    if (NORM == CMPQ_NORM_L1) return acc + fabsf(x);
    // the larger magnitude, as bit patterns (for finite values the order is the same): a NaN pattern sorts
    // above every number and so survives to the end, where it is reported
    return __uint_as_float(max(__float_as_uint(acc), __float_as_uint(x) & 0x7fffffffu));
}

// Two partial results combined: a sum, or a maximum for l_inf.
// the larger of two non-negative values, a NaN in either winning
__device__ __forceinline__ double max_keep_nan(double a, double b) { return (a != a) ? a : ((b != b || b > a) ? b : a); }

template <int NORM>
__device__ __forceinline__ double join(double a, double b) {
    return NORM == CMPQ_NORM_LINF ? max_keep_nan(a, b) : a + b;
}

template <int DT, int NORM>
__device__ __forceinline__ void accumulate8(const uint4& v, float (&acc)[8]) {
    float2 p0 = widen16x2<DT>(v.x), p1 = widen16x2<DT>(v.y);
    float2 p2 = widen16x2<DT>(v.z), p3 = widen16x2<DT>(v.w);
    acc[0] = fold<NORM>(p0.x, acc[0]);
    acc[1] = fold<NORM>(p0.y, acc[1]);
    acc[2] = fold<NORM>(p1.x, acc[2]);
    acc[3] = fold<NORM>(p1.y, acc[3]);
    acc[4] = fold<NORM>(p2.x, acc[4]);
    acc[5] = fold<NORM>(p2.y, acc[5]);
    acc[6] = fold<NORM>(p3.x, acc[6]);
    acc[7] = fold<NORM>(p3.y, acc[7]);
}

// partial[(row_block * tiles + tile) * kTileCols + c] = sum over the block's rows of X[t, tile*256+c]^2
// The fp64 running totals live in shared memory (slot [warp][i][lane] for column lane*8+i: conflict
// free), which keeps the register count low enough for 5 resident blocks per SM.
template <int DT, int NORM>
__global__ void __launch_bounds__(kStatsThreads, 5)
stats_partial_vec_kernel(const uint16_t* __restrict__ X, int64_t n_tokens, int64_t d_in, int64_t ldx,
                         int64_t rows_per_block, double* __restrict__ partial) {
    __shared__ double red[kStatsWarps][8][32];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t tile = blockIdx.x;
    const int64_t col = tile * kTileCols + lane * 8;
    const int64_t r0 = (int64_t)blockIdx.y * rows_per_block;
    int64_t r1 = r0 + rows_per_block;
    if (r1 > n_tokens) r1 = n_tokens;
#pragma unroll
    for (int i = 0; i < 8; ++i) red[warp][i][lane] = 0.0;

    if (col < d_in) {
        const uint16_t* p = X + col;
        float acc[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) acc[i] = 0.f;
        int since_flush = 0;
        int64_t r = r0 + warp;
        for (; r + 3 * kStatsWarps < r1; r += 4 * kStatsWarps) {
            uint4 v0 = __ldcs(reinterpret_cast<const uint4*>(p + r * ldx));
            uint4 v1 = __ldcs(reinterpret_cast<const uint4*>(p + (r + kStatsWarps) * ldx));
            uint4 v2 = __ldcs(reinterpret_cast<const uint4*>(p + (r + 2 * kStatsWarps) * ldx));
            uint4 v3 = __ldcs(reinterpret_cast<const uint4*>(p + (r + 3 * kStatsWarps) * ldx));
            accumulate8<DT, NORM>(v0, acc);
            accumulate8<DT, NORM>(v1, acc);
            accumulate8<DT, NORM>(v2, acc);
            accumulate8<DT, NORM>(v3, acc);
            since_flush += 4;
            if (since_flush >= kFlushRows) {
#pragma unroll
                for (int i = 0; i < 8; ++i) { red[warp][i][lane] = join<NORM>(red[warp][i][lane], (double)acc[i]); acc[i] = 0.f; }
                since_flush = 0;
            }
        }
        for (; r < r1; r += kStatsWarps) {
            uint4 v0 = __ldcs(reinterpret_cast<const uint4*>(p + r * ldx));
            accumulate8<DT, NORM>(v0, acc);
        }
#pragma unroll
        for (int i = 0; i < 8; ++i) red[warp][i][lane] = join<NORM>(red[warp][i][lane], (double)acc[i]);
    }
    __syncthreads();
    // thread c adds the eight warps' sums of column c in warp order
    const int c = threadIdx.x;
    double s = 0.0;
#pragma unroll
    for (int w = 0; w < kStatsWarps; ++w) s = join<NORM>(s, red[w][c & 7][c >> 3]);
    partial[((int64_t)blockIdx.y * gridDim.x + tile) * kTileCols + c] = s;
}

// Same contract for inputs that cannot be read with aligned 128-bit loads: one column per thread.
template <int DT, int NORM>
__global__ void __launch_bounds__(kStatsThreads)
stats_partial_scalar_kernel(const uint16_t* __restrict__ X, int64_t n_tokens, int64_t d_in,
                            int64_t ldx, int64_t rows_per_block, double* __restrict__ partial) {
    const int64_t tile = blockIdx.x;
    const int64_t col = tile * kTileCols + threadIdx.x;
    const int64_t r0 = (int64_t)blockIdx.y * rows_per_block;
    int64_t r1 = r0 + rows_per_block;
    if (r1 > n_tokens) r1 = n_tokens;
    double total = 0.0;
    if (col < d_in) {
        float acc = 0.f;
        int since_flush = 0;
        for (int64_t r = r0; r < r1; ++r) {
            float x = widen16<DT>(X[r * ldx + col]);
            acc = fold<NORM>(x, acc);
            if (++since_flush == kFlushRows) { total = join<NORM>(total, (double)acc); acc = 0.f; since_flush = 0; }
        }
        total = join<NORM>(total, (double)acc);
    }
    partial[((int64_t)blockIdx.y * gridDim.x + tile) * kTileCols + threadIdx.x] = total;
}

// sumsq[j] += sum over the row blocks of partial[rb][j]   (l_inf: the maximum instead of the sum), always in
// the same order: warp p of a block adds the row blocks p, p + 8, p + 16, ... of 32 columns (one per lane), then
// warp 0 adds the eight part sums in ascending p.
// A NaN or an infinity among the activations of a column (or an fp32 square beyond the fp32 range) makes
// the column's partial result non-finite: bit 0 of *nonfinite is set (nonfinite may be NULL).
constexpr int kCombineParts = 8;
__global__ void __launch_bounds__(32 * kCombineParts)
stats_combine_kernel(const double* __restrict__ partial, int64_t row_blocks, int64_t padded_cols, int64_t d_in,
                     double* __restrict__ sumsq, int take_max, int32_t* nonfinite) {
    __shared__ double part_sum[kCombineParts][32];
    const int lane = threadIdx.x & 31, part = threadIdx.x >> 5;
    const int64_t j = (int64_t)blockIdx.x * 32 + lane;
    double s = 0.0;
    if (j < d_in) {
        if (take_max) {
            for (int64_t rb = part; rb < row_blocks; rb += kCombineParts) s = max_keep_nan(s, partial[rb * padded_cols + j]);
        } else {
            for (int64_t rb = part; rb < row_blocks; rb += kCombineParts) s += partial[rb * padded_cols + j];
        }
    }
    part_sum[part][lane] = s;
    __syncthreads();
    if (part != 0 || j >= d_in) return;
    s = part_sum[0][lane];
#pragma unroll
    for (int p = 1; p < kCombineParts; ++p) s = take_max ? max_keep_nan(s, part_sum[p][lane]) : s + part_sum[p][lane];
    sumsq[j] = take_max ? max_keep_nan(sumsq[j], s) : sumsq[j] + s;
    if (nonfinite && !(fabs(s) <= 1.7976931348623157e308)) atomicOr(nonfinite, 1);
}

__global__ void stats_finalize_kernel(const double* __restrict__ sumsq, int64_t d_in,
                                      float* __restrict__ a, int take_root) {
    int64_t j = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (j < d_in) a[j] = (float)(take_root ? sqrt(sumsq[j]) : sumsq[j]);
}

template <int NORM>
static void launch_partial(const uint16_t* Xp, cmpq_dtype dt, bool vec, dim3 grid, int64_t n_tokens, int64_t d_in,
                           int64_t ldx, int64_t rows_per_block, double* partial, cudaStream_t st) {
    if (vec) {
        if (dt == CMPQ_F16)
            stats_partial_vec_kernel<CMPQ_F16, NORM><<<grid, kStatsThreads, 0, st>>>(Xp, n_tokens, d_in, ldx, rows_per_block, partial);
        else
            stats_partial_vec_kernel<CMPQ_BF16, NORM><<<grid, kStatsThreads, 0, st>>>(Xp, n_tokens, d_in, ldx, rows_per_block, partial);
    } else {
        if (dt == CMPQ_F16)
            stats_partial_scalar_kernel<CMPQ_F16, NORM><<<grid, kStatsThreads, 0, st>>>(Xp, n_tokens, d_in, ldx, rows_per_block, partial);
        else
            stats_partial_scalar_kernel<CMPQ_BF16, NORM><<<grid, kStatsThreads, 0, st>>>(Xp, n_tokens, d_in, ldx, rows_per_block, partial);
    }
}

// Launches the two statistic kernels with `partial` as scratch (row_blocks * tiles * 256 doubles).
cmpq_status launch_collect_stats_norm(const void* X, cmpq_dtype dt, int64_t n_tokens, int64_t d_in,
                                      int64_t ldx, cmpq_norm norm, double* sumsq, double* partial,
                                      int64_t row_blocks, cudaStream_t st, int32_t* nonfinite) {
    const int64_t ct = col_tiles(d_in);
    const int64_t rows_per_block = (n_tokens + row_blocks - 1) / row_blocks;
    const bool vec = aligned_to(X, 16) && (ldx % 8 == 0) && (d_in % 8 == 0);
    dim3 grid((unsigned)ct, (unsigned)row_blocks);
    const uint16_t* Xp = static_cast<const uint16_t*>(X);
    if (norm == CMPQ_NORM_L2) launch_partial<CMPQ_NORM_L2>(Xp, dt, vec, grid, n_tokens, d_in, ldx, rows_per_block, partial, st);
    else if (norm == CMPQ_NORM_L1) launch_partial<CMPQ_NORM_L1>(Xp, dt, vec, grid, n_tokens, d_in, ldx, rows_per_block, partial, st);
    else launch_partial<CMPQ_NORM_LINF>(Xp, dt, vec, grid, n_tokens, d_in, ldx, rows_per_block, partial, st);
    stats_combine_kernel<<<(unsigned)((d_in + 31) / 32), 32 * kCombineParts, 0, st>>>(partial, row_blocks, ct * kTileCols, d_in,
                                                                                   sumsq, norm == CMPQ_NORM_LINF, nonfinite);
    return launch_status();
}

cmpq_status launch_collect_stats(const void* X, cmpq_dtype dt, int64_t n_tokens, int64_t d_in,
                                 int64_t ldx, double* sumsq, double* partial, int64_t row_blocks,
                                 cudaStream_t st) {
    return launch_collect_stats_norm(X, dt, n_tokens, d_in, ldx, CMPQ_NORM_L2, sumsq, partial, row_blocks, st, nullptr);
}

const void* stats_kernel_address() {
    return reinterpret_cast<const void*>(&stats_partial_vec_kernel<CMPQ_BF16, CMPQ_NORM_L2>);
}

int64_t stats_row_blocks(int64_t d_in, int64_t n_tokens) {
    int sms = sm_count();
    if (sms <= 0) return 0;
    return row_blocks_for(d_in, n_tokens, sms);
}

}  // namespace cmpq

using namespace cmpq;

extern "C" cmpq_status cmpq_collect_stats_norm(const void* X, cmpq_dtype dt, int64_t n_tokens, int64_t d_in,
                                               int64_t ldx, cmpq_norm norm, double* acc, int32_t* nonfinite, void* ws,
                                               size_t ws_bytes, void* stream) {
    if (!acc || n_tokens < 0 || d_in < 1 || d_in > CMPQ_MAX_D_IN || ldx < d_in) return CMPQ_ERR_INVALID_ARG;
    if (dt != CMPQ_F16 && dt != CMPQ_BF16) return CMPQ_ERR_INVALID_ARG;
    if (norm != CMPQ_NORM_L2 && norm != CMPQ_NORM_L1 && norm != CMPQ_NORM_LINF) return CMPQ_ERR_INVALID_ARG;
    if (n_tokens > 0 && !X) return CMPQ_ERR_INVALID_ARG;
    if (!aligned_to(X, 2) || !aligned_to(acc, 8) || !aligned_to(nonfinite, 4)) return CMPQ_ERR_INVALID_ARG;
    if (!ws || !aligned_to(ws, 256) || ws_bytes < stats_ws_bytes(d_in)) return CMPQ_ERR_WORKSPACE;
    if (n_tokens == 0) return CMPQ_OK;
    int64_t rb = stats_row_blocks(d_in, n_tokens);
    if (rb <= 0) return CMPQ_ERR_CUDA;
    return launch_collect_stats_norm(X, dt, n_tokens, d_in, ldx, norm, acc, static_cast<double*>(ws), rb,
                                     static_cast<cudaStream_t>(stream), nonfinite);
}

extern "C" cmpq_status cmpq_collect_stats(const void* X, cmpq_dtype dt, int64_t n_tokens, int64_t d_in,
                                          int64_t ldx, double* sumsq, int32_t* nonfinite, void* ws, size_t ws_bytes,
                                          void* stream) {
    return cmpq_collect_stats_norm(X, dt, n_tokens, d_in, ldx, CMPQ_NORM_L2, sumsq, nonfinite, ws, ws_bytes, stream);
}

extern "C" cmpq_status cmpq_check_finite(const int32_t* nonfinite, void* stream) {
    if (!nonfinite) return CMPQ_ERR_INVALID_ARG;
    int32_t word = 0;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (cudaMemcpyAsync(&word, nonfinite, sizeof(word), cudaMemcpyDeviceToHost, st) != cudaSuccess) return CMPQ_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return CMPQ_ERR_CUDA;
    return word ? CMPQ_ERR_NONFINITE : CMPQ_OK;
}

extern "C" cmpq_status cmpq_finalize_stats_norm(const double* acc, int64_t d_in, cmpq_norm norm, float* a,
                                                void* stream) {
    if (!acc || !a || d_in < 1 || d_in > CMPQ_MAX_D_IN) return CMPQ_ERR_INVALID_ARG;
    if (norm != CMPQ_NORM_L2 && norm != CMPQ_NORM_L1 && norm != CMPQ_NORM_LINF) return CMPQ_ERR_INVALID_ARG;
    stats_finalize_kernel<<<(unsigned)((d_in + 255) / 256), 256, 0, static_cast<cudaStream_t>(stream)>>>(
        acc, d_in, a, norm == CMPQ_NORM_L2);
    return launch_status();
}

extern "C" cmpq_status cmpq_finalize_stats(const double* sumsq, int64_t d_in, float* a, void* stream) {
    return cmpq_finalize_stats_norm(sumsq, d_in, CMPQ_NORM_L2, a, stream);
}
