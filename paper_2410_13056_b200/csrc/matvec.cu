// Inference product of one token with a quantized layer (Section 6 of the paper: the input is split by
// the precision of its channels, each part multiplies its 2-, 3- or 4-bit sub-matrix through the
// channel's look-up table, the 16-bit outliers multiply the original input, everything is accumulated):
//     y_j = sum_i x_i * lut_i[code_ij]  +  sum_{(i,j,v) in O} x_i * v .
// The packed layout stores a channel's codes contiguously, so a thread owns 32 output columns and walks
// over channels; what has to come from HBM is the packed code stream (b/8 bytes per weight), once.
#include "common.cuh"

#include <cuda_bf16.h>

namespace cmpq {

constexpr int kMvThreads = 256;                       // 8 warps
constexpr int kMvWarps = kMvThreads / 32;
constexpr int kMvRowsPerWarp = 8;                     // channels a warp keeps in flight
constexpr int kMvRowsPerPass = kMvWarps * kMvRowsPerWarp;
constexpr int kMvCols = 1024;                         // output columns per block: 32 lanes x 32 columns
constexpr int kMvPad = kMvCols + 32;                  // one pad float per 32 columns: conflict-free both ways

// Channels per block (a multiple of kMvRowsPerPass), chosen so that large layers still fill the GPU a few
// times over while their partial sums stay small beside the code stream.
static int matvec_rows_per_block(int64_t d_in, int64_t d_out) {
    const int64_t tiles = (d_out + kMvCols - 1) / kMvCols;
    const int64_t blocks = tiles * ((d_in + kMvRowsPerPass - 1) / kMvRowsPerPass + 2);
    int64_t m = blocks / 592;
    if (m < 1) m = 1;
    if (m > 8) m = 8;
    return (int)(m * kMvRowsPerPass);
}

static int64_t matvec_max_chunks(int64_t d_in, int rows_per_block) {
    return (d_in + rows_per_block - 1) / rows_per_block + 2;  // three segments: at most two extra ragged chunks
}

size_t matvec_ws_bytes(int64_t d_in, int64_t d_out) {
    return round_up((size_t)matvec_max_chunks(d_in, matvec_rows_per_block(d_in, d_out)) * (size_t)d_out * sizeof(float), 256);
}

size_t by_column_ws_bytes(int64_t d_out) { return round_up((size_t)(d_out + 1) * sizeof(int), 256); }

// Chunk `slot` of the layer: which segment (bit width) it belongs to and which stored rows it covers.
// Chunks never straddle a segment, so the bit width is uniform in a block.
struct MvChunk {
    int c;          // bits per code, 0 = no such chunk
    int64_t r0, r1; // stored rows [r0, r1)
};

__device__ __forceinline__ MvChunk matvec_chunk(const int64_t* __restrict__ seg_rows, int64_t slot, int rb) {
    MvChunk ch;
    ch.c = 0;
    ch.r0 = ch.r1 = 0;
    int64_t first = 0;
#pragma unroll
    for (int s = 0; s < 3; ++s) {
        const int64_t n = seg_rows[s];
        const int64_t chunks = (n + rb - 1) / rb;
        if (ch.c == 0 && slot < chunks) {
            ch.c = s + 2;
            ch.r0 = first + slot * rb;
            ch.r1 = min(first + n, ch.r0 + rb);
        }
        slot -= chunks;
        first += n;
    }
    return ch;
}

__device__ __forceinline__ int64_t matvec_total_chunks(const int64_t* __restrict__ seg_rows, int rb) {
    return (seg_rows[0] + rb - 1) / rb + (seg_rows[1] + rb - 1) / rb + (seg_rows[2] + rb - 1) / rb;
}

// Code t (0..31) of a group of 32 codes held LSB-first in C words, as a byte offset into a float table.
template <int C, int T>
__device__ __forceinline__ uint32_t code_offset(const uint32_t (&w)[C]) {
    constexpr int pos = C * T, word = pos / 32, sh = pos % 32;
    uint32_t v;
    if (sh + C <= 32) v = w[word] >> sh;
    else v = __funnelshift_r(w[word], w[(word + 1 < C) ? word + 1 : word], sh);
    return (v & ((1u << C) - 1u)) << 2;
}

template <int C, int T>
struct MvAccumulate {
    static __device__ __forceinline__ void run(const uint32_t (&w)[C], const char* table, float (&acc)[32]) {
        acc[T] += *reinterpret_cast<const float*>(table + code_offset<C, T>(w));
        MvAccumulate<C, T + 1>::run(w, table, acc);
    }
};
template <int C>
struct MvAccumulate<C, 32> {
    static __device__ __forceinline__ void run(const uint32_t (&)[C], const char*, float (&)[32]) {}
};

// The C words of one group of 32 codes; words at or beyond `valid` read as 0.
template <int C>
__device__ __forceinline__ void load_group(const uint32_t* __restrict__ p, int valid, bool vec, uint32_t (&w)[C]) {
    if (C == 2 && vec && valid >= 2) {
        const uint2 v = __ldcs(reinterpret_cast<const uint2*>(p));
        w[0] = v.x;
        w[1] = v.y;
    } else if (C == 4 && vec && valid >= 4) {
        const uint4 v = __ldcs(reinterpret_cast<const uint4*>(p));
        w[0] = v.x;
        w[1] = v.y;
        w[2] = v.z;
        w[3] = v.w;
    } else {
#pragma unroll
        for (int t = 0; t < C; ++t) w[t] = (t < valid) ? __ldcs(p + t) : 0u;
    }
}

// One warp, up to kMvRowsPerWarp stored rows [r, r_end): every lane adds its 32 columns.
template <int C, int DT>
__device__ __forceinline__ void matvec_rows(const uint32_t* __restrict__ packed, const int64_t* __restrict__ row_off,
                                            const int32_t* __restrict__ perm, const float* __restrict__ lut,
                                            const uint16_t* __restrict__ x, int64_t r, int64_t r_end, int64_t group,
                                            int valid_words, bool base_vec, float* table /* [rows][16] of this warp */,
                                            float (&acc)[32]) {
    const int lane = threadIdx.x & 31;
    // table[q][k] = x_i * lut_i[k] for the rows of this pass: one multiplication per table entry instead
    // of one per weight
#pragma unroll
    for (int q = 0; q < kMvRowsPerWarp / 2; ++q) {
        const int rr = 2 * q + (lane >> 4);
        float v = 0.0f;
        if (r + rr < r_end) {
            const int32_t i = perm[r + rr];
            v = widen16<DT>(x[i]) * lut[(int64_t)i * CMPQ_LUT_STRIDE + (lane & 15)];
        }
        table[rr * 16 + (lane & 15)] = v;
    }
    uint32_t w[kMvRowsPerWarp][C];
#pragma unroll
    for (int q = 0; q < kMvRowsPerWarp; ++q) {
        if (r + q < r_end && valid_words > 0) {
            const int64_t off = row_off[r + q] + group * C;
            const bool vec = base_vec && (C == 2 ? (off & 1) == 0 : (off & 3) == 0);
            load_group<C>(packed + off, valid_words, vec, w[q]);
        } else {
#pragma unroll
            for (int t = 0; t < C; ++t) w[q][t] = 0u;
        }
    }
    __syncwarp();
#pragma unroll
    for (int q = 0; q < kMvRowsPerWarp; ++q)
        MvAccumulate<C, 0>::run(w[q], reinterpret_cast<const char*>(table + q * 16), acc);
    __syncwarp();
}

// partial[slot][j] = sum over the chunk's channels of x_i * lut_i[code_ij].
template <int DT>
__global__ void __launch_bounds__(kMvThreads)
matvec_partial_kernel(const uint32_t* __restrict__ packed, const int64_t* __restrict__ row_off,
                      const int32_t* __restrict__ perm, const int64_t* __restrict__ seg_rows,
                      const float* __restrict__ lut, const uint16_t* __restrict__ x, int64_t d_out,
                      int rows_per_block, int base_align, float* __restrict__ partial) {
    __shared__ float tables[kMvWarps][kMvRowsPerWarp * 16];
    __shared__ float red[kMvWarps][kMvPad];
    const MvChunk ch = matvec_chunk(seg_rows, blockIdx.y, rows_per_block);
    if (ch.c == 0) return;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t group = (int64_t)blockIdx.x * 32 + lane;  // group of 32 columns
    const int64_t words_per_row = (d_out * ch.c + 31) / 32;
    const int64_t left = words_per_row - group * ch.c;
    const int valid_words = (int)max((int64_t)0, min((int64_t)ch.c, left));
    float acc[32];
#pragma unroll
    for (int t = 0; t < 32; ++t) acc[t] = 0.0f;
    for (int64_t r = ch.r0 + warp * kMvRowsPerWarp; r < ch.r1; r += kMvRowsPerPass) {
        if (ch.c == 2)
            matvec_rows<2, DT>(packed, row_off, perm, lut, x, r, ch.r1, group, valid_words, base_align >= 8,
                               tables[warp], acc);
        else if (ch.c == 3)
            matvec_rows<3, DT>(packed, row_off, perm, lut, x, r, ch.r1, group, valid_words, false, tables[warp], acc);
        else
            matvec_rows<4, DT>(packed, row_off, perm, lut, x, r, ch.r1, group, valid_words, base_align >= 16,
                               tables[warp], acc);
    }
    // warps are summed in a fixed order; the staging is laid out so that both sides are conflict free
#pragma unroll
    for (int t = 0; t < 32; ++t) red[warp][lane * 33 + t] = acc[t];
    __syncthreads();
    float* out = partial + (int64_t)blockIdx.y * d_out + (int64_t)blockIdx.x * kMvCols;
    const int64_t cols_here = min((int64_t)kMvCols, d_out - (int64_t)blockIdx.x * kMvCols);
    for (int col = threadIdx.x; col < cols_here; col += kMvThreads) {
        float s = 0.0f;
#pragma unroll
        for (int wq = 0; wq < kMvWarps; ++wq) s += red[wq][col + (col >> 5)];
        out[col] = s;
    }
}

template <int DT>
__device__ __forceinline__ uint16_t narrow16(float v) {
    if (DT == CMPQ_BF16) return __bfloat16_as_ushort(__float2bfloat16_rn(v));
    return __half_as_ushort(__float2half_rn(v));
}

// y_j = (sum of the chunk partials, in chunk order) + (the column's outlier products, in row order).
// 32 columns per block; the 8 warps take every 8th chunk / every 8th outlier and are combined in order.
template <int DT>
__global__ void __launch_bounds__(kMvThreads)
matvec_finish_kernel(const float* __restrict__ partial, const int64_t* __restrict__ seg_rows, int rows_per_block,
                     int64_t d_out, const uint16_t* __restrict__ x, const int64_t* __restrict__ col_ptr,
                     const int32_t* __restrict__ c_rows, const uint16_t* __restrict__ c_vals,
                     float* __restrict__ y, uint16_t* __restrict__ y16) {
    __shared__ float part[kMvWarps][32];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t j = (int64_t)blockIdx.x * 32 + lane;
    const int64_t chunks = matvec_total_chunks(seg_rows, rows_per_block);
    float s = 0.0f;
    if (j < d_out) {
        for (int64_t q = warp; q < chunks; q += kMvWarps) s += partial[q * d_out + j];
        if (col_ptr != nullptr) {
            float so = 0.0f;
            const int64_t e1 = col_ptr[j + 1];
            for (int64_t e = col_ptr[j] + warp; e < e1; e += kMvWarps)
                so += widen16<DT>(x[c_rows[e]]) * widen16<DT>(c_vals[e]);
            s += so;
        }
    }
    part[warp][lane] = s;
    __syncthreads();
    if (warp == 0 && j < d_out) {
        float t = 0.0f;
#pragma unroll
        for (int wq = 0; wq < kMvWarps; ++wq) t += part[wq][lane];
        y[j] = t;
        if (y16 != nullptr) y16[j] = narrow16<DT>(t);
    }
}

// ---- outlier list regrouped by column -----------------------------------------------------------------
__global__ void column_count_kernel(const int32_t* __restrict__ cols, int64_t nnz, int* __restrict__ count) {
    const int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (e < nnz) atomicAdd(&count[cols[e]], 1);
}

// One block: col_ptr = exclusive prefix sums of count; count is cleared for its second use as a cursor.
__global__ void __launch_bounds__(1024)
column_scan_kernel(int* __restrict__ count, int64_t d_out, int64_t* __restrict__ col_ptr) {
    __shared__ int64_t warp_sum[32];
    __shared__ int64_t carry;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (threadIdx.x == 0) carry = 0;
    __syncthreads();
    for (int64_t base = 0; base < d_out; base += 1024) {
        const int64_t j = base + threadIdx.x;
        const int64_t v = j < d_out ? count[j] : 0;
        int64_t inc = v;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const int64_t o = __shfl_up_sync(0xffffffffu, inc, d);
            if (lane >= d) inc += o;
        }
        if (lane == 31) warp_sum[warp] = inc;
        __syncthreads();
        if (warp == 0) {
            const int64_t ws = warp_sum[lane];
            int64_t winc = ws;
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                const int64_t o = __shfl_up_sync(0xffffffffu, winc, d);
                if (lane >= d) winc += o;
            }
            warp_sum[lane] = winc - ws;  // exclusive over warps
        }
        __syncthreads();
        const int64_t excl = carry + warp_sum[warp] + inc - v;
        if (j < d_out) {
            col_ptr[j] = excl;
            count[j] = 0;
        }
        __syncthreads();
        if (threadIdx.x == 1023) carry = excl + v;
        __syncthreads();
    }
    if (threadIdx.x == 0) col_ptr[d_out] = carry;
}

__global__ void column_scatter_kernel(const int32_t* __restrict__ rows, const int32_t* __restrict__ cols,
                                      const uint16_t* __restrict__ vals, int64_t nnz,
                                      const int64_t* __restrict__ col_ptr, int* __restrict__ cursor,
                                      int32_t* __restrict__ c_rows, uint16_t* __restrict__ c_vals) {
    const int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (e >= nnz) return;
    const int32_t c = cols[e];
    const int64_t pos = col_ptr[c] + atomicAdd(&cursor[c], 1);
    c_rows[pos] = rows[e];
    c_vals[pos] = vals[e];
}

constexpr int kColSortCap = 2048;  // entries of one column ordered in shared memory

// One warp per column: the scatter left the column's entries in arbitrary order; put them in ascending
// row order (rows are distinct inside a column, so the rank of an entry is the number of smaller rows).
__global__ void __launch_bounds__(32)
column_sort_kernel(const int64_t* __restrict__ col_ptr, int32_t* __restrict__ c_rows, uint16_t* __restrict__ c_vals) {
    __shared__ int32_t srow[kColSortCap];
    __shared__ uint16_t sval[kColSortCap];
    const int lane = threadIdx.x;
    const int64_t b = col_ptr[blockIdx.x], e = col_ptr[blockIdx.x + 1];
    const int64_t n = e - b;
    if (n <= 1) return;
    if (n <= kColSortCap) {
        for (int64_t t = lane; t < n; t += 32) {
            srow[t] = c_rows[b + t];
            sval[t] = c_vals[b + t];
        }
        __syncwarp();
        for (int64_t t = lane; t < n; t += 32) {
            const int32_t r = srow[t];
            int rank = 0;
            for (int64_t u = 0; u < n; ++u) rank += srow[u] < r;
            c_rows[b + rank] = r;
            c_vals[b + rank] = sval[t];
        }
    } else if (lane == 0) {  // a column with thousands of outliers: plain insertion in place
        for (int64_t t = b + 1; t < e; ++t) {
            const int32_t r = c_rows[t];
            const uint16_t v = c_vals[t];
            int64_t u = t;
            while (u > b && c_rows[u - 1] > r) {
                c_rows[u] = c_rows[u - 1];
                c_vals[u] = c_vals[u - 1];
                --u;
            }
            c_rows[u] = r;
            c_vals[u] = v;
        }
    }
}

}  // namespace cmpq

using namespace cmpq;

extern "C" cmpq_status cmpq_outliers_by_column(const int32_t* rows, const int32_t* cols, const uint16_t* vals,
                                               int64_t nnz, int64_t d_out, int64_t* col_ptr, int32_t* c_rows,
                                               uint16_t* c_vals, void* ws, size_t ws_bytes, void* stream) {
    if (nnz < 0 || d_out < 1 || d_out > CMPQ_MAX_D_OUT || !col_ptr) return CMPQ_ERR_INVALID_ARG;
    if (nnz > 0 && (!rows || !cols || !vals || !c_rows || !c_vals)) return CMPQ_ERR_INVALID_ARG;
    if (nnz > (int64_t)CMPQ_MAX_D_IN * CMPQ_MAX_D_OUT) return CMPQ_ERR_INVALID_ARG;
    if (!aligned_to(col_ptr, 8)) return CMPQ_ERR_INVALID_ARG;
    if (!ws || !aligned_to(ws, 256) || ws_bytes < by_column_ws_bytes(d_out)) return CMPQ_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int* count = static_cast<int*>(ws);
    if (cudaMemsetAsync(count, 0, (size_t)(d_out + 1) * sizeof(int), st) != cudaSuccess) return CMPQ_ERR_CUDA;
    const unsigned blocks = (unsigned)((nnz + 255) / 256);
    if (nnz > 0) column_count_kernel<<<blocks, 256, 0, st>>>(cols, nnz, count);
    column_scan_kernel<<<1, 1024, 0, st>>>(count, d_out, col_ptr);
    if (nnz > 0) {
        column_scatter_kernel<<<blocks, 256, 0, st>>>(rows, cols, vals, nnz, col_ptr, count, c_rows, c_vals);
        column_sort_kernel<<<(unsigned)d_out, 32, 0, st>>>(col_ptr, c_rows, c_vals);
    }
    return launch_status();
}

extern "C" cmpq_status cmpq_matvec(const uint32_t* packed, const int64_t* row_off, const int32_t* perm,
                                   const int64_t* seg_rows, const float* lut, int64_t d_in, int64_t d_out,
                                   const void* x, cmpq_dtype dt, const int64_t* col_ptr, const int32_t* c_rows,
                                   const uint16_t* c_vals, float* y, void* y16, void* ws, size_t ws_bytes,
                                   void* stream) {
    if (!packed || !row_off || !perm || !seg_rows || !lut || !x || !y) return CMPQ_ERR_INVALID_ARG;
    if (d_in < 1 || d_in > CMPQ_MAX_D_IN || d_out < 1 || d_out > CMPQ_MAX_D_OUT) return CMPQ_ERR_INVALID_ARG;
    if (dt != CMPQ_F16 && dt != CMPQ_BF16) return CMPQ_ERR_INVALID_ARG;
    if (col_ptr && (!c_rows || !c_vals)) return CMPQ_ERR_INVALID_ARG;
    if (!aligned_to(packed, 4) || !aligned_to(row_off, 8) || !aligned_to(seg_rows, 8) || !aligned_to(lut, 4) ||
        !aligned_to(x, 2) || !aligned_to(y, 4) || (y16 && !aligned_to(y16, 2)) || (col_ptr && !aligned_to(col_ptr, 8)))
        return CMPQ_ERR_INVALID_ARG;
    if (!ws || !aligned_to(ws, 256) || ws_bytes < matvec_ws_bytes(d_in, d_out)) return CMPQ_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int rb = matvec_rows_per_block(d_in, d_out);
    float* partial = static_cast<float*>(ws);
    const int base_align = aligned_to(packed, 16) ? 16 : (aligned_to(packed, 8) ? 8 : 4);
    dim3 grid((unsigned)((d_out + kMvCols - 1) / kMvCols), (unsigned)matvec_max_chunks(d_in, rb));
    const unsigned fin_blocks = (unsigned)((d_out + 31) / 32);
    const uint16_t* xu = static_cast<const uint16_t*>(x);
    uint16_t* yu = static_cast<uint16_t*>(y16);
    if (dt == CMPQ_BF16) {
        matvec_partial_kernel<CMPQ_BF16><<<grid, kMvThreads, 0, st>>>(packed, row_off, perm, seg_rows, lut, xu, d_out,
                                                                      rb, base_align, partial);
        matvec_finish_kernel<CMPQ_BF16><<<fin_blocks, kMvThreads, 0, st>>>(partial, seg_rows, rb, d_out, xu, col_ptr,
                                                                           c_rows, c_vals, y, yu);
    } else {
        matvec_partial_kernel<CMPQ_F16><<<grid, kMvThreads, 0, st>>>(packed, row_off, perm, seg_rows, lut, xu, d_out,
                                                                     rb, base_align, partial);
        matvec_finish_kernel<CMPQ_F16><<<fin_blocks, kMvThreads, 0, st>>>(partial, seg_rows, rb, d_out, xu, col_ptr,
                                                                          c_rows, c_vals, y, yu);
    }
    return launch_status();
}
