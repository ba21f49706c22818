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
#ifndef CMPQ_MV_MIN_BLOCKS
#define CMPQ_MV_MIN_BLOCKS 2                          // resident blocks per SM the partial kernel is compiled for
#endif

// Channels per block: a multiple m <= 8 of kMvRowsPerPass, grown with the layer.  Measured on B200 the time
// hardly depends on m once there are a few blocks per SM (67 to 75 us for m = 2..12 at 8192 x 28672), single
// passes lose 20 % there (nothing to overlap the first loads with) and small layers want m = 1 or 2 to spread
// over every SM: aim at two to four resident rounds.
static int matvec_rows_per_block(int64_t d_in, int64_t d_out) {
    const int64_t tiles = (d_out + kMvCols - 1) / kMvCols;
    const int64_t blocks = tiles * ((d_in + kMvRowsPerPass - 1) / kMvRowsPerPass + 2);
    const int sms = sm_count();
    int64_t m = blocks / (4 * (int64_t)(sms > 0 ? sms : 148));
    if (m < 1) m = 1;
    if (m > 8) m = 8;
    return (int)(m * kMvRowsPerPass);
}

static int64_t matvec_max_chunks(int64_t d_in, int rows_per_block) {
    return (d_in + rows_per_block - 1) / rows_per_block + 2;  // three segments: at most two extra ragged chunks
}

// Sized for the smallest block (the most chunks), so the size does not depend on the device.
size_t matvec_ws_bytes(int64_t d_in, int64_t d_out) {
    return round_up((size_t)matvec_max_chunks(d_in, kMvRowsPerPass) * (size_t)d_out * sizeof(float), 256);
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

// ---- two channels per look-up ------------------------------------------------------------------------
// Two channels a, b of the same width C share one table of 2^(2C) sums  T[cb << C | ca] = t_a[ca] + t_b[cb]
// (t_i[k] = x_i * lut_i[k]), so one shared-memory load and one addition serve two weights.  The index
// streams are formed 32 columns at a time with word-wide logic: with M = the bits of every even-numbered
// code,  U = (wa & M) | ((wb & M) << C)  holds the 2C-bit indices of the even columns back to back, and
// V = ((wa & ~M) >> C) | (wb & ~M)  those of the odd columns (shifts run across the C words of the group).

// Mask word `word` of the even-numbered codes of width C: bit i of the stream is set iff (i mod 2C) < C.
template <int C>
__host__ __device__ constexpr uint32_t even_code_mask(int word) {
    uint32_t m = 0;
    for (int j = 0; j < 32; ++j)
        if (((word * 32 + j) % (2 * C)) < C) m |= 1u << j;
    return m;
}

template <int C>
__device__ __forceinline__ void pair_streams(const uint32_t (&wa)[C], const uint32_t (&wb)[C], uint32_t (&U)[C],
                                             uint32_t (&V)[C]) {
    uint32_t be[C], ao[C];
#pragma unroll
    for (int k = 0; k < C; ++k) {
        be[k] = wb[k] & even_code_mask<C>(k);
        ao[k] = wa[k] & ~even_code_mask<C>(k);
    }
#pragma unroll
    for (int k = 0; k < C; ++k) {
        const uint32_t up = (be[k] << C) | (k > 0 ? be[k > 0 ? k - 1 : 0] >> (32 - C) : 0u);
        const uint32_t down = (ao[k] >> C) | (k + 1 < C ? ao[k + 1 < C ? k + 1 : k] << (32 - C) : 0u);
        U[k] = (wa[k] & even_code_mask<C>(k)) | up;
        V[k] = down | (wb[k] & ~even_code_mask<C>(k));
    }
}

// Shared-memory address of table entry number S, an F-bit field at bit F*S of a stream of C words: the
// field is moved straight to bits [2, 2+F) (a byte offset into floats) and OR-ed into the table's address,
// which is aligned to the table's size, so one shift and one three-input logic operation produce the address.
template <int C, int F, int S>
__device__ __forceinline__ uint32_t entry_address(const uint32_t (&st)[C], uint32_t table_addr) {
    constexpr int pos = F * S, word = pos / 32, sh = pos % 32;
    constexpr uint32_t mask = ((1u << F) - 1u) << 2;
    uint32_t v;
    if constexpr (sh + F > 32) v = __funnelshift_r(st[word], st[(word + 1 < C) ? word + 1 : word], sh - 2);
    else if constexpr (sh >= 2) v = st[word] >> (sh - 2);
    else v = st[word] << (2 - sh);
    return (v & mask) | table_addr;
}

template <int BYTE_OFFSET>
__device__ __forceinline__ float load_shared_float(uint32_t addr) {
    float v;
    asm volatile("ld.shared.f32 %0, [%1+%2];" : "=f"(v) : "r"(addr), "n"(BYTE_OFFSET) : "memory");
    return v;
}

// acc[2s] += T_P[U_s], acc[2s+1] += T_P[V_s] for the 16 even and 16 odd columns of the group.
template <int C, int P, int S>
struct MvAccumulate {
    static __device__ __forceinline__ void run(const uint32_t (&U)[C], const uint32_t (&V)[C], uint32_t table_addr,
                                               float (&acc)[32]) {
        constexpr int table_bytes = 4 << (2 * C);
        acc[2 * S] += load_shared_float<P * table_bytes>(entry_address<C, 2 * C, S>(U, table_addr));
        acc[2 * S + 1] += load_shared_float<P * table_bytes>(entry_address<C, 2 * C, S>(V, table_addr));
        MvAccumulate<C, P, S + 1>::run(U, V, table_addr, acc);
    }
};
template <int C, int P>
struct MvAccumulate<C, P, 16> {
    static __device__ __forceinline__ void run(const uint32_t (&)[C], const uint32_t (&)[C], uint32_t, float (&)[32]) {}
};

template <int C, int P>
struct MvPairs {
    static __device__ __forceinline__ void run(const uint32_t (&w)[kMvRowsPerWarp][C], uint32_t table_addr,
                                               float (&acc)[32]) {
        uint32_t U[C], V[C];
        pair_streams<C>(w[2 * P], w[2 * P + 1], U, V);
        MvAccumulate<C, P, 0>::run(U, V, table_addr, acc);
        MvPairs<C, P + 1>::run(w, table_addr, acc);
    }
};
template <int C>
struct MvPairs<C, kMvRowsPerWarp / 2> {
    static __device__ __forceinline__ void run(const uint32_t (&)[kMvRowsPerWarp][C], uint32_t, float (&)[32]) {}
};

// One channel per look-up, for 4-bit channels: a pair table would have 256 entries, whose bank conflicts
// and construction cost more than the second load saves, so each row reads its own 16 values directly.
template <int C, int Q, int T>
struct MvAccumulateRow {
    static __device__ __forceinline__ void run(const uint32_t (&w)[C], uint32_t values_addr, float (&acc)[32]) {
        acc[T] += load_shared_float<Q * 64>(entry_address<C, C, T>(w, values_addr));
        MvAccumulateRow<C, Q, T + 1>::run(w, values_addr, acc);
    }
};
template <int C, int Q>
struct MvAccumulateRow<C, Q, 32> {
    static __device__ __forceinline__ void run(const uint32_t (&)[C], uint32_t, float (&)[32]) {}
};
template <int C, int Q>
struct MvRows {
    static __device__ __forceinline__ void run(const uint32_t (&w)[kMvRowsPerWarp][C], uint32_t values_addr,
                                               float (&acc)[32]) {
        MvAccumulateRow<C, Q, 0>::run(w[Q], values_addr, acc);
        MvRows<C, Q + 1>::run(w, values_addr, acc);
    }
};
template <int C>
struct MvRows<C, kMvRowsPerWarp> {
    static __device__ __forceinline__ void run(const uint32_t (&)[kMvRowsPerWarp][C], uint32_t, float (&)[32]) {}
};

#ifndef CMPQ_MV_PAIR_MAX_BITS
#define CMPQ_MV_PAIR_MAX_BITS 3  // widest channels that share a table between two channels
#endif
template <int C>
constexpr bool kMvUsePairs = (C <= CMPQ_MV_PAIR_MAX_BITS);

// ---- staging of the code words: asynchronous copies into a per-lane slot of shared memory -------------
// Every lane copies the C words of its own group for each row of a pass; word t of row q of lane l lands at
// stage[(q * C + t) * 32 + l] (conflict free).  Only the copying lane reads its words back, so waiting for
// the lane's own copy group is all the synchronisation the data needs.  Words at or beyond `valid`, and
// rows past the end, are zero-filled (a copy of source size 0 reads nothing).
template <int BYTES>
__device__ __forceinline__ void async_copy(uint32_t dst, const void* src, int src_bytes) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], %2, %3;" ::"r"(dst), "l"(src), "n"(BYTES), "r"(src_bytes)
                 : "memory");
}
__device__ __forceinline__ void async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void async_wait() {
    asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}

// Within a segment every channel has the same number of words, so the word offset of stored row r is
// off0 + (r - r0) * words_per_row with off0 = row_off[r0]: no load stands between a row and its copies.
template <int C>
__device__ __forceinline__ void stage_rows(const uint32_t* __restrict__ packed, int64_t off0, int64_t r0,
                                           int64_t words_per_row, int64_t r, int64_t r_end, int64_t group,
                                           int valid_words, uint32_t stage_addr /* shared address of this warp's stage */) {
    const int lane = threadIdx.x & 31;
#pragma unroll
    for (int q = 0; q < kMvRowsPerWarp; ++q) {
        const bool row_ok = (r + q < r_end) && valid_words > 0;
        const uint32_t* src = row_ok ? packed + off0 + (r + q - r0) * words_per_row + group * C : packed;
#pragma unroll
        for (int t = 0; t < C; ++t)
            async_copy<4>(stage_addr + ((q * C + t) * 32 + lane) * 4, row_ok && t < valid_words ? src + t : packed,
                          row_ok && t < valid_words ? 4 : 0);
    }
}

// The table values x_i * lut_i[k] of a pass are fetched in three steps spread over three passes, so that
// no step waits for the one before it: channel ids (perm) two passes ahead, the raw x_i and lut_i[k] one
// pass ahead, the product when the pass starts.  This lane holds rows 2q + (lane >> 4), entry k = lane & 15.
struct MvIds {
    int32_t i[kMvRowsPerWarp / 2];  // -1: no such row
};
struct MvRaw {
    uint16_t x[kMvRowsPerWarp / 2];
    float l[kMvRowsPerWarp / 2];
};

__device__ __forceinline__ MvIds load_ids(const int32_t* __restrict__ perm, int64_t r, int64_t r_end) {
    const int lane = threadIdx.x & 31;
    MvIds ids;
#pragma unroll
    for (int q = 0; q < kMvRowsPerWarp / 2; ++q) {
        const int64_t row = r + 2 * q + (lane >> 4);
        ids.i[q] = row < r_end ? perm[row] : -1;
    }
    return ids;
}

// The tables of a layer as the kernel reads them: fp32 as the final fit wrote them, or rounded to FP16
// (the stored format of Section 5.1), widened on the fly.
struct MvLut {
    const void* p;
    int is_f16;
    __device__ __forceinline__ float at(int64_t idx) const {
        return is_f16 ? __half2float(__ushort_as_half(static_cast<const uint16_t*>(p)[idx]))
                      : static_cast<const float*>(p)[idx];
    }
};

__device__ __forceinline__ MvRaw load_raw(const MvIds& ids, const MvLut& lut, const uint16_t* __restrict__ x) {
    const int lane = threadIdx.x & 31;
    MvRaw raw;
#pragma unroll
    for (int q = 0; q < kMvRowsPerWarp / 2; ++q) {
        raw.x[q] = ids.i[q] >= 0 ? x[ids.i[q]] : (uint16_t)0;
        raw.l[q] = ids.i[q] >= 0 ? lut.at((int64_t)ids.i[q] * CMPQ_LUT_STRIDE + (lane & 15)) : 0.0f;
    }
    return raw;
}

constexpr int kMvWarpTableBytes = (kMvRowsPerWarp / 2) * (4 << 8);   // four pair tables of 4-bit channels
constexpr int kMvWarpValueFloats = kMvRowsPerWarp * 16;              // t_i[k] of the rows of a pass
constexpr int kMvWarpStageBytes = kMvRowsPerWarp * 4 * 32 * 4;       // one pass of 4-bit code words
constexpr int kMvStages = 2;
constexpr int kMvTableRegion = kMvWarps * (kMvWarpTableBytes + kMvWarpValueFloats * 4);
constexpr int kMvSharedBytes = 1024 + kMvTableRegion + kMvWarps * kMvStages * kMvWarpStageBytes;
static_assert(kMvTableRegion >= kMvWarps * kMvPad * 4, "the reduction staging reuses the table space");

// One warp, all its passes over the chunk's rows: pass p computes while the words of pass p + 1 arrive.
template <int C, int DT>
__device__ __forceinline__ void matvec_warp(const uint32_t* __restrict__ packed, int64_t off0, int64_t r0,
                                            int64_t words_per_row, const int32_t* __restrict__ perm,
                                            const MvLut& lut, const uint16_t* __restrict__ x,
                                            int64_t r_first, int64_t r_end, int64_t group, int valid_words,
                                            float* values, float* tables, uint32_t stage_addr, float (&acc)[32]) {
    const int lane = threadIdx.x & 31;
    if (r_first >= r_end) return;
    stage_rows<C>(packed, off0, r0, words_per_row, r_first, r_end, group, valid_words, stage_addr);
    async_commit();
    MvRaw raw_now = load_raw(load_ids(perm, r_first, r_end), lut, x);
    MvIds ids_next = load_ids(perm, r_first + kMvRowsPerPass, r_end);
    int buf = 0;
    for (int64_t r = r_first; r < r_end; r += kMvRowsPerPass) {
        const int64_t rn = r + kMvRowsPerPass;
        if (rn < r_end)
            stage_rows<C>(packed, off0, r0, words_per_row, rn, r_end, group, valid_words,
                          stage_addr + (buf ^ 1) * kMvWarpStageBytes);
        async_commit();
        const MvRaw raw_next = load_raw(ids_next, lut, x);            // used in the next pass
        ids_next = load_ids(perm, rn + kMvRowsPerPass, r_end);        // used in the next pass
        // values[q][k] of this pass, then the pair tables: entry e of pair p = values[2p][e mod 2^C] +
        // values[2p+1][e div 2^C]
#pragma unroll
        for (int q = 0; q < kMvRowsPerWarp / 2; ++q)
            values[(2 * q + (lane >> 4)) * 16 + (lane & 15)] = widen16<DT>(raw_now.x[q]) * raw_now.l[q];
        __syncwarp();
        if constexpr (kMvUsePairs<C>) {
            constexpr int E = 1 << (2 * C);
#pragma unroll
            for (int idx0 = 0; idx0 < (kMvRowsPerWarp / 2) * E; idx0 += 32) {
                const int idx = idx0 + lane, pr = idx / E, e = idx % E;
                tables[idx] = values[(2 * pr) * 16 + (e & ((1 << C) - 1))] + values[(2 * pr + 1) * 16 + (e >> C)];
            }
        }
        async_wait<1>();  // the words of this pass have arrived (the next pass's group may still be in flight)
        uint32_t w[kMvRowsPerWarp][C];
        const uint32_t* st = reinterpret_cast<const uint32_t*>(__cvta_shared_to_generic(stage_addr + buf * kMvWarpStageBytes));
#pragma unroll
        for (int q = 0; q < kMvRowsPerWarp; ++q)
#pragma unroll
            for (int t = 0; t < C; ++t) w[q][t] = st[(q * C + t) * 32 + lane];
        __syncwarp();
        if constexpr (kMvUsePairs<C>) MvPairs<C, 0>::run(w, (uint32_t)__cvta_generic_to_shared(tables), acc);
        else MvRows<C, 0>::run(w, (uint32_t)__cvta_generic_to_shared(values), acc);
        __syncwarp();
        raw_now = raw_next;
        buf ^= 1;
    }
    async_wait<0>();
}

// partial[slot][j] = sum over the chunk's channels of x_i * lut_i[code_ij].
template <int DT>
__global__ void __launch_bounds__(kMvThreads, CMPQ_MV_MIN_BLOCKS)
matvec_partial_kernel(const uint32_t* __restrict__ packed, const int64_t* __restrict__ row_off,
                      const int32_t* __restrict__ perm, const int64_t* __restrict__ seg_rows,
                      const MvLut lut, const uint16_t* __restrict__ x, int64_t d_out,
                      int rows_per_block, float* __restrict__ partial) {
    extern __shared__ __align__(16) unsigned char raw[];
    // the finishing kernel may be scheduled from now on (it waits for this grid before it reads a partial sum)
    asm volatile("griddepcontrol.launch_dependents;");
    const MvChunk ch = matvec_chunk(seg_rows, blockIdx.y, rows_per_block);
    if (ch.c == 0) return;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    // the pair tables must sit on a multiple of their size (1 KB for 4-bit channels): align by hand
    const uint32_t raw_addr = (uint32_t)__cvta_generic_to_shared(raw);
    const uint32_t base_addr = (raw_addr + 1023u) & ~1023u;
    unsigned char* base = raw + (base_addr - raw_addr);
    float* tables = reinterpret_cast<float*>(base + warp * kMvWarpTableBytes);
    float* values = reinterpret_cast<float*>(base + kMvWarps * kMvWarpTableBytes) + warp * kMvWarpValueFloats;
    float* red = reinterpret_cast<float*>(base);  // [kMvWarps][kMvPad], used after the tables
    const uint32_t stage_addr = base_addr + kMvTableRegion + warp * kMvStages * kMvWarpStageBytes;
    const int64_t group = (int64_t)blockIdx.x * 32 + lane;  // group of 32 columns
    const int64_t words_per_row = (d_out * ch.c + 31) / 32;
    const int64_t left = words_per_row - group * ch.c;
    const int valid_words = (int)max((int64_t)0, min((int64_t)ch.c, left));
    float acc[32];
#pragma unroll
    for (int t = 0; t < 32; ++t) acc[t] = 0.0f;
    const int64_t r_first = ch.r0 + warp * kMvRowsPerWarp;
    const int64_t off0 = row_off[ch.r0];
    if (ch.c == 2)
        matvec_warp<2, DT>(packed, off0, ch.r0, words_per_row, perm, lut, x, r_first, ch.r1, group, valid_words, values,
                           tables, stage_addr, acc);
    else if (ch.c == 3)
        matvec_warp<3, DT>(packed, off0, ch.r0, words_per_row, perm, lut, x, r_first, ch.r1, group, valid_words, values,
                           tables, stage_addr, acc);
    else
        matvec_warp<4, DT>(packed, off0, ch.r0, words_per_row, perm, lut, x, r_first, ch.r1, group, valid_words, values,
                           tables, stage_addr, acc);
    __syncthreads();  // every warp is done with its tables: their space now stages the reduction
    // warps are summed in a fixed order; the staging is laid out so that both sides are conflict free
#pragma unroll
    for (int t = 0; t < 32; ++t) red[warp * kMvPad + lane * 33 + t] = acc[t];
    __syncthreads();
    float* out = partial + (int64_t)blockIdx.y * d_out + (int64_t)blockIdx.x * kMvCols;
    const int64_t cols_here = min((int64_t)kMvCols, d_out - (int64_t)blockIdx.x * kMvCols);
    for (int col = threadIdx.x; col < cols_here; col += kMvThreads) {
        float s = 0.0f;
#pragma unroll
        for (int wq = 0; wq < kMvWarps; ++wq) s += red[wq * kMvPad + col + (col >> 5)];
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
    // The outlier products need nothing from the partial kernel, so they run first: this kernel is launched
    // as a programmatic dependent of the partial kernel and may start while that one is still running.
    float so = 0.0f;
    if (j < d_out && col_ptr != nullptr) {
        const int64_t e0 = col_ptr[j], e1 = col_ptr[j + 1];
        for (int64_t e = e0 + warp; e < e1; e += 4 * kMvWarps) {  // four entries in flight, additions in order
            int32_t rw[4];
            uint16_t vv[4], xv[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const bool ok = e + u * kMvWarps < e1;
                rw[u] = ok ? c_rows[e + u * kMvWarps] : -1;
                vv[u] = ok ? c_vals[e + u * kMvWarps] : (uint16_t)0;
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) xv[u] = rw[u] >= 0 ? x[rw[u]] : (uint16_t)0;
#pragma unroll
            for (int u = 0; u < 4; ++u) so += widen16<DT>(xv[u]) * widen16<DT>(vv[u]);
        }
    }
    // From here on the partial sums are read: wait until the partial kernel has completed and its stores
    // are visible (returns at once when the kernel was launched without the dependency).
    asm volatile("griddepcontrol.wait;" ::: "memory");
    float s = 0.0f;
    if (j < d_out) {
        for (int64_t q = warp; q < chunks; q += 4 * kMvWarps) {  // absent partial sums read as 0
            float pv[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) pv[u] = (q + u * kMvWarps < chunks) ? __ldcg(partial + (q + u * kMvWarps) * d_out + j) : 0.0f;
#pragma unroll
            for (int u = 0; u < 4; ++u) s += pv[u];
        }
        s += so;
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

// The partial kernel needs more dynamic shared memory than the default limit: raise it once per device.
static bool matvec_allow_shared_memory() {
    static bool done[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return false;
    if (dev >= 0 && dev < 64 && done[dev]) return true;
    if (cudaFuncSetAttribute(matvec_partial_kernel<CMPQ_BF16>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             kMvSharedBytes) != cudaSuccess ||
        cudaFuncSetAttribute(matvec_partial_kernel<CMPQ_F16>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             kMvSharedBytes) != cudaSuccess)
        return false;
    if (dev >= 0 && dev < 64) done[dev] = true;
    return true;
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

static cmpq_status matvec_impl(const uint32_t* packed, const int64_t* row_off, const int32_t* perm,
                               const int64_t* seg_rows, const void* lut_p, int lut_is_f16, int64_t d_in, int64_t d_out,
                               const void* x, cmpq_dtype dt, const int64_t* col_ptr, const int32_t* c_rows,
                               const uint16_t* c_vals, float* y, void* y16, void* ws, size_t ws_bytes,
                               void* stream) {
    MvLut lut;
    lut.p = lut_p;
    lut.is_f16 = lut_is_f16;
    if (!packed || !row_off || !perm || !seg_rows || !lut_p || !x || !y) return CMPQ_ERR_INVALID_ARG;
    if (d_in < 1 || d_in > CMPQ_MAX_D_IN || d_out < 1 || d_out > CMPQ_MAX_D_OUT) return CMPQ_ERR_INVALID_ARG;
    if (dt != CMPQ_F16 && dt != CMPQ_BF16) return CMPQ_ERR_INVALID_ARG;
    if (col_ptr && (!c_rows || !c_vals)) return CMPQ_ERR_INVALID_ARG;
    if (!aligned_to(packed, 4) || !aligned_to(row_off, 8) || !aligned_to(seg_rows, 8) || !aligned_to(lut_p, lut_is_f16 ? 2 : 4) ||
        !aligned_to(x, 2) || !aligned_to(y, 4) || (y16 && !aligned_to(y16, 2)) || (col_ptr && !aligned_to(col_ptr, 8)))
        return CMPQ_ERR_INVALID_ARG;
    if (!ws || !aligned_to(ws, 256) || ws_bytes < matvec_ws_bytes(d_in, d_out)) return CMPQ_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int rb = matvec_rows_per_block(d_in, d_out);
    float* partial = static_cast<float*>(ws);
    if (!matvec_allow_shared_memory()) return CMPQ_ERR_CUDA;
    dim3 grid((unsigned)((d_out + kMvCols - 1) / kMvCols), (unsigned)matvec_max_chunks(d_in, rb));
    const unsigned fin_blocks = (unsigned)((d_out + 31) / 32);
    const uint16_t* xu = static_cast<const uint16_t*>(x);
    uint16_t* yu = static_cast<uint16_t*>(y16);
    // the finishing kernel is a programmatic dependent of the partial kernel: its launch and its outlier
    // products overlap the partial kernel, its griddepcontrol.wait orders the reads of the partial sums
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(fin_blocks);
    cfg.blockDim = dim3(kMvThreads);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = st;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const float* partial_in = partial;
    cudaError_t err;
    if (dt == CMPQ_BF16) {
        matvec_partial_kernel<CMPQ_BF16><<<grid, kMvThreads, kMvSharedBytes, st>>>(packed, row_off, perm, seg_rows, lut,
                                                                                   xu, d_out, rb, partial);
        err = cudaLaunchKernelEx(&cfg, matvec_finish_kernel<CMPQ_BF16>, partial_in, seg_rows, rb, d_out, xu, col_ptr,
                                 c_rows, c_vals, y, yu);
    } else {
        matvec_partial_kernel<CMPQ_F16><<<grid, kMvThreads, kMvSharedBytes, st>>>(packed, row_off, perm, seg_rows, lut,
                                                                                  xu, d_out, rb, partial);
        err = cudaLaunchKernelEx(&cfg, matvec_finish_kernel<CMPQ_F16>, partial_in, seg_rows, rb, d_out, xu, col_ptr,
                                 c_rows, c_vals, y, yu);
    }
    if (err != cudaSuccess) return CMPQ_ERR_CUDA;
    return launch_status();
}

extern "C" cmpq_status cmpq_matvec(const uint32_t* packed, const int64_t* row_off, const int32_t* perm,
                                   const int64_t* seg_rows, const float* lut, int64_t d_in, int64_t d_out,
                                   const void* x, cmpq_dtype dt, const int64_t* col_ptr, const int32_t* c_rows,
                                   const uint16_t* c_vals, float* y, void* y16, void* ws, size_t ws_bytes,
                                   void* stream) {
    return matvec_impl(packed, row_off, perm, seg_rows, lut, 0, d_in, d_out, x, dt, col_ptr, c_rows, c_vals, y, y16, ws,
                       ws_bytes, stream);
}

extern "C" cmpq_status cmpq_matvec_f16lut(const uint32_t* packed, const int64_t* row_off, const int32_t* perm,
                                          const int64_t* seg_rows, const uint16_t* lut16, int64_t d_in,
                                          int64_t d_out, const void* x, cmpq_dtype dt, const int64_t* col_ptr,
                                          const int32_t* c_rows, const uint16_t* c_vals, float* y, void* y16,
                                          void* ws, size_t ws_bytes, void* stream) {
    return matvec_impl(packed, row_off, perm, seg_rows, lut16, 1, d_in, d_out, x, dt, col_ptr, c_rows, c_vals, y, y16,
                       ws, ws_bytes, stream);
}
