// Outlier protection of CMPQ (Section 3.2.2).
//
//   O_act  the n_act channels with the largest activation statistic are kept whole
//   O_q    after a provisional channel-wise K-means of W' = W - O_act, the n_q entries with the
//          largest error |W' - W'_q| are kept as well (equal errors: smaller linear index first)
//
// Errors are non-negative, so their
// bit patterns order like integers: an exact three-pass radix select (12 + 10 + 10 bits) finds
// the bit pattern tau of the n_q-th largest error and how many entries equal to tau still
// belong to the set.  Per-row counts and one scan over the rows then give every row its slice
// of the output, and each row writes its entries in column order, which yields the list sorted
// by (row, col) without a sort.
//
// Where the errors come from depends on the K-means formulation.  The all-pairs kernel writes one
// fp32 error per weight and the kernels in this file read them.  The ordered formulation never
// writes them: the error of a weight depends only on its value, so the select and the per-row
// counts run on the value tables of the fit (every distinct value weighed with its count) and the
// emit step recomputes the errors of the rows that keep entries (kernels in lloyd_hist.cu).
#include "lloyd.cuh"
#include "select.cuh"

namespace cmpq {

// hist[d] += number of errors in non-act rows whose fixed bits match the prefix and whose
// digit (err >> shift) & (bins-1) equals d.  One block handles whole rows.
__global__ void __launch_bounds__(kSelThreads)
select_hist_kernel(const float* __restrict__ err, const uint8_t* __restrict__ is_act, int64_t d_in,
                   int64_t d_out, const SelectState* __restrict__ st, int shift, int bins,
                   unsigned int* __restrict__ hist) {
    __shared__ unsigned int local[kSelBins];
    for (int b = threadIdx.x; b < bins; b += blockDim.x) local[b] = 0;
    __syncthreads();
    const uint32_t prefix = st->prefix, mask = st->mask;
    for (int64_t row = blockIdx.x; row < d_in; row += gridDim.x) {
        if (is_act[row]) continue;
        const uint32_t* e = reinterpret_cast<const uint32_t*>(err + row * d_out);
        for (int64_t j = threadIdx.x; j < d_out; j += blockDim.x) {
            uint32_t u = e[j];
            if ((u & mask) == prefix) atomicAdd(&local[(u >> shift) & (bins - 1)], 1u);
        }
    }
    __syncthreads();
    for (int b = threadIdx.x; b < bins; b += blockDim.x)
        if (local[b]) atomicAdd(&hist[b], local[b]);
}

__global__ void __launch_bounds__(1024)
select_digit_kernel(unsigned int* __restrict__ hist, int shift, int bins, SelectState* st, int final_pass) {
    __shared__ int warp_totals[32];
    __shared__ int found_digit;
    __shared__ long long found_above;
    select_digit_block<1024>(hist, shift, bins, st, final_pass, warp_totals, &found_digit, &found_above);
}

// Per row: how many errors exceed tau and how many equal it.
__global__ void __launch_bounds__(kSelThreads)
row_count_kernel(const float* __restrict__ err, const uint8_t* __restrict__ is_act, int64_t d_out,
                 const SelectState* __restrict__ st, int32_t* __restrict__ gt,
                 int32_t* __restrict__ eq) {
    __shared__ int sg, se;
    const int64_t row = blockIdx.x;
    if (threadIdx.x == 0) { sg = 0; se = 0; }
    __syncthreads();
    int g = 0, q = 0;
    if (!is_act[row]) {
        const uint32_t tau = st->tau;
        const uint32_t* e = reinterpret_cast<const uint32_t*>(err + row * d_out);
        for (int64_t j = threadIdx.x; j < d_out; j += blockDim.x) {
            uint32_t u = e[j];
            g += u > tau ? 1 : 0;
            q += u == tau ? 1 : 0;
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        g += __shfl_xor_sync(0xffffffffu, g, o);
        q += __shfl_xor_sync(0xffffffffu, q, o);
    }
    if ((threadIdx.x & 31) == 0) { if (g) atomicAdd(&sg, g); if (q) atomicAdd(&se, q); }
    __syncthreads();
    if (threadIdx.x == 0) { gt[row] = sg; eq[row] = se; }
}

// One block walks the rows in order: entries equal to tau are taken from the lowest rows first
// until take_equal is used up; row_start is the exclusive scan of the rows' output counts.
__global__ void __launch_bounds__(1024)
row_scan_kernel(const int32_t* __restrict__ gt, const int32_t* __restrict__ eq,
                const uint8_t* __restrict__ is_act, int64_t d_in, int64_t d_out,
                const SelectState* __restrict__ st, int32_t* __restrict__ take_eq,
                int64_t* __restrict__ row_start) {
    __shared__ int warp_totals[32];
    const long long take_equal = st->take_equal;
    long long eq_before = 0, out_before = 0;
    // every thread owns kPer consecutive rows of a chunk: two block scans per chunk, loads up front
    constexpr int kPer = 4;
    for (int64_t base = 0; base < d_in; base += (int64_t)blockDim.x * kPer) {
        const int64_t i0 = base + (int64_t)threadIdx.x * kPer;
        int e[kPer], g[kPer], act[kPer];
#pragma unroll
        for (int u = 0; u < kPer; ++u) {
            const bool in = i0 + u < d_in;
            e[u] = in ? eq[i0 + u] : 0;
            g[u] = in ? gt[i0 + u] : 0;
            act[u] = in ? is_act[i0 + u] : 0;
        }
        int e_sum = 0;
#pragma unroll
        for (int u = 0; u < kPer; ++u) e_sum += e[u];
        int tot_e;
        long long my_eq_before = eq_before + block_exclusive_scan(e_sum, warp_totals, tot_e);
        int te[kPer], sel[kPer], sel_sum = 0;
#pragma unroll
        for (int u = 0; u < kPer; ++u) {
            const long long room = take_equal - my_eq_before;
            te[u] = room <= 0 ? 0 : (room < e[u] ? (int)room : e[u]);
            my_eq_before += e[u];
            sel[u] = i0 + u < d_in ? (act[u] ? (int)d_out : g[u] + te[u]) : 0;
            sel_sum += sel[u];
        }
        int tot_s;
        long long my_out_before = out_before + block_exclusive_scan(sel_sum, warp_totals, tot_s);
#pragma unroll
        for (int u = 0; u < kPer; ++u) {
            if (i0 + u < d_in) { take_eq[i0 + u] = te[u]; row_start[i0 + u] = my_out_before; }
            my_out_before += sel[u];
        }
        eq_before += tot_e;
        out_before += tot_s;
    }
    if (threadIdx.x == 0) row_start[d_in] = out_before;
}

// Each row writes its kept entries in column order.  Rows of O_act are copied whole.  In the
// other rows kept entries are rare: candidates (error >= tau) are gathered into a short list in
// shared memory, ordered by column by counting, and the first take_eq[row] of those equal to tau
// are kept next to all larger ones.  A row with more candidates than the list holds falls back
// to a scan-based ordered compaction.
__global__ void __launch_bounds__(kSelThreads)
emit_kernel(const uint16_t* __restrict__ W, int64_t ldw, const float* __restrict__ err,
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
    const uint32_t* e = reinterpret_cast<const uint32_t*>(err + row * d_out);
    const int ncand = gt[row] + eq[row];
    if (ncand <= kEmitListCap) {
        if (threadIdx.x == 0) list_n = 0;
        __syncthreads();
        for (int64_t j = threadIdx.x; j < d_out; j += blockDim.x) {
            uint32_t u = e[j];
            if (u >= tau) {
                int p = atomicAdd(&list_n, 1);
                list_col[p] = (int)j;
                list_eq[p] = u == tau ? 1 : 0;
            }
        }
        __syncthreads();
        const int n = list_n;
        for (int i = threadIdx.x; i < n; i += blockDim.x) {
            const int c = list_col[i];
            const int is_eq = list_eq[i];
            int before = 0, eq_before = 0;   // candidates / tau-candidates in lower columns
            for (int t = 0; t < n; ++t) {
                int lower = list_col[t] < c ? 1 : 0;
                before += lower;
                eq_before += lower & list_eq[t];
            }
            const bool keep = !is_eq || eq_before < te;
            if (keep) {
                // dropped tau-candidates are exactly those of tau-rank >= te, all after the kept ones
                int dropped_before = eq_before > te ? eq_before - te : 0;
                int64_t pos = out0 + before - dropped_before;
                rows[pos] = (int32_t)row;
                cols[pos] = c;
                vals[pos] = w[c];
            }
        }
        return;
    }
    int eq_seen = 0, written = 0;
    for (int64_t base = 0; base < d_out; base += blockDim.x) {
        int64_t j = base + threadIdx.x;
        bool in = j < d_out;
        uint32_t u = in ? e[j] : 0u;
        int is_eq = (in && u == tau) ? 1 : 0;
        int tot_eq;
        int eq_rank = eq_seen + block_exclusive_scan(is_eq, warp_totals, tot_eq);
        int keep = in && (u > tau || (is_eq && eq_rank < te)) ? 1 : 0;
        int tot_keep;
        int pos = written + block_exclusive_scan(keep, warp_totals, tot_keep);
        if (keep) {
            rows[out0 + pos] = (int32_t)row;
            cols[out0 + pos] = (int32_t)j;
            vals[out0 + pos] = w[j];
        }
        eq_seen += tot_eq;
        written += tot_keep;
    }
}

// packed outputs of a call that also packs (all NULL otherwise)
struct PackOut {
    uint32_t* packed;
    int64_t* row_off;
    int32_t* perm;
    int64_t* seg_rows;
};

struct OutlierWs {
    float* err;     // one fp32 error per weight: only the all-pairs formulation materialises them
    uint8_t* is_act;
    unsigned int* hist;
    SelectState* state;
    int32_t* gt;
    int32_t* eq;
    int32_t* take_eq;
    int64_t* row_start;
    char* tables;  // value tables of the ordered K-means
};

// The layout depends on the assignment method selected when the call is made: the ordered formulation keeps
// value tables (about 5 bytes per weight), the all-pairs formulation an fp32 error per weight.
static OutlierWs carve(Workspace& w, int64_t d_in, int64_t d_out) {
    const bool all_pairs = lloyd_assignment() == CMPQ_ASSIGN_ALL_PAIRS;
    OutlierWs o;
    o.err = all_pairs ? w.take<float>((size_t)d_in * (size_t)d_out) : nullptr;
    o.is_act = w.take<uint8_t>(d_in);
    o.hist = w.take<unsigned int>(kSelBins);
    o.state = w.take<SelectState>(1);
    o.gt = w.take<int32_t>(d_in);
    o.eq = w.take<int32_t>(d_in);
    o.take_eq = w.take<int32_t>(d_in);
    o.row_start = w.take<int64_t>(d_in + 1);
    o.tables = all_pairs ? nullptr : w.take<char>(lloyd_tables_bytes(d_in, d_out));
    return o;
}

size_t outliers_ws_bytes(int64_t d_in, int64_t d_out) {
    Workspace w(nullptr, 0);
    carve(w, d_in, d_out);
    return w.used;
}

cmpq_status extract_impl(const void* W, cmpq_dtype dt, int64_t d_in, int64_t d_out, int64_t ldw, const float* a,
                         const uint8_t* bits, int64_t n_act, int64_t n_q, int lloyd_iters, int32_t* rows,
                         int32_t* cols, uint16_t* vals, int64_t nnz_out, const OutlierWs& o, cudaStream_t st,
                         void* fit_cache = nullptr, bool tables_ready = false, const PackOut* po = nullptr,
                         int64_t* word_off = nullptr, int32_t* nonfinite = nullptr);
static cmpq_status check_extract_args(const void* W, cmpq_dtype dt, int64_t d_in, int64_t d_out, int64_t ldw,
                                      const float* a, const uint8_t* bits, int64_t n_act, int64_t n_q,
                                      int lloyd_iters, const int32_t* rows, const int32_t* cols,
                                      const uint16_t* vals, int64_t nnz_out);

}  // namespace cmpq

using namespace cmpq;

extern "C" void cmpq_default_counts(int64_t d_in, int64_t d_out, int64_t* n_act, int64_t* n_q) {
    if (n_act) *n_act = (45 * d_in) / 10000;
    if (n_q) *n_q = (5 * d_in * d_out) / 10000;
}

extern "C" cmpq_status cmpq_extract_outliers(const void* W, cmpq_dtype dt, int64_t d_in, int64_t d_out,
                                             int64_t ldw, const float* a, const uint8_t* bits,
                                             int64_t n_act, int64_t n_q, int lloyd_iters,
                                             int32_t* rows, int32_t* cols, uint16_t* vals,
                                             int64_t nnz_out, int32_t* nonfinite, void* ws, size_t ws_bytes,
                                             void* stream) {
    if (!aligned_to(nonfinite, 4)) return CMPQ_ERR_INVALID_ARG;
    const cmpq_status chk = check_extract_args(W, dt, d_in, d_out, ldw, a, bits, n_act, n_q, lloyd_iters, rows, cols, vals, nnz_out);
    if (chk != CMPQ_OK) return chk;
    if (!ws || !aligned_to(ws, 256) || ws_bytes < outliers_ws_bytes(d_in, d_out)) return CMPQ_ERR_WORKSPACE;
    Workspace wsp(ws, ws_bytes);
    OutlierWs o = carve(wsp, d_in, d_out);
    return extract_impl(W, dt, d_in, d_out, ldw, a, bits, n_act, n_q, lloyd_iters, rows, cols, vals, nnz_out, o,
                        static_cast<cudaStream_t>(stream), nullptr, false, nullptr, nullptr, nonfinite);
}

namespace cmpq {

cmpq_status extract_impl(const void* W, cmpq_dtype dt, int64_t d_in, int64_t d_out, int64_t ldw, const float* a,
                         const uint8_t* bits, int64_t n_act, int64_t n_q, int lloyd_iters, int32_t* rows,
                         int32_t* cols, uint16_t* vals, int64_t nnz_out, const OutlierWs& o, cudaStream_t st,
                         void* fit_cache, bool tables_ready, const PackOut* po, int64_t* word_off, int32_t* nonfinite) {
    const bool all_pairs = lloyd_assignment() == CMPQ_ASSIGN_ALL_PAIRS;
    const size_t tables_bytes = lloyd_tables_bytes(d_in, d_out);
    const uint16_t* Wp = static_cast<const uint16_t*>(W);

    // O_act: the channels of rank >= d_in - n_act in the ascending order of (a, id).  The same block also
    // resets the select and, for a call that packs, lays out the packed segments (widths alone decide it).
    cmpq_status s = launch_act_cut(a, d_in, n_act, o.is_act, o.state, (long long)n_q, o.hist, po ? bits : nullptr, d_out,
                                   po ? po->row_off : nullptr, po ? po->perm : nullptr, po ? po->seg_rows : nullptr,
                                   word_off, st);
    if (s != CMPQ_OK) return s;

    if (n_q > 0) {
        LloydArgs la{};
        la.W = static_cast<const uint16_t*>(W);
        la.d_in = d_in; la.d_out = d_out; la.ldw = ldw;
        la.bits = bits;
        la.iters = lloyd_iters;
        la.skip_row = o.is_act;
        // all pairs: one fp32 error per weight is written; ordered: the fit alone, errors are then
        // taken from the value tables
        la.err = all_pairs ? o.err : nullptr;
        la.fit_cache = fit_cache;
        la.tables_ready = tables_ready;
        la.nonfinite = nonfinite;
        la.side_hist = all_pairs ? nullptr : o.hist;
        s = all_pairs ? launch_lloyd(la, dt, st) : launch_lloyd_ordered(la, dt, o.tables, tables_bytes, st);
        if (s != CMPQ_OK) return s;
    }

    if (n_q > 0) {
        int sms = sm_count();
        if (sms <= 0) return CMPQ_ERR_CUDA;
        unsigned hist_blocks = (unsigned)((int64_t)sms * 8 < d_in ? (int64_t)sms * 8 : d_in);
        const int shifts[3] = {20, 10, 0};
        const int bins[3] = {4096, 1024, 1024};
        if (!all_pairs) {  // a lower bound of the threshold from the largest errors of the cluster sides
            s = launch_select_lower(o.state, o.hist, st);
            if (s != CMPQ_OK) return s;
        }
        for (int p = 0; p < 3; ++p) {
            if (all_pairs) {
                select_hist_kernel<<<hist_blocks, kSelThreads, 0, st>>>(o.err, o.is_act, d_in, d_out, o.state, shifts[p], bins[p], o.hist);
                select_digit_kernel<<<1, 1024, 0, st>>>(o.hist, shifts[p], bins[p], o.state, p == 2);
            } else {  // the last block of the histogram kernel to finish also fixes the digit
                s = launch_table_select_hist(o.tables, tables_bytes, dt, bits, o.is_act, d_in, d_out, o.state, shifts[p], bins[p], p == 2, o.hist, st);
                if (s != CMPQ_OK) return s;
            }
        }
        if (all_pairs) {
            row_count_kernel<<<(unsigned)d_in, kSelThreads, 0, st>>>(o.err, o.is_act, d_out, o.state, o.gt, o.eq);
        } else {
            s = launch_table_row_count(o.tables, tables_bytes, dt, bits, o.is_act, d_in, d_out, o.state, o.gt, o.eq, st);
            if (s != CMPQ_OK) return s;
        }
    } else {
        if (cudaMemsetAsync(o.gt, 0, (size_t)d_in * sizeof(int32_t), st) != cudaSuccess) return CMPQ_ERR_CUDA;
        if (cudaMemsetAsync(o.eq, 0, (size_t)d_in * sizeof(int32_t), st) != cudaSuccess) return CMPQ_ERR_CUDA;
    }
    row_scan_kernel<<<1, 1024, 0, st>>>(o.gt, o.eq, o.is_act, d_in, d_out, o.state, o.take_eq, o.row_start);
    if (nnz_out > 0) {
        // with n_q == 0 no row outside O_act keeps anything, so neither errors nor tables are read
        if (all_pairs || n_q == 0)
            emit_kernel<<<(unsigned)d_in, kSelThreads, 0, st>>>(Wp, ldw, o.err, o.is_act, d_out, o.state, o.gt, o.eq, o.take_eq, o.row_start, rows, cols, vals);
        else
            return launch_table_emit(o.tables, tables_bytes, dt, Wp, ldw, bits, o.is_act, d_in, d_out, o.state, o.gt, o.eq, o.take_eq, o.row_start, rows, cols, vals, st);
    }
    return launch_status();
}

static cmpq_status check_extract_args(const void* W, cmpq_dtype dt, int64_t d_in, int64_t d_out, int64_t ldw,
                                      const float* a, const uint8_t* bits, int64_t n_act, int64_t n_q,
                                      int lloyd_iters, const int32_t* rows, const int32_t* cols,
                                      const uint16_t* vals, int64_t nnz_out) {
    if (!W || !a || !bits) return CMPQ_ERR_INVALID_ARG;
    if (dt != CMPQ_F16 && dt != CMPQ_BF16) return CMPQ_ERR_INVALID_ARG;
    if (d_in < 1 || d_in > CMPQ_MAX_D_IN || d_out < 1 || d_out > CMPQ_MAX_D_OUT || ldw < d_out)
        return CMPQ_ERR_INVALID_ARG;
    if (n_act < 0 || n_act > d_in || n_q < 0 || n_q > (d_in - n_act) * d_out) return CMPQ_ERR_INVALID_ARG;
    if (nnz_out != n_act * d_out + n_q) return CMPQ_ERR_INVALID_ARG;
    if (nnz_out > 0 && (!rows || !cols || !vals)) return CMPQ_ERR_INVALID_ARG;
    if (lloyd_iters < 0 || lloyd_iters > CMPQ_MAX_LLOYD_ITERS) return CMPQ_ERR_INVALID_ARG;
    if (!aligned_to(W, 2)) return CMPQ_ERR_INVALID_ARG;
    if (d_in * d_out > 0x7fffffffLL) return CMPQ_ERR_UNSUPPORTED;  // 32-bit counters in the select
    return CMPQ_OK;
}

// Work space of the fused call: the outlier step's.  The final fit derives its tables from the provisional
// ones: in shared memory for nearly every channel, in place in the provisional tables for the others.
struct FusedWs {
    OutlierWs o;
};

static FusedWs carve_fused(Workspace& w, int64_t d_in, int64_t d_out) {
    FusedWs f;
    f.o = carve(w, d_in, d_out);
    return f;
}

size_t protect_quantize_ws_bytes(int64_t d_in, int64_t d_out) {
    Workspace w(nullptr, 0);
    carve_fused(w, d_in, d_out);
    return w.used;
}

size_t protect_quantize_pack_ws_bytes(int64_t d_in, int64_t d_out) {
    return protect_quantize_ws_bytes(d_in, d_out) + pack_ws_bytes(d_in, d_out);
}

cmpq_status launch_pack_layout(const uint8_t* bits, int64_t d_in, int64_t d_out, int64_t* row_off, int32_t* perm,
                               int64_t* seg_rows, int64_t* word_off, cudaStream_t st);
cmpq_status launch_pack_codes(const uint8_t* codes, const uint8_t* bits, int64_t d_in, int64_t d_out,
                              const int64_t* word_off, uint32_t* packed, cudaStream_t st);


}  // namespace cmpq

namespace cmpq {

// Sweep cache: [value tables of all channels][fits kept per (width, channel)]
struct SweepCache {
    char* tables;
    char* fits;
};

static SweepCache carve_sweep(void* cache, int64_t d_in, int64_t d_out) {
    Workspace w(cache, ~(size_t)0);
    SweepCache c;
    c.tables = w.take<char>(lloyd_tables_bytes(d_in, d_out));
    c.fits = w.take<char>(lloyd_fit_cache_bytes(d_in));
    return c;
}

static size_t sweep_cache_bytes(int64_t d_in, int64_t d_out) {
    return round_up(lloyd_tables_bytes(d_in, d_out), 256) + round_up(lloyd_fit_cache_bytes(d_in), 256);
}

// Outlier protection and final fit; with a sweep cache the provisional fit takes its value tables (and the
// fits already made) from there.
static cmpq_status protect_quantize_impl(const void* W, cmpq_dtype dt, int64_t d_in, int64_t d_out, int64_t ldw,
                                         const float* a, const uint8_t* bits, int64_t n_act, int64_t n_q,
                                         int lloyd_iters, int32_t* rows, int32_t* cols, uint16_t* vals,
                                         int64_t nnz_out, float* lut, uint8_t* codes, int32_t* inexact_rows,
                                         unsigned long long* sweeps, int32_t* nonfinite, void* ws, size_t ws_bytes,
                                         void* cache, cudaStream_t st, const PackOut* po = nullptr) {
    cmpq_status s = check_extract_args(W, dt, d_in, d_out, ldw, a, bits, n_act, n_q, lloyd_iters, rows, cols, vals, nnz_out);
    if (s != CMPQ_OK) return s;
    if (!lut || !aligned_to(lut, 4) || !aligned_to(nonfinite, 4)) return CMPQ_ERR_INVALID_ARG;
    if (!codes && !po) return CMPQ_ERR_INVALID_ARG;
    if (codes && !aligned_to(codes, 8)) return CMPQ_ERR_INVALID_ARG;
    if (po && (!po->packed || !po->row_off || !po->perm || !po->seg_rows || !aligned_to(po->packed, 4) ||
               !aligned_to(po->row_off, 8) || !aligned_to(po->perm, 4) || !aligned_to(po->seg_rows, 8)))
        return CMPQ_ERR_INVALID_ARG;
    const bool ordered = lloyd_assignment() != CMPQ_ASSIGN_ALL_PAIRS;
    if (po && !codes && !ordered) return CMPQ_ERR_UNSUPPORTED;  // the all-pairs kernel writes byte codes
    const size_t need = po ? protect_quantize_pack_ws_bytes(d_in, d_out) : protect_quantize_ws_bytes(d_in, d_out);
    if (!ws || !aligned_to(ws, 256) || ws_bytes < need) return CMPQ_ERR_WORKSPACE;
    Workspace wsp(ws, ws_bytes);
    FusedWs f = carve_fused(wsp, d_in, d_out);
    int64_t* word_off = po ? wsp.take<int64_t>(d_in) : nullptr;
    void* fit_cache = nullptr;
    char* final_tables = f.o.tables;  // the provisional tables are patched in place ...
    if (cache && ordered) {  // ... unless they are the cache's, which stay as they are: the work space's serve
        const SweepCache c = carve_sweep(cache, d_in, d_out);
        f.o.tables = c.tables;
        fit_cache = c.fits;
    }
    s = extract_impl(W, dt, d_in, d_out, ldw, a, bits, n_act, n_q, lloyd_iters, rows, cols, vals, nnz_out, f.o, st,
                     fit_cache, fit_cache != nullptr, po, word_off, nonfinite);
    if (s != CMPQ_OK) return s;
    // the list is sorted by row, so the first list position of a row is the start of the row's slice of
    // the output: the row index of the final fit is the scan the outlier step has just made
    LloydArgs la{};
    la.W = static_cast<const uint16_t*>(W);
    la.d_in = d_in; la.d_out = d_out; la.ldw = ldw;
    la.bits = bits;
    la.iters = lloyd_iters;
    la.row_ptr = f.o.row_start;
    la.cols = cols;
    la.lut = lut;
    la.codes = codes;
    la.inexact_rows = inexact_rows;
    la.sweeps = sweeps;
    la.nonfinite = nonfinite;
    const size_t tables_bytes = lloyd_tables_bytes(d_in, d_out);
    if (!ordered) {
        s = launch_lloyd(la, dt, st);
        if (s != CMPQ_OK || !po) return s;
        return launch_pack_codes(codes, bits, d_in, d_out, word_off, po->packed, st);
    }
    if (po) {  // the last assignment writes the packed words itself
        la.packed = po->packed;
        la.word_off = word_off;
    }
    // the provisional fit ran (and left its tables) only when entries had to be selected; a sweep cache
    // holds the tables of all channels in any case
    if (n_q > 0 || fit_cache) return launch_lloyd_ordered_patched(la, dt, f.o.tables, final_tables, tables_bytes, st);
    return launch_lloyd_ordered(la, dt, final_tables, tables_bytes, st);
}

}  // namespace cmpq

extern "C" cmpq_status cmpq_protect_and_quantize(const void* W, cmpq_dtype dt, int64_t d_in, int64_t d_out,
                                                 int64_t ldw, const float* a, const uint8_t* bits,
                                                 int64_t n_act, int64_t n_q, int lloyd_iters, int32_t* rows,
                                                 int32_t* cols, uint16_t* vals, int64_t nnz_out, float* lut,
                                                 uint8_t* codes, int32_t* inexact_rows,
                                                 unsigned long long* sweeps, int32_t* nonfinite, void* ws,
                                                 size_t ws_bytes, void* stream) {
    return protect_quantize_impl(W, dt, d_in, d_out, ldw, a, bits, n_act, n_q, lloyd_iters, rows, cols, vals, nnz_out,
                                 lut, codes, inexact_rows, sweeps, nonfinite, ws, ws_bytes, nullptr,
                                 static_cast<cudaStream_t>(stream));
}

extern "C" cmpq_status cmpq_protect_quantize_pack(const void* W, cmpq_dtype dt, int64_t d_in, int64_t d_out,
                                                  int64_t ldw, const float* a, const uint8_t* bits,
                                                  int64_t n_act, int64_t n_q, int lloyd_iters, int32_t* rows,
                                                  int32_t* cols, uint16_t* vals, int64_t nnz_out, float* lut,
                                                  uint8_t* codes, uint32_t* packed, int64_t* row_off,
                                                  int32_t* perm, int64_t* seg_rows, int32_t* inexact_rows,
                                                  unsigned long long* sweeps, int32_t* nonfinite, void* ws,
                                                  size_t ws_bytes, void* stream) {
    const PackOut po{packed, row_off, perm, seg_rows};
    return protect_quantize_impl(W, dt, d_in, d_out, ldw, a, bits, n_act, n_q, lloyd_iters, rows, cols, vals, nnz_out,
                                 lut, codes, inexact_rows, sweeps, nonfinite, ws, ws_bytes, nullptr,
                                 static_cast<cudaStream_t>(stream), &po);
}

extern "C" size_t cmpq_sweep_cache_bytes(int64_t d_in, int64_t d_out) {
    if (d_in < 1 || d_in > CMPQ_MAX_D_IN || d_out < 1 || d_out > CMPQ_MAX_D_OUT) return 0;
    return sweep_cache_bytes(d_in, d_out);
}

extern "C" cmpq_status cmpq_sweep_begin(const void* W, cmpq_dtype dt, int64_t d_in, int64_t d_out, int64_t ldw,
                                        int lloyd_iters, int32_t* nonfinite, void* cache, size_t cache_bytes,
                                        void* stream) {
    if (!W || (dt != CMPQ_F16 && dt != CMPQ_BF16) || !aligned_to(W, 2) || !aligned_to(nonfinite, 4)) return CMPQ_ERR_INVALID_ARG;
    if (d_in < 1 || d_in > CMPQ_MAX_D_IN || d_out < 1 || d_out > CMPQ_MAX_D_OUT || ldw < d_out) return CMPQ_ERR_INVALID_ARG;
    if (lloyd_iters < 0 || lloyd_iters > CMPQ_MAX_LLOYD_ITERS) return CMPQ_ERR_INVALID_ARG;
    if (!cache || !aligned_to(cache, 256) || cache_bytes < sweep_cache_bytes(d_in, d_out)) return CMPQ_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const SweepCache c = carve_sweep(cache, d_in, d_out);
    LloydArgs la{};
    la.W = static_cast<const uint16_t*>(W);
    la.d_in = d_in; la.d_out = d_out; la.ldw = ldw;
    la.nonfinite = nonfinite;
    cmpq_status s = launch_lloyd_tables(la, dt, c.tables, lloyd_tables_bytes(d_in, d_out), st);
    if (s != CMPQ_OK) return s;
    return launch_fit_cache_clear(c.fits, d_in, lloyd_iters, st);
}

extern "C" cmpq_status cmpq_sweep_budget(const void* W, cmpq_dtype dt, int64_t d_in, int64_t d_out, int64_t ldw,
                                         const float* a, const uint8_t* bits, int64_t n_act, int64_t n_q,
                                         int lloyd_iters, int32_t* rows, int32_t* cols, uint16_t* vals,
                                         int64_t nnz_out, float* lut, uint8_t* codes, int32_t* inexact_rows,
                                         unsigned long long* sweeps, void* cache, size_t cache_bytes, void* ws,
                                         size_t ws_bytes, void* stream) {
    if (!cache || !aligned_to(cache, 256)) return CMPQ_ERR_WORKSPACE;
    if (d_in >= 1 && d_in <= CMPQ_MAX_D_IN && d_out >= 1 && d_out <= CMPQ_MAX_D_OUT &&
        cache_bytes < sweep_cache_bytes(d_in, d_out))
        return CMPQ_ERR_WORKSPACE;
    return protect_quantize_impl(W, dt, d_in, d_out, ldw, a, bits, n_act, n_q, lloyd_iters, rows, cols, vals, nnz_out,
                                 lut, codes, inexact_rows, sweeps, nullptr, ws, ws_bytes, cache,
                                 static_cast<cudaStream_t>(stream));
}

extern "C" cmpq_status cmpq_sweep_budget_pack(const void* W, cmpq_dtype dt, int64_t d_in, int64_t d_out, int64_t ldw,
                                              const float* a, const uint8_t* bits, int64_t n_act, int64_t n_q,
                                              int lloyd_iters, int32_t* rows, int32_t* cols, uint16_t* vals,
                                              int64_t nnz_out, float* lut, uint8_t* codes, uint32_t* packed,
                                              int64_t* row_off, int32_t* perm, int64_t* seg_rows,
                                              int32_t* inexact_rows, unsigned long long* sweeps, void* cache,
                                              size_t cache_bytes, void* ws, size_t ws_bytes, void* stream) {
    if (!cache || !aligned_to(cache, 256)) return CMPQ_ERR_WORKSPACE;
    if (d_in >= 1 && d_in <= CMPQ_MAX_D_IN && d_out >= 1 && d_out <= CMPQ_MAX_D_OUT &&
        cache_bytes < sweep_cache_bytes(d_in, d_out))
        return CMPQ_ERR_WORKSPACE;
    const PackOut po{packed, row_off, perm, seg_rows};
    return protect_quantize_impl(W, dt, d_in, d_out, ldw, a, bits, n_act, n_q, lloyd_iters, rows, cols, vals, nnz_out,
                                 lut, codes, inexact_rows, sweeps, nullptr, ws, ws_bytes, cache,
                                 static_cast<cudaStream_t>(stream), &po);
}
