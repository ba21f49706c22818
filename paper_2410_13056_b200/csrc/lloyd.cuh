// Channel-wise K-means of CMPQ (Section 3.2.1; quantizer of Section 3): launch interface.
#pragma once

#include "common.cuh"

namespace cmpq {

// What one launch of the channel kernel reads and writes.
struct LloydArgs {
    const uint16_t* W;       // [d_in][ldw] 16-bit weights
    int64_t d_in, d_out, ldw;
    const uint8_t* bits;     // [d_in] in {2,3,4}
    int iters;               // centroid updates T
    // provisional fit (Section 3.2.2): rows flagged in skip_row are not fitted, every other
    // row writes err[i*d_out + j] = |x - nearest centroid|
    const uint8_t* skip_row; // [d_in] or NULL
    float* err;              // [d_in*d_out] or NULL
    // final fit: positions row_ptr[i]..row_ptr[i+1] of cols are set to +0 before fitting
    const int64_t* row_ptr;  // [d_in+1] or NULL
    const int32_t* cols;     // [nnz] or NULL
    float* lut;              // [d_in][16] or NULL
    uint8_t* codes;          // [d_in][d_out] or NULL
    // ordered formulation: the last assignment can write the packed bit streams itself (layout of cmpq_pack)
    uint32_t* packed;        // or NULL
    const int64_t* word_off; // [d_in] first word of every channel (with packed)
    int32_t* inexact_rows;   // optional counter
    unsigned long long* sweeps;  // optional counter of distance evaluations
    int32_t* nonfinite;      // optional flag word: bit 1 is set when a weight is a NaN or an infinity
    // ordered formulation, provisional fit of the outlier step: every fitted channel leaves the limits of
    // its clusters in the tables and adds the largest error of each cluster side to this histogram (by the
    // top 12 bits of the error pattern), from which a lower bound of the selection threshold follows
    unsigned int* side_hist; // [4096] or NULL
    // ordered formulation only: fits kept across calls on the same weights (budget sweeps).  fit_cache is
    // the block lloyd_fit_cache_bytes() describes; a channel whose fit for its width is already there
    // copies it instead of iterating, every other channel stores its fit there.
    void* fit_cache;         // or NULL
    bool tables_ready;       // the value tables of every row to be fitted are in place already
};

// The process-wide choice made by cmpq_set_lloyd_assignment.
cmpq_lloyd_assignment lloyd_assignment();

// All-pairs formulation: one fused kernel, every iteration evaluates every (weight, centroid) pair.
cmpq_status launch_lloyd(const LloydArgs& args, cmpq_dtype dt, cudaStream_t st);

// Ordered formulation: value table per channel, warp-per-channel iterations, streaming last
// assignment.  `tables` is device scratch of lloyd_tables_bytes(d_in, d_out) bytes, 256-byte aligned.
size_t lloyd_tables_bytes(int64_t d_in, int64_t d_out);
// Value tables of every row of args.W alone (no fit); args.skip_row / row_ptr are honoured.
cmpq_status launch_lloyd_tables(const LloydArgs& args, cmpq_dtype dt, void* tables, size_t tables_bytes,
                                cudaStream_t st);
// Provisional fits per (width, channel) kept between calls: [header 256 B][valid 3 x d_in bytes]
// [centroids 3 x d_in x 16 floats][thresholds 3 x d_in x 16 floats]; cleared by launch_fit_cache_clear.
size_t lloyd_fit_cache_bytes(int64_t d_in);
cmpq_status launch_fit_cache_clear(void* fit_cache, int64_t d_in, int iters, cudaStream_t st);
// Final fit whose value tables are derived from those a provisional ordered fit of the same weights left
// in prov_tables, which is only read (args.row_ptr / args.cols: the positions removed since).
cmpq_status launch_lloyd_ordered_patched(const LloydArgs& args, cmpq_dtype dt, void* prov_tables, void* tables,
                                         size_t tables_bytes, cudaStream_t st);

// Selection of the worst-fitted entries on the tables of a provisional ordered fit made with neither codes
// nor errors requested (state: the radix select's SelectState; see outliers.cu for the procedure).
// state->lower = the lower edge of the histogram bin in which the n_q-th largest of the cluster-side
// maxima lies (0 if there are fewer); clears the histogram.
cmpq_status launch_select_lower(void* state, unsigned int* hist, cudaStream_t st);
cmpq_status launch_table_select_hist(void* tables, size_t tables_bytes, cmpq_dtype dt, const uint8_t* bits,
                                     const uint8_t* is_act, int64_t d_in, int64_t d_out, void* state,
                                     int shift, int bins, int final_pass, unsigned int* hist, cudaStream_t st);
cmpq_status launch_table_row_count(void* tables, size_t tables_bytes, cmpq_dtype dt, const uint8_t* bits,
                                   const uint8_t* is_act, int64_t d_in, int64_t d_out, const void* state,
                                   int32_t* gt, int32_t* eq, cudaStream_t st);
cmpq_status launch_table_emit(void* tables, size_t tables_bytes, cmpq_dtype dt, const uint16_t* W, int64_t ldw,
                              const uint8_t* bits, const uint8_t* is_act, int64_t d_in, int64_t d_out,
                              const void* state, const int32_t* gt, const int32_t* eq, const int32_t* take_eq,
                              const int64_t* row_start, int32_t* rows, int32_t* cols, uint16_t* vals,
                              cudaStream_t st);

// events[0..3] (cudaEvent_t, or NULL to clear): recorded around the three kernels of the next ordered launch.
void set_lloyd_phase_events(void* const* events);
cmpq_status launch_lloyd_ordered(const LloydArgs& args, cmpq_dtype dt, void* tables, size_t tables_bytes,
                                 cudaStream_t st);

// Weighted fit (sens: [d_in][d_out] fp32 sensitivities): one block per channel, every (weight, centroid) pair
// evaluated in every iteration; writes args.lut / args.codes / args.sweeps, ignores the other outputs.
cmpq_status launch_lloyd_weighted(const LloydArgs& args, cmpq_dtype dt, const float* sens, cudaStream_t st);
// the same fit on the value tables (tables: as for launch_lloyd_ordered); args.skip_row is not used
cmpq_status launch_lloyd_weighted_tables(const LloydArgs& args, cmpq_dtype dt, const float* sens, void* tables,
                                         size_t tables_bytes, cudaStream_t st);

// Fills row_ptr[0..d_in] from a row-sorted coordinate list.
cmpq_status launch_row_ptr(const int32_t* rows, int64_t nnz, int64_t d_in, int64_t* row_ptr,
                           cudaStream_t st);

// out[i] = base + how many of the two rank cuts k0, k1 channel i reaches in the ascending order of (a, id)
// (a cut >= d_in is reached by nobody).
cmpq_status launch_rank_cut(const float* a, int64_t d_in, int64_t k0, int64_t k1, int base, uint8_t* out,
                            cudaStream_t st);

cmpq_status launch_act_cut(const float* a, int64_t d_in, int64_t n_act, uint8_t* is_act, void* select_state,
                           long long n_q, unsigned int* hist, const uint8_t* bits, int64_t d_out, int64_t* row_off,
                           int32_t* perm, int64_t* seg_rows, int64_t* word_off, cudaStream_t st);

// rank[i] = position of channel i in the ascending order of (a, id).
cmpq_status launch_rank(const float* a, int64_t d_in, int32_t* rank, cudaStream_t st);

}  // namespace cmpq
