/*
 * cmpq.h -- C ABI of the CMPQ quantization pass for one linear layer on one GPU.
 *
 * CMPQ (channel-wise mixed-precision quantization, arxiv 2410.13056) quantizes a
 * weight matrix W in R^{d_in x d_out} channel by channel, a channel being the row
 * W_{i,:} that multiplies input feature i (Section 3.2.1).  The pass is:
 *   statistic   a_j = ||X[:,j]||_2 over the calibration tokens     (Section 3.2.1)
 *   allocation  c in {2,3,4}^{d_in} for an average budget b         (Algorithm 1)
 *   outliers    O_act (whole channels, largest a) and O_q (entries a
 *               provisional K-means fits worst), kept in 16 bits    (Section 3.2.2)
 *   quantizer   per channel K-means with K = 2^{c_i}, nearest-centroid
 *               codes                                               (Sections 3, 3.2.1)
 *   packing     codes grouped by bit width into bit streams         (Sections 5.1, 6)
 * and, for the quantized layer, the product of one token with it   (Section 6).
 *
 * Conventions for every entry point
 *  - All array arguments are DEVICE pointers owned by the caller unless the
 *    parameter comment says "host".  The library allocates no memory; scratch space
 *    is the caller's `ws` buffer of at least cmpq_workspace_bytes(op, ...) bytes,
 *    256-byte aligned, whose contents are undefined before and after the call.
 *    The only state it keeps between calls is host state that the caller sets
 *    explicitly: the process-wide assignment method (cmpq_set_lloyd_assignment,
 *    which also decides what cmpq_workspace_bytes answers) and the one-shot event
 *    handles of cmpq_lloyd_phase_events; cmpq_collect_stats_static in addition
 *    owns a fixed device array (see there).
 *  - `stream` is a cudaStream_t passed as void* (NULL = default stream).  Calls
 *    only enqueue work; outputs are valid once the stream has been synchronised.
 *  - Matrices are row-major with a leading dimension in elements (ldx, ldw).
 *    16-bit floating inputs (cmpq_dtype) are passed as const void*.
 *  - Arguments are checked on the host before anything is launched.  A call
 *    returns CMPQ_OK or an error code and never throws, aborts or prints;
 *    after an error no output has been written.
 *  - Inputs must be finite.  Calls never look at their inputs on the host; the calls that read the
 *    activations or the weights take an optional device word `nonfinite` (int32, zeroed by the caller,
 *    may be NULL) into which the kernels OR bit 0 when an activation, and bit 1 when a weight, is a NaN or
 *    an infinity (they read every value anyway, so the test costs nothing).  The outputs of such a call are
 *    unspecified; the K-means iterations of the same call are skipped once the word is non-zero.
 *    cmpq_check_finite waits for the stream and turns the word into a status.
 *  - Results are deterministic: the same inputs give the same bytes.
 */
#ifndef CMPQ_H_
#define CMPQ_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    CMPQ_OK = 0,
    CMPQ_ERR_INVALID_ARG = 1, /* null pointer, negative size, budget outside [2,4], ... */
    CMPQ_ERR_UNSUPPORTED = 2, /* legal but outside what the kernels handle (see each call) */
    CMPQ_ERR_WORKSPACE = 3,   /* ws is NULL, misaligned or smaller than cmpq_workspace_bytes */
    CMPQ_ERR_CUDA = 4,        /* a CUDA runtime call failed */
    CMPQ_ERR_INTERNAL = 5,
    CMPQ_ERR_NONFINITE = 6    /* an input held a NaN or an infinity (answer of cmpq_check_finite) */
} cmpq_status;

typedef enum { CMPQ_F16 = 0, CMPQ_BF16 = 1 } cmpq_dtype;

/* Which norm of a channel's activations serves as the allocation criterion.  L2 is the paper's
 * choice (Section 3.2.1); L1 and LINF are the alternatives its norm-ablation table compares. */
typedef enum { CMPQ_NORM_L2 = 0, CMPQ_NORM_L1 = 1, CMPQ_NORM_LINF = 2 } cmpq_norm;

/* How Algorithm 1's "q-quantile" is read.  RANK: the floor(|b-3| d_in + 1/2)
 * channels with the smallest (b < 3) or largest (b > 3) statistic change width
 * (at b == 3 exactly: floor(0.01 d_in + 1/2) at each end); equal statistics are
 * ordered by channel id.  QUANTILE: thresholds are linearly interpolated
 * quantiles of a and the comparisons are strict, as the algorithm is printed. */
typedef enum { CMPQ_ALLOC_RANK = 0, CMPQ_ALLOC_QUANTILE = 1 } cmpq_alloc_mode;

/* How the K-means kernels find the nearest centroid of every weight (Section 3: each weight goes
 * to its nearest centroid; the rule itself is stated at cmpq_quantize_layer and is the same for
 * both).  Both give bit-identical centroids, codes and errors.
 *   CMPQ_ASSIGN_ORDERED    (default) the channel is sorted once; while the centroids are strictly
 *                          increasing with safe gaps, a cluster is a run of the sorted order and an
 *                          iteration only searches the K-1 run boundaries and reads prefix sums.
 *                          Iterations whose centroids do not allow this fall back to all pairs.
 *   CMPQ_ASSIGN_ALL_PAIRS  every iteration evaluates every (weight, centroid) pair on the fp32
 *                          pipes: the brute-force formulation, kept for measuring ALU throughput. */
typedef enum { CMPQ_ASSIGN_ORDERED = 0, CMPQ_ASSIGN_ALL_PAIRS = 1 } cmpq_lloyd_assignment;

typedef enum {
    CMPQ_OP_COLLECT_STATS = 0,
    CMPQ_OP_ALLOCATE_BITS = 1,
    CMPQ_OP_EXTRACT_OUTLIERS = 2,
    CMPQ_OP_QUANTIZE_LAYER = 3,
    CMPQ_OP_PACK = 4,
    CMPQ_OP_PROTECT_AND_QUANTIZE = 5,
    CMPQ_OP_OUTLIERS_BY_COLUMN = 6, /* d_in is ignored */
    CMPQ_OP_MATVEC = 7,
    CMPQ_OP_QUANTIZE_LAYER_PACKED = 8,
    CMPQ_OP_PROTECT_QUANTIZE_PACK = 9
} cmpq_op;

#define CMPQ_LUT_STRIDE 16      /* floats per channel in a look-up table */
#define CMPQ_MAX_D_OUT 32768    /* one thread block holds one channel */
#define CMPQ_MAX_D_IN 262144
#define CMPQ_MAX_LLOYD_ITERS 1000

/* ---- statistic (Section 3.2.1: per-channel L2 norm of the activation matrix X) --------------
 * sumsq[j] += sum_t X[t*ldx + j]^2 for the n_tokens rows given; call it once per chunk of
 * calibration tokens after zeroing sumsq (fp64, d_in entries).  Squares are formed in fp32
 * (exact for 16-bit inputs), partial sums in fp32 over at most 32 rows, the rest in fp64 in
 * a fixed order.  n_tokens may be 0.  X is [n_tokens][ldx] of `dt`, ldx >= d_in.
 * Because the squares are formed in fp32, a bf16 activation beyond about 1.8e19 in magnitude overflows
 * to infinity although it is finite: it is reported through `nonfinite` like a true infinity (fp16
 * inputs cannot get there).
 * ws: cmpq_workspace_bytes(CMPQ_OP_COLLECT_STATS, d_in, 0). */
cmpq_status cmpq_collect_stats(const void* X, cmpq_dtype dt, int64_t n_tokens, int64_t d_in,
                               int64_t ldx, double* sumsq, int32_t* nonfinite, void* ws, size_t ws_bytes,
                               void* stream);

/* Waits for `stream` and reads the word the calls above and below OR their findings into:
 * CMPQ_OK if it is zero, CMPQ_ERR_NONFINITE otherwise (CMPQ_ERR_INVALID_ARG for NULL). */
cmpq_status cmpq_check_finite(const int32_t* nonfinite, void* stream);

/* Same result as cmpq_collect_stats without any work space: the partial sums live in a fixed
 * 2 MiB array inside the library (the paper has no counterpart; this exists for callers that
 * cannot allocate device memory: code running inside another framework's memory plan, code that
 * must avoid the device-wide synchronisation an allocation implies, plug-ins that only receive
 * input and output buffers).  The array is held by every GPU that loads the library until the
 * process exits.  d_in <= CMPQ_STATIC_MAX_D_IN, else CMPQ_ERR_UNSUPPORTED; other checks as above.
 * The call allocates and frees nothing.  The first call on each device looks up the array's
 * device address (make that call before any stream capture starts).  All calls on a device share
 * the array: two calls whose kernels may overlap on the GPU (different streams, no ordering
 * between them) race on it; calls on one stream are safe.  Nothing needs clearing between calls:
 * each call overwrites every partial it later reads.  The number of partial sums may differ
 * from cmpq_collect_stats, so results agree to rounding (about 1e-7 relative), not bit for bit. */
#define CMPQ_STATIC_MAX_D_IN 32768
cmpq_status cmpq_collect_stats_static(const void* X, cmpq_dtype dt, int64_t n_tokens, int64_t d_in,
                                      int64_t ldx, double* sumsq, void* stream);

/* a[j] = (float) sqrt(sumsq[j]). */
cmpq_status cmpq_finalize_stats(const double* sumsq, int64_t d_in, float* a, void* stream);

/* The statistic for another norm (appendix of the paper, norm-ablation table).  Same contract as
 * cmpq_collect_stats / cmpq_finalize_stats with acc (fp64, d_in entries, zeroed by the caller
 * before the first chunk) accumulating
 *   CMPQ_NORM_L2    acc[j] += sum_t X[t][j]^2          a[j] = (float) sqrt(acc[j])   (identical to the calls above)
 *   CMPQ_NORM_L1    acc[j] += sum_t |X[t][j]|          a[j] = (float) acc[j]
 *   CMPQ_NORM_LINF  acc[j]  = max(acc[j], max_t |X[t][j]|)   a[j] = (float) acc[j]   (exact)
 * The criterion a then feeds cmpq_allocate_bits and cmpq_extract_outliers unchanged.  An unknown
 * norm is CMPQ_ERR_INVALID_ARG.  ws: cmpq_workspace_bytes(CMPQ_OP_COLLECT_STATS, d_in, 0). */
cmpq_status cmpq_collect_stats_norm(const void* X, cmpq_dtype dt, int64_t n_tokens, int64_t d_in,
                                    int64_t ldx, cmpq_norm norm, double* acc, int32_t* nonfinite, void* ws,
                                    size_t ws_bytes, void* stream);
cmpq_status cmpq_finalize_stats_norm(const double* acc, int64_t d_in, cmpq_norm norm, float* a,
                                     void* stream);

/* ---- allocation (Algorithm 1) ------------------------------------------------------------------
 * bits[i] in {2,3,4} from the statistic a (fp32, d_in entries, finite, >= 0) and the average
 * budget avg_bits in [2,4] (else CMPQ_ERR_INVALID_ARG).  order (optional, may be NULL) receives
 * the channel ids sorted ascending by (a, id).
 * ws: cmpq_workspace_bytes(CMPQ_OP_ALLOCATE_BITS, d_in, 0). */
cmpq_status cmpq_allocate_bits(const float* a, int64_t d_in, double avg_bits, cmpq_alloc_mode mode,
                               uint8_t* bits, int32_t* order, void* ws, size_t ws_bytes,
                               void* stream);

/* ---- outlier protection (Section 3.2.2) ------------------------------------------------------
 * O_act: the n_act channels with the largest (a, id), kept whole.  W' = W with those rows set
 * to +0.  Every channel of W' is fitted by K-means with K = 2^bits[i] and lloyd_iters updates
 * (start, tie and rounding rules: see cmpq_quantize_layer).  O_q: the n_q entries outside O_act
 * rows with the largest fp32 error |W' - W'_q|, equal errors by smaller i*d_out + j.
 * Output: the union as coordinate lists sorted by (row, col); vals are the original 16-bit
 * patterns of W.  nnz_out must equal n_act*d_out + n_q (the arrays' length).
 * W is [d_in][ldw] of `dt`, ldw >= d_out, 1 <= d_out <= CMPQ_MAX_D_OUT.
 * 0 <= n_act <= d_in, 0 <= n_q <= (d_in - n_act)*d_out.
 * ws: cmpq_workspace_bytes(CMPQ_OP_EXTRACT_OUTLIERS, d_in, d_out): about 5 bytes per weight of value
 * tables (2-byte key and 2-byte count prefix per possible distinct value, sums at every eighth), or one
 * fp32 error per weight while CMPQ_ASSIGN_ALL_PAIRS is selected -- cmpq_workspace_bytes answers for the
 * assignment method selected at the time it is asked. */
cmpq_status cmpq_extract_outliers(const void* W, cmpq_dtype dt, int64_t d_in, int64_t d_out,
                                  int64_t ldw, const float* a, const uint8_t* bits, int64_t n_act,
                                  int64_t n_q, int lloyd_iters, int32_t* rows, int32_t* cols,
                                  uint16_t* vals, int64_t nnz_out, int32_t* nonfinite, void* ws,
                                  size_t ws_bytes, void* stream);

/* ---- channel-wise non-uniform quantization (Sections 3 and 3.2.1, final step of 3.2.2) -------
 * W'' = W with the nnz listed positions (sorted by (row, col), e.g. from cmpq_extract_outliers;
 * rows/cols may be NULL when nnz == 0) set to +0.  For every channel i, K = 2^bits[i]:
 *   start       c_k = the ((2k+1) d_out)/(2K)-th smallest value (integer division)
 *   assignment  the first k minimising fabsf(x - c_k) in fp32
 *   update      c_k = (float)(sum of members in fp64 / count); an empty cluster keeps c_k
 * exactly lloyd_iters updates (1..CMPQ_MAX_LLOYD_ITERS; 0 is allowed and returns the start),
 * then a last assignment.  lut: [d_in][CMPQ_LUT_STRIDE] fp32, the first K entries valid, the
 * rest 0.  codes: [d_in][d_out] uint8, 8-byte aligned (else CMPQ_ERR_INVALID_ARG).
 * sens: NULL for the paper's unweighted K-means.  Otherwise [d_in][d_out] fp32 sensitivities s >= 0
 * (finite), one per weight: the update becomes the weighted mean  c_k = sum s x / sum s  over the
 * members (a cluster whose members' sensitivities sum to 0 keeps c_k); start and assignment are
 * unchanged.  The weighted sums are not exact in fp64, so they depend on the order of summation: the
 * result is deterministic (the same inputs give the same bytes) and agrees with a sequential sum to
 * rounding (centroids to about 1e-7 relative); with all s equal to one power of two it equals the
 * unweighted fit bit for bit whenever inexact_rows stays 0 there.  With CMPQ_ASSIGN_ORDERED the fit
 * works on the value tables: the sensitivities of the weights that share a value are added in 64-bit
 * fixed point (scaled by a power of two so that a channel's total stays below 2^52; a sensitivity
 * below 2^-(52 - ceil(log2 d_out)) of the channel's largest loses its low bits), and cluster sums are
 * differences of fp64 prefix sums over the distinct values.  With CMPQ_ASSIGN_ALL_PAIRS, and for a
 * channel with more than 11264 distinct values, every weight is scanned against every centroid in
 * every iteration.  inexact_rows is left untouched.
 * inexact_rows (optional device int32, caller zeroes it): incremented for every channel whose
 * dynamic range is so wide that fp64 cluster sums may depend on the order of summation; when
 * it stays 0 the centroids are independent of the summation order, hence reproducible bit
 * for bit by any other correct implementation.
 * sweeps (optional device uint64, caller zeroes it): receives, summed over the channels,
 * (assignment steps executed) * d_out * K, i.e. the number of (weight, centroid) distance
 * evaluations that assigning every weight against every centroid costs.  CMPQ_ASSIGN_ALL_PAIRS
 * performs exactly that many; CMPQ_ASSIGN_ORDERED reaches the same result with far fewer.
 * ws: cmpq_workspace_bytes(CMPQ_OP_QUANTIZE_LAYER, d_in, d_out). */
cmpq_status cmpq_quantize_layer(const void* W, cmpq_dtype dt, int64_t d_in, int64_t d_out,
                                int64_t ldw, const uint8_t* bits, const int32_t* rows,
                                const int32_t* cols, int64_t nnz, int lloyd_iters,
                                const float* sens, float* lut, uint8_t* codes,
                                int32_t* inexact_rows, unsigned long long* sweeps, int32_t* nonfinite,
                                void* ws, size_t ws_bytes, void* stream);

/* ---- outlier protection and quantization in one call (Section 3.2.2 with its final step) -------
 * Exactly cmpq_extract_outliers followed by cmpq_quantize_layer on the list it produced: the same
 * arguments, the same outputs bit for bit (rows/cols/vals, lut, codes, inexact_rows, sweeps of the
 * final fit).  Knowing both steps lets the library derive the value tables of the final fit from
 * those of the provisional fit (the two weight matrices differ only at the kept entries) instead
 * of reading and counting every weight a second time.
 * ws: cmpq_workspace_bytes(CMPQ_OP_PROTECT_AND_QUANTIZE, d_in, d_out). */
cmpq_status cmpq_protect_and_quantize(const void* W, cmpq_dtype dt, int64_t d_in, int64_t d_out,
                                      int64_t ldw, const float* a, const uint8_t* bits, int64_t n_act,
                                      int64_t n_q, int lloyd_iters, int32_t* rows, int32_t* cols,
                                      uint16_t* vals, int64_t nnz_out, float* lut, uint8_t* codes,
                                      int32_t* inexact_rows, unsigned long long* sweeps, int32_t* nonfinite,
                                      void* ws, size_t ws_bytes, void* stream);

/* ---- budget sweeps (the paper's limitations paragraph: a new memory budget means quantizing again) --
 * The value tables of a layer's channels depend on the weights alone, and a channel's provisional
 * K-means fit on its width and the iteration count alone.  A sweep over several budgets on the same
 * weights therefore keeps both in a caller-owned cache:
 *   cmpq_sweep_begin   counts the values of every channel of W once (no statistic needed) and marks the
 *                      cache empty of fits; lloyd_iters is the count every later call will use.
 *   cmpq_sweep_budget  is cmpq_protect_and_quantize -- same arguments, same outputs bit for bit -- except
 *                      that the provisional fit reads the cached tables, copies the fits already made for
 *                      a (channel, width) pair and adds the new ones to the cache.  W, d_in, d_out, ldw
 *                      and lloyd_iters must be those of cmpq_sweep_begin (a different lloyd_iters is
 *                      detected on the device and simply bypasses the kept fits); a, bits, n_act and n_q
 *                      may change from call to call.
 * cache: cmpq_sweep_cache_bytes(d_in, d_out) bytes of device memory, 256-byte aligned, untouched by the
 * caller between the calls (else CMPQ_ERR_WORKSPACE).  Calls on one cache must be ordered (one stream, or
 * streams joined by events: cmpq_sweep_begin needs the weights alone and may run beside the statistic).
 * With CMPQ_ASSIGN_ALL_PAIRS selected the cache is ignored.
 *   cmpq_sweep_budget_pack  is cmpq_protect_quantize_pack with the same use of the cache (the last assignment
 *                      writes the packed words; codes may be NULL).
 * ws of cmpq_sweep_budget: cmpq_workspace_bytes(CMPQ_OP_PROTECT_AND_QUANTIZE, d_in, d_out); of
 * cmpq_sweep_budget_pack: cmpq_workspace_bytes(CMPQ_OP_PROTECT_QUANTIZE_PACK, d_in, d_out). */
size_t cmpq_sweep_cache_bytes(int64_t d_in, int64_t d_out);
cmpq_status cmpq_sweep_begin(const void* W, cmpq_dtype dt, int64_t d_in, int64_t d_out, int64_t ldw,
                             int lloyd_iters, int32_t* nonfinite, void* cache, size_t cache_bytes, void* stream);
cmpq_status cmpq_sweep_budget(const void* W, cmpq_dtype dt, int64_t d_in, int64_t d_out, int64_t ldw,
                              const float* a, const uint8_t* bits, int64_t n_act, int64_t n_q,
                              int lloyd_iters, int32_t* rows, int32_t* cols, uint16_t* vals,
                              int64_t nnz_out, float* lut, uint8_t* codes, int32_t* inexact_rows,
                              unsigned long long* sweeps, void* cache, size_t cache_bytes, void* ws,
                              size_t ws_bytes, void* stream);
cmpq_status cmpq_sweep_budget_pack(const void* W, cmpq_dtype dt, int64_t d_in, int64_t d_out, int64_t ldw,
                                   const float* a, const uint8_t* bits, int64_t n_act, int64_t n_q,
                                   int lloyd_iters, int32_t* rows, int32_t* cols, uint16_t* vals,
                                   int64_t nnz_out, float* lut, uint8_t* codes, uint32_t* packed,
                                   int64_t* row_off, int32_t* perm, int64_t* seg_rows, int32_t* inexact_rows,
                                   unsigned long long* sweeps, void* cache, size_t cache_bytes, void* ws,
                                   size_t ws_bytes, void* stream);

/* Process-wide choice of the assignment method used by cmpq_extract_outliers and
 * cmpq_quantize_layer from the next call on (host state, no GPU work; thread-safe).
 * CMPQ_ERR_INVALID_ARG for an unknown value. */
cmpq_status cmpq_set_lloyd_assignment(cmpq_lloyd_assignment mode);
cmpq_lloyd_assignment cmpq_get_lloyd_assignment(void);

/* Timing aid for CMPQ_ASSIGN_ORDERED, which runs three kernels per K-means call (value table,
 * iterations, last assignment): the four cudaEvent_t handles given here are recorded on the call's
 * stream before the first and after each of the three kernels by the NEXT cmpq_extract_outliers or
 * cmpq_quantize_layer call, once; the library keeps no reference afterwards.  Pass four NULLs to
 * cancel; any other mix of NULLs is CMPQ_ERR_INVALID_ARG.  The events stay owned by the caller. */
cmpq_status cmpq_lloyd_phase_events(void* before_table, void* after_table, void* after_iterate,
                                    void* after_assign);

/* ---- packing (accounting of Section 5.1; per-precision sub-matrices of Section 6) -----------
 * Three segments in the order 2-, 3-, 4-bit channels, channels by ascending id inside a
 * segment.  perm[r] = channel stored at position r; row_off[r] = its first 32-bit word
 * (row_off[d_in] = total words = cmpq_packed_words); seg_rows[0..2] = channels per segment.
 * A channel's codes form an LSB-first bit stream (code j at bits [j*c, (j+1)*c)) cut into
 * little-endian 32-bit words, the last one zero padded.  packed must hold
 * cmpq_packed_words() words.  seg_rows is a DEVICE array of 3 int64.
 * ws: cmpq_workspace_bytes(CMPQ_OP_PACK, d_in, d_out). */
cmpq_status cmpq_pack(const uint8_t* codes, const uint8_t* bits, int64_t d_in, int64_t d_out,
                      uint32_t* packed, int64_t* row_off, int32_t* perm, int64_t* seg_rows,
                      void* ws, size_t ws_bytes, void* stream);

/* ---- final fit and packing in one call (Sections 3.2.1 / 3.2.2 with the storage of Section 5.1) ------
 * cmpq_quantize_layer_packed = cmpq_quantize_layer followed by cmpq_pack, and
 * cmpq_protect_quantize_pack = cmpq_protect_and_quantize followed by cmpq_pack: the same arguments and
 * the same outputs bit for bit (lut, codes, packed, row_off, perm, seg_rows, ...).  The last assignment
 * of the K-means writes the bit streams itself (the four threads that hold 32 neighbouring codes form
 * the 2, 3 or 4 words of that group), so the byte codes need not exist: codes may be NULL, and then
 * they are neither written nor read anywhere -- the call moves 2 bytes per weight less than the two
 * separate calls.  With CMPQ_ASSIGN_ALL_PAIRS selected, or with sensitivities given, the kernels still
 * produce byte codes: codes == NULL is then CMPQ_ERR_UNSUPPORTED, otherwise the packing runs as a
 * separate step inside the call.  packed must hold cmpq_packed_words() words.
 * ws: cmpq_workspace_bytes(CMPQ_OP_QUANTIZE_LAYER_PACKED / CMPQ_OP_PROTECT_QUANTIZE_PACK, d_in, d_out). */
cmpq_status cmpq_quantize_layer_packed(const void* W, cmpq_dtype dt, int64_t d_in, int64_t d_out,
                                       int64_t ldw, const uint8_t* bits, const int32_t* rows,
                                       const int32_t* cols, int64_t nnz, int lloyd_iters, const float* sens,
                                       float* lut, uint8_t* codes, uint32_t* packed, int64_t* row_off,
                                       int32_t* perm, int64_t* seg_rows, int32_t* inexact_rows,
                                       unsigned long long* sweeps, int32_t* nonfinite, void* ws, size_t ws_bytes,
                                       void* stream);
cmpq_status cmpq_protect_quantize_pack(const void* W, cmpq_dtype dt, int64_t d_in, int64_t d_out, int64_t ldw,
                                       const float* a, const uint8_t* bits, int64_t n_act, int64_t n_q,
                                       int lloyd_iters, int32_t* rows, int32_t* cols, uint16_t* vals,
                                       int64_t nnz_out, float* lut, uint8_t* codes, uint32_t* packed,
                                       int64_t* row_off, int32_t* perm, int64_t* seg_rows,
                                       int32_t* inexact_rows, unsigned long long* sweeps, int32_t* nonfinite,
                                       void* ws, size_t ws_bytes, void* stream);

/* ---- inference product of one token (Section 6: the figure of the real quantization process) ----
 * The input vector is split by the precision of its channels, every part multiplies its 2-, 3- or
 * 4-bit weight sub-matrix through the channel's look-up table, the 16-bit outliers multiply the
 * original input, and all products are accumulated:
 *     y[j] = sum_i x[i] * lut[i][code_ij]  +  sum over outliers (i, j, v) of x[i] * v .
 * packed, row_off, perm, seg_rows: exactly what cmpq_pack wrote for a [d_in][d_out] layer (the
 * codes are read from the packed segments; the byte codes are not needed).  lut: [d_in][16] fp32
 * as written by cmpq_quantize_layer.  x: d_in values of `dt`.  col_ptr / c_rows / c_vals: the
 * outliers grouped by column as written by cmpq_outliers_by_column (values of the same `dt`), or
 * three NULLs for a layer without outliers.  y: d_out fp32.  y16 (optional, may be NULL): the same
 * result rounded to nearest even into `dt` (the paper accumulates into 16-bit outputs).
 * Arithmetic: fp32; x[i]*lut[i][k] is formed once per table entry (for 2- and 3-bit channels the
 * entries of two neighbouring channels are added into one table first), a column's sum is taken
 * over blocks of channels in a fixed order, so the result is deterministic and differs from the
 * exact sum by at most a few hundred units of 2^-24 relative to sum_i |x[i] * w_ij|.
 * The call enqueues two kernels, the second as a programmatic dependent of the first (it starts
 * early and waits for the first before it reads its results); both complete in stream order.
 * 1 <= d_out <= CMPQ_MAX_D_OUT.  ws: cmpq_workspace_bytes(CMPQ_OP_MATVEC, d_in, d_out). */
cmpq_status cmpq_matvec(const uint32_t* packed, const int64_t* row_off, const int32_t* perm,
                        const int64_t* seg_rows, const float* lut, int64_t d_in, int64_t d_out,
                        const void* x, cmpq_dtype dt, const int64_t* col_ptr, const int32_t* c_rows,
                        const uint16_t* c_vals, float* y, void* y16, void* ws, size_t ws_bytes,
                        void* stream);

/* The outlier list of cmpq_extract_outliers (sorted by (row, col)) regrouped by output column for
 * cmpq_matvec (Section 6 keeps the outliers in a compressed sparse format): col_ptr[j] ..
 * col_ptr[j+1] (d_out + 1 int64) delimits column j's entries in c_rows / c_vals (nnz entries
 * each), which are ascending by row inside a column.  (row, col) pairs must be distinct and
 * 0 <= col < d_out.  nnz may be 0 (then only col_ptr is written and the list pointers may be NULL).
 * ws: cmpq_workspace_bytes(CMPQ_OP_OUTLIERS_BY_COLUMN, 1, d_out). */
cmpq_status cmpq_outliers_by_column(const int32_t* rows, const int32_t* cols, const uint16_t* vals,
                                    int64_t nnz, int64_t d_out, int64_t* col_ptr, int32_t* c_rows,
                                    uint16_t* c_vals, void* ws, size_t ws_bytes, void* stream);

/* The same product with the tables in their stored FP16 format (Section 5.1: 16 bits per centroid):
 * lut16 is [d_in][16] binary16 patterns as written by cmpq_store_lut(CMPQ_LUT_F16), widened exactly
 * when read; everything else as cmpq_matvec.  (4-bit tables are expanded with cmpq_load_lut first.) */
cmpq_status cmpq_matvec_f16lut(const uint32_t* packed, const int64_t* row_off, const int32_t* perm,
                               const int64_t* seg_rows, const uint16_t* lut16, int64_t d_in, int64_t d_out,
                               const void* x, cmpq_dtype dt, const int64_t* col_ptr, const int32_t* c_rows,
                               const uint16_t* c_vals, float* y, void* y16, void* ws, size_t ws_bytes,
                               void* stream);

/* ---- stored formats of the look-up tables (Section 5.1, memory usage) ----------------------------
 * The final fit returns fp32 centroids.  The paper stores them in FP16 (one 4-bit width tag and K
 * 16-bit centroids per channel: (4 + 8*16)/4096 = 0.03 bit per weight at 3 bits and 4096 weights per
 * channel) and reports a variant with 4 bits per centroid ((4 + 8*4)/4096 < 0.01).
 *   CMPQ_LUT_F16  uint16 [d_in][16]: every centroid rounded to the nearest binary16 value, ties to even
 *                 (centroids beyond +-65504 become infinities); entries at k >= K are 0.
 *   CMPQ_LUT_U4   12 bytes per channel.  The paper gives only the accounting; the reading taken is its own
 *                 uniform quantizer (Section 3, N = 4) over the K centroids of the channel: lo / hi = the
 *                 smallest / largest centroid, each rounded to binary16; D = (hi - lo)/15;
 *                 code_k = clamp(round_half_even((c_k - lo)/D), 0, 15), 0 when D == 0; decoded centroid
 *                 lo + code_k * D; every step one fp32 operation.  Bytes 0..7: code 2b in the low and code
 *                 2b+1 in the high nibble of byte b (0 at k >= K); bytes 8..11: lo, hi as little-endian
 *                 binary16.  The two grid ends cost 32 bits per channel more than the paper's accounting.
 * cmpq_store_lut: lut [d_in][16] fp32 (16-byte aligned) -> stored (cmpq_lut_bytes(fmt, d_in) bytes, 4-byte
 * aligned).  cmpq_load_lut: the inverse, fp32 tables that cmpq_matvec reads.  CMPQ_LUT_F32 is refused by
 * both (nothing to convert).  cmpq_table_bits_per_weight (host, bits_host is a HOST array): the paper's
 * accounting, (4 + K * bits per centroid [+ 32 for the 4-bit format's grid ends]) / d_out averaged over
 * the channels. */
typedef enum { CMPQ_LUT_F32 = 0, CMPQ_LUT_F16 = 1, CMPQ_LUT_U4 = 2 } cmpq_lut_format;
#define CMPQ_LUT_U4_BYTES 12
size_t cmpq_lut_bytes(cmpq_lut_format fmt, int64_t d_in);
cmpq_status cmpq_store_lut(const float* lut, const uint8_t* bits, int64_t d_in, cmpq_lut_format fmt, void* stored,
                           void* stream);
cmpq_status cmpq_load_lut(const void* stored, cmpq_lut_format fmt, const uint8_t* bits, int64_t d_in, float* lut,
                          void* stream);
double cmpq_table_bits_per_weight(const uint8_t* bits_host, int64_t d_in, int64_t d_out, cmpq_lut_format fmt,
                                  int count_grid_ends);

/* ---- layout conversion (Section 3.2.1: W in R^{d_in x d_out}, a channel is the row W_{i,:}) ----
 * Frameworks store a linear layer output-major, [d_out][d_in]; every call above takes the paper's
 * input-channel-major layout.  dst[c*ld_dst + r] = src[r*ld_src + c] for a [rows][cols] source of
 * 16-bit elements (raw patterns, fp16 or bf16 alike): call it with rows = d_out, cols = d_in to get
 * W [d_in][ld_dst >= d_out].  src and dst must not overlap.  1 <= rows, cols <= CMPQ_MAX_D_IN,
 * ld_src >= cols, ld_dst >= rows, else CMPQ_ERR_INVALID_ARG.  No work space. */
cmpq_status cmpq_transpose16(const void* src, int64_t rows, int64_t cols, int64_t ld_src, void* dst,
                             int64_t ld_dst, void* stream);

/* ---- measurement aids (no counterpart in the paper; nothing here is on the quantization path) ------
 * cmpq_alu_probe enqueues a kernel that performs, on register operands only and in eight independent
 * chains per thread, the arithmetic of a brute-force nearest-centroid assignment (Section 3): per
 * (value, centroid) pair one fp32 subtract and one compare/select (min of magnitudes).  `blocks` blocks of
 * 256 threads run `rounds` rounds of 8 x 16 pairs each; *evaluations (host, optional) receives the number
 * of pairs the launch evaluates, so 2 * evaluations / (event-timed duration) is this GPU's ceiling, at the
 * clocks of the moment, for the two-operation mix an all-pairs assignment needs.  sink: device scratch of
 * blocks * 256 floats (never written in practice).  1 <= rounds <= 2^24, 1 <= blocks <= 2^20. */
cmpq_status cmpq_alu_probe(int rounds, int blocks, float* sink, unsigned long long* evaluations, void* stream);

/* Registers per thread and static shared memory of a kernel of this library, as compiled (host call, no
 * GPU work).  Lets a stored profile of a kernel be recognised as stale after the kernel has changed. */
typedef enum {
    CMPQ_KERNEL_STATS_PARTIAL_VEC_BF16 = 0,   /* column reduction of cmpq_collect_stats, bf16, l2 */
    CMPQ_KERNEL_LLOYD_TABLE_BF16_4096 = 1     /* value-table kernel, bf16, 2048 < d_out <= 4096 */
} cmpq_kernel;
cmpq_status cmpq_kernel_resources(cmpq_kernel k, int* registers, int* static_smem_bytes);

/* ---- host helpers (pure functions, no GPU work) ----------------------------------------------- */
size_t cmpq_workspace_bytes(cmpq_op op, int64_t d_in, int64_t d_out);
/* Algorithm 1 in rank form: how many channels get 2 and 4 bits. */
void cmpq_alloc_counts(int64_t d_in, double avg_bits, int64_t* n2, int64_t* n4);
/* Section 3.2.2 budget: n_act = 45*d_in/10000, n_q = 5*d_in*d_out/10000 (integer division). */
void cmpq_default_counts(int64_t d_in, int64_t d_out, int64_t* n_act, int64_t* n_q);
/* Sum over channels of ceil(d_out*bits/32); bits_host is a HOST array. */
int64_t cmpq_packed_words(const uint8_t* bits_host, int64_t d_in, int64_t d_out);
const char* cmpq_status_string(cmpq_status s);

#ifdef __cplusplus
}
#endif
#endif /* CMPQ_H_ */
