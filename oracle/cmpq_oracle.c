/*
 * CMPQ oracle -- TEST INFRASTRUCTURE, NOT A PRODUCT PATH.
 *
 * A plain, slow, single-threaded CPU restatement of the CMPQ post-training
 * quantization pass for one linear layer (channel-wise mixed-precision
 * quantization, arxiv 2410.13056).  It exists only so that tests, the smoke
 * check and the benchmark's CPU-baseline leg can compare the CUDA library
 * against it.  It shares no code, header, table or helper with the CUDA
 * library and must never be called from it.
 *
 * Every function names the passage of the paper it follows.  Where the paper is
 * silent the reading taken is stated next to the code.  Floating point: sums in
 * fp64, distances in fp32 (a single subtraction and absolute value), no
 * blocking, no fusion, no reordering.  Compile with -O2 -ffp-contract=off and
 * never with -ffast-math.
 *
 * Notation (paper, Section 3.2.1): W in R^{d_in x d_out}, a channel is the row
 * W_{i,:} (one input channel, d_out weights); X in R^{n x d_in}; a in R^{d_in}
 * is the per-channel L2 norm of X; c in {2,3,4}^{d_in} the allocated bits;
 * K = 2^c centroids per channel.
 *
 * Pins (tests/test_oracle_*.py): closed forms for the statistic, allocation
 * invariants and numpy argsort, exhaustive optimal 1-D clustering on <= 16
 * points, sklearn's Lloyd from the same start, full-sort top-k, pack/unpack
 * round trip, the storage figures the paper prints; for the inference product:
 * unit inputs, exactly representable layers, a dense float64 matrix product and
 * the reconstruction error of the same layer; for the l1 / l_inf statistics:
 * numpy's vector norms, closed forms, chunking and the norm inequalities; for
 * the weighted update: constant weights change nothing, every non-empty
 * centroid is its members' weighted mean; for the stored table formats: numpy's
 * float16 conversion on every binade and rounding case, the grid end points, the
 * half-step error bound and a hand-worked channel.
 * Parity unpinned: none of the paper's perplexity tables can pin the
 * reconstruction error (no model weights exist here); oracle_recon_error is
 * pinned only against a dense float64 numpy evaluation of the same definition.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORACLE_F16 0
#define ORACLE_BF16 1

/* ---------------------------------------------------------------------------
 * 16-bit storage formats -> float (exact widening).
 * ------------------------------------------------------------------------- */
static float bits_to_float(uint32_t u) {
    float f;
    memcpy(&f, &u, 4);
    return f;
}

/* IEEE binary16: 1 sign, 5 exponent (bias 15), 10 fraction bits. */
static float half_to_float(uint16_t h) {
    int sign = (h >> 15) & 1;
    int e = (h >> 10) & 0x1f;
    int m = h & 0x3ff;
    double v;
    if (e == 0) {
        v = ldexp((double)m, -24); /* subnormal: m * 2^-10 * 2^-14 */
    } else if (e == 31) {
        v = m ? NAN : INFINITY;
    } else {
        v = ldexp((double)(1024 + m), e - 25); /* (1 + m/1024) * 2^(e-15) */
    }
    return (float)(sign ? -v : v);
}

/* bfloat16 is the upper half of an IEEE binary32. */
static float bf16_to_float(uint16_t h) { return bits_to_float((uint32_t)h << 16); }

float oracle_widen(uint16_t h, int dtype) {
    return dtype == ORACLE_F16 ? half_to_float(h) : bf16_to_float(h);
}

/* ---------------------------------------------------------------------------
 * Step 1.  Activation statistic (Section 3.2.1: the L2 norm of every column of X).
 *   sumsq_j += sum_t X[t,j]^2   in token order, fp64
 *   a_j      = (float) sqrt(sumsq_j)
 * The caller zeroes sumsq before the first chunk of tokens.
 * ------------------------------------------------------------------------- */
void oracle_collect_stats(const uint16_t* X, int dtype, int64_t n_tokens, int64_t d_in,
                          int64_t ldx, double* sumsq) {
    for (int64_t t = 0; t < n_tokens; ++t) {
        for (int64_t j = 0; j < d_in; ++j) {
            double x = (double)oracle_widen(X[t * ldx + j], dtype);
            sumsq[j] += x * x;
        }
    }
}

void oracle_finalize_stats(const double* sumsq, int64_t d_in, float* a) {
    for (int64_t j = 0; j < d_in; ++j) a[j] = (float)sqrt(sumsq[j]);
}

/* Other activation norms as the allocation criterion (appendix, norm ablation table:
 * the l1 and l_inf norms of the channel's activations are compared with l2).
 * norm 1: acc_j += sum_t |X[t,j]| ; norm 2 (l_inf): acc_j = max(acc_j, max_t |X[t,j]|);
 * norm 0 is the l2 statistic above.  The criterion a_j is acc_j itself (rounded to
 * fp32) for l1 and l_inf, its square root for l2. */
void oracle_collect_stats_norm(const uint16_t* X, int dtype, int64_t n_tokens, int64_t d_in,
                               int64_t ldx, int norm, double* acc) {
    for (int64_t t = 0; t < n_tokens; ++t)
        for (int64_t j = 0; j < d_in; ++j) {
            double x = (double)oracle_widen(X[t * ldx + j], dtype);
            if (norm == 0) acc[j] += x * x;
            else if (norm == 1) acc[j] += fabs(x);
            else if (fabs(x) > acc[j]) acc[j] = fabs(x);
        }
}

void oracle_finalize_stats_norm(const double* acc, int64_t d_in, int norm, float* a) {
    for (int64_t j = 0; j < d_in; ++j) a[j] = (float)(norm == 0 ? sqrt(acc[j]) : acc[j]);
}

/* ---------------------------------------------------------------------------
 * Step 2.  Channel-wise precision allocation (Algorithm 1).
 *
 * Reading of "q-quantile" (the paper does not define it):
 *  mode 0 (rank form, default): the number of channels that leave 3 bits is
 *     n = floor(|b-3| * d_in + 1/2); for b > 3 the n channels with the largest
 *     (a, index) get 4 bits, for b < 3 the n smallest get 2 bits, and for
 *     b == 3 exactly the bottom and the top floor(0.01*d_in + 1/2) channels get
 *     2 and 4 bits ("1st" and "99th" quantile).  This meets the budget to
 *     within 1/(2 d_in) and exactly when |b-3|*d_in is an integer.
 *  mode 1 (literal form): thresholds are linearly interpolated quantiles of a
 *     (position q*(d_in-1) in the ascending order statistics, fp64) compared
 *     strictly, exactly as the algorithm is printed.
 * ------------------------------------------------------------------------- */
void oracle_alloc_counts(int64_t d_in, double avg_bits, int64_t* n2, int64_t* n4) {
    *n2 = 0;
    *n4 = 0;
    if (avg_bits == 3.0) {
        int64_t n = (int64_t)floor(0.01 * (double)d_in + 0.5);
        *n2 = n;
        *n4 = n;
    } else {
        double t = fabs(avg_bits - 3.0) * (double)d_in;
        int64_t n = (int64_t)floor(t + 0.5);
        if (n > d_in) n = d_in;
        if (avg_bits > 3.0) *n4 = n; else *n2 = n;
    }
}

typedef struct { float a; int32_t idx; } key_idx;

static int cmp_key_idx(const void* pa, const void* pb) {
    const key_idx* x = (const key_idx*)pa;
    const key_idx* y = (const key_idx*)pb;
    if (x->a < y->a) return -1;
    if (x->a > y->a) return 1;
    return (x->idx > y->idx) - (x->idx < y->idx);
}

/* order[r] = id of the channel of rank r when channels are sorted ascending by
 * a, equal values by ascending id. */
static void rank_channels(const float* a, int64_t d_in, int32_t* order) {
    key_idx* keys = (key_idx*)malloc((size_t)d_in * sizeof(key_idx));
    for (int64_t i = 0; i < d_in; ++i) { keys[i].a = a[i]; keys[i].idx = (int32_t)i; }
    qsort(keys, (size_t)d_in, sizeof(key_idx), cmp_key_idx);
    for (int64_t r = 0; r < d_in; ++r) order[r] = keys[r].idx;
    free(keys);
}

static double interp_quantile(const float* a, const int32_t* order, int64_t d_in, double q) {
    double pos = q * (double)(d_in - 1);
    if (pos < 0.0) pos = 0.0;
    if (pos > (double)(d_in - 1)) pos = (double)(d_in - 1);
    int64_t lo = (int64_t)floor(pos);
    int64_t hi = lo + 1 < d_in ? lo + 1 : lo;
    double frac = pos - (double)lo;
    double vlo = (double)a[order[lo]];
    double vhi = (double)a[order[hi]];
    return vlo + (vhi - vlo) * frac;
}

/* returns 0, or 1 if avg_bits is outside [2,4] (Algorithm 1 requires b in [2,4]) */
int oracle_allocate_bits(const float* a, int64_t d_in, double avg_bits, int mode,
                         uint8_t* bits, int32_t* order_out) {
    if (!(avg_bits >= 2.0 && avg_bits <= 4.0) || d_in < 1) return 1;
    int32_t* order = (int32_t*)malloc((size_t)d_in * sizeof(int32_t));
    rank_channels(a, d_in, order);
    for (int64_t i = 0; i < d_in; ++i) bits[i] = 3; /* every channel starts at 3 bits */
    if (mode == 0) {
        int64_t n2, n4;
        oracle_alloc_counts(d_in, avg_bits, &n2, &n4);
        for (int64_t r = 0; r < n2; ++r) bits[order[r]] = 2;
        for (int64_t r = d_in - n4; r < d_in; ++r) bits[order[r]] = 4;
    } else {
        if (avg_bits > 3.0) {
            double l = interp_quantile(a, order, d_in, 1.0 - (avg_bits - 3.0));
            for (int64_t i = 0; i < d_in; ++i) if ((double)a[i] > l) bits[i] = 4;
        } else if (avg_bits < 3.0) {
            double s = interp_quantile(a, order, d_in, 3.0 - avg_bits);
            for (int64_t i = 0; i < d_in; ++i) if ((double)a[i] < s) bits[i] = 2;
        } else {
            double s = interp_quantile(a, order, d_in, 0.01);
            double l = interp_quantile(a, order, d_in, 0.99);
            for (int64_t i = 0; i < d_in; ++i) {
                if ((double)a[i] < s) bits[i] = 2;
                if ((double)a[i] > l) bits[i] = 4;
            }
        }
    }
    if (order_out) memcpy(order_out, order, (size_t)d_in * sizeof(int32_t));
    free(order);
    return 0;
}

/* Outlier counts (Section 3.2.2: 0.45 % of the channels, 0.05 % of the
 * entries); integer division so that the 0.5 % budget is never exceeded. */
void oracle_default_counts(int64_t d_in, int64_t d_out, int64_t* n_act, int64_t* n_q) {
    *n_act = (45 * d_in) / 10000;
    *n_q = (5 * d_in * d_out) / 10000;
}

/* ---------------------------------------------------------------------------
 * Channel-wise K-means (Section 3.2.1: every channel W_{i,:} is clustered on its
 * own with K = 2^bits centroids, e.g. K = 8 at 3 bits; quantizer of Section 3:
 * a value is replaced by the centroid nearest to it).
 *
 * The paper fixes neither the start, the iteration count, the handling of empty
 * clusters nor the rounding.  Reading taken:
 *   start      c_k = xs[((2k+1) N) / (2K)], xs = x sorted ascending (K evenly
 *              spaced order statistics, integer division)
 *   assignment first k minimising fabsf(x_i - c_k): fp32 subtraction, strict '<'
 *              scan k = 0..K-1, so that equal distances go to the lowest index
 *   update     S_k = sum of (double)x_i over the members (or sum s_i x_i),
 *              n_k = member count (or sum s_i); c_k = (float)(S_k / n_k) when the
 *              cluster has a member, unchanged otherwise
 *   exactly T updates, then one last assignment, which also gives
 *   err_i = min_k |x_i - c_k| (fp32).
 * x is canonicalised with x + 0.0f so that -0 and +0 are the same point.
 * sse_trace (optional, T+1 doubles) receives the fp64 sum of squared distances
 * of every assignment, in order.
 * ------------------------------------------------------------------------- */
static int cmp_float(const void* pa, const void* pb) {
    float x = *(const float*)pa, y = *(const float*)pb;
    return (x > y) - (x < y);
}

static double assign_all(const float* x, int64_t N, const float* c, int K, uint8_t* code,
                         float* err) {
    double sse = 0.0;
    for (int64_t i = 0; i < N; ++i) {
        float best = fabsf(x[i] - c[0]);
        int bk = 0;
        for (int k = 1; k < K; ++k) {
            float d = fabsf(x[i] - c[k]);
            if (d < best) { best = d; bk = k; }
        }
        code[i] = (uint8_t)bk;
        if (err) err[i] = best;
        sse += (double)best * (double)best;
    }
    return sse;
}

void oracle_lloyd(const float* x_in, int64_t N, int K, int T, const double* s, float* lut,
                  uint8_t* code, float* err, double* sse_trace) {
    float* x = (float*)malloc((size_t)N * sizeof(float));
    float* xs = (float*)malloc((size_t)N * sizeof(float));
    for (int64_t i = 0; i < N; ++i) x[i] = x_in[i] + 0.0f;
    memcpy(xs, x, (size_t)N * sizeof(float));
    qsort(xs, (size_t)N, sizeof(float), cmp_float);
    float c[16];
    for (int k = 0; k < K; ++k) c[k] = xs[((int64_t)(2 * k + 1) * N) / (2 * (int64_t)K)];
    for (int it = 0; it < T; ++it) {
        double sse = assign_all(x, N, c, K, code, NULL);
        if (sse_trace) sse_trace[it] = sse;
        double S[16], n[16];
        for (int k = 0; k < K; ++k) { S[k] = 0.0; n[k] = 0.0; }
        for (int64_t i = 0; i < N; ++i) {
            if (s) { S[code[i]] += s[i] * (double)x[i]; n[code[i]] += s[i]; }
            else   { S[code[i]] += (double)x[i];        n[code[i]] += 1.0; }
        }
        for (int k = 0; k < K; ++k) if (n[k] > 0.0) c[k] = (float)(S[k] / n[k]);
    }
    double sse = assign_all(x, N, c, K, code, err);
    if (sse_trace) sse_trace[T] = sse;
    for (int k = 0; k < 16; ++k) lut[k] = k < K ? c[k] : 0.0f;
    free(xs);
    free(x);
}

/* ---------------------------------------------------------------------------
 * Steps 3-6.  Outlier protection (Section 3.2.2).
 *   O_act : the n_act channels with the largest (a, index), kept whole.
 *   W'    : W with those rows set to +0  (W' = W - O_act).
 *   W'_q  : channel-wise K-means of W' with the allocated bits.
 *   O_q   : the n_q entries outside O_act rows with the largest |W' - W'_q|
 *           (fp32), equal errors by smaller linear index i*d_out + j; the
 *           selection is global over the matrix.
 *   O     : O_act + O_q as (row, col, original 16-bit pattern), sorted by
 *           (row, col).
 * Output arrays hold n_act*d_out + n_q entries.  lut1 (optional, d_in*16) and
 * err_out (optional, d_in*d_out; rows of O_act hold -1) expose the provisional
 * fit for tests.  Returns 0, or 1 on bad arguments.
 * ------------------------------------------------------------------------- */
typedef struct { float err; int64_t idx; } err_idx;

static int cmp_err_idx(const void* pa, const void* pb) {
    const err_idx* x = (const err_idx*)pa;
    const err_idx* y = (const err_idx*)pb;
    if (x->err > y->err) return -1; /* larger error first */
    if (x->err < y->err) return 1;
    return (x->idx > y->idx) - (x->idx < y->idx); /* then smaller index */
}

static int cmp_i64(const void* pa, const void* pb) {
    int64_t x = *(const int64_t*)pa, y = *(const int64_t*)pb;
    return (x > y) - (x < y);
}

int oracle_extract_outliers(const uint16_t* W, int dtype, int64_t d_in, int64_t d_out,
                            int64_t ldw, const float* a, const uint8_t* bits, int64_t n_act,
                            int64_t n_q, int T, int32_t* rows, int32_t* cols, uint16_t* vals,
                            float* lut1, float* err_out) {
    if (n_act < 0 || n_act > d_in || n_q < 0 || n_q > (d_in - n_act) * d_out) return 1;
    int32_t* order = (int32_t*)malloc((size_t)d_in * sizeof(int32_t));
    uint8_t* is_act = (uint8_t*)calloc((size_t)d_in, 1);
    rank_channels(a, d_in, order);
    for (int64_t r = d_in - n_act; r < d_in; ++r) is_act[order[r]] = 1;

    int64_t n_rest = (d_in - n_act) * d_out;
    err_idx* cand = (err_idx*)malloc((size_t)(n_rest > 0 ? n_rest : 1) * sizeof(err_idx));
    float* x = (float*)malloc((size_t)d_out * sizeof(float));
    float* err = (float*)malloc((size_t)d_out * sizeof(float));
    uint8_t* code = (uint8_t*)malloc((size_t)d_out);
    float lut[16];
    int64_t m = 0;
    for (int64_t i = 0; i < d_in; ++i) {
        for (int64_t j = 0; j < d_out; ++j)
            x[j] = is_act[i] ? 0.0f : oracle_widen(W[i * ldw + j], dtype);
        oracle_lloyd(x, d_out, 1 << bits[i], T, NULL, lut, code, err, NULL);
        if (lut1) memcpy(lut1 + i * 16, lut, sizeof(lut));
        for (int64_t j = 0; j < d_out; ++j) {
            if (err_out) err_out[i * d_out + j] = is_act[i] ? -1.0f : err[j];
            if (!is_act[i]) { cand[m].err = err[j]; cand[m].idx = i * d_out + j; ++m; }
        }
    }
    qsort(cand, (size_t)m, sizeof(err_idx), cmp_err_idx);

    /* union of the O_act rows and the n_q selected entries, sorted by (row, col) */
    int64_t nnz = n_act * d_out + n_q;
    int64_t* lin = (int64_t*)malloc((size_t)(nnz > 0 ? nnz : 1) * sizeof(int64_t));
    int64_t p = 0;
    for (int64_t i = 0; i < d_in; ++i)
        if (is_act[i]) for (int64_t j = 0; j < d_out; ++j) lin[p++] = i * d_out + j;
    for (int64_t r = 0; r < n_q; ++r) lin[p++] = cand[r].idx;
    qsort(lin, (size_t)nnz, sizeof(int64_t), cmp_i64);
    for (int64_t r = 0; r < nnz; ++r) {
        int64_t i = lin[r] / d_out, j = lin[r] % d_out;
        rows[r] = (int32_t)i;
        cols[r] = (int32_t)j;
        vals[r] = W[i * ldw + j];
    }
    free(lin); free(code); free(err); free(x); free(cand); free(is_act); free(order);
    return 0;
}

/* ---------------------------------------------------------------------------
 * Step 7.  Final quantization (Section 3.2.2: "Two types of outliers
 * O = O_act + O_q are removed from the weight matrix W, and the remaining
 * weights then undergo the quantization process to obtain W_q").
 * Removed entries become +0 and still take part in the clustering (W - O taken
 * literally); lut is [d_in][16] with the first 2^bits entries valid, rest 0.
 * sens (optional, [d_in][d_out], > 0) weights the centroid update only.
 * ------------------------------------------------------------------------- */
int oracle_quantize_layer(const uint16_t* W, int dtype, int64_t d_in, int64_t d_out, int64_t ldw,
                          const uint8_t* bits, const int32_t* rows, const int32_t* cols,
                          int64_t nnz, int T, const double* sens, float* lut, uint8_t* codes) {
    float* x = (float*)malloc((size_t)d_out * sizeof(float));
    int64_t p = 0;
    for (int64_t i = 0; i < d_in; ++i) {
        for (int64_t j = 0; j < d_out; ++j) x[j] = oracle_widen(W[i * ldw + j], dtype);
        while (p < nnz && rows[p] == i) { x[cols[p]] = 0.0f; ++p; }
        oracle_lloyd(x, d_out, 1 << bits[i], T, sens ? sens + i * d_out : NULL, lut + i * 16,
                     codes + i * d_out, NULL, NULL);
    }
    free(x);
    return p == nnz ? 0 : 1; /* rows must be sorted ascending */
}

/* ---------------------------------------------------------------------------
 * Step 8.  Bit-packing (Section 5.1 gives only the accounting: one small integer
 * per channel for its bit width, 2^c table entries, c bits per weight; the
 * inference figure of Section 6 groups the channels by precision).
 * Layout (ours): three segments in the order 2-bit, 3-bit, 4-bit channels;
 * inside a segment channels by ascending id (perm); the d_out codes of a
 * channel are an LSB-first bit stream (code j occupies bits [j*c, (j+1)*c))
 * cut into little-endian 32-bit words, the last word zero padded; row_off is
 * the exclusive prefix sum, in words, of ceil(d_out*c/32) in segment order.
 * ------------------------------------------------------------------------- */
int64_t oracle_packed_words(const uint8_t* bits, int64_t d_in, int64_t d_out) {
    int64_t words = 0;
    for (int64_t i = 0; i < d_in; ++i) words += (d_out * bits[i] + 31) / 32;
    return words;
}

void oracle_pack(const uint8_t* codes, const uint8_t* bits, int64_t d_in, int64_t d_out,
                 uint32_t* packed, int64_t* row_off, int32_t* perm, int64_t* seg_rows) {
    int64_t r = 0, off = 0;
    for (int c = 2; c <= 4; ++c) {
        seg_rows[c - 2] = 0;
        for (int64_t i = 0; i < d_in; ++i) {
            if (bits[i] != c) continue;
            int64_t words = (d_out * c + 31) / 32;
            perm[r] = (int32_t)i;
            row_off[r] = off;
            for (int64_t w = 0; w < words; ++w) packed[off + w] = 0;
            for (int64_t j = 0; j < d_out; ++j) {
                uint32_t code = codes[i * d_out + j];
                for (int t = 0; t < c; ++t) { /* one bit at a time */
                    int64_t pos = j * c + t;
                    if ((code >> t) & 1u) packed[off + pos / 32] |= 1u << (pos % 32);
                }
            }
            off += words;
            ++r;
            ++seg_rows[c - 2];
        }
    }
    row_off[d_in] = off;
}

void oracle_unpack(const uint32_t* packed, const int64_t* row_off, const int32_t* perm,
                   const uint8_t* bits, int64_t d_in, int64_t d_out, uint8_t* codes) {
    for (int64_t r = 0; r < d_in; ++r) {
        int64_t i = perm[r];
        int c = bits[i];
        for (int64_t j = 0; j < d_out; ++j) {
            uint32_t code = 0;
            for (int t = 0; t < c; ++t) {
                int64_t pos = j * c + t;
                code |= ((packed[row_off[r] + pos / 32] >> (pos % 32)) & 1u) << t;
            }
            codes[i * d_out + j] = (uint8_t)code;
        }
    }
}

/* Storage accounting of Section 5.1: bits per weight spent on the per-channel
 * metadata, i.e. (tag_bits + 2^c * lut_bits) / d_out averaged over channels. */
double oracle_metadata_bits_per_weight(const uint8_t* bits, int64_t d_in, int64_t d_out,
                                       int tag_bits, int lut_bits) {
    double total = 0.0;
    for (int64_t i = 0; i < d_in; ++i)
        total += (double)tag_bits + (double)(1 << bits[i]) * (double)lut_bits;
    return total / ((double)d_in * (double)d_out);
}

/* ---------------------------------------------------------------------------
 * Stored formats of the look-up tables (Section 5.1, memory usage: the tables are
 * kept in FP16, 16 bits per centroid, and a variant keeps them in 4 bits).
 *
 * FP16: every centroid is rounded to the nearest binary16 value, ties to even
 * (values beyond the binary16 range become infinities).
 *
 * 4 bit: the paper prints only the accounting, (1*4 + 8*4)/4096 bits per weight.
 * Reading taken: the uniform quantizer of Section 3 with N = 4 applied to the K
 * centroids of one channel.  lo and hi are the smallest and largest centroid of
 * the channel, each rounded to FP16 (they are stored with the codes: 32 more bits
 * per channel than the paper's accounting counts);  D = (hi - lo) / 15;
 * code_k = clamp(round((c_k - lo) / D), 0, 15) with round-half-to-even; D == 0
 * gives code 0.  Decoding: lo + code * D.  Every step is one fp32 operation
 * (subtract, divide, round, multiply, add), nothing fused.
 * Layout of a channel: 8 bytes of codes (code 2b in the low, code 2b+1 in the high
 * nibble of byte b; codes at k >= K are 0), then lo and hi as little-endian
 * binary16 patterns: 12 bytes.
 * ------------------------------------------------------------------------- */
static uint32_t float_to_bits(float f) {
    uint32_t u;
    memcpy(&u, &f, 4);
    return u;
}

/* float -> binary16, round to nearest, ties to even */
static uint16_t float_to_half(float f) {
    uint32_t u = float_to_bits(f);
    uint16_t sign = (uint16_t)((u >> 16) & 0x8000u);
    uint32_t mag = u & 0x7fffffffu;
    if (mag > 0x7f800000u) return (uint16_t)(sign | 0x7e00u);            /* NaN */
    if (mag == 0x7f800000u) return (uint16_t)(sign | 0x7c00u);           /* infinity */
    double v = fabs((double)f);
    if (v == 0.0) return sign;
    /* position on the binary16 grid: subnormal spacing 2^-24 below 2^-14, else 2^(e-10) */
    int e;
    (void)frexp(v, &e);              /* v = m * 2^e, 0.5 <= m < 1, so v in [2^(e-1), 2^e) */
    int ex = e - 1;                  /* floor(log2 v) */
    if (ex < -14) ex = -14;
    double ulp = ldexp(1.0, ex - 10);
    double q = v / ulp;              /* exact: a power-of-two scaling */
    double r = floor(q);
    double frac = q - r;
    if (frac > 0.5 || (frac == 0.5 && fmod(r, 2.0) == 1.0)) r += 1.0;
    /* r in [0, 2048]: 0..1023 subnormal (ex == -14 and v < 2^-14), 1024..2047 normal, 2048 = next binade */
    uint32_t n = (uint32_t)r;
    uint32_t h;
    if (ex == -14 && n < 1024u) {
        h = n;                                           /* subnormal or zero */
    } else {
        int be = ex + 15;                                /* biased exponent */
        if (n == 2048u) { n = 1024u; be += 1; }
        if (be >= 31) return (uint16_t)(sign | 0x7c00u); /* overflow */
        h = ((uint32_t)be << 10) | (n - 1024u);
    }
    return (uint16_t)(sign | h);
}

uint16_t oracle_float_to_half(float f) { return float_to_half(f); }

void oracle_lut_to_f16(const float* lut, const uint8_t* bits, int64_t d_in, uint16_t* out) {
    for (int64_t i = 0; i < d_in; ++i) {
        int K = 1 << bits[i];
        for (int k = 0; k < 16; ++k) out[i * 16 + k] = k < K ? float_to_half(lut[i * 16 + k]) : 0;
    }
}

void oracle_lut_from_f16(const uint16_t* in, int64_t d_in, float* lut) {
    for (int64_t i = 0; i < d_in * 16; ++i) lut[i] = half_to_float(in[i]);
}

void oracle_lut_to_u4(const float* lut, const uint8_t* bits, int64_t d_in, uint8_t* out) {
    for (int64_t i = 0; i < d_in; ++i) {
        const float* c = lut + i * 16;
        int K = 1 << bits[i];
        float lo = c[0], hi = c[0];
        for (int k = 1; k < K; ++k) {
            if (c[k] < lo) lo = c[k];
            if (c[k] > hi) hi = c[k];
        }
        uint16_t lo16 = float_to_half(lo), hi16 = float_to_half(hi);
        float flo = half_to_float(lo16), fhi = half_to_float(hi16);
        float span = fhi - flo;
        float D = span / 15.0f;
        uint8_t* o = out + i * 12;
        memset(o, 0, 8);
        for (int k = 0; k < K; ++k) {
            int code = 0;
            if (D > 0.0f) {
                float t = c[k] - flo;
                float r = nearbyintf(t / D);          /* default rounding mode: half to even */
                code = r < 0.0f ? 0 : (r > 15.0f ? 15 : (int)r);
            }
            o[k >> 1] |= (uint8_t)(code << (4 * (k & 1)));
        }
        o[8] = (uint8_t)(lo16 & 0xff); o[9] = (uint8_t)(lo16 >> 8);
        o[10] = (uint8_t)(hi16 & 0xff); o[11] = (uint8_t)(hi16 >> 8);
    }
}

void oracle_lut_from_u4(const uint8_t* in, const uint8_t* bits, int64_t d_in, float* lut) {
    for (int64_t i = 0; i < d_in; ++i) {
        const uint8_t* o = in + i * 12;
        int K = 1 << bits[i];
        float flo = half_to_float((uint16_t)(o[8] | (o[9] << 8)));
        float fhi = half_to_float((uint16_t)(o[10] | (o[11] << 8)));
        float span = fhi - flo;
        float D = span / 15.0f;
        for (int k = 0; k < 16; ++k) {
            int code = (o[k >> 1] >> (4 * (k & 1))) & 15;
            float step = (float)code * D;
            lut[i * 16 + k] = k < K ? flo + step : 0.0f;
        }
    }
}

/* ---------------------------------------------------------------------------
 * Step 9.  Reconstruction and output error (Section 3.2.2: inference uses the
 * quantized weights plus the kept outliers; Appendix, justification of the
 * allocation: the output changes by X (W - W^)).
 *   What_{ij} = lut_i[code_{ij}] + O_{ij},   E = || X (W - What) ||_F   in fp64.
 * t_step > 1 evaluates every t_step-th token only (a sample of the rows of X).
 * ------------------------------------------------------------------------- */
double oracle_recon_error(const uint16_t* X, const uint16_t* W, int dtype, int64_t n_tokens,
                          int64_t d_in, int64_t d_out, int64_t ldx, int64_t ldw,
                          const float* lut, const uint8_t* codes, const int32_t* rows,
                          const int32_t* cols, const uint16_t* vals, int64_t nnz,
                          int64_t t_step) {
    double* D = (double*)malloc((size_t)(d_in * d_out) * sizeof(double));
    for (int64_t i = 0; i < d_in; ++i)
        for (int64_t j = 0; j < d_out; ++j)
            D[i * d_out + j] = (double)oracle_widen(W[i * ldw + j], dtype) -
                               (double)lut[i * 16 + codes[i * d_out + j]];
    for (int64_t p = 0; p < nnz; ++p)
        D[(int64_t)rows[p] * d_out + cols[p]] -= (double)oracle_widen(vals[p], dtype);
    double* y = (double*)malloc((size_t)d_out * sizeof(double));
    double total = 0.0;
    if (t_step < 1) t_step = 1;
    for (int64_t t = 0; t < n_tokens; t += t_step) {
        for (int64_t j = 0; j < d_out; ++j) y[j] = 0.0;
        for (int64_t i = 0; i < d_in; ++i) {
            double x = (double)oracle_widen(X[t * ldx + i], dtype);
            for (int64_t j = 0; j < d_out; ++j) y[j] += x * D[i * d_out + j];
        }
        for (int64_t j = 0; j < d_out; ++j) total += y[j] * y[j];
    }
    free(y);
    free(D);
    return sqrt(total);
}

/* ---------------------------------------------------------------------------
 * Step 10.  Inference product of one token with the quantized layer (Section 6,
 * the figure of the real quantization process): the input is split by the
 * precision of its channels, each part multiplies its 2-, 3- or 4-bit weight
 * sub-matrix, the outliers multiply the original 16-bit input, and everything
 * is accumulated:
 *     y_j = sum_i x_i * lut_i[code_{ij}]  +  sum_{(i,j,v) in O} x_i * v .
 * Grouping by precision only reorders the sum over i, so the definition is
 * written out directly from the byte codes, in fp64, channel by channel.
 * yabs_j (optional) = sum of the absolute values of the same terms: the scale
 * a floating-point error bound of any summation order is stated against.
 * ------------------------------------------------------------------------- */
void oracle_matvec(const uint16_t* x, int dtype, int64_t d_in, int64_t d_out, const float* lut,
                   const uint8_t* codes, const int32_t* rows, const int32_t* cols,
                   const uint16_t* vals, int64_t nnz, double* y, double* yabs) {
    for (int64_t j = 0; j < d_out; ++j) {
        y[j] = 0.0;
        if (yabs) yabs[j] = 0.0;
    }
    for (int64_t i = 0; i < d_in; ++i) {
        double xi = (double)oracle_widen(x[i], dtype);
        for (int64_t j = 0; j < d_out; ++j) {
            double t = xi * (double)lut[i * 16 + codes[i * d_out + j]];
            y[j] += t;
            if (yabs) yabs[j] += fabs(t);
        }
    }
    for (int64_t p = 0; p < nnz; ++p) {
        double t = (double)oracle_widen(x[rows[p]], dtype) * (double)oracle_widen(vals[p], dtype);
        y[cols[p]] += t;
        if (yabs) yabs[cols[p]] += fabs(t);
    }
}

/* The outlier list regrouped by output column (the paper keeps the outliers in a
 * compressed sparse format for the inference kernel, Section 6): col_ptr[j] ..
 * col_ptr[j+1] delimits the entries of column j, inside a column ascending by
 * row.  Plain definition: stable counting by column of a list that is already
 * sorted by (row, col). */
void oracle_outliers_by_column(const int32_t* rows, const int32_t* cols, const uint16_t* vals,
                               int64_t nnz, int64_t d_out, int64_t* col_ptr, int32_t* c_rows,
                               uint16_t* c_vals) {
    for (int64_t j = 0; j <= d_out; ++j) col_ptr[j] = 0;
    for (int64_t p = 0; p < nnz; ++p) ++col_ptr[cols[p] + 1];
    for (int64_t j = 0; j < d_out; ++j) col_ptr[j + 1] += col_ptr[j];
    int64_t* next = (int64_t*)malloc((size_t)(d_out + 1) * sizeof(int64_t));
    memcpy(next, col_ptr, (size_t)(d_out + 1) * sizeof(int64_t));
    for (int64_t p = 0; p < nnz; ++p) {
        int64_t q = next[cols[p]]++;
        c_rows[q] = rows[p];
        c_vals[q] = vals[p];
    }
    free(next);
}

/* Whole pass for one layer, in the paper's order (used by the timed CPU
 * baseline): statistic -> Algorithm 1 -> O_act, provisional K-means, O_q ->
 * final K-means and codes -> packing.  Outputs are caller-allocated. */
int oracle_layer_pass(const uint16_t* X, const uint16_t* W, int dtype, int64_t n_tokens,
                      int64_t d_in, int64_t d_out, int64_t ldx, int64_t ldw, double avg_bits,
                      int64_t n_act, int64_t n_q, int T, float* a, uint8_t* bits,
                      int32_t* rows, int32_t* cols, uint16_t* vals, float* lut, uint8_t* codes,
                      uint32_t* packed, int64_t* row_off, int32_t* perm, int64_t* seg_rows) {
    double* sumsq = (double*)calloc((size_t)d_in, sizeof(double));
    oracle_collect_stats(X, dtype, n_tokens, d_in, ldx, sumsq);
    oracle_finalize_stats(sumsq, d_in, a);
    free(sumsq);
    int rc = oracle_allocate_bits(a, d_in, avg_bits, 0, bits, NULL);
    if (rc) return rc;
    rc = oracle_extract_outliers(W, dtype, d_in, d_out, ldw, a, bits, n_act, n_q, T, rows, cols,
                                 vals, NULL, NULL);
    if (rc) return rc;
    rc = oracle_quantize_layer(W, dtype, d_in, d_out, ldw, bits, rows, cols,
                               n_act * d_out + n_q, T, NULL, lut, codes);
    if (rc) return rc;
    oracle_pack(codes, bits, d_in, d_out, packed, row_off, perm, seg_rows);
    return 0;
}
