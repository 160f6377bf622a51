/*
 * SwiftPrune CPU oracle  --  TEST INFRASTRUCTURE, NOT A PRODUCT PATH.
 *
 * A plain, slow, obviously-correct restatement of the per-layer pruning pass of
 * SwiftPrune (arXiv 2501.16376): calibration statistics (Algorithm 1, step 1),
 * the contribution metric (Eq. 8), the EWMA running-threshold selection
 * (Algorithm 1 with the state rules of Table 2), the N:M group selection
 * (Section 3.3) and the write-back of pruned weights (Algorithm 1, "w_i = 0" /
 * "c_i = w_i").  It exists only so that tests, the smoke check and the
 * benchmark's CPU-baseline leg can compare the CUDA library against it.  It
 * shares no code with the CUDA library and must never be called from it.
 *
 * Conventions
 *   W   [R, n] row-major 16-bit floats (dtype 0 = IEEE binary16, 1 = bfloat16),
 *       leading dimension ldw (elements).  Row = one output neuron, column =
 *       one input channel (Section 2: rows are pruned independently).
 *   X   [T, n] row-major 16-bit floats, leading dimension ldx.
 *   colsq[q] = sum_t X[t,q]^2  -- the "x_q^2" of Eq. 8 (diagonal of X X^T,
 *       Section 2: H = 2 X X^T),  S = sum_q colsq[q]  (Algorithm 1, step 1).
 *   mask [R, ceil(n/32)] uint32, bit j of word k = keep flag of column 32k+j
 *       (1 = kept).
 *
 * Arithmetic
 *   Statistics are accumulated in fp64.  The selection functions exist in two
 *   precisions: "_f32" evaluates every operation of Eq. 8 / Algorithm 1 in
 *   IEEE binary32, one rounding per printed operation, in the printed order
 *   (the file must be compiled with -ffp-contract=off); "_f64" does the same in
 *   binary64 and is used to report the fp32-vs-fp64 gap.
 *
 *   The binary32 score is evaluated as
 *       u = x_q^2 / S ;  den = 1 - u ;  c = 0.5 / den ;  L = (w*w) * c
 *   which is Eq. 8 with the per-channel factor 1/(2(1 - x_q^2/S)) formed first.
 *   den == 0 (one channel holds all the energy) gives c = +inf by IEEE rules.
 *
 * Parity pins: every function below is pinned by tests/test_oracle_pins.py
 * (closed forms, brute force, hand-traced recurrences, textbook magnitude
 * pruning as a special case) except the mapping from a nominal sparsity to an
 * achieved sparsity, for which the paper prints no worked example: that
 * mapping is "parity unpinned".
 */
#include <math.h>
#include <stdint.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define SPO_F16 0
#define SPO_BF16 1

#define SPO_S_LITERAL_W2 1 /* Table 2 / Algorithm 1: S <- S - w_i^2 when pruned */
#define SPO_S_FROZEN 0     /* S stays at its initial value */
#define SPO_S_READING_X2 2 /* the other reading of Table 2's row S: S <- S - x_i^2 when pruned (S is a
                              sum of x^2, so the pruned channel's own share leaves it) */

/* ---- 16-bit float decoding (exact) ------------------------------------- */

static float spo_bits_to_float(uint32_t b)
{
    float f;
    memcpy(&f, &b, sizeof f);
    return f;
}

/* IEEE binary16 -> binary32, exact for every bit pattern. */
float spo_half_to_float(uint16_t h)
{
    uint32_t sign = (uint32_t)(h & 0x8000u) << 16;
    uint32_t expo = (h >> 10) & 0x1fu;
    uint32_t frac = h & 0x3ffu;
    if (expo == 0x1fu) /* inf / nan */
        return spo_bits_to_float(sign | 0x7f800000u | (frac << 13));
    if (expo == 0) { /* zero / subnormal: frac * 2^-24 */
        float v = (float)frac * (1.0f / 16777216.0f);
        return sign ? -v : v;
    }
    return spo_bits_to_float(sign | ((expo + 112u) << 23) | (frac << 13));
}

/* bfloat16 -> binary32: the 16 bits are the high half of the binary32 word. */
float spo_bf16_to_float(uint16_t h)
{
    return spo_bits_to_float((uint32_t)h << 16);
}

static inline float spo_decode(uint16_t bits, int dtype)
{
    return dtype == SPO_BF16 ? spo_bf16_to_float(bits) : spo_half_to_float(bits);
}

/* Vectorised decode for the tests that pin the two decoders against numpy. */
void spo_decode_array(const uint16_t *src, int dtype, int64_t count, float *dst)
{
    for (int64_t i = 0; i < count; ++i)
        dst[i] = spo_decode(src[i], dtype);
}

/* ---- Algorithm 1, step 1: statistics ----------------------------------- */

/*
 * colsq[q] += sum_t X[t,q]^2 in fp64 (values decoded exactly), tokens in
 * ascending order for every channel.  Channels are independent, so blocks of
 * channels may be given to different threads without changing any sum.
 */
void spo_colsq_accumulate(const uint16_t *X, int dtype, int64_t T, int64_t n,
                          int64_t ldx, double *colsq, int nthreads)
{
    const int64_t block = 64;
    const int64_t nblocks = (n + block - 1) / block;
    (void)nthreads;
#ifdef _OPENMP
#pragma omp parallel for schedule(static) num_threads(nthreads > 0 ? nthreads : 1)
#endif
    for (int64_t b = 0; b < nblocks; ++b) {
        int64_t q0 = b * block;
        int64_t q1 = q0 + block < n ? q0 + block : n;
        for (int64_t t = 0; t < T; ++t) {
            const uint16_t *row = X + t * ldx;
            for (int64_t q = q0; q < q1; ++q) {
                double v = (double)spo_decode(row[q], dtype);
                colsq[q] += v * v;
            }
        }
    }
}

/* S = sum_q colsq[q]  (Algorithm 1, step 1), fp64, ascending q. */
double spo_total(const double *colsq, int64_t n)
{
    double S = 0.0;
    for (int64_t q = 0; q < n; ++q)
        S += colsq[q];
    return S;
}

/* ---- Eq. 8: the contribution metric ------------------------------------ */

static inline float spo_score32(float w, float xq2, float S)
{
    float u = xq2 / S;
    float den = 1.0f - u;
    float c = 0.5f / den;
    float w2 = w * w;
    return w2 * c;
}

static inline double spo_score64(double w, double xq2, double S)
{
    return 0.5 * (w * w) / (1.0 - xq2 / S);
}

/* Per-channel factor c_q = 1 / (2 (1 - x_q^2 / S)) in binary32. */
void spo_channel_factor_f32(const float *colsq32, float S32, int64_t n, float *c)
{
    for (int64_t q = 0; q < n; ++q) {
        float u = colsq32[q] / S32;
        float den = 1.0f - u;
        c[q] = 0.5f / den;
    }
}

/* L[r,q] for a whole matrix with S fixed (binary32). L is [R, n] dense. */
void spo_score_f32(const uint16_t *W, int dtype, int64_t R, int64_t n, int64_t ldw,
                   const float *colsq32, float S32, float *L)
{
    for (int64_t r = 0; r < R; ++r)
        for (int64_t q = 0; q < n; ++q)
            L[r * n + q] = spo_score32(spo_decode(W[r * ldw + q], dtype), colsq32[q], S32);
}

/* Same in binary64, straight from Eq. 8. */
void spo_score_f64(const uint16_t *W, int dtype, int64_t R, int64_t n, int64_t ldw,
                   const double *colsq, double S, double *L)
{
    for (int64_t r = 0; r < R; ++r)
        for (int64_t q = 0; q < n; ++q)
            L[r * n + q] = spo_score64((double)spo_decode(W[r * ldw + q], dtype), colsq[q], S);
}

/* ---- Algorithm 1: EWMA running-threshold selection ---------------------- */

static inline void spo_set_keep(uint32_t *mask_row, int64_t i)
{
    mask_row[i >> 5] |= (uint32_t)1u << (i & 31);
}

/*
 * Algorithm 1 for every row, binary32.
 *   For i = 0 .. n-1 in ascending column order:
 *     L_i from Eq. 8 with the current S;
 *     if i == 0: est = L_0            (Table 2, initial value of est; dev = 0)
 *     if L_i < est - la*dev: prune (S <- S - w_i^2 in literal mode, w_i = 0)
 *     est <- (1-alpha) est + alpha L_i
 *     dev <- (1-beta) dev + beta |est - L_i|     (est already updated)
 *     c_i = w_i
 * Optional outputs (may be NULL): L_out, thr_out [R, n] hold L_i and the
 * threshold est - la*dev that L_i was tested against.
 * mask must hold R * ceil(n/32) words; it is overwritten.  Wout may be NULL.
 */
void spo_select_ewma_f32(const uint16_t *W, int dtype, int64_t R, int64_t n, int64_t ldw,
                         const float *colsq32, float S32,
                         float alpha, float beta, float la, int s_update,
                         uint32_t *mask, uint16_t *Wout, int64_t ldo,
                         float *L_out, float *thr_out, int nthreads)
{
    const int64_t words = (n + 31) / 32;
    const float one_minus_alpha = 1.0f - alpha;
    const float one_minus_beta = 1.0f - beta;
    (void)nthreads;
#ifdef _OPENMP
#pragma omp parallel for schedule(static) num_threads(nthreads > 0 ? nthreads : 1)
#endif
    for (int64_t r = 0; r < R; ++r) { /* rows are independent problems (the row loop of Algorithm 1 is parallel) */
        uint32_t *mrow = mask + r * words;
        for (int64_t k = 0; k < words; ++k)
            mrow[k] = 0;
        float S = S32;
        float est = 0.0f;
        float dev = 0.0f;
        for (int64_t i = 0; i < n; ++i) {
            uint16_t bits = W[r * ldw + i];
            float w = spo_decode(bits, dtype);
            float L = spo_score32(w, colsq32[i], S);
            if (i == 0)
                est = L;
            float la_dev = la * dev;
            float thr = est - la_dev;
            if (L < thr) {
                if (s_update == SPO_S_LITERAL_W2) {
                    float w2 = w * w;
                    S = S - w2;
                } else if (s_update == SPO_S_READING_X2) {
                    S = S - colsq32[i];
                }
                bits = 0; /* w_i = 0 */
            } else {
                spo_set_keep(mrow, i);
            }
            float keep_part = one_minus_alpha * est;
            float new_part = alpha * L;
            est = keep_part + new_part;
            float diff = fabsf(est - L);
            float dkeep = one_minus_beta * dev;
            float dnew = beta * diff;
            dev = dkeep + dnew;
            if (Wout)
                Wout[r * ldo + i] = bits; /* c_i = w_i */
            if (L_out)
                L_out[r * n + i] = L;
            if (thr_out)
                thr_out[r * n + i] = thr;
        }
    }
}

/* The same algorithm with every operation in binary64. */
void spo_select_ewma_f64(const uint16_t *W, int dtype, int64_t R, int64_t n, int64_t ldw,
                         const double *colsq, double S0,
                         double alpha, double beta, double la, int s_update,
                         uint32_t *mask, uint16_t *Wout, int64_t ldo,
                         double *L_out, double *thr_out, int nthreads)
{
    const int64_t words = (n + 31) / 32;
    (void)nthreads;
#ifdef _OPENMP
#pragma omp parallel for schedule(static) num_threads(nthreads > 0 ? nthreads : 1)
#endif
    for (int64_t r = 0; r < R; ++r) {
        uint32_t *mrow = mask + r * words;
        for (int64_t k = 0; k < words; ++k)
            mrow[k] = 0;
        double S = S0;
        double est = 0.0;
        double dev = 0.0;
        for (int64_t i = 0; i < n; ++i) {
            uint16_t bits = W[r * ldw + i];
            double w = (double)spo_decode(bits, dtype);
            double L = spo_score64(w, colsq[i], S);
            if (i == 0)
                est = L;
            double thr = est - la * dev;
            if (L < thr) {
                if (s_update == SPO_S_LITERAL_W2)
                    S = S - w * w;
                else if (s_update == SPO_S_READING_X2)
                    S = S - colsq[i];
                bits = 0;
            } else {
                spo_set_keep(mrow, i);
            }
            est = (1.0 - alpha) * est + alpha * L;
            dev = (1.0 - beta) * dev + beta * fabs(est - L);
            if (Wout)
                Wout[r * ldo + i] = bits;
            if (L_out)
                L_out[r * n + i] = L;
            if (thr_out)
                thr_out[r * n + i] = thr;
        }
    }
}

/* ---- Section 3.3: N:M group selection ----------------------------------- */

/* Strict order on scores with NaN placed above every number. */
static inline int spo_less32(float a, float b)
{
    if (isnan(a))
        return 0;
    if (isnan(b))
        return 1;
    return a < b;
}

/*
 * Every row is cut into contiguous groups of M columns starting at column 0;
 * in each group the M-N entries with the smallest L (Eq. 8, S fixed) are
 * pruned and N are kept.  Among equal scores the lower column is pruned first.
 * Selection is by repeated scan for the smallest remaining entry.
 * Requires n % M == 0, 0 < N < M <= 32 (returns -1 otherwise).
 */
int spo_select_nm_f32(const uint16_t *W, int dtype, int64_t R, int64_t n, int64_t ldw,
                      const float *colsq32, float S32, int N, int M,
                      uint32_t *mask, uint16_t *Wout, int64_t ldo,
                      float *L_out, int nthreads)
{
    if (M <= 0 || M > 32 || N <= 0 || N >= M || n % M != 0)
        return -1;
    const int64_t words = (n + 31) / 32;
    (void)nthreads;
#ifdef _OPENMP
#pragma omp parallel for schedule(static) num_threads(nthreads > 0 ? nthreads : 1)
#endif
    for (int64_t r = 0; r < R; ++r) {
        uint32_t *mrow = mask + r * words;
        for (int64_t k = 0; k < words; ++k)
            mrow[k] = 0;
        for (int64_t g = 0; g < n; g += M) {
            float L[32];
            int pruned[32];
            for (int j = 0; j < M; ++j) {
                L[j] = spo_score32(spo_decode(W[r * ldw + g + j], dtype), colsq32[g + j], S32);
                pruned[j] = 0;
                if (L_out)
                    L_out[r * n + g + j] = L[j];
            }
            for (int k = 0; k < M - N; ++k) { /* remove the smallest remaining */
                int best = -1;
                for (int j = 0; j < M; ++j) {
                    if (pruned[j])
                        continue;
                    if (best < 0 || spo_less32(L[j], L[best]))
                        best = j;
                }
                pruned[best] = 1;
            }
            for (int j = 0; j < M; ++j) {
                uint16_t bits = W[r * ldw + g + j];
                if (pruned[j])
                    bits = 0;
                else
                    spo_set_keep(mrow, g + j);
                if (Wout)
                    Wout[r * ldo + g + j] = bits;
            }
        }
    }
    return 0;
}

/* ---- Algorithm 1 write-back on its own: C = W (.) mask ------------------- */

void spo_apply_mask(const uint16_t *W, int64_t R, int64_t n, int64_t ldw,
                    const uint32_t *mask, uint16_t *Wout, int64_t ldo)
{
    const int64_t words = (n + 31) / 32;
    for (int64_t r = 0; r < R; ++r)
        for (int64_t i = 0; i < n; ++i) {
            int keep = (mask[r * words + (i >> 5)] >> (i & 31)) & 1u;
            Wout[r * ldo + i] = keep ? W[r * ldw + i] : (uint16_t)0;
        }
}

int spo_max_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
