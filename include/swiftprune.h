/*
 * swiftprune.h -- C ABI of the B200 (sm_100a) SwiftPrune pruning pass.
 *
 * The library implements the per-layer pruning pass of SwiftPrune
 * (arXiv 2501.16376): calibration statistics (Algorithm 1, step 1), the
 * Hessian-free contribution metric (Eq. 8), the EWMA running-threshold
 * selection that replaces sorting (Algorithm 1; state rules in Table 2; the
 * parameter la per pruning ratio in Table 3), the N:M group selection
 * (Section 3.3) and the write-back of the pruned weights (Algorithm 1,
 * "w_i = 0" / "c_i = w_i").
 *
 * General conventions
 *   - Unless a parameter says "host", every data pointer is a DEVICE pointer to
 *     memory owned by the caller, on the device the context was created for.
 *     The library owns only the context (O(d_in) device memory).
 *   - Calls enqueue work on the caller's stream (sp_stream = cudaStream_t passed
 *     as void*; NULL = the default stream) and return without synchronising,
 *     except sp_create, sp_destroy, sp_get_stats, sp_set_stats and sp_search_la, which say so.
 *   - Arguments are validated on the host before anything is launched; a
 *     non-SP_OK status means nothing was enqueued by that call.  No call
 *     throws, traps or aborts.
 *   - A weight matrix W is [n_rows, d_in] row-major 16-bit floats with leading
 *     dimension ldw (elements, >= d_in): one row per output neuron, one column
 *     per input channel.  Rows are pruned independently (Section 2; the row loop of
 *     Algorithm 1 runs in parallel).
 *   - A mask is [n_rows, ceil(d_in/32)] uint32, row-major, no padding between
 *     rows; bit j of word k of a row is the keep flag of column 32k+j
 *     (1 = kept, 0 = pruned; bits past d_in are 0).
 *   - Pruned weights are written as +0 (bit pattern 0x0000); kept weights are
 *     copied bit for bit.
 *   - Fast paths need 16-byte aligned base pointers and leading dimensions
 *     that are multiples of 8 elements; anything else is handled by slower
 *     element-wise paths with identical results.
 *   - One context belongs to one layer input of width d_in; layers that read
 *     the same input (q/k/v; gate/up) share it.  A context must not be used
 *     from two streams at once.
 */
#ifndef SWIFTPRUNE_H_
#define SWIFTPRUNE_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct sp_ctx sp_ctx; /* opaque, library-owned */
typedef void *sp_stream;      /* a cudaStream_t */

typedef enum {
    SP_OK = 0,
    SP_ERR_INVALID_ARG = 1, /* null pointer, negative size, unknown enum value */
    SP_ERR_SHAPE = 2,       /* ld < d_in, d_in % M != 0, size over a stated maximum */
    SP_ERR_DTYPE = 3,
    SP_ERR_STATE = 4,       /* selection or scoring before any calibration data */
    SP_ERR_DEGENERATE = 5,  /* S == 0 or non-finite statistics (sp_get_stats reports it) */
    SP_ERR_CUDA = 6,        /* a CUDA runtime call failed; see sp_last_cuda_error */
    SP_ERR_NOMEM = 7
} sp_status;

typedef enum { SP_F16 = 0, SP_BF16 = 1 } sp_dtype;

/* How the EWMA selection treats Algorithm 1's step "S = S - w_i^2" (Table 2, row S).
 * In binary32 the subtraction changes S only if w_i^2 reaches a quarter of the spacing of
 * floats at S, which calibration-scale statistics (S ~ tokens * d_in) never allow. */
typedef enum {
    SP_S_GATED = 0,      /* Algorithm 1 as printed, at scan speed: rows are scanned in parallel with
                            S at its initial value; a row holding a weight that could change S is
                            detected before that weight's tile is stored and finished
                            sequentially from there in the same kernel, so the result is the
                            printed algorithm for every row (the default) */
    SP_S_LITERAL_W2 = 1, /* the printed update, evaluated sequentially along every row */
    SP_S_FROZEN = 2,     /* S keeps its initial value whatever is pruned */
    SP_S_READING_X2 = 3, /* the other conceivable reading of that row of Table 2: S is a sum of
                            x^2, and a pruned weight takes its channel's x_i^2 out of it
                            ("S = S - x_i^2"); evaluated sequentially along every row.  This
                            changes S by tens of percent and is not what the paper prints:
                            offered for comparison */
    SP_S_LITERAL_SCAN = 4 /* the printed update again, but rows scanned by whole warps: every
                            256-column tile is decided by fix-point sweeps (decide with the S the
                            previous sweep's decisions imply, prefix-sum the pruned w^2, repeat
                            until nothing changes; a tile that does not settle in 8 sweeps hands
                            the row to the sequential walk and counts in SP_COUNTER_S_HAZARD).
                            Same decisions as SP_S_LITERAL_W2 up to re-association (the tolerance
                            of the scans); several times faster when rows are few and long */
} sp_s_update;

/* Parameters of Algorithm 1 (alpha, beta: Table 2; la: Table 3). */
typedef struct {
    float alpha;
    float beta;
    float la;
    int s_update; /* an sp_s_update */
} sp_ewma_params;

/* Entries of the optional device counter block passed to the selection calls. */
enum { SP_COUNTER_KEPT = 0, SP_COUNTER_S_HAZARD = 1, SP_NUM_COUNTERS = 2 };

/* ------------------------------------------------------------------ context */

/*
 * Creates the context for one layer input of d_in channels on CUDA device
 * `device` (1 <= d_in <= 2^20).  Allocates its device memory (statistics,
 * per-channel factors, partial sums) and synchronises with that device once.
 * The statistics start empty.
 */
sp_status sp_create(sp_ctx **out, int64_t d_in, int device);

/* Frees the context (synchronises with its device first).  NULL is allowed. */
sp_status sp_destroy(sp_ctx *ctx);

/* ------------------------------------------------------------------ calibration (Algorithm 1, step 1) */

/* Forgets all accumulated statistics. */
sp_status sp_calib_reset(sp_ctx *ctx, sp_stream stream);

/*
 * Adds one batch of calibration activations: for every channel q,
 *     colsq[q] += sum_t X[t, q]^2.
 * colsq[q] is the "x_q^2" of Eq. 8, i.e. the q-th diagonal entry of X X^T
 * (Section 2: H = 2 X X^T), and S = sum_q colsq[q] is Algorithm 1's step 1.
 * X is [n_tokens, d_in] row-major of `dtype` with leading dimension ldx
 * (elements).  n_tokens == 0 is a no-op.  Squares are exact in fp32; sums of
 * at most 8 squares are formed in fp32 and then accumulated in fp64.  The
 * result does not depend on run-to-run scheduling (no floating-point atomics).
 */
sp_status sp_calib_accumulate(sp_ctx *ctx, const void *X, sp_dtype dtype, int64_t n_tokens,
                              int64_t ldx, sp_stream stream);

/*
 * The same with flags.  The library's kernels are launched so that a kernel may be scheduled
 * while its predecessor on the stream drains; sp_calib_accumulate still reads X only after
 * everything queued earlier on the stream has completed (ordinary stream semantics: the
 * preceding kernel may be the one that writes X).  SP_CALIB_X_COMPLETE is the caller's promise
 * that X was complete before the operation that precedes this call on the stream began (e.g.
 * calibration data prepared long before, with library calls in between): the kernel then
 * streams X while that predecessor is still finishing and orders only its update of the
 * statistics after it.  With the flag set wrongly the statistics are silently wrong.
 */
enum { SP_CALIB_X_COMPLETE = 1 };
sp_status sp_calib_accumulate_ex(sp_ctx *ctx, const void *X, sp_dtype dtype, int64_t n_tokens,
                                 int64_t ldx, unsigned flags, sp_stream stream);

/*
 * One batch for each of several layer inputs (the inputs of one transformer block, say) in one
 * launch: the effect of sp_calib_accumulate_ex(ctxs[i], batches[i].X, dtype,
 * batches[i].n_tokens, batches[i].ldx, flags, stream) for every i - Algorithm 1's step 1 is a
 * sum per channel, and the channels of different inputs have nothing to do with each other.
 * The sums agree with those of the single calls to rounding (the tokens of a batch may be cut
 * into slabs differently, which moves the last bits of a sum) and are, like theirs,
 * reproducible bit for bit for a given sequence of calls.  For inputs so narrow or batches so
 * short that a launch of their own would be mostly ramp-up.  ctxs and batches are HOST arrays of n_items entries (1 <= n_items <=
 * SP_MAX_MULTI); the contexts must all be different (two batches of one launch cannot update
 * the same sums: SP_ERR_INVALID_ARG) and on one device; a batch with n_tokens == 0 is skipped;
 * batches that do not allow 16-byte access get launches of their own.
 */
typedef struct {
    const void *X;    /* device, [n_tokens, d_in of its context] of the call's dtype */
    int64_t n_tokens;
    int64_t ldx;      /* elements */
} sp_batch;
sp_status sp_calib_accumulate_multi(sp_ctx *const *ctxs /* host */,
                                    const sp_batch *batches /* host */, int n_items,
                                    sp_dtype dtype, unsigned flags, sp_stream stream);

/*
 * Finalisation of several contexts at once: S and the per-channel factors of Eq. 8 for every
 * listed context that has batches pending, by one launch (what sp_score(ctx, NULL, ...) does for
 * one context; the selection calls do it implicitly).  A context without calibration data gives
 * SP_ERR_STATE; a context may appear more than once.
 */
sp_status sp_finalize_multi(sp_ctx *const *ctxs /* host */, int n_items, sp_stream stream);

/*
 * Reads the statistics back to HOST buffers (any may be NULL) and synchronises
 * the stream: colsq_host[d_in] (fp64), *S_host, factor_host[d_in] (the fp32
 * per-channel factor c_q = 1/(2(1 - colsq[q]/S)) of Eq. 8), *n_tokens_host.
 * Returns SP_ERR_DEGENERATE if S is zero or not finite, SP_ERR_STATE if no
 * token has been accumulated.
 */
sp_status sp_get_stats(sp_ctx *ctx, double *colsq_host, double *S_host, float *factor_host,
                       int64_t *n_tokens_host, sp_stream stream);

/*
 * Replaces the statistics by colsq_host[d_in] (HOST, fp64) and a token count
 * (> 0), e.g. to resume from saved statistics.  Synchronises the stream.
 */
sp_status sp_set_stats(sp_ctx *ctx, const double *colsq_host, int64_t n_tokens, sp_stream stream);

/*
 * One-shot statistics without any allocation (the paper has no counterpart: this exists for
 * callers, not for the method).  Some programs must not allocate device memory while they
 * run: code executing inside a framework that owns the whole memory pool, a service that has
 * handed all remaining memory to its caches, a real-time loop that cannot afford the implicit
 * device-wide synchronisation of cudaMalloc/cudaFree.  sp_create allocates, so such callers
 * cannot use a context.  This call computes, for ONE batch X [n_tokens, d_in] (n_tokens >= 1),
 * what sp_calib_accumulate + finalisation compute, on the CURRENT device, and copies the
 * results into the caller's DEVICE buffers (each may be NULL): colsq_out[d_in] (fp64),
 * factor_out[d_in] (fp32 c_q of Eq. 8), S_out[1] (fp64).  Its working memory is a fixed array
 * inside the library image (about 4.4 MB per GPU, held until the process exits), hence:
 *   - d_in must be <= 16384, else SP_ERR_SHAPE and nothing is enqueued;
 *   - it calls no cudaMalloc/cudaFree and no allocating library routine;
 *   - all calls on one device share that array: calls whose GPU work may overlap (different
 *     streams, different threads) race and give wrong results - keep them on one stream or
 *     order them with events.  Nothing is kept between calls;
 *   - the first call on each device looks up the array's device address (a host-side,
 *     synchronous runtime query) and may make the CUDA runtime load the library's kernels,
 *     which can allocate; make that first call before starting any stream capture and before
 *     the phase in which nothing may be allocated.
 * Results agree with the context path to rounding (the token slabs may be cut differently).
 */
sp_status sp_calib_stats_noalloc(const void *X, sp_dtype dtype, int64_t n_tokens, int64_t d_in,
                                 int64_t ldx, double *colsq_out, float *factor_out, double *S_out,
                                 sp_stream stream);

/* ------------------------------------------------------------------ metric (Eq. 8) */

/*
 * Finalises the statistics (S and the per-channel factor c_q) if new batches
 * arrived since the last finalisation, and, if scores_out is not NULL, writes
 *     L[r, q] = (w[r,q] * w[r,q]) * c_q ,   c_q = 0.5 / (1 - colsq[q] / S)
 * as fp32 [n_rows, d_in] (dense, leading dimension d_in), which is Eq. 8 with S
 * at its initial value.  All operations are IEEE binary32 with one rounding
 * each, in exactly this order: u = colsq32/S32, den = 1-u, c = 0.5/den,
 * w2 = w*w (exact), L = w2*c.  W may be NULL when scores_out is NULL
 * (finalise only).  The selection calls finalise implicitly.
 */
sp_status sp_score(sp_ctx *ctx, const void *W, sp_dtype dtype, int64_t n_rows, int64_t ldw,
                   float *scores_out, sp_stream stream);

/* ------------------------------------------------------------------ selection */

/* Table 3: la for a pruning ratio in (0, 1).  The five listed ratios (0.5 .. 0.9)
 * return the printed values; other ratios are interpolated linearly between, or
 * extrapolated from, the nearest two (the paper gives no values there). */
sp_status sp_la_for_sparsity(float sparsity, float *la_out);

/*
 * Algorithm 1 (EWMA running threshold) on every row of W, fused with the
 * write-back.  Along each row, for i = 0 .. d_in-1:
 *     L_i as in sp_score;  est starts at L_0, dev at 0 (Table 2);
 *     prune w_i  iff  L_i < est - la * dev      (state before the update);
 *     est <- (1-alpha) est + alpha L_i;  dev <- (1-beta) dev + beta |est - L_i|
 *     (dev uses the updated est, as Algorithm 1 orders the two steps).
 * Column 0 of every row is therefore never pruned.
 *   sparsity   nominal pruning ratio; la = sp_la_for_sparsity(sparsity),
 *              alpha = beta = 0.125 (Section 4.2), SP_S_GATED.  The achieved ratio
 *              is only approximately the nominal one.
 *   mask_out   nullable; mask as described above.
 *   W_out      nullable; pruned copy of W with leading dimension ldo; may alias W
 *              exactly (same pointer, same ld) for in-place pruning.
 *   counters   nullable; SP_NUM_COUNTERS device uint64 the call ADDS to:
 *              [SP_COUNTER_KEPT] kept weights, [SP_COUNTER_S_HAZARD] rows that held a weight
 *              able to change S in binary32 and were therefore finished sequentially
 *              (SP_S_GATED only; 0 at calibration scale).
 * The scan evaluates the two recurrences as warp-level affine scans in fp32; results differ
 * from a sequential fp32 evaluation by re-association only.  A row that SP_S_GATED finishes
 * sequentially costs about as much as a thousand scanned rows: when the statistics are so
 * small that most rows need it, SP_S_LITERAL_W2 is the faster way to the same result.
 */
sp_status sp_select_unstructured(sp_ctx *ctx, const void *W, sp_dtype dtype, int64_t n_rows,
                                 int64_t ldw, float sparsity, uint32_t *mask_out, void *W_out,
                                 int64_t ldo, unsigned long long *counters, sp_stream stream);

/* Same with explicit parameters (0 < alpha, beta <= 1; la finite). */
sp_status sp_select_unstructured_ex(sp_ctx *ctx, const void *W, sp_dtype dtype, int64_t n_rows,
                                    int64_t ldw, const sp_ewma_params *params /* host */,
                                    uint32_t *mask_out, void *W_out, int64_t ldo,
                                    unsigned long long *counters, sp_stream stream);

/*
 * Diagnostic behind the paper's Fig. 2 (est and dev tracking the mean and the L1 deviation of L
 * along a row): writes, for every weight of every row, the state Algorithm 1 tests it against -
 * est_out[r, i] and dev_out[r, i] are est and dev BEFORE the update of element i (so
 * est_out[r, 0] = L_0, dev_out[r, 0] = 0) - and scores_out[r, i] = L_i; each fp32
 * [n_rows, d_in], dense, nullable.  Evaluated sequentially along each row in binary32 with one
 * rounding per operation (one thread per row: meant for a handful of rows, not for speed);
 * params->s_update selects whether "S = S - w_i^2" is applied to pruned weights.
 */
sp_status sp_ewma_trace(sp_ctx *ctx, const void *W, sp_dtype dtype, int64_t n_rows, int64_t ldw,
                        const sp_ewma_params *params /* host */, float *est_out, float *dev_out,
                        float *scores_out, sp_stream stream);

/*
 * Searches la for a requested pruning ratio (the paper tunes la per ratio by hand, Table 3, and
 * names "finding the optimal sparsity" and frequent re-pruning as the use, Sections 1 and 4.2).
 * With S frozen the pruned fraction is a non-increasing function of la, so the call bisects
 * la on [-8, 8]: each of the `iterations` (1..64) steps runs Algorithm 1 over W at the midpoint
 * in count-only mode (W is read, nothing is written).  For rows that allow 16-byte access
 * (W 16-byte aligned, ldw and d_in multiples of 8) the bisection state stays on the device and
 * the call SYNCHRONISES the stream once, at the end; otherwise the kept count is read back after
 * every step (one synchronisation per step).  *la_out (host) receives the visited la whose
 * pruned fraction is closest to target_sparsity, *achieved_out (host, nullable) that fraction.
 * Follow with sp_select_unstructured_ex(la) to prune.
 */
sp_status sp_search_la(sp_ctx *ctx, const void *W, sp_dtype dtype, int64_t n_rows, int64_t ldw,
                       float target_sparsity, float alpha, float beta, int iterations,
                       float *la_out /* host */, double *achieved_out /* host */,
                       sp_stream stream);

/*
 * Section 3.3: N:M selection fused with the write-back.  Every row is cut into
 * contiguous groups of M columns starting at column 0; in each group the N
 * weights with the largest L (as in sp_score) are kept and the M-N smallest are
 * pruned; among equal scores the lower column is pruned first; a NaN score
 * ranks above every number.  M is 4 or 8, 0 < N < M, d_in % M == 0
 * (else SP_ERR_SHAPE).  2:4 keeps two of every four.
 */
sp_status sp_select_nm(sp_ctx *ctx, const void *W, sp_dtype dtype, int64_t n_rows, int64_t ldw,
                       int N, int M, uint32_t *mask_out, void *W_out, int64_t ldo,
                       sp_stream stream);

/*
 * Grouped selection.  Layers that read the same input (q/k/v; gate/up) share a context and the
 * per-channel factors, and Algorithm 1 treats every row on its own (its row loop is
 * parallel), so their rows can be pruned by one launch: small layers then no longer pay a
 * launch and a ramp-up each.  mats (HOST array, 1 <= n_mats <= SP_MAX_GROUP) lists the
 * matrices, all of `dtype`; every entry follows the rules of the single-matrix call (mask_out
 * and W_out nullable, W_out may alias W exactly).  The result for each matrix is identical to
 * that of its own sp_select_unstructured[_ex] / sp_select_nm call.  Matrices that do not allow
 * 16-byte access, or (N:M) ask for different outputs than their neighbours, get launches of
 * their own.
 */
enum { SP_MAX_GROUP = 8 };
typedef struct {
    const void *W;
    int64_t n_rows;
    int64_t ldw;
    uint32_t *mask_out;
    void *W_out;
    int64_t ldo;
} sp_matrix;
sp_status sp_select_unstructured_group(sp_ctx *ctx, const sp_matrix *mats /* host */, int n_mats,
                                       sp_dtype dtype, float sparsity,
                                       unsigned long long *counters, sp_stream stream);
sp_status sp_select_unstructured_group_ex(sp_ctx *ctx, const sp_matrix *mats /* host */, int n_mats,
                                          sp_dtype dtype, const sp_ewma_params *params /* host */,
                                          unsigned long long *counters, sp_stream stream);
sp_status sp_select_nm_group(sp_ctx *ctx, const sp_matrix *mats /* host */, int n_mats,
                             sp_dtype dtype, int N, int M, sp_stream stream);

/*
 * Algorithm 1 on matrices that read DIFFERENT layer inputs (all layers of a transformer block,
 * say), in one launch where their layouts allow: item i is mats[i] pruned with the statistics of
 * ctxs[i] (HOST arrays of n_items entries, 1 <= n_items <= SP_MAX_MULTI; a context may appear
 * more than once; all contexts on one device, each with calibration data, else
 * SP_ERR_INVALID_ARG / SP_ERR_STATE; mats[i] must be at least ctxs[i]'s d_in wide).  The rows
 * of Algorithm 1 are independent problems whatever matrix they belong to, so the result for
 * each matrix is identical to that of its own sp_select_unstructured[_ex] call on its context;
 * what changes is the cost: one launch, whose tail the short rows fill, instead of one launch
 * and one ramp-up per layer input.  Every context with batches pending is finalised on `stream`
 * first (all of them by one launch).  counters (nullable, device) are totals over all items.  sp_select_nm_multi is the
 * same for the N:M rule of Section 3.3 (every ctxs[i]'s d_in a multiple of M, else
 * SP_ERR_SHAPE; matrices that ask for different outputs than their neighbours, or do not allow
 * 16-byte access, get launches of their own).
 */
enum { SP_MAX_MULTI = 16 };
sp_status sp_select_unstructured_multi(sp_ctx *const *ctxs /* host */,
                                       const sp_matrix *mats /* host */, int n_items,
                                       sp_dtype dtype, float sparsity,
                                       unsigned long long *counters, sp_stream stream);
sp_status sp_select_nm_multi(sp_ctx *const *ctxs /* host */, const sp_matrix *mats /* host */,
                             int n_items, sp_dtype dtype, int N, int M, sp_stream stream);
sp_status sp_select_unstructured_multi_ex(sp_ctx *const *ctxs /* host */,
                                          const sp_matrix *mats /* host */, int n_items,
                                          sp_dtype dtype, const sp_ewma_params *params /* host */,
                                          unsigned long long *counters, sp_stream stream);

/*
 * Section 3.3, compressed output: 2:4 selection (exactly as sp_select_nm with N = 2, M = 4)
 * written as the kept values plus per-group indices in the same pass, so that a consumer of
 * 2:4 sparsity needs no dense pruned matrix and no separate conversion step (Section 3.3 makes
 * the same point about the 2:4 pattern and sparse hardware).  The layout is this library's own:
 *   values_out  [n_rows, d_in/2] of `dtype`, leading dimension ldv (elements, >= d_in/2): the
 *               two kept weights of group g of a row at columns 2g, 2g+1, in column order,
 *               copied bit for bit;
 *   meta_out    [n_rows, ceil(d_in/32)] uint32, no padding between rows: bits 4g..4g+3 of
 *               word k describe group 8k+g as  idx0 | idx1 << 2,  idx0 < idx1 being the
 *               positions (0..3) of the kept weights inside the group; bits past d_in/4 groups
 *               are 0.
 * d_in % 4 == 0 (else SP_ERR_SHAPE).  The fast path needs values_out 8-byte aligned and
 * ldv % 4 == 0 in addition to the usual conditions on W.
 */
sp_status sp_select_24_compressed(sp_ctx *ctx, const void *W, sp_dtype dtype, int64_t n_rows,
                                  int64_t ldw, void *values_out, int64_t ldv, uint32_t *meta_out,
                                  sp_stream stream);

/*
 * Algorithm 1's write-back on its own: W_out = W where the mask bit is 1, +0
 * elsewhere.  W_out may alias W exactly.  Needs no context.
 */
sp_status sp_apply_mask(const void *W, sp_dtype dtype, int64_t n_rows, int64_t n_cols, int64_t ldw,
                        const uint32_t *mask, void *W_out, int64_t ldo, sp_stream stream);

/* ------------------------------------------------------------------ host-buffer variants */

/*
 * The same operations (Algorithm 1 step 1; Section 3.3; Algorithm 1) for data that lives in
 * HOST memory: X_host, W_host, mask_host and W_out_host are host pointers (pinned memory lets
 * the transfers overlap the kernels; pageable memory works but copies synchronously).  The
 * matrix is streamed through two device staging slots of 64 MiB owned by the context (created,
 * together with two internal streams, by the first such call on a context - that call
 * allocates): host->device copy, kernel and device->host copy of successive row chunks overlap.
 * Work is ordered after everything already queued on `stream`, and `stream` completes only
 * after the last result has reached the host; the calls themselves do not wait.  mask_host and
 * W_out_host may each be NULL; W_out_host may equal W_host (same ld) for in-place pruning.
 * Results are identical to the device-pointer calls.
 */
sp_status sp_calib_accumulate_host(sp_ctx *ctx, const void *X_host, sp_dtype dtype,
                                   int64_t n_tokens, int64_t ldx, sp_stream stream);
sp_status sp_select_nm_host(sp_ctx *ctx, const void *W_host, sp_dtype dtype, int64_t n_rows,
                            int64_t ldw, int N, int M, uint32_t *mask_host, void *W_out_host,
                            int64_t ldo, sp_stream stream);
sp_status sp_select_unstructured_host(sp_ctx *ctx, const void *W_host, sp_dtype dtype,
                                      int64_t n_rows, int64_t ldw, float sparsity,
                                      uint32_t *mask_host, void *W_out_host, int64_t ldo,
                                      sp_stream stream);

/* ------------------------------------------------------------------ diagnostics */

/*
 * Index checks of the debug build (python -m paper_2501_16376_b200.build --debug ->
 * libswiftprune_debug.so, same ABI).  In that build the kernels check the indices of their
 * stores; an out-of-range access is skipped and recorded instead of faulting (nothing traps).
 * *violations receives the number of skipped accesses on the current device since the last
 * clear (-1 in the release build, which compiles no checks); first_code / first_index /
 * first_limit (nullable) describe the first one (codes in csrc/sp_debug.cuh); clear != 0 resets
 * the records.  Synchronises the device.
 */
sp_status sp_debug_status(int *violations /* host */, int *first_code /* host */,
                          int64_t *first_index /* host */, int64_t *first_limit /* host */,
                          int clear);

const char *sp_status_string(sp_status status);
/* Text of the last CUDA error this thread saw inside the library ("" if none). */
const char *sp_last_cuda_error(void);
/* Kernels launched by the library since it was loaded (all threads). */
uint64_t sp_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* SWIFTPRUNE_H_ */
