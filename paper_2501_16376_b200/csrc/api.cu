// C ABI of the library: argument validation on the host, context management, dispatch to
// the kernel launchers.  Nothing here synchronises unless the header says so.
#include <algorithm>
#include <atomic>
#include <cmath>
#include <cstdio>
#include <cstring>
#include <new>
#include <vector>

#include <nvtx3/nvToolsExt.h>

#include "sp_internal.h"

namespace sp {

static thread_local char g_cuda_error[256] = "";
// readers of the per-translation-unit index-check records (debug build only; see sp_debug.cuh)
static DebugReader g_debug_readers[16];
static int g_debug_reader_count = 0;

void register_debug_reader(DebugReader reader) {
    if (g_debug_reader_count < 16) g_debug_readers[g_debug_reader_count++] = reader;
}

static std::atomic<uint64_t> g_launches{0};

sp_status cuda_fail(cudaError_t e) {
    snprintf(g_cuda_error, sizeof g_cuda_error, "%s: %s", cudaGetErrorName(e),
             cudaGetErrorString(e));
    return e == cudaErrorMemoryAllocation ? SP_ERR_NOMEM : SP_ERR_CUDA;
}

void count_launch(int n) { g_launches.fetch_add(static_cast<uint64_t>(n)); }

// Makes the context's device current for the scope of one call.
class DeviceGuard {
   public:
    explicit DeviceGuard(int device) {
        if (cudaGetDevice(&prev_) != cudaSuccess) prev_ = -1;
        if (prev_ != device) {
            err_ = cudaSetDevice(device);
            switched_ = err_ == cudaSuccess;
        }
    }
    ~DeviceGuard() {
        if (switched_ && prev_ >= 0) cudaSetDevice(prev_);
    }
    cudaError_t error() const { return err_; }

   private:
    int prev_ = -1;
    bool switched_ = false;
    cudaError_t err_ = cudaSuccess;
};

// NVTX range around one entry point: shows up in a timeline profile under the call's name;
// costs a function-pointer test when no profiler is attached.
class CallRange {
   public:
    explicit CallRange(const char *name) { nvtxRangePushA(name); }
    ~CallRange() { nvtxRangePop(); }
    CallRange(const CallRange &) = delete;
    CallRange &operator=(const CallRange &) = delete;
};
#define SP_CALL_RANGE() CallRange sp_call_range__(__func__)

static bool valid_dtype(sp_dtype d) { return d == SP_F16 || d == SP_BF16; }

static bool ewma_params_valid(const sp_ewma_params *params) {
    if (params == nullptr) return false;
    if (!(params->alpha > 0.0f) || !(params->alpha <= 1.0f) || !(params->beta > 0.0f) ||
        !(params->beta <= 1.0f) || !std::isfinite(params->la))
        return false;
    return params->s_update == SP_S_GATED || params->s_update == SP_S_FROZEN ||
           params->s_update == SP_S_LITERAL_W2 || params->s_update == SP_S_READING_X2 ||
           params->s_update == SP_S_LITERAL_SCAN;
}

static sp_status ensure_finalized(sp_ctx *ctx, cudaStream_t stream) {
    if (ctx->n_tokens <= 0) return SP_ERR_STATE;
    if (!ctx->dirty) return SP_OK;
    return launch_finalize(ctx, stream);
}

static sp_status check_matrix_args(const sp_ctx *ctx, const void *W, sp_dtype dtype,
                                   int64_t n_rows, int64_t ldw, const void *W_out, int64_t ldo) {
    if (ctx == nullptr) return SP_ERR_INVALID_ARG;
    if (!valid_dtype(dtype)) return SP_ERR_DTYPE;
    if (n_rows < 0) return SP_ERR_INVALID_ARG;
    if (W == nullptr && n_rows != 0) return SP_ERR_INVALID_ARG;  // an empty matrix has no address
    if (ldw < ctx->d_in) return SP_ERR_SHAPE;
    if (W_out != nullptr) {
        if (ldo < ctx->d_in) return SP_ERR_SHAPE;
        if (W_out == W && ldo != ldw) return SP_ERR_SHAPE;
    }
    return SP_OK;
}

}  // namespace sp

using namespace sp;

extern "C" {

sp_status sp_create(sp_ctx **out, int64_t d_in, int device) {
    SP_CALL_RANGE();
    if (out == nullptr) return SP_ERR_INVALID_ARG;
    *out = nullptr;
    if (d_in < 1 || d_in > kMaxDin) return SP_ERR_SHAPE;
    int count = 0;
    cudaError_t e = cudaGetDeviceCount(&count);
    if (e != cudaSuccess) return cuda_fail(e);
    if (device < 0 || device >= count) return SP_ERR_INVALID_ARG;
    DeviceGuard guard(device);
    if (guard.error() != cudaSuccess) return cuda_fail(guard.error());

    sp_ctx *ctx = new (std::nothrow) sp_ctx();
    if (ctx == nullptr) return SP_ERR_NOMEM;
    ctx->device = device;
    ctx->d_in = d_in;
    ctx->n_pad = (d_in + kStripChannels - 1) / kStripChannels * kStripChannels;
    ctx->strips = static_cast<int>(ctx->n_pad / kStripChannels);
    ctx->n_tokens = 0;
    ctx->slabs_valid = 0;
    ctx->dirty = false;
    ctx->host_pipe = nullptr;
    e = cudaDeviceGetAttribute(&ctx->sm_count, cudaDevAttrMultiProcessorCount, device);
    if (e != cudaSuccess) { delete ctx; return cuda_fail(e); }
    ctx->calib_blocks_per_sm = calib_query_blocks_per_sm();

    const size_t np = static_cast<size_t>(ctx->n_pad);
    constexpr int kBuffers = 6;
    void *ptrs[kBuffers] = {nullptr, nullptr, nullptr, nullptr, nullptr, nullptr};
    const size_t sizes[kBuffers] = {sizeof(double) * np * kMaxSlabs, sizeof(double) * np,
                                    sizeof(double) * static_cast<size_t>(ctx->strips),
                                    sizeof(float) * (np + kStripChannels),
                                    sizeof(DeviceScalars),
                                    sizeof(float) * ((np + 511) / 512 * 512 + 512)};
    for (int i = 0; i < kBuffers; ++i) {
        e = cudaMalloc(&ptrs[i], sizes[i]);
        if (e == cudaSuccess) e = cudaMemset(ptrs[i], 0, sizes[i]);
        if (e != cudaSuccess) {
            for (int j = 0; j <= i; ++j) cudaFree(ptrs[j]);
            delete ctx;
            return cuda_fail(e);
        }
    }
    ctx->partial = static_cast<double *>(ptrs[0]);
    ctx->colsq = static_cast<double *>(ptrs[1]);
    ctx->strip_sum = static_cast<double *>(ptrs[2]);
    ctx->factor = static_cast<float *>(ptrs[3]);
    ctx->scalars = static_cast<DeviceScalars *>(ptrs[4]);
    ctx->factor_pairs = static_cast<float *>(ptrs[5]);
    e = cudaDeviceSynchronize();
    if (e != cudaSuccess) { sp_destroy(ctx); return cuda_fail(e); }
    *out = ctx;
    return SP_OK;
}

sp_status sp_destroy(sp_ctx *ctx) {
    SP_CALL_RANGE();
    if (ctx == nullptr) return SP_OK;
    DeviceGuard guard(ctx->device);
    cudaDeviceSynchronize();
    host_pipe_destroy(ctx->host_pipe);
    cudaFree(ctx->partial);
    cudaFree(ctx->colsq);
    cudaFree(ctx->strip_sum);
    cudaFree(ctx->factor);
    cudaFree(ctx->factor_pairs);
    cudaFree(ctx->scalars);
    delete ctx;
    return SP_OK;
}

sp_status sp_calib_reset(sp_ctx *ctx, sp_stream stream) {
    SP_CALL_RANGE();
    (void)stream;  // the partial sums are overwritten, not cleared, by the next batch
    if (ctx == nullptr) return SP_ERR_INVALID_ARG;
    ctx->n_tokens = 0;
    ctx->slabs_valid = 0;
    ctx->dirty = false;
    return SP_OK;
}

sp_status sp_calib_accumulate_ex(sp_ctx *ctx, const void *X, sp_dtype dtype, int64_t n_tokens,
                                 int64_t ldx, unsigned flags, sp_stream stream) {
    SP_CALL_RANGE();
    if (ctx == nullptr) return SP_ERR_INVALID_ARG;
    if (!valid_dtype(dtype)) return SP_ERR_DTYPE;
    if (n_tokens < 0 || (flags & ~static_cast<unsigned>(SP_CALIB_X_COMPLETE)) != 0u)
        return SP_ERR_INVALID_ARG;
    if (n_tokens == 0) return SP_OK;
    if (X == nullptr) return SP_ERR_INVALID_ARG;
    if (ldx < ctx->d_in) return SP_ERR_SHAPE;
    DeviceGuard guard(ctx->device);
    if (guard.error() != cudaSuccess) return cuda_fail(guard.error());
    return launch_calib_accumulate(ctx, X, dtype, n_tokens, ldx, static_cast<cudaStream_t>(stream),
                                   (flags & SP_CALIB_X_COMPLETE) != 0u);
}

sp_status sp_calib_accumulate_multi(sp_ctx *const *ctxs, const sp_batch *batches, int n_items,
                                    sp_dtype dtype, unsigned flags, sp_stream stream) {
    SP_CALL_RANGE();
    if (ctxs == nullptr || batches == nullptr) return SP_ERR_INVALID_ARG;
    if (n_items < 1 || n_items > SP_MAX_MULTI) return SP_ERR_INVALID_ARG;
    if (!valid_dtype(dtype)) return SP_ERR_DTYPE;
    if ((flags & ~static_cast<unsigned>(SP_CALIB_X_COMPLETE)) != 0u) return SP_ERR_INVALID_ARG;
    for (int i = 0; i < n_items; ++i) {
        if (ctxs[i] == nullptr || batches[i].n_tokens < 0) return SP_ERR_INVALID_ARG;
        if (batches[i].n_tokens > 0 && batches[i].X == nullptr) return SP_ERR_INVALID_ARG;
        if (batches[i].ldx < ctxs[i]->d_in) return SP_ERR_SHAPE;
        if (ctxs[i]->device != ctxs[0]->device) return SP_ERR_INVALID_ARG;
        for (int k = 0; k < i; ++k)  // two batches of one launch cannot update the same sums
            if (ctxs[k] == ctxs[i]) return SP_ERR_INVALID_ARG;
    }
    DeviceGuard guard(ctxs[0]->device);
    if (guard.error() != cudaSuccess) return cuda_fail(guard.error());
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const bool x_complete = (flags & SP_CALIB_X_COMPLETE) != 0u;
    // batches that allow 16-byte access share launches of up to 8; the others go one by one
    sp_ctx *group_ctx[8];
    CalibItem group[8];
    int n_group = 0;
    auto flush = [&]() -> sp_status {
        sp_status st = SP_OK;
        if (n_group == 1)
            st = launch_calib_accumulate(group_ctx[0], group[0].X, dtype, group[0].n_tokens,
                                         group[0].ldx, s, x_complete);
        else if (n_group > 1)
            st = launch_calib_accumulate_multi(group_ctx, group, n_group, dtype, s, x_complete);
        n_group = 0;
        return st;
    };
    for (int i = 0; i < n_items; ++i) {
        const sp_batch &b = batches[i];
        if (b.n_tokens == 0) continue;
        if (!calib_multi_applies(ctxs[i], b.X, b.ldx, b.n_tokens)) {
            sp_status st = launch_calib_accumulate(ctxs[i], b.X, dtype, b.n_tokens, b.ldx, s, x_complete);
            if (st != SP_OK) return st;
            continue;
        }
        group_ctx[n_group] = ctxs[i];
        group[n_group] = CalibItem{b.X, b.n_tokens, b.ldx};
        if (++n_group == 8) {
            sp_status st = flush();
            if (st != SP_OK) return st;
        }
    }
    return flush();
}

sp_status sp_calib_accumulate(sp_ctx *ctx, const void *X, sp_dtype dtype, int64_t n_tokens,
                              int64_t ldx, sp_stream stream) {
    SP_CALL_RANGE();
    return sp_calib_accumulate_ex(ctx, X, dtype, n_tokens, ldx, 0u, stream);
}

sp_status sp_get_stats(sp_ctx *ctx, double *colsq_host, double *S_host, float *factor_host,
                       int64_t *n_tokens_host, sp_stream stream) {
    SP_CALL_RANGE();
    if (ctx == nullptr) return SP_ERR_INVALID_ARG;
    if (n_tokens_host != nullptr) *n_tokens_host = ctx->n_tokens;
    if (ctx->n_tokens <= 0) return SP_ERR_STATE;
    DeviceGuard guard(ctx->device);
    if (guard.error() != cudaSuccess) return cuda_fail(guard.error());
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    sp_status st = ensure_finalized(ctx, s);
    if (st != SP_OK) return st;
    DeviceScalars sc;
    cudaError_t e = cudaMemcpyAsync(&sc, ctx->scalars, sizeof sc, cudaMemcpyDeviceToHost, s);
    if (e == cudaSuccess && colsq_host != nullptr)
        e = cudaMemcpyAsync(colsq_host, ctx->colsq, sizeof(double) * ctx->d_in,
                            cudaMemcpyDeviceToHost, s);
    if (e == cudaSuccess && factor_host != nullptr)
        e = cudaMemcpyAsync(factor_host, ctx->factor, sizeof(float) * ctx->d_in,
                            cudaMemcpyDeviceToHost, s);
    if (e == cudaSuccess) e = cudaStreamSynchronize(s);
    if (e != cudaSuccess) return cuda_fail(e);
    if (S_host != nullptr) *S_host = sc.S;
    return (sc.flags & kFlagDegenerate) ? SP_ERR_DEGENERATE : SP_OK;
}

sp_status sp_set_stats(sp_ctx *ctx, const double *colsq_host, int64_t n_tokens, sp_stream stream) {
    SP_CALL_RANGE();
    if (ctx == nullptr || colsq_host == nullptr || n_tokens <= 0) return SP_ERR_INVALID_ARG;
    DeviceGuard guard(ctx->device);
    if (guard.error() != cudaSuccess) return cuda_fail(guard.error());
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    // The statistics become slab row 0 of the partial sums; the padding stays zero.
    cudaError_t e = cudaMemsetAsync(ctx->partial, 0, sizeof(double) * ctx->n_pad, s);
    if (e == cudaSuccess)
        e = cudaMemcpyAsync(ctx->partial, colsq_host, sizeof(double) * ctx->d_in,
                            cudaMemcpyHostToDevice, s);
    if (e == cudaSuccess) e = cudaStreamSynchronize(s);
    if (e != cudaSuccess) return cuda_fail(e);
    ctx->n_tokens = n_tokens;
    ctx->slabs_valid = 1;
    ctx->dirty = true;
    return SP_OK;
}

sp_status sp_calib_stats_noalloc(const void *X, sp_dtype dtype, int64_t n_tokens, int64_t d_in,
                                 int64_t ldx, double *colsq_out, float *factor_out, double *S_out,
                                 sp_stream stream) {
    SP_CALL_RANGE();
    if (!valid_dtype(dtype)) return SP_ERR_DTYPE;
    if (X == nullptr || n_tokens < 1) return SP_ERR_INVALID_ARG;
    if (d_in < 1 || d_in > calib_static_max_d_in()) return SP_ERR_SHAPE;
    if (ldx < d_in) return SP_ERR_SHAPE;
    int device = -1;
    cudaError_t e = cudaGetDevice(&device);
    if (e != cudaSuccess) return cuda_fail(e);
    return launch_calib_stats_static(device, X, dtype, n_tokens, d_in, ldx, colsq_out, factor_out,
                                     S_out, static_cast<cudaStream_t>(stream));
}

sp_status sp_score(sp_ctx *ctx, const void *W, sp_dtype dtype, int64_t n_rows, int64_t ldw,
                   float *scores_out, sp_stream stream) {
    SP_CALL_RANGE();
    if (ctx == nullptr) return SP_ERR_INVALID_ARG;
    if (scores_out != nullptr) {
        sp_status st = check_matrix_args(ctx, W, dtype, n_rows, ldw, nullptr, 0);
        if (st != SP_OK) return st;
    }
    if (ctx->n_tokens <= 0) return SP_ERR_STATE;
    DeviceGuard guard(ctx->device);
    if (guard.error() != cudaSuccess) return cuda_fail(guard.error());
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    sp_status st = ensure_finalized(ctx, s);
    if (st != SP_OK || scores_out == nullptr) return st;
    return launch_score(ctx, W, dtype, n_rows, ldw, scores_out, s);
}

sp_status sp_finalize_multi(sp_ctx *const *ctxs, int n_items, sp_stream stream) {
    SP_CALL_RANGE();
    if (ctxs == nullptr || n_items < 1 || n_items > SP_MAX_MULTI) return SP_ERR_INVALID_ARG;
    for (int i = 0; i < n_items; ++i) {
        if (ctxs[i] == nullptr || ctxs[i]->device != ctxs[0]->device) return SP_ERR_INVALID_ARG;
        if (ctxs[i]->n_tokens <= 0) return SP_ERR_STATE;
    }
    DeviceGuard guard(ctxs[0]->device);
    if (guard.error() != cudaSuccess) return cuda_fail(guard.error());
    return launch_finalize_pending(ctxs, n_items, static_cast<cudaStream_t>(stream));
}

sp_status sp_la_for_sparsity(float sparsity, float *la_out) {
    SP_CALL_RANGE();
    if (la_out == nullptr || !(sparsity > 0.0f) || !(sparsity < 1.0f)) return SP_ERR_INVALID_ARG;
    // Table 3: pruning ratio (%) -> la.
    static const double pct[5] = {50.0, 60.0, 70.0, 80.0, 90.0};
    static const double la[5] = {0.5, 0.2, -0.2, -0.9, -1.5};
    const double x = static_cast<double>(sparsity) * 100.0;
    for (int i = 0; i < 5; ++i) {
        if (std::fabs(x - pct[i]) < 1e-4) {
            *la_out = static_cast<float>(la[i]);
            return SP_OK;
        }
    }
    int i = 0;
    if (x >= pct[4]) {
        i = 3;
    } else {
        while (i < 3 && x >= pct[i + 1]) ++i;
    }
    const double t = (x - pct[i]) / (pct[i + 1] - pct[i]);
    *la_out = static_cast<float>(la[i] + t * (la[i + 1] - la[i]));
    return SP_OK;
}

sp_status sp_select_unstructured_ex(sp_ctx *ctx, const void *W, sp_dtype dtype, int64_t n_rows,
                                    int64_t ldw, const sp_ewma_params *params, uint32_t *mask_out,
                                    void *W_out, int64_t ldo, unsigned long long *counters,
                                    sp_stream stream) {
    SP_CALL_RANGE();
    sp_status st = check_matrix_args(ctx, W, dtype, n_rows, ldw, W_out, ldo);
    if (st != SP_OK) return st;
    if (!ewma_params_valid(params)) return SP_ERR_INVALID_ARG;
    if (ctx->n_tokens <= 0) return SP_ERR_STATE;
    DeviceGuard guard(ctx->device);
    if (guard.error() != cudaSuccess) return cuda_fail(guard.error());
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    st = ensure_finalized(ctx, s);
    if (st != SP_OK) return st;
    return launch_select_ewma(ctx, W, dtype, n_rows, ldw, *params, mask_out, W_out, ldo, counters, s);
}

sp_status sp_select_unstructured(sp_ctx *ctx, const void *W, sp_dtype dtype, int64_t n_rows,
                                 int64_t ldw, float sparsity, uint32_t *mask_out, void *W_out,
                                 int64_t ldo, unsigned long long *counters, sp_stream stream) {
    SP_CALL_RANGE();
    sp_ewma_params p;
    p.alpha = 0.125f;  // Section 4.2
    p.beta = 0.125f;
    p.s_update = SP_S_GATED;
    sp_status st = sp_la_for_sparsity(sparsity, &p.la);
    if (st != SP_OK) return st;
    return sp_select_unstructured_ex(ctx, W, dtype, n_rows, ldw, &p, mask_out, W_out, ldo, counters,
                                     stream);
}

// Validates a group of matrices and converts it to launch jobs.
static sp_status group_jobs(const sp_ctx *ctx, const sp_matrix *mats, int n_mats, sp_dtype dtype,
                            EwmaLaunchJob *jobs) {
    if (ctx == nullptr || mats == nullptr) return SP_ERR_INVALID_ARG;
    if (n_mats < 1 || n_mats > SP_MAX_GROUP) return SP_ERR_INVALID_ARG;
    for (int i = 0; i < n_mats; ++i) {
        const sp_matrix &m = mats[i];
        sp_status st = check_matrix_args(ctx, m.W, dtype, m.n_rows, m.ldw, m.W_out, m.ldo);
        if (st != SP_OK) return st;
        jobs[i] = EwmaLaunchJob{m.W, m.W_out, m.mask_out, m.n_rows, m.ldw, m.ldo};
    }
    return SP_OK;
}

sp_status sp_select_unstructured_group_ex(sp_ctx *ctx, const sp_matrix *mats, int n_mats,
                                          sp_dtype dtype, const sp_ewma_params *params,
                                          unsigned long long *counters, sp_stream stream) {
    SP_CALL_RANGE();
    EwmaLaunchJob jobs[SP_MAX_GROUP];
    sp_status st = group_jobs(ctx, mats, n_mats, dtype, jobs);
    if (st != SP_OK) return st;
    if (!ewma_params_valid(params)) return SP_ERR_INVALID_ARG;
    if (ctx->n_tokens <= 0) return SP_ERR_STATE;
    DeviceGuard guard(ctx->device);
    if (guard.error() != cudaSuccess) return cuda_fail(guard.error());
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    st = ensure_finalized(ctx, s);
    if (st != SP_OK) return st;
    return launch_select_ewma(ctx, jobs, n_mats, dtype, *params, counters, s);
}

sp_status sp_select_unstructured_group(sp_ctx *ctx, const sp_matrix *mats, int n_mats,
                                       sp_dtype dtype, float sparsity,
                                       unsigned long long *counters, sp_stream stream) {
    SP_CALL_RANGE();
    sp_ewma_params p;
    p.alpha = 0.125f;  // Section 4.2
    p.beta = 0.125f;
    p.s_update = SP_S_GATED;
    sp_status st = sp_la_for_sparsity(sparsity, &p.la);
    if (st != SP_OK) return st;
    return sp_select_unstructured_group_ex(ctx, mats, n_mats, dtype, &p, counters, stream);
}

sp_status sp_select_unstructured_multi_ex(sp_ctx *const *ctxs, const sp_matrix *mats, int n_items,
                                          sp_dtype dtype, const sp_ewma_params *params,
                                          unsigned long long *counters, sp_stream stream) {
    SP_CALL_RANGE();
    if (ctxs == nullptr || mats == nullptr) return SP_ERR_INVALID_ARG;
    if (n_items < 1 || n_items > SP_MAX_MULTI) return SP_ERR_INVALID_ARG;
    if (!ewma_params_valid(params)) return SP_ERR_INVALID_ARG;
    EwmaLaunchJob jobs[SP_MAX_MULTI];
    for (int i = 0; i < n_items; ++i) {
        const sp_matrix &m = mats[i];
        if (ctxs[i] == nullptr) return SP_ERR_INVALID_ARG;
        sp_status st = check_matrix_args(ctxs[i], m.W, dtype, m.n_rows, m.ldw, m.W_out, m.ldo);
        if (st != SP_OK) return st;
        if (ctxs[i]->device != ctxs[0]->device) return SP_ERR_INVALID_ARG;
        if (ctxs[i]->n_tokens <= 0) return SP_ERR_STATE;
        jobs[i] = EwmaLaunchJob{m.W, m.W_out, m.mask_out, m.n_rows, m.ldw, m.ldo, ctxs[i]};
    }
    // Longest rows first: the CTAs of a launch start in this order, and the launch ends soonest
    // when the rows that take longest are not the ones left for its tail.
    std::stable_sort(jobs, jobs + n_items, [](const EwmaLaunchJob &x, const EwmaLaunchJob &y) {
        return x.ctx->d_in > y.ctx->d_in;
    });
    DeviceGuard guard(ctxs[0]->device);
    if (guard.error() != cudaSuccess) return cuda_fail(guard.error());
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    sp_status fin = launch_finalize_pending(ctxs, n_items, s);  // one launch for all that need it
    if (fin != SP_OK) return fin;
    return launch_select_ewma(ctxs[0], jobs, n_items, dtype, *params, counters, s);
}

sp_status sp_select_unstructured_multi(sp_ctx *const *ctxs, const sp_matrix *mats, int n_items,
                                       sp_dtype dtype, float sparsity,
                                       unsigned long long *counters, sp_stream stream) {
    SP_CALL_RANGE();
    sp_ewma_params p;
    p.alpha = 0.125f;  // Section 4.2
    p.beta = 0.125f;
    p.s_update = SP_S_GATED;
    sp_status st = sp_la_for_sparsity(sparsity, &p.la);
    if (st != SP_OK) return st;
    return sp_select_unstructured_multi_ex(ctxs, mats, n_items, dtype, &p, counters, stream);
}

sp_status sp_select_nm_group(sp_ctx *ctx, const sp_matrix *mats, int n_mats, sp_dtype dtype, int N,
                             int M, sp_stream stream) {
    SP_CALL_RANGE();
    EwmaLaunchJob jobs[SP_MAX_GROUP];
    sp_status st = group_jobs(ctx, mats, n_mats, dtype, jobs);
    if (st != SP_OK) return st;
    if (M != 4 && M != 8) return SP_ERR_INVALID_ARG;
    if (N <= 0 || N >= M) return SP_ERR_INVALID_ARG;
    if (ctx->d_in % M != 0) return SP_ERR_SHAPE;
    if (ctx->n_tokens <= 0) return SP_ERR_STATE;
    DeviceGuard guard(ctx->device);
    if (guard.error() != cudaSuccess) return cuda_fail(guard.error());
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    st = ensure_finalized(ctx, s);
    if (st != SP_OK) return st;
    return launch_select_nm(ctx, jobs, n_mats, dtype, N, M, s);
}

sp_status sp_select_nm_multi(sp_ctx *const *ctxs, const sp_matrix *mats, int n_items,
                             sp_dtype dtype, int N, int M, sp_stream stream) {
    SP_CALL_RANGE();
    if (ctxs == nullptr || mats == nullptr) return SP_ERR_INVALID_ARG;
    if (n_items < 1 || n_items > SP_MAX_MULTI) return SP_ERR_INVALID_ARG;
    if (M != 4 && M != 8) return SP_ERR_INVALID_ARG;
    if (N <= 0 || N >= M) return SP_ERR_INVALID_ARG;
    EwmaLaunchJob jobs[SP_MAX_MULTI];
    for (int i = 0; i < n_items; ++i) {
        const sp_matrix &m = mats[i];
        if (ctxs[i] == nullptr) return SP_ERR_INVALID_ARG;
        sp_status st = check_matrix_args(ctxs[i], m.W, dtype, m.n_rows, m.ldw, m.W_out, m.ldo);
        if (st != SP_OK) return st;
        if (ctxs[i]->device != ctxs[0]->device) return SP_ERR_INVALID_ARG;
        if (ctxs[i]->d_in % M != 0) return SP_ERR_SHAPE;
        if (ctxs[i]->n_tokens <= 0) return SP_ERR_STATE;
        jobs[i] = EwmaLaunchJob{m.W, m.W_out, m.mask_out, m.n_rows, m.ldw, m.ldo, ctxs[i]};
    }
    DeviceGuard guard(ctxs[0]->device);
    if (guard.error() != cudaSuccess) return cuda_fail(guard.error());
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    sp_status fin = launch_finalize_pending(ctxs, n_items, s);  // one launch for all that need it
    if (fin != SP_OK) return fin;
    return launch_select_nm(ctxs[0], jobs, n_items, dtype, N, M, s);
}

sp_status sp_ewma_trace(sp_ctx *ctx, const void *W, sp_dtype dtype, int64_t n_rows, int64_t ldw,
                        const sp_ewma_params *params, float *est_out, float *dev_out,
                        float *scores_out, sp_stream stream) {
    SP_CALL_RANGE();
    sp_status st = check_matrix_args(ctx, W, dtype, n_rows, ldw, nullptr, 0);
    if (st != SP_OK) return st;
    if (params == nullptr || !(params->alpha > 0.0f) || !(params->alpha <= 1.0f) ||
        !(params->beta > 0.0f) || !(params->beta <= 1.0f) || !std::isfinite(params->la))
        return SP_ERR_INVALID_ARG;
    if (params->s_update != SP_S_GATED && params->s_update != SP_S_FROZEN &&
        params->s_update != SP_S_LITERAL_W2 && params->s_update != SP_S_READING_X2 &&
        params->s_update != SP_S_LITERAL_SCAN)
        return SP_ERR_INVALID_ARG;
    if (ctx->n_tokens <= 0) return SP_ERR_STATE;
    DeviceGuard guard(ctx->device);
    if (guard.error() != cudaSuccess) return cuda_fail(guard.error());
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    st = ensure_finalized(ctx, s);
    if (st != SP_OK) return st;
    return launch_ewma_trace(ctx, W, dtype, n_rows, ldw, *params, est_out, dev_out, scores_out, s);
}

sp_status sp_search_la(sp_ctx *ctx, const void *W, sp_dtype dtype, int64_t n_rows, int64_t ldw,
                       float target_sparsity, float alpha, float beta, int iterations,
                       float *la_out, double *achieved_out, sp_stream stream) {
    SP_CALL_RANGE();
    sp_status st = check_matrix_args(ctx, W, dtype, n_rows, ldw, nullptr, 0);
    if (st != SP_OK) return st;
    if (la_out == nullptr || !(target_sparsity > 0.0f) || !(target_sparsity < 1.0f) ||
        !(alpha > 0.0f) || !(alpha <= 1.0f) || !(beta > 0.0f) || !(beta <= 1.0f) ||
        iterations < 1 || iterations > 64 || n_rows < 1)
        return SP_ERR_INVALID_ARG;
    if (ctx->n_tokens <= 0) return SP_ERR_STATE;
    DeviceGuard guard(ctx->device);
    if (guard.error() != cudaSuccess) return cuda_fail(guard.error());
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    st = ensure_finalized(ctx, s);
    if (st != SP_OK) return st;
    // The pruned fraction never increases with la (the threshold est - la*dev only moves down
    // and, with S frozen, est and dev do not depend on the decisions): bisection on [-8, 8].
    // Rows that allow 16-byte access: the whole bisection runs on the device, one
    // synchronisation at the end.
    if (ewma_pair_path_applies(W, ldw, ctx->d_in))
        return launch_search_la_device(ctx, W, dtype, n_rows, ldw, target_sparsity, alpha, beta,
                                       iterations, la_out, achieved_out, s);
    const double total = static_cast<double>(n_rows) * static_cast<double>(ctx->d_in);
    float lo = -8.0f, hi = 8.0f, best_la = 0.0f;
    double best_gap = 2.0, best_frac = 0.0;
    unsigned long long *counters = ctx->scalars->search_counters;
    for (int it = 0; it < iterations; ++it) {
        sp_ewma_params p;
        p.alpha = alpha;
        p.beta = beta;
        p.la = 0.5f * (lo + hi);
        p.s_update = SP_S_FROZEN;
        cudaError_t e = cudaMemsetAsync(counters, 0, sizeof(unsigned long long) * SP_NUM_COUNTERS, s);
        if (e != cudaSuccess) return cuda_fail(e);
        st = launch_select_ewma(ctx, W, dtype, n_rows, ldw, p, nullptr, nullptr, ldw, counters, s);
        if (st != SP_OK) return st;
        unsigned long long host[SP_NUM_COUNTERS];
        e = cudaMemcpyAsync(host, counters, sizeof host, cudaMemcpyDeviceToHost, s);
        if (e == cudaSuccess) e = cudaStreamSynchronize(s);
        if (e != cudaSuccess) return cuda_fail(e);
        const double pruned = 1.0 - static_cast<double>(host[SP_COUNTER_KEPT]) / total;
        const double gap = std::fabs(pruned - static_cast<double>(target_sparsity));
        if (gap < best_gap) {
            best_gap = gap;
            best_la = p.la;
            best_frac = pruned;
        }
        if (pruned > static_cast<double>(target_sparsity))
            lo = p.la;  // too much pruned: raise la
        else
            hi = p.la;
    }
    *la_out = best_la;
    if (achieved_out != nullptr) *achieved_out = best_frac;
    return SP_OK;
}

sp_status sp_select_nm(sp_ctx *ctx, const void *W, sp_dtype dtype, int64_t n_rows, int64_t ldw,
                       int N, int M, uint32_t *mask_out, void *W_out, int64_t ldo,
                       sp_stream stream) {
    SP_CALL_RANGE();
    sp_status st = check_matrix_args(ctx, W, dtype, n_rows, ldw, W_out, ldo);
    if (st != SP_OK) return st;
    if (M != 4 && M != 8) return SP_ERR_INVALID_ARG;
    if (N <= 0 || N >= M) return SP_ERR_INVALID_ARG;
    if (ctx->d_in % M != 0) return SP_ERR_SHAPE;
    if (ctx->n_tokens <= 0) return SP_ERR_STATE;
    DeviceGuard guard(ctx->device);
    if (guard.error() != cudaSuccess) return cuda_fail(guard.error());
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    st = ensure_finalized(ctx, s);
    if (st != SP_OK) return st;
    return launch_select_nm(ctx, W, dtype, n_rows, ldw, N, M, mask_out, W_out, ldo, s);
}

sp_status sp_select_24_compressed(sp_ctx *ctx, const void *W, sp_dtype dtype, int64_t n_rows,
                                  int64_t ldw, void *values_out, int64_t ldv, uint32_t *meta_out,
                                  sp_stream stream) {
    SP_CALL_RANGE();
    sp_status st = check_matrix_args(ctx, W, dtype, n_rows, ldw, nullptr, 0);
    if (st != SP_OK) return st;
    if (n_rows > 0 && (values_out == nullptr || meta_out == nullptr)) return SP_ERR_INVALID_ARG;
    if (ctx->d_in % 4 != 0 || ldv < ctx->d_in / 2) return SP_ERR_SHAPE;
    if (ctx->n_tokens <= 0) return SP_ERR_STATE;
    DeviceGuard guard(ctx->device);
    if (guard.error() != cudaSuccess) return cuda_fail(guard.error());
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    st = ensure_finalized(ctx, s);
    if (st != SP_OK) return st;
    return launch_select_24_compressed(ctx, W, dtype, n_rows, ldw, values_out, ldv, meta_out, s);
}

sp_status sp_apply_mask(const void *W, sp_dtype dtype, int64_t n_rows, int64_t n_cols, int64_t ldw,
                        const uint32_t *mask, void *W_out, int64_t ldo, sp_stream stream) {
    SP_CALL_RANGE();
    if (!valid_dtype(dtype)) return SP_ERR_DTYPE;
    if (n_rows < 0 || n_cols < 0) return SP_ERR_INVALID_ARG;
    if ((W == nullptr || mask == nullptr || W_out == nullptr) && n_rows * n_cols != 0)
        return SP_ERR_INVALID_ARG;
    if (ldw < n_cols || ldo < n_cols) return SP_ERR_SHAPE;
    if (W_out == W && ldo != ldw) return SP_ERR_SHAPE;
    return launch_apply_mask(W, dtype, n_rows, n_cols, ldw, mask, W_out, ldo,
                             static_cast<cudaStream_t>(stream));
}

sp_status sp_calib_accumulate_host(sp_ctx *ctx, const void *X_host, sp_dtype dtype,
                                   int64_t n_tokens, int64_t ldx, sp_stream stream) {
    SP_CALL_RANGE();
    if (ctx == nullptr) return SP_ERR_INVALID_ARG;
    if (!valid_dtype(dtype)) return SP_ERR_DTYPE;
    if (n_tokens < 0) return SP_ERR_INVALID_ARG;
    if (n_tokens == 0) return SP_OK;
    if (X_host == nullptr) return SP_ERR_INVALID_ARG;
    if (ldx < ctx->d_in) return SP_ERR_SHAPE;
    DeviceGuard guard(ctx->device);
    if (guard.error() != cudaSuccess) return cuda_fail(guard.error());
    return host_calib_accumulate(ctx, X_host, dtype, n_tokens, ldx, static_cast<cudaStream_t>(stream));
}

sp_status sp_select_nm_host(sp_ctx *ctx, const void *W_host, sp_dtype dtype, int64_t n_rows,
                            int64_t ldw, int N, int M, uint32_t *mask_host, void *W_out_host,
                            int64_t ldo, sp_stream stream) {
    SP_CALL_RANGE();
    sp_status st = check_matrix_args(ctx, W_host, dtype, n_rows, ldw, W_out_host, ldo);
    if (st != SP_OK) return st;
    if (M != 4 && M != 8) return SP_ERR_INVALID_ARG;
    if (N <= 0 || N >= M) return SP_ERR_INVALID_ARG;
    if (ctx->d_in % M != 0) return SP_ERR_SHAPE;
    if (ctx->n_tokens <= 0) return SP_ERR_STATE;
    DeviceGuard guard(ctx->device);
    if (guard.error() != cudaSuccess) return cuda_fail(guard.error());
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    st = ensure_finalized(ctx, s);
    if (st != SP_OK) return st;
    return host_select(ctx, 0, W_host, dtype, n_rows, ldw, N, M, nullptr, mask_host, W_out_host, ldo, s);
}

sp_status sp_select_unstructured_host(sp_ctx *ctx, const void *W_host, sp_dtype dtype,
                                      int64_t n_rows, int64_t ldw, float sparsity,
                                      uint32_t *mask_host, void *W_out_host, int64_t ldo,
                                      sp_stream stream) {
    SP_CALL_RANGE();
    sp_status st = check_matrix_args(ctx, W_host, dtype, n_rows, ldw, W_out_host, ldo);
    if (st != SP_OK) return st;
    sp_ewma_params p;
    p.alpha = 0.125f;
    p.beta = 0.125f;
    p.s_update = SP_S_GATED;
    st = sp_la_for_sparsity(sparsity, &p.la);
    if (st != SP_OK) return st;
    if (ctx->n_tokens <= 0) return SP_ERR_STATE;
    DeviceGuard guard(ctx->device);
    if (guard.error() != cudaSuccess) return cuda_fail(guard.error());
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    st = ensure_finalized(ctx, s);
    if (st != SP_OK) return st;
    return host_select(ctx, 1, W_host, dtype, n_rows, ldw, 0, 0, &p, mask_host, W_out_host, ldo, s);
}

sp_status sp_debug_status(int *violations, int *first_code, int64_t *first_index,
                          int64_t *first_limit, int clear) {
    if (violations == nullptr) return SP_ERR_INVALID_ARG;
    *violations = -1;
    if (first_code != nullptr) *first_code = 0;
    if (first_index != nullptr) *first_index = 0;
    if (first_limit != nullptr) *first_limit = 0;
    if (g_debug_reader_count == 0) return SP_OK;  // release build: no checks compiled in
    cudaError_t e = cudaDeviceSynchronize();
    if (e != cudaSuccess) return cuda_fail(e);
    unsigned int total = 0;
    for (int i = 0; i < g_debug_reader_count; ++i) {
        DebugRecord r = {};
        e = g_debug_readers[i](&r, clear != 0);
        if (e != cudaSuccess) return cuda_fail(e);
        if (r.count != 0u && total == 0u) {
            if (first_code != nullptr) *first_code = r.code;
            if (first_index != nullptr) *first_index = r.index;
            if (first_limit != nullptr) *first_limit = r.limit;
        }
        total += r.count;
    }
    *violations = static_cast<int>(total);
    return SP_OK;
}

const char *sp_status_string(sp_status status) {
    switch (status) {
        case SP_OK: return "ok";
        case SP_ERR_INVALID_ARG: return "invalid argument";
        case SP_ERR_SHAPE: return "invalid shape or leading dimension";
        case SP_ERR_DTYPE: return "unsupported dtype";
        case SP_ERR_STATE: return "no calibration statistics accumulated";
        case SP_ERR_DEGENERATE: return "degenerate calibration statistics (S is zero or not finite)";
        case SP_ERR_CUDA: return "CUDA runtime error";
        case SP_ERR_NOMEM: return "out of memory";
    }
    return "unknown status";
}

const char *sp_last_cuda_error(void) { return g_cuda_error; }

uint64_t sp_launch_count(void) { return g_launches.load(); }

}  // extern "C"
