// Internal declarations shared by the translation units of the library.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "sp_debug.cuh"
#include "swiftprune.h"

namespace sp {

constexpr int kStripChannels = 256;  // channels covered by one warp-wide 16-byte load
constexpr int kMaxSlabs = 128;       // token slabs that own a row of partial sums
constexpr int kTile = 256;           // weights per warp tile (32 lanes x 8)
constexpr int64_t kMaxDin = 1 << 20;

// Status word written by the finalisation kernel.
constexpr int kFlagDegenerate = 1;

constexpr int64_t kEwmaMaxLaunchRows = int64_t(1) << 30;  // rows one EWMA launch can cover
constexpr int kEwmaMaxJobs = 16;                           // weight matrices, likewise

// Scalars produced by finalisation; lives in device memory inside the context.
struct DeviceScalars {
    double S;             // sum_q colsq[q]
    float S32;            // (float)S
    float hazard_w2;      // a weight with w^2 >= this could change S in "S - w^2" (binary32)
    int flags;            // kFlag*
    unsigned int ticket;  // arrival counter of the finalisation kernel (returns to 0)
    unsigned long long search_counters[SP_NUM_COUNTERS];  // scratch of sp_search_la
    // state of sp_search_la's bisection when it runs on the device
    float search_la, search_lo, search_hi, search_best_la;
    double search_best_gap, search_best_frac;
};

// Powers of a = 1-alpha and b = 1-beta that the scan kernel needs (a lane owns P consecutive
// weights), computed on the host in fp64 and rounded once.
struct ScanConstants {
    float alpha, beta, la;
    float a, b;            // 1-alpha, 1-beta (rounded in fp32 like the definition)
    float a_lane[32];      // a^(P*lane)
    float b_lane[32];
    float a_step[5];       // a^(P*2^k)
    float b_step[5];
};

struct HostPipe;  // staging slots and streams of the host-buffer entry points (host_pipe.cu)

}  // namespace sp

struct sp_ctx {
    int device;
    int sm_count;
    int64_t d_in;
    int64_t n_pad;             // d_in rounded up to a multiple of kStripChannels
    int strips;                // n_pad / kStripChannels
    int64_t n_tokens;          // host-side count
    int slabs_valid;           // slab rows of `partial` that hold data
    bool dirty;                // batches arrived since the last finalisation
    int calib_blocks_per_sm;   // measured occupancy of the accumulation kernel
    double *partial;           // [kMaxSlabs][n_pad] fp64 partial column sums
    double *colsq;             // [n_pad]
    double *strip_sum;         // [strips]
    float *factor;             // [n_pad + 256] c_q, zero in the padding
    float *factor_pairs;       // the same values in the layout of the EWMA pair kernel (calib.cu)
    sp::DeviceScalars *scalars;
    sp::HostPipe *host_pipe;   // created by the first host-buffer call
};

namespace sp {

// Thread-local CUDA error text and the global launch counter (api.cu).
sp_status cuda_fail(cudaError_t e);
void count_launch(int n = 1);
inline sp_status check_launch() {
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(e);
    count_launch();
    return SP_OK;
}

// calib.cu
int calib_query_blocks_per_sm();
sp_status launch_calib_accumulate(sp_ctx *ctx, const void *X, sp_dtype dtype, int64_t n_tokens,
                                  int64_t ldx, cudaStream_t stream, bool x_complete = false);
sp_status launch_finalize(sp_ctx *ctx, cudaStream_t stream);
sp_status launch_finalize_pending(sp_ctx *const *ctxs, int count, cudaStream_t stream);
// One batch for each of several contexts (all different) in one launch; every item must satisfy
// calib_multi_applies (16-byte access).
struct CalibItem {
    const void *X;
    int64_t n_tokens, ldx;
};
bool calib_multi_applies(const sp_ctx *ctx, const void *X, int64_t ldx, int64_t n_tokens);
sp_status launch_calib_accumulate_multi(sp_ctx *const *ctxs, const CalibItem *items, int count,
                                        sp_dtype dtype, cudaStream_t stream, bool x_complete);
int64_t calib_static_max_d_in();
sp_status launch_calib_stats_static(int device, const void *X, sp_dtype dtype, int64_t n_tokens,
                                    int64_t d_in, int64_t ldx, double *colsq_out,
                                    float *factor_out, double *S_out, cudaStream_t stream);

// elementwise.cu
sp_status launch_score(const sp_ctx *ctx, const void *W, sp_dtype dtype, int64_t n_rows,
                       int64_t ldw, float *scores, cudaStream_t stream);
sp_status launch_apply_mask(const void *W, sp_dtype dtype, int64_t n_rows, int64_t n_cols,
                            int64_t ldw, const uint32_t *mask, void *W_out, int64_t ldo,
                            cudaStream_t stream);

// select_nm_compressed.cu
sp_status launch_select_24_compressed(const sp_ctx *ctx, const void *W, sp_dtype dtype,
                                      int64_t n_rows, int64_t ldw, void *values, int64_t ldv,
                                      uint32_t *meta, cudaStream_t stream);

// One weight matrix of a selection launch that covers several.
struct EwmaLaunchJob {
    const void *W;
    void *W_out;     // nullable
    uint32_t *mask;  // nullable
    int64_t n_rows, ldw, ldo;
    const sp_ctx *ctx = nullptr;  // statistics to prune it with; null: those of the call's context
};

// select_nm.cu: N:M selection of up to kEwmaMaxJobs matrices (each with the statistics of its
// own context, or of `ctx`), in as few launches as their layouts and requested outputs allow
sp_status launch_select_nm(const sp_ctx *ctx, const EwmaLaunchJob *jobs, int n_jobs, sp_dtype dtype,
                           int N, int M, cudaStream_t stream);
inline sp_status launch_select_nm(const sp_ctx *ctx, const void *W, sp_dtype dtype, int64_t n_rows,
                                  int64_t ldw, int N, int M, uint32_t *mask, void *W_out,
                                  int64_t ldo, cudaStream_t stream) {
    const EwmaLaunchJob job{W, W_out, mask, n_rows, ldw, ldo};
    return launch_select_nm(ctx, &job, 1, dtype, N, M, stream);
}

// select_ewma.cu
// Algorithm 1 on several matrices of one dtype (each with the statistics of its own context, or
// of `ctx`), in as few launches as their layouts allow.
sp_status launch_select_ewma(const sp_ctx *ctx, const EwmaLaunchJob *jobs, int n_jobs,
                             sp_dtype dtype, const sp_ewma_params &p, unsigned long long *counters,
                             cudaStream_t stream, bool la_from_device = false);
inline sp_status launch_select_ewma(const sp_ctx *ctx, const void *W, sp_dtype dtype, int64_t n_rows,
                                    int64_t ldw, const sp_ewma_params &p, uint32_t *mask,
                                    void *W_out, int64_t ldo, unsigned long long *counters,
                                    cudaStream_t stream, bool la_from_device = false) {
    const EwmaLaunchJob job{W, W_out, mask, n_rows, ldw, ldo};
    return launch_select_ewma(ctx, &job, 1, dtype, p, counters, stream, la_from_device);
}
// True when launch_select_ewma would take the kernel that can read la from DeviceScalars.
bool ewma_pair_path_applies(const void *W, int64_t ldw, int64_t n);
sp_status launch_search_la_device(sp_ctx *ctx, const void *W, sp_dtype dtype, int64_t n_rows,
                                  int64_t ldw, float target, float alpha, float beta,
                                  int iterations, float *la_out, double *achieved_out,
                                  cudaStream_t stream);

// select_ewma_sweep.cu
sp_status launch_ewma_sweep(const sp_ctx *ctx, const void *W, sp_dtype dtype, int64_t n_rows,
                            int64_t ldw, const sp_ewma_params &p, uint32_t *mask, void *W_out,
                            int64_t ldo, unsigned long long *counters, cudaStream_t stream);

// select_ewma_tiled.cu
sp_status launch_ewma_literal_tiled(const sp_ctx *ctx, const void *W, sp_dtype dtype,
                                    int64_t n_rows, int64_t ldw, const sp_ewma_params &p,
                                    uint32_t *mask, void *W_out, int64_t ldo,
                                    unsigned long long *counters, cudaStream_t stream);

// host_pipe.cu
void host_pipe_destroy(HostPipe *hp);
sp_status host_calib_accumulate(sp_ctx *ctx, const void *X_host, sp_dtype dtype, int64_t n_tokens,
                                int64_t ldx, cudaStream_t stream);
sp_status host_select(sp_ctx *ctx, int kind, const void *W_host, sp_dtype dtype, int64_t n_rows,
                      int64_t ldw, int N, int M, const sp_ewma_params *params,
                      uint32_t *mask_host, void *W_out_host, int64_t ldo, cudaStream_t stream);

// Launch configuration with programmatic dependent launch allowed: the kernel may be scheduled
// while the previous kernel of the stream drains; every kernel launched this way executes
// griddepcontrol.wait before it touches memory an earlier kernel may still be writing.
struct PdlConfig {
    cudaLaunchConfig_t cfg;
    cudaLaunchAttribute attr[1];
    PdlConfig(dim3 grid, dim3 block, cudaStream_t stream) : cfg{}, attr{} {
        cfg.gridDim = grid;
        cfg.blockDim = block;
        cfg.dynamicSmemBytes = 0;
        cfg.stream = stream;
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
    }
};

sp_status launch_ewma_trace(const sp_ctx *ctx, const void *W, sp_dtype dtype, int64_t n_rows,
                            int64_t ldw, const sp_ewma_params &p, float *est_out, float *dev_out,
                            float *score_out, cudaStream_t stream);

inline bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

}  // namespace sp
