// Host-buffer entry points: the same kernels fed from, and drained to, host memory.
//
// A matrix that lives in host memory is cut into row chunks; each chunk is copied to one of two
// device staging slots on a copy-in stream, processed on the caller's stream, and (for the
// selection calls) its results are copied back on a copy-out stream, so that the transfer of
// chunk k+1, the kernel on chunk k and the read-back of chunk k-1 overlap.  Events order the
// three streams; nothing blocks the host (with pinned host memory; pageable memory makes the
// copies themselves synchronous, as usual).  The staging slots and streams belong to the
// context and are created on the first host-buffer call.
#include <new>

#include "sp_internal.h"

namespace sp {

constexpr size_t kStageBytes = size_t(64) << 20;  // per slot: input rows; output rows

struct HostPipe {
    cudaStream_t s_in = nullptr, s_out = nullptr;
    cudaEvent_t ev_in[2] = {nullptr, nullptr};    // chunk arrived in slot
    cudaEvent_t ev_done[2] = {nullptr, nullptr};  // kernel finished with slot
    cudaEvent_t ev_out[2] = {nullptr, nullptr};   // slot's results are back on the host
    cudaEvent_t ev_fork = nullptr;
    void *d_in[2] = {nullptr, nullptr};
    void *d_out[2] = {nullptr, nullptr};
    uint32_t *d_mask[2] = {nullptr, nullptr};
    int next_slot = 0;
};

void host_pipe_destroy(HostPipe *hp) {
    if (hp == nullptr) return;
    for (int i = 0; i < 2; ++i) {
        if (hp->ev_in[i]) cudaEventDestroy(hp->ev_in[i]);
        if (hp->ev_done[i]) cudaEventDestroy(hp->ev_done[i]);
        if (hp->ev_out[i]) cudaEventDestroy(hp->ev_out[i]);
        cudaFree(hp->d_in[i]);
        cudaFree(hp->d_out[i]);
        cudaFree(hp->d_mask[i]);
    }
    if (hp->ev_fork) cudaEventDestroy(hp->ev_fork);
    if (hp->s_in) cudaStreamDestroy(hp->s_in);
    if (hp->s_out) cudaStreamDestroy(hp->s_out);
    delete hp;
}

static sp_status host_pipe_get(sp_ctx *ctx, HostPipe **out) {
    if (ctx->host_pipe != nullptr) {
        *out = ctx->host_pipe;
        return SP_OK;
    }
    HostPipe *hp = new (std::nothrow) HostPipe();
    if (hp == nullptr) return SP_ERR_NOMEM;
    cudaError_t e = cudaStreamCreateWithFlags(&hp->s_in, cudaStreamNonBlocking);
    if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&hp->s_out, cudaStreamNonBlocking);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&hp->ev_fork, cudaEventDisableTiming);
    for (int i = 0; i < 2 && e == cudaSuccess; ++i) {
        e = cudaEventCreateWithFlags(&hp->ev_in[i], cudaEventDisableTiming);
        if (e == cudaSuccess) e = cudaEventCreateWithFlags(&hp->ev_done[i], cudaEventDisableTiming);
        if (e == cudaSuccess) e = cudaEventCreateWithFlags(&hp->ev_out[i], cudaEventDisableTiming);
        if (e == cudaSuccess) e = cudaMalloc(&hp->d_in[i], kStageBytes);
        if (e == cudaSuccess) e = cudaMalloc(&hp->d_out[i], kStageBytes);
        // one mask bit per 16-bit weight: 1/16 of the weight bytes, plus row padding
        if (e == cudaSuccess)
            e = cudaMalloc(reinterpret_cast<void **>(&hp->d_mask[i]), kStageBytes / 8);
    }
    if (e != cudaSuccess) {
        host_pipe_destroy(hp);
        return cuda_fail(e);
    }
    ctx->host_pipe = hp;
    *out = hp;
    return SP_OK;
}

#define SP_CUDA(call)                                 \
    do {                                              \
        cudaError_t e__ = (call);                     \
        if (e__ != cudaSuccess) return cuda_fail(e__); \
    } while (0)

// Rows of `width` elements per chunk such that the chunk and its mask fit their staging slots.
static int64_t chunk_rows_for(int64_t width) {
    const int64_t by_data = static_cast<int64_t>(kStageBytes) / (width * 2);
    const int64_t by_mask = static_cast<int64_t>(kStageBytes / 8) / (((width + 31) / 32) * 4);
    const int64_t rows = by_data < by_mask ? by_data : by_mask;
    return rows < 1 ? 0 : rows;
}

sp_status host_calib_accumulate(sp_ctx *ctx, const void *X_host, sp_dtype dtype, int64_t n_tokens,
                                int64_t ldx, cudaStream_t stream) {
    HostPipe *hp = nullptr;
    sp_status st = host_pipe_get(ctx, &hp);
    if (st != SP_OK) return st;
    const int64_t n = ctx->d_in;
    const int64_t chunk = chunk_rows_for(n);
    if (chunk == 0) return SP_ERR_SHAPE;
    const char *src = static_cast<const char *>(X_host);
    // the copy-in stream starts after whatever the caller has queued so far
    SP_CUDA(cudaEventRecord(hp->ev_fork, stream));
    SP_CUDA(cudaStreamWaitEvent(hp->s_in, hp->ev_fork, 0));
    for (int64_t t0 = 0; t0 < n_tokens; t0 += chunk) {
        const int64_t rows = n_tokens - t0 < chunk ? n_tokens - t0 : chunk;
        const int slot = hp->next_slot;
        hp->next_slot ^= 1;
        SP_CUDA(cudaStreamWaitEvent(hp->s_in, hp->ev_done[slot], 0));  // slot free again
        SP_CUDA(cudaMemcpy2DAsync(hp->d_in[slot], n * 2, src + t0 * ldx * 2, ldx * 2, n * 2, rows,
                                  cudaMemcpyHostToDevice, hp->s_in));
        SP_CUDA(cudaEventRecord(hp->ev_in[slot], hp->s_in));
        SP_CUDA(cudaStreamWaitEvent(stream, hp->ev_in[slot], 0));
        st = launch_calib_accumulate(ctx, hp->d_in[slot], dtype, rows, n, stream);
        if (st != SP_OK) return st;
        SP_CUDA(cudaEventRecord(hp->ev_done[slot], stream));
    }
    return SP_OK;
}

// kind: 0 = N:M (a = N, b = M), 1 = EWMA with explicit parameters.
sp_status host_select(sp_ctx *ctx, int kind, const void *W_host, sp_dtype dtype, int64_t n_rows,
                      int64_t ldw, int N, int M, const sp_ewma_params *params,
                      uint32_t *mask_host, void *W_out_host, int64_t ldo, cudaStream_t stream) {
    HostPipe *hp = nullptr;
    sp_status st = host_pipe_get(ctx, &hp);
    if (st != SP_OK) return st;
    const int64_t n = ctx->d_in;
    const int64_t chunk = chunk_rows_for(n);
    if (chunk == 0) return SP_ERR_SHAPE;
    const int64_t words = (n + 31) / 32;
    const char *src = static_cast<const char *>(W_host);
    char *dst = static_cast<char *>(W_out_host);
    SP_CUDA(cudaEventRecord(hp->ev_fork, stream));
    SP_CUDA(cudaStreamWaitEvent(hp->s_in, hp->ev_fork, 0));
    int used[2] = {0, 0};
    for (int64_t r0 = 0; r0 < n_rows; r0 += chunk) {
        const int64_t rows = n_rows - r0 < chunk ? n_rows - r0 : chunk;
        const int slot = hp->next_slot;
        hp->next_slot ^= 1;
        used[slot] = 1;
        SP_CUDA(cudaStreamWaitEvent(hp->s_in, hp->ev_done[slot], 0));
        SP_CUDA(cudaMemcpy2DAsync(hp->d_in[slot], n * 2, src + r0 * ldw * 2, ldw * 2, n * 2, rows,
                                  cudaMemcpyHostToDevice, hp->s_in));
        SP_CUDA(cudaEventRecord(hp->ev_in[slot], hp->s_in));
        SP_CUDA(cudaStreamWaitEvent(stream, hp->ev_in[slot], 0));
        SP_CUDA(cudaStreamWaitEvent(stream, hp->ev_out[slot], 0));  // previous results drained
        uint32_t *dmask = mask_host != nullptr ? hp->d_mask[slot] : nullptr;
        void *dout = W_out_host != nullptr ? hp->d_out[slot] : nullptr;
        if (kind == 0)
            st = launch_select_nm(ctx, hp->d_in[slot], dtype, rows, n, N, M, dmask, dout, n, stream);
        else
            st = launch_select_ewma(ctx, hp->d_in[slot], dtype, rows, n, *params, dmask, dout, n,
                                    nullptr, stream);
        if (st != SP_OK) return st;
        SP_CUDA(cudaEventRecord(hp->ev_done[slot], stream));
        SP_CUDA(cudaStreamWaitEvent(hp->s_out, hp->ev_done[slot], 0));
        if (dout != nullptr)
            SP_CUDA(cudaMemcpy2DAsync(dst + r0 * ldo * 2, ldo * 2, dout, n * 2, n * 2, rows,
                                      cudaMemcpyDeviceToHost, hp->s_out));
        if (dmask != nullptr)
            SP_CUDA(cudaMemcpyAsync(mask_host + r0 * words, dmask, rows * words * 4,
                                    cudaMemcpyDeviceToHost, hp->s_out));
        SP_CUDA(cudaEventRecord(hp->ev_out[slot], hp->s_out));
    }
    // the caller's stream completes only when every result is on the host
    for (int slot = 0; slot < 2; ++slot)
        if (used[slot]) SP_CUDA(cudaStreamWaitEvent(stream, hp->ev_out[slot], 0));
    return SP_OK;
}

}  // namespace sp
