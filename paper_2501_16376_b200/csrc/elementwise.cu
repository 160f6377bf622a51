// Materialised scores (Eq. 8 with S at its initial value) and the stand-alone write-back
// W_out = W (.) mask (Algorithm 1, "w_i = 0" / "c_i = w_i").  Both are plain streaming
// kernels: one warp per 256-element tile of a row, 16 bytes of weights per lane.
#include "sp_device.cuh"
#include "sp_internal.h"

namespace sp {

constexpr int kEwThreads = 256;
constexpr int kEwWarps = kEwThreads / 32;

template <bool BF16, bool VEC>
__global__ void __launch_bounds__(kEwThreads)
score_kernel(const uint16_t *__restrict__ W, int64_t ldw, int64_t n_rows, int64_t n,
             int tiles_per_row, int64_t total_tiles, const float *__restrict__ factor,
             float *__restrict__ scores) {
    const int lane = threadIdx.x & 31;
    const int64_t tile = static_cast<int64_t>(blockIdx.x) * kEwWarps + (threadIdx.x >> 5);
    if (tile >= total_tiles) return;
    const int64_t row = tile / tiles_per_row;
    const int64_t col = (tile - row * tiles_per_row) * kTile + lane * 8;
    if (col >= n) return;
    uint32_t p[4];
    load8<VEC, true>(W + row * ldw, col, n, p);
    float w[8], c[8];
    unpack8<BF16>(p, w);
    load_factor8(factor, col, c);
    float *dst = scores + row * n + col;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        if (col + j < n) dst[j] = __fmul_rn(__fmul_rn(w[j], w[j]), c[j]);
    }
}

template <bool VEC>
__global__ void __launch_bounds__(kEwThreads)
apply_mask_kernel(const uint16_t *__restrict__ W, int64_t ldw, int64_t n_rows, int64_t n,
                  int tiles_per_row, int64_t total_tiles, const uint32_t *__restrict__ mask,
                  int64_t mask_words, uint16_t *__restrict__ W_out, int64_t ldo) {
    const int lane = threadIdx.x & 31;
    const int64_t tile = static_cast<int64_t>(blockIdx.x) * kEwWarps + (threadIdx.x >> 5);
    if (tile >= total_tiles) return;
    const int64_t row = tile / tiles_per_row;
    const int64_t col = (tile - row * tiles_per_row) * kTile + lane * 8;
    if (col >= n) return;
    uint32_t p[4];
    load8<VEC, true>(W + row * ldw, col, n, p);
    const uint32_t word = __ldg(mask + row * mask_words + (col >> 5));
    const uint32_t keep8 = (word >> (col & 31)) & 0xffu;
    zero_pruned(p, keep8);
    store8<VEC>(W_out + row * ldo, col, n, p);
}

sp_status launch_score(const sp_ctx *ctx, const void *W, sp_dtype dtype, int64_t n_rows,
                       int64_t ldw, float *scores, cudaStream_t stream) {
    const int64_t n = ctx->d_in;
    const int tiles_per_row = static_cast<int>((n + kTile - 1) / kTile);
    const int64_t total_tiles = n_rows * tiles_per_row;
    if (total_tiles == 0) return SP_OK;
    const int64_t blocks = (total_tiles + kEwWarps - 1) / kEwWarps;
    if (blocks > 0x7fffffffLL) return SP_ERR_SHAPE;
    const bool vec = aligned16(W) && ldw % 8 == 0 && n % 8 == 0;
    const uint16_t *Wp = static_cast<const uint16_t *>(W);
#define SP_LAUNCH(B, V)                                                                 \
    score_kernel<B, V><<<static_cast<unsigned>(blocks), kEwThreads, 0, stream>>>(       \
        Wp, ldw, n_rows, n, tiles_per_row, total_tiles, ctx->factor, scores)
    if (dtype == SP_BF16) {
        if (vec) SP_LAUNCH(true, true); else SP_LAUNCH(true, false);
    } else {
        if (vec) SP_LAUNCH(false, true); else SP_LAUNCH(false, false);
    }
#undef SP_LAUNCH
    return check_launch();
}

sp_status launch_apply_mask(const void *W, sp_dtype dtype, int64_t n_rows, int64_t n_cols,
                            int64_t ldw, const uint32_t *mask, void *W_out, int64_t ldo,
                            cudaStream_t stream) {
    (void)dtype;  // a bit-level select: the two 16-bit types are handled alike
    const int64_t n = n_cols;
    const int tiles_per_row = static_cast<int>((n + kTile - 1) / kTile);
    const int64_t total_tiles = n_rows * tiles_per_row;
    if (total_tiles == 0) return SP_OK;
    const int64_t blocks = (total_tiles + kEwWarps - 1) / kEwWarps;
    if (blocks > 0x7fffffffLL) return SP_ERR_SHAPE;
    const bool vec = aligned16(W) && aligned16(W_out) && ldw % 8 == 0 && ldo % 8 == 0 && n % 8 == 0;
    const uint16_t *Wp = static_cast<const uint16_t *>(W);
    uint16_t *Op = static_cast<uint16_t *>(W_out);
    const int64_t words = (n + 31) / 32;
    if (vec)
        apply_mask_kernel<true><<<static_cast<unsigned>(blocks), kEwThreads, 0, stream>>>(
            Wp, ldw, n_rows, n, tiles_per_row, total_tiles, mask, words, Op, ldo);
    else
        apply_mask_kernel<false><<<static_cast<unsigned>(blocks), kEwThreads, 0, stream>>>(
            Wp, ldw, n_rows, n, tiles_per_row, total_tiles, mask, words, Op, ldo);
    return check_launch();
}

}  // namespace sp
