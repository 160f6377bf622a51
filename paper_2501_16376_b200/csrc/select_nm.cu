// N:M selection (Section 3.3) fused with score, mask emission and write-back.
//
// One lane owns 8 consecutive weights of a row (one 16-byte load), i.e. two groups of four or
// one group of eight; a group never straddles lanes, so the selection needs no cross-lane
// traffic.  Scores are L = (w*w)*c_q in binary32 (Eq. 8).  Within a group an element's rank
// is the number of elements that order before it (smaller score, or equal score and lower
// column); the M-N lowest ranks are pruned.  Scores are non-negative, so they are compared
// through their bit patterns as unsigned integers, which also puts NaN above every number.
// Each warp processes kNmTilesPerWarp tiles with all loads issued first.
#include "sp_device.cuh"
#include "sp_internal.h"

namespace sp {

constexpr int kNmThreads = 256;
constexpr int kNmWarps = kNmThreads / 32;
constexpr int kNmTilesPerWarp = 4;

// keep bits (bit e = element e of the group is kept) of one group of M scores.
template <int M>
__device__ __forceinline__ uint32_t nm_keep_bits(const uint32_t *key, int prune_count) {
    int rank[M];
#pragma unroll
    for (int i = 0; i < M; ++i) rank[i] = 0;
#pragma unroll
    for (int i = 0; i < M; ++i) {
#pragma unroll
        for (int j = i + 1; j < M; ++j) {
            const int gt = key[i] > key[j] ? 1 : 0;  // j orders before i
            rank[i] += gt;
            rank[j] += 1 - gt;                        // i orders before j (ties: lower column)
        }
    }
    uint32_t keep = 0;
#pragma unroll
    for (int i = 0; i < M; ++i) keep |= (rank[i] >= prune_count ? 1u : 0u) << i;
    return keep;
}

template <bool BF16, bool VEC, int M>
__global__ void __launch_bounds__(kNmThreads)
select_nm_kernel(const uint16_t *__restrict__ W, int64_t ldw, int64_t n, int tiles_per_row,
                 int64_t total_tiles, const float *__restrict__ factor, int prune_count,
                 uint32_t *__restrict__ mask, int64_t mask_words, uint16_t *__restrict__ W_out,
                 int64_t ldo) {
    const int lane = threadIdx.x & 31;
    const int64_t first_tile =
        (static_cast<int64_t>(blockIdx.x) * kNmWarps + (threadIdx.x >> 5)) * kNmTilesPerWarp;

    uint32_t p[kNmTilesPerWarp][4];
    int64_t row[kNmTilesPerWarp], col[kNmTilesPerWarp];
#pragma unroll
    for (int u = 0; u < kNmTilesPerWarp; ++u) {
        const int64_t tile = first_tile + u;
        row[u] = tile / tiles_per_row;
        col[u] = (tile - row[u] * tiles_per_row) * kTile + lane * 8;
        if (tile < total_tiles) {
            load8<VEC, true>(W + row[u] * ldw, col[u], n, p[u]);
        } else {
            p[u][0] = p[u][1] = p[u][2] = p[u][3] = 0u;
        }
    }
#pragma unroll
    for (int u = 0; u < kNmTilesPerWarp; ++u) {
        if (first_tile + u >= total_tiles) break;  // warp-uniform
        uint32_t keep8 = 0;
        if (col[u] < n) {
            float w[8], c[8];
            unpack8<BF16>(p[u], w);
            load_factor8(factor, col[u], c);
            uint32_t key[8];
#pragma unroll
            for (int j = 0; j < 8; ++j)
                key[j] = __float_as_uint(__fmul_rn(__fmul_rn(w[j], w[j]), c[j]));
            if constexpr (M == 4) {
                keep8 = nm_keep_bits<4>(key, prune_count) | (nm_keep_bits<4>(key + 4, prune_count) << 4);
            } else {
                keep8 = nm_keep_bits<8>(key, prune_count);
            }
            const int64_t left = n - col[u];
            if (left < 8) keep8 &= (1u << left) - 1u;
            if (W_out != nullptr) {
                zero_pruned(p[u], keep8);
                store8<VEC>(W_out + row[u] * ldo, col[u], n, p[u]);
            }
        }
        const uint32_t word = gather_mask_word(keep8, lane);
        if (mask != nullptr && (lane & 3) == 0 && col[u] < n)
            mask[row[u] * mask_words + (col[u] >> 5)] = word;
    }
}

sp_status launch_select_nm(const sp_ctx *ctx, const void *W, sp_dtype dtype, int64_t n_rows,
                           int64_t ldw, int N, int M, uint32_t *mask, void *W_out, int64_t ldo,
                           cudaStream_t stream) {
    const int64_t n = ctx->d_in;
    const int tiles_per_row = static_cast<int>((n + kTile - 1) / kTile);
    const int64_t total_tiles = n_rows * tiles_per_row;
    if (total_tiles == 0) return SP_OK;
    const int64_t tiles_per_block = static_cast<int64_t>(kNmWarps) * kNmTilesPerWarp;
    const int64_t blocks = (total_tiles + tiles_per_block - 1) / tiles_per_block;
    if (blocks > 0x7fffffffLL) return SP_ERR_SHAPE;
    const bool vec = aligned16(W) && ldw % 8 == 0 && n % 8 == 0 &&
                     (W_out == nullptr || (aligned16(W_out) && ldo % 8 == 0));
    const uint16_t *Wp = static_cast<const uint16_t *>(W);
    uint16_t *Op = static_cast<uint16_t *>(W_out);
    const int64_t words = (n + 31) / 32;
    const int prune_count = M - N;
    const unsigned grid = static_cast<unsigned>(blocks);
#define SP_LAUNCH(B, V, MM)                                                                  \
    select_nm_kernel<B, V, MM><<<grid, kNmThreads, 0, stream>>>(                              \
        Wp, ldw, n, tiles_per_row, total_tiles, ctx->factor, prune_count, mask, words, Op, ldo)
#define SP_LAUNCH_M(B, V)                                                                     \
    do {                                                                                      \
        if (M == 4) SP_LAUNCH(B, V, 4); else SP_LAUNCH(B, V, 8);                              \
    } while (0)
    if (dtype == SP_BF16) {
        if (vec) SP_LAUNCH_M(true, true); else SP_LAUNCH_M(true, false);
    } else {
        if (vec) SP_LAUNCH_M(false, true); else SP_LAUNCH_M(false, false);
    }
#undef SP_LAUNCH_M
#undef SP_LAUNCH
    return check_launch();
}

}  // namespace sp
