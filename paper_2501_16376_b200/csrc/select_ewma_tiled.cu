// Algorithm 1 exactly as printed (including "S = S - w_i^2" when a weight is pruned), one
// thread per row, binary32 with one rounding per operation - the same arithmetic, in the same
// order, as ewma_literal_kernel, so the result is bit-identical to it - but with the rows of a
// warp moved together: a warp owns 32 rows and walks them in tiles of 32 rows x 32 columns
// (64 bytes per row).  A tile comes in by asynchronous 16-byte copies, four lanes per row so
// that global accesses are whole 64-byte runs, into an eight-slot ring in shared memory
// (seven tiles ahead of the walk); lane r then reads row r of the tile in 16-byte chunks
// (XOR-swizzled: the eight lanes of a quarter warp hit eight different bank groups), writes
// the pruned chunks back in place, and the tile goes out with the mapping it came in with.
// Every lane is at the same column at the same time, so the per-channel factors are uniform
// loads.  The walk is one dependent chain per row (about 25 instructions per weight, each
// waiting for the one before it): with a few thousand rows there is at most one warp per
// scheduler to run, so the kernel is bound by instruction latency, not by memory.
#include <type_traits>

#include "sp_device.cuh"
#include "sp_internal.h"

namespace sp {

constexpr int kTiledStages = 8;  // ring slots (a power of two)
constexpr int kTiledCols = 32;   // columns per tile

template <bool BF16>
__global__ void __launch_bounds__(32)
ewma_literal_tiled_kernel(const uint16_t *__restrict__ W, int64_t ldw, int n_rows, int n,
                          const double *__restrict__ colsq, const float *__restrict__ factor,
                          const DeviceScalars *__restrict__ scalars, float alpha, float beta,
                          float la, uint32_t *__restrict__ mask, int mask_words,
                          uint16_t *__restrict__ W_out, int64_t ldo,
                          unsigned long long *__restrict__ counters) {
    const int lane = threadIdx.x;
    const int row_base = blockIdx.x * 32;
    const int tiles = (n + kTiledCols - 1) / kTiledCols;

    // copy mapping: instruction i moves rows 8i + (lane >> 2), 16-byte chunk (lane & 3)
    const int crow = lane >> 2, cchunk = lane & 3;
    const int rows_left = n_rows - row_base - crow;  // row 8i + crow exists iff 8i < rows_left
    const uint16_t *src = W + static_cast<int64_t>(row_base + crow) * ldw + cchunk * 8;
    uint16_t *dst = W_out != nullptr ? W_out + static_cast<int64_t>(row_base + crow) * ldo + cchunk * 8
                                     : nullptr;
    const int coff = crow * 4 + (cchunk ^ ((crow >> 1) & 3));  // uint4 index inside a tile
    // walk mapping: lane r reads row r; chunk k sits at r * 4 + (k ^ swz)
    const int swz = (lane >> 1) & 3;
    const bool row_ok = row_base + lane < n_rows;
    uint32_t *mrow = mask != nullptr && row_ok
                         ? mask + static_cast<int64_t>(row_base + lane) * mask_words
                         : nullptr;

    __shared__ __align__(16) uint4 ring[kTiledStages][32 * 4];
    auto issue_tile = [&](int t) {
        // d_in % 8 == 0: a 16-byte chunk is inside the row or outside as a whole
        if (t < tiles && t * kTiledCols + cchunk * 8 < n) {
            uint4 *slot = ring[t & (kTiledStages - 1)];
#pragma unroll
            for (int i = 0; i < 4; ++i)
                if (8 * i < rows_left)
                    cp_async16(slot + 32 * i + coff, src + static_cast<int64_t>(8 * i) * ldw + t * kTiledCols, 16);
        }
        cp_async_commit();
    };
#pragma unroll
    for (int t = 0; t < kTiledStages - 1; ++t) issue_tile(t);

    const float one_minus_alpha = __fsub_rn(1.0f, alpha);
    const float one_minus_beta = __fsub_rn(1.0f, beta);
    const float S0 = scalars->S32;
    float S = S0;
    float est = 0.0f, dev = 0.0f;
    uint32_t kept = 0;

    for (int tile = 0; tile < tiles; ++tile) {
        cp_async_wait<kTiledStages - 2>();
        // every lane's copies of this tile have landed, and every lane is done with the
        // previous tile, whose slot is refilled next
        __syncwarp();
        issue_tile(tile + kTiledStages - 1);
        uint4 *slot = ring[tile & (kTiledStages - 1)];
        uint4 *mine = slot + lane * 4;
        uint32_t word = 0;
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const int i0 = tile * kTiledCols + 8 * k;
            if (i0 >= n) break;  // warp-uniform
            uint4 v = mine[k ^ swz];
            uint32_t p[4] = {v.x, v.y, v.z, v.w};
            float w[8];
            unpack8<BF16>(p, w);
            const float4 c0 = __ldg(reinterpret_cast<const float4 *>(factor + i0));
            const float4 c1 = __ldg(reinterpret_cast<const float4 *>(factor + i0) + 1);
            const float cf[8] = {c0.x, c0.y, c0.z, c0.w, c1.x, c1.y, c1.z, c1.w};
            // The 8 elements of the chunk, in order.  FOLLOW_S: recompute the factor of an
            // element from the current S once a pruned weight has changed it (a lane whose S
            // still has its initial value keeps the finalised factor, which is the same three
            // operations on the same operands).
            uint32_t keep8;
            auto walk = [&](auto follow_s) {
                keep8 = 0;
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    float c = cf[j];
                    if (decltype(follow_s)::value) {
                        if (S != S0) {
                            const float u = __fdiv_rn(static_cast<float>(colsq[i0 + j]), S);
                            c = __fdiv_rn(0.5f, __fsub_rn(1.0f, u));
                        }
                    }
                    const float w2 = __fmul_rn(w[j], w[j]);
                    const float L = __fmul_rn(w2, c);
                    if (k == 0 && j == 0 && tile == 0) est = L;
                    const float thr = __fsub_rn(est, __fmul_rn(la, dev));
                    const bool prune = L < thr;
                    S = prune ? __fsub_rn(S, w2) : S;
                    keep8 |= prune ? 0u : 1u << j;
                    est = __fadd_rn(__fmul_rn(one_minus_alpha, est), __fmul_rn(alpha, L));
                    dev = __fadd_rn(__fmul_rn(one_minus_beta, dev),
                                    __fmul_rn(beta, fabsf(__fsub_rn(est, L))));
                }
            };
            // Usual case: no lane's S has moved, and none moves inside the chunk - the chunk is
            // straight-line code with the finalised factors.  Otherwise the chunk is walked
            // (again) from the state it started in, following S element by element.
            const float est_in = est, dev_in = dev, S_in = S;
            bool follow = __any_sync(kFullWarp, S_in != S0);
            if (!follow) {
                walk(std::false_type{});
                follow = __any_sync(kFullWarp, S != S_in);
            }
            if (follow) {
                est = est_in;
                dev = dev_in;
                S = S_in;
                walk(std::true_type{});
            }
            word |= keep8 << (8 * k);
            if (dst != nullptr) {
                zero_pruned(p, keep8);
                mine[k ^ swz] = make_uint4(p[0], p[1], p[2], p[3]);
            }
        }
        if (row_ok) kept += __popc(word);
        if (mrow != nullptr) mrow[tile] = word;
        if (dst != nullptr) {
            __syncwarp();  // the pruned tile is complete in shared memory
            if (tile * kTiledCols + cchunk * 8 < n) {
#pragma unroll
                for (int i = 0; i < 4; ++i)
                    if (8 * i < rows_left)
                        __stcs(reinterpret_cast<uint4 *>(dst + static_cast<int64_t>(8 * i) * ldo + tile * kTiledCols),
                               slot[32 * i + coff]);
            }
        }
    }
    if (counters != nullptr) {
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) kept += __shfl_xor_sync(kFullWarp, kept, off);
        if (lane == 0) atomicAdd(counters + SP_COUNTER_KEPT, static_cast<unsigned long long>(kept));
    }
}

sp_status launch_ewma_literal_tiled(const sp_ctx *ctx, const void *W, sp_dtype dtype,
                                    int64_t n_rows, int64_t ldw, const sp_ewma_params &p,
                                    uint32_t *mask, void *W_out, int64_t ldo,
                                    unsigned long long *counters, cudaStream_t stream) {
    const int64_t n = ctx->d_in;
    const int64_t blocks = (n_rows + 31) / 32;
    if (blocks > 0x7fffffffLL || n_rows > 0x7fffffffLL) return SP_ERR_SHAPE;
    const uint16_t *Wp = static_cast<const uint16_t *>(W);
    uint16_t *Op = static_cast<uint16_t *>(W_out);
    const int words = static_cast<int>((n + 31) / 32);
    const unsigned grid = static_cast<unsigned>(blocks);
    if (dtype == SP_BF16)
        ewma_literal_tiled_kernel<true><<<grid, 32, 0, stream>>>(
            Wp, ldw, static_cast<int>(n_rows), static_cast<int>(n), ctx->colsq, ctx->factor,
            ctx->scalars, p.alpha, p.beta, p.la, mask, words, Op, ldo, counters);
    else
        ewma_literal_tiled_kernel<false><<<grid, 32, 0, stream>>>(
            Wp, ldw, static_cast<int>(n_rows), static_cast<int>(n), ctx->colsq, ctx->factor,
            ctx->scalars, p.alpha, p.beta, p.la, mask, words, Op, ldo, counters);
    return check_launch();
}

}  // namespace sp
