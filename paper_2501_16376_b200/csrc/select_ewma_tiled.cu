// Algorithm 1 exactly as printed (including "S = S - w_i^2" when a weight is pruned), one
// thread per row, binary32 with one rounding per operation - the same arithmetic, in the same
// order, as ewma_literal_kernel, so the result is bit-identical to it - but with the rows moved
// in tiles: a CTA owns 32 rows and walks them in tiles of 32 rows x 32 columns (64 bytes per
// row).  A tile comes in by asynchronous 16-byte copies, four threads per row so that global
// accesses are whole 64-byte runs, into an eight-slot ring in shared memory (seven tiles ahead
// of the walk); the thread that walks row r reads it in 16-byte chunks (XOR-swizzled: the eight
// walkers of a warp hit eight different bank groups), writes the pruned chunks back in place,
// and the tile goes out with the mapping it came in with.  All walkers are at the same column
// at the same time, so the per-channel factors are uniform loads.
//
// The walk is one dependent chain per row (about 25 instructions per weight), and a layer has
// only 10^3..10^4 rows: the kernel is bound by instruction latency, not by memory.  The number
// of lanes of a warp that walk rows is a build option (kTiledWalkers: with 8 or 16 the same rows
// make more warps for each scheduler to interleave, at the price of idle lanes); measured, 32 is
// the best choice on the layer shapes of the benchmarks.
#include <type_traits>

#include "sp_device.cuh"
#include "sp_internal.h"

namespace sp {

constexpr int kTiledStages = 8;  // ring slots (a power of two)
constexpr int kTiledCols = 32;   // columns per tile
#ifndef SP_TILED_WALKERS
#define SP_TILED_WALKERS 32
#endif
constexpr int kTiledWalkers = SP_TILED_WALKERS;            // rows walked by one warp
constexpr int kTiledThreads = 32 * (32 / kTiledWalkers);   // threads of the CTA (32 rows)
constexpr int kTiledCopies = 128 / kTiledThreads;          // 16-byte copies per thread and tile
constexpr unsigned kWalkerMask = kTiledWalkers == 32 ? 0xffffffffu : (1u << kTiledWalkers) - 1u;
static_assert(kTiledWalkers == 8 || kTiledWalkers == 16 || kTiledWalkers == 32, "walkers per warp");

template <bool BF16>
__global__ void __launch_bounds__(kTiledThreads)
ewma_literal_tiled_kernel(const uint16_t *__restrict__ W, int64_t ldw, int n_rows, int n,
                          const double *__restrict__ colsq, const float *__restrict__ factor,
                          const DeviceScalars *__restrict__ scalars, float alpha, float beta,
                          float la, uint32_t *__restrict__ mask, int mask_words,
                          uint16_t *__restrict__ W_out, int64_t ldo,
                          unsigned long long *__restrict__ counters, int subtract_x2) {
    const int tid = threadIdx.x;
    const int lane = tid & 31;
    const int row_base = blockIdx.x * 32;
    const int tiles = (n + kTiledCols - 1) / kTiledCols;

    // copy mapping: copy c of thread tid moves the 16-byte chunk (idx & 3) of row (idx >> 2),
    // idx = c * kTiledThreads + tid; its place in a tile is row * 4 + (chunk ^ ((row >> 1) & 3))
    const int cchunk = tid & 3;  // kTiledThreads is a multiple of 4: the same for every copy
    // walk mapping: lanes below kTiledWalkers walk row  warp * kTiledWalkers + lane
    const bool walker = lane < kTiledWalkers;
    const int wrow = (tid >> 5) * kTiledWalkers + (walker ? lane : 0);
    const int swz = (wrow >> 1) & 3;
    const bool row_ok = walker && row_base + wrow < n_rows;
    uint32_t *mrow = mask != nullptr && row_ok
                         ? mask + static_cast<int64_t>(row_base + wrow) * mask_words
                         : nullptr;

    __shared__ __align__(16) uint4 ring[kTiledStages][32 * 4];
    auto issue_tile = [&](int t) {
        // d_in % 8 == 0: a 16-byte chunk is inside the row or outside as a whole
        if (t < tiles && t * kTiledCols + cchunk * 8 < n) {
            uint4 *slot = ring[t & (kTiledStages - 1)];
#pragma unroll
            for (int c = 0; c < kTiledCopies; ++c) {
                const int r = (c * kTiledThreads + tid) >> 2;
                if (row_base + r < n_rows)
                    cp_async16(slot + r * 4 + (cchunk ^ ((r >> 1) & 3)),
                               W + static_cast<int64_t>(row_base + r) * ldw + t * kTiledCols + cchunk * 8, 16);
            }
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

    float4 c0_next = __ldg(reinterpret_cast<const float4 *>(factor));
    float4 c1_next = __ldg(reinterpret_cast<const float4 *>(factor) + 1);
    for (int tile = 0; tile < tiles; ++tile) {
        cp_async_wait<kTiledStages - 2>();
        // every thread's copies of this tile have landed, and every thread is done with the
        // previous tile, whose slot is refilled next
        __syncthreads();
        issue_tile(tile + kTiledStages - 1);
        uint4 *slot = ring[tile & (kTiledStages - 1)];
        if (walker) {
            uint4 *mine = slot + wrow * 4;
            uint32_t word = 0;
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const int i0 = tile * kTiledCols + 8 * k;
                if (i0 >= n) break;  // uniform
                uint4 v = mine[k ^ swz];
                uint32_t p[4] = {v.x, v.y, v.z, v.w};
                float w[8];
                unpack8<BF16>(p, w);
                // the factors of this chunk were requested one chunk ago; those of the next one
                // are requested now (the factor array is padded with a tile of zeros)
                const float4 c0 = c0_next, c1 = c1_next;
                c0_next = __ldg(reinterpret_cast<const float4 *>(factor + i0 + 8));
                c1_next = __ldg(reinterpret_cast<const float4 *>(factor + i0 + 8) + 1);
                const float cf[8] = {c0.x, c0.y, c0.z, c0.w, c1.x, c1.y, c1.z, c1.w};
                // The 8 elements of the chunk, in order.  FOLLOW_S: recompute the factor of an
                // element from the current S once a pruned weight has changed it (a row whose S
                // still has its initial value keeps the finalised factor, which is the same
                // three operations on the same operands).
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
                        float dec = w2;
                        if (decltype(follow_s)::value) {  // the x_i^2 reading always walks this way
                            if (subtract_x2) dec = static_cast<float>(colsq[i0 + j]);
                        }
                        S = prune ? __fsub_rn(S, dec) : S;
                        keep8 |= prune ? 0u : 1u << j;
                        est = __fadd_rn(__fmul_rn(one_minus_alpha, est), __fmul_rn(alpha, L));
                        dev = __fadd_rn(__fmul_rn(one_minus_beta, dev),
                                        __fmul_rn(beta, fabsf(__fsub_rn(est, L))));
                    }
                };
                // Usual case: no walker's S has moved, and none moves inside the chunk - the
                // chunk is straight-line code with the finalised factors.  Otherwise the chunk
                // is walked (again) from the state it started in, following S element by element.
                const float est_in = est, dev_in = dev, S_in = S;
                bool follow = subtract_x2 != 0 || __any_sync(kWalkerMask, S_in != S0);
                if (!follow) {
                    walk(std::false_type{});
                    follow = __any_sync(kWalkerMask, S != S_in);
                }
                if (follow) {
                    est = est_in;
                    dev = dev_in;
                    S = S_in;
                    walk(std::true_type{});
                }
                word |= keep8 << (8 * k);
                if (W_out != nullptr) {
                    zero_pruned(p, keep8);
                    mine[k ^ swz] = make_uint4(p[0], p[1], p[2], p[3]);
                }
            }
            if (row_ok) kept += __popc(word);
            if (mrow != nullptr) mrow[tile] = word;
        }
        if (W_out != nullptr) {
            __syncthreads();  // the pruned tile is complete in shared memory
            if (tile * kTiledCols + cchunk * 8 < n) {
#pragma unroll
                for (int c = 0; c < kTiledCopies; ++c) {
                    const int r = (c * kTiledThreads + tid) >> 2;
                    if (row_base + r < n_rows)
                        __stcs(reinterpret_cast<uint4 *>(W_out + static_cast<int64_t>(row_base + r) * ldo +
                                                         tile * kTiledCols + cchunk * 8),
                               slot[r * 4 + (cchunk ^ ((r >> 1) & 3))]);
                }
            }
        }
    }
    if (counters != nullptr) {
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) kept += __shfl_xor_sync(kFullWarp, kept, off);
        if (lane == 0 && kept != 0)
            atomicAdd(counters + SP_COUNTER_KEPT, static_cast<unsigned long long>(kept));
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
        ewma_literal_tiled_kernel<true><<<grid, kTiledThreads, 0, stream>>>(
            Wp, ldw, static_cast<int>(n_rows), static_cast<int>(n), ctx->colsq, ctx->factor,
            ctx->scalars, p.alpha, p.beta, p.la, mask, words, Op, ldo, counters,
            p.s_update == SP_S_READING_X2 ? 1 : 0);
    else
        ewma_literal_tiled_kernel<false><<<grid, kTiledThreads, 0, stream>>>(
            Wp, ldw, static_cast<int>(n_rows), static_cast<int>(n), ctx->colsq, ctx->factor,
            ctx->scalars, p.alpha, p.beta, p.la, mask, words, Op, ldo, counters,
            p.s_update == SP_S_READING_X2 ? 1 : 0);
    return check_launch();
}

}  // namespace sp
