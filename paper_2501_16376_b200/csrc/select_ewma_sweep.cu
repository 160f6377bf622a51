// Algorithm 1 with its printed update "S = S - w_i^2" (Table 2, row S) evaluated in parallel
// along a row: fix-point sweeps over tiles (SP_S_LITERAL_SCAN).
//
// Once pruned weights change S, the score of element i depends on the decisions before it
// through S_i = S - (sum of the w_j^2 pruned before i), so the row is one causal chain.  A causal
// system has exactly one self-consistent assignment of decisions, and iterating "decide with the
// S_i that the previous decisions imply" reaches it: each sweep settles at least the next
// undecided element, in practice a whole tile within a few sweeps unless S is comparable to the
// pruned sum itself.  One warp owns one row and walks it in tiles of 256 weights (8 per lane):
//   sweep: S_i = S_0 - (pruned before the tile + exclusive prefix inside the tile, from the
//          previous sweep's decisions; zero in the first sweep) -> scores with the factor
//          0.5/(1 - x_i^2/S_i) -> the two recurrences as affine lane scans (as in
//          ewma_scan_kernel) -> decisions -> equal to the previous sweep's? then the tile is done;
//          else prefix-sum the pruned w^2 over the tile (lane-local + one lane scan) and repeat.
// A tile whose pruned sum cannot change S in binary32 is done after its first sweep (always, at
// calibration scale).  A tile that has not settled after kSweepLimit sweeps hands the rest of
// the row to the sequential walk (literal_walk) from the tile's first column, with the state and
// the S the row has there; such rows are counted in SP_COUNTER_S_HAZARD.
//
// Against the sequential kernels the arithmetic is re-associated (scans; S_i from a prefix sum
// instead of successive subtractions), so decisions agree with
// the oracle's literal mode under the tolerance band, not bit for bit.  What it buys: rows are
// scanned by whole warps, so a matrix with few, long rows (4096 x 14336: 4096 sequential chains
// for the thread-per-row kernel) no longer starves the GPU.
#include <math.h>

#include "ewma_common.cuh"

namespace sp {

constexpr int kSweepThreads = 256;
constexpr int kSweepWarps = kSweepThreads / 32;
constexpr int kSweepTile = 256;
constexpr int kSweepLimit = 8;

struct SweepConstants {
    float alpha, beta, la;
    float a, b;
    float a_lane[32], b_lane[32];  // a^(8 lane), b^(8 lane)
    float a_step[5], b_step[5];    // a^(8 2^k), b^(8 2^k)
};

__device__ __forceinline__ float lane_affine_scan8(float x, const float (&step)[5], int lane) {
#pragma unroll
    for (int k = 0; k < 5; ++k) {
        const float y = __shfl_up_sync(kFullWarp, x, 1 << k);
        if (lane >= (1 << k)) x = fmaf(step[k], y, x);
    }
    return x;
}

template <bool BF16, bool VEC>
__global__ void __launch_bounds__(kSweepThreads)
ewma_sweep_kernel(const uint16_t *__restrict__ W, int64_t ldw, int n_rows, int n,
                  const double *__restrict__ colsq, const float *__restrict__ factor,
                  const DeviceScalars *__restrict__ scalars,
                  const __grid_constant__ SweepConstants sc, uint32_t *__restrict__ mask,
                  int mask_words, uint16_t *__restrict__ W_out, int64_t ldo,
                  unsigned long long *__restrict__ counters) {
    pdl_launch_dependents();
    pdl_wait();
    const int lane = threadIdx.x & 31;
    const int row = blockIdx.x * kSweepWarps + (threadIdx.x >> 5);
    if (row >= n_rows) return;  // warp-uniform
    const uint16_t *wrow = W + static_cast<int64_t>(row) * ldw;
    uint16_t *orow = W_out != nullptr ? W_out + static_cast<int64_t>(row) * ldo : nullptr;
    uint32_t *mrow = mask != nullptr ? mask + static_cast<int64_t>(row) * mask_words : nullptr;

    const float alpha = sc.alpha, neg_alpha = -sc.alpha, a = sc.a, b = sc.b;
    const float la_beta = sc.la * sc.beta;
    const float a_lane = sc.a_lane[lane], b_lane = sc.b_lane[lane];
    const float S0 = scalars->S32;
    const int tiles = (n + kSweepTile - 1) / kSweepTile;
    float carry_E = 0.0f, carry_D = 0.0f;
    float P_in = 0.0f;  // w^2 pruned before the tile
    uint32_t kept = 0;
    unsigned long long walked = 0;

    for (int tile = 0; tile < tiles; ++tile) {
        const int col = tile * kSweepTile + lane * 8;
        uint32_t p[4];
        load8<VEC, true>(wrow, col, n, p);
        float w[8], w2[8], x32[8];
        unpack8<BF16>(p, w);
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            w2[j] = __fmul_rn(w[j], w[j]);
            x32[j] = col + j < n ? static_cast<float>(__ldg(colsq + col + j)) : 0.0f;
        }
        const float S_in = __fsub_rn(S0, P_in);

        float pre[8];  // pruned w^2 inside the tile before element j (previous sweep's decisions)
#pragma unroll
        for (int j = 0; j < 8; ++j) pre[j] = 0.0f;
        uint32_t prev8 = 0xffffffffu, prune8 = 0;
        float E_end = 0.0f, D_end = 0.0f, tile_pruned = 0.0f;
        bool settled = false;
        for (int sweep = 0; sweep < kSweepLimit && !settled; ++sweep) {
            float L[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const float S_i = __fsub_rn(S0, __fadd_rn(P_in, pre[j]));
                const float u = __fdiv_rn(x32[j], S_i);  // the factor of Eq. 8 at the current S
                L[j] = __fmul_rn(w2[j], __fdiv_rn(0.5f, __fsub_rn(1.0f, u)));
            }
            float cE = carry_E;
            if (tile == 0) cE = __shfl_sync(kFullWarp, L[0], 0) / alpha;  // est starts at L_0
            // E over the lane's elements from a zero state -> lane total -> scan
            float acc = L[0];
#pragma unroll
            for (int j = 1; j < 8; ++j) acc = fmaf(a, acc, L[j]);
            float incl = lane_affine_scan8(acc, sc.a_step, lane);
            float excl = __shfl_up_sync(kFullWarp, incl, 1);
            if (lane == 0) excl = 0.0f;
            const float E_in = fmaf(a_lane, cE, excl);
            float q[8], dabs[8];
            float E_run = E_in, D_loc = 0.0f;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                q[j] = fmaf(neg_alpha, E_run, L[j]);
                E_run = fmaf(a, E_run, L[j]);
                dabs[j] = fabsf(fmaf(alpha, E_run, -L[j]));
                D_loc = fmaf(b, D_loc, dabs[j]);
            }
            incl = lane_affine_scan8(D_loc, sc.b_step, lane);
            excl = __shfl_up_sync(kFullWarp, incl, 1);
            if (lane == 0) excl = 0.0f;
            float D_run = fmaf(b_lane, carry_D, excl);
            prune8 = 0;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                // the sign bit of L_i - est_{i-1} + la dev_{i-1} is the prune flag (NaN: kept)
                const float diff = fmaf(la_beta, D_run, q[j]);
                prune8 |= (__float_as_uint(diff) >> 31) << j;
                D_run = fmaf(b, D_run, dabs[j]);
            }
            if (tile == 0 && lane == 0) prune8 &= ~1u;  // column 0 is kept by definition
            const int left = n - col;
            if (left < 8) prune8 &= left > 0 ? ((1u << left) - 1u) : 0u;
            E_end = __shfl_sync(kFullWarp, E_run, 31);
            D_end = __shfl_sync(kFullWarp, D_run, 31);

            settled = sweep > 0 && __all_sync(kFullWarp, prune8 == prev8);
            if (!settled) {
                // pruned w^2 under these decisions: exclusive prefix inside the tile, and total
                float loc[8];
                float run = 0.0f;
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    loc[j] = run;
                    run = __fadd_rn(run, (prune8 >> j) & 1u ? w2[j] : 0.0f);
                }
                float sum = run;
#pragma unroll
                for (int k = 0; k < 5; ++k) {
                    const float y = __shfl_up_sync(kFullWarp, sum, 1 << k);
                    if (lane >= (1 << k)) sum = __fadd_rn(sum, y);
                }
                const float before = __fsub_rn(sum, run);  // lanes below
                tile_pruned = __shfl_sync(kFullWarp, sum, 31);
#pragma unroll
                for (int j = 0; j < 8; ++j) pre[j] = __fadd_rn(before, loc[j]);
                prev8 = prune8;
                // if the whole tile's pruned sum cannot move S, nothing can change in a next sweep
                if (sweep == 0 && __fsub_rn(S0, __fadd_rn(P_in, tile_pruned)) == S_in) settled = true;
            }
        }
        if (!settled) {
            // hand the rest of the row to the sequential walk, from this tile's first column
            if (lane == 0) {
                if (counters != nullptr) atomicAdd(counters + SP_COUNTER_S_HAZARD, 1ULL);
                float est = __fmul_rn(alpha, carry_E), dev = __fmul_rn(sc.beta, carry_D);
                walked = literal_walk<BF16>(wrow, orow, mrow, n, tile * kSweepTile, est, dev, colsq,
                                            factor, S0, sc.alpha, sc.beta, sc.la, false, S_in);
            }
            break;
        }
        carry_E = E_end;
        carry_D = D_end;
        P_in = __fadd_rn(P_in, tile_pruned);

        const int left = n - col;
        uint32_t keep8 = ~prune8 & 0xffu;
        if (left < 8) keep8 &= left > 0 ? ((1u << left) - 1u) : 0u;
        kept += __popc(keep8);
        if (orow != nullptr) {
            zero_pruned(p, keep8);
            store8<VEC>(orow, col, n, p);
        }
        const uint32_t word = gather_mask_word(keep8, lane);  // four lanes share a mask word
        if (mrow != nullptr && (lane & 3) == 0 && col < n) mrow[col >> 5] = word;
    }

    if (counters != nullptr) {
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) kept += __shfl_xor_sync(kFullWarp, kept, off);
        if (lane == 0 && kept + walked != 0ULL)
            atomicAdd(counters + SP_COUNTER_KEPT, static_cast<unsigned long long>(kept) + walked);
    }
}

sp_status launch_ewma_sweep(const sp_ctx *ctx, const void *W, sp_dtype dtype, int64_t n_rows,
                            int64_t ldw, const sp_ewma_params &p, uint32_t *mask, void *W_out,
                            int64_t ldo, unsigned long long *counters, cudaStream_t stream) {
    const int64_t n = ctx->d_in;
    if (n_rows == 0) return SP_OK;
    if (n_rows > 0x7fffffffLL) return SP_ERR_SHAPE;
    SweepConstants sc;
    sc.alpha = p.alpha;
    sc.beta = p.beta;
    sc.la = p.la;
    sc.a = 1.0f - p.alpha;
    sc.b = 1.0f - p.beta;
    const double a = static_cast<double>(sc.a), b = static_cast<double>(sc.b);
    for (int l = 0; l < 32; ++l) {
        sc.a_lane[l] = static_cast<float>(pow(a, 8.0 * l));
        sc.b_lane[l] = static_cast<float>(pow(b, 8.0 * l));
    }
    for (int k = 0; k < 5; ++k) {
        sc.a_step[k] = static_cast<float>(pow(a, 8.0 * (1 << k)));
        sc.b_step[k] = static_cast<float>(pow(b, 8.0 * (1 << k)));
    }
    const bool vec = aligned16(W) && ldw % 8 == 0 && n % 8 == 0 &&
                     (W_out == nullptr || (aligned16(W_out) && ldo % 8 == 0));
    PdlConfig pdl(dim3(static_cast<unsigned>((n_rows + kSweepWarps - 1) / kSweepWarps)),
                  dim3(kSweepThreads), stream);
    const uint16_t *Wp = static_cast<const uint16_t *>(W);
    uint16_t *Op = static_cast<uint16_t *>(W_out);
    const double *colsq = ctx->colsq;
    const float *factor = ctx->factor;
    const DeviceScalars *scalars = ctx->scalars;
    const int words = static_cast<int>((n + 31) / 32);
    const int rows = static_cast<int>(n_rows), nn = static_cast<int>(n);
    cudaError_t e;
#define SP_LAUNCH(B, V)                                                                        \
    e = cudaLaunchKernelEx(&pdl.cfg, ewma_sweep_kernel<B, V>, Wp, ldw, rows, nn, colsq, factor, \
                           scalars, sc, mask, words, Op, ldo, counters)
    if (dtype == SP_BF16) {
        if (vec) SP_LAUNCH(true, true); else SP_LAUNCH(true, false);
    } else {
        if (vec) SP_LAUNCH(false, true); else SP_LAUNCH(false, false);
    }
#undef SP_LAUNCH
    if (e != cudaSuccess) return cuda_fail(e);
    return check_launch();
}

}  // namespace sp
