// EWMA running-threshold selection (Algorithm 1; state rules of Table 2) fused with score,
// mask emission and write-back.
//
// Frozen-S path (scan kernel).  With S fixed, est and dev do not depend on the prune
// decisions: est_i = a est_{i-1} + alpha L_i and dev_i = b dev_{i-1} + beta |est_i - L_i|
// (a = 1-alpha, b = 1-beta) are first-order linear recurrences, evaluated as affine scans.
// One warp owns one row and walks it in tiles of 256 weights; a lane owns 8 consecutive
// weights.  Per tile: the lane runs both recurrences over its 8 elements from a zero state,
// a 5-step shuffle scan with the constant multipliers a^(8*2^k) combines the lane totals, and
// the state entering the lane (the scan's exclusive prefix plus a^(8*lane) times the state
// carried in from the previous tile) is folded back into the 8 local values.  Element i is
// tested against the state before its own update, est_{i-1} - la*dev_{i-1}; est_{-1} = L_0 and
// dev_{-1} = 0 (Table 2), so column 0 is never pruned.  The next tile's weights are loaded
// before the current tile is processed; only the two carried scalars serialise the tiles.
//
// Literal-S path (sequential kernel).  Algorithm 1's "S = S - w_i^2" makes L_i depend on
// earlier decisions, so the row is evaluated in order by one thread, every operation in
// binary32 with one rounding each.  It is a correctness path, not a fast one.
#include <math.h>

#include "sp_device.cuh"
#include "sp_internal.h"

namespace sp {

constexpr int kEwmaThreads = 256;
constexpr int kEwmaWarps = kEwmaThreads / 32;

template <bool BF16>
__device__ __forceinline__ uint32_t packed_abs_max(uint32_t acc, uint32_t v) {
    if constexpr (BF16) {
        __nv_bfloat162 a = *reinterpret_cast<__nv_bfloat162 *>(&acc);
        __nv_bfloat162 b = __habs2(*reinterpret_cast<__nv_bfloat162 *>(&v));
        __nv_bfloat162 m = __hmax2(a, b);
        return *reinterpret_cast<uint32_t *>(&m);
    } else {
        __half2 a = *reinterpret_cast<__half2 *>(&acc);
        __half2 b = __habs2(*reinterpret_cast<__half2 *>(&v));
        __half2 m = __hmax2(a, b);
        return *reinterpret_cast<uint32_t *>(&m);
    }
}

// Inclusive scan over lanes of x with the recurrence multiplier step[k] = m^(8*2^k).
__device__ __forceinline__ float lane_affine_scan(float x, const float (&step)[5], int lane) {
#pragma unroll
    for (int k = 0; k < 5; ++k) {
        const float y = __shfl_up_sync(kFullWarp, x, 1 << k);
        if (lane >= (1 << k)) x = fmaf(step[k], y, x);
    }
    return x;
}

template <bool BF16, bool VEC>
__global__ void __launch_bounds__(kEwmaThreads)
ewma_scan_kernel(const uint16_t *__restrict__ W, int64_t ldw, int64_t n_rows, int64_t n,
                 const float *__restrict__ factor, const DeviceScalars *__restrict__ scalars,
                 const __grid_constant__ ScanConstants sc, uint32_t *__restrict__ mask,
                 int64_t mask_words, uint16_t *__restrict__ W_out, int64_t ldo,
                 unsigned long long *__restrict__ counters) {
    const int lane = threadIdx.x & 31;
    const int64_t row = static_cast<int64_t>(blockIdx.x) * kEwmaWarps + (threadIdx.x >> 5);
    if (row >= n_rows) return;  // warp-uniform
    const uint16_t *wrow = W + row * ldw;
    uint16_t *orow = W_out != nullptr ? W_out + row * ldo : nullptr;
    uint32_t *mrow = mask != nullptr ? mask + row * mask_words : nullptr;

    const float alpha = sc.alpha, beta = sc.beta, neg_la = -sc.la, a = sc.a, b = sc.b;
    const float a_lane = sc.a_lane[lane], b_lane = sc.b_lane[lane];
    float a_step[5], b_step[5];
#pragma unroll
    for (int k = 0; k < 5; ++k) { a_step[k] = sc.a_step[k]; b_step[k] = sc.b_step[k]; }

    const int tiles = static_cast<int>((n + kTile - 1) / kTile);
    float carry_e = 0.0f, carry_d = 0.0f;
    uint32_t kept = 0;
    uint32_t wmax = 0;  // packed running max of |w| over this lane's elements

    uint32_t p_next[4];
    load8<VEC, true>(wrow, lane * 8, n, p_next);

    for (int tile = 0; tile < tiles; ++tile) {
        const int64_t col = static_cast<int64_t>(tile) * kTile + lane * 8;
        uint32_t p[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) p[k] = p_next[k];
        if (tile + 1 < tiles) load8<VEC, true>(wrow, col + kTile, n, p_next);

        float w[8], c[8], L[8];
        unpack8<BF16>(p, w);
        load_factor8(factor, col, c);  // zero past d_in: scores of padding are 0
#pragma unroll
        for (int k = 0; k < 4; ++k) wmax = packed_abs_max<BF16>(wmax, p[k]);
#pragma unroll
        for (int j = 0; j < 8; ++j) L[j] = __fmul_rn(__fmul_rn(w[j], w[j]), c[j]);

        if (tile == 0) carry_e = __shfl_sync(kFullWarp, L[0], 0);  // est starts at L_0

        // est: local recurrence from zero, lane scan, fold the incoming state back in
        float e[8];
        e[0] = alpha * L[0];
#pragma unroll
        for (int j = 1; j < 8; ++j) e[j] = fmaf(a, e[j - 1], alpha * L[j]);
        float incl = lane_affine_scan(e[7], a_step, lane);
        float excl = __shfl_up_sync(kFullWarp, incl, 1);
        if (lane == 0) excl = 0.0f;
        const float est_in = fmaf(a_lane, carry_e, excl);
#pragma unroll
        for (int j = 0; j < 8; ++j) e[j] = fmaf(sc.a_pow[j], est_in, e[j]);

        // dev: same with the inputs beta * |est_i - L_i|
        float d[8];
        d[0] = beta * fabsf(e[0] - L[0]);
#pragma unroll
        for (int j = 1; j < 8; ++j) d[j] = fmaf(b, d[j - 1], beta * fabsf(e[j] - L[j]));
        incl = lane_affine_scan(d[7], b_step, lane);
        excl = __shfl_up_sync(kFullWarp, incl, 1);
        if (lane == 0) excl = 0.0f;
        const float dev_in = fmaf(b_lane, carry_d, excl);
#pragma unroll
        for (int j = 0; j < 8; ++j) d[j] = fmaf(sc.b_pow[j], dev_in, d[j]);

        // decisions against the state before each element's update: element j is pruned iff
        // L_j - (est_{j-1} - la*dev_{j-1}) is negative.  The difference of two floats has the
        // exact sign (it is never rounded to zero, equal operands give +0, a NaN result is the
        // positive canonical NaN), so the prune flag is its sign bit; a byte permute with sign
        // replication turns two of them into the half-word mask of a packed pair.
        float diff[8];
        diff[0] = L[0] - fmaf(neg_la, dev_in, est_in);
#pragma unroll
        for (int j = 1; j < 8; ++j) diff[j] = L[j] - fmaf(neg_la, d[j - 1], e[j - 1]);
        uint32_t pm[4];
#pragma unroll
        for (int k = 0; k < 4; ++k)
            pm[k] = prmt(__float_as_uint(diff[2 * k]), __float_as_uint(diff[2 * k + 1]), 0xffbbu);
        uint32_t keep8 = ~halfmasks_to_bits(pm) & 0xffu;
        const int64_t left = n - col;
        if (left < 8) keep8 &= left > 0 ? ((1u << left) - 1u) : 0u;
        kept += __popc(keep8);

        carry_e = __shfl_sync(kFullWarp, e[7], 31);
        carry_d = __shfl_sync(kFullWarp, d[7], 31);

        if (orow != nullptr) {
#pragma unroll
            for (int k = 0; k < 4; ++k) p[k] &= ~pm[k];
            store8<VEC>(orow, col, n, p);
        }
        const uint32_t word = gather_mask_word(keep8, lane);
        if (mrow != nullptr && (lane & 3) == 0 && col < n) mrow[col >> 5] = word;
    }

    if (counters != nullptr) {
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) kept += __shfl_xor_sync(kFullWarp, kept, off);
        float2 m = unpack2<BF16>(wmax);
        float mx = fmaxf(m.x, m.y);
#pragma unroll
        for (int off = 16; off > 0; off >>= 1)
            mx = fmaxf(mx, __shfl_xor_sync(kFullWarp, mx, off));
        if (lane == 0) {
            atomicAdd(counters + SP_COUNTER_KEPT, static_cast<unsigned long long>(kept));
            if (!(mx * mx < scalars->hazard_w2)) atomicAdd(counters + SP_COUNTER_S_HAZARD, 1ULL);
        }
    }
}

// Algorithm 1 exactly as printed, one thread per row, binary32 with one rounding per operation.
template <bool BF16>
__global__ void __launch_bounds__(128)
ewma_literal_kernel(const uint16_t *__restrict__ W, int64_t ldw, int64_t n_rows, int64_t n,
                    const double *__restrict__ colsq, const DeviceScalars *__restrict__ scalars,
                    float alpha, float beta, float la, uint32_t *__restrict__ mask,
                    int64_t mask_words, uint16_t *__restrict__ W_out, int64_t ldo,
                    unsigned long long *__restrict__ counters) {
    const int64_t row = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (row >= n_rows) return;
    const uint16_t *wrow = W + row * ldw;
    const float one_minus_alpha = __fsub_rn(1.0f, alpha);
    const float one_minus_beta = __fsub_rn(1.0f, beta);
    float S = scalars->S32;
    float est = 0.0f, dev = 0.0f;
    uint32_t word = 0;
    unsigned long long kept = 0;
    for (int64_t i = 0; i < n; ++i) {
        uint16_t bits = wrow[i];
        const float w = BF16 ? __uint_as_float(static_cast<uint32_t>(bits) << 16)
                             : __half2float(__ushort_as_half(bits));
        const float x2 = static_cast<float>(colsq[i]);
        const float u = __fdiv_rn(x2, S);
        const float den = __fsub_rn(1.0f, u);
        const float c = __fdiv_rn(0.5f, den);
        const float w2 = __fmul_rn(w, w);
        const float L = __fmul_rn(w2, c);
        if (i == 0) est = L;
        const float thr = __fsub_rn(est, __fmul_rn(la, dev));
        if (L < thr) {
            S = __fsub_rn(S, w2);
            bits = 0;
        } else {
            word |= 1u << (i & 31);
            ++kept;
        }
        est = __fadd_rn(__fmul_rn(one_minus_alpha, est), __fmul_rn(alpha, L));
        dev = __fadd_rn(__fmul_rn(one_minus_beta, dev), __fmul_rn(beta, fabsf(__fsub_rn(est, L))));
        if (W_out != nullptr) W_out[row * ldo + i] = bits;
        if ((i & 31) == 31 || i == n - 1) {
            if (mask != nullptr) mask[row * mask_words + (i >> 5)] = word;
            word = 0;
        }
    }
    if (counters != nullptr) atomicAdd(counters + SP_COUNTER_KEPT, kept);
}

static void fill_scan_constants(const sp_ewma_params &p, ScanConstants &sc) {
    sc.alpha = p.alpha;
    sc.beta = p.beta;
    sc.la = p.la;
    sc.a = 1.0f - p.alpha;
    sc.b = 1.0f - p.beta;
    const double a = static_cast<double>(sc.a), b = static_cast<double>(sc.b);
    for (int j = 0; j < 8; ++j) {
        sc.a_pow[j] = static_cast<float>(pow(a, j + 1));
        sc.b_pow[j] = static_cast<float>(pow(b, j + 1));
    }
    for (int l = 0; l < 32; ++l) {
        sc.a_lane[l] = static_cast<float>(pow(a, 8.0 * l));
        sc.b_lane[l] = static_cast<float>(pow(b, 8.0 * l));
    }
    for (int k = 0; k < 5; ++k) {
        sc.a_step[k] = static_cast<float>(pow(a, 8.0 * (1 << k)));
        sc.b_step[k] = static_cast<float>(pow(b, 8.0 * (1 << k)));
    }
}

sp_status launch_select_ewma(const sp_ctx *ctx, const void *W, sp_dtype dtype, int64_t n_rows,
                             int64_t ldw, const sp_ewma_params &p, uint32_t *mask, void *W_out,
                             int64_t ldo, unsigned long long *counters, cudaStream_t stream) {
    const int64_t n = ctx->d_in;
    if (n_rows == 0) return SP_OK;
    const uint16_t *Wp = static_cast<const uint16_t *>(W);
    uint16_t *Op = static_cast<uint16_t *>(W_out);
    const int64_t words = (n + 31) / 32;
    const bool bf16 = dtype == SP_BF16;

    if (p.s_update == SP_S_LITERAL_W2) {
        const int64_t blocks = (n_rows + 127) / 128;
        if (blocks > 0x7fffffffLL) return SP_ERR_SHAPE;
        if (bf16)
            ewma_literal_kernel<true><<<static_cast<unsigned>(blocks), 128, 0, stream>>>(
                Wp, ldw, n_rows, n, ctx->colsq, ctx->scalars, p.alpha, p.beta, p.la, mask, words,
                Op, ldo, counters);
        else
            ewma_literal_kernel<false><<<static_cast<unsigned>(blocks), 128, 0, stream>>>(
                Wp, ldw, n_rows, n, ctx->colsq, ctx->scalars, p.alpha, p.beta, p.la, mask, words,
                Op, ldo, counters);
        return check_launch();
    }

    ScanConstants sc;
    fill_scan_constants(p, sc);
    const int64_t blocks = (n_rows + kEwmaWarps - 1) / kEwmaWarps;
    if (blocks > 0x7fffffffLL) return SP_ERR_SHAPE;
    const bool vec = aligned16(W) && ldw % 8 == 0 && n % 8 == 0 &&
                     (W_out == nullptr || (aligned16(W_out) && ldo % 8 == 0));
    const unsigned grid = static_cast<unsigned>(blocks);
#define SP_LAUNCH(B, V)                                                                      \
    ewma_scan_kernel<B, V><<<grid, kEwmaThreads, 0, stream>>>(                               \
        Wp, ldw, n_rows, n, ctx->factor, ctx->scalars, sc, mask, words, Op, ldo, counters)
    if (bf16) {
        if (vec) SP_LAUNCH(true, true); else SP_LAUNCH(true, false);
    } else {
        if (vec) SP_LAUNCH(false, true); else SP_LAUNCH(false, false);
    }
#undef SP_LAUNCH
    return check_launch();
}

}  // namespace sp
