// EWMA running-threshold selection (Algorithm 1; state rules of Table 2) fused with score,
// mask emission and write-back.
//
// Frozen-S path (scan kernels).  With S fixed, est and dev do not depend on the prune
// decisions: est_i = a est_{i-1} + alpha L_i and dev_i = b dev_{i-1} + beta |est_i - L_i|
// (a = 1-alpha, b = 1-beta) are first-order linear recurrences, evaluated as affine scans.
// One warp owns one row and walks it in tiles of 256 weights; a lane owns 8 consecutive
// weights.  Per tile and recurrence: the lane runs the recurrence over its elements from a zero
// state to get its total, a 5-step shuffle scan with the constant multipliers a^(8*2^k)
// combines the lane totals, and the lane obtains its true states from the state entering it
// (the scan's exclusive prefix plus a^(8*lane) times the state carried in from the previous
// tile).  Element i is tested against the state before its own update,
// est_{i-1} - la*dev_{i-1}; est_{-1} = L_0 and dev_{-1} = 0 (Table 2), so column 0 is never
// pruned.  Two kernels: ewma_pair_scan_kernel for rows that allow 16-byte access (the fast
// path: packed binary32 pairs, weights streamed through a shared-memory ring of asynchronous
// copies) and ewma_scan_kernel for any other pointer, stride or width.
//
// Drift gate (SP_S_GATED).  "S = S - w_i^2" (Table 2, row S) changes S in binary32 only when a
// pruned weight has w_i^2 >= DeviceScalars::hazard_w2.  The scan kernels test every tile for
// such a weight before they store anything of it; at the first tile that may hold one, the warp
// notes the column and the state of Algorithm 1 before it and stops storing, and once its scan
// loop has ended one of its lanes takes the row up again at that column and walks it
// sequentially with the printed update (literal_walk).  Up to that column the frozen and the
// printed rule are the same rule, so the result is Algorithm 1 as printed; the input is never
// overwritten ahead of the sequential walk, so pruning in place works as well.  A row that is
// walked this way costs about as much as a thousand scanned ones: the gate is a safety net for
// stray rows, and SP_S_LITERAL_W2 the mode for statistics so small that every row needs it.
//
// Literal-S path (sequential kernels, here and in select_ewma_tiled.cu).  Algorithm 1's
// "S = S - w_i^2" makes L_i depend on earlier decisions, so the row is evaluated in order by one
// thread, every operation in binary32 with one rounding each.  It is the exact path, bound by
// the latency of one dependent chain per row.
#include <math.h>

#include "ewma_common.cuh"

namespace sp {

#ifndef SP_EWMA_MIN_BLOCKS
#define SP_EWMA_MIN_BLOCKS 4
#endif
constexpr int kEwmaThreads = 256;
constexpr int kEwmaWarps = kEwmaThreads / 32;
constexpr int kEwmaPerLane = 8;                   // consecutive weights per lane
constexpr int kEwmaTile = 32 * kEwmaPerLane;      // weights per warp tile
#ifndef SP_EWMA_PAIR_THREADS
#define SP_EWMA_PAIR_THREADS 128
#endif
#ifndef SP_EWMA_PAIR_MIN_BLOCKS
#define SP_EWMA_PAIR_MIN_BLOCKS 7
#endif
constexpr int kPairThreads = SP_EWMA_PAIR_THREADS;
constexpr int kPairWarps = kPairThreads / 32;
#ifndef SP_EWMA_STAGES
#define SP_EWMA_STAGES 4
#endif
constexpr int kEwmaStages = SP_EWMA_STAGES;       // ring slots per warp (a power of two)
static_assert((kEwmaStages & (kEwmaStages - 1)) == 0, "ring size must be a power of two");

// Inclusive scan over lanes of x with the recurrence multiplier step[k] = m^(P*2^k).
__device__ __forceinline__ float lane_affine_scan(float x, const float (&step)[5], int lane) {
#pragma unroll
    for (int k = 0; k < 5; ++k) {
        const float y = __shfl_up_sync(kFullWarp, x, 1 << k);
        if (lane >= (1 << k)) x = fmaf(step[k], y, x);
    }
    return x;
}

// The matrices of one launch, each with the statistics it is pruned with (matrices that read
// different layer inputs can share a launch).  A job owns a whole number of CTAs, so the job of a
// CTA - and with it the row length and every pointer - is the same for all its warps.
struct EwmaJob {
    const uint16_t *W;
    uint16_t *W_out;  // nullable
    uint32_t *mask;   // nullable
    const float *factor_pairs;
    const DeviceScalars *scalars;
    const double *colsq;
    const float *factor;
    int ldw, ldo, n_rows;
    int n, mask_words;
    int first_cta;
};
struct EwmaJobTable {
    int count;
    int total_ctas;
    EwmaJob job[kEwmaMaxJobs];
};

// Drift gate: the rest of a row, from column `col` on, for a scan kernel that had to leave it
// (est, dev: the state of Algorithm 1 before that column).  Rarely taken, kept out of line.
template <bool BF16>
__device__ __noinline__ unsigned long long gate_walk(
    const uint16_t *wrow, uint16_t *orow, uint32_t *mrow, int n, int col, float est, float dev,
    const double *colsq, const float *factor, const DeviceScalars *scalars, float alpha, float beta,
    float la, unsigned long long *counters) {
    if (counters != nullptr) atomicAdd(counters + SP_COUNTER_S_HAZARD, 1ULL);
    return literal_walk<BF16>(wrow, orow, mrow, n, col, est, dev, colsq, factor, scalars->S32,
                              alpha, beta, la);
}

// The kernel carries the two states in scaled form, E = est/alpha and D = dev/beta:
//     E_i = a E_{i-1} + L_i ,   D_i = b D_{i-1} + |alpha E_i - L_i| ,
// and element i is pruned iff  L_i - alpha E_{i-1} + (la beta) D_{i-1} < 0.
// General scan kernel: element-wise access with bounds checks, any alignment, stride or width.
// COUNT: also produce the kept-weight count.  GATE: the drift gate described above.
template <bool BF16, bool COUNT, bool GATE>
__global__ void __launch_bounds__(kEwmaThreads, SP_EWMA_MIN_BLOCKS)
ewma_scan_kernel(const uint16_t *__restrict__ W, int ldw, int n_rows, int n,
                 const float *__restrict__ factor, const DeviceScalars *__restrict__ scalars,
                 const __grid_constant__ ScanConstants sc, uint32_t *__restrict__ mask,
                 int mask_words, uint16_t *__restrict__ W_out, int ldo,
                 unsigned long long *__restrict__ counters, const double *__restrict__ colsq) {
    pdl_launch_dependents();
    pdl_wait();  // the per-channel factors come from an earlier kernel of the stream
    const int lane = threadIdx.x & 31;
    const int row = blockIdx.x * kEwmaWarps + (threadIdx.x >> 5);
    if (row >= n_rows) return;  // warp-uniform
    const uint16_t *wrow = W + static_cast<int64_t>(row) * ldw;
    uint16_t *orow = W_out != nullptr ? W_out + static_cast<int64_t>(row) * ldo : nullptr;
    uint32_t *mrow = mask != nullptr ? mask + static_cast<int64_t>(row) * mask_words : nullptr;

    const float alpha = pinned(sc.alpha), neg_alpha = pinned(-sc.alpha);
    const float la_beta = pinned(sc.la * sc.beta);
    const float a = pinned(sc.a), b = pinned(sc.b);
    const float a_lane = pinned(sc.a_lane[lane]), b_lane = pinned(sc.b_lane[lane]);
    float a_step[5], b_step[5];
#pragma unroll
    for (int k = 0; k < 5; ++k) { a_step[k] = pinned(sc.a_step[k]); b_step[k] = pinned(sc.b_step[k]); }

    const int tiles = (n + kEwmaTile - 1) / kEwmaTile;
    float carry_E = 0.0f, carry_D = 0.0f;
    uint32_t kept = 0;
    int left_at = -1;  // GATE: column from which the row is walked sequentially
    const float hazard_w2 = GATE ? scalars->hazard_w2 : 0.0f;
    uint32_t p_next[4];
    load8<false, true>(wrow, lane * kEwmaPerLane, n, p_next);

    for (int tile = 0; tile < tiles; ++tile) {
        const int col = tile * kEwmaTile + lane * kEwmaPerLane;
        uint32_t p[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) p[k] = p_next[k];
        if (tile + 1 < tiles) load8<false, true>(wrow, col + kEwmaTile, n, p_next);

        float L[kEwmaPerLane], w[8], c[8];
        unpack8<BF16>(p, w);
        load_factor8(factor, col, c);  // zero past d_in: scores of padding are 0
#pragma unroll
        for (int j = 0; j < 8; ++j) L[j] = __fmul_rn(__fmul_rn(w[j], w[j]), c[j]);

        if (tile == 0) carry_E = __shfl_sync(kFullWarp, L[0], 0) / alpha;  // est starts at L_0
        if constexpr (GATE) {
            // a weight of this tile could change S if it were pruned: the sequential kernel
            // takes the row up from here (nothing of the tile has been stored yet)
            float w2max = 0.0f;
            bool odd = false;  // a NaN weight
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const float w2 = __fmul_rn(w[j], w[j]);
                odd = odd || !(w2 == w2);
                w2max = fmaxf(w2max, w2);
            }
            if (__any_sync(kFullWarp, odd || !(w2max < hazard_w2))) {
                left_at = tile * kEwmaTile;
                break;
            }
        }

        // Pass A: E over the lane's elements from a zero state -> lane total -> scan.
        float acc = L[0];
#pragma unroll
        for (int j = 1; j < kEwmaPerLane; ++j) acc = fmaf(a, acc, L[j]);
        float incl = lane_affine_scan(acc, a_step, lane);
        float excl = __shfl_up_sync(kFullWarp, incl, 1);
        if (lane == 0) excl = 0.0f;
        const float E_in = fmaf(a_lane, carry_E, excl);  // E before this lane's first element

        // Pass B: the true E from E_in; per element q_j = L_j - alpha E_{j-1} (the part of the
        // decision that does not need D) and |alpha E_j - L_j| (the input of D); D from a zero
        // state -> lane total -> scan.
        float q[kEwmaPerLane], dabs[kEwmaPerLane];
        float E_run = E_in, D_loc = 0.0f;
#pragma unroll
        for (int j = 0; j < kEwmaPerLane; ++j) {
            q[j] = fmaf(neg_alpha, E_run, L[j]);
            E_run = fmaf(a, E_run, L[j]);
            dabs[j] = fabsf(fmaf(alpha, E_run, -L[j]));
            D_loc = fmaf(b, D_loc, dabs[j]);
        }
        incl = lane_affine_scan(D_loc, b_step, lane);
        excl = __shfl_up_sync(kFullWarp, incl, 1);
        if (lane == 0) excl = 0.0f;
        const float D_in = fmaf(b_lane, carry_D, excl);

        // Pass C: the true D from D_in and the decisions against the state before each element's
        // update.  The sign bit of  L_i - est_{i-1} + la dev_{i-1}  is the prune flag (a NaN is
        // the positive canonical NaN: kept, as "L < threshold" is false); a byte permute with
        // sign replication turns two flags into the half-word mask of a packed pair of weights.
        float diff[kEwmaPerLane];
        float D_run = D_in;
#pragma unroll
        for (int j = 0; j < kEwmaPerLane; ++j) {
            diff[j] = fmaf(la_beta, D_run, q[j]);
            D_run = fmaf(b, D_run, dabs[j]);
        }
        uint32_t pm[4];
#pragma unroll
        for (int k = 0; k < 4; ++k)
            pm[k] = prmt(__float_as_uint(diff[2 * k]), __float_as_uint(diff[2 * k + 1]), 0xffbbu);
        uint32_t keep8 = ~halfmasks_to_bits(pm) & 0xffu;
        if (tile == 0 && lane == 0 && (keep8 & 1u) == 0u) {
            // column 0 is kept by definition (est starts at L_0); alpha*(L_0/alpha) may round up
            keep8 |= 1u;
            pm[0] &= 0xffff0000u;
        }
        const int left = n - col;
        if (left < kEwmaPerLane) keep8 &= left > 0 ? ((1u << left) - 1u) : 0u;
        if constexpr (COUNT) kept += __popc(keep8);

        carry_E = __shfl_sync(kFullWarp, E_run, 31);
        carry_D = __shfl_sync(kFullWarp, D_run, 31);

        if (orow != nullptr) {
#pragma unroll
            for (int k = 0; k < 4; ++k) p[k] &= ~pm[k];
            store8<false>(orow, col, n, p);
        }
        const uint32_t word = gather_mask_word(keep8, lane);  // four lanes share a mask word
        if (mrow != nullptr && (lane & 3) == 0 && col < n) mrow[col >> 5] = word;
    }

    unsigned long long walked = 0;
    if constexpr (GATE) {
        if (left_at >= 0 && lane == 0)
            walked = gate_walk<BF16>(wrow, orow, mrow, n, left_at, __fmul_rn(alpha, carry_E),
                                     __fmul_rn(sc.beta, carry_D), colsq, factor, scalars, sc.alpha,
                                     sc.beta, sc.la, counters);
    }
    if constexpr (COUNT) {
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) kept += __shfl_xor_sync(kFullWarp, kept, off);
        if (lane == 0 && kept + walked != 0ULL)
            atomicAdd(counters + SP_COUNTER_KEPT, static_cast<unsigned long long>(kept) + walked);
    }
}

// Paired-chain scan kernel for rows that allow 16-byte access.
//
// Same decomposition as ewma_scan_kernel (warp per row, two lane scans per tile), but a lane
// owns 16 consecutive weights (two 16-byte chunks) and a tile is 512 weights.  Each chunk is
// treated as two chains of 4 (elements 0-3 and 4-7) that advance together in the two halves of
// packed binary32 pairs (fma.rn.f32x2: one issue slot for two fused multiply-adds); the two
// chunks give every warp two independent instruction streams.  A later chain starts from the
// state the previous one ends in, which is known as soon as the previous chain's zero-state
// total is: E(4) = a^4 E(0) + T_0, E(8) = a^8 E(0) + (a^4 T_0 + T_1), ...
//
// Algebra used (scaled states E = est/alpha, D' = dev/(beta a)):
//     q_i  = L_i - alpha E_{i-1}                  (score minus the estimate it is tested against)
//     E_i  = a E_{i-1} + L_i
//     est_i - L_i = -a q_i   =>   D'_i = b D'_{i-1} + |q_i|
//     prune  <=>  q_i + kappa D'_{i-1} < 0 ,  kappa = la beta a .
// D' is a linear recurrence, so the state before element j of a chain entered with D'_in is
// Dloc_{j-1} + b^j D'_in (Dloc: the chain run from a zero state); the decision value is
// (q_j + kappa Dloc_{j-1}) + (kappa b^j) D'_in, whose first term is formed before the D scan
// and whose second needs one packed multiply-add per pair after it.
//
// The tile loop carries no special cases: the state before column 0 (est = L_0, Table 2) is set
// up before the loop such that the decision value of column 0 cannot be negative, the scan
// steps take their "has a partner lane" predicate from the shuffle itself, lane 0 folds the
// state carried in from the previous tile into its total before the scan (one lane rotation
// then gives every lane the state it starts from and lane 0 the state to carry on), and when
// the row is a whole number of tiles (FULL) there are no column guards.  Four tiles are
// processed per trip so that ring slots and address offsets are compile-time constants.
//
// Shared-memory ring: the copies of a tile are issued coalesced (instruction h moves the
// 16-byte chunk 32h + lane), while a lane reads chunks 2*lane and 2*lane + 1.  Chunk g is kept
// at position g ^ ((g >> 3) & 1): both the coalesced writes and the strided reads then touch
// eight different bank groups per quarter warp.
//
// The per-channel factors come from a copy of the factor array laid out for this kernel (see
// finalize_kernel): per 512-column tile, four 16-byte loads per lane, each contiguous across
// the warp, deliver the lane's 16 factors in pair order (columns 0,4,1,5 | 2,6,3,7 of a chunk).
struct PairConstants {
    float a4, b4;        // a^4, b^4: chain 0-3 -> chain 4-7
    float la;            // the decision constants kappa * b^j are formed on the device as
    float unit_b[4];     // la * (beta * a * b^j), the same way wherever la comes from
    int la_from_device;  // counting passes of the la search: la is DeviceScalars::search_la
    float hazard_scale;  // a^3 / 2, a little lowered (gate test on the chain totals)
};

struct TileConstants {
    float a_step[5], b_step[5];  // a^(16*2^k), b^(16*2^k)
    float a8, b8;
};

template <bool BF16, bool FULL, bool COUNT, bool GATE>
__global__ void __launch_bounds__(kPairThreads, SP_EWMA_PAIR_MIN_BLOCKS)
ewma_pair_scan_kernel(const __grid_constant__ EwmaJobTable jobs,
                      const __grid_constant__ ScanConstants sc,
                      const __grid_constant__ PairConstants pc,
                      const __grid_constant__ TileConstants wc,
                      unsigned long long *__restrict__ counters) {
    constexpr int kTile = 512;
    pdl_launch_dependents();
    pdl_wait();  // the per-channel factors come from an earlier kernel of the stream
    const int lane = threadIdx.x & 31;
    int jk = 0;  // the job of this CTA
    while (jk + 1 < jobs.count && static_cast<int>(blockIdx.x) >= jobs.job[jk + 1].first_cta) ++jk;
    const EwmaJob &job = jobs.job[jk];
    const int row = (static_cast<int>(blockIdx.x) - job.first_cta) * kPairWarps + (threadIdx.x >> 5);
    if (row >= job.n_rows) return;  // warp-uniform
    const int n = job.n;
    const int mask_words = job.mask_words;
    const float *__restrict__ factor_pairs = job.factor_pairs;
    const DeviceScalars *__restrict__ scalars = job.scalars;
    const uint16_t *wrow = job.W + static_cast<int64_t>(row) * job.ldw;
    uint16_t *const W_out = job.W_out;
    uint32_t *const mask = job.mask;
    uint16_t *olane = W_out != nullptr ? W_out + static_cast<int64_t>(row) * job.ldo + lane * 16 : nullptr;
    uint16_t *mlane = mask != nullptr
                          ? reinterpret_cast<uint16_t *>(mask + static_cast<int64_t>(row) * mask_words) + lane
                          : nullptr;
    const float4 *flane = reinterpret_cast<const float4 *>(factor_pairs) + lane;
    const int mask_halves = mask_words * 2;

    const float b = pinned(sc.b);
    const float2 a2 = make_float2(pinned(sc.a), pinned(sc.a));
    const float2 neg_alpha2 = make_float2(pinned(-sc.alpha), pinned(-sc.alpha));
    const float a4 = pinned(pc.a4), b4 = pinned(pc.b4), a8 = pinned(wc.a8), b8 = pinned(wc.b8);
    // lane 0 folds the state carried in from the previous tile into its total before the scan
    const float a16_lane0 = pinned(lane == 0 ? sc.a_step[1] : 0.0f);
    const float b16_lane0 = pinned(lane == 0 ? sc.b_step[1] : 0.0f);
    const int lane_below = (lane + 31) & 31;
    const bool is_lane0 = lane == 0;
    float la = pc.la;
    if constexpr (COUNT) {
        // the bisection of sp_search_la keeps its current la on the device
        if (pc.la_from_device) la = scalars->search_la;
    }
    float kappa_b[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) kappa_b[j] = __fmul_rn(la, pc.unit_b[j]);
    const float kappa = pinned(kappa_b[0]);
    const float2 kappa2 = make_float2(kappa, kappa);
    float2 kappa_b2[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) kappa_b2[j] = make_float2(pinned(kappa_b[j]), pinned(kappa_b[j]));
    uint32_t kept = 0;
    float hz_thr = 0.0f;
    if constexpr (GATE) hz_thr = scalars->hazard_w2 * pc.hazard_scale;

    constexpr int kSlot = 64;  // uint4 per warp and stage
    __shared__ __align__(16) uint4 ring[kPairWarps * kEwmaStages * kSlot];
    __shared__ int gate_snap[GATE ? kPairWarps : 1][4 + 32];
    uint4 *my_ring = ring + (threadIdx.x >> 5) * kEwmaStages * kSlot;
    const int wpos = lane ^ ((lane >> 3) & 1);               // where this lane's copies go
    const int rpos_a = 2 * lane + ((lane >> 2) & 1);         // where chunk 2*lane sits
    const int rpos_b = 2 * lane + 1 - ((lane >> 2) & 1);     // where chunk 2*lane + 1 sits
    const int tiles = (n + kTile - 1) / kTile;
    auto issue_tile = [&](int t, int slot) {
        if (t < tiles) {
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int c = t * kTile + (32 * h + lane) * 8;
                if (FULL || c < n) cp_async16(my_ring + slot * kSlot + 32 * h + wpos, wrow + c, 16);
            }
        }
        cp_async_commit();
    };
#pragma unroll
    for (int t = 0; t < kEwmaStages - 1; ++t) issue_tile(t, t);

    // State before column 0: est = L_0, i.e. E = L_0 / alpha, lowered by one ulp when rounding
    // would make  L_0 - alpha E  negative, so that column 0 is never pruned (Table 2).
    float carry_E, carry_D = 0.0f;
    {
        cp_async_wait<kEwmaStages - 2>();
        const float w0 = unpack_lo<BF16>(my_ring[rpos_a].x);  // lane 0: its own copy of chunk 0
        const float L0 = __fmul_rn(__fmul_rn(w0, w0), __ldg(factor_pairs));
        float e = L0 / sc.alpha;
        if (fmaf(-sc.alpha, e, L0) < 0.0f) e = __uint_as_float(__float_as_uint(e) - 1u);
        carry_E = is_lane0 ? e : 0.0f;  // only lane 0's copy of the carried states is used
    }

    float4 cf_next[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) cf_next[i] = __ldg(flane + 32 * i);
    if constexpr (GATE) {
        if (is_lane0) gate_snap[threadIdx.x >> 5][0] = -1;  // no column recorded yet
    }
    for (int t0 = 0; t0 < tiles; t0 += kEwmaStages) {
#pragma unroll
        for (int u = 0; u < kEwmaStages; ++u) {
            const int tile = t0 + u;
            if (tile >= tiles) break;  // warp-uniform
            const int col = tile * kTile + lane * 16;
            // factors in pair order: (0,4,1,5) (2,6,3,7) of either chunk; zero past d_in
            float4 cf[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {  // those of the next tile are requested now
                cf[i] = cf_next[i];
                cf_next[i] = __ldg(flane + (tile + 1) * 128 + 32 * i);  // padded by one tile
            }
            issue_tile(tile + kEwmaStages - 1, (u + kEwmaStages - 1) & (kEwmaStages - 1));
            cp_async_wait<kEwmaStages - 1>();
            __syncwarp();  // the copies of this tile were made by other lanes
            uint4 v[2];
            v[0] = my_ring[u * kSlot + rpos_a];
            v[1] = my_ring[u * kSlot + rpos_b];
            bool in_row[2];
            uint32_t p[2][4];
            float2 L2[2][4];  // chunk x: (L_j, L_{j+4})
            float2 acc[2];
#pragma unroll
            for (int x = 0; x < 2; ++x) {
                in_row[x] = FULL || col + 8 * x < n;
                if (!in_row[x]) v[x] = make_uint4(0u, 0u, 0u, 0u);
                p[x][0] = v[x].x; p[x][1] = v[x].y; p[x][2] = v[x].z; p[x][3] = v[x].w;
                float2 w2;
                w2 = make_float2(unpack_lo<BF16>(p[x][0]), unpack_lo<BF16>(p[x][2]));
                L2[x][0] = __fmul2_rn(__fmul2_rn(w2, w2), make_float2(cf[2 * x].x, cf[2 * x].y));
                w2 = make_float2(unpack_hi<BF16>(p[x][0]), unpack_hi<BF16>(p[x][2]));
                L2[x][1] = __fmul2_rn(__fmul2_rn(w2, w2), make_float2(cf[2 * x].z, cf[2 * x].w));
                w2 = make_float2(unpack_lo<BF16>(p[x][1]), unpack_lo<BF16>(p[x][3]));
                L2[x][2] = __fmul2_rn(__fmul2_rn(w2, w2), make_float2(cf[2 * x + 1].x, cf[2 * x + 1].y));
                w2 = make_float2(unpack_hi<BF16>(p[x][1]), unpack_hi<BF16>(p[x][3]));
                L2[x][3] = __fmul2_rn(__fmul2_rn(w2, w2), make_float2(cf[2 * x + 1].z, cf[2 * x + 1].w));
                // E: the chunk's two chains from a zero state
                acc[x] = L2[x][0];
#pragma unroll
                for (int j = 1; j < 4; ++j) acc[x] = __ffma2_rn(a2, acc[x], L2[x][j]);
            }
            // chunk totals -> lane total (+ a^16 carry in lane 0) -> scan over lanes
            const float tot_a = fmaf(a4, acc[0].x, acc[0].y), tot_b = fmaf(a4, acc[1].x, acc[1].y);
            const float lane_tot = fmaf(a8, tot_a, tot_b);
            if constexpr (GATE) {
                // Every score is at least w^2 / 2 and a chain's zero-state total at least a^3
                // times any of its 4 scores, so four totals below the scaled bound rule out a
                // weight that could change S (a NaN fails the test as well).  Otherwise the
                // sequential kernel takes the row up from this tile: nothing of it has been
                // stored yet, and nothing more of the row is stored or counted here.
                const float m4 = fmaxf(fmaxf(acc[0].x, acc[0].y), fmaxf(acc[1].x, acc[1].y));
                if (__any_sync(kFullWarp, !(lane_tot == lane_tot) || !(m4 < hz_thr))) {
                    // (rare) remember the column, the scaled state before it and the count so
                    // far - only the first time - and stop storing: the outputs are off from here
                    int *snap = gate_snap[threadIdx.x >> 5];
                    const bool first = snap[0] < 0;
                    __syncwarp();
                    if (first) {
                        snap[4 + lane] = static_cast<int>(kept);
                        if (is_lane0) {
                            snap[0] = tile * kTile;
                            snap[1] = __float_as_int(carry_E);
                            snap[2] = __float_as_int(carry_D);
                        }
                    }
                    olane = nullptr;
                    mlane = nullptr;
                }
            }
            float incl = lane_affine_scan_pred(fmaf(a16_lane0, carry_E, lane_tot), wc.a_step);
            float rot = __shfl_sync(kFullWarp, incl, lane_below);
            const float e0 = is_lane0 ? carry_E : rot;  // E before element 0
            carry_E = rot;
            float2 E2[2];
            E2[0].x = e0;
            E2[0].y = fmaf(a4, e0, acc[0].x);           // before element 4
            E2[1].x = fmaf(a8, e0, tot_a);              // before element 8
            E2[1].y = fmaf(a4, E2[1].x, acc[1].x);      // before element 12

            float2 r2[2][4], dl[2];
#pragma unroll
            for (int x = 0; x < 2; ++x) {
                float2 q2[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    q2[j] = __ffma2_rn(neg_alpha2, E2[x], L2[x][j]);
                    E2[x] = __ffma2_rn(a2, E2[x], L2[x][j]);
                }
                r2[x][0] = q2[0];
                r2[x][1].x = fmaf(kappa, fabsf(q2[0].x), q2[1].x);
                r2[x][1].y = fmaf(kappa, fabsf(q2[0].y), q2[1].y);
                dl[x].x = fmaf(b, fabsf(q2[0].x), fabsf(q2[1].x));
                dl[x].y = fmaf(b, fabsf(q2[0].y), fabsf(q2[1].y));
#pragma unroll
                for (int j = 2; j < 4; ++j) {
                    r2[x][j] = __ffma2_rn(kappa2, dl[x], q2[j]);
                    dl[x].x = fmaf(b, dl[x].x, fabsf(q2[j].x));
                    dl[x].y = fmaf(b, dl[x].y, fabsf(q2[j].y));
                }
            }
            const float dtot_a = fmaf(b4, dl[0].x, dl[0].y), dtot_b = fmaf(b4, dl[1].x, dl[1].y);
            incl = lane_affine_scan_pred(
                fmaf(b16_lane0, carry_D, fmaf(b8, dtot_a, dtot_b)), wc.b_step);
            rot = __shfl_sync(kFullWarp, incl, lane_below);
            const float d0 = is_lane0 ? carry_D : rot;  // D' before element 0
            carry_D = rot;
            float2 D2[2];
            D2[0].x = d0;
            D2[0].y = fmaf(b4, d0, dl[0].x);
            D2[1].x = fmaf(b8, d0, dtot_a);
            D2[1].y = fmaf(b4, D2[1].x, dl[1].x);

            uint32_t keep16 = 0;
#pragma unroll
            for (int x = 0; x < 2; ++x) {
                // Decision values; their sign bits are the prune flags (a NaN is the positive
                // canonical NaN: kept, as "L < threshold" is false).
                float2 diff2[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) diff2[j] = __ffma2_rn(kappa_b2[j], D2[x], r2[x][j]);
                uint32_t pm[4];
                pm[0] = prmt(__float_as_uint(diff2[0].x), __float_as_uint(diff2[1].x), 0xffbbu);
                pm[1] = prmt(__float_as_uint(diff2[2].x), __float_as_uint(diff2[3].x), 0xffbbu);
                pm[2] = prmt(__float_as_uint(diff2[0].y), __float_as_uint(diff2[1].y), 0xffbbu);
                pm[3] = prmt(__float_as_uint(diff2[2].y), __float_as_uint(diff2[3].y), 0xffbbu);
                uint32_t keep8 = ~halfmasks_to_bits(pm) & 0xffu;
                if (!in_row[x]) keep8 = 0u;
                keep16 |= keep8 << (8 * x);
                if (olane != nullptr && in_row[x] &&
                    SP_IN_RANGE(col + 8 * x + 7, job.ldo, kDbgEwmaColumn)) {
#pragma unroll
                    for (int k = 0; k < 4; ++k) p[x][k] &= ~pm[k];
                    __stcs(reinterpret_cast<uint4 *>(olane + tile * kTile + 8 * x),
                           make_uint4(p[x][0], p[x][1], p[x][2], p[x][3]));
                }
            }
            if constexpr (COUNT) kept += __popc(keep16);
            // two mask bytes per lane: a little-endian half word holds columns 16k .. 16k+15
            if (mlane != nullptr && (FULL || tile * 32 + lane < mask_halves) &&
                SP_IN_RANGE(tile * 32 + lane, mask_halves, kDbgEwmaMask))
                mlane[tile * 32] = static_cast<uint16_t>(keep16);
            __syncwarp();  // all lanes have read this slot before it is refilled
        }
    }

    unsigned long long walked = 0;
    if constexpr (GATE) {
        __syncwarp();
        const int *snap = gate_snap[threadIdx.x >> 5];
        if (snap[0] >= 0) {  // the scan stopped storing at column snap[0]: walk the rest
            kept = static_cast<uint32_t>(snap[4 + lane]);  // kept before that column
            if (is_lane0)
                walked = gate_walk<BF16>(
                    wrow, W_out != nullptr ? W_out + static_cast<int64_t>(row) * job.ldo : nullptr,
                    mask != nullptr ? mask + static_cast<int64_t>(row) * mask_words : nullptr, n,
                    snap[0], __fmul_rn(sc.alpha, __int_as_float(snap[1])),
                    __fmul_rn(pc.unit_b[0], __int_as_float(snap[2])), job.colsq, job.factor, scalars,
                    sc.alpha, sc.beta, la, counters);
        }
    }
    if constexpr (COUNT) {
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) kept += __shfl_xor_sync(kFullWarp, kept, off);
        if (lane == 0 && kept + walked != 0ULL)
            atomicAdd(counters + SP_COUNTER_KEPT, static_cast<unsigned long long>(kept) + walked);
    }
}

// The sequential path for rows that do not allow 16-byte access (ewma_literal_tiled_kernel
// handles those that do): one thread per row, whole rows.
template <bool BF16>
__global__ void __launch_bounds__(128)
ewma_literal_kernel(const uint16_t *__restrict__ W, int64_t ldw, int64_t n_rows, int64_t n,
                    const double *__restrict__ colsq, const float *__restrict__ factor,
                    const DeviceScalars *__restrict__ scalars, float alpha, float beta, float la,
                    uint32_t *__restrict__ mask, int64_t mask_words,
                    uint16_t *__restrict__ W_out, int64_t ldo,
                    unsigned long long *__restrict__ counters, int subtract_x2) {
    const int64_t row = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (row >= n_rows) return;
    const unsigned long long kept = literal_walk<BF16>(
        W + row * ldw, W_out != nullptr ? W_out + row * ldo : nullptr,
        mask != nullptr ? mask + row * mask_words : nullptr, n, 0, 0.0f, 0.0f, colsq, factor,
        scalars->S32, alpha, beta, la, subtract_x2 != 0);
    if (counters != nullptr) atomicAdd(counters + SP_COUNTER_KEPT, kept);
}

// Diagnostic: the state Algorithm 1 tests every weight against (est and dev before the update
// of element i) and the score L_i, written out along each row; one thread per row, sequential,
// binary32 with one rounding per operation like the literal kernel (S updated when s_update
// says so).  This is the data behind the paper's Fig. 2 (est / dev tracking the mean and the
// L1 deviation of L along a row).
template <bool BF16>
__global__ void __launch_bounds__(128)
ewma_trace_kernel(const uint16_t *__restrict__ W, int64_t ldw, int64_t n_rows, int64_t n,
                  const double *__restrict__ colsq, const DeviceScalars *__restrict__ scalars,
                  float alpha, float beta, float la, int literal_s, float *__restrict__ est_out,
                  float *__restrict__ dev_out, float *__restrict__ score_out) {
    const int64_t row = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (row >= n_rows) return;
    const uint16_t *wrow = W + row * ldw;
    const float one_minus_alpha = __fsub_rn(1.0f, alpha);
    const float one_minus_beta = __fsub_rn(1.0f, beta);
    float S = scalars->S32;
    float est = 0.0f, dev = 0.0f;
    for (int64_t i = 0; i < n; ++i) {
        const uint16_t bits = wrow[i];
        const float w = BF16 ? __uint_as_float(static_cast<uint32_t>(bits) << 16)
                             : __half2float(__ushort_as_half(bits));
        const float u = __fdiv_rn(static_cast<float>(colsq[i]), S);
        const float c = __fdiv_rn(0.5f, __fsub_rn(1.0f, u));
        const float w2 = __fmul_rn(w, w);
        const float L = __fmul_rn(w2, c);
        if (i == 0) est = L;
        if (est_out != nullptr) est_out[row * n + i] = est;
        if (dev_out != nullptr) dev_out[row * n + i] = dev;
        if (score_out != nullptr) score_out[row * n + i] = L;
        const float thr = __fsub_rn(est, __fmul_rn(la, dev));
        if (L < thr && literal_s) S = __fsub_rn(S, literal_s == 2 ? static_cast<float>(colsq[i]) : w2);
        est = __fadd_rn(__fmul_rn(one_minus_alpha, est), __fmul_rn(alpha, L));
        dev = __fadd_rn(__fmul_rn(one_minus_beta, dev), __fmul_rn(beta, fabsf(__fsub_rn(est, L))));
    }
}

sp_status launch_ewma_trace(const sp_ctx *ctx, const void *W, sp_dtype dtype, int64_t n_rows,
                            int64_t ldw, const sp_ewma_params &p, float *est_out, float *dev_out,
                            float *score_out, cudaStream_t stream) {
    if (n_rows == 0) return SP_OK;
    const int64_t blocks = (n_rows + 127) / 128;
    if (blocks > 0x7fffffffLL) return SP_ERR_SHAPE;
    const uint16_t *Wp = static_cast<const uint16_t *>(W);
    const int literal = p.s_update == SP_S_FROZEN ? 0 : (p.s_update == SP_S_READING_X2 ? 2 : 1);  // gated = as printed
    if (dtype == SP_BF16)
        ewma_trace_kernel<true><<<static_cast<unsigned>(blocks), 128, 0, stream>>>(
            Wp, ldw, n_rows, ctx->d_in, ctx->colsq, ctx->scalars, p.alpha, p.beta, p.la, literal,
            est_out, dev_out, score_out);
    else
        ewma_trace_kernel<false><<<static_cast<unsigned>(blocks), 128, 0, stream>>>(
            Wp, ldw, n_rows, ctx->d_in, ctx->colsq, ctx->scalars, p.alpha, p.beta, p.la, literal,
            est_out, dev_out, score_out);
    return check_launch();
}

static void fill_scan_constants(const sp_ewma_params &p, ScanConstants &sc) {
    sc.alpha = p.alpha;
    sc.beta = p.beta;
    sc.la = p.la;
    sc.a = 1.0f - p.alpha;
    sc.b = 1.0f - p.beta;
    const double a = static_cast<double>(sc.a), b = static_cast<double>(sc.b);
    for (int l = 0; l < 32; ++l) {
        sc.a_lane[l] = static_cast<float>(pow(a, static_cast<double>(kEwmaPerLane) * l));
        sc.b_lane[l] = static_cast<float>(pow(b, static_cast<double>(kEwmaPerLane) * l));
    }
    for (int k = 0; k < 5; ++k) {
        sc.a_step[k] = static_cast<float>(pow(a, static_cast<double>(kEwmaPerLane) * (1 << k)));
        sc.b_step[k] = static_cast<float>(pow(b, static_cast<double>(kEwmaPerLane) * (1 << k)));
    }
}

bool ewma_pair_path_applies(const void *W, int64_t ldw, int64_t n) {
    return aligned16(W) && ldw % 8 == 0 && n % 8 == 0;
}

namespace {

bool job_is_vector(const EwmaLaunchJob &j, int64_t n) {
    return aligned16(j.W) && j.ldw % 8 == 0 && n % 8 == 0 &&
           (j.W_out == nullptr || (aligned16(j.W_out) && j.ldo % 8 == 0));
}

// Statistics a job is pruned with: its own context's, else those of the call's context.
inline const sp_ctx *job_ctx(const EwmaLaunchJob &j, const sp_ctx *ctx) {
    return j.ctx != nullptr ? j.ctx : ctx;
}

// Device-side table of the jobs [first, first + count); false if there are too many rows.
bool fill_job_table(const sp_ctx *ctx, const EwmaLaunchJob *jobs, int first, int count,
                    EwmaJobTable &t) {
    t.count = count;
    int64_t ctas = 0;
    for (int i = 0; i < count; ++i) {
        const EwmaLaunchJob &j = jobs[first + i];
        const sp_ctx *c = job_ctx(j, ctx);
        EwmaJob &d = t.job[i];
        d.W = static_cast<const uint16_t *>(j.W);
        d.W_out = static_cast<uint16_t *>(j.W_out);
        d.mask = j.mask;
        d.factor_pairs = c->factor_pairs;
        d.scalars = c->scalars;
        d.colsq = c->colsq;
        d.factor = c->factor;
        d.ldw = static_cast<int>(j.ldw);
        d.ldo = static_cast<int>(j.ldo);
        d.n_rows = static_cast<int>(j.n_rows);
        d.n = static_cast<int>(c->d_in);
        d.mask_words = static_cast<int>((c->d_in + 31) / 32);
        d.first_cta = static_cast<int>(ctas);
        ctas += (j.n_rows + kPairWarps - 1) / kPairWarps;
    }
    t.total_ctas = static_cast<int>(ctas);
    return ctas <= 0x7fffffffLL;
}

// The frozen-S scan (with the drift gate, if asked for) over jobs that share one launch: all of
// them allow 16-byte access, or there is a single job.
sp_status launch_scan_group(const sp_ctx *ctx, const EwmaLaunchJob *jobs, int first, int count,
                            sp_dtype dtype, const sp_ewma_params &p,
                            unsigned long long *counters, cudaStream_t stream,
                            bool la_from_device) {
    const bool bf16 = dtype == SP_BF16;
    const bool gated = p.s_update == SP_S_GATED;
    EwmaJobTable table{};
    if (!fill_job_table(ctx, jobs, first, count, table)) return SP_ERR_SHAPE;
    if (table.total_ctas == 0) return SP_OK;

    ScanConstants sc;
    fill_scan_constants(p, sc);
    cudaError_t launch_err = cudaSuccess;
    const sp_ctx *c0 = job_ctx(jobs[first], ctx);
    const bool vec = job_is_vector(jobs[first], c0->d_in);  // groups are uniform in this respect
    if (vec) {
        const double a = static_cast<double>(sc.a), b = static_cast<double>(sc.b);
        PairConstants pc{};
        pc.a4 = static_cast<float>(pow(a, 4.0));
        pc.b4 = static_cast<float>(pow(b, 4.0));
        pc.la = p.la;
        for (int j = 0; j < 4; ++j)
            pc.unit_b[j] = static_cast<float>(static_cast<double>(p.beta) * sc.a * pow(b, j));
        pc.la_from_device = la_from_device ? 1 : 0;
        pc.hazard_scale = static_cast<float>(pow(a, 3.0) * 0.5 * (1.0 - 1.0 / 1024.0));
        TileConstants wc;
        for (int k = 0; k < 5; ++k) {
            wc.a_step[k] = static_cast<float>(pow(a, 16.0 * (1 << k)));
            wc.b_step[k] = static_cast<float>(pow(b, 16.0 * (1 << k)));
        }
        wc.a8 = sc.a_step[0];
        wc.b8 = sc.b_step[0];
        bool full_tiles = true;  // every row of the launch a whole number of tiles
        for (int i = 0; i < count; ++i) full_tiles = full_tiles && table.job[i].n % 512 == 0;
        PdlConfig pdlp(dim3(static_cast<unsigned>(table.total_ctas)), dim3(kPairThreads), stream);
#define SP_LAUNCH_P(B, F, C, G)                                                              \
    launch_err = cudaLaunchKernelEx(&pdlp.cfg, ewma_pair_scan_kernel<B, F, C, G>, table, sc,  \
                                    pc, wc, counters)
#define SP_LAUNCH_PC(B, F, C)                                                                \
    do {                                                                                     \
        if (gated) SP_LAUNCH_P(B, F, C, true); else SP_LAUNCH_P(B, F, C, false);             \
    } while (0)
#define SP_LAUNCH_PF(B, F)                                                                   \
    do {                                                                                     \
        if (counters != nullptr) SP_LAUNCH_PC(B, F, true); else SP_LAUNCH_PC(B, F, false);   \
    } while (0)
        if (bf16) {
            if (full_tiles) SP_LAUNCH_PF(true, true); else SP_LAUNCH_PF(true, false);
        } else {
            if (full_tiles) SP_LAUNCH_PF(false, true); else SP_LAUNCH_PF(false, false);
        }
#undef SP_LAUNCH_PF
#undef SP_LAUNCH_PC
#undef SP_LAUNCH_P
    } else {
        const EwmaJob &j = table.job[0];
        const int n = j.n, words = j.mask_words;
        const float *factor = j.factor;
        const DeviceScalars *scalars = j.scalars;
        const double *colsq = j.colsq;
        const int64_t ldw = j.ldw, ldo = j.ldo, n_rows = j.n_rows;
        PdlConfig pdl(dim3(static_cast<unsigned>((j.n_rows + kEwmaWarps - 1) / kEwmaWarps)),
                      dim3(kEwmaThreads), stream);
#define SP_LAUNCH_S(B, C, G)                                                                 \
    launch_err = cudaLaunchKernelEx(&pdl.cfg, ewma_scan_kernel<B, C, G>, j.W, ldw, n_rows, n, \
                                    factor, scalars, sc, j.mask, words, j.W_out, ldo,         \
                                    counters, colsq)
#define SP_LAUNCH_SC(B, C)                                                                   \
    do {                                                                                     \
        if (gated) SP_LAUNCH_S(B, C, true); else SP_LAUNCH_S(B, C, false);                   \
    } while (0)
        if (bf16) {
            if (counters != nullptr) SP_LAUNCH_SC(true, true); else SP_LAUNCH_SC(true, false);
        } else {
            if (counters != nullptr) SP_LAUNCH_SC(false, true); else SP_LAUNCH_SC(false, false);
        }
#undef SP_LAUNCH_SC
#undef SP_LAUNCH_S
    }
    if (launch_err != cudaSuccess) return cuda_fail(launch_err);
    return check_launch();
}

sp_status launch_literal(const sp_ctx *ctx, const EwmaLaunchJob &j, sp_dtype dtype,
                         const sp_ewma_params &p, unsigned long long *counters,
                         cudaStream_t stream) {
    const int64_t n = ctx->d_in;
    if (j.n_rows == 0) return SP_OK;
    if (job_is_vector(j, n))  // rows that allow 16-byte access: the same arithmetic, rows moved in tiles
        return launch_ewma_literal_tiled(ctx, j.W, dtype, j.n_rows, j.ldw, p, j.mask, j.W_out, j.ldo,
                                         counters, stream);
    const int64_t blocks = (j.n_rows + 127) / 128;
    if (blocks > 0x7fffffffLL) return SP_ERR_SHAPE;
    const unsigned lgrid = static_cast<unsigned>(blocks);
    const uint16_t *Wp = static_cast<const uint16_t *>(j.W);
    uint16_t *Op = static_cast<uint16_t *>(j.W_out);
    const int64_t words = (n + 31) / 32;
    if (dtype == SP_BF16)
        ewma_literal_kernel<true><<<lgrid, 128, 0, stream>>>(
            Wp, j.ldw, j.n_rows, n, ctx->colsq, ctx->factor, ctx->scalars, p.alpha, p.beta, p.la,
            j.mask, words, Op, j.ldo, counters, p.s_update == SP_S_READING_X2 ? 1 : 0);
    else
        ewma_literal_kernel<false><<<lgrid, 128, 0, stream>>>(
            Wp, j.ldw, j.n_rows, n, ctx->colsq, ctx->factor, ctx->scalars, p.alpha, p.beta, p.la,
            j.mask, words, Op, j.ldo, counters, p.s_update == SP_S_READING_X2 ? 1 : 0);
    return check_launch();
}

}  // namespace

sp_status launch_select_ewma(const sp_ctx *ctx, const EwmaLaunchJob *jobs_in, int n_jobs,
                             sp_dtype dtype, const sp_ewma_params &p, unsigned long long *counters,
                             cudaStream_t stream, bool la_from_device) {
    // Cut every matrix into pieces of at most kEwmaMaxLaunchRows rows ...
    EwmaLaunchJob pieces[64];
    int n_pieces = 0;
    for (int i = 0; i < n_jobs; ++i) {
        const EwmaLaunchJob &j = jobs_in[i];
        const int64_t words = (job_ctx(j, ctx)->d_in + 31) / 32;
        if (j.n_rows < 0 || j.ldw > 0x7fffffffLL || j.ldo > 0x7fffffffLL) return SP_ERR_SHAPE;
        for (int64_t r0 = 0; r0 < j.n_rows; r0 += kEwmaMaxLaunchRows) {
            if (n_pieces == 64) return SP_ERR_SHAPE;
            EwmaLaunchJob &q = pieces[n_pieces++];
            q = j;
            q.n_rows = j.n_rows - r0 < kEwmaMaxLaunchRows ? j.n_rows - r0 : kEwmaMaxLaunchRows;
            q.W = static_cast<const uint16_t *>(j.W) + r0 * j.ldw;
            if (j.W_out != nullptr) q.W_out = static_cast<uint16_t *>(j.W_out) + r0 * j.ldo;
            if (j.mask != nullptr) q.mask = j.mask + r0 * words;
        }
    }
    if (p.s_update == SP_S_LITERAL_SCAN) {
        for (int i = 0; i < n_pieces; ++i) {
            const EwmaLaunchJob &j = pieces[i];
            sp_status st = launch_ewma_sweep(job_ctx(j, ctx), j.W, dtype, j.n_rows, j.ldw, p, j.mask,
                                             j.W_out, j.ldo, counters, stream);
            if (st != SP_OK) return st;
        }
        return SP_OK;
    }
    if (p.s_update == SP_S_LITERAL_W2 || p.s_update == SP_S_READING_X2) {
        for (int i = 0; i < n_pieces; ++i) {
            sp_status st = launch_literal(job_ctx(pieces[i], ctx), pieces[i], dtype, p, counters, stream);
            if (st != SP_OK) return st;
        }
        return SP_OK;
    }
    // ... and give consecutive pieces that allow 16-byte access one launch.
    int first = 0;
    while (first < n_pieces) {
        int count = 1;
        if (job_is_vector(pieces[first], job_ctx(pieces[first], ctx)->d_in)) {
            int64_t bits = pieces[first].n_rows;
            while (first + count < n_pieces && count < kEwmaMaxJobs &&
                   job_is_vector(pieces[first + count], job_ctx(pieces[first + count], ctx)->d_in)) {
                const int64_t more = pieces[first + count].n_rows;
                if (bits + more > kEwmaMaxLaunchRows) break;
                bits += more;
                ++count;
            }
        }
        sp_status st = launch_scan_group(ctx, pieces, first, count, dtype, p, counters, stream,
                                         la_from_device);
        if (st != SP_OK) return st;
        first += count;
    }
    return SP_OK;
}

// Bisection of la on the device: no host round trip between the counting passes.
__global__ void search_init_kernel(DeviceScalars *s, float lo, float hi) {
    s->search_lo = lo;
    s->search_hi = hi;
    s->search_la = 0.5f * (lo + hi);
    s->search_best_la = 0.0f;
    s->search_best_gap = 2.0;
    s->search_best_frac = 0.0;
    for (int i = 0; i < SP_NUM_COUNTERS; ++i) s->search_counters[i] = 0ULL;
}

__global__ void search_step_kernel(DeviceScalars *s, double total, double target) {
    const float la = s->search_la;
    const double pruned = 1.0 - static_cast<double>(s->search_counters[SP_COUNTER_KEPT]) / total;
    const double gap = fabs(pruned - target);
    if (gap < s->search_best_gap) {
        s->search_best_gap = gap;
        s->search_best_la = la;
        s->search_best_frac = pruned;
    }
    if (pruned > target)
        s->search_lo = la;  // too much pruned: raise la
    else
        s->search_hi = la;
    s->search_la = 0.5f * (s->search_lo + s->search_hi);
    for (int i = 0; i < SP_NUM_COUNTERS; ++i) s->search_counters[i] = 0ULL;
}

sp_status launch_search_la_device(sp_ctx *ctx, const void *W, sp_dtype dtype, int64_t n_rows,
                                  int64_t ldw, float target, float alpha, float beta,
                                  int iterations, float *la_out, double *achieved_out,
                                  cudaStream_t stream) {
    DeviceScalars *sc = ctx->scalars;
    const double total = static_cast<double>(n_rows) * static_cast<double>(ctx->d_in);
    search_init_kernel<<<1, 1, 0, stream>>>(sc, -8.0f, 8.0f);
    sp_status st = check_launch();
    if (st != SP_OK) return st;
    sp_ewma_params p;
    p.alpha = alpha;
    p.beta = beta;
    p.la = 0.0f;  // unused: the kernel reads DeviceScalars::search_la
    p.s_update = SP_S_FROZEN;
    for (int it = 0; it < iterations; ++it) {
        st = launch_select_ewma(ctx, W, dtype, n_rows, ldw, p, nullptr, nullptr, ldw,
                                sc->search_counters, stream, /*la_from_device=*/true);
        if (st != SP_OK) return st;
        search_step_kernel<<<1, 1, 0, stream>>>(sc, total, static_cast<double>(target));
        st = check_launch();
        if (st != SP_OK) return st;
    }
    float best_la = 0.0f;
    double best_frac = 0.0;
    cudaError_t e = cudaMemcpyAsync(&best_la, &sc->search_best_la, sizeof(float),
                                    cudaMemcpyDeviceToHost, stream);
    if (e == cudaSuccess)
        e = cudaMemcpyAsync(&best_frac, &sc->search_best_frac, sizeof(double),
                            cudaMemcpyDeviceToHost, stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize(stream);
    if (e != cudaSuccess) return cuda_fail(e);
    *la_out = best_la;
    if (achieved_out != nullptr) *achieved_out = best_frac;
    return SP_OK;
}

}  // namespace sp
