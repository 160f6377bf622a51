// N:M selection (Section 3.3) fused with score, mask emission and write-back.
//
// Work layout.  The column axis is cut into strips of 256 columns; a warp owns one strip and a
// slab of consecutive rows, a lane owns 8 consecutive columns of the strip (one 16-byte access
// per row), i.e. two groups of four or one group of eight: a group never straddles lanes, so
// the selection needs no cross-lane traffic.  The 8 per-channel factors c_q of the lane's
// columns are loaded once and stay in registers for the whole slab, and several rows are kept
// in flight per lane: in select_nm_stream_kernel (rows that allow 16-byte access) through a
// small per-lane ring in shared memory filled by asynchronous copies (a lane only reads what it
// copied itself), in select_nm_kernel (any other layout, element-wise access) in registers.
//
// Selection.  Scores are L = (w*w)*c_q in binary32 (Eq. 8); they are non-negative, so they are
// compared through their bit patterns as unsigned integers, which also ranks NaN above every
// number.  Element i orders before element j when L_i < L_j, or L_i == L_j and i < j; an
// element is kept when at least M-N elements of its group order before it.  The counts of all
// 8 elements of a lane live in the bytes of two registers, biased so that a byte's top bit is
// the keep flag; a byte permute with sign replication turns those bits into the 16-bit masks
// that zero the pruned weights, and a two-way dot product packs them into the 8 mask bits.
#include "nm_rank.cuh"
#include "sp_device.cuh"
#include "sp_internal.h"

namespace sp {

// Tuning knobs (compile-time): rows kept in flight per lane (general kernel), resident CTAs per
// SM asked of ptxas, the fewest rows a warp gets and the warps per SM the launcher aims for.
#ifndef SP_NM_ROWS_IN_FLIGHT
#define SP_NM_ROWS_IN_FLIGHT 4
#endif
#ifndef SP_NM_MIN_BLOCKS
#define SP_NM_MIN_BLOCKS 8
#endif
#ifndef SP_NM_MIN_ROWS
#define SP_NM_MIN_ROWS 8
#endif
#ifndef SP_NM_TARGET_WARPS
#define SP_NM_TARGET_WARPS 256
#endif
#ifndef SP_NM_THREADS
#define SP_NM_THREADS 128
#endif
constexpr int kNmMaxJobs = 16;  // matrices one launch can cover
constexpr int kNmThreads = SP_NM_THREADS;
constexpr int kNmWarps = kNmThreads / 32;
constexpr int kNmRowsInFlight = SP_NM_ROWS_IN_FLIGHT;

// One row of one lane: score, rank, masks, write-back.  Returns the 8 keep bits.
template <bool BF16, int M>
__device__ __forceinline__ uint32_t nm_process_row(uint32_t (&p)[4], const float (&c)[8],
                                                   uint32_t bias_lo, uint32_t bias_hi,
                                                   uint32_t valid, uint16_t *out_row, int64_t col,
                                                   int64_t n) {
    float w[8];
    unpack8<BF16>(p, w);
    uint32_t key[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) key[j] = __float_as_uint(__fmul_rn(__fmul_rn(w[j], w[j]), c[j]));
    // half-word masks from the top bit of each rank field (sign replication)
    uint32_t m[4];
    if constexpr (M == 4) {
        uint32_t ra, rb;
        nm_rank_bytes<4>(key, bias_lo, bias_hi, ra, rb);
        m[0] = prmt(ra, 0u, 0x9988u);
        m[1] = prmt(ra, 0u, 0xbbaau);
        m[2] = prmt(rb, 0u, 0x9988u);
        m[3] = prmt(rb, 0u, 0xbbaau);
    } else {
        masks_from_nibbles(nm_rank_nibbles8(key, bias_lo), m);  // bias_lo holds the nibble bias
    }
    if (out_row != nullptr) {
#pragma unroll
        for (int k = 0; k < 4; ++k) p[k] &= m[k];
        store8<false>(out_row, col, n, p);
    }
    return halfmasks_to_bits(m) & valid;
}

template <bool BF16, int M>
__global__ void __launch_bounds__(kNmThreads, SP_NM_MIN_BLOCKS)
select_nm_kernel(const uint16_t *__restrict__ W, int ldw, int n_rows, int64_t n,
                 int rows_per_warp, const float *__restrict__ factor, int prune_count,
                 uint32_t *__restrict__ mask, int mask_words, uint16_t *__restrict__ W_out,
                 int ldo) {
    pdl_launch_dependents();
    pdl_wait();  // the per-channel factors come from an earlier kernel of the stream
    const int lane = threadIdx.x & 31;
    const int64_t col = static_cast<int64_t>(blockIdx.x) * kStripChannels + lane * 8;
    const int slab = blockIdx.y * kNmWarps + (threadIdx.x >> 5);
    const int64_t row_begin64 = static_cast<int64_t>(slab) * rows_per_warp;
    if (row_begin64 >= n_rows) return;  // warp-uniform
    const int row_begin = static_cast<int>(row_begin64);
    const int rows = min(n_rows - row_begin, rows_per_warp);

    float c[8];
    load_factor8(factor, col, c);  // zero past d_in
    const int64_t left = n - col;
    const uint32_t valid = left >= 8 ? 0xffu : (left > 0 ? (1u << left) - 1u : 0u);
    // M == 4: rank bytes in two registers; M == 8: rank nibbles in one (see nm_rank.cuh)
    const uint32_t bias_lo =
        M == 4 ? static_cast<uint32_t>(0x80 - prune_count) * 0x01010101u + 0x03020100u
               : static_cast<uint32_t>(8 - prune_count) * 0x11111111u + 0x76543210u;
    const uint32_t bias_hi = bias_lo;
    const bool store_word = mask != nullptr && (lane & 3) == 0 && left > 0;

    // Row pointers advance by whole rows; row index times leading dimension is a 32x32->64
    // multiply-add on the current pointer.
    const uint16_t *wp = W + static_cast<int64_t>(row_begin) * ldw;
    uint16_t *op = W_out != nullptr ? W_out + static_cast<int64_t>(row_begin) * ldo : nullptr;
    uint32_t *mp = mask != nullptr ? mask + static_cast<int64_t>(row_begin) * mask_words + (col >> 5)
                                   : nullptr;

    int r = 0;
    for (; r + kNmRowsInFlight <= rows; r += kNmRowsInFlight) {
        uint32_t p[kNmRowsInFlight][4];
#pragma unroll
        for (int u = 0; u < kNmRowsInFlight; ++u)
            load8<false, true>(wp + static_cast<int64_t>(u) * ldw, col, n, p[u]);
#pragma unroll
        for (int u = 0; u < kNmRowsInFlight; ++u) {
            uint16_t *orow = op != nullptr ? op + static_cast<int64_t>(u) * ldo : nullptr;
            const uint32_t keep8 =
                nm_process_row<BF16, M>(p[u], c, bias_lo, bias_hi, valid, orow, col, n);
            const uint32_t word = gather_mask_word(keep8, lane);
            if (store_word) mp[static_cast<int64_t>(u) * mask_words] = word;
        }
        wp += static_cast<int64_t>(kNmRowsInFlight) * ldw;
        if (op != nullptr) op += static_cast<int64_t>(kNmRowsInFlight) * ldo;
        if (mp != nullptr) mp += static_cast<int64_t>(kNmRowsInFlight) * mask_words;
    }
    for (; r < rows; ++r) {  // fewer than kNmRowsInFlight rows left in the slab
        uint32_t p[4];
        load8<false, true>(wp, col, n, p);
        const uint32_t keep8 =
            nm_process_row<BF16, M>(p, c, bias_lo, bias_hi, valid, op, col, n);
        const uint32_t word = gather_mask_word(keep8, lane);
        if (store_word) *mp = word;
        wp += ldw;
        if (op != nullptr) op += ldo;
        if (mp != nullptr) mp += mask_words;
    }
}

// Streaming kernel for rows that allow 16-byte access (the fast path).  Same work layout and
// selection as select_nm_kernel; what differs is the bookkeeping around it: scores are formed
// two at a time in packed binary32 pairs (mul.rn.f32x2, each half rounded like a scalar
// product), the rows run through a four-slot per-lane ring whose slots are compile-time
// constants (four rows per trip), every lane stores its own mask byte (byte k of a
// little-endian mask word holds columns 8k .. 8k+7) instead of assembling words across lanes,
// and when the strip is whole (FULL: d_in a multiple of 256) there are no column guards.
// OUT / MASK: the pruned weights / the keep mask are requested.  The launch covers a table of
// matrices, each with the per-channel factors of the input it reads (layers of one input, or all
// layers of a block).  A matrix owns whole CTAs - strips x groups of kNmWarps slabs, strips
// fastest - so the matrix of a CTA, and with it the width and every pointer, is CTA-uniform.
struct NmJob {
    const uint16_t *W;
    uint16_t *W_out;  // nullable
    uint32_t *mask;   // nullable
    const float *factor;
    int ldw, ldo, n_rows;
    int n, mask_words, strips;
    int first_cta;
};
struct NmJobTable {
    int count;
    int total_ctas;
    NmJob job[kNmMaxJobs];
};

template <bool BF16, bool FULL, int M, bool OUT, bool MASK>
__global__ void __launch_bounds__(kNmThreads, SP_NM_MIN_BLOCKS)
select_nm_stream_kernel(const __grid_constant__ NmJobTable jobs, int rows_per_warp,
                        int prune_count) {
    pdl_launch_dependents();
    pdl_wait();  // the per-channel factors come from an earlier kernel of the stream
    const int lane = threadIdx.x & 31;
    int jk = 0;  // the matrix of this CTA
    while (jk + 1 < jobs.count && static_cast<int>(blockIdx.x) >= jobs.job[jk + 1].first_cta) ++jk;
    const NmJob &job = jobs.job[jk];
    const int local = static_cast<int>(blockIdx.x) - job.first_cta;
    const int slab_group = local / job.strips;
    const int col = (local - slab_group * job.strips) * kStripChannels + lane * 8;
    const int n = job.n, mask_words = job.mask_words;
    const float *__restrict__ factor = job.factor;
    const uint16_t *const W = job.W;
    uint16_t *const W_out = job.W_out;
    uint32_t *const mask = job.mask;
    const int ldw = job.ldw, ldo = job.ldo, n_rows = job.n_rows;
    const int row_begin = (slab_group * kNmWarps + (threadIdx.x >> 5)) * rows_per_warp;
    if (row_begin >= n_rows) return;  // warp-uniform
    const int rows = min(n_rows - row_begin, rows_per_warp);
    const bool in_row = FULL || col < n;  // d_in % 8 == 0: a chunk is inside or outside as a whole

    float2 cp[4];  // factors of columns (0,1) (2,3) (4,5) (6,7) of the chunk, zero past d_in
    {
        float c[8];
        load_factor8(factor, col, c);
#pragma unroll
        for (int k = 0; k < 4; ++k) cp[k] = make_float2(c[2 * k], c[2 * k + 1]);
    }
    // M == 4: rank bytes in two registers; M == 8: rank nibbles in one (see nm_rank.cuh)
    const uint32_t bias =
        M == 4 ? static_cast<uint32_t>(0x80 - prune_count) * 0x01010101u + 0x03020100u
               : static_cast<uint32_t>(8 - prune_count) * 0x11111111u + 0x76543210u;

    const uint16_t *src = W + static_cast<int64_t>(row_begin) * ldw + (in_row ? col : 0);
    uint16_t *dst = OUT ? W_out + static_cast<int64_t>(row_begin) * ldo + (in_row ? col : 0) : nullptr;
    const int mask_pitch = mask_words * 4;  // bytes per mask row
    const bool in_mask = FULL || (col >> 3) < mask_pitch;
    uint8_t *mdst = MASK ? reinterpret_cast<uint8_t *>(mask + static_cast<int64_t>(row_begin) * mask_words) +
                               (in_mask ? col >> 3 : 0)
                         : nullptr;

    constexpr int kStages = 4;
    __shared__ __align__(16) uint4 ring[kNmWarps * kStages * 32];
    uint4 *my_ring = ring + (threadIdx.x >> 5) * kStages * 32 + lane;
    auto issue = [&](int rr, int slot) {
        if (rr < rows && in_row)
            cp_async16(my_ring + slot * 32, src + static_cast<int64_t>(rr) * ldw, 16);
        cp_async_commit();
    };
#pragma unroll
    for (int rr = 0; rr < kStages - 1; ++rr) issue(rr, rr);

    // One row of this lane: wait for its copy, score, rank, masks, write-back.
    auto process = [&](int rr, int slot) {
        issue(rr + kStages - 1, (slot + kStages - 1) & (kStages - 1));
        cp_async_wait<kStages - 1>();
        uint4 v = make_uint4(0u, 0u, 0u, 0u);
        if (in_row) v = my_ring[slot * 32];
        uint32_t p[4] = {v.x, v.y, v.z, v.w};
        uint32_t key[8];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const float2 w2 = unpack2<BF16>(p[k]);
            const float2 L2 = __fmul2_rn(__fmul2_rn(w2, w2), cp[k]);
            key[2 * k] = __float_as_uint(L2.x);
            key[2 * k + 1] = __float_as_uint(L2.y);
        }
        // half-word masks from the top bit of each rank field (sign replication)
        uint32_t m[4];
        if constexpr (M == 4) {
            uint32_t ra, rb;
            nm_rank_bytes<4>(key, bias, bias, ra, rb);
            m[0] = prmt(ra, 0u, 0x9988u);
            m[1] = prmt(ra, 0u, 0xbbaau);
            m[2] = prmt(rb, 0u, 0x9988u);
            m[3] = prmt(rb, 0u, 0xbbaau);
        } else {
            masks_from_nibbles(nm_rank_nibbles8(key, bias), m);
        }
        if (OUT && in_row && SP_IN_RANGE(row_begin + rr, n_rows, kDbgNmRow) &&
            SP_IN_RANGE(col + 7, ldo, kDbgNmColumn)) {
            __stcs(reinterpret_cast<uint4 *>(dst + static_cast<int64_t>(rr) * ldo),
                   make_uint4(p[0] & m[0], p[1] & m[1], p[2] & m[2], p[3] & m[3]));
        }
        if (MASK && in_mask) {
            const uint32_t keep8 = in_row ? halfmasks_to_bits(m) & 0xffu : 0u;
            mdst[static_cast<int64_t>(rr) * mask_pitch] = static_cast<uint8_t>(keep8);
        }
    };
    int r0 = 0;
    for (; r0 + kStages <= rows; r0 += kStages) {  // four rows per trip: static ring slots
#pragma unroll
        for (int u = 0; u < kStages; ++u) process(r0 + u, u);
    }
    for (int rr = r0; rr < rows; ++rr) process(rr, rr & (kStages - 1));  // r0 % kStages == 0
}

namespace {

bool nm_job_is_vector(const EwmaLaunchJob &j, int64_t n) {
    return aligned16(j.W) && j.ldw % 8 == 0 && n % 8 == 0 &&
           (j.W_out == nullptr || (aligned16(j.W_out) && j.ldo % 8 == 0));
}

inline const sp_ctx *nm_job_ctx(const EwmaLaunchJob &j, const sp_ctx *ctx) {
    return j.ctx != nullptr ? j.ctx : ctx;
}

// Jobs [first, first + count) in one launch: either all of them allow 16-byte access and ask
// for the same outputs, or count == 1.
sp_status launch_nm_group(const sp_ctx *ctx, const EwmaLaunchJob *jobs, int first, int count,
                          sp_dtype dtype, int N, int M, cudaStream_t stream) {
    int64_t row_strips = 0, total_rows = 0;  // warps' worth of work: rows x 256-column strips
    for (int i = 0; i < count; ++i) {
        row_strips += jobs[first + i].n_rows * nm_job_ctx(jobs[first + i], ctx)->strips;
        total_rows += jobs[first + i].n_rows;
    }
    if (total_rows == 0) return SP_OK;
    // Short slabs, i.e. many warps (measured: 8 rows per warp for the LLaMA-sized layers is 3-7 %
    // faster than 16-32, and than 4 once the SM clock is held down by the power cap).
    const int64_t target_warps = static_cast<int64_t>(ctx->sm_count) * SP_NM_TARGET_WARPS;
    int64_t rows_per_warp = (row_strips + target_warps - 1) / target_warps;
    rows_per_warp = (rows_per_warp + kNmRowsInFlight - 1) / kNmRowsInFlight * kNmRowsInFlight;
    if (rows_per_warp < SP_NM_MIN_ROWS) rows_per_warp = SP_NM_MIN_ROWS;

    const EwmaLaunchJob &j0 = jobs[first];
    const sp_ctx *c0 = nm_job_ctx(j0, ctx);
    const int64_t n = c0->d_in;
    const bool vec = nm_job_is_vector(j0, n);
    if (!vec) {
        // element-wise kernel (a single matrix, grid = strips x slab groups): keep gridDim.y legal
        // for very tall matrices by giving each warp more rows
        const int64_t max_grid_y = 65535;
        if ((j0.n_rows + rows_per_warp * kNmWarps - 1) / (rows_per_warp * kNmWarps) > max_grid_y) {
            rows_per_warp = (j0.n_rows + max_grid_y * kNmWarps - 1) / (max_grid_y * kNmWarps);
            rows_per_warp = (rows_per_warp + kNmRowsInFlight - 1) / kNmRowsInFlight * kNmRowsInFlight;
        }
        if (rows_per_warp > 0x7fffffffLL) return SP_ERR_SHAPE;
    }
    NmJobTable table{};
    int64_t ctas = 0;
    for (;;) {  // the CTAs of the launch; a grid that would not fit gets longer slabs
        table.count = count;
        ctas = 0;
        for (int i = 0; i < count; ++i) {
            const EwmaLaunchJob &j = jobs[first + i];
            const sp_ctx *c = nm_job_ctx(j, ctx);
            if (j.n_rows > 0x7fffffffLL || j.ldw > 0x7fffffffLL || j.ldo > 0x7fffffffLL) return SP_ERR_SHAPE;
            NmJob &d = table.job[i];
            d.W = static_cast<const uint16_t *>(j.W);
            d.W_out = static_cast<uint16_t *>(j.W_out);
            d.mask = j.mask;
            d.factor = c->factor;
            d.ldw = static_cast<int>(j.ldw);
            d.ldo = static_cast<int>(j.ldo);
            d.n_rows = static_cast<int>(j.n_rows);
            d.n = static_cast<int>(c->d_in);
            d.mask_words = static_cast<int>((c->d_in + 31) / 32);
            d.strips = c->strips;
            d.first_cta = static_cast<int>(ctas);
            const int64_t slabs = (j.n_rows + rows_per_warp - 1) / rows_per_warp;
            ctas += (slabs + kNmWarps - 1) / kNmWarps * c->strips;
        }
        if (ctas <= 0x7fffffffLL) break;
        rows_per_warp *= 2;
        if (rows_per_warp > 0x7fffffffLL) return SP_ERR_SHAPE;
    }
    table.total_ctas = static_cast<int>(ctas);
    const uint16_t *Wp = static_cast<const uint16_t *>(j0.W);
    uint16_t *Op = static_cast<uint16_t *>(j0.W_out);
    uint32_t *mask = j0.mask;
    const int words = static_cast<int>((n + 31) / 32);
    const int prune_count = M - N;
    const int rpw = static_cast<int>(rows_per_warp);
    const float *factor = c0->factor;
    cudaError_t launch_err = cudaSuccess;
    const int64_t slabs0 = (j0.n_rows + rows_per_warp - 1) / rows_per_warp;
    PdlConfig pdl(vec ? dim3(static_cast<unsigned>(ctas))
                      : dim3(static_cast<unsigned>(c0->strips),
                             static_cast<unsigned>((slabs0 + kNmWarps - 1) / kNmWarps)),
                  dim3(kNmThreads), stream);
#define SP_LAUNCH(B, MM)                                                                     \
    launch_err = cudaLaunchKernelEx(&pdl.cfg, select_nm_kernel<B, MM>, Wp,                    \
                                    static_cast<int>(j0.ldw), static_cast<int>(j0.n_rows), n, \
                                    rpw, factor, prune_count, mask, words, Op,                \
                                    static_cast<int>(j0.ldo))
#define SP_LAUNCH_M(B)                                                                        \
    do {                                                                                      \
        if (M == 8) SP_LAUNCH(B, 8); else SP_LAUNCH(B, 4);                                    \
    } while (0)
#define SP_LAUNCH_ST(B, F, MM, O, K)                                                         \
    launch_err = cudaLaunchKernelEx(&pdl.cfg, select_nm_stream_kernel<B, F, MM, O, K>, table, \
                                    rpw, prune_count)
#define SP_LAUNCH_STO(B, F, MM)                                                               \
    do {                                                                                      \
        if (Op != nullptr && mask != nullptr) SP_LAUNCH_ST(B, F, MM, true, true);             \
        else if (Op != nullptr) SP_LAUNCH_ST(B, F, MM, true, false);                          \
        else SP_LAUNCH_ST(B, F, MM, false, true);                                             \
    } while (0)
#define SP_LAUNCH_STM(B, F)                                                                   \
    do {                                                                                      \
        if (M == 8) SP_LAUNCH_STO(B, F, 8); else SP_LAUNCH_STO(B, F, 4);                      \
    } while (0)
    bool full = true;  // every matrix a whole number of strips wide
    for (int i = 0; i < count; ++i) full = full && table.job[i].n % kStripChannels == 0;
    if (vec) {
        if (dtype == SP_BF16) {
            if (full) SP_LAUNCH_STM(true, true); else SP_LAUNCH_STM(true, false);
        } else {
            if (full) SP_LAUNCH_STM(false, true); else SP_LAUNCH_STM(false, false);
        }
    } else if (dtype == SP_BF16) {
        SP_LAUNCH_M(true);
    } else {
        SP_LAUNCH_M(false);
    }
#undef SP_LAUNCH_STM
#undef SP_LAUNCH_STO
#undef SP_LAUNCH_ST
#undef SP_LAUNCH_M
#undef SP_LAUNCH
    if (launch_err != cudaSuccess) return cuda_fail(launch_err);
    return check_launch();
}

}  // namespace

sp_status launch_select_nm(const sp_ctx *ctx, const EwmaLaunchJob *jobs_in, int n_jobs,
                           sp_dtype dtype, int N, int M, cudaStream_t stream) {
    // jobs that produce nothing are dropped; consecutive jobs that allow 16-byte access and ask
    // for the same outputs share a launch
    EwmaLaunchJob jobs[kNmMaxJobs];
    int count = 0;
    for (int i = 0; i < n_jobs; ++i) {
        if (jobs_in[i].n_rows == 0 || (jobs_in[i].mask == nullptr && jobs_in[i].W_out == nullptr)) continue;
        if (count == kNmMaxJobs) return SP_ERR_INVALID_ARG;
        jobs[count++] = jobs_in[i];
    }
    int first = 0;
    while (first < count) {
        int group = 1;
        if (nm_job_is_vector(jobs[first], nm_job_ctx(jobs[first], ctx)->d_in)) {
            while (first + group < count &&
                   nm_job_is_vector(jobs[first + group], nm_job_ctx(jobs[first + group], ctx)->d_in) &&
                   (jobs[first + group].mask != nullptr) == (jobs[first].mask != nullptr) &&
                   (jobs[first + group].W_out != nullptr) == (jobs[first].W_out != nullptr))
                ++group;
        }
        sp_status st = launch_nm_group(ctx, jobs, first, group, dtype, N, M, stream);
        if (st != SP_OK) return st;
        first += group;
    }
    return SP_OK;
}

}  // namespace sp
