// Calibration statistics (Algorithm 1, step 1): streaming column sums of squares over the
// tokens x d_in activations, and the finalisation that turns them into S and the
// per-channel factor of Eq. 8.
//
// Layout of the work: the channel axis is cut into strips of 256 channels (one warp-wide
// 16-byte load per activation row), the token axis into slabs.  One CTA owns one
// (strip, slab) cell; its 8 warps take rows slab_begin + warp, + 8, ... and keep 8 rows in
// flight per lane.  Squares are exact in fp32 (formed straight from the 16-bit values by the
// mixed-precision fused multiply-add); the sum of the 8 in-flight squares is formed in fp32 and
// added to an fp64 accumulator.  The CTA adds its 256 sums to row `slab` of the
// partial-sum array, which no other CTA touches: there are no floating-point atomics, so the
// statistics are reproducible bit for bit for a given sequence of batches.
#include <mutex>

#include "sp_device.cuh"
#include "sp_internal.h"

namespace sp {

constexpr int kCalibThreads = 256;
constexpr int kCalibWarps = kCalibThreads / 32;
constexpr int kRowsInFlight = 8;
constexpr int kFinalGroups = 4;  // slab groups summed in parallel by the finalisation kernel
constexpr int kFinalThreads = kFinalGroups * kStripChannels;
constexpr int kFinalMaxJobs = 16;  // contexts one finalisation launch can cover

// One activation matrix of an accumulate launch.  I: the type of its sizes - 64-bit for a single
// matrix, whose sizes the kernel reads from the constant bank wherever it uses them; 32-bit for a
// table of matrices, where the sizes of the CTA's matrix live in registers for the whole kernel.
template <class I>
struct CalibMatrixT {
    const uint16_t *X;
    double *partial;
    I ldx, n_tokens, n, n_pad, rows_per_slab;
    int strips, first_fresh_slab, first_cta;
};

// Launch arguments, in two shapes with one kernel body.  CalibOne: a single matrix on a
// strips x slabs grid.  CalibMany: several matrices (the inputs of one transformer block, say)
// in one launch for inputs so small that a launch of their own would be mostly ramp-up; a matrix
// owns strips x slabs consecutive CTAs of a 1-D grid, strips fastest.
struct CalibOne {
    using Matrix = CalibMatrixT<int64_t>;
    Matrix m;
    __device__ __forceinline__ const Matrix &cell(int &strip, int &slab) const {
        strip = blockIdx.x;
        slab = blockIdx.y;
        return m;
    }
};
constexpr int kCalibMaxJobs = 8;
struct CalibMany {
    using Matrix = CalibMatrixT<int>;
    int count;
    Matrix job[kCalibMaxJobs];
    __device__ __forceinline__ const Matrix &cell(int &strip, int &slab) const {
        int jk = 0;
        while (jk + 1 < count && static_cast<int>(blockIdx.x) >= job[jk + 1].first_cta) ++jk;
        const int local = static_cast<int>(blockIdx.x) - job[jk].first_cta;
        slab = local / job[jk].strips;
        strip = local - slab * job[jk].strips;
        return job[jk];
    }
};

template <bool BF16, bool VEC, class Args>
__global__ void __launch_bounds__(kCalibThreads, VEC ? 4 : 1)  // 16-byte path: 4 CTAs per SM
calib_accumulate_kernel(const __grid_constant__ Args args, int x_complete) {
    // Programmatic dependent launch: the next kernel in the stream may start as soon as this
    // grid's CTAs are all resident.  X is read only after everything queued earlier on the
    // stream has completed - the kernel before this one may be the one that writes X - unless
    // the caller vouches that X was complete before that (x_complete): then the streaming phase
    // overlaps the tail of the previous kernel and only the read-modify-write of the partial
    // sums below waits for it.
    pdl_launch_dependents();
    if (!x_complete) pdl_wait();
    int strip, slab;
    const typename Args::Matrix &a = args.cell(strip, slab);
    using I = decltype(a.ldx);
    const uint16_t *__restrict__ X = a.X;
    const I ldx = a.ldx, n = a.n;
    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    const I col = static_cast<I>(strip) * kStripChannels + lane * 8;
    const I row_begin = static_cast<I>(slab) * a.rows_per_slab;
    const I row_end = min(a.n_tokens, row_begin + a.rows_per_slab);

    double acc[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) acc[j] = 0.0;

    for (I r = row_begin + warp; r < row_end; r += kCalibWarps * kRowsInFlight) {
        uint32_t v[kRowsInFlight][4];
#pragma unroll
        for (int u = 0; u < kRowsInFlight; ++u) {
            const I rr = r + static_cast<I>(u) * kCalibWarps;
            if (rr < row_end) {
                load8<VEC, true>(X + static_cast<int64_t>(rr) * ldx, col, n, v[u]);
            } else {
                v[u][0] = v[u][1] = v[u][2] = v[u][3] = 0u;
            }
        }
        float s[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) s[j] = 0.0f;
#pragma unroll
        for (int u = 0; u < kRowsInFlight; ++u) {
#pragma unroll
            for (int k = 0; k < 4; ++k) fma_square2<BF16>(v[u][k], s[2 * k], s[2 * k + 1]);
        }
#pragma unroll
        for (int j = 0; j < 8; ++j) acc[j] += static_cast<double>(s[j]);
    }

    // Combine the 8 warps in a fixed order, then add to this cell's row of `partial`.
    __shared__ double sm[kCalibWarps][kStripChannels];
#pragma unroll
    for (int j = 0; j < 8; ++j) sm[warp][lane * 8 + j] = acc[j];
    __syncthreads();
    pdl_wait();  // earlier kernels' partial sums are final
    // (the matrix is looked up again rather than carried through the loop in registers)
    int strip_out, slab_out;
    const typename Args::Matrix &b = args.cell(strip_out, slab_out);
    const int t = threadIdx.x;
    const int64_t ch = static_cast<int64_t>(strip_out) * kStripChannels + t;
    if (ch < b.n) {
        double sum = 0.0;
#pragma unroll
        for (int w = 0; w < kCalibWarps; ++w) sum += sm[w][t];
        const int64_t at = static_cast<int64_t>(slab_out) * b.n_pad + ch;
        double *dst = b.partial + at;
        if (SP_IN_RANGE(at, kMaxSlabs * static_cast<int64_t>(b.n_pad), kDbgCalibPartial)) {
            if (slab_out >= b.first_fresh_slab)
                *dst = sum;
            else
                *dst += sum;
        }
    }
}

// Finalisation.  CTA `strip` sums its 256 channels over the valid slab rows (four slab groups
// in parallel, each in ascending order, then the groups in order), writes colsq and its strip
// total; the last CTA to arrive adds the strip totals in
// ascending order to S and writes the per-channel factor for every channel:
//     u = colsq32 / S32 ;  den = 1 - u ;  c = 0.5 / den          (binary32, round to nearest)
// No CTA waits for another one (the last arrival does the tail), so the kernel cannot hang.
__device__ __forceinline__ void finalize_strip(
    const double *__restrict__ partial, int slabs_valid, int64_t n, int64_t n_pad, int strips,
    double *__restrict__ colsq, double *__restrict__ strip_sum, float *__restrict__ factor,
    float *__restrict__ factor_pairs, DeviceScalars *__restrict__ scalars, int strip) {
    __shared__ double part[kFinalGroups][kStripChannels];
    __shared__ double red[kStripChannels];
    __shared__ bool is_last;
    pdl_launch_dependents();
    pdl_wait();  // all partial sums are in place
    const int t = threadIdx.x & (kStripChannels - 1);  // channel within the strip
    const int g = threadIdx.x / kStripChannels;        // slab group
    const int64_t ch = static_cast<int64_t>(strip) * kStripChannels + t;
    // Group g adds a contiguous range of slabs in ascending order (eight loads in flight);
    // the groups are then added in ascending order: a fixed summation order.
    const int per_group = (slabs_valid + kFinalGroups - 1) / kFinalGroups;
    const int s_begin = g * per_group;
    const int s_end = min(slabs_valid, s_begin + per_group);
    double v = 0.0;
    if (ch < n) {
        const double *src = partial + ch;
        int s = s_begin;
        for (; s + 8 <= s_end; s += 8) {
            double x[8];
#pragma unroll
            for (int k = 0; k < 8; ++k) x[k] = __ldcg(src + static_cast<int64_t>(s + k) * n_pad);
#pragma unroll
            for (int k = 0; k < 8; ++k) v += x[k];
        }
        for (; s < s_end; ++s) v += __ldcg(src + static_cast<int64_t>(s) * n_pad);
    }
    part[g][t] = v;
    __syncthreads();
    if (g == 0) {
        v = part[0][t];
#pragma unroll
        for (int k = 1; k < kFinalGroups; ++k) v += part[k][t];
        colsq[ch] = v;  // ch < n_pad always; padding gets 0
        red[t] = v;
    }
    __syncthreads();
    for (int half = kStripChannels / 2; half > 0; half >>= 1) {
        if (threadIdx.x < half) red[threadIdx.x] += red[threadIdx.x + half];
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        strip_sum[strip] = red[0];
        __threadfence();
        unsigned int ticket = atomicAdd(&scalars->ticket, 1u);
        is_last = (ticket == static_cast<unsigned int>(strips) - 1u);
    }
    __syncthreads();
    if (!is_last) return;
    __threadfence();

    // S: thread i < 256 adds the strip totals i, i+256, ... in ascending order, then the same
    // fixed tree as above combines the 256 partial sums (deterministic, loads in parallel).
    if (threadIdx.x < kStripChannels) {
        double acc = 0.0;
        for (int s = threadIdx.x; s < strips; s += kStripChannels) acc += __ldcg(strip_sum + s);
        red[threadIdx.x] = acc;
    }
    __syncthreads();
    for (int half = kStripChannels / 2; half > 0; half >>= 1) {
        if (threadIdx.x < half) red[threadIdx.x] += red[threadIdx.x + half];
        __syncthreads();
    }
    const double S = red[0];
    const float S32 = static_cast<float>(S);
    if (threadIdx.x == 0) {
        int flags = 0;
        if (!(S > 0.0) || isinf(S) || isnan(S) || isinf(S32)) flags |= kFlagDegenerate;
        // "S - w^2" leaves S unchanged in binary32 whenever w^2 is below a quarter of the
        // spacing of floats at S: 2^(e-25) for S in [2^e, 2^(e+1)).
        float hazard = 0.0f;
        if (!flags) {
            const int e = static_cast<int>((__float_as_uint(S32) >> 23) & 0xffu);
            hazard = e > 25 ? __uint_as_float(static_cast<uint32_t>(e - 25) << 23) : 0.0f;
        }
        scalars->S = S;
        scalars->S32 = S32;
        scalars->hazard_w2 = hazard;
        scalars->flags = flags;
        scalars->ticket = 0u;
    }
    // per-channel factors, four channels per thread in flight
    for (int64_t q0 = threadIdx.x; q0 < n_pad; q0 += 4 * kFinalThreads) {
        double x[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const int64_t q = q0 + static_cast<int64_t>(k) * kFinalThreads;
            x[k] = q < n ? __ldcg(colsq + q) : 0.0;
        }
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const int64_t q = q0 + static_cast<int64_t>(k) * kFinalThreads;
            if (q < n_pad) {
                float c = 0.0f;
                if (q < n) {
                    const float u = __fdiv_rn(static_cast<float>(x[k]), S32);
                    const float den = __fsub_rn(1.0f, u);
                    c = __fdiv_rn(0.5f, den);
                }
                factor[q] = c;
                // Second copy for the EWMA pair kernel, whose lanes own 16 consecutive columns
                // of a 512-column tile and pair column j of a chunk of 8 with column j + 4:
                // [tile][float4 i = 2 * chunk + pos / 4][lane][pos % 4], pos = place of the
                // column in the order 0,4,1,5,2,6,3,7.
                if (factor_pairs != nullptr) {
                    const int64_t e = q & 7;
                    const int64_t pos = e < 4 ? 2 * e : 2 * (e - 4) + 1;
                    const int64_t r = q & 511, ln = r >> 4, ch = (r >> 3) & 1;
                    const int64_t at = (q & ~int64_t(511)) + (2 * ch + (pos >> 2)) * 128 + ln * 4 + (pos & 3);
                    if (SP_IN_RANGE(at, (n_pad + 511) / 512 * 512 + 512, kDbgFactorPairs)) factor_pairs[at] = c;
                }
            }
        }
    }
}

__global__ void __launch_bounds__(kFinalThreads)
finalize_kernel(const double *__restrict__ partial, int slabs_valid, int64_t n, int64_t n_pad,
                int strips, double *__restrict__ colsq, double *__restrict__ strip_sum,
                float *__restrict__ factor, float *__restrict__ factor_pairs,
                DeviceScalars *__restrict__ scalars) {
    finalize_strip(partial, slabs_valid, n, n_pad, strips, colsq, strip_sum, factor, factor_pairs,
                   scalars, blockIdx.x);
}

// Several contexts in one launch: context j owns the CTAs [first_cta, first_cta + strips) and has
// its own arrival counter, so the contexts do not wait for each other either.
struct FinalJob {
    const double *partial;
    double *colsq, *strip_sum;
    float *factor, *factor_pairs;
    DeviceScalars *scalars;
    int64_t n, n_pad;
    int slabs_valid, strips, first_cta;
};
struct FinalJobTable {
    int count;
    FinalJob job[kFinalMaxJobs];
};

__global__ void __launch_bounds__(kFinalThreads)
finalize_multi_kernel(const __grid_constant__ FinalJobTable jobs) {
    int jk = 0;
    while (jk + 1 < jobs.count && static_cast<int>(blockIdx.x) >= jobs.job[jk + 1].first_cta) ++jk;
    const FinalJob &j = jobs.job[jk];
    finalize_strip(j.partial, j.slabs_valid, j.n, j.n_pad, j.strips, j.colsq, j.strip_sum, j.factor,
                   j.factor_pairs, j.scalars, static_cast<int>(blockIdx.x) - j.first_cta);
}

template <bool BF16, bool VEC>
static int query_blocks_per_sm() {
    int blocks = 0;
    cudaError_t e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(
        &blocks, calib_accumulate_kernel<BF16, VEC, CalibOne>, kCalibThreads, 0);
    if (e != cudaSuccess || blocks < 1) blocks = 1;
    return blocks;
}

int calib_query_blocks_per_sm() { return query_blocks_per_sm<false, true>(); }

// Slabs and rows per slab for one activation matrix of a launch that covers `total_strips`
// strips in all (its own, plus those of the other matrices of a multi-input launch).
static void calib_partition(const sp_ctx *ctx, int64_t n_tokens, int64_t total_strips,
                            int64_t &slabs, int64_t &rows_per_slab) {
    // One resident wave: strips x slabs CTAs fill the GPU once, every CTA gets the same rows.
    const int64_t resident = static_cast<int64_t>(ctx->sm_count) * ctx->calib_blocks_per_sm;
    slabs = resident / total_strips;
    if (slabs < 1) slabs = 1;
    if (slabs > kMaxSlabs) slabs = kMaxSlabs;
    const int64_t min_rows = kCalibWarps * kRowsInFlight;  // at least one full step per warp
    const int64_t max_slabs_by_rows = (n_tokens + min_rows - 1) / min_rows;
    if (slabs > max_slabs_by_rows) slabs = max_slabs_by_rows;
    rows_per_slab = (n_tokens + slabs - 1) / slabs;
    rows_per_slab = (rows_per_slab + kCalibWarps - 1) / kCalibWarps * kCalibWarps;
    slabs = (n_tokens + rows_per_slab - 1) / rows_per_slab;
}

sp_status launch_calib_accumulate(sp_ctx *ctx, const void *X, sp_dtype dtype, int64_t n_tokens,
                                  int64_t ldx, cudaStream_t stream, bool x_complete) {
    const int64_t n = ctx->d_in;
    int64_t slabs, rows_per_slab;
    calib_partition(ctx, n_tokens, ctx->strips, slabs, rows_per_slab);

    const bool vec = aligned16(X) && (ldx % 8 == 0) && (n % 8 == 0);
    const bool bf16 = dtype == SP_BF16;
    dim3 grid(static_cast<unsigned>(ctx->strips), static_cast<unsigned>(slabs));
    PdlConfig pdl(grid, dim3(kCalibThreads), stream);
    CalibOne args{};
    args.m.X = static_cast<const uint16_t *>(X);
    args.m.partial = ctx->partial;
    args.m.ldx = ldx;
    args.m.n_tokens = n_tokens;
    args.m.n = n;
    args.m.n_pad = ctx->n_pad;
    args.m.rows_per_slab = rows_per_slab;
    args.m.strips = ctx->strips;
    args.m.first_fresh_slab = ctx->slabs_valid;
    args.m.first_cta = 0;
    const int x_ok = x_complete ? 1 : 0;
    cudaError_t launch_err = cudaSuccess;
#define SP_LAUNCH(B, V) \
    launch_err = cudaLaunchKernelEx(&pdl.cfg, calib_accumulate_kernel<B, V, CalibOne>, args, x_ok)
    if (bf16) {
        if (vec) SP_LAUNCH(true, true); else SP_LAUNCH(true, false);
    } else {
        if (vec) SP_LAUNCH(false, true); else SP_LAUNCH(false, false);
    }
#undef SP_LAUNCH
    if (launch_err != cudaSuccess) return cuda_fail(launch_err);
    sp_status st = check_launch();
    if (st != SP_OK) return st;
    if (slabs > ctx->slabs_valid) ctx->slabs_valid = static_cast<int>(slabs);
    ctx->n_tokens += n_tokens;
    ctx->dirty = true;
    return SP_OK;
}

bool calib_multi_applies(const sp_ctx *ctx, const void *X, int64_t ldx, int64_t n_tokens) {
    return aligned16(X) && ldx % 8 == 0 && ctx->d_in % 8 == 0 && ldx < (int64_t(1) << 30) &&
           n_tokens < (int64_t(1) << 30);  // the table kernel computes with 32-bit sizes
}

sp_status launch_calib_accumulate_multi(sp_ctx *const *ctxs, const CalibItem *items, int count,
                                        sp_dtype dtype, cudaStream_t stream, bool x_complete) {
    if (count > kCalibMaxJobs) return SP_ERR_INVALID_ARG;
    int64_t total_strips = 0;
    for (int i = 0; i < count; ++i) total_strips += ctxs[i]->strips;
    CalibMany table{};
    table.count = count;
    int64_t ctas = 0;
    int64_t slabs_of[kCalibMaxJobs];
    for (int i = 0; i < count; ++i) {
        sp_ctx *c = ctxs[i];
        int64_t slabs, rows_per_slab;
        calib_partition(c, items[i].n_tokens, total_strips, slabs, rows_per_slab);
        slabs_of[i] = slabs;
        CalibMany::Matrix &j = table.job[i];
        j.X = static_cast<const uint16_t *>(items[i].X);
        j.partial = c->partial;
        j.ldx = static_cast<int>(items[i].ldx);  // calib_multi_applies: all below 2^31
        j.n_tokens = static_cast<int>(items[i].n_tokens);
        j.n = static_cast<int>(c->d_in);
        j.n_pad = static_cast<int>(c->n_pad);
        j.rows_per_slab = static_cast<int>(rows_per_slab);
        j.strips = c->strips;
        j.first_fresh_slab = c->slabs_valid;
        j.first_cta = static_cast<int>(ctas);
        ctas += slabs * c->strips;
    }
    PdlConfig pdl(dim3(static_cast<unsigned>(ctas)), dim3(kCalibThreads), stream);
    const int x_ok = x_complete ? 1 : 0;
    cudaError_t e =
        dtype == SP_BF16
            ? cudaLaunchKernelEx(&pdl.cfg, calib_accumulate_kernel<true, true, CalibMany>, table, x_ok)
            : cudaLaunchKernelEx(&pdl.cfg, calib_accumulate_kernel<false, true, CalibMany>, table, x_ok);
    if (e != cudaSuccess) return cuda_fail(e);
    sp_status st = check_launch();
    if (st != SP_OK) return st;
    for (int i = 0; i < count; ++i) {
        sp_ctx *c = ctxs[i];
        if (slabs_of[i] > c->slabs_valid) c->slabs_valid = static_cast<int>(slabs_of[i]);
        c->n_tokens += items[i].n_tokens;
        c->dirty = true;
    }
    return SP_OK;
}

// Finalises every context of the list that has batches pending, in one launch when there are
// several (a context may appear more than once).
sp_status launch_finalize_pending(sp_ctx *const *ctxs, int count, cudaStream_t stream) {
    sp_ctx *todo[kFinalMaxJobs];
    int n_todo = 0;
    for (int i = 0; i < count; ++i) {
        sp_ctx *c = ctxs[i];
        if (!c->dirty) continue;
        bool seen = false;
        for (int k = 0; k < n_todo; ++k) seen = seen || todo[k] == c;
        if (seen) continue;
        if (n_todo == kFinalMaxJobs) {  // more distinct contexts than one table holds
            sp_status st = launch_finalize(c, stream);
            if (st != SP_OK) return st;
            continue;
        }
        todo[n_todo++] = c;
    }
    if (n_todo == 0) return SP_OK;
    if (n_todo == 1) return launch_finalize(todo[0], stream);
    FinalJobTable table{};
    table.count = n_todo;
    int ctas = 0;
    for (int i = 0; i < n_todo; ++i) {
        sp_ctx *c = todo[i];
        FinalJob &j = table.job[i];
        j.partial = c->partial;
        j.colsq = c->colsq;
        j.strip_sum = c->strip_sum;
        j.factor = c->factor;
        j.factor_pairs = c->factor_pairs;
        j.scalars = c->scalars;
        j.n = c->d_in;
        j.n_pad = c->n_pad;
        j.slabs_valid = c->slabs_valid;
        j.strips = c->strips;
        j.first_cta = ctas;
        ctas += c->strips;
    }
    PdlConfig pdl(dim3(static_cast<unsigned>(ctas)), dim3(kFinalThreads), stream);
    cudaError_t e = cudaLaunchKernelEx(&pdl.cfg, finalize_multi_kernel, table);
    if (e != cudaSuccess) return cuda_fail(e);
    sp_status st = check_launch();
    if (st != SP_OK) return st;
    for (int i = 0; i < n_todo; ++i) todo[i]->dirty = false;
    return SP_OK;
}

sp_status launch_finalize(sp_ctx *ctx, cudaStream_t stream) {
    PdlConfig pdl(dim3(ctx->strips), dim3(kFinalThreads), stream);
    const double *partial = ctx->partial;
    cudaError_t e = cudaLaunchKernelEx(&pdl.cfg, finalize_kernel, partial, ctx->slabs_valid,
                                       ctx->d_in, ctx->n_pad, ctx->strips, ctx->colsq,
                                       ctx->strip_sum, ctx->factor, ctx->factor_pairs,
                                       ctx->scalars);
    if (e != cudaSuccess) return cuda_fail(e);
    sp_status st = check_launch();
    if (st == SP_OK) ctx->dirty = false;
    return st;
}

// ---------------------------------------------------------------------------------------------
// Allocation-free one-shot statistics.
//
// Same two kernels as above, but every byte of working memory comes from one file-scope device
// array instead of a context obtained with cudaMalloc.  The array is part of the library image:
// each GPU that loads the library carries it (about 4.4 MB) until the process exits.  All calls
// on a device share it, so two calls whose work overlaps on the GPU would overwrite each other's
// partial sums; nothing in it needs to survive from one call to the next.
constexpr int64_t kStaticMaxDin = 16384;
constexpr int64_t kStaticPartialDoubles = int64_t(1) << 19;  // 4 MiB of partial sums

struct StaticScratch {
    double partial[kStaticPartialDoubles];
    double colsq[kStaticMaxDin];
    double strip_sum[kStaticMaxDin / kStripChannels];
    float factor[kStaticMaxDin];
    DeviceScalars scalars;
};

static __device__ __align__(256) unsigned char g_static_scratch[sizeof(StaticScratch)];

constexpr int kMaxDevices = 64;
struct StaticDeviceState {
    StaticScratch *scratch = nullptr;  // device address of g_static_scratch on this device
    int sm_count = 0;
    int blocks_per_sm = 0;
};
static StaticDeviceState g_static_state[kMaxDevices];
static std::mutex g_static_mutex;

// In host code `g_static_scratch` is only a handle for the runtime, not an address the GPU can
// use; the address on the current device has to be asked for.  Done once per device.
static sp_status static_setup(int device, StaticDeviceState **out) {
    if (device < 0 || device >= kMaxDevices) return SP_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lock(g_static_mutex);
    StaticDeviceState &st = g_static_state[device];
    if (st.scratch == nullptr) {
        void *ptr = nullptr;
        cudaError_t e = cudaGetSymbolAddress(&ptr, g_static_scratch);
        if (e != cudaSuccess) return cuda_fail(e);
        int sms = 0;
        e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device);
        if (e != cudaSuccess) return cuda_fail(e);
        st.sm_count = sms;
        st.blocks_per_sm = calib_query_blocks_per_sm();
        st.scratch = static_cast<StaticScratch *>(ptr);
    }
    *out = &st;
    return SP_OK;
}

int64_t calib_static_max_d_in() { return kStaticMaxDin; }

sp_status launch_calib_stats_static(int device, const void *X, sp_dtype dtype, int64_t n_tokens,
                                    int64_t d_in, int64_t ldx, double *colsq_out,
                                    float *factor_out, double *S_out, cudaStream_t stream) {
    StaticDeviceState *st = nullptr;
    sp_status status = static_setup(device, &st);
    if (status != SP_OK) return status;
    StaticScratch *sc = st->scratch;

    const int64_t n = d_in;
    const int64_t n_pad = (n + kStripChannels - 1) / kStripChannels * kStripChannels;
    const int strips = static_cast<int>(n_pad / kStripChannels);
    // same slab rule as the context path, additionally bounded by the fixed partial-sum area
    int64_t slabs = static_cast<int64_t>(st->sm_count) * st->blocks_per_sm / strips;
    if (slabs < 1) slabs = 1;
    if (slabs > kMaxSlabs) slabs = kMaxSlabs;
    if (slabs > kStaticPartialDoubles / n_pad) slabs = kStaticPartialDoubles / n_pad;
    const int64_t min_rows = kCalibWarps * kRowsInFlight;
    const int64_t max_slabs_by_rows = (n_tokens + min_rows - 1) / min_rows;
    if (slabs > max_slabs_by_rows) slabs = max_slabs_by_rows;
    int64_t rows_per_slab = (n_tokens + slabs - 1) / slabs;
    rows_per_slab = (rows_per_slab + kCalibWarps - 1) / kCalibWarps * kCalibWarps;
    slabs = (n_tokens + rows_per_slab - 1) / rows_per_slab;

    // The arrival counter of the finalisation kernel must start at zero whatever an earlier
    // call left behind; every other field is written before it is read.
    cudaError_t e = cudaMemsetAsync(&sc->scalars, 0, sizeof(DeviceScalars), stream);
    if (e != cudaSuccess) return cuda_fail(e);

    const bool vec = aligned16(X) && (ldx % 8 == 0) && (n % 8 == 0);
    const bool bf16 = dtype == SP_BF16;
    dim3 grid(static_cast<unsigned>(strips), static_cast<unsigned>(slabs));
    CalibOne args{};
    args.m.X = static_cast<const uint16_t *>(X);
    args.m.partial = sc->partial;
    args.m.ldx = ldx;
    args.m.n_tokens = n_tokens;
    args.m.n = n;
    args.m.n_pad = n_pad;
    args.m.rows_per_slab = rows_per_slab;
    args.m.strips = strips;
    args.m.first_fresh_slab = 0;
    args.m.first_cta = 0;
#define SP_LAUNCH(B, V) \
    calib_accumulate_kernel<B, V, CalibOne><<<grid, kCalibThreads, 0, stream>>>(args, /*x_complete=*/0)
    if (bf16) {
        if (vec) SP_LAUNCH(true, true); else SP_LAUNCH(true, false);
    } else {
        if (vec) SP_LAUNCH(false, true); else SP_LAUNCH(false, false);
    }
#undef SP_LAUNCH
    status = check_launch();
    if (status != SP_OK) return status;
    finalize_kernel<<<strips, kFinalThreads, 0, stream>>>(
        sc->partial, static_cast<int>(slabs), n, n_pad, strips, sc->colsq, sc->strip_sum,
        sc->factor, /*factor_pairs=*/nullptr, &sc->scalars);
    status = check_launch();
    if (status != SP_OK) return status;

    if (colsq_out != nullptr) {
        e = cudaMemcpyAsync(colsq_out, sc->colsq, sizeof(double) * n, cudaMemcpyDeviceToDevice, stream);
        if (e != cudaSuccess) return cuda_fail(e);
    }
    if (factor_out != nullptr) {
        e = cudaMemcpyAsync(factor_out, sc->factor, sizeof(float) * n, cudaMemcpyDeviceToDevice, stream);
        if (e != cudaSuccess) return cuda_fail(e);
    }
    if (S_out != nullptr) {
        e = cudaMemcpyAsync(S_out, &sc->scalars.S, sizeof(double), cudaMemcpyDeviceToDevice, stream);
        if (e != cudaSuccess) return cuda_fail(e);
    }
    return SP_OK;
}

}  // namespace sp
