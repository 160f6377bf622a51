// 2:4 selection (Section 3.3) emitted directly in a compressed form: the two kept weights of
// every group of four, packed, plus a 4-bit index record per group.  Section 3.3 notes that
// sparse tensor-core hardware consumes a 2:4 result as it is, with no conversion step; this
// kernel writes values and indices in the same pass that selects them, so no dense pruned
// matrix has to be written and re-read.  The layout is this library's own, documented in the
// header: values [rows, d_in/2] (kept weights in column order), metadata [rows, ceil(d_in/32)]
// uint32 with bits 4g..4g+3 of word k describing group 8k+g as  idx0 | idx1 << 2  (idx0 < idx1,
// the positions of the two kept weights inside the group).
//
// Work layout and selection are those of select_nm.cu: a warp owns a 256-column strip and a
// slab of rows, a lane owns 8 columns (two groups), the factors of its columns stay in registers.
// select_24_compressed_stream_kernel is the path for aligned rows, select_24_compressed_kernel
// (element-wise access) the one for any other layout.
#include "nm_rank.cuh"
#include "sp_device.cuh"
#include "sp_internal.h"

namespace sp {

constexpr int kNmcThreads = 128;
constexpr int kNmcWarps = kNmcThreads / 32;
constexpr int kNmcRowsInFlight = 4;

// keep nibble (exactly two bits set) -> idx0 | idx1 << 2, 4 bits per entry, entry k at bits 4k.
// 0011->(0,1)=0x4  0101->(0,2)=0x8  0110->(1,2)=0x9  1001->(0,3)=0xc  1010->(1,3)=0xd  1100->(2,3)=0xe
constexpr unsigned long long kMetaOfNibble =
    (0x4ull << (4 * 0x3)) | (0x8ull << (4 * 0x5)) | (0x9ull << (4 * 0x6)) | (0xcull << (4 * 0x9)) |
    (0xdull << (4 * 0xa)) | (0xeull << (4 * 0xc));

// The two kept 16-bit weights of a group held in (lo: elements 0,1; hi: elements 2,3), packed.
__device__ __forceinline__ uint32_t pick_pair(uint32_t lo, uint32_t hi, uint32_t meta) {
    const uint32_t i0 = meta & 3u, i1 = meta >> 2;
    // element i is bytes 2i, 2i+1 of the byte pool {lo, hi}
    const uint32_t sel = (i0 + (i1 << 8)) * 0x22u + 0x1010u;
    return prmt(lo, hi, sel);
}

template <bool BF16>
__global__ void __launch_bounds__(kNmcThreads, 8)
select_24_compressed_kernel(const uint16_t *__restrict__ W, int ldw, int n_rows, int64_t n,
                            int rows_per_warp, const float *__restrict__ factor,
                            uint16_t *__restrict__ values, int ldv, uint32_t *__restrict__ meta,
                            int meta_words) {
    pdl_launch_dependents();
    pdl_wait();  // the per-channel factors come from an earlier kernel of the stream
    const int lane = threadIdx.x & 31;
    const int64_t col = static_cast<int64_t>(blockIdx.x) * kStripChannels + lane * 8;
    const int slab = blockIdx.y * kNmcWarps + (threadIdx.x >> 5);
    const int64_t row_begin64 = static_cast<int64_t>(slab) * rows_per_warp;
    if (row_begin64 >= n_rows) return;  // warp-uniform
    const int row_begin = static_cast<int>(row_begin64);
    const int rows = min(n_rows - row_begin, rows_per_warp);

    float c[8];
    load_factor8(factor, col, c);  // zero past d_in
    const int64_t left = n - col;  // a multiple of 4
    const uint32_t bias = static_cast<uint32_t>(0x80 - 2) * 0x01010101u + 0x03020100u;
    const bool store_word = (lane & 3) == 0 && left > 0;

    const uint16_t *wp = W + static_cast<int64_t>(row_begin) * ldw;
    uint16_t *vp = values + static_cast<int64_t>(row_begin) * ldv + (col >> 1);
    uint32_t *mp = meta + static_cast<int64_t>(row_begin) * meta_words + (col >> 5);

    for (int r0 = 0; r0 < rows; r0 += kNmcRowsInFlight) {
        uint32_t p[kNmcRowsInFlight][4];
#pragma unroll
        for (int u = 0; u < kNmcRowsInFlight; ++u) {
            if (r0 + u < rows) {
                load8<false, true>(wp + static_cast<int64_t>(u) * ldw, col, n, p[u]);
            } else {
                p[u][0] = p[u][1] = p[u][2] = p[u][3] = 0u;
            }
        }
#pragma unroll
        for (int u = 0; u < kNmcRowsInFlight; ++u) {
            if (r0 + u >= rows) break;  // warp-uniform
            float w[8];
            unpack8<BF16>(p[u], w);
            uint32_t key[8];
#pragma unroll
            for (int j = 0; j < 8; ++j)
                key[j] = __float_as_uint(__fmul_rn(__fmul_rn(w[j], w[j]), c[j]));
            uint32_t ra, rb;
            nm_rank_bytes<4>(key, bias, bias, ra, rb);
            uint32_t m[4];
            m[0] = prmt(ra, 0u, 0x9988u);
            m[1] = prmt(ra, 0u, 0xbbaau);
            m[2] = prmt(rb, 0u, 0x9988u);
            m[3] = prmt(rb, 0u, 0xbbaau);
            const uint32_t keep8 = halfmasks_to_bits(m);
            const uint32_t meta0 = static_cast<uint32_t>(kMetaOfNibble >> (4 * (keep8 & 0xfu))) & 0xfu;
            uint32_t meta1 = static_cast<uint32_t>(kMetaOfNibble >> (4 * (keep8 >> 4))) & 0xfu;
            const uint32_t v0 = pick_pair(p[u][0], p[u][1], meta0);
            const uint32_t v1 = pick_pair(p[u][2], p[u][3], meta1);
            if (left < 8) meta1 = 0u;  // the lane's second group lies past d_in
            uint16_t *vrow = vp + static_cast<int64_t>(u) * ldv;
            if (left >= 8) {
                vrow[0] = static_cast<uint16_t>(v0 & 0xffffu);
                vrow[1] = static_cast<uint16_t>(v0 >> 16);
                vrow[2] = static_cast<uint16_t>(v1 & 0xffffu);
                vrow[3] = static_cast<uint16_t>(v1 >> 16);
            } else if (left > 0) {
                vrow[0] = static_cast<uint16_t>(v0 & 0xffffu);
                vrow[1] = static_cast<uint16_t>(v0 >> 16);
            }
            const uint32_t word = gather_mask_word(left > 0 ? (meta0 | (meta1 << 4)) : 0u, lane);
            if (store_word) mp[static_cast<int64_t>(u) * meta_words] = word;
        }
        wp += static_cast<int64_t>(kNmcRowsInFlight) * ldw;
        vp += static_cast<int64_t>(kNmcRowsInFlight) * ldv;
        mp += static_cast<int64_t>(kNmcRowsInFlight) * meta_words;
    }
}

// Streaming kernel for rows that allow 16-byte reads and 8-byte value writes (the fast path):
// the same selection and records, with the rows run through a four-slot per-lane ring of
// asynchronous copies (four rows per trip: static slots), scores formed two at a time in packed
// binary32 pairs, and the lane's two 4-bit records stored as one byte (byte k of a little-endian
// metadata word describes groups 2k and 2k+1) instead of assembling words across lanes.
// FULL: d_in is a multiple of 256, no column guards.
template <bool BF16, bool FULL>
__global__ void __launch_bounds__(kNmcThreads, 8)
select_24_compressed_stream_kernel(const uint16_t *__restrict__ W, int ldw, int n_rows, int n,
                                   int rows_per_warp, const float *__restrict__ factor,
                                   uint16_t *__restrict__ values, int ldv,
                                   uint32_t *__restrict__ meta, int meta_words) {
    pdl_launch_dependents();
    pdl_wait();  // the per-channel factors come from an earlier kernel of the stream
    const int lane = threadIdx.x & 31;
    const int col = blockIdx.x * kStripChannels + lane * 8;
    const int slab = blockIdx.y * kNmcWarps + (threadIdx.x >> 5);
    const int64_t row_begin64 = static_cast<int64_t>(slab) * rows_per_warp;
    if (row_begin64 >= n_rows) return;  // warp-uniform
    const int row_begin = static_cast<int>(row_begin64);
    const int rows = min(n_rows - row_begin, rows_per_warp);
    const bool in_row = FULL || col < n;  // d_in % 8 == 0: a chunk is inside or outside as a whole

    float2 cp[4];  // factors of columns (0,1) (2,3) (4,5) (6,7) of the chunk, zero past d_in
    {
        float c[8];
        load_factor8(factor, col, c);
#pragma unroll
        for (int k = 0; k < 4; ++k) cp[k] = make_float2(c[2 * k], c[2 * k + 1]);
    }
    const uint32_t bias = static_cast<uint32_t>(0x80 - 2) * 0x01010101u + 0x03020100u;
    const uint16_t *src = W + static_cast<int64_t>(row_begin) * ldw + (in_row ? col : 0);
    uint16_t *vdst = values + static_cast<int64_t>(row_begin) * ldv + (in_row ? col >> 1 : 0);
    const int meta_pitch = meta_words * 4;  // bytes per metadata row
    const bool in_meta = FULL || (col >> 3) < meta_pitch;
    uint8_t *mdst = reinterpret_cast<uint8_t *>(meta + static_cast<int64_t>(row_begin) * meta_words) +
                    (in_meta ? col >> 3 : 0);

    constexpr int kStages = 4;
    __shared__ __align__(16) uint4 ring[kNmcWarps * kStages * 32];
    uint4 *my_ring = ring + (threadIdx.x >> 5) * kStages * 32 + lane;
    auto issue = [&](int rr, int slot) {
        if (rr < rows && in_row)
            cp_async16(my_ring + slot * 32, src + static_cast<int64_t>(rr) * ldw, 16);
        cp_async_commit();
    };
#pragma unroll
    for (int rr = 0; rr < kStages - 1; ++rr) issue(rr, rr);

    auto process = [&](int rr, int slot) {
        issue(rr + kStages - 1, (slot + kStages - 1) & (kStages - 1));
        cp_async_wait<kStages - 1>();
        uint4 v = make_uint4(0u, 0u, 0u, 0u);
        if (in_row) v = my_ring[slot * 32];
        const uint32_t p[4] = {v.x, v.y, v.z, v.w};
        uint32_t key[8];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const float2 w2 = unpack2<BF16>(p[k]);
            const float2 L2 = __fmul2_rn(__fmul2_rn(w2, w2), cp[k]);
            key[2 * k] = __float_as_uint(L2.x);
            key[2 * k + 1] = __float_as_uint(L2.y);
        }
        uint32_t ra, rb;
        nm_rank_bytes<4>(key, bias, bias, ra, rb);
        uint32_t m[4];
        m[0] = prmt(ra, 0u, 0x9988u);
        m[1] = prmt(ra, 0u, 0xbbaau);
        m[2] = prmt(rb, 0u, 0x9988u);
        m[3] = prmt(rb, 0u, 0xbbaau);
        const uint32_t keep8 = halfmasks_to_bits(m);
        const uint32_t meta0 = static_cast<uint32_t>(kMetaOfNibble >> (4 * (keep8 & 0xfu))) & 0xfu;
        const uint32_t meta1 = static_cast<uint32_t>(kMetaOfNibble >> (4 * (keep8 >> 4))) & 0xfu;
        if (in_row)
            *reinterpret_cast<uint2 *>(vdst + static_cast<int64_t>(rr) * ldv) =
                make_uint2(pick_pair(p[0], p[1], meta0), pick_pair(p[2], p[3], meta1));
        if (in_meta)
            mdst[static_cast<int64_t>(rr) * meta_pitch] =
                static_cast<uint8_t>(in_row ? meta0 | (meta1 << 4) : 0u);
    };
    int r0 = 0;
    for (; r0 + kStages <= rows; r0 += kStages) {  // four rows per trip: static ring slots
#pragma unroll
        for (int u = 0; u < kStages; ++u) process(r0 + u, u);
    }
    for (int rr = r0; rr < rows; ++rr) process(rr, rr & (kStages - 1));  // r0 % kStages == 0
}

sp_status launch_select_24_compressed(const sp_ctx *ctx, const void *W, sp_dtype dtype,
                                      int64_t n_rows, int64_t ldw, void *values, int64_t ldv,
                                      uint32_t *meta, cudaStream_t stream) {
    const int64_t n = ctx->d_in;
    if (n_rows == 0) return SP_OK;
    if (n_rows > 0x7fffffffLL || ldw > 0x7fffffffLL || ldv > 0x7fffffffLL) return SP_ERR_SHAPE;
    const int strips = ctx->strips;
    const int64_t target_warps = static_cast<int64_t>(ctx->sm_count) * 64;
    int64_t rows_per_warp = (n_rows * strips + target_warps - 1) / target_warps;
    rows_per_warp = (rows_per_warp + kNmcRowsInFlight - 1) / kNmcRowsInFlight * kNmcRowsInFlight;
    if (rows_per_warp < 2 * kNmcRowsInFlight) rows_per_warp = 2 * kNmcRowsInFlight;
    const int64_t max_grid_y = 65535;
    if ((n_rows + rows_per_warp * kNmcWarps - 1) / (rows_per_warp * kNmcWarps) > max_grid_y) {
        rows_per_warp = (n_rows + max_grid_y * kNmcWarps - 1) / (max_grid_y * kNmcWarps);
        rows_per_warp = (rows_per_warp + kNmcRowsInFlight - 1) / kNmcRowsInFlight * kNmcRowsInFlight;
    }
    const int64_t slabs = (n_rows + rows_per_warp - 1) / rows_per_warp;
    const dim3 grid(static_cast<unsigned>(strips),
                    static_cast<unsigned>((slabs + kNmcWarps - 1) / kNmcWarps));
    const bool vec = aligned16(W) && ldw % 8 == 0 && n % 8 == 0 &&
                     (reinterpret_cast<uintptr_t>(values) & 7u) == 0 && ldv % 4 == 0;
    PdlConfig pdl(grid, dim3(kNmcThreads), stream);
    const uint16_t *Wp = static_cast<const uint16_t *>(W);
    uint16_t *Vp = static_cast<uint16_t *>(values);
    const float *factor = ctx->factor;
    const int words = static_cast<int>((n + 31) / 32);
    const int rpw = static_cast<int>(rows_per_warp);
    cudaError_t e;
#define SP_LAUNCH(B)                                                                           \
    e = cudaLaunchKernelEx(&pdl.cfg, select_24_compressed_kernel<B>, Wp,                        \
                           static_cast<int>(ldw), static_cast<int>(n_rows), n, rpw, factor, Vp, \
                           static_cast<int>(ldv), meta, words)
#define SP_LAUNCH_ST(B, F)                                                                     \
    e = cudaLaunchKernelEx(&pdl.cfg, select_24_compressed_stream_kernel<B, F>, Wp,              \
                           static_cast<int>(ldw), static_cast<int>(n_rows),                     \
                           static_cast<int>(n), rpw, factor, Vp, static_cast<int>(ldv), meta,   \
                           words)
    const bool full = n % kStripChannels == 0;
    if (vec) {
        if (dtype == SP_BF16) {
            if (full) SP_LAUNCH_ST(true, true); else SP_LAUNCH_ST(true, false);
        } else {
            if (full) SP_LAUNCH_ST(false, true); else SP_LAUNCH_ST(false, false);
        }
    } else if (dtype == SP_BF16) {
        SP_LAUNCH(true);
    } else {
        SP_LAUNCH(false);
    }
#undef SP_LAUNCH_ST
#undef SP_LAUNCH
    if (e != cudaSuccess) return cuda_fail(e);
    return check_launch();
}

}  // namespace sp
