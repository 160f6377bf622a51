// Pieces shared by the EWMA selection kernels (Algorithm 1 with S frozen: the two recurrences
// of Table 2 evaluated as affine scans): packed helpers, the lane scan, and the algebra of the
// paired chains.
//
// Scaled states E = est/alpha and D' = dev/(beta a), a = 1-alpha, b = 1-beta:
//     q_i  = L_i - alpha E_{i-1}                  (score minus the estimate it is tested against)
//     E_i  = a E_{i-1} + L_i
//     est_i - L_i = -a q_i   =>   D'_i = b D'_{i-1} + |q_i|
//     prune  <=>  q_i + kappa D'_{i-1} < 0 ,  kappa = la beta a .
// A lane owns 16 consecutive weights (two 16-byte chunks); each chunk is two chains of 4
// (elements 0-3 and 4-7) that advance together in the two halves of packed binary32 pairs.
#pragma once

#include "sp_device.cuh"
#include "sp_internal.h"

namespace sp {

// Running packed maximum of |w| (two 16-bit floats per word); a NaN weight is dropped.
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

// Keeps a kernel parameter in a register for the whole kernel (the compiler would otherwise be
// free to re-read it from the constant bank at every use).
__device__ __forceinline__ float pinned(float v) {
    float r;
    asm volatile("mov.f32 %0, %1;" : "=f"(r) : "f"(v));
    return r;
}

// One step of the inclusive lane scan: x += m * (x of the lane `delta` below), for lanes that
// have such a lane.  The shuffle's own predicate output says whether the source lane exists, so
// no comparison on the lane index is needed.
template <int DELTA>
__device__ __forceinline__ float lane_scan_step(float x, float m) {
    float r;
    asm volatile(
        "{\n\t"
        ".reg .pred p;\n\t"
        ".reg .f32 y;\n\t"
        "shfl.sync.up.b32 y|p, %1, %2, 0, 0xffffffff;\n\t"
        "mov.f32 %0, %1;\n\t"
        "@p fma.rn.f32 %0, %3, y, %1;\n\t"
        "}"
        : "=&f"(r)
        : "f"(x), "n"(DELTA), "f"(m));
    return r;
}
__device__ __forceinline__ float lane_affine_scan_pred(float x, const float (&step)[5]) {
    x = lane_scan_step<1>(x, step[0]);
    x = lane_scan_step<2>(x, step[1]);
    x = lane_scan_step<4>(x, step[2]);
    x = lane_scan_step<8>(x, step[3]);
    x = lane_scan_step<16>(x, step[4]);
    return x;
}

template <bool BF16>
__device__ __forceinline__ float unpack_lo(uint32_t u) {
    if constexpr (BF16) return __uint_as_float(u << 16);
    else return __half2float(__ushort_as_half(static_cast<unsigned short>(u & 0xffffu)));
}
template <bool BF16>
__device__ __forceinline__ float unpack_hi(uint32_t u) {
    if constexpr (BF16) return __uint_as_float(u & 0xffff0000u);
    else return __half2float(__ushort_as_half(static_cast<unsigned short>(u >> 16)));
}

// The state before column 0 is est = L_0 (Table 2), i.e. E = L_0 / alpha, lowered by one ulp
// when rounding would make  L_0 - alpha E  negative, so that column 0 is never pruned.
__device__ __forceinline__ float ewma_start_state(float L0, float alpha) {
    float e = L0 / alpha;
    if (fmaf(-alpha, e, L0) < 0.0f) e = __uint_as_float(__float_as_uint(e) - 1u);
    return e;
}

// Scores of one 16-byte chunk in pair order, (L_j, L_{j+4}) for j = 0..3, from the packed
// weights and the chunk's two factor quads (columns 0,4,1,5 | 2,6,3,7).
template <bool BF16>
__device__ __forceinline__ void chunk_scores(const uint32_t (&p)[4], const float4 &c01,
                                             const float4 &c23, float2 (&L2)[4]) {
    float2 w2;
    w2 = make_float2(unpack_lo<BF16>(p[0]), unpack_lo<BF16>(p[2]));
    L2[0] = __fmul2_rn(__fmul2_rn(w2, w2), make_float2(c01.x, c01.y));
    w2 = make_float2(unpack_hi<BF16>(p[0]), unpack_hi<BF16>(p[2]));
    L2[1] = __fmul2_rn(__fmul2_rn(w2, w2), make_float2(c01.z, c01.w));
    w2 = make_float2(unpack_lo<BF16>(p[1]), unpack_lo<BF16>(p[3]));
    L2[2] = __fmul2_rn(__fmul2_rn(w2, w2), make_float2(c23.x, c23.y));
    w2 = make_float2(unpack_hi<BF16>(p[1]), unpack_hi<BF16>(p[3]));
    L2[3] = __fmul2_rn(__fmul2_rn(w2, w2), make_float2(c23.z, c23.w));
}

// Prune flags of one chunk from its eight decision values (pair order): the sign bit of a
// decision value is the prune flag (a NaN is the positive canonical NaN: kept, as
// "L < threshold" is false).  pm[k]: half-word masks of the packed weight pair k (0xffff where
// pruned); returns the 8 keep bits.
__device__ __forceinline__ uint32_t chunk_decide(const float2 (&diff2)[4], uint32_t (&pm)[4]) {
    pm[0] = prmt(__float_as_uint(diff2[0].x), __float_as_uint(diff2[1].x), 0xffbbu);
    pm[1] = prmt(__float_as_uint(diff2[2].x), __float_as_uint(diff2[3].x), 0xffbbu);
    pm[2] = prmt(__float_as_uint(diff2[0].y), __float_as_uint(diff2[1].y), 0xffbbu);
    pm[3] = prmt(__float_as_uint(diff2[2].y), __float_as_uint(diff2[3].y), 0xffbbu);
    return ~halfmasks_to_bits(pm) & 0xffu;
}

// Algorithm 1 exactly as printed along one row from column i_begin (a multiple of 32) on, by
// one thread, binary32 with one rounding per operation; est / dev are the state before that
// column (ignored for column 0, where est starts at L_0).  subtract_x2: the other reading of
// Table 2's row S, a pruned weight takes its channel's x_i^2 (not w_i^2) out of S.  Element-wise access with bounds
// checks.  While S still has its initial value the per-channel factor computed at finalisation
// is used: it was formed by the same three operations from the same S, so the result is
// bit-identical to recomputing it; once a pruned weight has changed S the factor is recomputed
// for every element.  S0 is the initial S (the one the finalised factors belong to), S_begin
// the value S has at column i_begin when weights before it have been pruned already.  Returns
// the number of kept weights.
template <bool BF16>
__device__ __forceinline__ unsigned long long literal_walk(
    const uint16_t *__restrict__ wrow, uint16_t *__restrict__ orow, uint32_t *__restrict__ mrow,
    int64_t n, int64_t i_begin, float est, float dev, const double *__restrict__ colsq,
    const float *__restrict__ factor, float S0, float alpha, float beta, float la,
    bool subtract_x2 = false, float S_begin = -1.0f) {
    const float one_minus_alpha = __fsub_rn(1.0f, alpha);
    const float one_minus_beta = __fsub_rn(1.0f, beta);
    float S = S_begin >= 0.0f ? S_begin : S0;  // S_begin: S has already moved before i_begin
    uint32_t word = 0;
    unsigned long long kept = 0;
    // two chunks are kept in flight ahead of the one being evaluated
    uint32_t ahead[2][4];
    load8<false, true>(wrow, i_begin, n, ahead[0]);
    load8<false, true>(wrow, i_begin + 8, n, ahead[1]);
    for (int64_t i0 = i_begin; i0 < n; i0 += 8) {
        uint32_t p[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            p[k] = ahead[0][k];
            ahead[0][k] = ahead[1][k];
        }
        load8<false, true>(wrow, i0 + 16, n, ahead[1]);
        float w[8];
        unpack8<BF16>(p, w);
        uint32_t keep8 = 0;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const int64_t i = i0 + j;
            if (i < n) {
                float c;
                if (S == S0) {
                    c = __ldg(factor + i);
                } else {
                    const float u = __fdiv_rn(static_cast<float>(colsq[i]), S);
                    c = __fdiv_rn(0.5f, __fsub_rn(1.0f, u));
                }
                const float w2 = __fmul_rn(w[j], w[j]);
                const float L = __fmul_rn(w2, c);
                if (i == 0) est = L;
                const float thr = __fsub_rn(est, __fmul_rn(la, dev));
                if (L < thr) {
                    S = __fsub_rn(S, subtract_x2 ? static_cast<float>(colsq[i]) : w2);
                } else {
                    keep8 |= 1u << j;
                }
                est = __fadd_rn(__fmul_rn(one_minus_alpha, est), __fmul_rn(alpha, L));
                dev = __fadd_rn(__fmul_rn(one_minus_beta, dev),
                                __fmul_rn(beta, fabsf(__fsub_rn(est, L))));
            }
        }
        kept += __popc(keep8);
        if (orow != nullptr) {
            zero_pruned(p, keep8);
            store8<false>(orow, i0, n, p);
        }
        word |= keep8 << (i0 & 31);
        if ((i0 & 31) == 24 || i0 + 8 >= n) {
            if (mrow != nullptr && SP_IN_RANGE(i0 >> 5, (n + 31) / 32, kDbgWalkMask)) mrow[i0 >> 5] = word;
            word = 0;
        }
    }
    return kept;
}

}  // namespace sp
