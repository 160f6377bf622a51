// Device-side helpers: 16-bit float decoding, 8-element vector access with ragged tails,
// mask-word assembly.  Every kernel of the library views a row as chunks of 8 consecutive
// elements (16 bytes) owned by one lane; a warp covers a 256-element tile.
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "sp_debug.cuh"

namespace sp {

constexpr unsigned kFullWarp = 0xffffffffu;

// Two packed 16-bit floats -> two fp32 values (exact).
template <bool BF16>
__device__ __forceinline__ float2 unpack2(uint32_t u) {
    if constexpr (BF16) {
        return make_float2(__uint_as_float(u << 16), __uint_as_float(u & 0xffff0000u));
    } else {
        __half2 h = *reinterpret_cast<__half2 *>(&u);
        return __half22float2(h);
    }
}

template <bool BF16>
__device__ __forceinline__ void unpack8(const uint32_t (&p)[4], float (&w)[8]) {
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        float2 f = unpack2<BF16>(p[k]);
        w[2 * k] = f.x;
        w[2 * k + 1] = f.y;
    }
}

// s0 += lo^2, s1 += hi^2 for the two 16-bit floats of a packed word, with the mixed-precision
// fused multiply-add of sm_100 (16-bit operands, binary32 addend and result): the square of a
// 16-bit float is exact in binary32 and the sum is rounded once, so the result is the one that
// converting the operand first and a binary32 fma would give, without the conversions.
template <bool BF16>
__device__ __forceinline__ void fma_square2(uint32_t p, float &s0, float &s1) {
    unsigned short lo, hi;
    asm("mov.b32 {%0, %1}, %2;" : "=h"(lo), "=h"(hi) : "r"(p));
    if constexpr (BF16) {
        asm("fma.rn.f32.bf16 %0, %1, %1, %0;" : "+f"(s0) : "h"(lo));
        asm("fma.rn.f32.bf16 %0, %1, %1, %0;" : "+f"(s1) : "h"(hi));
    } else {
        asm("fma.rn.f32.f16 %0, %1, %1, %0;" : "+f"(s0) : "h"(lo));
        asm("fma.rn.f32.f16 %0, %1, %1, %0;" : "+f"(s1) : "h"(hi));
    }
}

// Loads elements [col, col+8) of a row into four packed words; elements at or past n read
// as zero.  VEC: 16-byte access (requires 16-byte aligned row start, n % 8 == 0, col % 8 == 0).
// STREAM: the data is read once (bypass L1, evict-first behaviour).
template <bool VEC, bool STREAM>
__device__ __forceinline__ void load8(const uint16_t *__restrict__ row, int64_t col, int64_t n,
                                      uint32_t (&p)[4]) {
    if constexpr (VEC) {
        if (col < n) {
            const uint4 *src = reinterpret_cast<const uint4 *>(row + col);
            uint4 v = STREAM ? __ldcs(src) : __ldg(src);
            p[0] = v.x; p[1] = v.y; p[2] = v.z; p[3] = v.w;
        } else {
            p[0] = p[1] = p[2] = p[3] = 0u;
        }
    } else {
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            uint32_t lo = 0, hi = 0;
            if (col + 2 * k < n) lo = row[col + 2 * k];
            if (col + 2 * k + 1 < n) hi = row[col + 2 * k + 1];
            p[k] = lo | (hi << 16);
        }
    }
}

template <bool VEC>
__device__ __forceinline__ void store8(uint16_t *__restrict__ row, int64_t col, int64_t n,
                                       const uint32_t (&p)[4]) {
    if constexpr (VEC) {
        if (col < n) {
            uint4 v = make_uint4(p[0], p[1], p[2], p[3]);
            __stcs(reinterpret_cast<uint4 *>(row + col), v);
        }
    } else {
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            if (col + 2 * k < n) row[col + 2 * k] = static_cast<uint16_t>(p[k] & 0xffffu);
            if (col + 2 * k + 1 < n) row[col + 2 * k + 1] = static_cast<uint16_t>(p[k] >> 16);
        }
    }
}

// Eight per-channel factors for columns [col, col+8); the factor array is padded with zeros
// to a multiple of 256 entries, so the 16-byte loads never leave it.
__device__ __forceinline__ void load_factor8(const float *__restrict__ factor, int64_t col,
                                             float (&c)[8]) {
    const float4 *src = reinterpret_cast<const float4 *>(factor + col);
    float4 a = __ldg(src);
    float4 b = __ldg(src + 1);
    c[0] = a.x; c[1] = a.y; c[2] = a.z; c[3] = a.w;
    c[4] = b.x; c[5] = b.y; c[6] = b.z; c[7] = b.w;
}

// Zeroes the 16-bit halves of the packed words whose keep bit (bit j of `keep`, j = element
// index within the chunk) is clear.
__device__ __forceinline__ void zero_pruned(uint32_t (&p)[4], uint32_t keep) {
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        uint32_t m = ((keep >> (2 * k)) & 1u ? 0x0000ffffu : 0u) |
                     ((keep >> (2 * k + 1)) & 1u ? 0xffff0000u : 0u);
        p[k] &= m;
    }
}

// Programmatic dependent launch: let the next kernel of the stream be scheduled early / wait
// until every earlier kernel of the stream has completed and its writes are visible.  Both are
// no-ops for kernels launched without the attribute.
__device__ __forceinline__ void pdl_launch_dependents() {
    asm volatile("griddepcontrol.launch_dependents;");
}
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// Asynchronous 16-byte copy global -> shared (bypassing L1).  src_bytes < 16 zero-fills the
// rest; src_bytes == 0 reads nothing.
__device__ __forceinline__ void cp_async16(void *smem_dst, const void *gmem_src, int src_bytes) {
    const uint32_t dst = static_cast<uint32_t>(__cvta_generic_to_shared(smem_dst));
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(gmem_src),
                 "r"(src_bytes)
                 : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
    asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}

// mbarrier + bulk asynchronous copy (cp.async.bulk, the 1-D form of the TMA unit).
__device__ __forceinline__ uint32_t smem_addr(const void *p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_fence_init() {
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes)
                 : "memory");
}
// Bulk copy global -> shared of `bytes` (a multiple of 16; both addresses 16-byte aligned),
// completing on the mbarrier.  No multicast; the source is memory of this GPU.
__device__ __forceinline__ void bulk_load(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
        "l"(src), "r"(bytes), "r"(bar)
        : "memory");
}
// Waits for the phase with the given parity; gives up (false) after a bounded number of polls.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
    for (uint32_t spin = 0; spin < (1u << 22); ++spin) {
        uint32_t done;
        asm volatile(
            "{\n\t"
            ".reg .pred p;\n\t"
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t"
            "}"
            : "=r"(done)
            : "r"(bar), "r"(parity)
            : "memory");
        if (done) return true;
    }
    return false;
}

// prmt.b32 in its generic mode: result byte k is byte (sel nibble k & 7) of the pair {a, b};
// when bit 3 of the nibble is set the byte's sign bit is replicated over the whole byte.
__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel) {
    uint32_t d;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(sel));
    return d;
}

// Four half-word masks m[k] (each 16-bit half is 0xffff or 0, element 2k in the low half) ->
// the 8-bit pattern with bit e set where element e's half is 0xffff.  Uses the signed
// two-way dot product: a half of 0xffff is -1, and the weights are -(1 << e).
__device__ __forceinline__ uint32_t halfmasks_to_bits(const uint32_t (&m)[4]) {
    int acc = 0;
    acc = __dp2a_lo(static_cast<int>(m[0]), 0x0000feff, acc);  // weights -1, -2
    acc = __dp2a_lo(static_cast<int>(m[1]), 0x0000f8fc, acc);  // -4, -8
    acc = __dp2a_lo(static_cast<int>(m[2]), 0x0000e0f0, acc);  // -16, -32
    acc = __dp2a_lo(static_cast<int>(m[3]), 0x000080c0, acc);  // -64, -128
    return static_cast<uint32_t>(acc);
}

// Each lane holds the 8 keep bits of its chunk.  Returns, in lanes with (lane & 3) == 0, the
// 32-bit mask word covering the chunks of lanes lane .. lane+3.
__device__ __forceinline__ uint32_t gather_mask_word(uint32_t keep8, int lane) {
    uint32_t v = keep8 << (8 * (lane & 3));
    v |= __shfl_xor_sync(kFullWarp, v, 1);
    v |= __shfl_xor_sync(kFullWarp, v, 2);
    return v;
}

}  // namespace sp
