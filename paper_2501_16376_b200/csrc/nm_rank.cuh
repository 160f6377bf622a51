// Rank counting for N:M selection, shared by the kernels that select N of M.
#pragma once

#include "sp_device.cuh"

namespace sp {

// if (a > b) r += MOVE, as a compare and one predicated add.
template <uint32_t MOVE>
__device__ __forceinline__ void add_if_greater(uint32_t &r, uint32_t a, uint32_t b) {
    asm("{\n\t.reg .pred p;\n\tsetp.gt.u32 p, %1, %2;\n\t@p add.u32 %0, %0, %3;\n\t}"
        : "+r"(r)
        : "r"(a), "r"(b), "n"(MOVE));
}

// if (a > b) { ra += 1 << (8*I); rb -= 1 << (8*J); }
template <int I, int J>
__device__ __forceinline__ void move_across(uint32_t &ra, uint32_t &rb, uint32_t a, uint32_t b) {
    asm("{\n\t.reg .pred p;\n\tsetp.gt.u32 p, %2, %3;\n\t@p add.u32 %0, %0, %4;\n\t"
        "@p sub.u32 %1, %1, %5;\n\t}"
        : "+r"(ra), "+r"(rb)
        : "r"(a), "r"(b), "n"(1u << (8 * I)), "n"(1u << (8 * J)));
}

template <int I, int J>
__device__ __forceinline__ void rank_pair(uint32_t &r, const uint32_t *key) {
    add_if_greater<(1u << (8 * I)) - (1u << (8 * J))>(r, key[I], key[J]);
}

// Ranks of one lane's 8 scores, one byte per element (elements 0..3 in ra, 4..7 in rb).
// A byte holds  bias + (number of elements of the group that order before this element)  with
// bias = 0x80 - (M - N), so its top bit is set exactly when the element is kept.  For a pair
// i < j the constant part counts "i orders before j"; when key_i > key_j the count moves from
// j's byte to i's byte.  No byte can overflow or borrow: the counts stay within 0..M-1.
template <int M>
__device__ __forceinline__ void nm_rank_bytes(const uint32_t (&key)[8], uint32_t bias_lo,
                                              uint32_t bias_hi, uint32_t &ra, uint32_t &rb) {
    ra = bias_lo;  // bias + 0x03020100: byte j receives one count per i < j of its group
    rb = bias_hi;  // same for M == 4; bias + 0x07060504 for M == 8
    rank_pair<0, 1>(ra, key); rank_pair<0, 2>(ra, key); rank_pair<0, 3>(ra, key);
    rank_pair<1, 2>(ra, key); rank_pair<1, 3>(ra, key); rank_pair<2, 3>(ra, key);
    rank_pair<0, 1>(rb, key + 4); rank_pair<0, 2>(rb, key + 4); rank_pair<0, 3>(rb, key + 4);
    rank_pair<1, 2>(rb, key + 4); rank_pair<1, 3>(rb, key + 4); rank_pair<2, 3>(rb, key + 4);
    if constexpr (M == 8) {
#define SP_ROW(I)                                                                             \
    move_across<I, 0>(ra, rb, key[I], key[4]); move_across<I, 1>(ra, rb, key[I], key[5]);      \
    move_across<I, 2>(ra, rb, key[I], key[6]); move_across<I, 3>(ra, rb, key[I], key[7]);
        SP_ROW(0) SP_ROW(1) SP_ROW(2) SP_ROW(3)
#undef SP_ROW
    }
}

}  // namespace sp
