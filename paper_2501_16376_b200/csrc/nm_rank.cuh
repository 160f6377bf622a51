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

template <int I, int J>
__device__ __forceinline__ void rank_pair(uint32_t &r, const uint32_t *key) {
    add_if_greater<(1u << (8 * I)) - (1u << (8 * J))>(r, key[I], key[J]);
}

// M == 4: ranks of one lane's 8 scores (two groups), one byte per element (elements 0..3 in
// ra, 4..7 in rb).  A byte holds  bias + (number of elements of the group that order before
// this element)  with bias = 0x80 - (M - N), so its top bit is set exactly when the element is
// kept.  For a pair
// i < j the constant part counts "i orders before j"; when key_i > key_j the count moves from
// j's byte to i's byte.  No byte can overflow or borrow: the counts stay within 0..M-1.
template <int M>
__device__ __forceinline__ void nm_rank_bytes(const uint32_t (&key)[8], uint32_t bias_lo,
                                              uint32_t bias_hi, uint32_t &ra, uint32_t &rb) {
    ra = bias_lo;  // bias + 0x03020100: byte j receives one count per i < j of its group
    rb = bias_hi;  // the same constant: both registers hold one group of four
    rank_pair<0, 1>(ra, key); rank_pair<0, 2>(ra, key); rank_pair<0, 3>(ra, key);
    rank_pair<1, 2>(ra, key); rank_pair<1, 3>(ra, key); rank_pair<2, 3>(ra, key);
    rank_pair<0, 1>(rb, key + 4); rank_pair<0, 2>(rb, key + 4); rank_pair<0, 3>(rb, key + 4);
    rank_pair<1, 2>(rb, key + 4); rank_pair<1, 3>(rb, key + 4); rank_pair<2, 3>(rb, key + 4);
}

// M == 8 with all eight ranks in the nibbles of one register: nibble j holds
// bias + (number of elements that order before element j), bias = 8 - (M - N), so the nibble's
// top bit is the keep flag and every pair costs one compare and one predicated add.
// bias_nibbles = bias * 0x11111111 + 0x76543210 (nibble j starts with one count per i < j).
__device__ __forceinline__ uint32_t nm_rank_nibbles8(const uint32_t (&key)[8],
                                                     uint32_t bias_nibbles) {
    uint32_t r = bias_nibbles;
#define SP_PAIR(I, J) add_if_greater<(1u << (4 * I)) - (1u << (4 * J))>(r, key[I], key[J]);
    SP_PAIR(0, 1)
    SP_PAIR(0, 2)
    SP_PAIR(0, 3)
    SP_PAIR(0, 4)
    SP_PAIR(0, 5)
    SP_PAIR(0, 6)
    SP_PAIR(0, 7)
    SP_PAIR(1, 2)
    SP_PAIR(1, 3)
    SP_PAIR(1, 4)
    SP_PAIR(1, 5)
    SP_PAIR(1, 6)
    SP_PAIR(1, 7)
    SP_PAIR(2, 3)
    SP_PAIR(2, 4)
    SP_PAIR(2, 5)
    SP_PAIR(2, 6)
    SP_PAIR(2, 7)
    SP_PAIR(3, 4)
    SP_PAIR(3, 5)
    SP_PAIR(3, 6)
    SP_PAIR(3, 7)
    SP_PAIR(4, 5)
    SP_PAIR(4, 6)
    SP_PAIR(4, 7)
    SP_PAIR(5, 6)
    SP_PAIR(5, 7)
    SP_PAIR(6, 7)
#undef SP_PAIR
    return r;
}

// Half-word masks (element 2k in the low half of m[k]) from the nibble top bits of r: the odd
// elements' flags are byte sign bits of r, the even elements' those of r << 4.
__device__ __forceinline__ void masks_from_nibbles(uint32_t r, uint32_t (&m)[4]) {
    const uint32_t even = r << 4;
    m[0] = prmt(even, r, 0xcc88u);
    m[1] = prmt(even, r, 0xdd99u);
    m[2] = prmt(even, r, 0xeeaau);
    m[3] = prmt(even, r, 0xffbbu);
}

}  // namespace sp
