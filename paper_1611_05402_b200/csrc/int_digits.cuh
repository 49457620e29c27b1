// Fixed-point digits for the integer contractions of the SGD engines (uniform grids).
#pragma once

#include "common.cuh"

namespace zipml {

// ---- integer contraction (uniform grids) ---------------------------------------------------------
// Both phases contract small unsigned codes with an fp32 vector that is constant for many rows (w in
// phase A, the residuals in phase B).  That vector is turned, once per step, into fixed point:
// value ~ delta * W with |W| <= QMAX, and W into NS balanced base-128 digits in [-64, 63], each an
// int8.  Codes times digits are integer products (dp4a, or the int8 tensor-core MMA below), the digit sums are combined
// exactly in 64 bits, and the only rounding is the one quantization of the vector, 2^-27 of its
// largest entry with four digits.  (Three digits, 2^-20, are not enough: the error of w is the same
// for every row, survives the minibatch mean and is amplified where residuals are small against the
// dots; measured 1.3e-5 on the gradient of clustered 3-bit codes.)
template <int CB>
struct IntPath {
    static constexpr int NS = 4;
    static constexpr int QMAX = 133000000;                         // below 63 * (128^NS - 1) / 127
    static constexpr int NG = 8 / CB;                              // groups of four codes in a 32-bit word
};

// The four codes of group g of a word, one per byte: byte b holds feature b * NG + g of the word.
template <int CB>
__device__ __forceinline__ uint32_t group_bytes(uint32_t u, int g) {
    if constexpr (CB == 8) return u;
    else if constexpr (CB == 4) return (u >> (4 * g)) & 0x0F0F0F0Fu;
    else return (u >> (2 * g)) & 0x03030303u;
}

template <int NS>
__device__ __forceinline__ void balanced_digits(int W, int (&d)[NS]) {
#pragma unroll
    for (int s = 0; s < NS - 1; ++s) {
        d[s] = ((W + 64) & 127) - 64;
        W = (W - d[s]) >> 7;
    }
    d[NS - 1] = W;
}

__device__ __forceinline__ uint32_t pack_bytes(int b0, int b1, int b2, int b3) {
    return (uint32_t)(b0 & 255) | ((uint32_t)(b1 & 255) << 8) | ((uint32_t)(b2 & 255) << 16) | ((uint32_t)(b3 & 255) << 24);
}

// Digit words of four values: out.x/.y/.z/.w = digit 0..3 of (v0, v1, v2, v3), one value per byte.
template <int NS>
__device__ __forceinline__ uint4 digit_words(const float (&v)[4], float inv_delta) {
    int d[4][NS];
#pragma unroll
    for (int b = 0; b < 4; ++b) balanced_digits<NS>(__float2int_rn(v[b] * inv_delta), d[b]);
    uint4 o;
    o.x = pack_bytes(d[0][0], d[1][0], d[2][0], d[3][0]);
    o.y = pack_bytes(d[0][1], d[1][1], d[2][1], d[3][1]);
    o.z = pack_bytes(d[0][2], d[1][2], d[2][2], d[3][2]);
    o.w = (NS == 4) ? pack_bytes(d[0][NS - 1], d[1][NS - 1], d[2][NS - 1], d[3][NS - 1]) : 0u;
    return o;
}

template <int NS>
__device__ __forceinline__ long long combine_digits(const int (&acc)[NS]) {
    long long t = 0;
#pragma unroll
    for (int s = 0; s < NS; ++s) t += (long long)acc[s] << (7 * s);
    return t;
}

// ---- int8 tensor-core contraction ------------------------------------------------------------------
// D += A (16 x 32, unsigned bytes, row-major) * B (32 x 8, signed bytes, column-major), 32-bit sums.
// Lane = 4 * g + t.  A: a0 = (row g, k 4t..4t+3), a1 = (row g+8, same k), a2, a3 = the same rows at k+16;
// B: b0 = (k 4t..4t+3, column g), b1 = k+16;  D: d0, d1 = (row g, columns 2t, 2t+1), d2, d3 = row g+8.
// With the digit words of four entries as B's columns 0..3 (columns 4..7 zero) one instruction
// contracts 16 x 32 codes with all four digits.
__device__ __forceinline__ void mma_u8s8(int (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
    asm("mma.sync.aligned.m16n8k32.row.col.s32.u8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3]) : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// The same with a zero accumulator coming in: the first product of a sum needs no cleared registers.
__device__ __forceinline__ void mma_u8s8_first(int (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
    asm("mma.sync.aligned.m16n8k32.row.col.s32.u8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%10,%10,%10};"
                 : "=r"(d[0]), "=r"(d[1]), "=r"(d[2]), "=r"(d[3]) : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1), "r"(0));
}

// Fragment loads from shared memory (ldmatrix, 8 x 8 matrices of 16-bit elements = 8 rows of 16 bytes).
// Lanes 8j..8j+7 give the row addresses of matrix j (16-byte aligned, shared-memory byte addresses);
// lane 4g + t receives from matrix j the four bytes 4t..4t+3 of its row g -- for byte data exactly an
// A fragment register (rows x k) or, with rows = columns of B, a B fragment register.
__device__ __forceinline__ void ldsm_x4(uint32_t (&r)[4], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr) : "memory");
}
__device__ __forceinline__ void ldsm_x2(uint32_t& r0, uint32_t& r1, uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x2.shared.b16 {%0,%1}, [%2];" : "=r"(r0), "=r"(r1) : "r"(addr) : "memory");
}
// Transposed: lane 4g + t receives from matrix j the 16-bit elements (row 2t, column g) and (row 2t+1,
// column g), i.e. bytes {2g, 2g+1} of row 2t in the low half and of row 2t+1 in the high half.
__device__ __forceinline__ void ldsm_x4_trans(uint32_t (&r)[4], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr) : "memory");
}

// Bytes (f0..f3) of four rows -> for each of the four features the bytes of the four rows.
__device__ __forceinline__ void transpose4x4(uint32_t x0, uint32_t x1, uint32_t x2, uint32_t x3, uint32_t (&t)[4]) {
    const uint32_t lo01 = __byte_perm(x0, x1, 0x5140), hi01 = __byte_perm(x0, x1, 0x7362);
    const uint32_t lo23 = __byte_perm(x2, x3, 0x5140), hi23 = __byte_perm(x2, x3, 0x7362);
    t[0] = __byte_perm(lo01, lo23, 0x5410);
    t[1] = __byte_perm(lo01, lo23, 0x7632);
    t[2] = __byte_perm(hi01, hi23, 0x5410);
    t[3] = __byte_perm(hi01, hi23, 0x7632);
}

}  // namespace zipml
