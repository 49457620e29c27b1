// Fixed-point digits for the integer contractions of the SGD engines (uniform grids).
#pragma once

#include "common.cuh"

namespace zipml {

// ---- integer contraction (uniform grids) ---------------------------------------------------------
// Both phases contract small unsigned codes with an fp32 vector that is constant for many rows (w in
// phase A, the residuals in phase B).  That vector is turned, once per step, into fixed point:
// value ~ delta * W with |W| <= QMAX, and W into NS balanced base-128 digits in [-64, 63], each an
// int8.  Four codes times four digits are then one dp4a into an int32, the digit sums are combined
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

}  // namespace zipml
