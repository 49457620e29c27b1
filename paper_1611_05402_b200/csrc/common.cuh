// Device helpers shared by the kernels: the counter-based random numbers, the pinned fp32
// rounding decision, container widths and a few warp/block reductions.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/zipml.h"

namespace zipml {

// Device-side status word values (ORed is not needed: first error wins).
struct DeviceStatus {
    int code;          // ZIPML_OK or a ZIPML_ERR_* value, set with atomicCAS from 0
    int detail;        // where a wait gave up, or 0
};

__device__ __forceinline__ void set_status(DeviceStatus* st, int code, int detail) {
    if (atomicCAS(&st->code, 0, code) == 0) st->detail = detail;
}

__host__ __device__ __forceinline__ int container_bits(int bits) {
    return (bits == 1 || bits == 2) ? 2 : (bits == 3 || bits == 4) ? 4 : (bits >= 5 && bits <= 8) ? 8 : 0;
}

// ---------------------------------------------------------------------------------------------
// Philox4x32-10 (Salmon et al., SC'11), written from its published round function.
// ---------------------------------------------------------------------------------------------
struct Philox4 {
    uint32_t v[4];
};

__device__ __forceinline__ Philox4 philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                                 uint32_t k0, uint32_t k1) {
    constexpr uint32_t kMul0 = 0xD2511F53u, kMul1 = 0xCD9E8D57u;
    constexpr uint32_t kWeyl0 = 0x9E3779B9u, kWeyl1 = 0xBB67AE85u;
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const uint32_t hi0 = __umulhi(kMul0, c0), lo0 = kMul0 * c0;
        const uint32_t hi1 = __umulhi(kMul1, c2), lo1 = kMul1 * c2;
        c0 = hi1 ^ c1 ^ k0;
        c1 = lo1;
        c2 = hi0 ^ c3 ^ k1;
        c3 = lo0;
        k0 += kWeyl0;
        k1 += kWeyl1;
    }
    Philox4 out;
    out.v[0] = c0; out.v[1] = c1; out.v[2] = c2; out.v[3] = c3;
    return out;
}

// Random block of the sample feature pair (2p, 2p+1) of row `row`: words {2p copy 1, 2p copy 2,
// 2p+1 copy 1, 2p+1 copy 2}; the top 24 bits of a word are the uniform integer.
// `draw` numbers further independent pairs of quantizations of the same samples (0: the two samples of the SGD path).
__device__ __forceinline__ Philox4 sample_block(uint64_t seed, uint64_t row, uint32_t pair, uint32_t draw) {
    return philox4x32_10((uint32_t)row, (uint32_t)(row >> 32), pair, draw, (uint32_t)seed, (uint32_t)(seed >> 32));
}

// Uniform 24-bit integer for coordinate `coord` of the model (stream 3) / gradient (stream 4)
// quantizer at (epoch, step).
__device__ __forceinline__ uint32_t vector_u24(uint64_t seed, uint32_t epoch, uint32_t step, uint32_t coord,
                                               uint32_t stream) {
    const Philox4 b = philox4x32_10(coord >> 2, step, epoch, stream, (uint32_t)seed, (uint32_t)(seed >> 32));
    return b.v[coord & 3u] >> 8;
}

// up <=> u24 * 2^-24 < p, both sides fp32 (the product is exact).  Since u24 is an integer below 2^24 and
// p * 2^24 is exact in fp32, that is u24 < ceil(p * 2^24): the threshold is computed once per element (one
// conversion; int <-> float conversions issue at a sixteenth of the FMA rate) and compared as integers for
// both copies.  p <= 0 or NaN gives 0 (never up), p >= 1 gives at least 2^24 (always up).
__device__ __forceinline__ uint32_t up_threshold(float p) { return __float2uint_ru(__fmul_rn(p, 16777216.0f)); }
__device__ __forceinline__ uint32_t round_up_if(uint32_t cell, uint32_t threshold, uint32_t word) {
    return cell + ((word >> 8) < threshold ? 1u : 0u);
}

// Cell and up-probability on a uniform grid of s intervals (s < 2^22): t = (v - lo) * inv with every
// operation rounded on its own (no contraction into an FMA), cell = clamp(floor t, 0, s-1), p = t - cell.
// The floor needs no conversion instruction: 2^23 + t' rounded down keeps floor(t') in its mantissa.
// A NaN lands in cell 0 with p = NaN (never up); -inf in cell 0, +inf in the last cell, always up.
__device__ __forceinline__ void uniform_cell(float v, float lo, float inv, int s, uint32_t& cell, float& p) {
    const float t = __fmul_rn(__fsub_rn(v, lo), inv);
    const float tc = fmaxf(t, 0.0f);                                        // NaN -> 0
    float fl = __fsub_rn(__fadd_rd(tc, 8388608.0f), 8388608.0f);            // floor(tc), exact for tc < 2^23
    fl = fminf(fl, (float)(s - 1));
    cell = __float_as_uint(__fadd_rn(fl, 8388608.0f)) & 0x7FFFFFu;
    p = __fsub_rn(t, fl);
}

// Regulariser applied to y = x - lr g, coordinate by coordinate (paper Eq. (proxupdate); reg 4: the
// least-squares SVM term of the Supplement).  cst is the per-call constant in fp32: 1/(1 + lr c),
// lr lambda or lr c.  Every operation is one IEEE fp32 rounding.
__device__ __forceinline__ float regularise(float y, float x_old, int reg, float cst) {
    if (reg == ZIPML_REG_L2) return __fmul_rn(y, cst);
    if (reg == ZIPML_REG_L1) {
        const float mag = __fsub_rn(fabsf(y), cst);
        return mag > 0.0f ? copysignf(mag, y) : 0.0f;
    }
    if (reg == ZIPML_REG_NONNEG) return y > 0.0f ? y : 0.0f;
    if (reg == ZIPML_REG_LSSVM) return __fmaf_rn(-cst, x_old, y);
    return y;
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// Sum over the block in a fixed order (warp results combined by thread 0); every thread gets the
// result.  `scratch` holds at least 33 doubles.  Ends with the block synchronised.
__device__ __forceinline__ double block_sum(double v, double* scratch) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = (blockDim.x + 31) >> 5;
    v = warp_sum(v);
    __syncthreads();
    if (lane == 0) scratch[warp] = v;
    __syncthreads();
    if (threadIdx.x == 0) {
        double t = 0.0;
        for (int w = 0; w < nwarps; ++w) t += scratch[w];
        scratch[32] = t;
    }
    __syncthreads();
    return scratch[32];
}

// The same for a maximum of non-negative values.
__device__ __forceinline__ double block_max(double v, double* scratch) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = (blockDim.x + 31) >> 5;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmax(v, __shfl_xor_sync(0xffffffffu, v, o));
    __syncthreads();
    if (lane == 0) scratch[warp] = v;
    __syncthreads();
    if (threadIdx.x == 0) {
        double t = 0.0;
        for (int w = 0; w < nwarps; ++w) t = fmax(t, scratch[w]);
        scratch[32] = t;
    }
    __syncthreads();
    return scratch[32];
}

// Order-preserving map float -> uint32 so that integer atomicMin/Max order floats (-0 < +0).
__device__ __forceinline__ uint32_t float_order_key(float f) {
    const uint32_t b = __float_as_uint(f);
    return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}

__device__ __forceinline__ float float_from_order_key(uint32_t k) {
    return __uint_as_float((k & 0x80000000u) ? (k & 0x7fffffffu) : ~k);
}

// ---------------------------------------------------------------------------------------------
// Unpacking a 32-bit word of codes into floats.  A code byte is dropped into the mantissa of 2^23
// with one byte permute, and subtracting 2^23 leaves the exact integer: no int->float conversion
// instruction (they issue at a fraction of the FMA rate).
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ float byte_to_float(uint32_t bytes, int i) {
    return __uint_as_float(__byte_perm(bytes, 0x4B000000u, 0x7650 + i)) - 8388608.0f;
}

template <int CB>
__device__ __forceinline__ void unpack_word(uint32_t w, float (&c)[32 / CB]) {
    if constexpr (CB == 8) {
#pragma unroll
        for (int i = 0; i < 4; ++i) c[i] = byte_to_float(w, i);
    } else if constexpr (CB == 4) {
        const uint32_t even = w & 0x0F0F0F0Fu, odd = (w >> 4) & 0x0F0F0F0Fu;
#pragma unroll
        for (int i = 0; i < 4; ++i) { c[2 * i] = byte_to_float(even, i); c[2 * i + 1] = byte_to_float(odd, i); }
    } else {
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const uint32_t t = (w >> (2 * k)) & 0x03030303u;
#pragma unroll
            for (int i = 0; i < 4; ++i) c[4 * i + k] = byte_to_float(t, i);
        }
    }
}

template <int CB>
__device__ __forceinline__ int code_at(uint32_t w, int i) {
    return (int)((w >> (i * CB)) & ((1u << CB) - 1u));
}


}  // namespace zipml
