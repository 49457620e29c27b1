// Column range scan and the quantize + pack kernel (paper Section 2.1; Supplement "Randomized
// Quantization" and "Column Scaling"): two independent unbiased stochastic roundings of every
// sample element onto its feature's level grid, written as two bit-packed planes.
#include "common.cuh"
#include "internal.h"

namespace zipml {

// ---------------------------------------------------------------------------------------------
// Column range.  A tile is 32*VEC columns wide; blockDim = (32, 8): x walks the columns (one VEC-wide
// load per thread, a warp reads 128*VEC contiguous bytes of a row), y walks rows.  Row chunks are
// spread over gridDim.y; results meet in order-preserving integer atomics (min/max are exact and
// order independent).
// ---------------------------------------------------------------------------------------------
__global__ void range_init_kernel(uint32_t* lo_key, uint32_t* hi_key, int64_t n) {
    const int64_t j = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (j < n) { lo_key[j] = 0xffffffffu; hi_key[j] = 0u; }
}

template <int VEC>
__global__ void __launch_bounds__(256) range_scan_kernel(const float* __restrict__ A, int64_t m, int64_t n,
                                                         int64_t lda, int64_t rows_per_block, uint32_t* lo_key,
                                                         uint32_t* hi_key, DeviceStatus* status) {
    __shared__ float s_lo[8][32 * VEC];
    __shared__ float s_hi[8][32 * VEC];
    const int64_t j0 = ((int64_t)blockIdx.x * 32 + threadIdx.x) * VEC;
    const int64_t r0 = (int64_t)blockIdx.y * rows_per_block;
    const int64_t r1 = min(m, r0 + rows_per_block);
    float lo[VEC], hi[VEC];
    bool bad = false;
#pragma unroll
    for (int v = 0; v < VEC; ++v) { lo[v] = INFINITY; hi[v] = -INFINITY; }
    if (j0 < n) {
        for (int64_t r = r0 + threadIdx.y; r < r1; r += 8) {
            float val[VEC];
            bool have[VEC];
            if constexpr (VEC == 4) {
                if (j0 + 3 < n) {
                    const float4 q = __ldg(reinterpret_cast<const float4*>(A + r * lda + j0));
                    val[0] = q.x; val[1] = q.y; val[2] = q.z; val[3] = q.w;
                    have[0] = have[1] = have[2] = have[3] = true;
                } else {
#pragma unroll
                    for (int v = 0; v < VEC; ++v) {
                        have[v] = j0 + v < n;
                        val[v] = have[v] ? __ldg(A + r * lda + j0 + v) : 0.0f;
                    }
                }
            } else {
                val[0] = __ldg(A + r * lda + j0);
                have[0] = true;
            }
#pragma unroll
            for (int v = 0; v < VEC; ++v) {
                if (!have[v]) continue;
                bad |= !(fabsf(val[v]) <= 3.402823466e+38f);
                lo[v] = fminf(lo[v], val[v]);
                hi[v] = fmaxf(hi[v], val[v]);
            }
        }
    }
#pragma unroll
    for (int v = 0; v < VEC; ++v) { s_lo[threadIdx.y][threadIdx.x * VEC + v] = lo[v]; s_hi[threadIdx.y][threadIdx.x * VEC + v] = hi[v]; }
    if (bad) set_status(status, ZIPML_ERR_NONFINITE, 1);
    __syncthreads();
    const int t = threadIdx.y * 32 + threadIdx.x;
    if (t < 32 * VEC) {
        const int64_t j = (int64_t)blockIdx.x * 32 * VEC + t;
        if (j < n) {
            float a = s_lo[0][t], b = s_hi[0][t];
#pragma unroll
            for (int y = 1; y < 8; ++y) { a = fminf(a, s_lo[y][t]); b = fmaxf(b, s_hi[y][t]); }
            if (a <= b) {  // at least one row seen
                atomicMin(lo_key + j, float_order_key(a));
                atomicMax(hi_key + j, float_order_key(b));
            }
        }
    }
}

__global__ void range_finalize_kernel(const uint32_t* lo_key, const uint32_t* hi_key, int64_t n, int s,
                                      float* lo_out, float* hi_out, float* inv_out, float* step_out) {
    const int64_t j = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= n) return;
    const float lo = float_from_order_key(lo_key[j]), hi = float_from_order_key(hi_key[j]);
    const float range = __fsub_rn(hi, lo);
    lo_out[j] = lo;
    if (hi_out) hi_out[j] = hi;
    if (inv_out) inv_out[j] = range > 0.0f ? __fdiv_rn((float)s, range) : 0.0f;
    if (step_out) step_out[j] = __fdiv_rn(range, (float)s);
}

int launch_column_range(zipml_ctx* ctx, const float* A, int64_t m, int64_t n, int64_t lda, int s,
                        uint32_t* key_scratch, float* lo_out, float* hi_out, float* inv_out, float* step_out) {
    uint32_t* lo_key = key_scratch;
    uint32_t* hi_key = key_scratch + n;
    const unsigned nb = (unsigned)((n + 255) / 256);
    range_init_kernel<<<nb, 256, 0, ctx->stream>>>(lo_key, hi_key, n);
    const bool vec = (lda % 4 == 0) && ((reinterpret_cast<uintptr_t>(A) & 15) == 0);
    const int width = vec ? 128 : 32;
    const int64_t col_tiles = (n + width - 1) / width;
    // enough row chunks to give every SM a few blocks, at least 64 rows each
    int64_t chunks = (int64_t)ctx->sm_count * 8 / col_tiles;
    chunks = chunks < 1 ? 1 : chunks;
    int64_t rows_per_block = (m + chunks - 1) / chunks;
    rows_per_block = rows_per_block < 64 ? 64 : rows_per_block;
    chunks = (m + rows_per_block - 1) / rows_per_block;
    if (chunks > 65535) { rows_per_block = (m + 65534) / 65535; chunks = (m + rows_per_block - 1) / rows_per_block; }
    const dim3 grid((unsigned)col_tiles, (unsigned)chunks), block(32, 8);
    if (vec) range_scan_kernel<4><<<grid, block, 0, ctx->stream>>>(A, m, n, lda, rows_per_block, lo_key, hi_key, ctx->d_status);
    else range_scan_kernel<1><<<grid, block, 0, ctx->stream>>>(A, m, n, lda, rows_per_block, lo_key, hi_key, ctx->d_status);
    range_finalize_kernel<<<nb, 256, 0, ctx->stream>>>(lo_key, hi_key, n, s, lo_out, hi_out, inv_out, step_out);
    ctx->launches += 3;
    return cuda_status(cudaGetLastError());
}

// ---------------------------------------------------------------------------------------------
// Quantize + pack.  One thread produces one 32-bit word of each plane: FPW = 32/CB consecutive
// features of one row.  It reads them as float4s when the row is 16-byte aligned, decides the cell
// and the up-probability in pinned fp32 arithmetic, draws one Philox block per feature pair (four
// words = two features x two copies) and writes the two words.  Words past the last feature are
// written as zero so that the planes are fully defined.
// ---------------------------------------------------------------------------------------------
template <int CB, bool TABLE>
__global__ void __launch_bounds__(256) quantize_kernel(const float* __restrict__ A, int64_t m, int64_t n, int64_t lda,
                                                       int bits, const float* __restrict__ lo,
                                                       const float* __restrict__ inv, const float* __restrict__ levels,
                                                       uint64_t seed, uint32_t* __restrict__ plane1,
                                                       uint32_t* __restrict__ plane2, int64_t row_words, bool vec_ok) {
    constexpr int FPW = 32 / CB;
    const int64_t id = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (id >= m * row_words) return;
    const int64_t row = id / row_words;
    const int64_t q = id - row * row_words;
    const int64_t j0 = q * FPW;
    const int L = 1 << bits, s = L - 1;
    uint32_t w1 = 0u, w2 = 0u;
    if (j0 < n) {
        float v[FPW];
        const float* src = A + row * lda + j0;
        if (vec_ok && j0 + FPW <= n) {
#pragma unroll
            for (int i = 0; i < FPW / 4; ++i) {
                const float4 t = __ldg(reinterpret_cast<const float4*>(src) + i);
                v[4 * i] = t.x; v[4 * i + 1] = t.y; v[4 * i + 2] = t.z; v[4 * i + 3] = t.w;
            }
        } else {
#pragma unroll
            for (int i = 0; i < FPW; ++i) v[i] = (j0 + i < n) ? __ldg(src + i) : 0.0f;
        }
#pragma unroll
        for (int pr = 0; pr < FPW / 2; ++pr) {
            const int64_t ja = j0 + 2 * pr;
            if (ja >= n) break;
            const Philox4 rnd = sample_block(seed, (uint64_t)row, (uint32_t)(ja >> 1));
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int64_t j = ja + h;
                if (j >= n) break;
                uint32_t cell;
                float p;
                if (!TABLE) {
                    uniform_cell(v[2 * pr + h], __ldg(lo + j), __ldg(inv + j), s, cell, p);
                } else {
                    const float* lev = levels + j * L;
                    const float val = v[2 * pr + h];
                    int l = 0;
                    for (int i = 1; i <= s - 1; ++i) l = (__ldg(lev + i) <= val) ? i : l;
                    const float base = __ldg(lev + l);
                    const float width = __fsub_rn(__ldg(lev + l + 1), base);
                    cell = (uint32_t)l;
                    p = width > 0.0f ? __fdiv_rn(__fsub_rn(val, base), width) : 0.0f;
                }
                const uint32_t c1 = round_up_if(cell, p, rnd.v[2 * h]);
                const uint32_t c2 = round_up_if(cell, p, rnd.v[2 * h + 1]);
                w1 |= c1 << ((2 * pr + h) * CB);
                w2 |= c2 << ((2 * pr + h) * CB);
            }
        }
    }
    plane1[row * row_words + q] = w1;
    plane2[row * row_words + q] = w2;
}

int launch_quantize(zipml_ctx* ctx, const float* A, int64_t m, int64_t n, int64_t lda, int bits, int level_mode,
                    const float* lo, const float* inv, const float* levels, uint64_t seed, uint8_t* plane1,
                    uint8_t* plane2, int64_t row_bytes) {
    const int cb = container_bits(bits);
    const int64_t row_words = row_bytes / 4;
    const int64_t total = m * row_words;
    const int64_t blocks = (total + 255) / 256;
    if (blocks > 0x7fffffffLL) return ZIPML_ERR_WORKSPACE;
    const bool vec_ok = (lda % 4 == 0) && ((reinterpret_cast<uintptr_t>(A) & 15) == 0);
    uint32_t* p1 = reinterpret_cast<uint32_t*>(plane1);
    uint32_t* p2 = reinterpret_cast<uint32_t*>(plane2);
    const bool table = level_mode == ZIPML_LEVELS_TABLE;
#define ZIPML_LAUNCH_Q(CB_, T_)                                                                         \
    quantize_kernel<CB_, T_><<<(unsigned)blocks, 256, 0, ctx->stream>>>(A, m, n, lda, bits, lo, inv, levels, seed, p1, \
                                                                        p2, row_words, vec_ok)
    if (cb == 2) { if (table) ZIPML_LAUNCH_Q(2, true); else ZIPML_LAUNCH_Q(2, false); }
    else if (cb == 4) { if (table) ZIPML_LAUNCH_Q(4, true); else ZIPML_LAUNCH_Q(4, false); }
    else { ZIPML_LAUNCH_Q(8, false); }
#undef ZIPML_LAUNCH_Q
    ctx->launches += 1;
    return cuda_status(cudaGetLastError());
}

}  // namespace zipml
