// Polynomial estimator over several independent quantizations of the samples (paper Section 4.1 "Quantizing
// Polynomials": Q(P) = sum_i m_i prod_{j <= i} Q_j(a)^T x, unbiased for P(a^T x) because the factors of a product
// are independent) and the sample mean of c_k Q(a_k) that Section 4.2's protocol uses as the gradient
// (c_k = b_k Q(P)_k, Q = Q_{d+1}).  Both read packed planes on the grid of a zipml_dataset.
#include "common.cuh"
#include "internal.h"

namespace zipml {

constexpr int kPolyMaxDegree = ZIPML_POLY_MAX_DEGREE;

struct PolyArgs {
    const uint32_t* plane[kPolyMaxDegree];
    double coef[kPolyMaxDegree + 1];
    int d;
};

// A warp per sample: the dots of its d planes one after the other (fp32 products in runs of at most 8 words per
// lane, combined in double), the running product and the polynomial's value in double.
template <int CB, bool TABLE>
__global__ void __launch_bounds__(256) poly_rows_kernel(const PolyArgs a, int64_t row_words, int64_t m, int64_t n,
                                                        const float* __restrict__ wtab, const double* __restrict__ base_in,
                                                        const float* __restrict__ scale, double* __restrict__ rows_out) {
    constexpr int FPW = 32 / CB;
    const int lane = threadIdx.x & 31;
    const int64_t warp_global = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int64_t nwarps = ((int64_t)gridDim.x * blockDim.x) >> 5;
    const int64_t words = (n + FPW - 1) / FPW;
    const double base = *base_in;
    for (int64_t k = warp_global; k < m; k += nwarps) {
        double value = a.coef[0], prod = 1.0;
#pragma unroll 1
        for (int i = 1; i <= a.d; ++i) {
            const uint32_t* row = a.plane[i - 1] + k * row_words;
            double z = 0.0;
            for (int64_t q0 = 0; q0 < words; q0 += 32 * 8) {
                float acc = 0.0f;
#pragma unroll 2
                for (int s = 0; s < 8; ++s) {
                    const int64_t q = q0 + s * 32 + lane;
                    if (q < words) {
                        const uint32_t u = __ldg(row + q);
                        if constexpr (!TABLE) {
                            float c[FPW];
                            unpack_word<CB>(u, c);
#pragma unroll
                            for (int e = 0; e < FPW; ++e) {
                                const int64_t j = q * FPW + e;
                                acc = fmaf(c[e], (j < n) ? __ldg(wtab + j) : 0.0f, acc);
                            }
                        } else {
#pragma unroll
                            for (int e = 0; e < FPW; ++e) {
                                const int64_t j = q * FPW + e;
                                if (j < n) acc += __ldg(wtab + (int64_t)code_at<CB>(u, e) * n + j);
                            }
                        }
                    }
                }
                z += (double)acc;
            }
            z = warp_sum(z) + base;
            prod *= z;
            value += a.coef[i] * prod;
        }
        if (lane == 0) rows_out[k] = scale ? (double)__ldg(scale + k) * value : value;
    }
}

// Partial sums of c_k * code (uniform grid) or c_k * level (table) over a chunk of rows: a thread per word column.
template <int CB, bool TABLE>
__global__ void __launch_bounds__(128) plane_mean_partial_kernel(const uint32_t* __restrict__ plane, int64_t row_words, int64_t m,
                                                                 int64_t n, int L, const float* __restrict__ levels,
                                                                 const double* __restrict__ c, int64_t rows_per_block,
                                                                 double* __restrict__ partial /* [row chunks][n + 1] */) {
    constexpr int FPW = 32 / CB;
    const int64_t q = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int64_t words = (n + FPW - 1) / FPW;
    const int64_t k0 = (int64_t)blockIdx.y * rows_per_block, k1 = min(m, k0 + rows_per_block);
    double acc[FPW];
#pragma unroll
    for (int e = 0; e < FPW; ++e) acc[e] = 0.0;
    double csum = 0.0;
    if (q < words) {
        for (int64_t k = k0; k < k1; ++k) {
            const uint32_t u = __ldg(plane + k * row_words + q);
            const double ck = __ldg(c + k);
            csum += ck;
#pragma unroll
            for (int e = 0; e < FPW; ++e) {
                const int64_t j = q * FPW + e;
                if constexpr (!TABLE) acc[e] += ck * (double)code_at<CB>(u, e);
                else if (j < n) acc[e] += ck * (double)__ldg(levels + j * L + code_at<CB>(u, e));
            }
        }
        double* out = partial + (int64_t)blockIdx.y * (n + 1);
#pragma unroll
        for (int e = 0; e < FPW; ++e) {
            const int64_t j = q * FPW + e;
            if (j < n) out[j] = acc[e];
        }
        if (q == 0) out[n] = csum;
    }
}

__global__ void plane_mean_finish_kernel(const double* __restrict__ partial, int chunks, int64_t n, int64_t m, bool table,
                                         const float* __restrict__ lo, const float* __restrict__ step, float* __restrict__ g_out) {
    const int64_t j = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= n) return;
    double s = 0.0, cs = 0.0;
    for (int r = 0; r < chunks; ++r) { s += partial[(int64_t)r * (n + 1) + j]; cs += partial[(int64_t)r * (n + 1) + n]; }
    const double v = table ? s : (double)lo[j] * cs + (double)step[j] * s;
    g_out[j] = (float)(v / (double)m);
}

int launch_poly_rows(zipml_ctx* ctx, const zipml_dataset* d, const uint8_t* const* planes, int degree, const double* coef,
                     const float* wtab, const double* base, const float* scale, double* rows_out) {
    PolyArgs a;
    for (int i = 0; i < kPolyMaxDegree; ++i) a.plane[i] = i < degree ? reinterpret_cast<const uint32_t*>(planes[i]) : nullptr;
    for (int i = 0; i <= kPolyMaxDegree; ++i) a.coef[i] = i <= degree ? coef[i] : 0.0;
    a.d = degree;
    const int cb = container_bits(d->bits);
    const bool table = d->level_mode == ZIPML_LEVELS_TABLE;
    int blocks = ctx->sm_count * 8;
    const int64_t need = (d->m + 7) / 8;
    if (blocks > need) blocks = (int)need;
    const int64_t rw = d->row_bytes / 4;
#define ZIPML_LAUNCH_P(CB_, T_) poly_rows_kernel<CB_, T_><<<blocks, 256, 0, ctx->stream>>>(a, rw, d->m, d->n, wtab, base, scale, rows_out)
    if (cb == 2) { if (table) ZIPML_LAUNCH_P(2, true); else ZIPML_LAUNCH_P(2, false); }
    else if (cb == 4) { if (table) ZIPML_LAUNCH_P(4, true); else ZIPML_LAUNCH_P(4, false); }
    else { ZIPML_LAUNCH_P(8, false); }
#undef ZIPML_LAUNCH_P
    ++ctx->launches;
    return cuda_status(cudaGetLastError());
}

int plane_mean_chunks(const zipml_ctx* ctx, int64_t m) {
    int64_t chunks = (m + 255) / 256;                  // at least 256 rows per chunk, at most four chunks per SM
    const int64_t cap = (int64_t)ctx->sm_count * 4;
    return (int)(chunks > cap ? cap : (chunks < 1 ? 1 : chunks));
}

int launch_plane_mean(zipml_ctx* ctx, const zipml_dataset* d, const uint8_t* plane, const double* c, double* partial,
                      float* g_out) {
    const int cb = container_bits(d->bits), fpw = 32 / cb;
    const bool table = d->level_mode == ZIPML_LEVELS_TABLE;
    const int chunks = plane_mean_chunks(ctx, d->m);
    const int64_t rows_per_block = (d->m + chunks - 1) / chunks;
    const int64_t words = (d->n + fpw - 1) / fpw;
    const dim3 grid((unsigned)((words + 127) / 128), (unsigned)chunks);
    const uint32_t* p = reinterpret_cast<const uint32_t*>(plane);
    const int64_t rw = d->row_bytes / 4;
    const int L = 1 << d->bits;
#define ZIPML_LAUNCH_M(CB_, T_) \
    plane_mean_partial_kernel<CB_, T_><<<grid, 128, 0, ctx->stream>>>(p, rw, d->m, d->n, L, d->levels, c, rows_per_block, partial)
    if (cb == 2) { if (table) ZIPML_LAUNCH_M(2, true); else ZIPML_LAUNCH_M(2, false); }
    else if (cb == 4) { if (table) ZIPML_LAUNCH_M(4, true); else ZIPML_LAUNCH_M(4, false); }
    else { ZIPML_LAUNCH_M(8, false); }
#undef ZIPML_LAUNCH_M
    plane_mean_finish_kernel<<<(unsigned)((d->n + 255) / 256), 256, 0, ctx->stream>>>(partial, chunks, d->n, d->m, table, d->feat_lo,
                                                                                       d->feat_step, g_out);
    ctx->launches += 2;
    return cuda_status(cudaGetLastError());
}

}  // namespace zipml
