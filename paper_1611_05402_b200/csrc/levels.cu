// Variance-optimal level placement (paper Section 3): a one-pass per-feature histogram over equal
// bins of the normalised range ("Discretization"), then the dynamic programme
//   T(k, m) = min_j T(k-1, j) + V(j, m)
// over the bin edges ("Dynamic Programming with Candidate Points") in exact 64-bit integers.
#include "common.cuh"
#include "internal.h"

namespace zipml {

// ---------------------------------------------------------------------------------------------
// Histogram.  A block owns 32 features and a chunk of rows and keeps 32 x bins counters in shared
// memory (row stride bins+1, so that lanes hitting the same bin of different features fall into
// different banks).  blockDim = (32, 8): a warp reads 128 contiguous bytes of a row.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) histogram_kernel(const float* __restrict__ A, int64_t m, int64_t n, int64_t lda,
                                                        int bins, int64_t rows_per_block,
                                                        const float* __restrict__ lo, const float* __restrict__ inv,
                                                        uint32_t* __restrict__ counts) {
    extern __shared__ uint32_t s_hist[];
    const int stride = bins + 1;
    const int t = threadIdx.y * 32 + threadIdx.x;
    for (int i = t; i < 32 * stride; i += 256) s_hist[i] = 0u;
    __syncthreads();
    const int64_t j = (int64_t)blockIdx.x * 32 + threadIdx.x;
    if (j < n) {
        const float flo = __ldg(lo + j), finv = __ldg(inv + j);
        const int64_t r0 = (int64_t)blockIdx.y * rows_per_block;
        const int64_t r1 = min(m, r0 + rows_per_block);
        uint32_t* mine = s_hist + threadIdx.x * stride;
        for (int64_t r = r0 + threadIdx.y; r < r1; r += 8) {
            uint32_t cell;
            float p;
            uniform_cell(__ldg(A + r * lda + j), flo, finv, bins, cell, p);
            atomicAdd(mine + cell, 1u);
        }
    }
    __syncthreads();
    for (int i = t; i < 32 * bins; i += 256) {
        const int f = i / bins, c = i - f * bins;
        const int64_t jj = (int64_t)blockIdx.x * 32 + f;
        const uint32_t v = s_hist[f * stride + c];
        if (jj < n && v) atomicAdd(counts + jj * bins + c, v);
    }
}

int launch_histogram(zipml_ctx* ctx, const float* A, int64_t m, int64_t n, int64_t lda, int bins, const float* lo,
                     const float* inv, uint32_t* counts) {
    cudaError_t e = cudaMemsetAsync(counts, 0, sizeof(uint32_t) * (size_t)(n * bins), ctx->stream);
    if (e != cudaSuccess) return cuda_status(e);
    const size_t smem = sizeof(uint32_t) * 32 * (size_t)(bins + 1);
    if (smem > (size_t)ctx->smem_optin) return ZIPML_ERR_WORKSPACE;
    e = cudaFuncSetAttribute(histogram_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return cuda_status(e);
    const int64_t col_tiles = (n + 31) / 32;
    int64_t chunks = (int64_t)ctx->sm_count * 2 / col_tiles;
    chunks = chunks < 1 ? 1 : chunks;
    int64_t rows_per_block = (m + chunks - 1) / chunks;
    rows_per_block = rows_per_block < 256 ? 256 : rows_per_block;
    chunks = (m + rows_per_block - 1) / rows_per_block;
    if (chunks > 65535) { rows_per_block = (m + 65534) / 65535; chunks = (m + rows_per_block - 1) / rows_per_block; }
    histogram_kernel<<<dim3((unsigned)col_tiles, (unsigned)chunks), dim3(32, 8), smem, ctx->stream>>>(
        A, m, n, lda, bins, rows_per_block, lo, inv, counts);
    ctx->launches += 1;
    return cuda_status(cudaGetLastError());
}

// ---------------------------------------------------------------------------------------------
// Level DP: one block per feature.  With bin centres at odd positions x_i = 2i+1 (units of 1/(2M))
// and edges at even positions, the variance of the points of [d_j, d_m] is
//   4 M^2 V(j, m) = sum c_i (2m - x_i)(x_i - 2j) = 2(j+m) S1 - S2 - 4jm S0
// with S_p the sums of c_i x_i^p over the bins j..m-1, taken from prefix sums.  Everything is an
// exact integer below 2^63 (up to 10^9 points, 1024 bins), so the result does not depend on the
// order of evaluation.  Ties go to the smallest j.
// ---------------------------------------------------------------------------------------------
constexpr int kDpThreads = 256;

__global__ void __launch_bounds__(kDpThreads) levels_dp_kernel(const uint32_t* __restrict__ counts, int bins, int s,
                                                               const float* __restrict__ lo,
                                                               const float* __restrict__ hi,
                                                               float* __restrict__ levels_out,
                                                               unsigned long long* __restrict__ objective_out) {
    extern __shared__ unsigned long long s_mem[];
    const int M = bins, M1 = bins + 1;
    unsigned long long* P0 = s_mem;
    unsigned long long* P1 = P0 + M1;
    unsigned long long* P2 = P1 + M1;
    unsigned long long* Ta = P2 + M1;
    unsigned long long* Tb = Ta + M1;
    unsigned short* arg = reinterpret_cast<unsigned short*>(Tb + M1);   // (s+1) x M1
    __shared__ int s_idx[17];
    const int64_t j_feat = blockIdx.x;
    const uint32_t* cnt = counts + j_feat * M;

    // prefix sums of c, c x, c x^2: every thread sums a run of bins, the runs' totals are scanned by warp 0
    {
        __shared__ unsigned long long tot[3][kDpThreads];
        const int per = (M + kDpThreads - 1) / kDpThreads;
        const int i_begin = min(M, (int)threadIdx.x * per), i_end = min(M, i_begin + per);
        unsigned long long a0 = 0, a1 = 0, a2 = 0;
        for (int i = i_begin; i < i_end; ++i) {
            const unsigned long long c = cnt[i], x = 2ull * i + 1ull;
            a0 += c; a1 += c * x; a2 += c * x * x;
        }
        tot[0][threadIdx.x] = a0; tot[1][threadIdx.x] = a1; tot[2][threadIdx.x] = a2;
        __syncthreads();
        if (threadIdx.x < 3) {                     // exclusive scan of one of the three rows (256 additions)
            unsigned long long run = 0;
            for (int t = 0; t < kDpThreads; ++t) { const unsigned long long v = tot[threadIdx.x][t]; tot[threadIdx.x][t] = run; run += v; }
        }
        __syncthreads();
        a0 = tot[0][threadIdx.x]; a1 = tot[1][threadIdx.x]; a2 = tot[2][threadIdx.x];
        if (threadIdx.x == 0) P0[0] = P1[0] = P2[0] = 0;
        for (int i = i_begin; i < i_end; ++i) {
            const unsigned long long c = cnt[i], x = 2ull * i + 1ull;
            a0 += c; a1 += c * x; a2 += c * x * x;
            P0[i + 1] = a0; P1[i + 1] = a1; P2[i + 1] = a2;
        }
    }
    __syncthreads();
    auto cost = [&](int j, int mm) -> unsigned long long {
        const unsigned long long S0 = P0[mm] - P0[j], S1 = P1[mm] - P1[j], S2 = P2[mm] - P2[j];
        return 2ull * (unsigned long long)(j + mm) * S1 - S2 - 4ull * (unsigned long long)j * (unsigned long long)mm * S0;
    };
    for (int mm = 1 + threadIdx.x; mm <= M; mm += kDpThreads) { Ta[mm] = cost(0, mm); arg[1 * M1 + mm] = 0; }
    __syncthreads();
    unsigned long long* prev = Ta;
    unsigned long long* cur = Tb;
    // The interval cost satisfies the quadrangle inequality (a point of [b,c) adds (2d-2c)(2b-2a) >= 0 to
    // w(a,d) + w(b,c) - w(a,c) - w(b,d), points left and right of it add non-negative amounts too), so the
    // leftmost minimiser j*(m) of prev[j] + cost(j, m) does not decrease with m.  Anchors -- every 32nd m
    // and m = M -- are minimised over their whole range by a warp each; every other m then only scans from
    // its lower anchor's minimiser to its upper anchor's.  The minima, and with ascending scans and strict
    // comparisons the leftmost minimisers, are those of the full scan.
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    constexpr int kStride = 32;
    for (int k = 2; k <= s; ++k) {
        const int first_anchor = (k + kStride - 1) / kStride;          // anchors at kStride * a, a >= first_anchor, and at M
        const int n_mult = M / kStride >= first_anchor ? M / kStride - first_anchor + 1 : 0;
        const bool m_extra = (M % kStride) != 0 || n_mult == 0;         // M itself, if it is not a multiple already
        const int n_anchor = n_mult + (m_extra ? 1 : 0);
        for (int a = warp; a < n_anchor; a += kDpThreads / 32) {
            const int mm = a < n_mult ? (first_anchor + a) * kStride : M;
            unsigned long long best = ~0ull;
            int bj = 0x7fffffff;
            for (int j = k - 1 + lane; j <= mm - 1; j += 32) {
                const unsigned long long c = prev[j] + cost(j, mm);
                if (c < best) { best = c; bj = j; }
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                const unsigned long long ob = __shfl_xor_sync(0xffffffffu, best, o);
                const int oj = __shfl_xor_sync(0xffffffffu, bj, o);
                if (ob < best || (ob == best && oj < bj)) { best = ob; bj = oj; }
            }
            if (lane == 0) { cur[mm] = best; arg[k * M1 + mm] = (unsigned short)bj; }
        }
        __syncthreads();
        for (int mm = k + threadIdx.x; mm <= M; mm += kDpThreads) {
            if (mm == M || (mm % kStride == 0 && mm / kStride >= first_anchor)) continue;      // an anchor
            const int below = (mm / kStride) * kStride;
            int above = below + kStride;
            if (above > M) above = M;
            const int j_lo = (below / kStride >= first_anchor && below >= k) ? (int)arg[k * M1 + below] : k - 1;
            const int j_hi = min((int)arg[k * M1 + above], mm - 1);
            unsigned long long best = ~0ull;
            int bj = j_lo;
            for (int j = j_lo; j <= j_hi; ++j) {
                const unsigned long long c = prev[j] + cost(j, mm);
                if (c < best) { best = c; bj = j; }
            }
            cur[mm] = best;
            arg[k * M1 + mm] = (unsigned short)bj;
        }
        __syncthreads();
        unsigned long long* t = prev; prev = cur; cur = t;
    }
    if (threadIdx.x == 0) {
        if (objective_out) objective_out[j_feat] = prev[M];
        int mm = M;
        for (int k = s; k >= 1; --k) { s_idx[k] = mm; mm = arg[k * M1 + mm]; }
        s_idx[0] = 0;
    }
    __syncthreads();
    if (threadIdx.x <= s) {
        const float flo = lo[j_feat], fhi = hi[j_feat];
        const float range = __fsub_rn(fhi, flo);
        const float frac = __fdiv_rn((float)s_idx[threadIdx.x], (float)M);
        float v = __fadd_rn(flo, __fmul_rn(range, frac));
        if (threadIdx.x == 0) v = flo;
        if (threadIdx.x == s) v = fhi;
        levels_out[j_feat * (s + 1) + threadIdx.x] = v;
    }
}

int launch_levels_dp(zipml_ctx* ctx, const uint32_t* counts, int64_t n, int bins, int s, const float* lo,
                     const float* hi, float* levels_out, uint64_t* objective_out) {
    const size_t smem = sizeof(unsigned long long) * 5 * (size_t)(bins + 1) + sizeof(unsigned short) * (size_t)(s + 1) * (bins + 1);
    if (smem > (size_t)ctx->smem_optin) return ZIPML_ERR_WORKSPACE;
    cudaError_t e = cudaFuncSetAttribute(levels_dp_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return cuda_status(e);
    if (n > 0x7fffffffLL) return ZIPML_ERR_WORKSPACE;
    levels_dp_kernel<<<(unsigned)n, kDpThreads, smem, ctx->stream>>>(
        counts, bins, s, lo, hi, levels_out, reinterpret_cast<unsigned long long*>(objective_out));
    ctx->launches += 1;
    return cuda_status(cudaGetLastError());
}

}  // namespace zipml
