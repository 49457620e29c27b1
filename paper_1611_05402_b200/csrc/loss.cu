// Training loss (paper Eq. (leastsquares) with l = a^T x - b) on the dense samples, its unbiased
// estimate from the two code planes, and the allocation-free variant of the latter.
#include <mutex>

#include "common.cuh"
#include "int_digits.cuh"
#include "internal.h"

namespace zipml {

// ---------------------------------------------------------------------------------------------
// Loss estimate from the two planes: 1/(2m) sum_k (Q1(a_k)^T x - b_k)(Q2(a_k)^T x - b_k).
// A small kernel first writes w_j = step_j x_j (or the level*x table) and the base lo^T x to
// scratch; the streaming kernel then takes one row per warp.
// ---------------------------------------------------------------------------------------------
__global__ void loss_prepare_kernel(const float* __restrict__ lo, const float* __restrict__ step,
                                    const float* __restrict__ levels, const float* __restrict__ x, int64_t n, int L,
                                    bool table, float* __restrict__ wtab, double* __restrict__ base_out) {
    __shared__ double red[40];
    double base = 0.0;
    for (int64_t j = threadIdx.x; j < n; j += blockDim.x) {
        const float xv = x[j];
        if (!table) {
            wtab[j] = step[j] * xv;
            base += (double)lo[j] * (double)xv;
        } else {
            for (int c = 0; c < L; ++c) wtab[(int64_t)c * n + j] = levels[j * L + c] * xv;
        }
    }
    base = block_sum(base, red);
    if (threadIdx.x == 0) *base_out = base;
}

// w = step * x (or level * x per code) and lo^T x for a data set's grid: shared by the loss and the polynomial estimator.
int launch_code_weights(zipml_ctx* ctx, const zipml_dataset* d, const float* x, float* wtab, double* base) {
    loss_prepare_kernel<<<1, 1024, 0, ctx->stream>>>(d->feat_lo, d->feat_step, d->levels, x, d->n, 1 << d->bits,
                                                     d->level_mode == ZIPML_LEVELS_TABLE, wtab, base);
    ++ctx->launches;
    return cuda_status(cudaGetLastError());
}

template <int CB, bool TABLE>
__global__ void __launch_bounds__(256) loss_codes_kernel(const uint32_t* __restrict__ p1, const uint32_t* __restrict__ p2,
                                                         int64_t row_words, int64_t m, int64_t n,
                                                         const float* __restrict__ wtab, const double* __restrict__ base_in,
                                                         const float* __restrict__ b, double* __restrict__ partials) {
    constexpr int FPW = 32 / CB;
    __shared__ double red[40];
    const int lane = threadIdx.x & 31;
    const int64_t warp_global = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int64_t nwarps = ((int64_t)gridDim.x * blockDim.x) >> 5;
    const int64_t words = (n + FPW - 1) / FPW;
    const double base = *base_in;
    double total = 0.0;
    for (int64_t k = warp_global; k < m; k += nwarps) {
        const uint32_t* row1 = p1 + k * row_words;
        const uint32_t* row2 = p2 + k * row_words;
        double d1 = 0.0, d2 = 0.0;
        for (int64_t q0 = 0; q0 < words; q0 += 32 * 8) {
            float acc1 = 0.0f, acc2 = 0.0f;
#pragma unroll 2
            for (int s = 0; s < 8; ++s) {
                const int64_t q = q0 + s * 32 + lane;
                if (q < words) {
                    const uint32_t u1 = __ldg(row1 + q), u2 = __ldg(row2 + q);
                    if constexpr (!TABLE) {
                        float c1[FPW], c2[FPW];
                        unpack_word<CB>(u1, c1);
                        unpack_word<CB>(u2, c2);
#pragma unroll
                        for (int i = 0; i < FPW; ++i) {
                            const int64_t j = q * FPW + i;
                            const float wv = (j < n) ? __ldg(wtab + j) : 0.0f;
                            acc1 = fmaf(c1[i], wv, acc1);
                            acc2 = fmaf(c2[i], wv, acc2);
                        }
                    } else {
#pragma unroll
                        for (int i = 0; i < FPW; ++i) {
                            const int64_t j = q * FPW + i;
                            if (j < n) {
                                acc1 += __ldg(wtab + (int64_t)code_at<CB>(u1, i) * n + j);
                                acc2 += __ldg(wtab + (int64_t)code_at<CB>(u2, i) * n + j);
                            }
                        }
                    }
                }
            }
            d1 += (double)acc1;
            d2 += (double)acc2;
        }
        d1 = warp_sum(d1) + base;
        d2 = warp_sum(d2) + base;
        const double bk = (double)__ldg(b + k);
        if (lane == 0) total += (d1 - bk) * (d2 - bk);
    }
    total = block_sum(total, red);
    if (threadIdx.x == 0) partials[blockIdx.x] = total;
}

// ---------------------------------------------------------------------------------------------
// Level tables whose level * x table fits shared memory.  Every block stages a table of GROUP sums: GB bits of a
// code word (GB / CB neighbouring codes) index one entry that already holds the sum of their level * x products, so a
// word costs 32 / GB look-ups instead of 32 / CB.  Entry (group value v, group p of a word, word q of the row) sits at
// (v * NP + p) * wpad + q with wpad a multiple of 32: the lanes of a warp -- consecutive words q, whatever their codes --
// read 32 different banks.  EB is the number of index bits kept of a group (7 for byte groups of 3-bit codes in 4-bit
// fields, whose bit 7 is always clear; else GB).  A warp takes four rows at a time (their loads are in flight
// together) and folds the eight row sums with a halving butterfly.  From global memory every look-up of a warp
// touched up to 32 cache lines (426 GB/s of packed codes on 500,000 x 512 3-bit rows).
// ---------------------------------------------------------------------------------------------
constexpr int kTableRows = 4;                             // rows per warp and pass

template <int CB, int GB, int EB>
__global__ void __launch_bounds__(1024) loss_codes_table_kernel(const uint32_t* __restrict__ p1, const uint32_t* __restrict__ p2,
                                                                int64_t row_words, int64_t m, int64_t n, int L, int wpad,
                                                                const float* __restrict__ levels, const float* __restrict__ x,
                                                                const float* __restrict__ b, double* __restrict__ partials) {
    constexpr int FPW = 32 / CB, NP = 32 / GB, CPG = GB / CB, E = 1 << EB;
    extern __shared__ float tab[];                        // [E][NP][wpad], then the single products [L][n + n / 32 + 1]
    __shared__ double red[40];
    const int words = (int)((n + FPW - 1) / FPW);
    // the products level * x of single codes first (levels read in their own order), feature j of code c at
    // c * npad + j + j / 32: the group sums below read features NP * CPG apart, which that skew spreads over the banks
    float* single = tab + (size_t)E * NP * wpad;
    const int npad = (int)(n + n / 32 + 1);
    for (int64_t idx = threadIdx.x; idx < n * L; idx += blockDim.x) {
        const int j = (int)(idx / L), c = (int)(idx % L);
        single[c * npad + j + (j >> 5)] = __ldg(levels + idx) * __ldg(x + j);
    }
    __syncthreads();
    for (int vp = threadIdx.x / wpad; vp < E * NP; vp += blockDim.x / wpad) {   // (wpad divides the block size or exceeds it: see the host)
        const int p = vp % NP, v = vp / NP;
        for (int q = threadIdx.x % wpad; q < wpad; q += blockDim.x) {
            float sum = 0.0f;
#pragma unroll
            for (int s = 0; s < CPG; ++s) {
                const int c = (v >> (CB * s)) & ((1 << CB) - 1);
                const int64_t j = ((int64_t)q * NP + p) * CPG + s;
                if (c < L && q < words && j < n) sum += single[c * npad + (int)j + (int)(j >> 5)];
            }
            tab[(size_t)vp * wpad + q] = sum;
        }
    }
    __syncthreads();
    const int lane = threadIdx.x & 31;
    const int64_t warp_global = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int64_t nwarps = ((int64_t)gridDim.x * blockDim.x) >> 5;
    const int stride = NP * wpad;
    double total = 0.0;
    for (int64_t k0 = warp_global * kTableRows; k0 < m; k0 += nwarps * kTableRows) {
        const uint32_t* row1 = p1 + k0 * row_words;
        const uint32_t* row2 = p2 + k0 * row_words;
        const int nr = m - k0 < kTableRows ? (int)(m - k0) : kTableRows;   // rows past the end read as zero words
        double d[2 * kTableRows];
#pragma unroll
        for (int i = 0; i < 2 * kTableRows; ++i) d[i] = 0.0;
        for (int qb = 0; qb < words; qb += 256) {         // fp32 sums of at most 8 words' look-ups, then double
            float acc[2 * kTableRows];
#pragma unroll
            for (int i = 0; i < 2 * kTableRows; ++i) acc[i] = 0.0f;
            const int qe = words < qb + 256 ? words : qb + 256;
            for (int q = qb + lane; q < qe; q += 32) {
                uint32_t u[2 * kTableRows];
#pragma unroll
                for (int i = 0; i < 2 * kTableRows; ++i)
                    u[i] = (i >> 1) < nr ? __ldcs(((i & 1) ? row2 : row1) + (i >> 1) * row_words + q) : 0u;
                const float* tq = tab + q;
#pragma unroll
                for (int i = 0; i < 2 * kTableRows; ++i)
#pragma unroll
                    for (int p = 0; p < NP; ++p) acc[i] += tq[(int)((u[i] >> (GB * p)) & (uint32_t)(E - 1)) * stride + p * wpad];
            }
#pragma unroll
            for (int i = 0; i < 2 * kTableRows; ++i) d[i] += (double)acc[i];
        }
        // d[2 r + plane]: lanes 16.. keep rows 2, 3, then lanes with bit 3 keep the odd row; both planes of that row go on
        static_assert(kTableRows == 4, "the butterfly below folds four rows");
        const bool hi16 = lane & 16, hi8 = lane & 8;
        double w[4], z[2];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const double keep = hi16 ? d[j + 4] : d[j], send = hi16 ? d[j] : d[j + 4];
            w[j] = keep + __shfl_xor_sync(0xffffffffu, send, 16);
        }
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            const double keep = hi8 ? w[j + 2] : w[j], send = hi8 ? w[j] : w[j + 2];
            z[j] = keep + __shfl_xor_sync(0xffffffffu, send, 8);
        }
#pragma unroll
        for (int o = 4; o > 0; o >>= 1) {
            z[0] += __shfl_xor_sync(0xffffffffu, z[0], o);
            z[1] += __shfl_xor_sync(0xffffffffu, z[1], o);
        }
        const int64_t k = k0 + (hi16 ? 2 : 0) + (hi8 ? 1 : 0);
        if ((lane & 7) == 0 && k < m) {
            const double bk = (double)__ldg(b + k);
            total += (z[0] - bk) * (z[1] - bk);
        }
    }
    total = block_sum(total, red);
    if (threadIdx.x == 0) partials[blockIdx.x] = total;
}

// ---------------------------------------------------------------------------------------------
// The same estimate for uniform grids on the int8 tensor cores: a pure streaming pass (no step-to-step
// dependency), so it shows what the unpack-and-dot arithmetic of the SGD step reaches against HBM.
// w = step * x becomes four balanced base-128 int8 digits per entry (one rounding, 2^-27 of the
// largest |w|); a warp takes 16 rows, its lanes load 16 bytes of codes per row and 64-byte span
// straight from global memory (rows g and g+8 of lane group g; four lanes cover the span), and every
// 8 bytes of a lane's 16 are one mma.sync m16n8k32 (u8 x s8) against the matching 8 bytes of each
// digit's vector (digits in the byte order of the codes, so the operand's k order is simply the
// lane's own byte order).  Digit sums are exact (32-bit sums moved into 64 bits before they can
// wrap, whatever the row length); they are combined in double.
// ---------------------------------------------------------------------------------------------
// Digit vectors of w: wdig[group][digit][byte of the row], row_bytes rounded up to 64 per vector.
template <int CB>
__global__ void __launch_bounds__(1024) loss_digits_kernel(const float* __restrict__ lo, const float* __restrict__ step,
                                                           const float* __restrict__ x, int64_t n, int64_t vec_bytes,
                                                           signed char* __restrict__ wdig, double* __restrict__ base_out) {
    constexpr int NG = IntPath<CB>::NG, NS = IntPath<CB>::NS, FPW = 32 / CB;
    __shared__ double red[40];
    __shared__ float smax[32];
    double base = 0.0;
    float wm = 0.0f;
    for (int64_t j = threadIdx.x; j < n; j += blockDim.x) {
        const float xv = x[j];
        wm = fmaxf(wm, fabsf(step[j] * xv));
        base += (double)lo[j] * (double)xv;
    }
    for (int o = 16; o > 0; o >>= 1) wm = fmaxf(wm, __shfl_xor_sync(0xffffffffu, wm, o));
    if ((threadIdx.x & 31) == 0) smax[threadIdx.x >> 5] = wm;
    base = block_sum(base, red);                  // its barriers also publish smax
    float wmax = 0.0f;
    for (int w = 0; w < (int)(blockDim.x >> 5); ++w) wmax = fmaxf(wmax, smax[w]);
    const float inv = wmax > 0.0f ? (float)IntPath<CB>::QMAX / wmax : 0.0f;
    if (threadIdx.x == 0) { base_out[0] = base; base_out[1] = (double)wmax / (double)IntPath<CB>::QMAX; }
    // feature j sits in byte (j / FPW) * 4 + (j % FPW) / NG of the row, code group (j % FPW) % NG
    for (int64_t idx = threadIdx.x; idx < vec_bytes * NG; idx += blockDim.x) {
        const int64_t byte = idx / NG;
        const int g = (int)(idx - byte * NG);
        const int64_t j = (byte >> 2) * FPW + (byte & 3) * NG + g;
        int d[NS];
        balanced_digits<NS>(j < n ? __float2int_rn(step[j] * x[j] * inv) : 0, d);
#pragma unroll
        for (int s = 0; s < NS; ++s) wdig[((int64_t)g * NS + s) * vec_bytes + byte] = (signed char)d[s];
    }
}

constexpr int64_t kLossFlushSpans = 1024;

template <int CB>
__global__ void __launch_bounds__(512) loss_codes_imma_kernel(const unsigned char* __restrict__ p1, const unsigned char* __restrict__ p2,
                                                              int64_t row_bytes, int64_t m, int64_t vec_bytes,
                                                              const signed char* __restrict__ wdig, const double* __restrict__ base_in,
                                                              const float* __restrict__ b, double* __restrict__ partials) {
    constexpr int NG = IntPath<CB>::NG, NS = IntPath<CB>::NS;
    __shared__ double red[40];
    const int lane = threadIdx.x & 31, gl = lane >> 2, tl = lane & 3;
    const int64_t warp_global = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int64_t nwarps = ((int64_t)gridDim.x * blockDim.x) >> 5;
    const double base = base_in[0], delta = base_in[1];
    const int64_t nblocks = (m + 15) / 16;
    const int64_t nspans = (row_bytes + 63) / 64;
    double total = 0.0;
    for (int64_t blk = warp_global; blk < nblocks; blk += nwarps) {
        const int64_t ra = min(blk * 16 + gl, m - 1), rh = min(blk * 16 + gl + 8, m - 1);
        const unsigned char* a1 = p1 + ra * row_bytes + 16 * tl;
        const unsigned char* h1 = p1 + rh * row_bytes + 16 * tl;
        const unsigned char* a2 = p2 + ra * row_bytes + 16 * tl;
        const unsigned char* h2 = p2 + rh * row_bytes + 16 * tl;
        // A span adds at most 2 * 32 * 255 * 64 to a 32-bit digit sum: they are moved into 64-bit sums every
        // kLossFlushSpans spans (2^20 * 1024 < 2^31), so rows of any admitted length stay exact.
        long long s1[4] = {0, 0, 0, 0}, s2[4] = {0, 0, 0, 0};
        for (int64_t sp0 = 0; sp0 < nspans; sp0 += kLossFlushSpans) {
        int c1[4] = {0, 0, 0, 0}, c2[4] = {0, 0, 0, 0};
        const int64_t sp1 = min(nspans, sp0 + kLossFlushSpans);
#pragma unroll 2
        for (int64_t sp = sp0; sp < sp1; ++sp) {
            const int64_t off = sp * 64;
            uint4 ua = make_uint4(0u, 0u, 0u, 0u), uh = ua, va = ua, vh = ua;
            if (off + 16 * tl < row_bytes) {                      // rows are whole multiples of 16 bytes
                ua = __ldcs(reinterpret_cast<const uint4*>(a1 + off));
                uh = __ldcs(reinterpret_cast<const uint4*>(h1 + off));
                va = __ldcs(reinterpret_cast<const uint4*>(a2 + off));
                vh = __ldcs(reinterpret_cast<const uint4*>(h2 + off));
            }
#pragma unroll
            for (int g = 0; g < NG; ++g) {
                uint4 bd = make_uint4(0u, 0u, 0u, 0u);            // digit gl of this lane's 16 bytes
                if (gl < NS) bd = __ldg(reinterpret_cast<const uint4*>(wdig + ((int64_t)g * NS + gl) * vec_bytes + off + 16 * tl));
                mma_u8s8(c1, group_bytes<CB>(ua.x, g), group_bytes<CB>(uh.x, g), group_bytes<CB>(ua.y, g), group_bytes<CB>(uh.y, g), bd.x, bd.y);
                mma_u8s8(c1, group_bytes<CB>(ua.z, g), group_bytes<CB>(uh.z, g), group_bytes<CB>(ua.w, g), group_bytes<CB>(uh.w, g), bd.z, bd.w);
                mma_u8s8(c2, group_bytes<CB>(va.x, g), group_bytes<CB>(vh.x, g), group_bytes<CB>(va.y, g), group_bytes<CB>(vh.y, g), bd.x, bd.y);
                mma_u8s8(c2, group_bytes<CB>(va.z, g), group_bytes<CB>(vh.z, g), group_bytes<CB>(va.w, g), group_bytes<CB>(vh.w, g), bd.z, bd.w);
            }
        }
#pragma unroll
        for (int e = 0; e < 4; ++e) { s1[e] += c1[e]; s2[e] += c2[e]; }
        }
        // lane t < 2 holds digits 2t, 2t+1 of rows g (s[0], s[1]) and g+8 (s[2], s[3])
        double v[4];
#pragma unroll
        for (int e = 0; e < 2; ++e) {
            const double q1 = (double)s1[2 * e] + 128.0 * (double)s1[2 * e + 1];
            const double q2 = (double)s2[2 * e] + 128.0 * (double)s2[2 * e + 1];
            v[2 * e] = q1 + 16384.0 * __shfl_down_sync(0xffffffffu, q1, 1);
            v[2 * e + 1] = q2 + 16384.0 * __shfl_down_sync(0xffffffffu, q2, 1);
        }
        if (tl == 0) {
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                const int64_t k = blk * 16 + gl + 8 * e;
                if (k < m) {
                    const double bk = (double)__ldg(b + k);
                    total += (v[2 * e] * delta + base - bk) * (v[2 * e + 1] * delta + base - bk);
                }
            }
        }
    }
    total = block_sum(total, red);
    if (threadIdx.x == 0) partials[blockIdx.x] = total;
}

__global__ void loss_finish_kernel(const double* __restrict__ partials, int count, double scale, double* out) {
    __shared__ double red[40];
    double v = 0.0;
    for (int i = threadIdx.x; i < count; i += blockDim.x) v += partials[i];
    v = block_sum(v, red);
    if (threadIdx.x == 0) *out = v * scale;
}

int launch_loss_codes(zipml_ctx* ctx, const zipml_dataset* d, const float* b, const float* x, double* partials,
                      int max_partials, double* loss_out) {
    const int cb = container_bits(d->bits);
    const bool table = d->level_mode == ZIPML_LEVELS_TABLE;
    const int L = 1 << d->bits;
    // scratch behind the partials: base and the fixed-point unit (2 doubles), then the w table or digit vectors
    double* base = partials + max_partials;
    float* wtab = reinterpret_cast<float*>(base + 2);
    if (!table) {
        // digit vectors take (8 / cb) * 4 * roundup64(row_bytes) bytes (the caller reserved them from the stride)
        const int64_t vec_bytes = (d->row_bytes + 63) / 64 * 64;
        signed char* wdig = reinterpret_cast<signed char*>(wtab);
        int blocks = ctx->sm_count * 2;                            // 2 x 16 warps per SM, 16 rows per warp and turn
        if (blocks > max_partials) blocks = max_partials;
        const int64_t need = ((d->m + 15) / 16 + 15) / 16;
        if (blocks > need) blocks = (int)need;
#define ZIPML_LAUNCH_LI(CB_) \
    loss_digits_kernel<CB_><<<1, 1024, 0, ctx->stream>>>(d->feat_lo, d->feat_step, x, d->n, vec_bytes, wdig, base); \
    loss_codes_imma_kernel<CB_><<<blocks, 512, 0, ctx->stream>>>(d->plane1, d->plane2, d->row_bytes, d->m, vec_bytes, wdig, base, b, partials)
        if (cb == 2) { ZIPML_LAUNCH_LI(2); } else if (cb == 4) { ZIPML_LAUNCH_LI(4); } else { ZIPML_LAUNCH_LI(8); }
#undef ZIPML_LAUNCH_LI
        loss_finish_kernel<<<1, 256, 0, ctx->stream>>>(partials, blocks, 1.0 / (2.0 * (double)d->m), loss_out);
        ctx->launches += 3;
        return cuda_status(cudaGetLastError());
    }
    if (table) {
        // group sums of the level * x table in shared memory: the widest group whose table fits (padding features of
        // the last word read as zero there); none fits: the look-ups below go to global memory
        const int fpw = 32 / cb;
        const int64_t words = (d->n + fpw - 1) / fpw;
        const int64_t wpad = (words + 31) / 32 * 32;
        const int64_t room = (int64_t)ctx->smem_optin - 1024;
        const uint32_t* q1 = reinterpret_cast<const uint32_t*>(d->plane1);
        const uint32_t* q2 = reinterpret_cast<const uint32_t*>(d->plane2);
        for (int gb = 8; gb >= cb; gb >>= 1) {
            const int eb = (gb == 8 && cb == 4 && L <= 8) ? 7 : gb;
            const int64_t smem = (int64_t)sizeof(float) * (((int64_t)1 << eb) * (32 / gb) * wpad + (int64_t)L * (d->n + d->n / 32 + 1));
            if (smem > room) continue;
            // one block of 1024 threads per SM, or several of 512 where the table is small
            int per_sm = (int)((int64_t)ctx->smem_optin / (smem + 2048));
            per_sm = per_sm < 1 ? 1 : per_sm > 4 ? 4 : per_sm;
            int threads = per_sm == 1 ? 1024 : 512;
            while (wpad < threads && threads % wpad != 0) threads -= 32;   // the staging loop wants wpad | threads (or wpad >= threads)
            int blocks = ctx->sm_count * per_sm;
            if (blocks > max_partials) blocks = max_partials;
            const int64_t need = (d->m + 4 * (threads / 32) - 1) / (4 * (threads / 32));
            if (blocks > need) blocks = (int)need;
#define ZIPML_LAUNCH_LT(CB_, GB_, EB_)                                                                                     \
    do {                                                                                                                   \
        cudaError_t e_ = cudaFuncSetAttribute(loss_codes_table_kernel<CB_, GB_, EB_>,                                      \
                                              cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);                     \
        if (e_ != cudaSuccess) return cuda_status(e_);                                                                     \
        loss_codes_table_kernel<CB_, GB_, EB_><<<blocks, threads, (size_t)smem, ctx->stream>>>(                            \
            q1, q2, d->row_bytes / 4, d->m, d->n, L, (int)wpad, d->levels, x, b, partials);                                       \
    } while (0)
            if (cb == 2) { if (gb == 8) ZIPML_LAUNCH_LT(2, 8, 8); else if (gb == 4) ZIPML_LAUNCH_LT(2, 4, 4); else ZIPML_LAUNCH_LT(2, 2, 2); }
            else { if (gb == 8 && eb == 7) ZIPML_LAUNCH_LT(4, 8, 7); else if (gb == 8) ZIPML_LAUNCH_LT(4, 8, 8); else ZIPML_LAUNCH_LT(4, 4, 4); }
#undef ZIPML_LAUNCH_LT
            loss_finish_kernel<<<1, 256, 0, ctx->stream>>>(partials, blocks, 1.0 / (2.0 * (double)d->m), loss_out);
            ctx->launches += 2;
            return cuda_status(cudaGetLastError());
        }
    }
    loss_prepare_kernel<<<1, 1024, 0, ctx->stream>>>(d->feat_lo, d->feat_step, d->levels, x, d->n, L, table, wtab, base);
    ++ctx->launches;
    int blocks = ctx->sm_count * 8;
    if (blocks > max_partials) blocks = max_partials;
    const int64_t need = (d->m + 7) / 8;
    if (blocks > need) blocks = (int)need;
    const uint32_t* p1 = reinterpret_cast<const uint32_t*>(d->plane1);
    const uint32_t* p2 = reinterpret_cast<const uint32_t*>(d->plane2);
    const int64_t rw = d->row_bytes / 4;
#define ZIPML_LAUNCH_L(CB_, T_) \
    loss_codes_kernel<CB_, T_><<<blocks, 256, 0, ctx->stream>>>(p1, p2, rw, d->m, d->n, wtab, base, b, partials)
    if (cb == 2) { if (table) ZIPML_LAUNCH_L(2, true); else ZIPML_LAUNCH_L(2, false); }
    else if (cb == 4) { if (table) ZIPML_LAUNCH_L(4, true); else ZIPML_LAUNCH_L(4, false); }
    else { ZIPML_LAUNCH_L(8, false); }
#undef ZIPML_LAUNCH_L
    loss_finish_kernel<<<1, 256, 0, ctx->stream>>>(partials, blocks, 1.0 / (2.0 * (double)d->m), loss_out);
    ctx->launches += 2;
    return cuda_status(cudaGetLastError());
}

// ---------------------------------------------------------------------------------------------
// Dense loss on the original samples: one row per warp, fp32 products over runs of 32*8 elements,
// doubles across runs, lanes, warps and blocks; block partials are summed in order by one block.
// ---------------------------------------------------------------------------------------------
template <bool VEC>
__global__ void __launch_bounds__(256) loss_dense_kernel(const float* __restrict__ A, int64_t m, int64_t n, int64_t lda,
                                                         const float* __restrict__ b, const float* __restrict__ x,
                                                         double* __restrict__ partials) {
    __shared__ double red[40];
    const int lane = threadIdx.x & 31;
    const int64_t warp_global = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int64_t nwarps = ((int64_t)gridDim.x * blockDim.x) >> 5;
    double total = 0.0;
    for (int64_t k = warp_global; k < m; k += nwarps) {
        const float* row = A + k * lda;
        double d = 0.0;
        if constexpr (VEC) {
            const int64_t n4 = n >> 2;
            for (int64_t q0 = 0; q0 < n4; q0 += 32 * 8) {
                float acc = 0.0f;
#pragma unroll 4
                for (int s = 0; s < 8; ++s) {
                    const int64_t q = q0 + s * 32 + lane;
                    if (q < n4) {
                        const float4 av = __ldg(reinterpret_cast<const float4*>(row) + q);
                        const float4 xv = __ldg(reinterpret_cast<const float4*>(x) + q);
                        acc = fmaf(av.x, xv.x, acc); acc = fmaf(av.y, xv.y, acc);
                        acc = fmaf(av.z, xv.z, acc); acc = fmaf(av.w, xv.w, acc);
                    }
                }
                d += (double)acc;
            }
            for (int64_t j = (n4 << 2) + lane; j < n; j += 32) d += (double)(__ldg(row + j) * __ldg(x + j));
        } else {
            for (int64_t j0 = 0; j0 < n; j0 += 32 * 8) {
                float acc = 0.0f;
#pragma unroll 4
                for (int s = 0; s < 8; ++s) {
                    const int64_t j = j0 + s * 32 + lane;
                    if (j < n) acc = fmaf(__ldg(row + j), __ldg(x + j), acc);
                }
                d += (double)acc;
            }
        }
        d = warp_sum(d);
        const double r = d - (double)__ldg(b + k);
        if (lane == 0) total += r * r;
    }
    total = block_sum(total, red);
    if (threadIdx.x == 0) partials[blockIdx.x] = total;
}

int launch_loss_dense(zipml_ctx* ctx, const float* A, int64_t m, int64_t n, int64_t lda, const float* b, const float* x,
                      double* partials, int max_partials, double* loss_out) {
    int blocks = ctx->sm_count * 8;
    if (blocks > max_partials) blocks = max_partials;
    const int64_t need = (m + 7) / 8;
    if (blocks > need) blocks = (int)need;
    const bool vec = (lda % 4 == 0) && ((reinterpret_cast<uintptr_t>(A) & 15) == 0) && ((reinterpret_cast<uintptr_t>(x) & 15) == 0);
    if (vec) loss_dense_kernel<true><<<blocks, 256, 0, ctx->stream>>>(A, m, n, lda, b, x, partials);
    else loss_dense_kernel<false><<<blocks, 256, 0, ctx->stream>>>(A, m, n, lda, b, x, partials);
    loss_finish_kernel<<<1, 256, 0, ctx->stream>>>(partials, blocks, 1.0 / (2.0 * (double)m), loss_out);
    ctx->launches += 2;
    return cuda_status(cudaGetLastError());
}

}  // namespace zipml

namespace zipml {

// ---------------------------------------------------------------------------------------------
// Loss estimate from the two planes for callers that cannot allocate device memory.
//
// Some hosts of this library run where cudaMalloc is off limits: inside a region that must not
// synchronise the device (an allocation can), under a memory pool that owns every byte of the GPU,
// or in a real-time loop with a fixed memory budget.  zipml_loss (CODES) needs scratch -- the
// per-step table w = step*x (or level*x) and one partial sum per block -- which it takes from the
// context's workspace, allocated on demand.  This variant takes the same scratch from a fixed array
// that is part of the loaded library image instead, so it never allocates; the price is an upper
// bound on the problem size and one shared array per device.
// ---------------------------------------------------------------------------------------------
constexpr int kStaticLossPartials = 1024;
constexpr int kStaticLossTableFloats = 1 << 18;        // n (uniform) or 2^bits * n (table) must fit
constexpr size_t kStaticLossBytes = sizeof(double) * (kStaticLossPartials + 2) + sizeof(float) * kStaticLossTableFloats;

static __device__ __align__(256) unsigned char g_static_loss_scratch[kStaticLossBytes];

constexpr int kMaxDevices = 64;
struct StaticLossDevice {
    bool ready = false;
    unsigned char* scratch = nullptr;   // device address of g_static_loss_scratch on this device
    int sm_count = 0;
};
static StaticLossDevice g_static_loss_devices[kMaxDevices];
static std::mutex g_static_loss_lock;           // two host threads may make a device's first call together

// Once per device, with that device current: in host code the array's name is only a handle, the
// kernels need the device address, which cudaGetSymbolAddress returns.
static int static_loss_setup(int device, StaticLossDevice** out) {
    if (device < 0 || device >= kMaxDevices) return ZIPML_ERR_INVALID_ARG;
    StaticLossDevice& d = g_static_loss_devices[device];
    std::lock_guard<std::mutex> guard(g_static_loss_lock);
    if (!d.ready) {
        void* p = nullptr;
        cudaError_t e = cudaGetSymbolAddress(&p, g_static_loss_scratch);
        if (e != cudaSuccess) return cuda_status(e);
        e = cudaDeviceGetAttribute(&d.sm_count, cudaDevAttrMultiProcessorCount, device);
        if (e != cudaSuccess) return cuda_status(e);
        d.scratch = static_cast<unsigned char*>(p);
        d.ready = true;
    }
    *out = &d;
    return ZIPML_OK;
}

}  // namespace zipml

extern "C" int zipml_loss_codes_static(int device, void* cuda_stream, const zipml_dataset* data, const float* b,
                                       const float* x, double* loss_out) {
    using namespace zipml;
    if (!b || !x || !loss_out) return ZIPML_ERR_INVALID_ARG;
    const int bad = check_dataset(data);          // the same checks as every other entry point (plane alignment included)
    if (bad != ZIPML_OK) return bad;
    if (data->layout != ZIPML_LAYOUT_ROWS) return ZIPML_ERR_UNSUPPORTED;
    const int cb = container_bits(data->bits);
    const bool table = data->level_mode == ZIPML_LEVELS_TABLE;
    const int L = 1 << data->bits;
    const int64_t table_floats = (table ? (int64_t)L : 1) * data->n;
    if (table_floats > kStaticLossTableFloats) return ZIPML_ERR_WORKSPACE;   // beyond the fixed scratch

    int prev = -1;
    if (cudaGetDevice(&prev) != cudaSuccess) return cuda_status(cudaGetLastError());
    if (prev != device && cudaSetDevice(device) != cudaSuccess) return cuda_status(cudaGetLastError());
    StaticLossDevice* dev = nullptr;
    int rc = static_loss_setup(device, &dev);
    if (rc == ZIPML_OK) {
        cudaStream_t stream = reinterpret_cast<cudaStream_t>(cuda_stream);
        double* partials = reinterpret_cast<double*>(dev->scratch);
        double* base = partials + kStaticLossPartials;
        float* wtab = reinterpret_cast<float*>(base + 2);
        // every slot that is read is written first by this call: nothing has to start at zero
        loss_prepare_kernel<<<1, 1024, 0, stream>>>(data->feat_lo, data->feat_step, data->levels, x, data->n, L, table,
                                                    wtab, base);
        int blocks = dev->sm_count * 8;
        if (blocks > kStaticLossPartials) blocks = kStaticLossPartials;
        const int64_t need = (data->m + 7) / 8;
        if (blocks > need) blocks = (int)need;
        const uint32_t* p1 = reinterpret_cast<const uint32_t*>(data->plane1);
        const uint32_t* p2 = reinterpret_cast<const uint32_t*>(data->plane2);
        const int64_t rw = data->row_bytes / 4;
#define ZIPML_LAUNCH_SL(CB_, T_) \
    loss_codes_kernel<CB_, T_><<<blocks, 256, 0, stream>>>(p1, p2, rw, data->m, data->n, wtab, base, b, partials)
        if (cb == 2) { if (table) ZIPML_LAUNCH_SL(2, true); else ZIPML_LAUNCH_SL(2, false); }
        else if (cb == 4) { if (table) ZIPML_LAUNCH_SL(4, true); else ZIPML_LAUNCH_SL(4, false); }
        else { ZIPML_LAUNCH_SL(8, false); }
#undef ZIPML_LAUNCH_SL
        loss_finish_kernel<<<1, 256, 0, stream>>>(partials, blocks, 1.0 / (2.0 * (double)data->m), loss_out);
        rc = cuda_status(cudaGetLastError());
    }
    if (prev != device) (void)cudaSetDevice(prev);
    return rc;
}
