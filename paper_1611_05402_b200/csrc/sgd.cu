// Mini-batch SGD over double-sampled packed codes (Supplement "Double Sampling", footnote form;
// "End-to-end Quantization"), and the code-plane loss estimate.
//
// Decomposition.  A minibatch tile (B rows x n features, two planes) is cut into na feature
// parts x nb row parts; CTA (ai, bi) owns one piece for the whole call and keeps its slice of the
// model in shared memory.  Per step:
//   phase A  partial dots of the CTA's rows over its features, both planes       -> pd (global)
//   barrier  (only if na > 1)
//   phase B  residuals of its rows from all feature parts; partial gradient of its features
//            over its rows                                                         -> pg, ps (global)
//   barrier  (only if more than one CTA)
//   phase C  every CTA sums the row parts of its own features in a fixed order, applies the
//            optional gradient quantizer and updates its model slice.  CTAs that share a feature
//            part do this redundantly and reach bit-identical slices, so no model exchange and no
//            third barrier is needed.
// For a uniform grid value = lo_j + code * step_j, so with w_j = step_j * x_j
//   q^T x = sum_j lo_j x_j + sum_j code_j w_j,
//   g_j   = [ lo_j * sum_k (r1_k + r2_k) + step_j * sum_k (c1_kj r2_k + c2_kj r1_k) ] / (2 B_t),
// i.e. both phases contract raw integer codes with an fp32 vector.  Level tables use lookups into
// per-step tables level*x (phase A) and level (phase B) laid out [code][slot][word] so that a warp
// reading consecutive words is bank-conflict free.
//
// Accuracy: fp32 lane partials over short runs, combined in double across lanes, warps and CTAs.
// Determinism: every reduction has a fixed order; no floating-point atomics.
//
// The same kernel runs "stepwise" (one launch per phase, kernel boundaries as barriers, model in
// global memory) or "persistent" (one cooperative launch, bounded-spin grid barriers).
#include "common.cuh"
#include "internal.h"

namespace zipml {

constexpr int kSgdThreads = 256;
constexpr int kSgdWarps = kSgdThreads / 32;
constexpr long long kBarrierSpinLimit = 1ll << 21;

enum : int { kPhaseA = 1, kPhaseB = 2, kPhaseC = 4, kPhaseAll = 7 };

struct SgdArgs {
    const uint32_t* p1;
    const uint32_t* p2;
    int64_t row_words;      // plane stride in 32-bit words
    int64_t m, n;
    int bits;
    const float* lo;
    const float* step;
    const float* levels;
    const float* b;
    float* x;
    float* grad_out;        // null or 2n
    int64_t batch, first_step, num_steps;
    const int32_t* order;   // device copy of the batch order, or null
    float lr;
    int model_bits, grad_bits;
    uint64_t seed;
    uint32_t epoch;
    int na, nb;             // feature parts, row parts
    int wc;                 // words per feature part (multiple of 32)
    int rc;                 // rows per row part
    double* pd;             // [2][na][batch][2]   partial dots
    float* pg;              // [2][nb][na*wc*FPW]  partial code gradients (table mode: value gradients)
    double* ps;             // [2][nb]             partial sums of r1 + r2
    unsigned* barrier;      // grid barrier counter (zeroed before a persistent launch)
    DeviceStatus* status;
    int phases;             // mask of kPhase*
    int persistent;
};

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

// Bounded grid barrier: arrive with a release, spin on an acquire load.  Returns false (and records
// ZIPML_ERR_TIMEOUT) if the other CTAs do not show up within the spin limit, or if any CTA has
// already recorded an error; the caller then leaves the kernel.
__device__ __forceinline__ bool grid_barrier(unsigned* counter, unsigned target, DeviceStatus* status, int where) {
    __shared__ int s_ok;
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        atomicAdd(counter, 1u);
        int ok = 0;
        for (long long it = 0; it < kBarrierSpinLimit; ++it) {
            unsigned v;
            asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(counter) : "memory");
            if (v >= target) { ok = 1; break; }
            if ((it & 1023) == 1023) {
                if (*reinterpret_cast<volatile int*>(&status->code) != 0) break;
                __nanosleep(200);
            }
        }
        if (!ok) set_status(status, ZIPML_ERR_TIMEOUT, where);
        s_ok = ok;
    }
    __syncthreads();
    return s_ok != 0;
}

// Scale and quantizer parameters of the row-scaled stochastic quantizer (Supplement Eq. (quant2)
// with M = ||v||_2, sign-magnitude, sm = 2^(bits-1)-1 intervals).
struct VecQuant {
    float M;
    int sm;
    uint64_t seed;
    uint32_t epoch, step, stream;
    __device__ __forceinline__ float apply(float v, uint32_t coord) const {
        if (!(M > 0.0f)) return 0.0f;
        const float t = __fmul_rn(__fdiv_rn(fabsf(v), M), (float)sm);
        float fl = floorf(t);
        fl = fl > (float)(sm - 1) ? (float)(sm - 1) : fl;
        const float p = __fsub_rn(t, fl);
        const uint32_t u = vector_u24(seed, epoch, step, coord, stream);
        const uint32_t mag = (uint32_t)fl + ((__fmul_rn((float)u, 5.9604644775390625e-08f) < p) ? 1u : 0u);
        const float q = __fmul_rn(M, __fdiv_rn((float)mag, (float)sm));
        return v < 0.0f ? -q : q;
    }
};

__device__ __forceinline__ float l2_norm_smem(const float* v, int count, double* red) {
    double ss = 0.0;
    for (int i = threadIdx.x; i < count; i += kSgdThreads) ss += (double)v[i] * (double)v[i];
    return (float)sqrt(block_sum(ss, red));
}

// Shared memory plan, F = wc * FPW features per CTA:
//   red[40] double            block reductions
//   dpart[2*kSgdWarps] double per-(row, segment) partial dots when a row is split over warps
//   xs[F] float               model slice
//   tab float                 uniform: w[F], layout [u][word][4] (u-th float4 of a word);
//                             table: WL[L*F] = level*x then LV[L*F] = level, layout [code][slot][word];
//                             tab[0..F) doubles as the gradient slice in phase C
//   gred[kSgdThreads*FPW]     cross-group reduction of phase B
//   res[2*rc]                 residuals r1, r2 of the CTA's rows
template <int CB, bool TABLE>
__global__ void __launch_bounds__(kSgdThreads) sgd_kernel(const SgdArgs a) {
    constexpr int FPW = 32 / CB;
    extern __shared__ __align__(16) unsigned char s_raw[];
    const int L = 1 << a.bits;
    const int F = a.wc * FPW;
    double* red = reinterpret_cast<double*>(s_raw);
    double* dpart = red + 40;
    float* xs = reinterpret_cast<float*>(dpart + 2 * kSgdWarps);
    float* tab = xs + F;
    float* gred = tab + (TABLE ? 2 * L * F : F);
    float* res = gred + kSgdThreads * FPW;
    float* gs = tab;

    const int ai = blockIdx.x % a.na, bi = blockIdx.x / a.na;
    const int G = a.na * a.nb;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t words_needed = (a.n + FPW - 1) / FPW;
    const int64_t w0 = (int64_t)ai * a.wc;                        // first word of this feature part
    const int wcnt = (int)max((int64_t)0, min((int64_t)a.wc, words_needed - w0));
    const int64_t j0 = w0 * FPW;                                  // first feature
    const int fcnt = (int)max((int64_t)0, min((int64_t)F, a.n - j0));
    const int64_t npad = (int64_t)a.na * F;
    unsigned barriers_done = 0;

    if (a.persistent || (a.phases & (kPhaseA | kPhaseC))) {
        for (int f = threadIdx.x; f < F; f += kSgdThreads) xs[f] = (f < fcnt) ? a.x[j0 + f] : 0.0f;
    }
    if (TABLE && (a.persistent || (a.phases & kPhaseB))) {
        float* LV = tab + L * F;
        for (int idx = threadIdx.x; idx < L * F; idx += kSgdThreads) {
            const int q = idx % a.wc, ci = idx / a.wc, i = ci % FPW, c = ci / FPW;
            const int f = q * FPW + i;
            LV[idx] = (f < fcnt) ? __ldg(a.levels + (j0 + f) * L + c) : 0.0f;
        }
    }
    __syncthreads();

    for (int64_t it = a.first_step; it < a.first_step + a.num_steps; ++it) {
        const int64_t t = a.order ? (int64_t)a.order[it] : it;
        const int64_t r0 = t * a.batch;
        const int bt = (int)min(a.batch, a.m - r0);
        const int k0 = bi * a.rc;                                 // first batch-local row of this CTA
        const int rcnt = max(0, min(a.rc, bt - k0));
        const int par = (int)(it & 1);
        double* pd = a.pd + (size_t)par * a.na * a.batch * 2;
        float* pg = a.pg + (size_t)par * a.nb * npad;
        double* ps = a.ps + (size_t)par * a.nb;
        const bool last = (it == a.first_step + a.num_steps - 1);

        // ------------------------------------------------------------------ phase A: dots
        if (a.phases & kPhaseA) {
            VecQuant q3{0.0f, 1, a.seed, a.epoch, (uint32_t)it, 3u};
            if (a.model_bits > 0) { q3.M = l2_norm_smem(xs, F, red); q3.sm = (1 << (a.model_bits - 1)) - 1; }
            double base = 0.0;
            if constexpr (!TABLE) {
                for (int q = threadIdx.x; q < a.wc; q += kSgdThreads) {
#pragma unroll
                    for (int i = 0; i < FPW; ++i) {
                        const int f = q * FPW + i;
                        float xv = xs[f];
                        if (a.model_bits > 0) xv = q3.apply(xv, (uint32_t)(j0 + f));
                        float sv = 0.0f, lv = 0.0f;
                        if (f < fcnt) { sv = __ldg(a.step + j0 + f); lv = __ldg(a.lo + j0 + f); }
                        tab[((i >> 2) * a.wc + q) * 4 + (i & 3)] = sv * xv;
                        base += (double)lv * (double)xv;
                    }
                }
                base = block_sum(base, red);   // ends with a barrier: w is complete
            } else {
                for (int f = threadIdx.x; f < F; f += kSgdThreads) {
                    float xv = xs[f];
                    if (a.model_bits > 0) xv = q3.apply(xv, (uint32_t)(j0 + f));
                    const int q = f / FPW, i = f % FPW;
                    for (int c = 0; c < L; ++c) {
                        const float lv = (f < fcnt) ? __ldg(a.levels + (j0 + f) * L + c) : 0.0f;
                        tab[(c * FPW + i) * a.wc + q] = lv * xv;
                    }
                }
                __syncthreads();
            }

            // tasks = rows x segments; a row is split over S warps when the CTA has fewer rows than warps
            const int chunks = (wcnt + 31) / 32;
            int S = 1;
            if (rcnt > 0 && rcnt < kSgdWarps) S = max(1, min(chunks, kSgdWarps / rcnt));
            const int cps = (chunks + S - 1) / S;
            const int ntasks = rcnt * S;
            for (int task = warp; task < ntasks; task += kSgdWarps) {
                const int r = task / S, seg = task - r * S;
                const uint32_t* row1 = a.p1 + (r0 + k0 + r) * a.row_words + w0;
                const uint32_t* row2 = a.p2 + (r0 + k0 + r) * a.row_words + w0;
                float acc1[2] = {0.0f, 0.0f}, acc2[2] = {0.0f, 0.0f};
                const int c_end = min(chunks, (seg + 1) * cps);
#pragma unroll 2
                for (int c = seg * cps; c < c_end; ++c) {
                    const int q = c * 32 + lane;
                    if (q < wcnt) {
                        const uint32_t u1 = __ldg(row1 + q), u2 = __ldg(row2 + q);
                        if constexpr (!TABLE) {
                            float c1[FPW], c2[FPW];
                            unpack_word<CB>(u1, c1);
                            unpack_word<CB>(u2, c2);
#pragma unroll
                            for (int u = 0; u < FPW / 4; ++u) {
                                const float4 wv = *reinterpret_cast<const float4*>(tab + (u * a.wc + q) * 4);
                                acc1[u & 1] = fmaf(c1[4 * u + 0], wv.x, acc1[u & 1]);
                                acc1[u & 1] = fmaf(c1[4 * u + 1], wv.y, acc1[u & 1]);
                                acc1[u & 1] = fmaf(c1[4 * u + 2], wv.z, acc1[u & 1]);
                                acc1[u & 1] = fmaf(c1[4 * u + 3], wv.w, acc1[u & 1]);
                                acc2[u & 1] = fmaf(c2[4 * u + 0], wv.x, acc2[u & 1]);
                                acc2[u & 1] = fmaf(c2[4 * u + 1], wv.y, acc2[u & 1]);
                                acc2[u & 1] = fmaf(c2[4 * u + 2], wv.z, acc2[u & 1]);
                                acc2[u & 1] = fmaf(c2[4 * u + 3], wv.w, acc2[u & 1]);
                            }
                        } else {
#pragma unroll
                            for (int i = 0; i < FPW; ++i) {
                                acc1[i & 1] += tab[(code_at<CB>(u1, i) * FPW + i) * a.wc + q];
                                acc2[i & 1] += tab[(code_at<CB>(u2, i) * FPW + i) * a.wc + q];
                            }
                        }
                    }
                }
                const double d1 = warp_sum((double)acc1[0] + (double)acc1[1]);
                const double d2 = warp_sum((double)acc2[0] + (double)acc2[1]);
                if (lane == 0) {
                    if (S == 1) {
                        __stcg(pd + ((size_t)ai * a.batch + k0 + r) * 2 + 0, d1 + base);
                        __stcg(pd + ((size_t)ai * a.batch + k0 + r) * 2 + 1, d2 + base);
                    } else {
                        dpart[2 * task] = d1;
                        dpart[2 * task + 1] = d2;
                    }
                }
            }
            if (S > 1) {
                __syncthreads();
                if (threadIdx.x < rcnt) {
                    double d1 = base, d2 = base;
                    for (int sg = 0; sg < S; ++sg) { d1 += dpart[2 * (threadIdx.x * S + sg)]; d2 += dpart[2 * (threadIdx.x * S + sg) + 1]; }
                    __stcg(pd + ((size_t)ai * a.batch + k0 + threadIdx.x) * 2 + 0, d1);
                    __stcg(pd + ((size_t)ai * a.batch + k0 + threadIdx.x) * 2 + 1, d2);
                }
            }
        }
        if (a.persistent && a.na > 1) {
            ++barriers_done;
            if (!grid_barrier(a.barrier, (unsigned)G * barriers_done, a.status, 1)) return;
        } else {
            __syncthreads();
        }

        // ------------------------------------------------------------------ phase B: gradient
        if (a.phases & kPhaseB) {
            double ssum = 0.0;
            for (int r = threadIdx.x; r < rcnt; r += kSgdThreads) {
                double d1 = 0.0, d2 = 0.0;
                for (int p = 0; p < a.na; ++p) {
                    d1 += __ldcg(pd + ((size_t)p * a.batch + k0 + r) * 2 + 0);
                    d2 += __ldcg(pd + ((size_t)p * a.batch + k0 + r) * 2 + 1);
                }
                const double bk = (double)__ldg(a.b + r0 + k0 + r);
                const float r1 = (float)(d1 - bk), r2 = (float)(d2 - bk);
                res[2 * r] = r1;
                res[2 * r + 1] = r2;
                ssum += (double)r1 + (double)r2;
            }
            ssum = block_sum(ssum, red);       // ends with a barrier: residuals are complete
            if (threadIdx.x == 0 && ai == 0) __stcg(ps + bi, ssum);

            const int lanes_q = min(kSgdThreads, ((wcnt + 31) / 32) * 32);
            const int ngroups = lanes_q > 0 ? kSgdThreads / lanes_q : 1;
            const int group = lanes_q > 0 ? threadIdx.x / lanes_q : 0;
            const int ql = lanes_q > 0 ? threadIdx.x % lanes_q : 0;
            const float* LV = tab + L * F;
            for (int qb = 0; qb < wcnt; qb += lanes_q) {
                const int q = qb + ql;
                const bool active = (group < ngroups) && (q < wcnt);
                float acc[FPW];
#pragma unroll
                for (int i = 0; i < FPW; ++i) acc[i] = 0.0f;
                if (active) {
                    const uint32_t* col1 = a.p1 + (r0 + k0) * a.row_words + w0 + q;
                    const uint32_t* col2 = a.p2 + (r0 + k0) * a.row_words + w0 + q;
#pragma unroll 2
                    for (int r = group; r < rcnt; r += ngroups) {
                        const uint32_t u1 = __ldg(col1 + (int64_t)r * a.row_words);
                        const uint32_t u2 = __ldg(col2 + (int64_t)r * a.row_words);
                        const float r1 = res[2 * r], r2 = res[2 * r + 1];
                        if constexpr (!TABLE) {
                            float c1[FPW], c2[FPW];
                            unpack_word<CB>(u1, c1);
                            unpack_word<CB>(u2, c2);
#pragma unroll
                            for (int i = 0; i < FPW; ++i) acc[i] = fmaf(c1[i], r2, fmaf(c2[i], r1, acc[i]));
                        } else {
#pragma unroll
                            for (int i = 0; i < FPW; ++i) {
                                const float l1 = LV[(code_at<CB>(u1, i) * FPW + i) * a.wc + q];
                                const float l2 = LV[(code_at<CB>(u2, i) * FPW + i) * a.wc + q];
                                acc[i] = fmaf(l1, r2, fmaf(l2, r1, acc[i]));
                            }
                        }
                    }
                }
                if (ngroups > 1) {
                    __syncthreads();
                    if (active) {
#pragma unroll
                        for (int i = 0; i < FPW; ++i) gred[(group * FPW + i) * lanes_q + ql] = acc[i];
                    }
                    __syncthreads();
                    if (active && group == 0) {
#pragma unroll
                        for (int i = 0; i < FPW; ++i) {
                            float tsum = gred[i * lanes_q + ql];
                            for (int gidx = 1; gidx < ngroups; ++gidx) tsum += gred[(gidx * FPW + i) * lanes_q + ql];
                            acc[i] = tsum;
                        }
                    }
                }
                if (active && group == 0) {
                    float4* dst = reinterpret_cast<float4*>(pg + (size_t)bi * npad + (size_t)(w0 + q) * FPW);
#pragma unroll
                    for (int u = 0; u < FPW / 4; ++u) __stcg(dst + u, make_float4(acc[4 * u], acc[4 * u + 1], acc[4 * u + 2], acc[4 * u + 3]));
                }
            }
        }
        if (a.persistent && G > 1) {
            ++barriers_done;
            if (!grid_barrier(a.barrier, (unsigned)G * barriers_done, a.status, 2)) return;
        } else {
            __syncthreads();
        }

        // ------------------------------------------------------------------ phase C: reduce, update
        if (a.phases & kPhaseC) {
            double ssum = 0.0;
            if constexpr (!TABLE) {
                for (int p = 0; p < a.nb; ++p) ssum += __ldcg(ps + p);
            }
            const double scale = 1.0 / (2.0 * (double)bt);
            for (int f = threadIdx.x; f < F; f += kSgdThreads) {
                float g = 0.0f;
                if (f < fcnt) {
                    double acc = 0.0;
                    for (int p = 0; p < a.nb; ++p) acc += (double)__ldcg(pg + (size_t)p * npad + j0 + f);
                    if constexpr (!TABLE) acc = (double)__ldg(a.lo + j0 + f) * ssum + (double)__ldg(a.step + j0 + f) * acc;
                    g = (float)(acc * scale);
                    if (last && a.grad_out && bi == 0) a.grad_out[j0 + f] = g;
                }
                gs[f] = g;
            }
            __syncthreads();
            VecQuant q4{0.0f, 1, a.seed, a.epoch, (uint32_t)it, 4u};
            if (a.grad_bits > 0) { q4.M = l2_norm_smem(gs, F, red); q4.sm = (1 << (a.grad_bits - 1)) - 1; }
            for (int f = threadIdx.x; f < fcnt; f += kSgdThreads) {
                float g = gs[f];
                if (a.grad_bits > 0) g = q4.apply(g, (uint32_t)(j0 + f));
                if (last && a.grad_out && bi == 0) a.grad_out[a.n + j0 + f] = g;
                xs[f] = fmaf(-a.lr, g, xs[f]);
            }
            __syncthreads();
            if (!a.persistent && bi == 0)
                for (int f = threadIdx.x; f < fcnt; f += kSgdThreads) a.x[j0 + f] = xs[f];
        }
    }
    if (a.persistent && bi == 0)
        for (int f = threadIdx.x; f < fcnt; f += kSgdThreads) a.x[j0 + f] = xs[f];
}

// ---------------------------------------------------------------------------------------------
// Host side: partition plan, workspace, launches
// ---------------------------------------------------------------------------------------------
struct SgdPlan {
    int na, nb, wc, rc;
    size_t smem;
    int max_ctas;           // co-resident CTAs for the persistent launch
};

template <int CB, bool TABLE>
static size_t sgd_smem_bytes(int wc, int rc, int bits) {
    constexpr int FPW = 32 / CB;
    const size_t F = (size_t)wc * FPW, L = (size_t)1 << bits;
    size_t bytes = sizeof(double) * (40 + 2 * kSgdWarps);
    bytes += sizeof(float) * (F + (TABLE ? 2 * L * F : F) + (size_t)kSgdThreads * FPW + 2 * (size_t)rc);
    return bytes;
}

static size_t sgd_smem_any(int cb, bool table, int wc, int rc, int bits) {
    if (cb == 2) return table ? sgd_smem_bytes<2, true>(wc, rc, bits) : sgd_smem_bytes<2, false>(wc, rc, bits);
    if (cb == 4) return table ? sgd_smem_bytes<4, true>(wc, rc, bits) : sgd_smem_bytes<4, false>(wc, rc, bits);
    return sgd_smem_bytes<8, false>(wc, rc, bits);
}

static const void* sgd_kernel_ptr(int cb, bool table) {
    if (cb == 2) return table ? (const void*)sgd_kernel<2, true> : (const void*)sgd_kernel<2, false>;
    if (cb == 4) return table ? (const void*)sgd_kernel<4, true> : (const void*)sgd_kernel<4, false>;
    return (const void*)sgd_kernel<8, false>;
}

static int round_up(int v, int q) { return (v + q - 1) / q * q; }

// Chooses the CTA grid.  Feature parts are the fewest that fit shared memory unless the exchange
// volume (na * 2B doubles of dots + nb * n floats of gradient per step) says otherwise; row parts
// fill the remaining CTAs while every CTA keeps at least a warp's worth of rows.
static int make_plan(const zipml_ctx* ctx, const zipml_dataset* d, const zipml_sgd_params* p, SgdPlan* plan) {
    const int cb = container_bits(d->bits);
    const bool table = d->level_mode == ZIPML_LEVELS_TABLE;
    const int fpw = 32 / cb;
    const int64_t words = (d->n + fpw - 1) / fpw;
    const int64_t B = p->batch < d->m ? p->batch : d->m;
    const size_t smem_cap = (size_t)ctx->smem_optin;
    const bool need_full = p->model_bits > 0 || p->grad_bits > 0;
    const int sms = ctx->sm_count > 0 ? ctx->sm_count : 1;

    auto fits = [&](int na, int nb, int* wc_out, int* rc_out, size_t* smem_out) {
        const int wc = round_up((int)((words + na - 1) / na), 32);
        const int rc = (int)((B + nb - 1) / nb);
        const size_t s = sgd_smem_any(cb, table, wc, rc, d->bits);
        *wc_out = wc; *rc_out = rc; *smem_out = s;
        return s <= smem_cap;
    };
    int best_na = 0, best_nb = 0;
    if (p->grid_feature_parts > 0 || p->grid_row_parts > 0) {
        best_na = p->grid_feature_parts > 0 ? p->grid_feature_parts : 1;
        best_nb = p->grid_row_parts > 0 ? p->grid_row_parts : 1;
        if ((int64_t)best_na * 32 > round_up((int)words, 32)) best_na = (int)((words + 31) / 32);
        if (best_nb > B) best_nb = (int)B;
    } else {
        double best_cost = 0.0;
        const int na_max = (int)((words + 31) / 32);
        for (int na = 1; na <= na_max && na <= sms; ++na) {
            if (need_full && na > 1) break;
            int nb = sms / na;
            const int64_t nb_rows = (B + kSgdWarps - 1) / kSgdWarps;     // at least a warp's worth of rows each
            if (nb > nb_rows) nb = (int)nb_rows;
            if (nb < 1) nb = 1;
            int wc, rc; size_t s;
            if (!fits(na, nb, &wc, &rc, &s)) continue;
            // per-step critical path model: streamed bytes per CTA + exchanged bytes + barrier count
            const double tile = 2.0 * (double)rc * wc * 4.0;
            const double exch = (na > 1 ? (double)na * 2.0 * (double)B * 8.0 : 0.0) + (double)nb * (double)d->n * 4.0 / na;
            const double cost = tile + 0.25 * exch + (na > 1 ? 65536.0 : 0.0);
            if (best_na == 0 || cost < best_cost) { best_cost = cost; best_na = na; best_nb = nb; }
        }
        if (best_na == 0) return ZIPML_ERR_WORKSPACE;
    }
    if (need_full && best_na > 1) return ZIPML_ERR_WORKSPACE;
    int wc, rc; size_t s;
    if (!fits(best_na, best_nb, &wc, &rc, &s)) return ZIPML_ERR_WORKSPACE;
    plan->na = best_na; plan->nb = best_nb; plan->wc = wc; plan->rc = rc; plan->smem = s;
    plan->max_ctas = 0;
    return ZIPML_OK;
}

struct SgdScratch {
    size_t pd_off, pg_off, ps_off, bar_off, order_off, total;
};

static SgdScratch sgd_scratch(const zipml_dataset* d, const zipml_sgd_params* p, const SgdPlan& plan, int64_t T) {
    const int fpw = 32 / container_bits(d->bits);
    const int64_t B = p->batch < d->m ? p->batch : d->m;
    SgdScratch s;
    size_t off = 0;
    s.pd_off = off; off += carve_size(sizeof(double) * 2 * (size_t)plan.na * (size_t)B * 2);
    s.pg_off = off; off += carve_size(sizeof(float) * 2 * (size_t)plan.nb * (size_t)plan.na * plan.wc * fpw);
    s.ps_off = off; off += carve_size(sizeof(double) * 2 * (size_t)plan.nb);
    s.bar_off = off; off += carve_size(sizeof(unsigned) * 4);
    s.order_off = off; off += carve_size(sizeof(int32_t) * (size_t)(p->batch_order ? T : 0));
    s.total = off;
    return s;
}

size_t sgd_workspace_bytes(const zipml_ctx* ctx, const zipml_dataset* d, const zipml_sgd_params* p) {
    SgdPlan plan;
    if (make_plan(ctx, d, p, &plan) != ZIPML_OK) return 0;
    const int64_t T = (d->m + p->batch - 1) / p->batch;
    return sgd_scratch(d, p, plan, T).total;
}

int launch_sgd_epoch(zipml_ctx* ctx, const zipml_dataset* d, const float* b, float* x, const zipml_sgd_params* p,
                     int64_t first_step, int64_t num_steps, float* grad_out) {
    SgdPlan plan;
    int rc = make_plan(ctx, d, p, &plan);
    if (rc != ZIPML_OK) return rc;
    const int cb = container_bits(d->bits);
    const bool table = d->level_mode == ZIPML_LEVELS_TABLE;
    const int64_t T = (d->m + p->batch - 1) / p->batch;
    const SgdScratch sc = sgd_scratch(d, p, plan, T);
    rc = ws_reserve(ctx, sc.total);
    if (rc != ZIPML_OK) return rc;

    const void* kernel = sgd_kernel_ptr(cb, table);
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)plan.smem);
    if (e != cudaSuccess) return cuda_status(e);
    int per_sm = 0;
    e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, kSgdThreads, plan.smem);
    if (e != cudaSuccess) return cuda_status(e);
    const int G = plan.na * plan.nb;
    const bool can_persist = ctx->cooperative && per_sm > 0 && G <= per_sm * ctx->sm_count;
    int engine = p->engine;
    if (engine == ZIPML_ENGINE_AUTO) engine = can_persist ? ZIPML_ENGINE_PERSISTENT : ZIPML_ENGINE_STEPWISE;
    if (engine == ZIPML_ENGINE_PERSISTENT && !can_persist) return ZIPML_ERR_WORKSPACE;

    SgdArgs a;
    a.p1 = reinterpret_cast<const uint32_t*>(d->plane1);
    a.p2 = reinterpret_cast<const uint32_t*>(d->plane2);
    a.row_words = d->row_bytes / 4;
    a.m = d->m; a.n = d->n; a.bits = d->bits;
    a.lo = d->feat_lo; a.step = d->feat_step; a.levels = d->levels;
    a.b = b; a.x = x; a.grad_out = grad_out;
    a.batch = p->batch < d->m ? p->batch : d->m;
    if (p->batch >= d->m) a.batch = d->m;
    a.lr = p->lr; a.model_bits = p->model_bits; a.grad_bits = p->grad_bits;
    a.seed = p->seed; a.epoch = (uint32_t)p->epoch;
    a.na = plan.na; a.nb = plan.nb; a.wc = plan.wc; a.rc = plan.rc;
    a.pd = reinterpret_cast<double*>(ctx->ws + sc.pd_off);
    a.pg = reinterpret_cast<float*>(ctx->ws + sc.pg_off);
    a.ps = reinterpret_cast<double*>(ctx->ws + sc.ps_off);
    a.barrier = reinterpret_cast<unsigned*>(ctx->ws + sc.bar_off);
    a.status = ctx->d_status;
    a.order = nullptr;
    if (p->batch_order) {
        int32_t* dev_order = reinterpret_cast<int32_t*>(ctx->ws + sc.order_off);
        e = cudaMemcpyAsync(dev_order, p->batch_order, sizeof(int32_t) * (size_t)T, cudaMemcpyHostToDevice, ctx->stream);
        if (e != cudaSuccess) return cuda_status(e);
        a.order = dev_order;
    }

    if (engine == ZIPML_ENGINE_PERSISTENT) {
        // barrier targets are 32-bit: at most 2 barriers per step and G arrivals per barrier
        const int64_t max_steps = (int64_t)(0x7fffffffLL / (2LL * G));
        for (int64_t s0 = first_step; s0 < first_step + num_steps; s0 += max_steps) {
            e = cudaMemsetAsync(a.barrier, 0, sizeof(unsigned) * 4, ctx->stream);
            if (e != cudaSuccess) return cuda_status(e);
            a.first_step = s0;
            a.num_steps = (first_step + num_steps - s0 < max_steps) ? first_step + num_steps - s0 : max_steps;
            a.phases = kPhaseAll; a.persistent = 1;
            SgdArgs last_chunk_args = a;
            if (s0 + a.num_steps < first_step + num_steps) last_chunk_args.grad_out = nullptr;
            void* params[] = {&last_chunk_args};
            e = cudaLaunchCooperativeKernel(kernel, dim3((unsigned)G), dim3(kSgdThreads), params, plan.smem, ctx->stream);
            if (e != cudaSuccess) return cuda_status(e);
            ctx->launches += 1;
        }
        return ZIPML_OK;
    }

    a.persistent = 0;
    for (int64_t s = first_step; s < first_step + num_steps; ++s) {
        a.first_step = s; a.num_steps = 1;
        SgdArgs step_args = a;
        if (s != first_step + num_steps - 1) step_args.grad_out = nullptr;
        for (int ph : {kPhaseA, kPhaseB, kPhaseC}) {
            step_args.phases = ph;
            void* params[] = {&step_args};
            e = cudaLaunchKernel(kernel, dim3((unsigned)G), dim3(kSgdThreads), params, plan.smem, ctx->stream);
            if (e != cudaSuccess) return cuda_status(e);
            ctx->launches += 1;
        }
    }
    return ZIPML_OK;
}

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
    // scratch behind the partials: base (1 double) then the w table
    double* base = partials + max_partials;
    float* wtab = reinterpret_cast<float*>(base + 2);
    loss_prepare_kernel<<<1, 1024, 0, ctx->stream>>>(d->feat_lo, d->feat_step, d->levels, x, d->n, L, table, wtab, base);
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
    ctx->launches += 3;
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

// Once per device, with that device current: in host code the array's name is only a handle, the
// kernels need the device address, which cudaGetSymbolAddress returns.
static int static_loss_setup(int device, StaticLossDevice** out) {
    if (device < 0 || device >= kMaxDevices) return ZIPML_ERR_INVALID_ARG;
    StaticLossDevice& d = g_static_loss_devices[device];
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
    if (!data || data->struct_size != sizeof(zipml_dataset) || !b || !x || !loss_out) return ZIPML_ERR_INVALID_ARG;
    const int cb = container_bits(data->bits);
    if (cb == 0) return ZIPML_ERR_UNSUPPORTED;
    const bool table = data->level_mode == ZIPML_LEVELS_TABLE;
    if (!table && data->level_mode != ZIPML_LEVELS_UNIFORM) return ZIPML_ERR_INVALID_ARG;
    if (table && data->bits == 8) return ZIPML_ERR_UNSUPPORTED;
    if (data->m <= 0 || data->n <= 0 || !data->plane1 || !data->plane2) return ZIPML_ERR_INVALID_ARG;
    if (data->row_bytes % 16 != 0 || data->row_bytes < zipml_row_bytes(data->n, data->bits)) return ZIPML_ERR_INVALID_ARG;
    if (table ? !data->levels : (!data->feat_lo || !data->feat_step)) return ZIPML_ERR_INVALID_ARG;
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
