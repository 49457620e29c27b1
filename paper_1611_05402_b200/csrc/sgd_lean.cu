// Lean engine of zipml_sgd_epoch: one persistent cooperative launch per call, built for steps
// whose code tile is small (Supplement "Double Sampling", footnote form; "End-to-end Quantization").
//
// When a minibatch holds a few hundred kilobytes of codes a step is not bound by HBM but by the
// chain  dots -> residuals -> partial gradients -> sum over the CTAs -> update -> new model at
// every CTA, which every step has to walk once.  Measured on B200: straight-line code whose
// footprint exceeds about 32 KB issues at about six cycles per instruction and warp (the
// instruction cache streams it from L2 every time round), and a CTA-wide barrier, an L2 round
// trip and a store becoming visible to another SM cost about 30, 300 and 420 cycles.  So this
// kernel is written for few instructions, few barriers and two exchanges per step:
//   * the minibatch is cut into nb row parts, one CTA each; a CTA sees whole rows, so a row's two
//     dots are complete inside one warp and the residuals never leave the CTA;
//   * all arithmetic on codes is fp32 FMA on unpacked codes in tight rolled loops, sums across
//     lanes, warps and CTAs are taken in double in a fixed order (results do not depend on timing);
//   * the code tiles do not depend on the model: one thread keeps bulk asynchronous copies
//     (cp.async.bulk + mbarrier transaction counts) several steps ahead in a ring of shared-memory
//     slots, one contiguous copy per plane and step;
//   * exchange by self-validating packets {fp32 value, step tag} written with one 64-bit store and
//     polled by their readers (no grid barrier, no fence): every CTA sends, for each feature, its
//     rows' part of the gradient to the feature's owner ([feature][writer] layout, so an owner reads
//     a contiguous run); the owner -- a group of P lanes per feature -- adds the nb parts, applies
//     the optional gradient quantizer and the update to the master value it keeps in shared
//     memory, and publishes what the next step sees (Q3 of it when the model quantizer is on);
//     every CTA collects that vector and turns it into w = step * x~ (or the level-times-model
//     table).  The first model takes the same route: the loop starts with a publish-only round.
//   A packet of step t is overwritten only after everything of step t that its readers needed has
//   been collected (the next write of a partial gradient follows the writer's collection of the
//   model, which the owner publishes after reading; the next publication follows the collection
//   of all partial gradients of the next step), so single buffers suffice.
// Every wait is bounded: when one gives up it records ZIPML_ERR_TIMEOUT, later waits of that CTA
// are skipped and the CTA still sends and publishes, so the launch always ends.
#include <string.h>

#include "sgd_common.cuh"

namespace zipml {

constexpr int kLeanThreads = 256;
constexpr int kLeanWarps = kLeanThreads / 32;
constexpr int kLeanMaxSlots = 8;
constexpr long long kLeanSpinLimit = 1ll << 22;

struct LeanArgs {
    const uint32_t* p1;
    const uint32_t* p2;
    const float* lo;
    const float* step;
    const float* levels;
    const float* b;
    float* x;
    float* grad_out;             // null or 2n
    float* model_out;            // null or n: the model the last executed step's gradient saw
    const int32_t* order;        // device copy of the batch order, or null
    unsigned long long* rs;      // [n][nb]   partial gradients, per feature the nb writers
    unsigned long long* ag;      // [n]       the model the next step sees
    unsigned long long* gn;      // [nb][2]   partial squared gradient norms (hi, lo)
    unsigned long long* xn;      // [nb][2]   partial squared model norms (hi, lo)
    unsigned long long* trace;
    DeviceStatus* status;
    int64_t m, batch, first_step, num_steps;
    uint64_t seed;
    uint32_t epoch;
    float lr;
    int reg;                     // ZIPML_REG_* and its fp32 constant
    float reg_cst;
    int n, bits, row_words, words;   // words = ceil(n / codes per word) <= row_words
    int model_bits, grad_bits;
    int nb, rc, slots;
    int sub_shift;               // a CTA owns 2^sub_shift consecutive features
    int p_shift;                 // 2^p_shift lanes share the sum of one owned feature
    int trace_steps;
};

struct LeanShared {
    double red[kLeanWarps];      // block sums
    double wbase[kLeanWarps];    // per-warp parts of lo^T x~
    double ssum[kLeanWarps];     // per-warp sums of the residuals
    unsigned long long full[kLeanMaxSlots];
    int abort_flag;
    int pad;
};

__device__ __forceinline__ void lean_store(unsigned long long* p, float v, uint32_t tag) {
    __stcg(p, ((unsigned long long)tag << 32) | (unsigned long long)__float_as_uint(v));
}
__device__ __forceinline__ unsigned long long lean_load(const unsigned long long* p) {
    unsigned long long v;
    asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}

// Polls up to four packets (p[0], p[stride], ...; the first `cnt`) until each carries `tag`.
__device__ __forceinline__ void lean_poll4(const unsigned long long* p, int stride, int cnt, uint32_t tag, float (&v)[4],
                                           LeanShared* sh, DeviceStatus* status, int where) {
    unsigned long long w[4] = {0, 0, 0, 0};
    bool ok = false;
    if (!*reinterpret_cast<volatile int*>(&sh->abort_flag)) {
#pragma unroll 1
        for (long long spin = 0; spin < kLeanSpinLimit && !ok; ++spin) {
            ok = true;
#pragma unroll
            for (int u = 0; u < 4; ++u)
                if (u < cnt) { w[u] = lean_load(p + (size_t)u * stride); ok = ok && ((uint32_t)(w[u] >> 32) == tag); }
            if (!ok && spin >= 32) __nanosleep(64);
        }
        if (!ok) { sh->abort_flag = 1; set_status(status, ZIPML_ERR_TIMEOUT, where); }
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) v[u] = (ok && u < cnt) ? __uint_as_float((uint32_t)w[u]) : 0.0f;
}

// l2 norm of a vector whose squared entries are spread over the threads of all CTAs: block sum,
// one packet pair per CTA, every warp adds the nb pairs in the same order.
__device__ __noinline__ float lean_norm(double v, unsigned long long* buf, uint32_t tag, int nb, LeanShared* sh,
                                        DeviceStatus* status, int where) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    v = warp_sum(v);
    __syncthreads();
    if (lane == 0) sh->red[warp] = v;
    __syncthreads();
    if (threadIdx.x == 0) {
        double t = 0.0;
        for (int w = 0; w < kLeanWarps; ++w) t += sh->red[w];
        const float hi = (float)t;
        lean_store(buf + 2 * (size_t)blockIdx.x, hi, tag);
        lean_store(buf + 2 * (size_t)blockIdx.x + 1, (float)(t - (double)hi), tag);
    }
    double part = 0.0;                                              // all 2*nb packets, hi and lo parts alike
#pragma unroll 1
    for (int i0 = lane; i0 < 2 * nb; i0 += 128) {
        float h[4];
        lean_poll4(buf + i0, 32, min(4, (2 * nb - i0 + 31) >> 5), tag, h, sh, status, where);
        part += ((double)h[0] + (double)h[1]) + ((double)h[2] + (double)h[3]);
    }
    return (float)sqrt(warp_sum(part));
}

__device__ __noinline__ float lean_quant(float v, float M, int sm, uint64_t seed, uint32_t epoch, uint32_t step,
                                         uint32_t stream, uint32_t coord) {
    VecQuant q{M, sm, seed, epoch, step, stream};
    return q.apply(v, coord);
}

__device__ __forceinline__ void lean_mark(const LeanArgs& a, int64_t it, int id) {
    if (a.trace && blockIdx.x == 0 && threadIdx.x == 0 && it >= a.first_step && it - a.first_step < a.trace_steps) {
        unsigned long long t;
        asm volatile("mov.u64 %0, %clock64;" : "=l"(t));
        a.trace[(it - a.first_step) * 8 + id] = t;
    }
}

// Shared memory after LeanShared, Fp = row_words * FPW (feature slots of a row, padding included):
//   uniform: wv[Fp]  w = step * x~, [slot i][word q];  los[Fp], steps[Fp]  lo and step by feature
//   table:   tab[L*Fp] level * x~ and lev[L*Fp] levels, both [code][slot i][word q]
//   xown[sub]        master model of the owned features;  gsub[sub]  their gradient of the current step
//   res[2*rc]        residuals (r1, r2) per row
//   gred[256*FPW]    cross-group sums of phase B (parts narrower than the CTA)
//   ring[slots][2][rc][row_words]  code tiles
template <int CB, bool TABLE>
__global__ void __launch_bounds__(kLeanThreads, 1) sgd_lean_kernel(const LeanArgs a) {
    constexpr int FPW = 32 / CB;
    constexpr int LOGF = (CB == 8) ? 2 : (CB == 4) ? 3 : 4;
    extern __shared__ __align__(16) unsigned char s_raw[];
    LeanShared* sh = reinterpret_cast<LeanShared*>(s_raw);
    const int rw = a.row_words, nw = a.words, n = a.n;
    const int Fp = rw * FPW;
    const int L = 1 << a.bits;
    const int sub = 1 << a.sub_shift;
    float* tab = reinterpret_cast<float*>(s_raw + ((sizeof(LeanShared) + 15) & ~(size_t)15));
    float* wv = tab;                                     // uniform
    float* los = tab + Fp;
    float* steps = los + Fp;
    float* lev = tab + (size_t)L * Fp;                   // table
    float* xown = tab + (TABLE ? 2 * (size_t)L * Fp : 3 * (size_t)Fp);
    float* gsub = xown + ((sub + 3) & ~3);
    float* res = gsub + ((sub + 3) & ~3);
    float* gred = res + ((2 * a.rc + 3) & ~3);
    uint32_t* ring = reinterpret_cast<uint32_t*>(
        (reinterpret_cast<uintptr_t>(gred + kLeanThreads * FPW) + 127) & ~(uintptr_t)127);
    const size_t slot_words = (size_t)2 * a.rc * rw;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int bi = blockIdx.x, nb = a.nb;
    const int k0 = bi * a.rc;
    const int64_t step_end = a.first_step + a.num_steps;

    auto step_rows = [&](int64_t it, int64_t& r0, int& bt, int& rcnt) {
        const int64_t t = a.order ? (int64_t)a.order[it] : it;
        r0 = t * a.batch;
        bt = (int)min(a.batch, a.m - r0);
        rcnt = max(0, min(a.rc, bt - k0));
    };
    // the tile of step `it` into its slot: one contiguous piece per plane (thread 0 only)
    auto issue_tile = [&](int64_t it, int slot) {
        int64_t r0; int bt, rcnt;
        step_rows(it, r0, bt, rcnt);
        uint64_t* full = reinterpret_cast<uint64_t*>(sh->full + slot);
        const uint32_t bytes = (uint32_t)rcnt * (uint32_t)rw * 4u;
        mbar_arrive_expect_tx(full, 2u * bytes);
        if (rcnt > 0) {
            uint32_t* dst = ring + (size_t)slot * slot_words;
            const size_t src = (size_t)(r0 + k0) * rw;
            bulk_copy_g2s(dst, a.p1 + src, bytes, full);
            bulk_copy_g2s(dst + (size_t)a.rc * rw, a.p2 + src, bytes, full);
        }
    };

    if (tid == 0) {
        for (int s = 0; s < a.slots; ++s) mbar_init(reinterpret_cast<uint64_t*>(sh->full + s), 1);
        sh->abort_flag = 0;
        mbar_fence_init();
    }
    for (int f = tid; f < Fp; f += kLeanThreads) {
        const int q = f >> LOGF, i = f & (FPW - 1);
        if constexpr (TABLE) {
            for (int c = 0; c < L; ++c) lev[(c * FPW + i) * rw + q] = (f < n) ? __ldg(a.levels + (size_t)f * L + c) : 0.0f;
        } else {
            los[f] = (f < n) ? __ldg(a.lo + f) : 0.0f;
            steps[f] = (f < n) ? __ldg(a.step + f) : 0.0f;
        }
    }
    for (int k = tid; k < sub; k += kLeanThreads) xown[k] = (bi * sub + k < n) ? a.x[bi * sub + k] : 0.0f;
    __syncthreads();
    if (tid == 0)
        for (int s = 0; s + 1 < a.slots && a.first_step + s < step_end; ++s) issue_tile(a.first_step + s, s);

    // thread roles: owner group of P lanes per owned feature; word column and row group of phase B
    const int P = 1 << a.p_shift;
    const int pp = tid & (P - 1);
    const int kpt = kLeanThreads >> a.p_shift;                     // owned features handled per pass
    const int lanes_q = min(kLeanThreads, ((nw + 31) / 32) * 32);
    const int ngroups = kLeanThreads / lanes_q;
    const int group = tid / lanes_q, ql = tid - group * lanes_q;

    int slot = 0;                                                  // slot and mbarrier parity of the current step's tile
    uint32_t parity = 0;
    for (int64_t it = a.first_step - 1; it < step_end; ++it) {
        const uint32_t tag = (uint32_t)(it - a.first_step) + 2u;   // the publish-only round uses 1
        const bool last = (it == step_end - 1);
        float gq_M = 0.0f;                                         // Q4 scale of this step
        if (it >= a.first_step) {
            lean_mark(a, it, 0);
            // refill the slot of the previous step: every thread has passed the barrier that closed it
            if (tid == 0 && it + a.slots - 1 < step_end) issue_tile(it + a.slots - 1, slot == 0 ? a.slots - 1 : slot - 1);
            int64_t r0; int bt, rcnt;
            step_rows(it, r0, bt, rcnt);
            if (!*reinterpret_cast<volatile int*>(&sh->abort_flag)) {
                bool ok = false;
#pragma unroll 1
                for (long long spin = 0; spin < kCopySpinLimit && !ok; ++spin)
                    ok = mbar_try_wait(reinterpret_cast<uint64_t*>(sh->full + slot), parity);
                if (!ok) { sh->abort_flag = 1; set_status(a.status, ZIPML_ERR_TIMEOUT, 6); }
            }
            const uint32_t* t1 = ring + (size_t)slot * slot_words;
            const uint32_t* t2 = t1 + (size_t)a.rc * rw;
            lean_mark(a, it, 1);

            // ---------------------------------------------------------- phase A: dots and residuals
            double base = 0.0;                                     // lo^T x~ (uniform grids)
            if constexpr (!TABLE) {
#pragma unroll
                for (int w = 0; w < kLeanWarps; ++w) base += sh->wbase[w];
            }
            double srow = 0.0;
#pragma unroll 1
            for (int r = warp; r < rcnt; r += kLeanWarps) {
                const float bl = __ldg(a.b + r0 + k0 + r);
                const uint32_t* row1 = t1 + (size_t)r * rw;
                const uint32_t* row2 = t2 + (size_t)r * rw;
                float acc1 = 0.0f, acc2 = 0.0f;
#pragma unroll 1
                for (int q = lane; q < nw; q += 32) {
                    const uint32_t u1 = row1[q], u2 = row2[q];
                    if constexpr (!TABLE) {
                        float c1[FPW], c2[FPW];
                        unpack_word<CB>(u1, c1);
                        unpack_word<CB>(u2, c2);
#pragma unroll
                        for (int i = 0; i < FPW; ++i) {
                            const float w = wv[i * rw + q];
                            acc1 = fmaf(c1[i], w, acc1);
                            acc2 = fmaf(c2[i], w, acc2);
                        }
                    } else {
#pragma unroll
                        for (int i = 0; i < FPW; ++i) {
                            acc1 += tab[(code_at<CB>(u1, i) * FPW + i) * rw + q];
                            acc2 += tab[(code_at<CB>(u2, i) * FPW + i) * rw + q];
                        }
                    }
                }
                const double d1 = warp_sum((double)acc1), d2 = warp_sum((double)acc2);
                if (lane == 0) {
                    const float r1 = (float)(d1 + base - (double)bl), r2 = (float)(d2 + base - (double)bl);
                    res[2 * r] = r1;
                    res[2 * r + 1] = r2;
                    srow += (double)r1 + (double)r2;
                }
            }
            if (lane == 0) sh->ssum[warp] = srow;
            __syncthreads();
            lean_mark(a, it, 2);

            // ---------------------------------------------------------- phase B: the rows' part of the gradient
            double S = 0.0;                                        // sum of r1 + r2 over the CTA's rows
            if constexpr (!TABLE) {
#pragma unroll
                for (int w = 0; w < kLeanWarps; ++w) S += sh->ssum[w];
            }
#pragma unroll 1
            for (int q0 = 0; q0 < nw; q0 += lanes_q) {
                const int q = q0 + ql;
                const bool active = group < ngroups && q < nw;
                float acc[FPW];
#pragma unroll
                for (int i = 0; i < FPW; ++i) acc[i] = 0.0f;
                if (active) {
#pragma unroll 1
                    for (int r = group; r < rcnt; r += ngroups) {
                        const uint32_t u1 = t1[(size_t)r * rw + q], u2 = t2[(size_t)r * rw + q];
                        const float2 rv = *reinterpret_cast<const float2*>(res + 2 * r);
                        if constexpr (!TABLE) {
                            float c1[FPW], c2[FPW];
                            unpack_word<CB>(u1, c1);
                            unpack_word<CB>(u2, c2);
#pragma unroll
                            for (int i = 0; i < FPW; ++i) acc[i] = fmaf(c1[i], rv.y, fmaf(c2[i], rv.x, acc[i]));
                        } else {
#pragma unroll
                            for (int i = 0; i < FPW; ++i) {
                                const float l1 = lev[(code_at<CB>(u1, i) * FPW + i) * rw + q];
                                const float l2 = lev[(code_at<CB>(u2, i) * FPW + i) * rw + q];
                                acc[i] = fmaf(l1, rv.y, fmaf(l2, rv.x, acc[i]));
                            }
                        }
                    }
                }
                // the groups' sums meet in shared memory ([group][feature of the pass]); then one thread per
                // feature adds them in order and sends the feature's packet
                if (q0 > 0) __syncthreads();
                if (active) {
#pragma unroll
                    for (int i = 0; i < FPW; ++i) gred[(group * lanes_q + ql) * FPW + i] = acc[i];
                }
                __syncthreads();
#pragma unroll 1
                for (int fl = tid; fl < lanes_q * FPW; fl += kLeanThreads) {
                    const int f = q0 * FPW + fl;
                    if (f < n) {
                        float v = gred[fl];
                        for (int g = 1; g < ngroups; ++g) v += gred[g * lanes_q * FPW + fl];
                        if constexpr (!TABLE) v = (float)((double)los[f] * S + (double)steps[f] * (double)v);
                        lean_store(a.rs + (size_t)f * nb + bi, v, tag);
                    }
                }
            }
            if (++slot == a.slots) { slot = 0; parity ^= 1u; }
            lean_mark(a, it, 3);

            // ---------------------------------------------------------- owners: sum the parts, update
            const double scale = 1.0 / (2.0 * (double)bt);
            double gsq = 0.0;
#pragma unroll 1
            for (int kb = 0; kb < sub; kb += kpt) {
                const int k = kb + (tid >> a.p_shift);
                const int f = bi * sub + k;
                const bool mine = k < sub && f < n;
                double t = 0.0;
                if (mine) {
                    const unsigned long long* src = a.rs + (size_t)f * nb;
#pragma unroll 1
                    for (int w0 = pp; w0 < nb; w0 += 4 * P) {
                        float v[4];
                        const int cnt = min(4, (nb - w0 + P - 1) >> a.p_shift);
                        lean_poll4(src + w0, P, cnt, tag, v, sh, a.status, 2);
                        t += ((double)v[0] + (double)v[1]) + ((double)v[2] + (double)v[3]);
                    }
                }
                for (int o = 1; o < P; o <<= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
                if (mine && pp == 0) {
                    const float g = (float)(t * scale);
                    if (last && a.grad_out) a.grad_out[f] = g;
                    gsub[k] = g;
                    gsq += (double)g * (double)g;
                }
            }
            lean_mark(a, it, 4);
            if (a.grad_bits > 0) gq_M = lean_norm(gsq, a.gn, tag, nb, sh, a.status, 3);
#pragma unroll 1
            for (int kb = 0; kb < sub; kb += kpt) {
                const int k = kb + (tid >> a.p_shift);
                const int f = bi * sub + k;
                if (k < sub && f < n && pp == 0) {
                    float g = gsub[k];
                    if (a.grad_bits > 0)
                        g = lean_quant(g, gq_M, (1 << (a.grad_bits - 1)) - 1, a.seed, a.epoch, (uint32_t)it, 4u, (uint32_t)f);
                    if (last && a.grad_out) a.grad_out[n + f] = g;
                    xown[k] = regularise(fmaf(-a.lr, g, xown[k]), xown[k], a.reg, a.reg_cst);
                }
            }
        }
        if (last) break;

        // -------------------------------------------------------------- publish what the next step sees
        float xq_M = 0.0f;
        if (a.model_bits > 0) {
            double xsq = 0.0;
            for (int kb = 0; kb < sub; kb += kpt) {
                const int k = kb + (tid >> a.p_shift);
                if (k < sub && bi * sub + k < n && pp == 0) xsq += (double)xown[k] * (double)xown[k];
            }
            xq_M = lean_norm(xsq, a.xn, tag, nb, sh, a.status, 8);
        }
#pragma unroll 1
        for (int kb = 0; kb < sub; kb += kpt) {
            const int k = kb + (tid >> a.p_shift);
            const int f = bi * sub + k;
            if (k < sub && f < n && pp == 0) {
                float xt = xown[k];
                if (a.model_bits > 0)
                    xt = lean_quant(xt, xq_M, (1 << (a.model_bits - 1)) - 1, a.seed, a.epoch, (uint32_t)(it + 1), 3u, (uint32_t)f);
                if (a.model_out && it + 2 == step_end) a.model_out[f] = xt;
                lean_store(a.ag + f, xt, tag);
            }
        }
        lean_mark(a, it, 5);

        // -------------------------------------------------------------- collect the model, build w
        double bpart = 0.0;
#pragma unroll 1
        for (int f0 = tid; f0 < Fp; f0 += 4 * kLeanThreads) {
            float xt[4];
            const int cnt = f0 >= n ? 0 : min(4, (n - f0 + kLeanThreads - 1) / kLeanThreads);
            lean_poll4(a.ag + f0, kLeanThreads, cnt, tag, xt, sh, a.status, 4);
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int f = f0 + u * kLeanThreads;
                if (f < Fp) {
                    const int q = f >> LOGF, i = f & (FPW - 1);
                    if constexpr (!TABLE) {
                        wv[i * rw + q] = steps[f] * xt[u];
                        bpart += (double)los[f] * (double)xt[u];
                    } else {
                        for (int c = 0; c < L; ++c) tab[(c * FPW + i) * rw + q] = lev[(c * FPW + i) * rw + q] * xt[u];
                    }
                }
            }
        }
        if constexpr (!TABLE) {
            bpart = warp_sum(bpart);
            if (lane == 0) sh->wbase[warp] = bpart;
        }
        lean_mark(a, it, 6);
        __syncthreads();
        lean_mark(a, it, 7);
    }
    // owners return the master model
    for (int kb = 0; kb < sub; kb += kpt) {
        const int k = kb + (tid >> a.p_shift);
        if (k < sub && bi * sub + k < n && pp == 0) a.x[bi * sub + k] = xown[k];
    }
}

// ---------------------------------------------------------------------------------------------
// Host side
// ---------------------------------------------------------------------------------------------
struct LeanPlan {
    int nb, rc, slots, sub_shift, p_shift;
    size_t smem;
};

static size_t lean_smem_bytes(int cb, bool table, int row_words, int bits, int sub, int rc, int slots) {
    const size_t fpw = 32 / cb, Fp = (size_t)row_words * fpw, L = (size_t)1 << bits;
    size_t bytes = (sizeof(LeanShared) + 15) & ~(size_t)15;
    bytes += sizeof(float) * ((table ? 2 * L * Fp : 3 * Fp) + 2 * (size_t)((sub + 3) & ~3) + (size_t)((2 * rc + 3) & ~3) + (size_t)kLeanThreads * fpw);
    bytes += 128;                                                   // slack to align the ring to 128 bytes
    bytes += sizeof(uint32_t) * (size_t)slots * 2 * rc * row_words;
    return bytes;
}

static const void* lean_kernel_ptr(int cb, bool table) {
    if (cb == 2) return table ? (const void*)sgd_lean_kernel<2, true> : (const void*)sgd_lean_kernel<2, false>;
    if (cb == 4) return table ? (const void*)sgd_lean_kernel<4, true> : (const void*)sgd_lean_kernel<4, false>;
    return (const void*)sgd_lean_kernel<8, false>;
}

static int make_lean_plan(const zipml_ctx* ctx, const zipml_dataset* d, const zipml_sgd_params* p, LeanPlan* plan) {
    const int cb = container_bits(d->bits);
    const bool table = d->level_mode == ZIPML_LEVELS_TABLE;
    const int64_t B = p->batch < d->m ? p->batch : d->m;
    const int64_t row_words = d->row_bytes / 4;
    const int sms = ctx->sm_count > 0 ? ctx->sm_count : 1;
    if (d->n > (1 << 20) || row_words > (1 << 18)) return ZIPML_ERR_WORKSPACE;
    int64_t nb = p->grid_row_parts > 0 ? p->grid_row_parts : 32;
    if (p->grid_row_parts <= 0 && nb * 8 > B) nb = B / 8;           // automatic: at least 8 rows per CTA
    if (nb > sms) nb = sms;
    if (nb > B) nb = B;
    if (nb < 1) nb = 1;
    const size_t cap = (size_t)ctx->smem_optin;
    const int64_t nb_max = B < sms ? B : sms;
    // the requested number of row parts is a hint: more parts are used when a tile does not fit
    for (;; ++nb) {
        if (nb > nb_max) return ZIPML_ERR_WORKSPACE;
        LeanPlan r;
        r.rc = (int)((B + nb - 1) / nb);
        r.nb = (int)((B + r.rc - 1) / r.rc);                        // no CTA without rows in a full batch
        const int64_t per = (d->n + r.nb - 1) / r.nb;
        r.sub_shift = 0;
        while (((int64_t)1 << r.sub_shift) < per) ++r.sub_shift;
        r.p_shift = 0;
        while (r.p_shift < 5 && ((int64_t)2 << (r.sub_shift + r.p_shift)) <= kLeanThreads && (1 << r.p_shift) < r.nb) ++r.p_shift;
        if ((uint64_t)2 * r.rc * row_words * 4 >= (1u << 20)) continue;                     // mbarrier tx-count range
        int slots = kLeanMaxSlots;
        while (slots >= 2 && lean_smem_bytes(cb, table, (int)row_words, d->bits, 1 << r.sub_shift, r.rc, slots) > cap) --slots;
        if (slots < 2) continue;
        r.slots = slots;
        r.smem = lean_smem_bytes(cb, table, (int)row_words, d->bits, 1 << r.sub_shift, r.rc, slots);
        *plan = r;
        return ZIPML_OK;
    }
}

int launch_sgd_lean(zipml_ctx* ctx, const zipml_dataset* d, const float* b, float* x, const zipml_sgd_params* p,
                    int64_t first_step, int64_t num_steps, float* grad_out) {
    if (!ctx->cooperative) return ZIPML_ERR_WORKSPACE;
    const int cb = container_bits(d->bits);
    const bool table = d->level_mode == ZIPML_LEVELS_TABLE;
    const int fpw = 32 / cb;
    const int64_t T = (d->m + p->batch - 1) / p->batch;
    LeanPlan plan;
    int rc = make_lean_plan(ctx, d, p, &plan);
    if (rc != ZIPML_OK) return rc;
    const void* kernel = lean_kernel_ptr(cb, table);
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)plan.smem);
    if (e != cudaSuccess) return cuda_status(e);
    int per_sm = 0;
    e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, kLeanThreads, plan.smem);
    if (e != cudaSuccess) return cuda_status(e);
    if (per_sm < 1 || plan.nb > per_sm * ctx->sm_count) return ZIPML_ERR_WORKSPACE;

    size_t off = 0;
    auto piece = [&](size_t bytes) { const size_t o = off; off += carve_size(bytes); return o; };
    const size_t n_rs = (size_t)d->n * plan.nb, n_ag = (size_t)d->n, n_nm = 2 * (size_t)plan.nb;
    const size_t o_ll = piece(sizeof(unsigned long long) * (n_rs + n_ag + 2 * n_nm));
    const size_t ll_bytes = off - o_ll;
    const size_t o_ord = piece(sizeof(int32_t) * (size_t)(p->batch_order ? T : 0));
    rc = ws_reserve(ctx, off);
    if (rc != ZIPML_OK) return rc;

    LeanArgs a;
    memset(&a, 0, sizeof(a));
    a.p1 = reinterpret_cast<const uint32_t*>(d->plane1);
    a.p2 = reinterpret_cast<const uint32_t*>(d->plane2);
    a.lo = d->feat_lo; a.step = d->feat_step; a.levels = d->levels;
    a.b = b; a.x = x; a.grad_out = grad_out; a.model_out = p->model_out;
    a.rs = reinterpret_cast<unsigned long long*>(ctx->ws + o_ll);
    a.ag = a.rs + n_rs;
    a.gn = a.ag + n_ag;
    a.xn = a.gn + n_nm;
    a.trace = reinterpret_cast<unsigned long long*>(p->trace);
    a.trace_steps = p->trace ? p->trace_steps : 0;
    a.status = ctx->d_status;
    a.m = d->m; a.batch = p->batch < d->m ? p->batch : d->m;
    a.seed = p->seed; a.epoch = (uint32_t)p->epoch; a.lr = p->lr; a.reg = p->reg; a.reg_cst = reg_constant(p);
    a.n = (int)d->n; a.bits = d->bits; a.row_words = (int)(d->row_bytes / 4);
    a.words = (int)((d->n + fpw - 1) / fpw);
    a.model_bits = p->model_bits; a.grad_bits = p->grad_bits;
    a.nb = plan.nb; a.rc = plan.rc; a.slots = plan.slots;
    a.sub_shift = plan.sub_shift; a.p_shift = plan.p_shift;
    if (p->batch_order) {
        int32_t* dev_order = reinterpret_cast<int32_t*>(ctx->ws + o_ord);
        e = cudaMemcpyAsync(dev_order, p->batch_order, sizeof(int32_t) * (size_t)T, cudaMemcpyHostToDevice, ctx->stream);
        if (e != cudaSuccess) return cuda_status(e);
        a.order = dev_order;
    }
    // packet tags are 32-bit step counters starting at 1
    const int64_t max_steps = 0x7ffffff0LL;
    for (int64_t s0 = first_step; s0 < first_step + num_steps; s0 += max_steps) {
        e = cudaMemsetAsync(ctx->ws + o_ll, 0, ll_bytes, ctx->stream);
        if (e != cudaSuccess) return cuda_status(e);
        LeanArgs chunk = a;
        chunk.first_step = s0;
        chunk.num_steps = (first_step + num_steps - s0 < max_steps) ? first_step + num_steps - s0 : max_steps;
        if (s0 + chunk.num_steps < first_step + num_steps) { chunk.grad_out = nullptr; chunk.model_out = nullptr; }
        void* params[] = {&chunk};
        e = cudaLaunchCooperativeKernel(kernel, dim3((unsigned)plan.nb), dim3(kLeanThreads), params, plan.smem, ctx->stream);
        if (e != cudaSuccess) return cuda_status(e);
        ctx->launches += 1;
    }
    ctx->last_engine = ZIPML_ENGINE_LEAN;
    return ZIPML_OK;
}

}  // namespace zipml
