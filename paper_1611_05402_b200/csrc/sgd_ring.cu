// Ring engine of zipml_sgd_epoch: one persistent cooperative launch per call, built for steps
// whose code tile is large (Supplement "Double Sampling", footnote form; "End-to-end Quantization").
//
// The minibatch tile is cut into na feature parts x nb row parts, one CTA each (at most one CTA per
// SM).  Inside a CTA one warp is a producer and the others are consumers:
//   * the producer walks the sequence of row chunks that the arithmetic will need -- for every
//     step the chunks of phase A in order, then (if the tile has more than one chunk) the chunks
//     of phase B in reverse order, so that the most recently streamed rows are fetched again
//     first, while they are still in L2 -- and fills a ring of shared-memory slots with bulk
//     asynchronous copies (cp.async.bulk + mbarrier transaction counts).  None of this depends on
//     the model, so the producer runs ahead across phases and steps as far as the ring allows and
//     HBM latency never sits on the step-to-step dependency chain;
//   * consumers wait for a slot, compute on it and hand it back (one arrival per consumer warp).
// Per step:  phase A dots -> residuals (through pd and a grid barrier if na > 1);
//            phase B partial gradients of the CTA's rows -> pg, ps; grid barrier;
//            reduce-scatter: CTA (ai, bi) sums the nb row parts of its own sub-slice of feature
//            part ai in a fixed order, applies the optional gradient quantizer (one more barrier
//            for the norm) and the update, and publishes the new sub-slice; grid barrier;
//            all-gather: every CTA reads the new model of its feature part.
// Every wait is bounded: when one gives up it records ZIPML_ERR_TIMEOUT, later waits of that CTA
// are skipped and the CTA still arrives at every barrier, so the launch always ends.
#include "sgd_common.cuh"

namespace zipml {

constexpr int kRingConsumers = 256;
constexpr int kRingWarps = kRingConsumers / 32;
constexpr int kRingThreads = kRingConsumers + 32;
constexpr int kRingMaxSlots = 8;

__device__ __forceinline__ void consumer_sync() { asm volatile("bar.sync 1, %0;" ::"n"(kRingConsumers) : "memory"); }

// Sum over the consumer threads in a fixed order; every consumer gets the result.
__device__ __forceinline__ double consumer_sum(double v, double* scratch) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    v = warp_sum(v);
    consumer_sync();
    if (lane == 0) scratch[warp] = v;
    consumer_sync();
    double t = 0.0;
#pragma unroll
    for (int w = 0; w < kRingWarps; ++w) t += scratch[w];
    return t;
}

struct RingShared {
    double red[16];
    double misc[8];
    unsigned long long full[kRingMaxSlots];
    unsigned long long empty[kRingMaxSlots];
    int abort_flag;
    int pad;
};

// Bounded wait on an mbarrier phase; after the first failure of this CTA every wait is skipped.
__device__ __forceinline__ void ring_wait(unsigned long long* bar, uint32_t parity, volatile int* abort_flag,
                                          DeviceStatus* status, int where) {
    if (*abort_flag) return;
    for (long long spin = 0; spin < kCopySpinLimit; ++spin)
        if (mbar_try_wait(reinterpret_cast<uint64_t*>(bar), parity)) return;
    *abort_flag = 1;
    set_status(status, ZIPML_ERR_TIMEOUT, where);
}

// Grid barrier among the consumers of all CTAs (the producer warps do not take part).
__device__ __forceinline__ void ring_grid_barrier(unsigned* counter, unsigned target, RingShared* sh, DeviceStatus* status,
                                                  int where) {
    consumer_sync();
    if (threadIdx.x == 0) {
        __threadfence();
        atomicAdd(counter, 1u);
        if (!sh->abort_flag) {
            bool ok = false;
            for (long long it = 0; it < kBarrierSpinLimit; ++it) {
                unsigned v;
                asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(counter) : "memory");
                if (v >= target) { ok = true; break; }
                if ((it & 1023) == 1023) {
                    if (*reinterpret_cast<volatile int*>(&status->code) != 0) break;
                    __nanosleep(200);
                }
            }
            if (!ok) { sh->abort_flag = 1; set_status(status, ZIPML_ERR_TIMEOUT, where); }
        }
    }
    consumer_sync();
}

// Shared memory plan, F = wc * FPW features per CTA:
//   RingShared
//   xs[F] float                model of the CTA's feature part
//   tab float                  uniform: w[F] ([u][word][4]); table: WL[L*F] then LV[L*F] ([code][slot][word])
//   gsub[sub] float            gradient of the CTA's own sub-slice
//   gred[kRingConsumers*FPW]   cross-group reduction of phase B
//   res[2*rc] float            residuals
//   ring[slots][2][cr][wc] u32 code chunks
template <int CB, bool TABLE>
__global__ void __launch_bounds__(kRingThreads) sgd_ring_kernel(const SgdArgs a) {
    constexpr int FPW = 32 / CB;
    extern __shared__ __align__(16) unsigned char s_raw[];
    RingShared* sh = reinterpret_cast<RingShared*>(s_raw);
    const int L = 1 << a.bits;
    const int F = a.wc * FPW;
    float* xs = reinterpret_cast<float*>(s_raw + ((sizeof(RingShared) + 15) & ~(size_t)15));
    float* tab = xs + F;
    float* gsub = tab + (TABLE ? 2 * L * F : F);
    float* gred = gsub + a.sub;
    float* res = gred + kRingConsumers * FPW;
    uint32_t* ring = reinterpret_cast<uint32_t*>(res + ((2 * a.rc + 3) & ~3));
    const size_t slot_words = (size_t)2 * a.cr * a.wc;

    const int ai = blockIdx.x % a.na, bi = blockIdx.x / a.na;
    const int G = a.na * a.nb;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t words_needed = (a.n + FPW - 1) / FPW;
    const int64_t w0 = (int64_t)ai * a.wc;
    const int wcnt = (int)max((int64_t)0, min((int64_t)a.wc, words_needed - w0));    // >= 1: no empty parts
    const int wcopy = (wcnt + 3) & ~3;
    const int64_t j0 = w0 * FPW;
    const int fcnt = (int)max((int64_t)0, min((int64_t)F, a.n - j0));
    const int64_t npad = (int64_t)a.na * F;
    const int k0 = bi * a.rc;
    const int slots = a.stages;
    const int64_t step_end = a.first_step + a.num_steps;

    auto step_rows = [&](int64_t it, int64_t& r0, int& bt, int& rcnt) {
        const int64_t t = a.order ? (int64_t)a.order[it] : it;
        r0 = t * a.batch;
        bt = (int)min(a.batch, a.m - r0);
        rcnt = max(0, min(a.rc, bt - k0));
    };

    if (threadIdx.x == 0) {
        for (int s = 0; s < slots; ++s) {
            mbar_init(reinterpret_cast<uint64_t*>(sh->full + s), 1);
            mbar_init(reinterpret_cast<uint64_t*>(sh->empty + s), kRingWarps);
        }
        sh->abort_flag = 0;
        mbar_fence_init();
    }
    __syncthreads();

    // ================================================================== producer warp
    if (warp == kRingWarps) {
        int slot = 0;
        uint32_t phase = 0;
        const uint32_t row_bytes = (uint32_t)wcopy * 4u;
        const bool contiguous = (a.row_words == a.wc) && (wcopy == a.wc);
        for (int64_t it = a.first_step; it < step_end; ++it) {
            if (*reinterpret_cast<volatile int*>(&sh->abort_flag)) break;   // a wait gave up: start no more copies
            int64_t r0; int bt, rcnt;
            step_rows(it, r0, bt, rcnt);
            const int C = (rcnt + a.cr - 1) / a.cr;
            const int nseq = C <= 1 ? C : 2 * C;
            for (int s = 0; s < nseq; ++s) {
                const int chunk = s < C ? s : 2 * C - 1 - s;
                const int rows = min(a.cr, rcnt - chunk * a.cr);
                uint64_t* full = reinterpret_cast<uint64_t*>(sh->full + slot);
                if (lane == 0) {
                    ring_wait(sh->empty + slot, phase ^ 1u, &sh->abort_flag, a.status, 5);
                    mbar_arrive_expect_tx(full, 2u * (uint32_t)rows * row_bytes);
                }
                __syncwarp();
                uint32_t* dst = ring + (size_t)slot * slot_words;
                const int64_t first = r0 + k0 + (int64_t)chunk * a.cr;
                if (contiguous) {
                    if (lane < 2)
                        bulk_copy_g2s(dst + (size_t)lane * a.cr * a.wc, (lane == 0 ? a.p1 : a.p2) + first * a.row_words,
                                      (uint32_t)rows * row_bytes, full);
                } else {
                    for (int i = lane; i < 2 * rows; i += 32) {
                        const int plane = i & 1, r = i >> 1;
                        bulk_copy_g2s(dst + ((size_t)plane * a.cr + r) * a.wc,
                                      (plane == 0 ? a.p1 : a.p2) + (first + r) * a.row_words + w0, row_bytes, full);
                    }
                }
                if (++slot == slots) { slot = 0; phase ^= 1u; }
            }
        }
        return;
    }

    // ================================================================== consumers
    for (int f = threadIdx.x; f < F; f += kRingConsumers) xs[f] = (f < fcnt) ? a.x[j0 + f] : 0.0f;
    if constexpr (TABLE) {
        float* LVw = tab + L * F;
        for (int idx = threadIdx.x; idx < L * F; idx += kRingConsumers) {
            const int q = idx % a.wc, ci = idx / a.wc, i = ci % FPW, c = ci / FPW;
            const int f = q * FPW + i;
            LVw[idx] = (f < fcnt) ? __ldg(a.levels + (j0 + f) * L + c) : 0.0f;
        }
    }
    // squared norm of the whole model for the first step's model quantizer
    double xnorm2 = 0.0;
    if (a.model_bits > 0) {
        double ss = 0.0;
        for (int64_t j = threadIdx.x; j < a.n; j += kRingConsumers) { const double v = (double)a.x[j]; ss += v * v; }
        xnorm2 = consumer_sum(ss, sh->red);
    }
    consumer_sync();

    // step-invariant thread roles
    const int lanes_q = min(kRingConsumers, ((wcnt + 31) / 32) * 32);
    const int ngroups = kRingConsumers / lanes_q;
    const int group = threadIdx.x / lanes_q;
    const int ql = threadIdx.x % lanes_q;
    const int qpasses = (wcnt + lanes_q - 1) / lanes_q;                      // > 1 only for parts wider than the CTA
    const int sub0 = min(F, bi * a.sub), sub1 = min(F, sub0 + a.sub);        // own sub-slice of the feature part
    const float* LV = tab + L * F;
    const int chunks_w = (wcnt + 31) / 32;
    unsigned barriers_done = 0;
    int slot = 0;
    uint32_t phase = 0;

    for (int64_t it = a.first_step; it < step_end; ++it) {
        int64_t r0; int bt, rcnt;
        step_rows(it, r0, bt, rcnt);
        const int C = (rcnt + a.cr - 1) / a.cr;
        const bool last = (it == step_end - 1);

        // -------------------------------------------------------------- model seen by the step
        VecQuant q3{0.0f, 1, a.seed, a.epoch, (uint32_t)it, 3u};
        if (a.model_bits > 0) { q3.M = (float)sqrt(xnorm2); q3.sm = (1 << (a.model_bits - 1)) - 1; }
        double base = 0.0;
        if constexpr (!TABLE) {
            for (int q = threadIdx.x; q < a.wc; q += kRingConsumers) {
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
            base = consumer_sum(base, sh->red);
        } else {
            for (int f = threadIdx.x; f < F; f += kRingConsumers) {
                float xv = xs[f];
                if (a.model_bits > 0) xv = q3.apply(xv, (uint32_t)(j0 + f));
                const int q = f / FPW, i = f % FPW;
                for (int c = 0; c < L; ++c) tab[(c * FPW + i) * a.wc + q] = LV[(c * FPW + i) * a.wc + q] * xv;
            }
            consumer_sync();
        }

        // -------------------------------------------------------------- phase A: dots
        const bool dots_local = (a.na == 1);
        const int slot_a = slot;                 // slot of the single chunk when C == 1
        for (int chunk = 0; chunk < C; ++chunk) {
            const int rows = min(a.cr, rcnt - chunk * a.cr);
            ring_wait(sh->full + slot, phase, &sh->abort_flag, a.status, 6);
            const uint32_t* t1 = ring + (size_t)slot * slot_words;
            const uint32_t* t2 = t1 + (size_t)a.cr * a.wc;
            for (int lr = warp; lr < rows; lr += kRingWarps) {
                const uint32_t* row1 = t1 + (size_t)lr * a.wc;
                const uint32_t* row2 = t2 + (size_t)lr * a.wc;
                float acc1[2] = {0.0f, 0.0f}, acc2[2] = {0.0f, 0.0f};
#pragma unroll 4
                for (int c = 0; c < chunks_w; ++c) {
                    const int q = c * 32 + lane;
                    if (q < wcnt) {
                        const uint32_t u1 = row1[q], u2 = row2[q];
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
                const double d1 = warp_sum((double)acc1[0] + (double)acc1[1]) + base;
                const double d2 = warp_sum((double)acc2[0] + (double)acc2[1]) + base;
                if (lane == 0) {
                    const int r = chunk * a.cr + lr;
                    if (dots_local) {
                        const double bk = (double)__ldg(a.b + r0 + k0 + r);
                        res[2 * r] = (float)(d1 - bk);
                        res[2 * r + 1] = (float)(d2 - bk);
                    } else {
                        __stcg(a.pd + ((size_t)ai * a.batch + k0 + r) * 2 + 0, d1);
                        __stcg(a.pd + ((size_t)ai * a.batch + k0 + r) * 2 + 1, d2);
                    }
                }
            }
            if (C > 1) {                         // hand the slot back; phase B fetches the chunk again
                __syncwarp();
                if (lane == 0) mbar_arrive(reinterpret_cast<uint64_t*>(sh->empty + slot));
                if (++slot == slots) { slot = 0; phase ^= 1u; }
            }
        }
        if (!dots_local) ring_grid_barrier(a.barrier, (unsigned)G * ++barriers_done, sh, a.status, 1);
        else consumer_sync();

        // -------------------------------------------------------------- phase B: gradient
        double ssum = 0.0;
        for (int r = threadIdx.x; r < rcnt; r += kRingConsumers) {
            float r1, r2;
            if (dots_local) {
                r1 = res[2 * r];
                r2 = res[2 * r + 1];
            } else {
                double d1 = 0.0, d2 = 0.0;
                for (int p = 0; p < a.na; ++p) {
                    d1 += __ldcg(a.pd + ((size_t)p * a.batch + k0 + r) * 2 + 0);
                    d2 += __ldcg(a.pd + ((size_t)p * a.batch + k0 + r) * 2 + 1);
                }
                const double bk = (double)__ldg(a.b + r0 + k0 + r);
                r1 = (float)(d1 - bk);
                r2 = (float)(d2 - bk);
                res[2 * r] = r1;
                res[2 * r + 1] = r2;
            }
            ssum += (double)r1 + (double)r2;
        }
        ssum = consumer_sum(ssum, sh->red);      // residuals are complete after its barriers
        if (threadIdx.x == 0 && ai == 0) __stcg(a.ps + bi, ssum);

        // parts wider than the consumer count (qpasses > 1) are planned as one retained chunk (C <= 1),
        // so the chunk sequence below is walked exactly once whenever chunks are fetched again
        for (int qp = 0; qp < qpasses; ++qp) {
            const int q = qp * lanes_q + ql;
            const bool active = (group < ngroups) && (q < wcnt);
            float acc[FPW];
#pragma unroll
            for (int i = 0; i < FPW; ++i) acc[i] = 0.0f;
            for (int ci = 0; ci < C; ++ci) {
                const int chunk = C - 1 - ci;
                const int rows = min(a.cr, rcnt - chunk * a.cr);
                int use_slot = slot_a;
                if (C > 1) {
                    ring_wait(sh->full + slot, phase, &sh->abort_flag, a.status, 7);
                    use_slot = slot;
                }
                if (active) {
                    const uint32_t* col1 = ring + (size_t)use_slot * slot_words + q;
                    const uint32_t* col2 = col1 + (size_t)a.cr * a.wc;
                    const float* rr = res + 2 * chunk * a.cr;
#pragma unroll 4
                    for (int lr = group; lr < rows; lr += ngroups) {
                        const uint32_t u1 = col1[(size_t)lr * a.wc];
                        const uint32_t u2 = col2[(size_t)lr * a.wc];
                        const float r1 = rr[2 * lr], r2 = rr[2 * lr + 1];
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
                if (C > 1) {
                    __syncwarp();
                    if (lane == 0) mbar_arrive(reinterpret_cast<uint64_t*>(sh->empty + slot));
                    if (++slot == slots) { slot = 0; phase ^= 1u; }
                }
            }
            if (ngroups > 1) {
                consumer_sync();
                if (active) {
#pragma unroll
                    for (int i = 0; i < FPW; ++i) gred[(group * FPW + i) * lanes_q + ql] = acc[i];
                }
                consumer_sync();
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
                float4* dst = reinterpret_cast<float4*>(a.pg + (size_t)bi * npad + (size_t)(w0 + q) * FPW);
#pragma unroll
                for (int u = 0; u < FPW / 4; ++u) __stcg(dst + u, make_float4(acc[4 * u], acc[4 * u + 1], acc[4 * u + 2], acc[4 * u + 3]));
            }
        }
        if (C == 1) {                            // the retained single chunk goes back now
            __syncwarp();
            if (lane == 0) mbar_arrive(reinterpret_cast<uint64_t*>(sh->empty + slot));
            if (++slot == slots) { slot = 0; phase ^= 1u; }
        }
        ring_grid_barrier(a.barrier, (unsigned)G * ++barriers_done, sh, a.status, 2);

        // -------------------------------------------------------------- reduce-scatter: own sub-slice
        double stot = 0.0;
        if constexpr (!TABLE) {
            double part = 0.0;
            if (warp == 0) {
                for (int p = lane; p < a.nb; p += 32) part += __ldcg(a.ps + p);
                part = warp_sum(part);
            }
            if (threadIdx.x == 0) sh->misc[0] = part;
            consumer_sync();
            stot = sh->misc[0];
        }
        const double scale = 1.0 / (2.0 * (double)bt);
        double gsq = 0.0;
        for (int f = sub0 + 4 * threadIdx.x; f < sub1; f += 4 * kRingConsumers) {
            double acc[4] = {0.0, 0.0, 0.0, 0.0};
            const float4* src = reinterpret_cast<const float4*>(a.pg + j0 + f);
#pragma unroll 8
            for (int p = 0; p < a.nb; ++p) {
                const float4 v = __ldcg(src + (size_t)p * (npad / 4));
                acc[0] += (double)v.x; acc[1] += (double)v.y; acc[2] += (double)v.z; acc[3] += (double)v.w;
            }
            float g[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                g[e] = 0.0f;
                if (f + e < fcnt) {
                    double v = acc[e];
                    if constexpr (!TABLE) v = (double)__ldg(a.lo + j0 + f + e) * stot + (double)__ldg(a.step + j0 + f + e) * v;
                    g[e] = (float)(v * scale);
                    if (last && a.grad_out) a.grad_out[j0 + f + e] = g[e];
                }
                gsq += (double)g[e] * (double)g[e];
            }
            *reinterpret_cast<float4*>(gsub + (f - sub0)) = make_float4(g[0], g[1], g[2], g[3]);
        }
        VecQuant q4{0.0f, 1, a.seed, a.epoch, (uint32_t)it, 4u};
        if (a.grad_bits > 0) {
            gsq = consumer_sum(gsq, sh->red);
            if (threadIdx.x == 0) __stcg(a.gn + blockIdx.x, gsq);
            ring_grid_barrier(a.barrier, (unsigned)G * ++barriers_done, sh, a.status, 3);
            double part = 0.0;
            if (warp == 0) {
                for (int p = lane; p < G; p += 32) part += __ldcg(a.gn + p);
                part = warp_sum(part);
            }
            if (threadIdx.x == 0) sh->misc[1] = part;
            consumer_sync();
            q4.M = (float)sqrt(sh->misc[1]);
            q4.sm = (1 << (a.grad_bits - 1)) - 1;
        } else {
            consumer_sync();                     // gsub is complete
        }
        double xsq = 0.0;
        for (int f = sub0 + threadIdx.x; f < sub1; f += kRingConsumers) {
            float xn = 0.0f;
            if (f < fcnt) {
                float g = gsub[f - sub0];
                if (a.grad_bits > 0) g = q4.apply(g, (uint32_t)(j0 + f));
                if (last && a.grad_out) a.grad_out[a.n + j0 + f] = g;
                xn = fmaf(-a.lr, g, xs[f]);
                xsq += (double)xn * (double)xn;
            }
            __stcg(a.xg + j0 + f, xn);
        }
        if (a.model_bits > 0) {
            xsq = consumer_sum(xsq, sh->red);
            if (threadIdx.x == 0) __stcg(a.gn + G + blockIdx.x, xsq);
        }
        ring_grid_barrier(a.barrier, (unsigned)G * ++barriers_done, sh, a.status, 4);

        // -------------------------------------------------------------- all-gather: new model of the part
        for (int f = 4 * threadIdx.x; f < F; f += 4 * kRingConsumers)
            *reinterpret_cast<float4*>(xs + f) = __ldcg(reinterpret_cast<const float4*>(a.xg + j0 + f));
        if (a.model_bits > 0) {
            double part = 0.0;
            if (warp == 0) {
                for (int p = lane; p < G; p += 32) part += __ldcg(a.gn + G + p);
                part = warp_sum(part);
            }
            if (threadIdx.x == 0) sh->misc[2] = part;
            consumer_sync();
            xnorm2 = sh->misc[2];
        } else {
            consumer_sync();
        }
    }
    if (bi == 0)
        for (int f = threadIdx.x; f < fcnt; f += kRingConsumers) a.x[j0 + f] = xs[f];
}

// ---------------------------------------------------------------------------------------------
// Host side
// ---------------------------------------------------------------------------------------------
struct RingPlan {
    int na, nb, wc, rc, cr, slots, sub;
    size_t smem;
};

static size_t ring_smem_bytes(int cb, bool table, int wc, int rc, int bits, int sub, int cr, int slots) {
    const int fpw = 32 / cb;
    const size_t F = (size_t)wc * fpw, L = (size_t)1 << bits;
    size_t bytes = (sizeof(RingShared) + 15) & ~(size_t)15;
    bytes += sizeof(float) * (F + (table ? 2 * L * F : F) + (size_t)sub + (size_t)kRingConsumers * fpw + (size_t)((2 * rc + 3) & ~3));
    bytes += sizeof(uint32_t) * (size_t)slots * 2 * cr * wc;
    return bytes;
}

static const void* ring_kernel_ptr(int cb, bool table) {
    if (cb == 2) return table ? (const void*)sgd_ring_kernel<2, true> : (const void*)sgd_ring_kernel<2, false>;
    if (cb == 4) return table ? (const void*)sgd_ring_kernel<4, true> : (const void*)sgd_ring_kernel<4, false>;
    return (const void*)sgd_ring_kernel<8, false>;
}

static int ring_round_up(int v, int q) { return (v + q - 1) / q * q; }

static int make_ring_plan(const zipml_ctx* ctx, const zipml_dataset* d, const zipml_sgd_params* p, RingPlan* plan) {
    const int cb = container_bits(d->bits);
    const bool table = d->level_mode == ZIPML_LEVELS_TABLE;
    const int fpw = 32 / cb;
    const int64_t words = (d->n + fpw - 1) / fpw;
    const int64_t B = p->batch < d->m ? p->batch : d->m;
    const size_t cap = (size_t)ctx->smem_optin;
    const int sms = ctx->sm_count > 0 ? ctx->sm_count : 1;

    auto shape = [&](int na, int nb, RingPlan* out) -> bool {
        RingPlan r;
        r.wc = ring_round_up((int)((words + na - 1) / na), 32);
        r.na = (int)((words + r.wc - 1) / r.wc);              // no empty feature parts
        r.rc = (int)((B + nb - 1) / nb);
        r.nb = (int)((B + r.rc - 1) / r.rc);                  // no CTA without rows in a full batch
        const int F = r.wc * fpw;
        r.sub = ring_round_up((F + r.nb - 1) / r.nb, 4);
        // a part wider than the consumer count needs the whole tile in one retained chunk
        const bool wide = r.wc > kRingConsumers;
        // chunk: about 32 KiB of codes, at least one row, at most the CTA's rows
        int cr = (int)(32768 / (2 * (size_t)r.wc * 4));
        cr = cr < 1 ? 1 : cr;
        cr = cr > r.rc ? r.rc : cr;
        if (wide) cr = r.rc;
        r.cr = cr;
        if (sizeof(uint32_t) * 2 * (size_t)cr * r.wc >= (1u << 20)) return false;   // mbarrier tx-count range
        int slots = kRingMaxSlots;
        while (slots >= 2 && ring_smem_bytes(cb, table, r.wc, r.rc, d->bits, r.sub, cr, slots) > cap) --slots;
        if (slots < 2) return false;
        r.slots = slots;
        r.smem = ring_smem_bytes(cb, table, r.wc, r.rc, d->bits, r.sub, cr, slots);
        *out = r;
        return true;
    };

    if (p->grid_feature_parts > 0 || p->grid_row_parts > 0) {
        int na = p->grid_feature_parts > 0 ? p->grid_feature_parts : 1;
        int nb = p->grid_row_parts > 0 ? p->grid_row_parts : 1;
        if ((int64_t)na * 32 > ring_round_up((int)words, 32)) na = (int)((words + 31) / 32);
        if (nb > B) nb = (int)B;
        return shape(na, nb, plan) ? ZIPML_OK : ZIPML_ERR_WORKSPACE;
    }
    bool found = false;
    double best_cost = 0.0;
    const int na_max = (int)((words + 31) / 32);
    for (int na = 1; na <= na_max && na <= sms; ++na) {
        int nb = sms / na;
        if (nb > B) nb = (int)B;
        if (nb < 1) nb = 1;
        RingPlan r;
        if (!shape(na, nb, &r)) continue;
        if (r.na * r.nb > sms) continue;
        // per-step model in bytes moved through one CTA: its tile twice, plus what it exchanges
        const double tile = 2.0 * 2.0 * (double)r.rc * r.wc * 4.0;
        const double exch = (r.na > 1 ? (double)r.na * 2.0 * r.rc * 8.0 + 2.0 * r.rc * 8.0 : 0.0) +
                            (double)r.nb * r.sub * 4.0 + (double)r.wc * fpw * 4.0 * 2.0;
        const double cost = tile + 4.0 * exch + (r.na > 1 ? 32768.0 : 0.0);
        if (!found || cost < best_cost) { found = true; best_cost = cost; *plan = r; }
    }
    return found ? ZIPML_OK : ZIPML_ERR_WORKSPACE;
}

int launch_sgd_ring(zipml_ctx* ctx, const zipml_dataset* d, const float* b, float* x, const zipml_sgd_params* p,
                    int64_t first_step, int64_t num_steps, float* grad_out, bool probe_only) {
    if (!ctx->cooperative) return ZIPML_ERR_WORKSPACE;
    const int cb = container_bits(d->bits);
    const bool table = d->level_mode == ZIPML_LEVELS_TABLE;
    const int fpw = 32 / cb;
    const int64_t T = (d->m + p->batch - 1) / p->batch;
    RingPlan plan;
    int rc = make_ring_plan(ctx, d, p, &plan);
    if (rc != ZIPML_OK) return rc;
    const void* kernel = ring_kernel_ptr(cb, table);
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)plan.smem);
    if (e != cudaSuccess) return cuda_status(e);
    int per_sm = 0;
    e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, kRingThreads, plan.smem);
    if (e != cudaSuccess) return cuda_status(e);
    const int G = plan.na * plan.nb;
    if (per_sm < 1 || G > per_sm * ctx->sm_count) return ZIPML_ERR_WORKSPACE;
    if (probe_only) return ZIPML_OK;

    const int64_t B = p->batch < d->m ? p->batch : d->m;
    const size_t npad = (size_t)plan.na * plan.wc * fpw;
    size_t off = 0;
    auto piece = [&](size_t bytes) { const size_t o = off; off += carve_size(bytes); return o; };
    const size_t o_pd = piece(sizeof(double) * (size_t)plan.na * (size_t)B * 2);
    const size_t o_pg = piece(sizeof(float) * (size_t)plan.nb * npad);
    const size_t o_ps = piece(sizeof(double) * (size_t)plan.nb);
    const size_t o_xg = piece(sizeof(float) * npad);
    const size_t o_gn = piece(sizeof(double) * 2 * (size_t)G);
    const size_t o_bar = piece(sizeof(unsigned) * 4);
    const size_t o_ord = piece(sizeof(int32_t) * (size_t)(p->batch_order ? T : 0));
    rc = ws_reserve(ctx, off);
    if (rc != ZIPML_OK) return rc;

    SgdArgs a;
    a.p1 = reinterpret_cast<const uint32_t*>(d->plane1);
    a.p2 = reinterpret_cast<const uint32_t*>(d->plane2);
    a.row_words = d->row_bytes / 4;
    a.m = d->m; a.n = d->n; a.bits = d->bits;
    a.lo = d->feat_lo; a.step = d->feat_step; a.levels = d->levels;
    a.b = b; a.x = x; a.grad_out = grad_out;
    a.batch = B;
    a.first_step = first_step; a.num_steps = num_steps;
    a.lr = p->lr; a.model_bits = p->model_bits; a.grad_bits = p->grad_bits;
    a.seed = p->seed; a.epoch = (uint32_t)p->epoch;
    a.na = plan.na; a.nb = plan.nb; a.wc = plan.wc; a.rc = plan.rc; a.stages = plan.slots;
    a.cr = plan.cr; a.sub = plan.sub;
    a.pd = reinterpret_cast<double*>(ctx->ws + o_pd);
    a.pg = reinterpret_cast<float*>(ctx->ws + o_pg);
    a.ps = reinterpret_cast<double*>(ctx->ws + o_ps);
    a.xg = reinterpret_cast<float*>(ctx->ws + o_xg);
    a.gn = reinterpret_cast<double*>(ctx->ws + o_gn);
    a.barrier = reinterpret_cast<unsigned*>(ctx->ws + o_bar);
    a.status = ctx->d_status;
    a.order = nullptr;
    a.phases = kPhaseAll; a.persistent = 1;
    if (p->batch_order) {
        int32_t* dev_order = reinterpret_cast<int32_t*>(ctx->ws + o_ord);
        e = cudaMemcpyAsync(dev_order, p->batch_order, sizeof(int32_t) * (size_t)T, cudaMemcpyHostToDevice, ctx->stream);
        if (e != cudaSuccess) return cuda_status(e);
        a.order = dev_order;
    }
    // barrier targets are 32-bit: at most 4 barriers per step and G arrivals per barrier
    const int64_t max_steps = (int64_t)(0x7fffffffLL / (4LL * G));
    for (int64_t s0 = first_step; s0 < first_step + num_steps; s0 += max_steps) {
        e = cudaMemsetAsync(a.barrier, 0, sizeof(unsigned) * 4, ctx->stream);
        if (e != cudaSuccess) return cuda_status(e);
        SgdArgs chunk = a;
        chunk.first_step = s0;
        chunk.num_steps = (first_step + num_steps - s0 < max_steps) ? first_step + num_steps - s0 : max_steps;
        if (s0 + chunk.num_steps < first_step + num_steps) chunk.grad_out = nullptr;
        void* params[] = {&chunk};
        e = cudaLaunchCooperativeKernel(kernel, dim3((unsigned)G), dim3(kRingThreads), params, plan.smem, ctx->stream);
        if (e != cudaSuccess) return cuda_status(e);
        ctx->launches += 1;
    }
    return ZIPML_OK;
}

}  // namespace zipml
