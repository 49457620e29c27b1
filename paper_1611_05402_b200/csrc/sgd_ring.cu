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
// Per step:  phase A dots -> residuals (with na > 1 the partial dots of a row meet first);
//            phase B partial gradients of the CTA's rows;
//            reduce-scatter: CTA (ai, bi) collects the nb row parts of its own sub-slice of feature
//            part ai, sums them in a fixed order, applies the optional gradient quantizer (one more
//            exchange for the norm) and the update, and publishes the new sub-slice;
//            all-gather: every CTA collects the new model of its feature part.
// Exchange.  Nothing here uses a grid barrier.  Every exchanged number travels as an 8-byte packet
// {fp32 value, step tag} written with one 64-bit store; a reader polls the packet until the tag is
// the current step's, so the data announces itself and one L2 round trip replaces "write, fence,
// count arrivals, poll the counter, read".  Buffers are zeroed before a launch and tags start at 1.
// A packet of step t is overwritten only by a CTA that has already collected everything of step t
// that depends on its readers, so single buffers suffice; the two exchanges that couple CTAs of
// different feature parts (dots, gradient norm) alternate between two buffers by step parity.
// Every wait is bounded: when one gives up it records ZIPML_ERR_TIMEOUT, later waits of that CTA
// are skipped and the CTA still publishes everything, so the launch always ends.
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

// ---- packets ---------------------------------------------------------------------------------
__device__ __forceinline__ void ll_store(unsigned long long* p, float v, uint32_t tag) {
    __stcg(p, ((unsigned long long)tag << 32) | (unsigned long long)__float_as_uint(v));
}
__device__ __forceinline__ void ll_store_double(unsigned long long* p, double v, uint32_t tag) {
    const float hi = (float)v;
    ll_store(p, hi, tag);
    ll_store(p + 1, (float)(v - (double)hi), tag);
}
__device__ __forceinline__ unsigned long long ll_load(const unsigned long long* p) {
    unsigned long long v;
    asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}
constexpr long long kPacketSpinLimit = 1ll << 22;

// Collects `count` contiguous packets of the current step into dst (shared memory), the consumer
// threads taking them four at a time so that their loads are in flight together.
__device__ __forceinline__ void ll_gather(const unsigned long long* src, int count, uint32_t tag, float* dst,
                                          RingShared* sh, DeviceStatus* status, int where) {
    for (int i0 = threadIdx.x; i0 < count; i0 += 4 * kRingConsumers) {
        unsigned long long v[4];
        bool ok = false;
        if (!*reinterpret_cast<volatile int*>(&sh->abort_flag)) {
            for (long long spin = 0; spin < kPacketSpinLimit && !ok; ++spin) {
                ok = true;
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int i = i0 + u * kRingConsumers;
                    if (i < count) { v[u] = ll_load(src + i); ok = ok && ((uint32_t)(v[u] >> 32) == tag); }
                }
            }
            if (!ok) { sh->abort_flag = 1; set_status(status, ZIPML_ERR_TIMEOUT, where); }
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int i = i0 + u * kRingConsumers;
            if (i < count) dst[i] = ok ? __uint_as_float((uint32_t)v[u]) : 0.0f;
        }
    }
}

// Shared memory plan, F = wc * FPW features per CTA:
//   RingShared
//   xs[F] float                 model of the CTA's feature part
//   tab float                   uniform: w[F] ([u][word][4]); table: WL[L*F] then LV[L*F] ([code][slot][word])
//   gsub[sub] float             gradient of the CTA's own sub-slice
//   gbuf[nb*(sub+2)] float      collected row parts of the own sub-slice (+ residual sums)
//   dsum[sub+2] double          their sums
//   nbuf[4*G] float             collected partial norms
//   gred[kRingConsumers*FPW]    cross-group reduction of phase B
//   res[2*rc] float             residuals
//   bsm[2][rc] float            labels of the current and the next step's rows
//   ring[slots][2][cr][wc] u32  code chunks
template <int CB, bool TABLE>
__global__ void __launch_bounds__(kRingThreads) sgd_ring_kernel(const SgdArgs a) {
    constexpr int FPW = 32 / CB;
    extern __shared__ __align__(16) unsigned char s_raw[];
    RingShared* sh = reinterpret_cast<RingShared*>(s_raw);
    const int L = 1 << a.bits;
    const int F = a.wc * FPW;
    const int G = a.na * a.nb;
    const int subp = a.sub + 2;                                  // packets per (owner, writer)
    float* xs = reinterpret_cast<float*>(s_raw + ((sizeof(RingShared) + 15) & ~(size_t)15));
    float* tab = xs + F;
    float* gsub = tab + (TABLE ? 2 * L * F : F);
    float* gbuf = gsub + a.sub;
    double* dsum = reinterpret_cast<double*>(gbuf + ((a.nb * subp + 3) & ~3));
    float* nbuf = reinterpret_cast<float*>(dsum + ((subp + 1) & ~1));
    float* gred = nbuf + 4 * G;
    float* res = gred + kRingConsumers * FPW;
    float* bsm = res + ((2 * a.rc + 3) & ~3);
    uint32_t* ring = reinterpret_cast<uint32_t*>(bsm + ((2 * a.rc + 3) & ~3));
    const size_t slot_words = (size_t)2 * a.cr * a.wc;

    const int ai = blockIdx.x % a.na, bi = blockIdx.x / a.na;
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
    {   // labels of the first step's rows
        int64_t r0; int bt, rcnt;
        step_rows(a.first_step, r0, bt, rcnt);
        float* bcur = bsm + (size_t)(a.first_step & 1) * a.rc;
        for (int r = threadIdx.x; r < rcnt; r += kRingConsumers) bcur[r] = __ldg(a.b + r0 + k0 + r);
    }
    consumer_sync();

    // step-invariant thread roles
    const int lanes_q = min(kRingConsumers, ((wcnt + 31) / 32) * 32);
    const int ngroups = kRingConsumers / lanes_q;
    const int group = threadIdx.x / lanes_q;
    const int ql = threadIdx.x % lanes_q;
    const int sub0 = min(F, bi * a.sub), sub1 = min(F, sub0 + a.sub);        // own sub-slice of the feature part
    const float* LV = tab + L * F;
    const int chunks_w = (wcnt + 31) / 32;
    int slot = 0;
    uint32_t phase = 0;
    // where this CTA's packets go and come from
    unsigned long long* rs_mine = a.ll_rs + (size_t)ai * a.nb * a.nb * subp;                 // + (owner*nb + writer)*subp
    const unsigned long long* rs_own = rs_mine + (size_t)bi * a.nb * subp;                   // collected by this owner
    unsigned long long* ag_part = a.ll_ag + j0;
    unsigned long long* ag_norm = a.ll_ag + npad;

    for (int64_t it = a.first_step; it < step_end; ++it) {
        int64_t r0; int bt, rcnt;
        step_rows(it, r0, bt, rcnt);
        const int C = (rcnt + a.cr - 1) / a.cr;
        const bool last = (it == step_end - 1);
        const uint32_t tag = (uint32_t)(it - a.first_step) + 1u;
        const int par = (int)(it & 1);
        const float* bcur = bsm + (size_t)par * a.rc;

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
        unsigned long long* pd_mine = a.ll_pd + (((size_t)par * a.nb + bi) * a.na + ai) * a.rc * 4;
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
                                acc1[0] = fmaf(c1[4 * u + 0], wv.x, acc1[0]);
                                acc1[1] = fmaf(c1[4 * u + 1], wv.y, acc1[1]);
                                acc1[0] = fmaf(c1[4 * u + 2], wv.z, acc1[0]);
                                acc1[1] = fmaf(c1[4 * u + 3], wv.w, acc1[1]);
                                acc2[0] = fmaf(c2[4 * u + 0], wv.x, acc2[0]);
                                acc2[1] = fmaf(c2[4 * u + 1], wv.y, acc2[1]);
                                acc2[0] = fmaf(c2[4 * u + 2], wv.z, acc2[0]);
                                acc2[1] = fmaf(c2[4 * u + 3], wv.w, acc2[1]);
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
                        const double bk = (double)bcur[r];
                        res[2 * r] = (float)(d1 - bk);
                        res[2 * r + 1] = (float)(d2 - bk);
                    } else {
                        ll_store_double(pd_mine + (size_t)r * 4, d1, tag);
                        ll_store_double(pd_mine + (size_t)r * 4 + 2, d2, tag);
                    }
                }
            }
            if (C > 1) {                         // hand the slot back; phase B fetches the chunk again
                __syncwarp();
                if (lane == 0) mbar_arrive(reinterpret_cast<uint64_t*>(sh->empty + slot));
                if (++slot == slots) { slot = 0; phase ^= 1u; }
            }
        }
        if (!dots_local) {
            // every row's dot is the sum, in part order, of the na partial dots published for it
            const unsigned long long* pd_row = a.ll_pd + ((size_t)par * a.nb + bi) * a.na * a.rc * 4;
            for (int r = threadIdx.x; r < rcnt; r += kRingConsumers) {
                double d1 = 0.0, d2 = 0.0;
                bool good = !*reinterpret_cast<volatile int*>(&sh->abort_flag);
                for (int p = 0; p < a.na && good; ++p) {
                    const unsigned long long* src = pd_row + ((size_t)p * a.rc + r) * 4;
                    unsigned long long v[4];
                    bool ok = false;
                    for (long long spin = 0; spin < kPacketSpinLimit && !ok; ++spin) {
                        ok = true;
#pragma unroll
                        for (int u = 0; u < 4; ++u) { v[u] = ll_load(src + u); ok = ok && ((uint32_t)(v[u] >> 32) == tag); }
                    }
                    if (!ok) { sh->abort_flag = 1; set_status(a.status, ZIPML_ERR_TIMEOUT, 1); good = false; break; }
                    d1 += (double)__uint_as_float((uint32_t)v[0]) + (double)__uint_as_float((uint32_t)v[1]);
                    d2 += (double)__uint_as_float((uint32_t)v[2]) + (double)__uint_as_float((uint32_t)v[3]);
                }
                const double bk = (double)bcur[r];
                res[2 * r] = good ? (float)(d1 - bk) : 0.0f;
                res[2 * r + 1] = good ? (float)(d2 - bk) : 0.0f;
            }
        }
        consumer_sync();                         // residuals are complete

        // -------------------------------------------------------------- phase B: gradient
        double ssum = 0.0;
        for (int r = threadIdx.x; r < rcnt; r += kRingConsumers) ssum += (double)res[2 * r] + (double)res[2 * r + 1];
        ssum = consumer_sum(ssum, sh->red);
        {
            const int q = ql;
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
                // feature f of the part belongs to owner f / sub; its packet sits in that owner's block for this writer
#pragma unroll
                for (int i = 0; i < FPW; ++i) {
                    const int f = q * FPW + i;
                    const int owner = f / a.sub;
                    ll_store(rs_mine + ((size_t)owner * a.nb + bi) * subp + (f - owner * a.sub), acc[i], tag);
                }
            }
        }
        if (C == 1) {                            // the retained single chunk goes back now
            __syncwarp();
            if (lane == 0) mbar_arrive(reinterpret_cast<uint64_t*>(sh->empty + slot));
            if (++slot == slots) { slot = 0; phase ^= 1u; }
        }
        // owners also wait for the slots of features past the part's last code word and of their
        // sub-slice's unused tail: those carry zeros
        for (int f = wcnt * FPW + threadIdx.x; f < a.nb * a.sub; f += kRingConsumers) {
            const int owner = f / a.sub;
            ll_store(rs_mine + ((size_t)owner * a.nb + bi) * subp + (f - owner * a.sub), 0.0f, tag);
        }
        // the residual sum goes to every owner of the part, behind the gradient packets
        for (int o = threadIdx.x; o < a.nb; o += kRingConsumers)
            ll_store_double(rs_mine + ((size_t)o * a.nb + bi) * subp + a.sub, ssum, tag);
        // labels of the next step's rows, fetched while the packets travel
        if (!last) {
            int64_t r0n; int btn, rcntn;
            step_rows(it + 1, r0n, btn, rcntn);
            float* bnext = bsm + (size_t)(par ^ 1) * a.rc;
            for (int r = threadIdx.x; r < rcntn; r += kRingConsumers) bnext[r] = __ldg(a.b + r0n + k0 + r);
        }

        // -------------------------------------------------------------- reduce-scatter: own sub-slice
        const int nsub = sub1 - sub0;            // features this CTA owns (may be 0 for the last owners)
        ll_gather(rs_own, a.nb * subp, tag, gbuf, sh, a.status, 2);
        consumer_sync();
        if (a.nb <= 32) {
            for (int k = threadIdx.x; k < subp; k += kRingConsumers) {
                double t = 0.0;
                for (int w = 0; w < a.nb; ++w) t += (double)gbuf[w * subp + k];
                dsum[k] = t;
            }
        } else {
            for (int k = warp; k < subp; k += kRingWarps) {
                double t = 0.0;
                for (int w = lane; w < a.nb; w += 32) t += (double)gbuf[w * subp + k];
                t = warp_sum(t);
                if (lane == 0) dsum[k] = t;
            }
        }
        consumer_sync();
        const double stot = dsum[a.sub] + dsum[a.sub + 1];
        const double scale = 1.0 / (2.0 * (double)bt);
        double gsq = 0.0;
        for (int k = threadIdx.x; k < nsub; k += kRingConsumers) {
            const int f = sub0 + k;
            float g = 0.0f;
            if (f < fcnt) {
                double v = dsum[k];
                if constexpr (!TABLE) v = (double)__ldg(a.lo + j0 + f) * stot + (double)__ldg(a.step + j0 + f) * v;
                g = (float)(v * scale);
                if (last && a.grad_out) a.grad_out[j0 + f] = g;
            }
            gsub[k] = g;
            gsq += (double)g * (double)g;
        }
        VecQuant q4{0.0f, 1, a.seed, a.epoch, (uint32_t)it, 4u};
        if (a.grad_bits > 0) {
            gsq = consumer_sum(gsq, sh->red);
            unsigned long long* gn = a.ll_gn + (size_t)par * G * 2;
            if (threadIdx.x == 0) ll_store_double(gn + (size_t)blockIdx.x * 2, gsq, tag);
            ll_gather(gn, 2 * G, tag, nbuf, sh, a.status, 3);
            consumer_sync();
            double part = 0.0;
            if (warp == 0) {
                for (int p = lane; p < G; p += 32) part += (double)nbuf[2 * p] + (double)nbuf[2 * p + 1];
                part = warp_sum(part);
            }
            if (threadIdx.x == 0) sh->misc[1] = part;
            consumer_sync();
            q4.M = (float)sqrt(sh->misc[1]);
            q4.sm = (1 << (a.grad_bits - 1)) - 1;
        }
        double xsq = 0.0;
        for (int k = threadIdx.x; k < nsub; k += kRingConsumers) {
            const int f = sub0 + k;
            float xn = 0.0f;
            if (f < fcnt) {
                float g = gsub[k];
                if (a.grad_bits > 0) g = q4.apply(g, (uint32_t)(j0 + f));
                if (last && a.grad_out) a.grad_out[a.n + j0 + f] = g;
                xn = fmaf(-a.lr, g, xs[f]);
                xsq += (double)xn * (double)xn;
            }
            ll_store(ag_part + f, xn, tag);
        }
        if (a.model_bits > 0) {
            xsq = consumer_sum(xsq, sh->red);
            if (threadIdx.x == 0) ll_store_double(ag_norm + (size_t)blockIdx.x * 2, xsq, tag);
        }

        // -------------------------------------------------------------- all-gather: new model of the part
        consumer_sync();                         // everybody is done with xs of this step
        ll_gather(ag_part, F, tag, xs, sh, a.status, 4);
        if (a.model_bits > 0) {
            ll_gather(ag_norm, 2 * G, tag, nbuf + 2 * G, sh, a.status, 8);
            consumer_sync();
            double part = 0.0;
            if (warp == 0) {
                for (int p = lane; p < G; p += 32) part += (double)nbuf[2 * G + 2 * p] + (double)nbuf[2 * G + 2 * p + 1];
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

static size_t ring_smem_bytes(int cb, bool table, int wc, int rc, int bits, int sub, int cr, int slots, int nb, int G) {
    const int fpw = 32 / cb;
    const size_t F = (size_t)wc * fpw, L = (size_t)1 << bits;
    const size_t subp = (size_t)sub + 2;
    size_t bytes = (sizeof(RingShared) + 15) & ~(size_t)15;
    bytes += sizeof(float) * (F + (table ? 2 * L * F : F) + (size_t)sub + (((size_t)nb * subp + 3) & ~(size_t)3));
    bytes += sizeof(double) * ((subp + 1) & ~(size_t)1);
    bytes += sizeof(float) * (4 * (size_t)G + (size_t)kRingConsumers * fpw + 2 * (size_t)((2 * rc + 3) & ~3));
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
        while (slots >= 2 && ring_smem_bytes(cb, table, r.wc, r.rc, d->bits, r.sub, cr, slots, r.nb, r.na * r.nb) > cap) --slots;
        if (slots < 2) return false;
        r.slots = slots;
        r.smem = ring_smem_bytes(cb, table, r.wc, r.rc, d->bits, r.sub, cr, slots, r.nb, r.na * r.nb);
        *out = r;
        return true;
    };

    const int na_min = (int)((words + kRingConsumers - 1) / kRingConsumers);
    if (p->grid_feature_parts > 0 || p->grid_row_parts > 0) {
        int na = p->grid_feature_parts > 0 ? p->grid_feature_parts : 1;
        int nb = p->grid_row_parts > 0 ? p->grid_row_parts : 1;
        if ((int64_t)na * 32 > ring_round_up((int)words, 32)) na = (int)((words + 31) / 32);
        if (na < na_min) na = na_min;          // the request is a hint: parts never exceed one word column per thread
        if (nb > B) nb = (int)B;
        return shape(na, nb, plan) ? ZIPML_OK : ZIPML_ERR_WORKSPACE;
    }
    bool found = false;
    double best_cost = 0.0;
    const int na_max = (int)((words + 31) / 32);
    for (int na = na_min; na <= na_max && na <= sms; ++na) {
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
    const size_t subp = (size_t)plan.sub + 2;
    const size_t n_pd = plan.na > 1 ? 2 * (size_t)plan.nb * plan.na * plan.rc * 4 : 0;
    const size_t n_rs = (size_t)G * plan.nb * subp;
    const size_t n_gn = 2 * (size_t)G * 2;
    const size_t n_ag = npad + 2 * (size_t)G;
    const size_t o_ll = piece(sizeof(unsigned long long) * (n_pd + n_rs + n_gn + n_ag));
    const size_t ll_bytes = off - o_ll;
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
    a.pd = nullptr; a.pg = nullptr; a.ps = nullptr; a.barrier = nullptr;
    a.ll_pd = reinterpret_cast<unsigned long long*>(ctx->ws + o_ll);
    a.ll_rs = a.ll_pd + n_pd;
    a.ll_gn = a.ll_rs + n_rs;
    a.ll_ag = a.ll_gn + n_gn;
    a.status = ctx->d_status;
    a.order = nullptr;
    a.phases = kPhaseAll; a.persistent = 1;
    if (p->batch_order) {
        int32_t* dev_order = reinterpret_cast<int32_t*>(ctx->ws + o_ord);
        e = cudaMemcpyAsync(dev_order, p->batch_order, sizeof(int32_t) * (size_t)T, cudaMemcpyHostToDevice, ctx->stream);
        if (e != cudaSuccess) return cuda_status(e);
        a.order = dev_order;
    }
    // packet tags are 32-bit step counters starting at 1
    const int64_t max_steps = 0x7fffffffLL;
    for (int64_t s0 = first_step; s0 < first_step + num_steps; s0 += max_steps) {
        e = cudaMemsetAsync(ctx->ws + o_ll, 0, ll_bytes, ctx->stream);
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
