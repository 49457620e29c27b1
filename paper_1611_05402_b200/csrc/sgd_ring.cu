// Ring engine of zipml_sgd_epoch: one persistent cooperative launch per call, built for steps
// whose code tile is large (Supplement "Double Sampling", footnote form; "End-to-end Quantization").
//
// The minibatch tile is cut into na feature parts x nb row parts, one CTA each (at most one CTA per
// SM).  Inside a CTA one warp is a producer and the others are consumers:
//   * the producer walks the sequence of row chunks that the arithmetic will need -- for every
//     step the chunks of phase A in order, then (if the tile has more than one chunk) the chunks
//     of phase B in reverse order, so that the most recently streamed rows are fetched again
//     first, while they are still in L2 -- and fills a ring of shared-memory slots with bulk
//     asynchronous copies (mbarrier transaction counts): for uniform grids one 2-D tensor-map box of
//     32 rows of one plane per slot, its rows four words wider than the part so that they lie wc + 4
//     words apart in shared memory (fragment loads of 8 rows then hit 8 different bank groups); for
//     level tables both planes of a chunk per slot.  None of this depends on the model, so the
//     producer runs ahead across phases and steps as far as the ring allows and HBM latency never
//     sits on the step-to-step dependency chain;
//   * consumers wait for a slot, compute on it and hand it back (one arrival per consumer warp).
// Uniform grids contract on the int8 tensor cores (mma.sync m16n8k32, u8 x s8 -> s32): the fp32
// vector that meets the codes (w = step * x~ in phase A, the residuals in phase B) is turned once
// per step into four balanced base-128 digits per entry, stored as the B operand's columns; the
// code bytes are the A operand, loaded with ldmatrix straight from the tile in phase A (16 rows x
// 32 bytes) and with a transposing ldmatrix plus two byte permutes in phase B (16 byte columns x
// 32 rows); 4- and 2-bit codes are split into their groups by a shift and a mask per fragment
// register, each group meeting its own digit vectors.  Digit sums are exact 32-bit integers, combined
// in 64 bits (or exactly in double); warps meet through shared-memory integer atomics, whose order
// cannot change the result.  Level tables use fp32 look-ups.
// Per step:  phase A dots -> residuals (with na > 1 the partial dots of a row meet first);
//            phase B partial gradients of the CTA's rows;
//            reduce-scatter: CTA (ai, bi) collects the nb row parts of its own sub-slice of feature
//            part ai, sums them in a fixed order, applies the optional gradient quantizer (one more
//            exchange for the norm) and the update, and publishes the new sub-slice;
//            all-gather: every CTA collects, word by word, the model its feature part will see in
//            the next step (the owners keep the fp32 master of their sub-slice to themselves and
//            publish Q3 of it when the model quantizer is on) and turns it into w = step * x~.
// Exchange.  Nothing here uses a grid barrier.  Every exchanged number travels as an 8-byte packet
// {fp32 value, step tag} written with one 64-bit store; a reader polls the packet until the tag is
// the current step's, so the data announces itself and one L2 round trip replaces "write, fence,
// count arrivals, poll the counter, read".  Buffers are zeroed before a launch and tags start at 1.
// A packet of step t is overwritten only by a CTA that has already collected everything of step t
// that depends on its readers, so single buffers suffice; the two exchanges that couple CTAs of
// different feature parts (dots, gradient norm) alternate between two buffers by step parity.
// Every wait is bounded: when one gives up it records ZIPML_ERR_TIMEOUT, later waits of that CTA
// are skipped and the CTA still publishes everything, so the launch always ends.
#include <cuda.h>
#include <string.h>

#include "int_digits.cuh"
#include "sgd_common.cuh"

namespace zipml {

constexpr int kRingConsumers = 256;
constexpr int kRingWarps = kRingConsumers / 32;
constexpr int kRingThreads = kRingConsumers + 32;
constexpr int kRingMaxSlots = 8;
constexpr int kRingTasks = 8;              // integer phase B: accumulator sets (8 words of one group) per warp

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
    double dpart[8 * 16];          // [task][8] partial sums of split row blocks
    double misc[8];
    double wbase[16];              // per-warp parts of lo^T x~ over the CTA's feature part
    float fmax[32];                // per-warp maxima: [0..15] |w| of the word stage, [16..31] |residual|
    unsigned long long full[kRingMaxSlots];
    unsigned long long empty[kRingMaxSlots];
    int abort_flag;
    int pad;
    uint4 zero16;                  // sixteen zero bytes: the unused columns of the digit operands point here
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

__device__ __forceinline__ void trace_mark(const SgdArgs& a, int64_t it, int slot_id) {
    if (a.trace && blockIdx.x == 0 && threadIdx.x == 0 && it - a.first_step < a.trace_steps) {
        unsigned long long t;
        asm volatile("mov.u64 %0, %clock64;" : "=l"(t));
        a.trace[(it - a.first_step) * 8 + slot_id] = t;
    }
}

// 2-D tiled bulk copy global -> shared through a tensor map (rows x words box); x in elements must make
// x * 4 bytes a multiple of 16, the destination is 128-byte aligned.
__device__ __forceinline__ void tensor_copy_g2s(void* dst_smem, const CUtensorMap* tm, int x, int y, uint64_t* bar) {
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                 ::"r"(smem_u32(dst_smem)), "l"(reinterpret_cast<uint64_t>(tm)), "r"(x), "r"(y), "r"(smem_u32(bar)) : "memory");
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

// Waits, with back-off, until `count` sentinel packets (src[i * stride], one per contributor) carry the
// current step's tag.  Only `count` threads poll, so the wait costs L2 little; the full collection that
// follows then finds (almost) every packet in place and still checks each tag itself.
__device__ __forceinline__ void ll_wait_sentinels(const unsigned long long* src, int stride, int count, uint32_t tag,
                                                  RingShared* sh, DeviceStatus* status, int where) {
    for (int i = threadIdx.x; i < count; i += kRingConsumers) {
        if (*reinterpret_cast<volatile int*>(&sh->abort_flag)) break;
        bool ok = false;
        for (long long spin = 0; spin < kPacketSpinLimit; ++spin) {
            if ((uint32_t)(ll_load(src + (size_t)i * stride) >> 32) == tag) { ok = true; break; }
            __nanosleep(spin < 64 ? 32 : 256);
        }
        if (!ok) { sh->abort_flag = 1; set_status(status, ZIPML_ERR_TIMEOUT, where); }
    }
    consumer_sync();
}

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

// Eight values per lane -> their eight sums over the warp with 9 shuffles instead of 40: in each of
// the first three steps a lane hands half of what it holds to its partner and keeps (and adds) the
// other half.  Afterwards lane L holds sum number (L >> 2) & 7, complete, in a fixed order.
template <typename T>
__device__ __forceinline__ T reduce8(const T (&v)[8], int lane) {
    const bool up16 = (lane & 16) != 0, up8 = (lane & 8) != 0, up4 = (lane & 4) != 0;
    T w4[4], w2[2];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const T send = up16 ? v[i] : v[i + 4], keep = up16 ? v[i + 4] : v[i];
        w4[i] = keep + __shfl_xor_sync(0xffffffffu, send, 16);
    }
#pragma unroll
    for (int i = 0; i < 2; ++i) {
        const T send = up8 ? w4[i] : w4[i + 2], keep = up8 ? w4[i + 2] : w4[i];
        w2[i] = keep + __shfl_xor_sync(0xffffffffu, send, 8);
    }
    const T send = up4 ? w2[0] : w2[1], keep = up4 ? w2[1] : w2[0];
    T w1 = keep + __shfl_xor_sync(0xffffffffu, send, 4);
    w1 += __shfl_xor_sync(0xffffffffu, w1, 2);
    w1 += __shfl_xor_sync(0xffffffffu, w1, 1);
    return w1;
}

// Maximum over the consumer threads (values >= 0); `slot` = 0 or 16 picks the half of sh->fmax.
__device__ __forceinline__ float consumer_max(float v, RingShared* sh, int slot) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    if ((threadIdx.x & 31) == 0) sh->fmax[slot + (threadIdx.x >> 5)] = v;
    consumer_sync();
    float m = 0.0f;
#pragma unroll
    for (int w = 0; w < kRingWarps; ++w) m = fmaxf(m, sh->fmax[slot + w]);
    return m;
}

// Shared memory plan, F = wc * FPW features per CTA:
//   RingShared
//   tab                         uniform: digits of w as B operands, bytes [k-slab of 8 words][group][digit][32];
//                               table: WL[L*F] then LV[L*F] floats ([code][slot][word])
//   xown[sub] float             master model of the CTA's own sub-slice
//   gsub[sub] float             gradient of the own sub-slice
//   gbuf[nb*(sub+2)] float      collected row parts of the own sub-slice (+ residual sums)
//   nbuf[2*G] float             collected partial norms
//   gred[kRingConsumers*FPW]    table: cross-group reduction of phase B
//   res[2*rc] float             residuals
//   rdig[ceil(rc/32)][2][4][32] bytes  uniform: digits of the residuals as B operands: per 32 rows, per
//                               residual (r1, r2), per digit a 32-byte k vector (row order of phase B)
//   dacc[rc][2][4] int          uniform: digit sums of the dots per (row, plane), filled by the warps' atomics
//   bsm[2][rc] float            labels of the current and the next step's rows
//   ring[slots][planes][cr][pitch] u32  code chunks (uniform: one plane per slot, pitch = wc + 4; table: both, pitch = wc)
template <int CB, bool TABLE>
__global__ void __launch_bounds__(kRingThreads, 1) sgd_ring_kernel(const SgdArgs a, const __grid_constant__ CUtensorMap tm1,
                                                                  const __grid_constant__ CUtensorMap tm2) {
    constexpr int FPW = 32 / CB;
    constexpr int NS = IntPath<CB>::NS, NG = IntPath<CB>::NG;
    constexpr float QMAXF = (float)IntPath<CB>::QMAX;
    extern __shared__ __align__(16) unsigned char s_raw[];
    RingShared* sh = reinterpret_cast<RingShared*>(s_raw);
    const int L = 1 << a.bits;
    const int F = a.wc * FPW;
    const int G = a.na * a.nb;
    const int subp = a.sub + 2;                                  // packets per (owner, writer)
    float* tab = reinterpret_cast<float*>(s_raw + ((sizeof(RingShared) + 15) & ~(size_t)15));
    float* xown = tab + (TABLE ? 2 * L * F : F);
    float* gsub = xown + a.sub;
    float* gbuf = gsub + a.sub;
    float* nbuf = gbuf + ((a.nb * subp + 3) & ~3);
    float* gred = nbuf + ((2 * G + 3) & ~3);
    float* res = gred + (TABLE ? kRingConsumers * FPW : 0);
    unsigned char* rdig = reinterpret_cast<unsigned char*>(res + ((2 * a.rc + 3) & ~3));
    int* dacc = reinterpret_cast<int*>(rdig + (size_t)((a.rc + 31) / 32) * 256);
    float* bsm = reinterpret_cast<float*>(dacc + (TABLE ? 0 : 8 * a.rc));
    uint32_t* ring = reinterpret_cast<uint32_t*>(
        (reinterpret_cast<uintptr_t>(bsm + ((2 * a.rc + 3) & ~3)) + 127) & ~(uintptr_t)127);      // tensor copies want 128 bytes
    const int pitch = a.pitch;
    constexpr int PPS = TABLE ? 2 : 1;           // planes per ring slot
    const size_t slot_words = (size_t)PPS * a.cr * pitch;

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
        sh->zero16 = make_uint4(0u, 0u, 0u, 0u);
        mbar_fence_init();
    }
    __syncthreads();

    // ================================================================== producer warp
    if (warp == kRingWarps) {
        int slot = 0;
        uint32_t phase = 0;
        const uint32_t row_bytes = (uint32_t)wcopy * 4u;
        const bool contiguous = (a.row_words == a.wc) && (wcopy == a.wc) && (pitch == a.wc);
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
                uint32_t* dst = ring + (size_t)slot * slot_words;
                const int64_t first = r0 + k0 + (int64_t)chunk * a.cr;
                if constexpr (!TABLE) {
                    // one slot per plane: rows of `row_bytes` bytes, `pitch` words apart
#pragma unroll 1
                    for (int pl = 0; pl < 2; ++pl) {
                        uint64_t* fullp = reinterpret_cast<uint64_t*>(sh->full + slot);
                        uint32_t* dstp = ring + (size_t)slot * slot_words;
                        if (a.use_tmap) {
                            // one box of cr rows x pitch words (64-bit elements): the four words past the part
                            // (the neighbour's, or zeros past the row) and the rows past the chunk come along
                            // unused; the box's dense rows are exactly `pitch` words apart
                            if (lane == 0) {
                                ring_wait(sh->empty + slot, phase ^ 1u, &sh->abort_flag, a.status, 5);
                                mbar_arrive_expect_tx(fullp, (uint32_t)a.cr * (uint32_t)pitch * 4u);
                                tensor_copy_g2s(dstp, pl == 0 ? &tm1 : &tm2, (int)(w0 >> 1), (int)first, fullp);
                            }
                            __syncwarp();
                        } else {
                            if (lane == 0) {
                                ring_wait(sh->empty + slot, phase ^ 1u, &sh->abort_flag, a.status, 5);
                                mbar_arrive_expect_tx(fullp, (uint32_t)rows * row_bytes);
                            }
                            __syncwarp();
                            const uint32_t* src = (pl == 0 ? a.p1 : a.p2) + first * a.row_words + w0;
                            for (int r = lane; r < rows; r += 32)
                                bulk_copy_g2s(dstp + (size_t)r * pitch, src + (size_t)r * a.row_words, row_bytes, fullp);
                        }
                        if (++slot == slots) { slot = 0; phase ^= 1u; }
                    }
                    continue;
                }
                if (a.use_tmap) {
                    // one box of cr rows x wc words per plane; rows past the chunk (the next rows of the
                    // plane, or zeros past its end) come along and are never used
                    if (lane == 0) {
                        ring_wait(sh->empty + slot, phase ^ 1u, &sh->abort_flag, a.status, 5);
                        mbar_arrive_expect_tx(full, 2u * (uint32_t)a.cr * (uint32_t)a.wc * 4u);
                        tensor_copy_g2s(dst, &tm1, (int)w0, (int)first, full);
                        tensor_copy_g2s(dst + (size_t)a.cr * pitch, &tm2, (int)w0, (int)first, full);
                    }
                    __syncwarp();
                } else {
                    if (lane == 0) {
                        ring_wait(sh->empty + slot, phase ^ 1u, &sh->abort_flag, a.status, 5);
                        mbar_arrive_expect_tx(full, 2u * (uint32_t)rows * row_bytes);
                    }
                    __syncwarp();
                    if (contiguous) {
                        if (lane < 2)
                            bulk_copy_g2s(dst + (size_t)lane * a.cr * pitch, (lane == 0 ? a.p1 : a.p2) + first * a.row_words,
                                          (uint32_t)rows * row_bytes, full);
                    } else {
                        for (int i = lane; i < 2 * rows; i += 32) {
                            const int plane = i & 1, r = i >> 1;
                            bulk_copy_g2s(dst + ((size_t)plane * a.cr + r) * pitch,
                                          (plane == 0 ? a.p1 : a.p2) + (first + r) * a.row_words + w0, row_bytes, full);
                        }
                    }
                }
                if (++slot == slots) { slot = 0; phase ^= 1u; }
            }
        }
        return;
    }

    // ================================================================== consumers
    const float* LV = tab + L * F;
    if constexpr (TABLE) {
        float* LVw = tab + L * F;
        for (int idx = threadIdx.x; idx < L * F; idx += kRingConsumers) {
            const int q = idx % a.wc, ci = idx / a.wc, i = ci % FPW, c = ci / FPW;
            const int f = q * FPW + i;
            LVw[idx] = (f < fcnt) ? __ldg(a.levels + (j0 + f) * L + c) : 0.0f;
        }
        consumer_sync();
    }
    // Turns the model values of this thread's word (as the gradient will see them) into what phase A
    // reads; every consumer calls it, `have` says whether the thread holds a word (parts are at most
    // one word per consumer wide).  Returns delta_w, the value of one fixed-point unit of w.
    uint32_t* wd32 = reinterpret_cast<uint32_t*>(tab);      // uniform: digits of w, [k-slab][group][digit][8 words]
    double base_w = 0.0;                         // lo^T x~ over the CTA's feature part (uniform grids)
    auto word_stage = [&](bool have, int q, const float (&xt)[FPW]) -> double {
        if constexpr (!TABLE) {
            float wv[FPW];
            float lsum = 0.0f, m = 0.0f;
#pragma unroll
            for (int i = 0; i < FPW; ++i) {
                const int f = q * FPW + i;
                float sv = 0.0f, lv = 0.0f;
                if (have && f < fcnt) { sv = __ldg(a.step + j0 + f); lv = __ldg(a.lo + j0 + f); }
                wv[i] = sv * xt[i];
                lsum = fmaf(lv, xt[i], lsum);
                m = fmaxf(m, fabsf(wv[i]));
            }
            {
                const double wb = warp_sum((double)lsum);
                if (lane == 0) sh->wbase[warp] = wb;
            }
            const float wmax = consumer_max(m, sh, 0);     // its barrier also publishes wbase
            base_w = 0.0;
#pragma unroll
            for (int w = 0; w < kRingWarps; ++w) base_w += sh->wbase[w];
            const float inv = wmax > 0.0f ? QMAXF / wmax : 0.0f;
            if (have) {
#pragma unroll
                for (int g = 0; g < NG; ++g) {
                    // B operand of phase A: per k-slab (8 words), group and digit a 32-byte k vector
                    const float v4[4] = {wv[0 * NG + g], wv[1 * NG + g], wv[2 * NG + g], wv[3 * NG + g]};
                    const uint4 o = digit_words<NS>(v4, inv);
                    uint32_t* dst = wd32 + (size_t)(((q >> 3) * NG + g) * NS) * 8 + (q & 7);
                    dst[0] = o.x; dst[8] = o.y; dst[16] = o.z; dst[24] = o.w;
                }
            }
            return (double)wmax / (double)QMAXF;
        } else {
            if (have) {
#pragma unroll
                for (int i = 0; i < FPW; ++i)
                    for (int c = 0; c < L; ++c) tab[(c * FPW + i) * a.wc + q] = LV[(c * FPW + i) * a.wc + q] * xt[i];
            }
            return 0.0;
        }
    };

    // own sub-slice of the feature part, and who acts for feature k of it: a thread when few CTAs
    // contribute, lane 0 of a warp (whose lanes split the contributors) when many do
    const int sub0 = min(F, bi * a.sub), sub1 = min(F, sub0 + a.sub);
    const int nsub = sub1 - sub0;
    const bool warp_path = a.nb > 32;
    const int kstart = warp_path ? warp : threadIdx.x, kstride = warp_path ? kRingWarps : kRingConsumers;
    const bool actor = !warp_path || lane == 0;

    // first step: model from the caller's vector
    double delta_w = 0.0;                        // one fixed-point unit of w, renewed with the model every step
    {
        VecQuant q3{0.0f, 1, a.seed, a.epoch, (uint32_t)a.first_step, 3u};
        if (a.model_bits > 0) {
            double ss = 0.0;
            for (int64_t j = threadIdx.x; j < a.n; j += kRingConsumers) { const double v = (double)a.x[j]; ss += v * v; }
            q3.M = (float)sqrt(consumer_sum(ss, sh->red));
            q3.sm = (1 << (a.model_bits - 1)) - 1;
        }
        {
            const int q = threadIdx.x;
            const bool have = q < a.wc;
            float xt[FPW];
#pragma unroll
            for (int i = 0; i < FPW; ++i) {
                const int f = q * FPW + i;
                xt[i] = (have && f < fcnt) ? a.x[j0 + f] : 0.0f;
                if (a.model_bits > 0 && have) xt[i] = q3.apply(xt[i], (uint32_t)(j0 + f));
                if (a.model_out && a.num_steps == 1 && bi == 0 && have && f < fcnt) a.model_out[j0 + f] = xt[i];
            }
            delta_w = word_stage(have, q, xt);
        }
        for (int k = threadIdx.x; k < nsub; k += kRingConsumers) xown[k] = (sub0 + k < fcnt) ? a.x[j0 + sub0 + k] : 0.0f;
        if constexpr (!TABLE)
            for (int i = threadIdx.x; i < 8 * a.rc; i += kRingConsumers) dacc[i] = 0;
        int64_t r0; int bt, rcnt;
        step_rows(a.first_step, r0, bt, rcnt);
        float* bcur = bsm + (size_t)(a.first_step & 1) * a.rc;
        for (int r = threadIdx.x; r < rcnt; r += kRingConsumers) bcur[r] = __ldg(a.b + r0 + k0 + r);
    }
    consumer_sync();

    // step-invariant thread roles of phase B and where this CTA's packets go and come from
    const int lanes_q = min(kRingConsumers, ((wcnt + 31) / 32) * 32);
    const int ngroups = kRingConsumers / lanes_q;
    const int group = threadIdx.x / lanes_q;
    const int ql = threadIdx.x % lanes_q;
    const int chunks_w = (wcnt + 31) / 32;
    const int kw8 = (wcnt + 7) / 8;              // k-slabs (8 words) per code group in the integer path
    unsigned long long* rs_mine = a.ll_rs + (size_t)ai * a.nb * a.nb * subp;                 // + (owner*nb + writer)*subp
    const unsigned long long* rs_own = rs_mine + (size_t)bi * a.nb * subp;                   // collected by this owner
    unsigned long long* ag_part = a.ll_ag + j0;
    int rs_off[FPW];                             // packet of feature i of this thread's word, for the writer bi
#pragma unroll
    for (int i = 0; i < FPW; ++i) {
        const int f = ql * FPW + i;
        const int owner = min(f / a.sub, a.nb - 1);
        rs_off[i] = (owner * a.nb + bi) * subp + (f - owner * a.sub);
    }
    int slot = 0;
    uint32_t phase = 0;

    for (int64_t it = a.first_step; it < step_end; ++it) {
        int64_t r0; int bt, rcnt;
        step_rows(it, r0, bt, rcnt);
        const int C = (rcnt + a.cr - 1) / a.cr;
        const bool last = (it == step_end - 1);
        const uint32_t tag = (uint32_t)(it - a.first_step) + 1u;
        const int par = (int)(it & 1);
        const float* bcur = bsm + (size_t)par * a.rc;
        trace_mark(a, it, 0);

        // labels of the next step's rows: requested now, parked in shared memory at the end of the step
        float breg = 0.0f;
        int rcnt_next = 0;
        int64_t r0_next = 0;
        if (!last) {
            int btn;
            step_rows(it + 1, r0_next, btn, rcnt_next);
            if ((int)threadIdx.x < rcnt_next) breg = __ldg(a.b + r0_next + k0 + threadIdx.x);
        }

        // -------------------------------------------------------------- phase A: dots
        const bool dots_local = (a.na == 1);
        unsigned long long* pd_mine = a.ll_pd + (((size_t)par * a.nb + bi) * a.na + ai) * a.rc * 4;
        int slot_a = slot, slot_a2 = slot;       // slot(s) of the single chunk when C == 1 (uniform: one per plane)
        // A warp takes four rows at a time: one load of w's digit words serves them all and the
        // eight (row, plane) sums are independent chains.  When the tile has fewer row blocks than warps
        // (single-chunk tiles only) a block's words are split over S warps.
        constexpr int RB = 4;
        int S = 1;
        {
            const int nblk_all = (rcnt + RB - 1) / RB;
            if (TABLE && C == 1 && nblk_all > 0 && nblk_all < kRingWarps) S = max(1, min(chunks_w, kRingWarps / nblk_all));
        }
        const int cps = (chunks_w + S - 1) / S;
        double wsum = 0.0;                       // r1 + r2 (one of them per lane) over what this thread finished
        float rmax = 0.0f;                       // and the largest |residual| this thread produced
        const int vmine = (lane >> 2) & 7;       // after the butterfly a lane holds sum number vmine = 2*row + plane
        for (int chunk = 0; chunk < C; ++chunk) {
            const int rows = min(a.cr, rcnt - chunk * a.cr);
            ring_wait(sh->full + slot, phase, &sh->abort_flag, a.status, 6);
            const uint32_t* t1 = ring + (size_t)slot * slot_words;
            const uint32_t* t2 = t1 + (size_t)a.cr * pitch;
            if constexpr (!TABLE) {
                // Integer dots on the tensor cores, one plane (one ring slot) after the other.  A k-slab is
                // 8 words (32 bytes of codes) of a row; a warp takes every kRingWarps-th slab for the chunk's
                // one or two blocks of 16 rows: the code bytes come as A fragments straight from the tile
                // (ldmatrix), each code group of the bytes meets its own digit vectors of w (B fragments,
                // ldmatrix), all in the same accumulators.  The warps' digit sums meet in dacc (integer sums:
                // the order of the atomics does not matter).  Rows past the chunk's last one are read (clamped
                // to the slot) and dropped; words past the part's last one meet zero digits.
                const int gl = lane >> 2, tl = lane & 3, lm = lane >> 3, l8 = lane & 7;
                const uint32_t wbase_addr = smem_u32(wd32), zero_addr = smem_u32(&sh->zero16);
#pragma unroll 1
                for (int pl = 0; pl < 2; ++pl) {
                    if (pl == 1) ring_wait(sh->full + slot, phase, &sh->abort_flag, a.status, 6);
                    const uint32_t tile_addr = smem_u32(ring + (size_t)slot * slot_words);
                    int c[2][4] = {{0, 0, 0, 0}, {0, 0, 0, 0}};
                    const uint32_t arow0 = tile_addr + (uint32_t)min(l8 + (lm & 1) * 8, a.cr - 1) * (uint32_t)pitch * 4u + (lm >> 1) * 16u;
                    const uint32_t arow1 = tile_addr + (uint32_t)min(16 + l8 + (lm & 1) * 8, a.cr - 1) * (uint32_t)pitch * 4u + (lm >> 1) * 16u;
                    const bool two_blocks = rows > 16;
#pragma unroll 2
                    for (int ks = warp; ks < kw8; ks += kRingWarps) {
                        uint32_t bf[NG][2], ar0[4], ar1[4];
                        ldsm_x4(ar0, arow0 + (uint32_t)ks * 32u);
                        ldsm_x4(ar1, (two_blocks ? arow1 : arow0) + (uint32_t)ks * 32u);
#pragma unroll
                        for (int g = 0; g < NG; ++g)
                            ldsm_x2(bf[g][0], bf[g][1],
                                    l8 < NS ? wbase_addr + (uint32_t)(((ks * NG + g) * NS + l8) * 32 + (lm & 1) * 16) : zero_addr);
#pragma unroll
                        for (int g = 0; g < NG; ++g) {
                            mma_u8s8(c[0], group_bytes<CB>(ar0[0], g), group_bytes<CB>(ar0[1], g), group_bytes<CB>(ar0[2], g),
                                     group_bytes<CB>(ar0[3], g), bf[g][0], bf[g][1]);
                            mma_u8s8(c[1], group_bytes<CB>(ar1[0], g), group_bytes<CB>(ar1[1], g), group_bytes<CB>(ar1[2], g),
                                     group_bytes<CB>(ar1[3], g), bf[g][0], bf[g][1]);
                        }
                    }
                    if (tl < 2) {                        // columns 2t, 2t+1 are digits; dacc is [row][plane][digit]
#pragma unroll
                        for (int rb = 0; rb < 2; ++rb) {
                            const int la = rb * 16 + gl, lh = la + 8;
                            int* d = dacc + (size_t)(chunk * a.cr + la) * 8 + pl * 4 + 2 * tl;
                            if (la < rows) { atomicAdd(d, c[rb][0]); atomicAdd(d + 1, c[rb][1]); }
                            if (lh < rows) { atomicAdd(d + 64, c[rb][2]); atomicAdd(d + 65, c[rb][3]); }
                        }
                    }
                    if (C > 1) {                         // hand the slot back; phase B fetches the chunk again
                        __syncwarp();
                        if (lane == 0) mbar_arrive(reinterpret_cast<uint64_t*>(sh->empty + slot));
                    } else if (pl == 0) {
                        slot_a = slot;                   // the single chunk stays: plane 1 here, plane 2 in the next slot
                    } else {
                        slot_a2 = slot;
                    }
                    if (++slot == slots) { slot = 0; phase ^= 1u; }
                }
            } else {
                const int nblk = (rows + RB - 1) / RB;
                for (int task = warp; task < nblk * S; task += kRingWarps) {
                    const int blk = task / S, seg = task - blk * S;
                    const uint32_t* rowp1 = t1 + (size_t)(blk * RB) * pitch;
                    const uint32_t* rowp2 = t2 + (size_t)(blk * RB) * pitch;
                    float fa[2 * RB];
#pragma unroll
                    for (int v = 0; v < 2 * RB; ++v) fa[v] = 0.0f;
                    const int c_end = min(chunks_w, (seg + 1) * cps);
#pragma unroll 2
                    for (int c = seg * cps; c < c_end; ++c) {
                        const int q = c * 32 + lane;
                        if (q < wcnt) {
                            uint32_t u[2 * RB];      // rows past the chunk's last one read leftovers of the slot; never used
#pragma unroll
                            for (int r = 0; r < RB; ++r) { u[2 * r] = rowp1[(size_t)r * pitch + q]; u[2 * r + 1] = rowp2[(size_t)r * pitch + q]; }
#pragma unroll
                            for (int i = 0; i < FPW; ++i) {
#pragma unroll
                                for (int v = 0; v < 2 * RB; ++v) fa[v] += tab[(code_at<CB>(u[v], i) * FPW + i) * a.wc + q];
                            }
                        }
                    }
                    double pv[2 * RB];
#pragma unroll
                    for (int v = 0; v < 2 * RB; ++v) pv[v] = (double)fa[v];
                    const double dsum = reduce8(pv, lane);
                    if ((lane & 3) == 0) {
                        const int lr = blk * RB + (vmine >> 1), plane = vmine & 1;
                        const int r = chunk * a.cr + lr;
                        if (S > 1) {
                            sh->dpart[task * 8 + vmine] = dsum;
                        } else if (lr < rows) {
                            if (dots_local) {
                                const float rv = (float)(dsum - (double)bcur[r]);
                                res[2 * r + plane] = rv;
                                wsum += (double)rv;
                                rmax = fmaxf(rmax, fabsf(rv));
                            } else {
                                ll_store_double(pd_mine + (size_t)r * 4 + 2 * plane, dsum, tag);
                            }
                        }
                    }
                }
            }
            if (TABLE && C > 1) {                // hand the slot back; phase B fetches the chunk again
                __syncwarp();
                if (lane == 0) mbar_arrive(reinterpret_cast<uint64_t*>(sh->empty + slot));
                if (++slot == slots) { slot = 0; phase ^= 1u; }
            }
        }
        if constexpr (!TABLE) {                  // one thread per (row, plane) takes the digit sums and clears them
            consumer_sync();
            for (int idx = threadIdx.x; idx < 2 * rcnt; idx += kRingConsumers) {
                const int4 dv = *reinterpret_cast<const int4*>(dacc + (size_t)idx * 4);
                *reinterpret_cast<int4*>(dacc + (size_t)idx * 4) = make_int4(0, 0, 0, 0);
                const int dd[NS] = {dv.x, dv.y, dv.z, dv.w};
                const double d = (double)combine_digits<NS>(dd) * delta_w + base_w;
                const int r = idx >> 1, plane = idx & 1;
                if (dots_local) {
                    const float rv = (float)(d - (double)bcur[r]);
                    res[idx] = rv;
                    wsum += (double)rv;
                    rmax = fmaxf(rmax, fabsf(rv));
                } else {
                    ll_store_double(pd_mine + (size_t)r * 4 + 2 * plane, d, tag);
                }
            }
        } else if (S > 1) {                      // single chunk: one thread per (row, plane) adds the segments in order
            consumer_sync();
            if ((int)threadIdx.x < 2 * rcnt) {
                const int r = threadIdx.x >> 1, plane = threadIdx.x & 1;
                const int blk = r / RB, vv = 2 * (r - blk * RB) + plane;
                double d = 0.0;
                for (int sg = 0; sg < S; ++sg) d += sh->dpart[(blk * S + sg) * 8 + vv];
                if (dots_local) {
                    const float rv = (float)(d - (double)bcur[r]);
                    res[2 * r + plane] = rv;
                    wsum += (double)rv;
                    rmax = fmaxf(rmax, fabsf(rv));
                } else {
                    ll_store_double(pd_mine + (size_t)r * 4 + 2 * plane, d, tag);
                }
            }
        }
        wsum = warp_sum(wsum);
        if (dots_local) {
            if (lane == 0) sh->red[warp] = wsum;
        } else {
            // every row's dot is the sum, in part order, of the na partial dots published for it
            const unsigned long long* pd_row = a.ll_pd + ((size_t)par * a.nb + bi) * a.na * a.rc * 4;
            double part = 0.0;
            for (int r = threadIdx.x; r < rcnt; r += kRingConsumers) {
                double d1 = 0.0, d2 = 0.0;
                bool good = !*reinterpret_cast<volatile int*>(&sh->abort_flag);
                // four parts at a time, their sixteen packets in flight together
                for (int p0 = 0; p0 < a.na && good; p0 += 4) {
                    const unsigned long long* src = pd_row + ((size_t)p0 * a.rc + r) * 4;
                    const int np = min(4, a.na - p0);
                    unsigned long long v[4][4];
                    bool ok = false;
                    for (long long spin = 0; spin < kPacketSpinLimit && !ok; ++spin) {
                        ok = true;
#pragma unroll
                        for (int pp = 0; pp < 4; ++pp)
                            if (pp < np) {
#pragma unroll
                                for (int u = 0; u < 4; ++u) {
                                    v[pp][u] = ll_load(src + (size_t)pp * a.rc * 4 + u);
                                    ok = ok && ((uint32_t)(v[pp][u] >> 32) == tag);
                                }
                            }
                    }
                    if (!ok) { sh->abort_flag = 1; set_status(a.status, ZIPML_ERR_TIMEOUT, 1); good = false; break; }
#pragma unroll
                    for (int pp = 0; pp < 4; ++pp)
                        if (pp < np) {
                            d1 += (double)__uint_as_float((uint32_t)v[pp][0]) + (double)__uint_as_float((uint32_t)v[pp][1]);
                            d2 += (double)__uint_as_float((uint32_t)v[pp][2]) + (double)__uint_as_float((uint32_t)v[pp][3]);
                        }
                }
                const double bk = (double)bcur[r];
                const float r1 = good ? (float)(d1 - bk) : 0.0f, r2 = good ? (float)(d2 - bk) : 0.0f;
                res[2 * r] = r1;
                res[2 * r + 1] = r2;
                part += (double)r1 + (double)r2;
                rmax = fmaxf(rmax, fmaxf(fabsf(r1), fabsf(r2)));
            }
            part = warp_sum(part);
            if (lane == 0) sh->red[warp] = part;
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) rmax = fmaxf(rmax, __shfl_xor_sync(0xffffffffu, rmax, o));
        if (lane == 0) sh->fmax[16 + warp] = rmax;
        consumer_sync();                         // residuals, their per-warp sums and maxima are complete
        double delta_r = 0.0;                    // one fixed-point unit of the residuals of this step
        if constexpr (!TABLE) {
            float rho = 0.0f;
#pragma unroll
            for (int w = 0; w < kRingWarps; ++w) rho = fmaxf(rho, sh->fmax[16 + w]);
            const float inv = rho > 0.0f ? QMAXF / rho : 0.0f;
            delta_r = (double)rho / (double)QMAXF;
            // digits of the residuals as B operands of phase B: per 32 rows and residual, per digit, 32 bytes
            // in the row order the transposed code fragments come in (k = 16h + 4t + e <-> row 16h + 2t +
            // (e & 1) + 8 (e >> 1)); rows past the batch count as zero
            uint32_t* rd32w = reinterpret_cast<uint32_t*>(rdig);
            for (int kk = threadIdx.x; kk < 8 * ((rcnt + 31) / 32); kk += kRingConsumers) {
                const int rbase = (kk >> 3) * 32 + ((kk >> 2) & 1) * 16 + 2 * (kk & 3);
                float v1[4], v2[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const int k = rbase + (e & 1) + 8 * (e >> 1);
                    v1[e] = k < rcnt ? res[2 * k] : 0.0f;
                    v2[e] = k < rcnt ? res[2 * k + 1] : 0.0f;
                }
                const uint4 o1 = digit_words<NS>(v1, inv), o2 = digit_words<NS>(v2, inv);
                uint32_t* d1 = rd32w + (size_t)((kk >> 3) * 2 * NS) * 8 + (kk & 7);
                d1[0] = o1.x; d1[8] = o1.y; d1[16] = o1.z; d1[24] = o1.w;
                d1[32] = o2.x; d1[40] = o2.y; d1[48] = o2.z; d1[56] = o2.w;
            }
            consumer_sync();
        }
        trace_mark(a, it, 1);

        // -------------------------------------------------------------- phase B: gradient
        if constexpr (!TABLE) {
            // Integer gradient parts on the tensor cores, one plane (one ring slot) after the other.  A task
            // is a 16-byte column of the tile over its 32 rows; a warp keeps the accumulators of its columns
            // (every kRingWarps-th) across the chunks.  A transposing ldmatrix hands each lane the bytes
            // {2g, 2g+1} of rows {2t, 2t+1} of the four 8-row groups; two permutes per half turn them into A
            // fragments "byte 2g (or 2g+1) of the column, four rows", i.e. features x rows with the row order
            // the residual digits were stored in.  Each code group of the bytes meets the residual digits
            // (plane 1 those of r2, plane 2 those of r1) in its own accumulators.
            constexpr int TI = (CB == 2) ? kRingTasks / 2 : kRingTasks;       // columns per warp
            const int gl = lane >> 2, tl = lane & 3, lm = lane >> 3, l8 = lane & 7;
            const uint32_t rbase_addr = smem_u32(rdig), zero_addr = smem_u32(&sh->zero16);
            const int ncol = (wcnt + 3) / 4;
            const unsigned sub_magic = (unsigned)((0x100000000ull + (unsigned)a.sub - 1) / (unsigned)a.sub);   // ceil(2^32 / sub)
            int acc[TI][NG][4];
#pragma unroll
            for (int ti = 0; ti < TI; ++ti)
#pragma unroll
                for (int g = 0; g < NG; ++g)
#pragma unroll
                    for (int e = 0; e < 4; ++e) acc[ti][g][e] = 0;
            for (int ci = 0; ci < C; ++ci) {
                const int chunk = C - 1 - ci;
                const int slab = chunk * a.cr / 32;              // chunks are 32 rows, or the tile is one chunk
#pragma unroll 1
                for (int pl = 0; pl < 2; ++pl) {
                    int use_slot = pl ? slot_a2 : slot_a;
                    if (C > 1) {
                        ring_wait(sh->full + slot, phase, &sh->abort_flag, a.status, 7);
                        use_slot = slot;
                    }
                    // digits of r2 for plane 1, of r1 for plane 2; rows past the chunk carry zero digits
                    uint32_t b0, b1;
                    ldsm_x2(b0, b1, l8 < NS ? rbase_addr + (uint32_t)(((slab * 2 + (1 - pl)) * NS + l8) * 32 + (lm & 1) * 16) : zero_addr);
                    const uint32_t row_addr = smem_u32(ring + (size_t)use_slot * slot_words) +
                                              (uint32_t)min(lane, a.cr - 1) * (uint32_t)pitch * 4u;
                    // four columns at a time: their loads are issued together, then the permutes and MMAs
#pragma unroll
                    for (int t0 = 0; t0 < TI; t0 += 4) {
                        uint32_t r4[4][4];
#pragma unroll
                        for (int tj = 0; tj < 4; ++tj) {
                            const int col = min(warp + (t0 + tj) * kRingWarps, ncol - 1);      // clamped: results dropped below
                            ldsm_x4_trans(r4[tj], row_addr + (uint32_t)col * 16u);
                        }
#pragma unroll
                        for (int tj = 0; tj < 4; ++tj) {
                            if (warp + (t0 + tj) * kRingWarps < ncol) {
                                const uint32_t pel = __byte_perm(r4[tj][0], r4[tj][1], 0x6420), pol = __byte_perm(r4[tj][0], r4[tj][1], 0x7531);
                                const uint32_t peh = __byte_perm(r4[tj][2], r4[tj][3], 0x6420), poh = __byte_perm(r4[tj][2], r4[tj][3], 0x7531);
#pragma unroll
                                for (int g = 0; g < NG; ++g)
                                    mma_u8s8(acc[t0 + tj][g], group_bytes<CB>(pel, g), group_bytes<CB>(pol, g), group_bytes<CB>(peh, g),
                                             group_bytes<CB>(poh, g), b0, b1);
                            }
                        }
                    }
                    if (C > 1) {
                        __syncwarp();
                        if (lane == 0) mbar_arrive(reinterpret_cast<uint64_t*>(sh->empty + slot));
                        if (++slot == slots) { slot = 0; phase ^= 1u; }
                    }
                }
            }
            if (C == 1) {                        // the retained single chunk goes back now, both planes
                __syncwarp();
                if (lane == 0) {
                    mbar_arrive(reinterpret_cast<uint64_t*>(sh->empty + slot_a));
                    mbar_arrive(reinterpret_cast<uint64_t*>(sh->empty + slot_a2));
                }
            }
            // columns 2t, 2t+1 of lane t < 2 are digits 2t, 2t+1: combine, add the pair of lanes, send.
            // Accumulator rows g, g+8 are bytes 2g, 2g+1 of the column.
#pragma unroll
            for (int ti = 0; ti < TI; ++ti) {
                const int col = warp + ti * kRingWarps;
                if (col < ncol) {
#pragma unroll
                    for (int g = 0; g < NG; ++g) {
#pragma unroll
                        for (int odd = 0; odd < 2; ++odd) {
                            // digit pair of this lane in double (exact), the other pair comes from lane t+1
                            const double pair = (double)acc[ti][g][2 * odd] + 128.0 * (double)acc[ti][g][2 * odd + 1];
                            const double upper = __shfl_down_sync(0xffffffffu, pair, 1);
                            const int byte_in_part = col * 16 + 2 * gl + odd;
                            const int q = byte_in_part >> 2, b = byte_in_part & 3;
                            if (tl == 0 && q < wcnt) {
                                const int f = q * FPW + b * NG + g;
                                const int owner = min((int)__umulhi((unsigned)f, sub_magic), a.nb - 1);     // f / sub, f < 2^16
                                ll_store(rs_mine + ((size_t)owner * a.nb + bi) * subp + (f - owner * a.sub),
                                         (float)((pair + 16384.0 * upper) * delta_r), tag);
                            }
                        }
                    }
                }
            }
        } else
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
                        const uint32_t* col2 = col1 + (size_t)a.cr * pitch;
                        const float* rr = res + 2 * chunk * a.cr;
#pragma unroll 4
                        for (int lr = group; lr < rows; lr += ngroups) {
                            const uint32_t u1 = col1[(size_t)lr * pitch];
                            const uint32_t u2 = col2[(size_t)lr * pitch];
                            const float2 rv = *reinterpret_cast<const float2*>(rr + 2 * lr);
                            const float r1 = rv.x, r2 = rv.y;
#pragma unroll
                            for (int i = 0; i < FPW; ++i) {
                                const float l1 = LV[(code_at<CB>(u1, i) * FPW + i) * a.wc + q];
                                const float l2 = LV[(code_at<CB>(u2, i) * FPW + i) * a.wc + q];
                                acc[i] = fmaf(l1, r2, fmaf(l2, r1, acc[i]));
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
#pragma unroll
                    for (int i = 0; i < FPW; ++i) ll_store(rs_mine + rs_off[i], acc[i], tag);
                }
            }
        if (TABLE && C == 1) {                   // the retained single chunk goes back now
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
        if ((int)threadIdx.x < a.nb) {
            double ssum = 0.0;
#pragma unroll
            for (int w = 0; w < kRingWarps; ++w) ssum += sh->red[w];
            for (int o = threadIdx.x; o < a.nb; o += kRingConsumers)
                ll_store_double(rs_mine + ((size_t)o * a.nb + bi) * subp + a.sub, ssum, tag);
        }
        trace_mark(a, it, 2);

        // -------------------------------------------------------------- reduce-scatter: own sub-slice
        ll_wait_sentinels(rs_own + a.sub, subp, a.nb, tag, sh, a.status, 2);      // each contributor's residual sum
        ll_gather(rs_own, a.nb * subp, tag, gbuf, sh, a.status, 2);
        consumer_sync();
        trace_mark(a, it, 3);
        double stot = 0.0;
        if (warp_path) {
            double t = 0.0;
            for (int w = lane; w < a.nb; w += 32) t += (double)gbuf[w * subp + a.sub] + (double)gbuf[w * subp + a.sub + 1];
            stot = warp_sum(t);
        } else {
            for (int w = 0; w < a.nb; ++w) stot += (double)gbuf[w * subp + a.sub] + (double)gbuf[w * subp + a.sub + 1];
        }
        const double scale = 1.0 / (2.0 * (double)bt);
        double gsq = 0.0;
        for (int k = kstart; k < nsub; k += kstride) {
            double t = 0.0;
            if (warp_path) {
                for (int w = lane; w < a.nb; w += 32) t += (double)gbuf[w * subp + k];
                t = warp_sum(t);
            } else {
                for (int w = 0; w < a.nb; ++w) t += (double)gbuf[w * subp + k];
            }
            if (actor) {
                const int f = sub0 + k;
                float g = 0.0f;
                if (f < fcnt) {
                    if constexpr (!TABLE) t = (double)__ldg(a.lo + j0 + f) * stot + (double)__ldg(a.step + j0 + f) * t;
                    g = (float)(t * scale);
                    if (last && a.grad_out) a.grad_out[j0 + f] = g;
                }
                gsub[k] = g;
                gsq += (double)g * (double)g;
            }
        }
        VecQuant q4{0.0f, 1, a.seed, a.epoch, (uint32_t)it, 4u};
        if (a.grad_bits > 0) {
            gsq = consumer_sum(gsq, sh->red);
            unsigned long long* gn = a.ll_gn + (size_t)par * G * 2;
            if (threadIdx.x == 0) ll_store_double(gn + (size_t)blockIdx.x * 2, gsq, tag);
            ll_gather(gn, 2 * G, tag, nbuf, sh, a.status, 3);
            consumer_sync();
            double part = 0.0;
            for (int p = lane; p < G; p += 32) part += (double)nbuf[2 * p] + (double)nbuf[2 * p + 1];
            q4.M = (float)sqrt(warp_sum(part));  // every warp adds the same numbers in the same order
            q4.sm = (1 << (a.grad_bits - 1)) - 1;
        }
        double xsq = 0.0;
        for (int k = kstart; k < nsub; k += kstride) {
            if (actor) {
                const int f = sub0 + k;
                float xn = 0.0f;
                if (f < fcnt) {
                    float g = gsub[k];
                    if (a.grad_bits > 0) g = q4.apply(g, (uint32_t)(j0 + f));
                    if (last && a.grad_out) a.grad_out[a.n + j0 + f] = g;
                    xn = regularise(fmaf(-a.lr, g, xown[k]), xown[k], a.reg, a.reg_cst);
                }
                xown[k] = xn;
                xsq += (double)xn * (double)xn;
            }
        }
        trace_mark(a, it, 4);
        if (last) break;

        // what the next step's gradient will see: Q3 of the new model, or the model itself
        VecQuant q3{0.0f, 1, a.seed, a.epoch, (uint32_t)(it + 1), 3u};
        if (a.model_bits > 0) {
            xsq = consumer_sum(xsq, sh->red);
            unsigned long long* xnp = a.ll_ag + npad + (size_t)par * G * 2;
            if (threadIdx.x == 0) ll_store_double(xnp + (size_t)blockIdx.x * 2, xsq, tag);
            ll_gather(xnp, 2 * G, tag, nbuf, sh, a.status, 8);
            consumer_sync();
            double part = 0.0;
            for (int p = lane; p < G; p += 32) part += (double)nbuf[2 * p] + (double)nbuf[2 * p + 1];
            q3.M = (float)sqrt(warp_sum(part));
            q3.sm = (1 << (a.model_bits - 1)) - 1;
        }
        for (int k = kstart; k < nsub; k += kstride) {
            if (actor) {
                const int f = sub0 + k;
                float xt = xown[k];
                if (a.model_bits > 0 && f < fcnt) xt = q3.apply(xt, (uint32_t)(j0 + f));
                if (a.model_out && it + 2 == a.first_step + a.num_steps && f < fcnt) a.model_out[j0 + f] = xt;
                ll_store(ag_part + f, xt, tag);
            }
        }
        trace_mark(a, it, 5);

        // -------------------------------------------------------------- all-gather: the part's model, word by word
        ll_wait_sentinels(ag_part, a.sub, (F + a.sub - 1) / a.sub, tag, sh, a.status, 4);  // each owner's first feature
        trace_mark(a, it, 6);
        {
            const int q = threadIdx.x;
            const bool have = q < a.wc;
            float xt[FPW];
#pragma unroll
            for (int i = 0; i < FPW; ++i) xt[i] = 0.0f;
            if (have) {
                const unsigned long long* src = ag_part + (size_t)q * FPW;
                unsigned long long v[FPW];
                bool ok = false;
                if (!*reinterpret_cast<volatile int*>(&sh->abort_flag)) {
                    for (long long spin = 0; spin < kPacketSpinLimit && !ok; ++spin) {
                        ok = true;
#pragma unroll
                        for (int i = 0; i < FPW; ++i) { v[i] = ll_load(src + i); ok = ok && ((uint32_t)(v[i] >> 32) == tag); }
                    }
                    if (!ok) { sh->abort_flag = 1; set_status(a.status, ZIPML_ERR_TIMEOUT, 4); }
                }
#pragma unroll
                for (int i = 0; i < FPW; ++i) xt[i] = ok ? __uint_as_float((uint32_t)v[i]) : 0.0f;
            }
            delta_w = word_stage(have, q, xt);
        }
        {
            float* bnext = bsm + (size_t)(par ^ 1) * a.rc;
            if ((int)threadIdx.x < rcnt_next) bnext[threadIdx.x] = breg;
            for (int r = threadIdx.x + kRingConsumers; r < rcnt_next; r += kRingConsumers) bnext[r] = __ldg(a.b + r0_next + k0 + r);
        }
        consumer_sync();
        trace_mark(a, it, 7);
    }
    consumer_sync();
    // every owner returns its sub-slice of the master model
    for (int k = threadIdx.x; k < nsub; k += kRingConsumers)
        if (sub0 + k < fcnt) a.x[j0 + sub0 + k] = xown[k];
}

// ---------------------------------------------------------------------------------------------
// Host side
// ---------------------------------------------------------------------------------------------
struct RingPlan {
    int na, nb, wc, rc, cr, slots, sub, pitch;
    size_t smem;
};

// Rows of a chunk lie `pitch` words apart in shared memory.  The integer path reads 8 rows x 4 words per
// tensor-core fragment load; a pitch of wc (a multiple of 32 words) would put all rows in the same banks.
static int ring_pitch(bool table, int wc) { return table ? wc : wc + 4; }

static size_t ring_smem_bytes(int cb, bool table, int wc, int rc, int bits, int sub, int cr, int slots, int nb, int G) {
    const int fpw = 32 / cb;
    const size_t F = (size_t)wc * fpw, L = (size_t)1 << bits;
    const size_t subp = (size_t)sub + 2;
    size_t bytes = (sizeof(RingShared) + 15) & ~(size_t)15;
    bytes += sizeof(float) * ((table ? 2 * L * F : F) + 2 * (size_t)sub + (((size_t)nb * subp + 3) & ~(size_t)3));
    bytes += sizeof(float) * (((2 * (size_t)G + 3) & ~(size_t)3) + (table ? (size_t)kRingConsumers * fpw : 0) + 2 * (size_t)((2 * rc + 3) & ~3));
    bytes += 256 * (size_t)((rc + 31) / 32) + (table ? 0 : sizeof(int) * 8 * (size_t)rc) + 128;   // + slack to align the ring
    bytes += sizeof(uint32_t) * (size_t)slots * (table ? 2 : 1) * cr * ring_pitch(table, wc);   // uniform: one plane per slot
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
        // chunk: about 64 KiB of codes (eight 4-row blocks of a full-width part: one per consumer warp)
        int cr = (int)(65536 / (2 * (size_t)r.wc * 4));
        cr = (cr + 3) & ~3;                                   // phase B walks a slot four rows at a time
        cr = cr < 4 ? 4 : cr;
        if (cr > ((r.rc + 3) & ~3) || wide) cr = (r.rc + 3) & ~3;
        if (!table) cr = r.rc <= 16 ? 16 : 32;                // integer path: fragments of 16 rows, k-slabs of 32 rows
        r.cr = cr;
        r.pitch = ring_pitch(table, r.wc);
        if (sizeof(uint32_t) * 2 * (size_t)cr * r.wc >= (1u << 20)) return false;   // mbarrier tx-count range
        int slots = kRingMaxSlots;
        while (slots >= 2 && ring_smem_bytes(cb, table, r.wc, r.rc, d->bits, r.sub, cr, slots, r.nb, r.na * r.nb) > cap) --slots;
        if (slots < 2) return false;
        r.slots = slots;
        r.smem = ring_smem_bytes(cb, table, r.wc, r.rc, d->bits, r.sub, cr, slots, r.nb, r.na * r.nb);
        *out = r;
        return true;
    };

    // parts are at most one word per consumer wide; phase B of the integer path keeps at most kRingTasks
    // accumulator sets per warp (8 words x groups each), which caps 2-bit parts at 128 words
    const int wc_max = table ? kRingConsumers : min(kRingConsumers, 64 * kRingTasks / (8 / cb));
    const int na_min = (int)((words + wc_max - 1) / wc_max);
    if (p->grid_feature_parts > 0 || p->grid_row_parts > 0) {
        int na = p->grid_feature_parts > 0 ? p->grid_feature_parts : 1;
        int nb = p->grid_row_parts > 0 ? p->grid_row_parts : 1;
        if ((int64_t)na * 32 > ring_round_up((int)words, 32)) na = (int)((words + 31) / 32);
        if (na < na_min) na = na_min;          // the request is a hint: parts never exceed one word column per thread
        if (nb > B) nb = (int)B;
        // more row parts than asked for when the tile of a part does not fit shared memory
        for (; nb <= B && na * nb <= sms; ++nb)
            if (shape(na, nb, plan)) return ZIPML_OK;
        return ZIPML_ERR_WORKSPACE;
    }
    // Fewest feature parts (widest contiguous row pieces).  Row parts: small steps are bound by the
    // exchange, whose cost grows with the number of CTAs, not by the tile -- measured on 0.25-1 MiB
    // steps, 32 row parts beat 148 by 10-25 % -- so use more than 32 only to keep a CTA's share of the
    // step's codes under 256 KiB, and never fewer than 8 rows per CTA.  If shared memory refuses the
    // shape, try more feature parts.
    bool found = false;
    for (int na = na_min; na <= (int)((words + 31) / 32) && na <= sms && !found; ++na) {
        const double step_bytes = 2.0 * (double)B * (double)words * 4.0;
        int nb = (int)(step_bytes / na / 262144.0) + 1;
        if (nb < 32) nb = 32;
        if (nb > sms / na) nb = sms / na;
        if ((int64_t)nb * 8 > B) nb = (int)(B / 8);
        if (nb < 1) nb = 1;
        RingPlan r;
        if (!shape(na, nb, &r) || r.na * r.nb > sms) continue;
        *plan = r;
        found = true;
    }
    return found ? ZIPML_OK : ZIPML_ERR_WORKSPACE;
}

static int64_t plane_wc_check(int wc) { return (int64_t)wc; }

// Tensor maps over the two planes seen as m x row_words matrices of 32-bit words.  The encoder is a
// driver entry point looked up through the runtime (no link against the driver library).
static int encode_plane_maps(zipml_ctx* ctx, const zipml_dataset* d, int box_words, int cr, bool wide_elements, CUtensorMap* out) {
    typedef CUresult (*EncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                 const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                 CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
    if (!ctx->tmap_encode) {
        void* fn = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess || !fn) {
            (void)cudaGetLastError();
            return ZIPML_ERR_CUDA;
        }
        ctx->tmap_encode = fn;
    }
    // 32-bit elements, or 64-bit ones for boxes wider than 256 words (a box dimension holds at most 256 elements)
    const int esz = wide_elements ? 8 : 4;
    const int box_elems = box_words * 4 / esz;
    if (box_elems > 256 || cr > 256 || (box_words * 4) % 16 != 0) return ZIPML_ERR_WORKSPACE;
    const cuuint64_t gdim[2] = {(cuuint64_t)(d->row_bytes / esz), (cuuint64_t)d->m};
    const cuuint64_t gstride[1] = {(cuuint64_t)d->row_bytes};
    const cuuint32_t box[2] = {(cuuint32_t)box_elems, (cuuint32_t)cr};
    const cuuint32_t estr[2] = {1, 1};
    const void* planes[2] = {d->plane1, d->plane2};
    for (int i = 0; i < 2; ++i) {
        const CUresult r = reinterpret_cast<EncodeFn>(ctx->tmap_encode)(
            &out[i], wide_elements ? CU_TENSOR_MAP_DATA_TYPE_UINT64 : CU_TENSOR_MAP_DATA_TYPE_UINT32, 2, const_cast<void*>(planes[i]), gdim, gstride, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) return ZIPML_ERR_CUDA;
    }
    return ZIPML_OK;
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
    const size_t n_ag = npad + 4 * (size_t)G;
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
    a.b = b; a.x = x; a.grad_out = grad_out; a.model_out = p->model_out;
    a.batch = B;
    a.first_step = first_step; a.num_steps = num_steps;
    a.lr = p->lr; a.reg = p->reg; a.reg_cst = reg_constant(p); a.model_bits = p->model_bits; a.grad_bits = p->grad_bits;
    a.seed = p->seed; a.epoch = (uint32_t)p->epoch;
    a.na = plan.na; a.nb = plan.nb; a.wc = plan.wc; a.rc = plan.rc; a.stages = plan.slots;
    a.cr = plan.cr; a.sub = plan.sub; a.pitch = plan.pitch;
    a.pd = nullptr; a.pg = nullptr; a.ps = nullptr; a.barrier = nullptr;
    a.ll_pd = reinterpret_cast<unsigned long long*>(ctx->ws + o_ll);
    a.ll_rs = a.ll_pd + n_pd;
    a.ll_gn = a.ll_rs + n_rs;
    a.ll_ag = a.ll_gn + n_gn;
    a.status = ctx->d_status;
    a.order = nullptr;
    a.phases = kPhaseAll; a.persistent = 1;
    a.trace = reinterpret_cast<unsigned long long*>(p->trace); a.trace_steps = p->trace ? p->trace_steps : 0;
    if (p->batch_order) {
        int32_t* dev_order = reinterpret_cast<int32_t*>(ctx->ws + o_ord);
        e = cudaMemcpyAsync(dev_order, p->batch_order, sizeof(int32_t) * (size_t)T, cudaMemcpyHostToDevice, ctx->stream);
        if (e != cudaSuccess) return cuda_status(e);
        a.order = dev_order;
    }
    // strided row pieces go through two tensor maps (plane 1, plane 2): box = cr rows x wc words
    CUtensorMap tmaps[2];
    memset(tmaps, 0, sizeof(tmaps));
    a.use_tmap = 0;
    if (d->m < 0x7fffffffLL && a.row_words < 0x7fffffffLL) {
        if (table) {
            if (a.row_words != plane_wc_check(plan.wc) && encode_plane_maps(ctx, d, plan.wc, plan.cr, false, tmaps) == ZIPML_OK)
                a.use_tmap = 1;
        } else if (encode_plane_maps(ctx, d, plan.pitch, plan.cr, true, tmaps) == ZIPML_OK) {
            a.use_tmap = 1;                    // uniform grids: one padded box per plane and chunk
        }
    }
    // packet tags are 32-bit step counters starting at 1
    const int64_t max_steps = 0x7fffffffLL;
    for (int64_t s0 = first_step; s0 < first_step + num_steps; s0 += max_steps) {
        e = cudaMemsetAsync(ctx->ws + o_ll, 0, ll_bytes, ctx->stream);
        if (e != cudaSuccess) return cuda_status(e);
        SgdArgs chunk = a;
        chunk.first_step = s0;
        chunk.num_steps = (first_step + num_steps - s0 < max_steps) ? first_step + num_steps - s0 : max_steps;
        if (s0 + chunk.num_steps < first_step + num_steps) { chunk.grad_out = nullptr; chunk.model_out = nullptr; }
        void* params[] = {&chunk, &tmaps[0], &tmaps[1]};
        e = cudaLaunchCooperativeKernel(kernel, dim3((unsigned)G), dim3(kRingThreads), params, plan.smem, ctx->stream);
        if (e != cudaSuccess) return cuda_status(e);
        ctx->launches += 1;
    }
    ctx->last_engine = ZIPML_ENGINE_RING;
    return ZIPML_OK;
}

}  // namespace zipml
