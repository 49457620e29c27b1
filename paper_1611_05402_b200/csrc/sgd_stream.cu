// Stream engine of zipml_sgd_epoch: large minibatch tiles on uniform grids, fp32 model and gradient.
//
// A step of the double-sampled minibatch SGD (paper Eq. (double) in its symmetrised form, footnote
// of "Double Sampling"; update in full precision, "End-to-end Quantization") is two passes over the
// step's code tile: the dots q1^T x, q2^T x of every row (pass A), then the gradient
// 1/(2B) sum_k [q1_k r2_k + q2_k r1_k] (pass B), with r = dot - b between them.  Both passes feed the
// int8 tensor cores with code bytes exactly as they lie in memory: pass A streams the tile from HBM
// and leaves it in L2, pass B re-reads it from L2.  Every warp moves its own bytes through a private
// ring of shared-memory stages with cp.async, several stages ahead of the arithmetic (in pass A a
// lane reads back only what it copied itself: no barrier; in pass B one __syncwarp per stage).
//
//   pass A   a CTA takes one column part of the row (a run of 64-byte spans) for 256 rows, a warp 16
//            of them; the part's digits of w = step * x (four balanced base-128 int8 digits) are
//            staged once per CTA.  Code bytes are the A operand of mma.sync m16n8k32 (u8 x s8), the
//            digits the B operand's columns; digit sums are exact integers, combined in 64 bits and
//            added to dots[plane][row] with integer atomics (order-free).
//   barrier  one grid barrier per step: every dot is complete.
//   resid.   every CTA computes all residuals (2B values), their common fixed-point scale and digits
//            (shared memory), redundantly and identically.
//   pass B   a CTA owns whole column blocks (64 bytes of the row = 512 / CB features) for all rows
//            of the step, so its gradient entries never leave it.  The contraction runs over rows:
//            a stage holds 32 rows x 64 bytes; a lane takes 8 bytes of 8 of them, transposes 4 x 4 byte
//            blocks with byte permutes and feeds (features x rows) fragments; the residual digits are
//            the B operand.
//   update   the owner updates its features of x (kept in shared memory for the whole launch), turns
//            w = step * x into digits for the next step and raises a per-block flag; pass A of the
//            next step waits only for the flags of the blocks it reads (no second grid barrier).
//
// The digit scale of w must be known to writers and readers without another exchange: it is a bound,
// |w_j(t+1)| <= max|w(t)| + lr * max_j(step_j * max|a_j|) * max_k|r_k(t)|, whose pieces every CTA
// already holds after the step's barrier (owners publish their part of max|w| and of lo^T x with
// the flags).  The bound costs a few of the 27 fixed-point bits while the model is still near zero.
#include <stdlib.h>
#include <string.h>

#include "int_digits.cuh"
#include "sgd_common.cuh"

namespace zipml {

constexpr int kStreamThreads = 512;
constexpr int kStreamWarps = kStreamThreads / 32;
constexpr int kStreamMaxBatch = 8192;      // residual digits of a step live in shared memory
constexpr int kStreamMaxOwn = 4;           // column blocks per CTA
constexpr int kStreamStages = 4;           // ring stages per warp
constexpr int kStreamStageBytes = 2048;    // pass A: 4 x 32 lanes x 16 B; pass B: 32 rows x 64 B
constexpr int kStreamRingBytes = kStreamWarps * kStreamStages * kStreamStageBytes;
constexpr int kStreamBlock = 64;           // bytes of a column block = one span
constexpr int kStreamMaxPartSpans = 64;    // spans of a pass-A column part

struct StreamArgs {
    const unsigned char* p1;
    const unsigned char* p2;
    int64_t row_bytes, m;
    int n, bits;
    const float* lo;
    const float* step;
    const float* b;
    float* x;
    float* grad_out;
    int64_t batch, first_step, num_steps;
    const int32_t* order;
    float lr;
    int reg;                 // ZIPML_REG_* and its fp32 constant
    float reg_cst;
    int ca;                  // pass A: column parts of the row
    int spans;               // 64-byte spans of a row = pass B's column blocks
    int part_spans;          // most spans a part holds
    int bpc;                 // column blocks per CTA
    int bpad;                // batch rounded up to 32
    int union_bytes;         // shared memory shared by pass A's digits and pass B's residual digits + sums
    int l2_prefetch;         // eighths of the next step's tile to ask L2 for while pass B runs (0..8)
    int64_t vec_bytes;       // bytes of one digit vector (spans * 64)
    signed char* wdig;       // [NG][NS][vec_bytes] digits of w, in the byte order of the codes
    unsigned* ready;         // [spans] number of digit versions published for the block
    long long* dots;         // [3][2][bpad] fixed-point dots of the step (three steps in rotation)
    float* wmax_part;        // [2][G] owners' max |w| (by step parity)
    double* base_part;       // [2][G] owners' part of lo^T x
    unsigned* barrier;
    DeviceStatus* status;
    unsigned long long* trace;
    int trace_steps;
};

__device__ __forceinline__ void stream_mark(const StreamArgs& a, int64_t t_rel, int k) {
    if (a.trace && blockIdx.x == 0 && threadIdx.x == 0 && t_rel < a.trace_steps) a.trace[t_rel * 8 + k] = (unsigned long long)clock64();
}

__device__ __forceinline__ unsigned ld_acquire_u32(const unsigned* p) {
    unsigned v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
// Flag store that follows one __threadfence() covering everything published before it.
__device__ __forceinline__ void st_relaxed_u32(unsigned* p, unsigned v) {
    asm volatile("st.relaxed.gpu.global.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ void red_add_s64(long long* p, long long v) {
    asm volatile("red.relaxed.gpu.global.add.u64 [%0], %1;" ::"l"(__cvta_generic_to_global(p)), "l"(v) : "memory");
}
__device__ __forceinline__ void prefetch_l2(const void* p) { asm volatile("prefetch.global.L2 [%0];" ::"l"(p)); }
__device__ __forceinline__ uint64_t l2_evict_first_policy() {
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}
__device__ __forceinline__ uint64_t l2_evict_normal_policy() {
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_normal.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}
// 16-byte global -> shared copy with an L2 policy, under a predicate (no branch around it): nothing is
// copied where `on` is false.
__device__ __forceinline__ void cp_async16_if(bool on, uint32_t dst, const void* src, uint64_t policy) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %0, 0;\n\t"
        "@p cp.async.cg.shared.global.L2::cache_hint [%1], [%2], 16, %3;\n\t}"
        ::"r"((int)on), "r"(dst), "l"(src), "l"(policy) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ void l2_prefetch_bulk(const void* src, uint32_t bytes) {
    asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(src), "r"(bytes) : "memory");
}

// Two maxima and a sum over the block in one round; every thread combines the warps' results in the
// same fixed order, so every thread (and every CTA given the same inputs) gets the same bits.
// Its two barriers come after the caller's earlier shared-memory writes and before anyone returns.
__device__ __forceinline__ void block_reduce_mms(float& m1, float& m2, double& s, float* shf, double* shd) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        m1 = fmaxf(m1, __shfl_xor_sync(0xffffffffu, m1, o));
        m2 = fmaxf(m2, __shfl_xor_sync(0xffffffffu, m2, o));
        s += __shfl_xor_sync(0xffffffffu, s, o);
    }
    const int warp = threadIdx.x >> 5;
    __syncthreads();
    if ((threadIdx.x & 31) == 0) { shf[warp] = m1; shf[kStreamWarps + warp] = m2; shd[warp] = s; }
    __syncthreads();
    m1 = 0.0f; m2 = 0.0f; s = 0.0;
#pragma unroll
    for (int w = 0; w < kStreamWarps; ++w) { m1 = fmaxf(m1, shf[w]); m2 = fmaxf(m2, shf[kStreamWarps + w]); s += shd[w]; }
}

__device__ __forceinline__ int fixed_point(float v, float inv) {
    const int W = __float2int_rn(v * inv);
    return max(-IntPath<8>::QMAX, min(IntPath<8>::QMAX, W));
}

template <int CB>
__global__ void __launch_bounds__(kStreamThreads, 1) sgd_stream_kernel(const StreamArgs a) {
    constexpr int NG = IntPath<CB>::NG, NS = IntPath<CB>::NS, FPW = 32 / CB;
    constexpr int CW = kStreamBlock, S = kStreamStages;
    constexpr int QMAX = IntPath<CB>::QMAX;
    static_assert(NS == 4, "four digits");
    extern __shared__ __align__(128) unsigned char smem[];
    unsigned char* ring = smem;                                                  // [warps][S][stage]
    unsigned char* uni = smem + kStreamRingBytes;
    signed char* wds = reinterpret_cast<signed char*>(uni);                      // pass A: [NG * NS][part_spans * 64]
    signed char* rdig = reinterpret_cast<signed char*>(uni);                     // pass B: [2][NS][bpad + 16]
    int* gacc = reinterpret_cast<int*>(uni + (size_t)2 * NS * (a.bpad + 16));    // pass B: [bpc][NG][CW][NS], one pad word per 32
    float* own = reinterpret_cast<float*>(uni + a.union_bytes);                  // [3][bpc * CW * NG]: lo, step, x of the own features
    double2* rres = reinterpret_cast<double2*>(ring);                            // dots minus labels, between the passes
    __shared__ double shd[kStreamWarps];
    __shared__ float shf[2 * kStreamWarps];

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, gl = lane >> 2, tl = lane & 3;
    const int cta = blockIdx.x, G = gridDim.x;
    const int n = a.n;
    const int64_t rb = a.row_bytes, vb = a.vec_bytes;
    const int cb0 = min(a.spans, cta * a.bpc), cb1 = min(a.spans, cb0 + a.bpc);
    const int own_bytes = (cb1 - cb0) * CW, own_n = own_bytes * NG, own_cap = a.bpc * CW * NG;
    signed char* dstage = reinterpret_cast<signed char*>(ring);                  // update: [NG * NS][own_bytes]
    float* lo_o = own;
    float* st_o = own + own_cap;
    float* x_o = own + 2 * own_cap;
    const float smax = (float)((1 << a.bits) - 1);
    const uint32_t ring_w = smem_u32(ring) + (uint32_t)warp * S * kStreamStageBytes;
    const int pstride = a.part_spans * 64 + 64;            // bytes between the digit vectors in wds (64 more: no bank conflicts)
    const int rstride = a.bpad + 16;                       // bytes between the residual digit vectors

    // ---- set-up: every CTA scans the model once (identical arithmetic everywhere)
    float cmax = 0.0f, wm = 0.0f;
    double base = 0.0;
    for (int j = tid; j < n; j += kStreamThreads) {
        const float l = a.lo[j], s = a.step[j], xv = a.x[j];
        cmax = fmaxf(cmax, fabsf(s) * fmaxf(fabsf(l), fabsf(l + s * smax)));
        wm = fmaxf(wm, fabsf(s * xv));
        base += (double)l * (double)xv;
    }
    block_reduce_mms(cmax, wm, base, shf, shd);
    float bound = wm;                      // digit scale of the w that the coming step reads

    // own features into shared memory; digits of w for the first step, from the caller's model
    {
        const float inv = bound > 0.0f ? (float)QMAX / bound : 0.0f;
        for (int idx = tid; idx < own_n; idx += kStreamThreads) {
            const int bl = idx / NG, grp = idx - bl * NG;
            const int64_t byte = (int64_t)cb0 * CW + bl;
            const int64_t j = (byte >> 2) * FPW + (byte & 3) * NG + grp;
            const bool real = j < n;
            const float l = real ? a.lo[j] : 0.0f, s = real ? a.step[j] : 0.0f, xv = real ? a.x[j] : 0.0f;
            lo_o[idx] = l; st_o[idx] = s; x_o[idx] = xv;
            int d[NS];
            balanced_digits<NS>(real ? fixed_point(s * xv, inv) : 0, d);
#pragma unroll
            for (int k = 0; k < NS; ++k) a.wdig[((int64_t)grp * NS + k) * vb + byte] = (signed char)d[k];
        }
        __syncthreads();
        if (tid == 0) {
            __threadfence();
            for (int c = cb0; c < cb1; ++c) st_relaxed_u32(a.ready + c, 1u);
        }
    }

    for (int64_t t_rel = 0; t_rel < a.num_steps; ++t_rel) {
        const int64_t it = a.first_step + t_rel;
        const bool last = t_rel + 1 == a.num_steps;
        const int64_t bt_idx = a.order ? (int64_t)a.order[it] : it;
        const int64_t row0 = bt_idx * a.batch;
        const int bt = (int)min(a.batch, a.m - row0);
        const unsigned char* t1 = a.p1 + row0 * rb;
        const unsigned char* t2 = a.p2 + row0 * rb;
        long long* dots = a.dots + (size_t)(t_rel % 3) * 2 * a.bpad;
        stream_mark(a, t_rel, 0);
        if (warp == kStreamWarps - 1)          // the step's labels are read right after the barrier: have them in L2 by then
            for (int k = lane * 32; k < bt; k += 32 * 32) prefetch_l2(a.b + row0 + k);

        // ------------------------------------------------------------------ pass A: dots
        {
            const int nrb = (bt + 15) >> 4, nrg = (nrb + kStreamWarps - 1) / kStreamWarps;
            const int units = a.ca * nrg;
#pragma unroll 1
            for (int u = cta; u < units; u += G) {
                const int rg = u / a.ca, part = u - rg * a.ca;
                const int s0 = (int)((int64_t)part * a.spans / a.ca), s1 = (int)((int64_t)(part + 1) * a.spans / a.ca);
                const int rblk = rg * kStreamWarps + warp;
                const bool active = rblk < nrb;
                // A lane copies 16 bytes of rows g and g+8 of both planes per span.  Copies of rows past the
                // batch or bytes past the row are skipped: what the stage then holds meets zero digits
                // (pad features) or is never stored (pad rows).
                const bool ok_a = active && rblk * 16 + gl < bt, ok_h = active && rblk * 16 + gl + 8 < bt;
                const uint32_t off_a = (uint32_t)(rblk * 16 + gl) * (uint32_t)rb + 16 * tl, off_h = off_a + 8 * (uint32_t)rb;
                const int sp_end = min(s1, (int)((rb - 16 * tl + 63) / 64));      // spans whose 16 bytes of this lane lie in the row
                const uint32_t stage0 = ring_w + lane * 16;
                const uint64_t keep = l2_evict_normal_policy();
                auto issue = [&](int sp) {
                    if (sp < sp_end) {
                        const uint32_t dst = stage0 + (uint32_t)((sp - s0) & (S - 1)) * kStreamStageBytes;
                        const uint32_t o = (uint32_t)sp * 64;
                        cp_async16_if(ok_a, dst, t1 + (off_a + o), keep);
                        cp_async16_if(ok_a, dst + 1024, t2 + (off_a + o), keep);
                        cp_async16_if(ok_h, dst + 512, t1 + (off_h + o), keep);
                        cp_async16_if(ok_h, dst + 1536, t2 + (off_h + o), keep);
                    }
                    cp_async_commit();
                };
                // the codes do not depend on the model: start copying before looking at the flags
#pragma unroll
                for (int k = 0; k < S - 1; ++k) issue(s0 + k);
                {
                    const unsigned want = (unsigned)(t_rel + 1);
                    for (int f = s0 + tid; f < s1; f += kStreamThreads) {
                        long long spin = 0;
                        while (ld_acquire_u32(a.ready + f) < want) {
                            if (++spin > kBarrierSpinLimit) { set_status(a.status, ZIPML_ERR_TIMEOUT, 20); break; }
                            if ((spin & 63) == 63) {
                                if (*reinterpret_cast<volatile int*>(&a.status->code) != 0) break;
                                __nanosleep(100);
                            }
                        }
                    }
                    __syncthreads();
                    const int pb16 = (s1 - s0) * 4;                        // 16-byte pieces of one digit vector
                    for (int idx = tid; idx < NG * NS * pb16; idx += kStreamThreads) {
                        const int v = idx / pb16, q = idx - v * pb16;
                        *reinterpret_cast<uint4*>(wds + (size_t)v * pstride + q * 16) =
                            __ldcg(reinterpret_cast<const uint4*>(a.wdig + (int64_t)v * vb + (int64_t)s0 * 64 + q * 16));
                    }
                    __syncthreads();
                }
                // group g's codes stay where they are in the byte (one mask): its sums come out 2^(g CB) times too large
                int c1[NG][4], c2[NG][4];
#pragma unroll
                for (int g = 0; g < NG; ++g)
#pragma unroll
                    for (int e = 0; e < 4; ++e) { c1[g][e] = 0; c2[g][e] = 0; }
                if (active) {
                    const unsigned char* stage_r = ring + (size_t)warp * S * kStreamStageBytes + lane * 16;
                    const signed char* dig_r = wds + (size_t)gl * pstride + 16 * tl;       // lanes with gl < NS read digit gl
#pragma unroll 1
                    for (int sp = s0; sp < s1; ++sp) {
                        issue(sp + S - 1);
                        cp_async_wait<S - 1>();
                        const unsigned char* st = stage_r + (size_t)((sp - s0) & (S - 1)) * kStreamStageBytes;
                        const uint4 ua = *reinterpret_cast<const uint4*>(st);
                        const uint4 uh = *reinterpret_cast<const uint4*>(st + 512);
                        const uint4 va = *reinterpret_cast<const uint4*>(st + 1024);
                        const uint4 vh = *reinterpret_cast<const uint4*>(st + 1536);
#pragma unroll
                        for (int g = 0; g < NG; ++g) {
                            constexpr uint32_t kLow = CB == 8 ? 0xFFFFFFFFu : CB == 4 ? 0x0F0F0F0Fu : 0x03030303u;
                            const uint32_t mk = kLow << (g * CB);
                            uint4 bd = make_uint4(0u, 0u, 0u, 0u);
                            if (gl < NS) bd = *reinterpret_cast<const uint4*>(dig_r + (size_t)g * NS * pstride + (sp - s0) * 64);
                            mma_u8s8(c1[g], ua.x & mk, uh.x & mk, ua.y & mk, uh.y & mk, bd.x, bd.y);
                            mma_u8s8(c1[g], ua.z & mk, uh.z & mk, ua.w & mk, uh.w & mk, bd.z, bd.w);
                            mma_u8s8(c2[g], va.x & mk, vh.x & mk, va.y & mk, vh.y & mk, bd.x, bd.y);
                            mma_u8s8(c2[g], va.z & mk, vh.z & mk, va.w & mk, vh.w & mk, bd.z, bd.w);
                        }
                    }
                }
                cp_async_wait<0>();
                // lane t < 2 holds digits 2t, 2t+1 of rows g (c[0], c[1]) and g+8 (c[2], c[3])
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    long long q1 = 0, q2 = 0;
#pragma unroll
                    for (int g = 0; g < NG; ++g) {         // exact: the sums are multiples of 2^(g CB)
                        q1 += (long long)(c1[g][2 * e] >> (g * CB)) + 128ll * (long long)(c1[g][2 * e + 1] >> (g * CB));
                        q2 += (long long)(c2[g][2 * e] >> (g * CB)) + 128ll * (long long)(c2[g][2 * e + 1] >> (g * CB));
                    }
                    const long long v1 = q1 + 16384ll * __shfl_down_sync(0xffffffffu, q1, 1);
                    const long long v2 = q2 + 16384ll * __shfl_down_sync(0xffffffffu, q2, 1);
                    const int k = rblk * 16 + gl + 8 * e;
                    if (active && tl == 0 && k < bt) {
                        // (a reduction that returns nothing: the warp does not wait for an old value it never reads)
                        red_add_s64(dots + k, v1);
                        red_add_s64(dots + a.bpad + k, v2);
                    }
                }
                __syncthreads();           // the next unit overwrites the staged digits
            }
        }
        stream_mark(a, t_rel, 1);
        if (!grid_barrier(a.barrier, (unsigned)((t_rel + 1) * G), a.status, 21)) return;
        stream_mark(a, t_rel, 2);

        // HBM is idle from here to the next step's first pass: part of the next tile can travel to L2 now
        // (the whole of it would push this step's tile out before the second pass has read it)
        if (a.l2_prefetch && !last && warp == kStreamWarps - 1 && lane < 2) {
            const int64_t itn = it + 1;
            const int64_t rown = (a.order ? (int64_t)a.order[itn] : itn) * a.batch;
            const int64_t bytes = min(a.batch, a.m - rown) * rb;          // a multiple of 16
            const int64_t per = ((bytes / 16 + G - 1) / G) * 16;
            const int64_t lo_b = min(bytes, per * cta), hi_b = min(bytes, lo_b + (per * a.l2_prefetch / 128) * 16);
            const unsigned char* srcn = (lane == 0 ? a.p1 : a.p2) + rown * rb;
            for (int64_t o = lo_b; o < hi_b; o += 32768) l2_prefetch_bulk(srcn + o, (uint32_t)min((int64_t)32768, hi_b - o));
        }

        // ------------------------------------------------------------------ residuals (every CTA, all rows)
        // clear the dots two steps ahead (its last readers passed the previous barrier)
        {
            long long* z = a.dots + (size_t)((t_rel + 2) % 3) * 2 * a.bpad;
            for (int i = cta * kStreamThreads + tid; i < 2 * a.bpad; i += G * kStreamThreads) z[i] = 0;
        }
        const double delta_w = (double)bound / (double)QMAX;
        float rmax = 0.0f, pm = 0.0f;
        double pb = 0.0;
        if (t_rel > 0) {                   // the owners' parts of max |w| and lo^T x of the model this step saw
            const size_t par = (size_t)(t_rel & 1) * G;
            for (int i = tid; i < G; i += kStreamThreads) { pm = fmaxf(pm, __ldcg(a.wmax_part + par + i)); pb += __ldcg(a.base_part + par + i); }
        }
        for (int k0 = tid; k0 < bt; k0 += 4 * kStreamThreads) {           // four rows' loads in flight together
            long long v1[4], v2[4];
            float bk[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const int k = k0 + q * kStreamThreads;
                if (k < bt) { v1[q] = __ldcg(dots + k); v2[q] = __ldcg(dots + a.bpad + k); bk[q] = a.b[row0 + k]; }
            }
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const int k = k0 + q * kStreamThreads;
                if (k < bt) rres[k] = make_double2((double)v1[q] * delta_w - (double)bk[q], (double)v2[q] * delta_w - (double)bk[q]);
            }
        }
        block_reduce_mms(rmax, pm, pb, shf, shd);          // rmax is not known yet: this round carries pm and pb
        if (t_rel > 0) { wm = pm; base = pb; }
        stream_mark(a, t_rel, 6);
        // r = delta_w V + lo^T x - b in double, rounded to fp32 once; the same on every CTA
        for (int k = tid; k < bt; k += kStreamThreads) {
            const double2 d = rres[k];
            rmax = fmaxf(rmax, fmaxf(fabsf((float)(d.x + base)), fabsf((float)(d.y + base))));
        }
        {
            float unused = 0.0f;
            double none = 0.0;
            block_reduce_mms(rmax, unused, none, shf, shd);
        }
        stream_mark(a, t_rel, 7);
        const float inv_r = rmax > 0.0f ? (float)QMAX / rmax : 0.0f;
        const double delta_r = (double)rmax / (double)QMAX;
        double rsum = 0.0;                 // sum of all fixed-point residuals (exact in double)
        // a thread takes rows t, t+4, t+8, t+12 of a group of 16: their digits are one 32-bit word of pass B's operand
        for (int q4 = tid; q4 < a.bpad / 4; q4 += kStreamThreads) {
            const int kb = (q4 >> 2) * 16 + (q4 & 3);
            uint32_t w1[NS] = {0u, 0u, 0u, 0u}, w2[NS] = {0u, 0u, 0u, 0u};
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int k = kb + 4 * i;
                int R1 = 0, R2 = 0;
                if (k < bt) {
                    const double2 d = rres[k];
                    R1 = fixed_point((float)(d.x + base), inv_r);
                    R2 = fixed_point((float)(d.y + base), inv_r);
                }
                rsum += (double)R1 + (double)R2;
                int d1[NS], d2[NS];
                balanced_digits<NS>(R1, d1);
                balanced_digits<NS>(R2, d2);
#pragma unroll
                for (int q = 0; q < NS; ++q) { w1[q] |= (uint32_t)(d1[q] & 255) << (8 * i); w2[q] |= (uint32_t)(d2[q] & 255) << (8 * i); }
            }
#pragma unroll
            for (int q = 0; q < NS; ++q) {
                *reinterpret_cast<uint32_t*>(rdig + (size_t)q * rstride + 4 * q4) = w2[q];             // plane 1 meets r2
                *reinterpret_cast<uint32_t*>(rdig + (size_t)(NS + q) * rstride + 4 * q4) = w1[q];      // plane 2 meets r1
            }
        }
        for (int i = tid; i < (cb1 - cb0) * NG * CW * NS * 33 / 32; i += kStreamThreads) gacc[i] = 0;
        {
            float u1 = 0.0f, u2 = 0.0f;
            block_reduce_mms(u1, u2, rsum, shf, shd);      // its barriers publish rdig and the cleared sums
        }
        // scale of the next model's digits: a bound that writers and readers both know now
        // (the regularisers only pull towards zero, except the least-squares SVM term with lr c > 2)
        const float grow = a.reg == ZIPML_REG_LSSVM ? fmaxf(1.0f, fabsf(1.0f - a.reg_cst)) : 1.0f;
        const float bound_next = (wm * grow + fabsf(a.lr) * cmax * rmax) * 1.0001f;
        stream_mark(a, t_rel, 3);

        // ------------------------------------------------------------------ pass B: gradient of the own blocks
        {
            const int nrb = (bt + 31) >> 5;
            const int mine = nrb > warp ? (nrb - 1 - warp) / kStreamWarps + 1 : 0;     // 32-row blocks of this warp
            const int per_c = 2 * mine, total = (cb1 - cb0) * per_c;
            // Iteration i: column block i / per_c, then (row block, plane); newest rows first (likeliest in L2).
            // A stage holds 32 rows x 64 bytes, row-major; a lane copies 16 bytes of rows l/4, l/4+8, l/4+16,
            // l/4+24.  Copies of rows past the batch or of bytes past the row are skipped: the former meet
            // zero residual digits, the latter end in sums of pad features that nobody reads.  Lane 4g+t
            // then takes the 8 bytes of column piece g from rows t, t+4, t+8, t+12 (and 16 more): for one
            // load the four t's read four consecutive rows, 256 contiguous bytes, no bank conflict; the
            // residual digits are stored in the matching row order.
            const uint32_t rb32 = (uint32_t)rb;
            const uint32_t stage0 = ring_w + lane * 16;
            const uint64_t dead = l2_evict_first_policy();    // the tile is not read again: its lines may leave L2 first
            const uint64_t keep = l2_evict_normal_policy();
            int i_ci = 0, i_rem = 0;                       // issue side: column block and position within it
            auto issue = [&]() {
                if (i_ci < cb1 - cb0) {
                    const int r0 = (nrb - 1 - warp - kStreamWarps * (i_rem >> 1)) * 32 + gl;
                    const uint32_t coff = (uint32_t)(cb0 + i_ci) * CW + tl * 16;
                    if (coff < rb32) {
                        const unsigned char* tp = ((i_rem & 1) ? t2 : t1) + coff;
                        const uint32_t dst = stage0 + (uint32_t)((i_ci * per_c + i_rem) & (S - 1)) * kStreamStageBytes;
                        const uint32_t o = (uint32_t)r0 * rb32;
                        // A 128-byte line holds two column blocks.  Once this CTA has read both, nobody reads the
                        // line again this step: only then may it leave L2 ahead of the rest.
                        const uint64_t pol = (i_ci > 0 && ((cb0 + i_ci) & 1)) ? dead : keep;
#pragma unroll
                        for (int k = 0; k < 4; ++k) cp_async16_if(r0 + 8 * k < bt, dst + k * 512, tp + (o + 8 * k * rb32), pol);
                    }
                    if (++i_rem == per_c) { i_rem = 0; ++i_ci; }
                }
                cp_async_commit();
            };
            int acc[NG][2][2][4];
#pragma unroll
            for (int g = 0; g < NG; ++g)
#pragma unroll
                for (int w = 0; w < 2; ++w)
#pragma unroll
                    for (int u = 0; u < 2; ++u)
#pragma unroll
                        for (int e = 0; e < 4; ++e) acc[g][w][u][e] = 0;
            if (total > 0) {
#pragma unroll
                for (int k = 0; k < S - 1; ++k) issue();
            }
            const unsigned char* stage_r = ring + (size_t)warp * S * kStreamStageBytes + tl * 64 + gl * 8;
            const signed char* rd_lane = rdig + (size_t)(gl & (NS - 1)) * rstride + 4 * tl;
            int ci = 0, rem = 0;
#pragma unroll 1
            for (int i = 0; i < total; ++i) {
                cp_async_wait<S - 2>();    // this lane's copies of stage i have landed ...
                __syncwarp();              // ... and everyone's; and everyone is done reading stage i - 1,
                issue();                   // which this refills
                const int r0 = (nrb - 1 - warp - kStreamWarps * (rem >> 1)) * 32;
                const unsigned char* st = stage_r + (size_t)(i & (S - 1)) * kStreamStageBytes;
                uint2 lo4[4], hi4[4];
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    lo4[k] = *reinterpret_cast<const uint2*>(st + k * 256);            // row t + 4k
                    hi4[k] = *reinterpret_cast<const uint2*>(st + 1024 + k * 256);     // row 16 + t + 4k
                }
                uint32_t b0 = 0u, b1 = 0u;
                if (gl < NS) {
                    const signed char* rd = rd_lane + (size_t)((rem & 1) * NS) * rstride + r0;
                    b0 = *reinterpret_cast<const uint32_t*>(rd);
                    b1 = *reinterpret_cast<const uint32_t*>(rd + 16);
                }
#pragma unroll
                for (int w = 0; w < 2; ++w) {
                    uint32_t ta[4], th[4];
                    if (w == 0) { transpose4x4(lo4[0].x, lo4[1].x, lo4[2].x, lo4[3].x, ta); transpose4x4(hi4[0].x, hi4[1].x, hi4[2].x, hi4[3].x, th); }
                    else { transpose4x4(lo4[0].y, lo4[1].y, lo4[2].y, lo4[3].y, ta); transpose4x4(hi4[0].y, hi4[1].y, hi4[2].y, hi4[3].y, th); }
#pragma unroll
                    for (int g = 0; g < NG; ++g) {
                        // Both groups of a byte meet the same residual digits, so the sums may nest: accumulator g
                        // takes the byte with the groups below g cleared (g = 0: the byte as it is, no mask at
                        // all), i.e. sum_{h >= g} 2^(h CB) code_h; group g is the difference of two neighbours.
                        const uint32_t mk = 0x01010101u * (uint32_t)((0xFFu << (g * CB)) & 0xFFu);
#pragma unroll
                        for (int u = 0; u < 2; ++u)
                            mma_u8s8(acc[g][w][u], ta[2 * u] & mk, ta[2 * u + 1] & mk, th[2 * u] & mk, th[2 * u + 1] & mk, b0, b1);
                    }
                }
                if (++rem == per_c) {
                    // lane t < 2: acc[g][w][u][0..1] = digits 2t, 2t+1 of byte 4w+2u of the lane's bytes, [2..3] of byte 4w+2u+1
                    // entry e lives at e + e / 32: the eight lane groups, 32 entries apart, hit eight banks
                    const int e0 = ci * NG * CW * NS;
#pragma unroll
                    for (int g = 0; g < NG; ++g)
#pragma unroll
                        for (int w = 0; w < 2; ++w)
#pragma unroll
                            for (int u = 0; u < 2; ++u) {
                                if (tl < 2) {
                                    const int e = e0 + (g * CW + gl * 8 + 4 * w + 2 * u) * NS + 2 * tl;
                                    int* p = gacc + e + (e >> 5);
                                    // (exact: the difference is 2^(g CB) times the group's sum)
#pragma unroll
                                    for (int q = 0; q < 4; ++q) {
                                        const int above = g + 1 < NG ? acc[g + 1 < NG ? g + 1 : g][w][u][q] : 0;
                                        atomicAdd(p + (q >> 1) * NS + (q & 1), (acc[g][w][u][q] - above) >> (g * CB));
                                    }
                                }
                            }
#pragma unroll
                    for (int g = 0; g < NG; ++g)
#pragma unroll
                        for (int w = 0; w < 2; ++w)
#pragma unroll
                            for (int u = 0; u < 2; ++u)
#pragma unroll
                                for (int e = 0; e < 4; ++e) acc[g][w][u][e] = 0;
                    rem = 0;
                    ++ci;
                }
            }
            cp_async_wait<0>();
        }
        __syncthreads();
        stream_mark(a, t_rel, 4);

        // ------------------------------------------------------------------ update of the own features, digits of the next w
        {
            const double scale = 1.0 / (2.0 * (double)bt);
            const double lo_term = delta_r * rsum;
            const float inv = bound_next > 0.0f ? (float)QMAX / bound_next : 0.0f;
            float pmax = 0.0f, unused = 0.0f;
            double pbase = 0.0;
            for (int idx = tid; idx < own_n; idx += kStreamThreads) {
                const int bl = idx / NG, grp = idx - bl * NG;
                const int64_t byte = (int64_t)cb0 * CW + bl;
                const int64_t j = (byte >> 2) * FPW + (byte & 3) * NG + grp;
                int W = 0;
                if (j < n) {
                    const int cl = bl / CW, bb = bl - cl * CW;
                    const int e = ((cl * NG + grp) * CW + bb) * NS;
                    const int* src = gacc + e + (e >> 5);
                    const int sv[NS] = {src[0], src[1], src[2], src[3]};
                    const long long Sj = combine_digits<NS>(sv);
                    const float l = lo_o[idx], st = st_o[idx];
                    const float g = (float)(((double)l * lo_term + (double)st * (delta_r * (double)Sj)) * scale);
                    if (last && a.grad_out) { a.grad_out[j] = g; a.grad_out[n + j] = g; }
                    const float xn = regularise(fmaf(-a.lr, g, x_o[idx]), x_o[idx], a.reg, a.reg_cst);
                    x_o[idx] = xn;
                    a.x[j] = xn;
                    const float w = st * xn;
                    pmax = fmaxf(pmax, fabsf(w));
                    pbase += (double)l * (double)xn;
                    W = fixed_point(w, inv);
                }
                if (!last) {               // digits meet in shared memory (the ring is idle) and leave as 16-byte stores
                    int d[NS];
                    balanced_digits<NS>(W, d);
#pragma unroll
                    for (int k = 0; k < NS; ++k) dstage[(grp * NS + k) * own_bytes + bl] = (signed char)d[k];
                }
            }
            if (last) break;
            block_reduce_mms(pmax, unused, pbase, shf, shd);
            {
                const int p16 = own_bytes / 16;
                for (int idx = tid; idx < NG * NS * p16; idx += kStreamThreads) {
                    const int v = idx / p16, q = idx - v * p16;
                    *reinterpret_cast<uint4*>(a.wdig + (int64_t)v * vb + (int64_t)cb0 * CW + q * 16) =
                        *reinterpret_cast<const uint4*>(dstage + v * own_bytes + q * 16);
                }
            }
            __syncthreads();               // every digit store of the CTA is issued; the ring is free again
            if (tid == 0) {
                const size_t par = (size_t)((t_rel + 1) & 1) * G;
                a.wmax_part[par + cta] = pmax;
                a.base_part[par + cta] = pbase;
                __threadfence();
                for (int c = cb0; c < cb1; ++c) st_relaxed_u32(a.ready + c, (unsigned)(t_rel + 2));
            }
            bound = bound_next;
        }
        stream_mark(a, t_rel, 5);
    }
}

// ---------------------------------------------------------------------------------------------
// Host side
// ---------------------------------------------------------------------------------------------
static const void* stream_kernel_ptr(int cb) {
    if (cb == 2) return reinterpret_cast<const void*>(&sgd_stream_kernel<2>);
    if (cb == 4) return reinterpret_cast<const void*>(&sgd_stream_kernel<4>);
    return reinterpret_cast<const void*>(&sgd_stream_kernel<8>);
}

int launch_sgd_stream(zipml_ctx* ctx, const zipml_dataset* d, const float* b, float* x, const zipml_sgd_params* p,
                      int64_t first_step, int64_t num_steps, float* grad_out, bool only_if_profitable) {
    if (!ctx->cooperative) return ZIPML_ERR_WORKSPACE;
    if (d->level_mode != ZIPML_LEVELS_UNIFORM || p->model_bits != 0 || p->grad_bits != 0) return ZIPML_ERR_WORKSPACE;
    if (d->n > (1 << 30) / 8) return ZIPML_ERR_WORKSPACE;
    const int cb = container_bits(d->bits);
    const int ng = 8 / cb, cw = kStreamBlock;
    // (model_out: with an fp32 model the last step's gradient saw the model as it stood before that step; this
    // engine keeps no copy of it, so the request is declined like the quantized model itself)
    if (p->model_out) return ZIPML_ERR_WORKSPACE;
    const int64_t T = (d->m + p->batch - 1) / p->batch;
    const int64_t B = p->batch < d->m ? p->batch : d->m;
    if (B > kStreamMaxBatch) return ZIPML_ERR_WORKSPACE;
    const int bpad = (int)((B + 31) / 32 * 32);
    const int64_t rb = d->row_bytes;
    const int64_t spans = (rb + 63) / 64;
    int G = ctx->sm_count;
    if (p->grid_row_parts > 0 && p->grid_row_parts < G) G = p->grid_row_parts;      // tuning: fewer CTAs
    int64_t bpc = (spans + G - 1) / G;
    if (bpc > kStreamMaxOwn) {             // the hint does not fit: plan for the whole device
        G = ctx->sm_count;
        bpc = (spans + G - 1) / G;
    }
    if (bpc > kStreamMaxOwn) return ZIPML_ERR_WORKSPACE;
    G = (int)((spans + bpc - 1) / bpc);
    // worth it only where the rows are wide enough to occupy the device (measured against the ring engine on
    // 16 KB rows: ahead at every batch from 128 to 8192 rows, 10.7 vs 25.8 us per step at 128)
    if (only_if_profitable && (G < ctx->sm_count / 2 || B < 32)) return ZIPML_ERR_WORKSPACE;
    // pass A: 256-row groups x column parts, about one unit per CTA
    const int64_t nrg = ((B + 15) / 16 + kStreamWarps - 1) / kStreamWarps;
    int64_t ca = G / nrg;
    if (ca < (spans + kStreamMaxPartSpans - 1) / kStreamMaxPartSpans) ca = (spans + kStreamMaxPartSpans - 1) / kStreamMaxPartSpans;
    if (ca < 1) ca = 1;
    if (ca > spans) ca = spans;
    const int part_spans = (int)((spans + ca - 1) / ca);
    const int64_t vec_bytes = spans * 64;

    const size_t pass_a = (size_t)ng * 4 * (part_spans * 64 + 64);
    const size_t pass_b = (size_t)2 * 4 * (bpad + 16) + sizeof(int) * (size_t)bpc * ng * cw * 4 * 33 / 32;
    const size_t uni = ((pass_a > pass_b ? pass_a : pass_b) + 127) / 128 * 128;
    const size_t smem = (size_t)kStreamRingBytes + uni + sizeof(float) * 3 * (size_t)bpc * cw * ng;
    if (smem > (size_t)ctx->smem_optin) return ZIPML_ERR_WORKSPACE;
    const void* kernel = stream_kernel_ptr(cb);
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return cuda_status(e);
    int per_sm = 0;
    e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, kStreamThreads, smem);
    if (e != cudaSuccess) return cuda_status(e);
    if (per_sm < 1 || G > per_sm * ctx->sm_count) return ZIPML_ERR_WORKSPACE;

    size_t off = 0;
    auto piece = [&](size_t bytes) { const size_t o = off; off += carve_size(bytes); return o; };
    // zeroed before a launch: barrier counter, flags, dots
    const size_t o_bar = piece(sizeof(unsigned) * 64);
    const size_t o_ready = piece(sizeof(unsigned) * (size_t)spans);
    const size_t o_dots = piece(sizeof(long long) * 3 * 2 * (size_t)bpad);
    const size_t zero_bytes = off;
    const size_t o_wdig = piece((size_t)ng * 4 * vec_bytes);
    const size_t o_wmax = piece(sizeof(float) * 2 * (size_t)G);
    const size_t o_base = piece(sizeof(double) * 2 * (size_t)G);
    const size_t o_ord = piece(sizeof(int32_t) * (size_t)(p->batch_order ? T : 0));
    int rc = ws_reserve(ctx, off);
    if (rc != ZIPML_OK) return rc;

    StreamArgs a;
    memset(&a, 0, sizeof(a));
    a.p1 = d->plane1; a.p2 = d->plane2; a.row_bytes = rb; a.m = d->m; a.n = (int)d->n; a.bits = d->bits;
    a.lo = d->feat_lo; a.step = d->feat_step; a.b = b; a.x = x; a.grad_out = grad_out;
    a.batch = B; a.lr = p->lr; a.reg = p->reg; a.reg_cst = reg_constant(p);
    a.ca = (int)ca; a.spans = (int)spans; a.part_spans = part_spans; a.bpc = (int)bpc; a.bpad = bpad;
    a.union_bytes = (int)uni; a.vec_bytes = vec_bytes;
    // The whole next tile where two tiles fit L2 with room to spare, a quarter of it where one and a half do
    // (measured on 64 MB tiles in a 126 MB L2: 2/8 gains 3 %, 8/8 loses 6 %); zipml_sgd_params.stream_prefetch overrides
    int l2_bytes = 0;
    cudaDeviceGetAttribute(&l2_bytes, cudaDevAttrL2CacheSize, ctx->device);
    const int64_t step_bytes = 2 * B * rb;
    a.l2_prefetch = 9 * step_bytes <= 4 * (int64_t)l2_bytes ? 8 : 3 * step_bytes <= 2 * (int64_t)l2_bytes ? 2 : 0;
    if (p->stream_prefetch >= 1 && p->stream_prefetch <= 9) a.l2_prefetch = p->stream_prefetch - 1;    // the caller's choice
    a.barrier = reinterpret_cast<unsigned*>(ctx->ws + o_bar);
    a.ready = reinterpret_cast<unsigned*>(ctx->ws + o_ready);
    a.dots = reinterpret_cast<long long*>(ctx->ws + o_dots);
    a.wdig = reinterpret_cast<signed char*>(ctx->ws + o_wdig);
    a.wmax_part = reinterpret_cast<float*>(ctx->ws + o_wmax);
    a.base_part = reinterpret_cast<double*>(ctx->ws + o_base);
    a.status = ctx->d_status;
    a.trace = reinterpret_cast<unsigned long long*>(p->trace);
    a.trace_steps = p->trace ? p->trace_steps : 0;
    if (p->batch_order) {
        int32_t* dev_order = reinterpret_cast<int32_t*>(ctx->ws + o_ord);
        e = cudaMemcpyAsync(dev_order, p->batch_order, sizeof(int32_t) * (size_t)T, cudaMemcpyHostToDevice, ctx->stream);
        if (e != cudaSuccess) return cuda_status(e);
        a.order = dev_order;
    }
    // the barrier counter and the flag versions are 32-bit step counts
    const int64_t max_steps = (int64_t)(0x7fffffff / G) - 2;
    for (int64_t s0 = first_step; s0 < first_step + num_steps; s0 += max_steps) {
        e = cudaMemsetAsync(ctx->ws, 0, zero_bytes, ctx->stream);
        if (e != cudaSuccess) return cuda_status(e);
        StreamArgs chunk = a;
        chunk.first_step = s0;
        chunk.num_steps = (first_step + num_steps - s0 < max_steps) ? first_step + num_steps - s0 : max_steps;
        if (s0 + chunk.num_steps < first_step + num_steps) chunk.grad_out = nullptr;
        if (s0 > first_step) { chunk.trace = nullptr; chunk.trace_steps = 0; }
        void* params[] = {&chunk};
        e = cudaLaunchCooperativeKernel(kernel, dim3((unsigned)G), dim3(kStreamThreads), params, smem, ctx->stream);
        if (e != cudaSuccess) return cuda_status(e);
        ctx->launches += 1;
    }
    ctx->last_engine = ZIPML_ENGINE_STREAM;
    return ZIPML_OK;
}

}  // namespace zipml
