// Cluster engine of zipml_sgd_epoch: one persistent launch of a single thread-block cluster, built
// for steps whose code tile is small (Supplement "Double Sampling", footnote form; "End-to-end
// Quantization").
//
// A small step is bound by the chain  dots -> residuals -> partial gradients -> sum over the CTAs ->
// update -> new model at every CTA.  Measured on B200, a value handed from one SM to another through
// L2 (store, poll) takes about 1000 cycles; a bulk copy from shared memory into the shared memory
// of another CTA of the cluster that completes a transaction count on the receiver's mbarrier
// takes about 320 cycles for 256 bytes (st.async: 230), and the receiver waits on local shared
// memory.  So here the minibatch is cut into nb <= 16 row parts, one CTA each, all in one cluster:
//   * phase A: a warp takes rows, its lanes the words of a row; fp32 FMA on unpacked codes against
//     w = step * x~ (or a level-times-model table), the two dots of a row summed across the warp
//     in double; residuals stay in the CTA;
//   * phase B: a thread takes a word column, adds code * residual over the CTA's rows; the CTA's
//     part of the gradient (for uniform grids lo * sum(r) + step * sum(code * r)) lands in
//     shared memory;
//   * reduce-scatter: CTA o owns features [o * sub, (o + 1) * sub); every CTA bulk-copies slice o of
//     its part into owner o's receive buffer (one copy instruction per owner); the owner waits on
//     its mbarrier, adds the nb parts in a fixed order, applies the optional gradient quantizer and
//     the update to its master copy and writes what the next step sees (Q3 of it when the model
//     quantizer is on) into a staging buffer;
//   * all-gather: the owner bulk-copies the staging buffer to every CTA's model vector; every CTA
//     waits on its mbarrier and builds w.  The first model takes the same route: the loop starts
//     with a publish-only round.
//   * the code tiles do not depend on the model: bulk copies from global memory run several steps
//     ahead in a ring of shared-memory slots (one contiguous copy per plane and step).
// Buffer reuse: a CTA overwrites its part (and sends the next one) only after it has received the
// model of the step from every owner, and an owner publishes only after all parts of the step have
// landed in its buffer; an owner overwrites its staging buffer only after the parts of the next
// step have arrived, which their senders issued after the model had landed everywhere.  So single
// buffers suffice and no copy can still be reading a buffer that is being rewritten.
// Every wait is a bounded wait on a local mbarrier: when one gives up the CTA records
// ZIPML_ERR_TIMEOUT, skips its later waits and still issues every copy, so the launch ends; all CTAs
// meet at a cluster barrier before they exit (nobody's shared memory goes away under a copy).
#include <string.h>

#include "sgd_common.cuh"

namespace zipml {

constexpr int kCluThreads = 512;
constexpr int kCluWarps = kCluThreads / 32;
constexpr int kCluMaxSlots = 8;
constexpr int kCluMaxCtas = 16;                   // one bulk copy per warp and destination: at most kCluWarps CTAs
static_assert(kCluMaxCtas <= kCluWarps, "a warp per destination CTA");

struct ClusterArgs {
    const uint32_t* p1;
    const uint32_t* p2;
    const float* lo;
    const float* step;
    const float* levels;
    const float* b;
    float* x;
    float* grad_out;             // null or 2n
    const int32_t* order;        // device copy of the batch order, or null
    unsigned long long* trace;
    DeviceStatus* status;
    int64_t m, batch, first_step, num_steps;
    uint64_t seed;
    uint32_t epoch;
    float lr;
    int n, bits, row_words, words;   // words = ceil(n / codes per word) <= row_words
    int model_bits, grad_bits;
    int nb, rc, slots;
    int sub;                     // a CTA owns `sub` consecutive features (a multiple of 4)
    int p_shift;                 // 2^p_shift lanes share the sum of one owned feature
    int trace_steps;
};

struct ClusterShared {
    double red[kCluWarps];       // block sums
    double wbase[kCluWarps];     // per-warp parts of lo^T x~
    double ssum[kCluWarps];      // per-warp sums of the residuals
    double nrm_g[kCluMaxCtas];   // partial squared gradient norms, one per CTA
    double nrm_x[kCluMaxCtas];   // partial squared model norms
    unsigned long long full[kCluMaxSlots];
    unsigned long long rs_bar, ag_bar, gn_bar, xn_bar;
    int abort_flag;
    int pad;
};

__device__ __forceinline__ uint32_t cluster_addr(const void* local_smem, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_u32(local_smem)), "r"(rank));
    return r;
}
// shared::cta -> shared::cluster bulk copy; completes `bytes` on the mbarrier at the destination CTA.
__device__ __forceinline__ void bulk_copy_s2c(uint32_t dst_cluster, const void* src_smem, uint32_t bytes, uint32_t bar_cluster) {
    asm volatile("cp.async.bulk.shared::cluster.shared::cta.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst_cluster), "r"(smem_u32(src_smem)), "r"(bytes), "r"(bar_cluster) : "memory");
}
__device__ __forceinline__ void store_async_f64(uint32_t dst_cluster, double v, uint32_t bar_cluster) {
    asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.b64 [%0], %1, [%2];"
                 ::"r"(dst_cluster), "l"(__double_as_longlong(v)), "r"(bar_cluster) : "memory");
}
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}

// Bounded wait on a local mbarrier phase; after the first failure of this CTA every wait is skipped.
__device__ __forceinline__ void clu_wait(unsigned long long* bar, uint32_t parity, ClusterShared* sh, DeviceStatus* status, int where) {
    if (*reinterpret_cast<volatile int*>(&sh->abort_flag)) return;
#pragma unroll 1
    for (long long spin = 0; spin < kCopySpinLimit; ++spin)
        if (mbar_try_wait(reinterpret_cast<uint64_t*>(bar), parity)) return;
    sh->abort_flag = 1;
    set_status(status, ZIPML_ERR_TIMEOUT, where);
}

// l2 norm of a vector whose squared entries are spread over the threads of all CTAs: block sum, one
// double per CTA stored into every CTA's table, added there in CTA order.
__device__ __noinline__ float clu_norm(double v, double* table, unsigned long long* bar, uint32_t parity, int nb,
                                       ClusterShared* sh, DeviceStatus* status, int where) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    v = warp_sum(v);
    __syncthreads();
    if (lane == 0) sh->red[warp] = v;
    if (threadIdx.x == 0) mbar_arrive_expect_tx(reinterpret_cast<uint64_t*>(bar), 8u * (uint32_t)nb);
    __syncthreads();
    if ((int)threadIdx.x < nb) {
        double t = 0.0;
        for (int w = 0; w < kCluWarps; ++w) t += sh->red[w];
        store_async_f64(cluster_addr(table + blockIdx.x, threadIdx.x), t, cluster_addr(bar, threadIdx.x));
    }
    clu_wait(bar, parity, sh, status, where);
    double t = 0.0;
    for (int c = 0; c < nb; ++c) t += table[c];
    return (float)sqrt(t);
}

__device__ __noinline__ float clu_quant(float v, float M, int sm, uint64_t seed, uint32_t epoch, uint32_t step,
                                        uint32_t stream, uint32_t coord) {
    VecQuant q{M, sm, seed, epoch, step, stream};
    return q.apply(v, coord);
}

__device__ __forceinline__ void clu_mark(const ClusterArgs& a, int64_t it, int id) {
    if (a.trace && blockIdx.x == 0 && threadIdx.x == 0 && it >= a.first_step && it - a.first_step < a.trace_steps) {
        unsigned long long t;
        asm volatile("mov.u64 %0, %clock64;" : "=l"(t));
        a.trace[(it - a.first_step) * 8 + id] = t;
    }
}

// Shared memory after ClusterShared; Fp = row_words * FPW feature slots of a row (padding included),
// Fs = nb * sub >= n features as the owners cut them:
//   uniform: wv[Fp]  w = step * x~, [slot i][word q];  los[Fp], steps[Fp]  lo and step by feature
//   table:   tab[L*Fp] level * x~ and lev[L*Fp] levels, both [code][slot i][word q]
//   xs[Fs]           the model this step sees (all-gather destination)
//   gpart[Fs]        this CTA's part of the gradient (reduce-scatter source)
//   gbuf[nb][sub]    the nb parts of the owned features (reduce-scatter destination)
//   xpub[sub], xown[sub], gsub[sub]   staging of the published slice, master model, gradient of the step
//   res[2*rc]        residuals (r1, r2) per row;   bsm[rc]  labels of the step's rows
//   gred[256*FPW]    cross-group sums of phase B (parts narrower than the CTA)
//   ring[slots][2][rc][row_words]  code tiles
template <int CB, bool TABLE>
__global__ void __launch_bounds__(kCluThreads, 1) sgd_cluster_kernel(const ClusterArgs a) {
    constexpr int FPW = 32 / CB;
    constexpr int LOGF = (CB == 8) ? 2 : (CB == 4) ? 3 : 4;
    extern __shared__ __align__(16) unsigned char s_raw[];
    ClusterShared* sh = reinterpret_cast<ClusterShared*>(s_raw);
    const int rw = a.row_words, nw = a.words, n = a.n;
    const int Fp = rw * FPW;
    const int L = 1 << a.bits;
    const int sub = a.sub;
    const int nb = a.nb;
    const int Fs = nb * sub;
    float* tab = reinterpret_cast<float*>(s_raw + ((sizeof(ClusterShared) + 15) & ~(size_t)15));
    float* wv = tab;                                     // uniform
    float* los = tab + Fp;
    float* steps = los + Fp;
    float* lev = tab + (size_t)L * Fp;                   // table
    float* xs = tab + (TABLE ? 2 * (size_t)L * Fp : 3 * (size_t)Fp);
    float* gpart = xs + Fs;
    float* gbuf = gpart + Fs;
    float* xpub = gbuf + Fs;
    float* xown = xpub + sub;
    float* gsub = xown + sub;
    float* res = gsub + sub;
    float* bsm = res + ((2 * a.rc + 3) & ~3);
    float* gred = bsm + ((a.rc + 3) & ~3);
    uint32_t* ring = reinterpret_cast<uint32_t*>(
        (reinterpret_cast<uintptr_t>(gred + kCluThreads * FPW) + 127) & ~(uintptr_t)127);
    const size_t slot_words = (size_t)2 * a.rc * rw;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int bi = blockIdx.x;                           // the grid is one cluster: block index = rank
    const int k0 = bi * a.rc;
    const int64_t step_end = a.first_step + a.num_steps;

    auto step_rows = [&](int64_t it, int64_t& r0, int& bt, int& rcnt) {
        const int64_t t = a.order ? (int64_t)a.order[it] : it;
        r0 = t * a.batch;
        bt = (int)min(a.batch, a.m - r0);
        rcnt = max(0, min(a.rc, bt - k0));
    };
    // the tile of step `it` into `slot`: one contiguous piece per plane (one thread)
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
        mbar_init(reinterpret_cast<uint64_t*>(&sh->rs_bar), 1);
        mbar_init(reinterpret_cast<uint64_t*>(&sh->ag_bar), 1);
        mbar_init(reinterpret_cast<uint64_t*>(&sh->gn_bar), 1);
        mbar_init(reinterpret_cast<uint64_t*>(&sh->xn_bar), 1);
        sh->abort_flag = 0;
        mbar_fence_init();
    }
    for (int f = tid; f < Fp; f += kCluThreads) {
        const int q = f >> LOGF, i = f & (FPW - 1);
        if constexpr (TABLE) {
            for (int c = 0; c < L; ++c) lev[(c * FPW + i) * rw + q] = (f < n) ? __ldg(a.levels + (size_t)f * L + c) : 0.0f;
        } else {
            los[f] = (f < n) ? __ldg(a.lo + f) : 0.0f;
            steps[f] = (f < n) ? __ldg(a.step + f) : 0.0f;
        }
    }
    for (int f = tid; f < Fs; f += kCluThreads) gpart[f] = 0.0f;       // features past n stay zero
    for (int k = tid; k < sub; k += kCluThreads) xown[k] = (bi * sub + k < n) ? a.x[bi * sub + k] : 0.0f;
    __syncthreads();
    if (tid == 0)
        for (int s = 0; s < a.slots && a.first_step + s < step_end; ++s) issue_tile(a.first_step + s, s);
    cluster_sync_all();                                  // every CTA's barriers exist before anyone copies into it

    // thread roles: owner group of P lanes per owned feature; word column and row group of phase B
    const int P = 1 << a.p_shift;
    const int pp = tid & (P - 1);
    const int kpt = kCluThreads >> a.p_shift;                      // owned features handled per pass
    const int lanes_q = min(kCluThreads, ((nw + 31) / 32) * 32);
    const int ngroups = kCluThreads / lanes_q;
    const int group = tid / lanes_q, ql = tid - group * lanes_q;
    const uint32_t slice_bytes = (uint32_t)sub * 4u;

    int slot = 0;                                                  // slot and mbarrier parity of the current step's tile
    uint32_t parity = 0;
    uint32_t ag_parity = 0, rs_parity = 0, gn_parity = 0, xn_parity = 0;
    // rows of the current step (set at the end of the previous round) and the batch index one step further on
    int64_t r0 = 0;
    int bt = 1, rcnt = 0;
    int64_t t_ahead = a.order ? (int64_t)a.order[a.first_step] : a.first_step;
    for (int64_t it = a.first_step - 1; it < step_end; ++it) {
        const bool last = (it == step_end - 1);
        // arm this round's receive barriers (tx counts may arrive earlier; the phase cannot complete before this)
        if (tid == 0) {
            if (it >= a.first_step) mbar_arrive_expect_tx(reinterpret_cast<uint64_t*>(&sh->rs_bar), (uint32_t)Fs * 4u);
            if (!last) mbar_arrive_expect_tx(reinterpret_cast<uint64_t*>(&sh->ag_bar), (uint32_t)Fs * 4u);
        }
        float gq_M = 0.0f;                                         // Q4 scale of this step
        if (it >= a.first_step) {
            clu_mark(a, it, 0);
            clu_wait(sh->full + slot, parity, sh, a.status, 6);
            const uint32_t* t1 = ring + (size_t)slot * slot_words;
            const uint32_t* t2 = t1 + (size_t)a.rc * rw;
            clu_mark(a, it, 1);

            // ---------------------------------------------------------- phase A: dots and residuals
            double base = 0.0;                                     // lo^T x~ (uniform grids)
            if constexpr (!TABLE) {
#pragma unroll
                for (int w = 0; w < kCluWarps; ++w) base += sh->wbase[w];
            }
            double srow = 0.0;
#pragma unroll 1
            for (int r = warp; r < rcnt; r += kCluWarps) {
                const uint32_t* row1 = t1 + (size_t)r * rw;
                const uint32_t* row2 = t2 + (size_t)r * rw;
                float acc1 = 0.0f, acc2 = 0.0f;
#pragma unroll 2
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
                // both sums with one butterfly: the upper half-warp ends up with plane 2, the lower with plane 1
                const bool up = (lane & 16) != 0;
                double d = (double)(up ? acc2 : acc1) + __shfl_xor_sync(0xffffffffu, (double)(up ? acc1 : acc2), 16);
#pragma unroll
                for (int o = 8; o > 0; o >>= 1) d += __shfl_xor_sync(0xffffffffu, d, o);
                if ((lane & 15) == 0) {
                    const float rv = (float)(d + base - (double)bsm[r]);
                    res[2 * r + (up ? 1 : 0)] = rv;
                    srow += (double)rv;
                }
            }
            srow += __shfl_xor_sync(0xffffffffu, srow, 16);
            if (lane == 0) sh->ssum[warp] = srow;
            __syncthreads();
            clu_mark(a, it, 2);

            // ---------------------------------------------------------- phase B: the rows' part of the gradient
            double S = 0.0;                                        // sum of r1 + r2 over the CTA's rows
            if constexpr (!TABLE) {
#pragma unroll
                for (int w = 0; w < kCluWarps; ++w) S += sh->ssum[w];
            }
#pragma unroll 1
            for (int q0 = 0; q0 < nw; q0 += lanes_q) {
                const int q = q0 + ql;
                const bool active = group < ngroups && q < nw;
                float acc[FPW];
#pragma unroll
                for (int i = 0; i < FPW; ++i) acc[i] = 0.0f;
                if (active) {
#pragma unroll 2
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
                // feature adds them in order and writes the feature's entry of the CTA's part
                if (q0 > 0) __syncthreads();
                if (active) {
#pragma unroll
                    for (int i = 0; i < FPW; ++i) gred[(group * lanes_q + ql) * FPW + i] = acc[i];
                }
                __syncthreads();
#pragma unroll 1
                for (int fl = tid; fl < lanes_q * FPW; fl += kCluThreads) {
                    const int f = q0 * FPW + fl;
                    if (f < n) {
                        float v = gred[fl];
                        for (int g = 1; g < ngroups; ++g) v += gred[g * lanes_q * FPW + fl];
                        if constexpr (!TABLE) v = (float)((double)los[f] * S + (double)steps[f] * (double)v);
                        gpart[f] = v;
                    }
                }
            }
            // reduce-scatter: slice o of the part goes to owner o
            fence_async_smem();
            __syncthreads();
            // (one copy per warp: the copies of one warp's lanes would be issued one after the other)
            if (lane == 0 && warp < nb)
                bulk_copy_s2c(cluster_addr(gbuf + (size_t)bi * sub, warp), gpart + (size_t)warp * sub, slice_bytes,
                              cluster_addr(&sh->rs_bar, warp));
            // the tile is consumed: refill its slot while the parts travel
            if (tid == 1 && it + a.slots < step_end) issue_tile(it + a.slots, slot);
            if (++slot == a.slots) { slot = 0; parity ^= 1u; }
            clu_mark(a, it, 3);

            // ---------------------------------------------------------- owners: sum the parts, update
            clu_wait(&sh->rs_bar, rs_parity, sh, a.status, 2);
            rs_parity ^= 1u;
            const double scale = 1.0 / (2.0 * (double)bt);
            double gsq = 0.0;
#pragma unroll 1
            for (int kb = 0; kb < sub; kb += kpt) {
                const int k = kb + (tid >> a.p_shift);
                const int f = bi * sub + k;
                const bool mine = k < sub && f < n;
                double t = 0.0;
                if (mine)
                    for (int w = pp; w < nb; w += P) t += (double)gbuf[w * sub + k];
                for (int o = 1; o < P; o <<= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
                if (mine && pp == 0) {
                    const float g = (float)(t * scale);
                    if (last && a.grad_out) a.grad_out[f] = g;
                    gsub[k] = g;
                    gsq += (double)g * (double)g;
                }
            }
            clu_mark(a, it, 4);
            if (a.grad_bits > 0) {
                gq_M = clu_norm(gsq, sh->nrm_g, &sh->gn_bar, gn_parity, nb, sh, a.status, 3);
                gn_parity ^= 1u;
            }
#pragma unroll 1
            for (int kb = 0; kb < sub; kb += kpt) {
                const int k = kb + (tid >> a.p_shift);
                const int f = bi * sub + k;
                if (k < sub && f < n && pp == 0) {
                    float g = gsub[k];
                    if (a.grad_bits > 0)
                        g = clu_quant(g, gq_M, (1 << (a.grad_bits - 1)) - 1, a.seed, a.epoch, (uint32_t)it, 4u, (uint32_t)f);
                    if (last && a.grad_out) a.grad_out[n + f] = g;
                    xown[k] = fmaf(-a.lr, g, xown[k]);
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
            xq_M = clu_norm(xsq, sh->nrm_x, &sh->xn_bar, xn_parity, nb, sh, a.status, 8);
            xn_parity ^= 1u;
        }
#pragma unroll 1
        for (int kb = 0; kb < sub; kb += kpt) {
            const int k = kb + (tid >> a.p_shift);
            const int f = bi * sub + k;
            if (k < sub && pp == 0) {
                float xt = (f < n) ? xown[k] : 0.0f;
                if (a.model_bits > 0 && f < n)
                    xt = clu_quant(xt, xq_M, (1 << (a.model_bits - 1)) - 1, a.seed, a.epoch, (uint32_t)(it + 1), 3u, (uint32_t)f);
                xpub[k] = xt;
            }
        }
        // labels of the next step's rows: requested now, parked in shared memory after the model has arrived
        r0 = t_ahead * a.batch;
        bt = (int)min(a.batch, a.m - r0);
        rcnt = max(0, min(a.rc, bt - k0));
        if (it + 2 < step_end) t_ahead = a.order ? (int64_t)a.order[it + 2] : it + 2;
        float breg = 0.0f;
        if (tid < rcnt) breg = __ldg(a.b + r0 + k0 + tid);
        fence_async_smem();
        __syncthreads();
        if (lane == 0 && warp < nb)
            bulk_copy_s2c(cluster_addr(xs + (size_t)bi * sub, warp), xpub, slice_bytes, cluster_addr(&sh->ag_bar, warp));
        clu_mark(a, it, 5);

        // -------------------------------------------------------------- the model arrives; build w
        clu_wait(&sh->ag_bar, ag_parity, sh, a.status, 4);
        ag_parity ^= 1u;
        double bpart = 0.0;
#pragma unroll 1
        for (int f = tid; f < Fp; f += kCluThreads) {
            const float xt = (f < n) ? xs[f] : 0.0f;
            const int q = f >> LOGF, i = f & (FPW - 1);
            if constexpr (!TABLE) {
                wv[i * rw + q] = steps[f] * xt;
                bpart += (double)los[f] * (double)xt;
            } else {
                for (int c = 0; c < L; ++c) tab[(c * FPW + i) * rw + q] = lev[(c * FPW + i) * rw + q] * xt;
            }
        }
        if constexpr (!TABLE) {
            bpart = warp_sum(bpart);
            if (lane == 0) sh->wbase[warp] = bpart;
        }
        if (tid < rcnt) bsm[tid] = breg;
        for (int r = tid + kCluThreads; r < rcnt; r += kCluThreads) bsm[r] = __ldg(a.b + r0 + k0 + r);
        clu_mark(a, it, 6);
        __syncthreads();
        clu_mark(a, it, 7);
    }
    // owners return the master model
    for (int kb = 0; kb < sub; kb += kpt) {
        const int k = kb + (tid >> a.p_shift);
        if (k < sub && bi * sub + k < n && pp == 0) a.x[bi * sub + k] = xown[k];
    }
    cluster_sync_all();                                  // nobody leaves while a copy may still target it
}

// ---------------------------------------------------------------------------------------------
// Host side
// ---------------------------------------------------------------------------------------------
struct ClusterPlan {
    int nb, rc, slots, sub, p_shift;
    size_t smem;
};

static size_t cluster_smem_bytes(int cb, bool table, int row_words, int bits, int nb, int sub, int rc, int slots) {
    const size_t fpw = 32 / cb, Fp = (size_t)row_words * fpw, L = (size_t)1 << bits, Fs = (size_t)nb * sub;
    size_t bytes = (sizeof(ClusterShared) + 15) & ~(size_t)15;
    bytes += sizeof(float) * ((table ? 2 * L * Fp : 3 * Fp) + 3 * Fs + 3 * (size_t)sub + (size_t)((2 * rc + 3) & ~3) +
                              (size_t)((rc + 3) & ~3) + (size_t)kCluThreads * fpw);
    bytes += 128;                                                   // slack to align the ring to 128 bytes
    bytes += sizeof(uint32_t) * (size_t)slots * 2 * rc * row_words;
    return bytes;
}

static const void* cluster_kernel_ptr(int cb, bool table) {
    if (cb == 2) return table ? (const void*)sgd_cluster_kernel<2, true> : (const void*)sgd_cluster_kernel<2, false>;
    if (cb == 4) return table ? (const void*)sgd_cluster_kernel<4, true> : (const void*)sgd_cluster_kernel<4, false>;
    return (const void*)sgd_cluster_kernel<8, false>;
}

static int make_cluster_plan(const zipml_ctx* ctx, const zipml_dataset* d, const zipml_sgd_params* p, ClusterPlan* plan) {
    const int cb = container_bits(d->bits);
    const bool table = d->level_mode == ZIPML_LEVELS_TABLE;
    const int64_t B = p->batch < d->m ? p->batch : d->m;
    const int64_t row_words = d->row_bytes / 4;
    if (d->n > (1 << 18) || row_words > (1 << 16)) return ZIPML_ERR_WORKSPACE;
    int64_t nb = p->grid_row_parts > 0 ? p->grid_row_parts : kCluMaxCtas;
    if (p->grid_row_parts <= 0 && nb * 8 > B) nb = B / 8;           // automatic: at least 8 rows per CTA
    if (nb > kCluMaxCtas) nb = kCluMaxCtas;
    if (nb > B) nb = B;
    if (nb < 1) nb = 1;
    const size_t cap = (size_t)ctx->smem_optin;
    const int64_t nb_max = B < kCluMaxCtas ? B : kCluMaxCtas;
    // the requested number of row parts is a hint: more parts are used when a tile does not fit
    for (;; ++nb) {
        if (nb > nb_max) return ZIPML_ERR_WORKSPACE;
        ClusterPlan r;
        r.rc = (int)((B + nb - 1) / nb);
        r.nb = (int)((B + r.rc - 1) / r.rc);                        // no CTA without rows in a full batch
        const int64_t per = (d->n + r.nb - 1) / r.nb;
        r.sub = (int)((per + 3) & ~(int64_t)3);                     // slices are copied in 16-byte units
        r.p_shift = 0;
        while (r.p_shift < 5 && ((int64_t)r.sub << (r.p_shift + 1)) <= kCluThreads && (1 << r.p_shift) < r.nb) ++r.p_shift;
        if ((uint64_t)2 * r.rc * row_words * 4 >= (1u << 20)) continue;                     // mbarrier tx-count range
        if ((uint64_t)r.nb * r.sub * 4 >= (1u << 20)) continue;
        int slots = kCluMaxSlots;
        while (slots >= 2 && cluster_smem_bytes(cb, table, (int)row_words, d->bits, r.nb, r.sub, r.rc, slots) > cap) --slots;
        if (slots < 2) continue;
        r.slots = slots;
        r.smem = cluster_smem_bytes(cb, table, (int)row_words, d->bits, r.nb, r.sub, r.rc, slots);
        *plan = r;
        return ZIPML_OK;
    }
}

int launch_sgd_cluster(zipml_ctx* ctx, const zipml_dataset* d, const float* b, float* x, const zipml_sgd_params* p,
                       int64_t first_step, int64_t num_steps, float* grad_out) {
    const int cb = container_bits(d->bits);
    const bool table = d->level_mode == ZIPML_LEVELS_TABLE;
    const int fpw = 32 / cb;
    const int64_t T = (d->m + p->batch - 1) / p->batch;
    ClusterPlan plan;
    int rc = make_cluster_plan(ctx, d, p, &plan);
    if (rc != ZIPML_OK) return rc;
    const void* kernel = cluster_kernel_ptr(cb, table);
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)plan.smem);
    if (e != cudaSuccess) return cuda_status(e);
    if (plan.nb > 8) {
        e = cudaFuncSetAttribute(kernel, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
        if (e != cudaSuccess) return cuda_status(e);
    }
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = dim3((unsigned)plan.nb);
    cfg.blockDim = dim3(kCluThreads);
    cfg.dynamicSmemBytes = plan.smem;
    cfg.stream = ctx->stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)plan.nb;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    int clusters = 0;
    e = cudaOccupancyMaxActiveClusters(&clusters, kernel, &cfg);
    if (e != cudaSuccess) { (void)cudaGetLastError(); return ZIPML_ERR_WORKSPACE; }
    if (clusters < 1) return ZIPML_ERR_WORKSPACE;

    size_t off = 0;
    auto piece = [&](size_t bytes) { const size_t o = off; off += carve_size(bytes); return o; };
    const size_t o_ord = piece(sizeof(int32_t) * (size_t)(p->batch_order ? T : 0));
    rc = ws_reserve(ctx, off > 0 ? off : 256);
    if (rc != ZIPML_OK) return rc;

    ClusterArgs a;
    memset(&a, 0, sizeof(a));
    a.p1 = reinterpret_cast<const uint32_t*>(d->plane1);
    a.p2 = reinterpret_cast<const uint32_t*>(d->plane2);
    a.lo = d->feat_lo; a.step = d->feat_step; a.levels = d->levels;
    a.b = b; a.x = x; a.grad_out = grad_out;
    a.trace = reinterpret_cast<unsigned long long*>(p->trace);
    a.trace_steps = p->trace ? p->trace_steps : 0;
    a.status = ctx->d_status;
    a.m = d->m; a.batch = p->batch < d->m ? p->batch : d->m;
    a.first_step = first_step; a.num_steps = num_steps;
    a.seed = p->seed; a.epoch = (uint32_t)p->epoch; a.lr = p->lr;
    a.n = (int)d->n; a.bits = d->bits; a.row_words = (int)(d->row_bytes / 4);
    a.words = (int)((d->n + fpw - 1) / fpw);
    a.model_bits = p->model_bits; a.grad_bits = p->grad_bits;
    a.nb = plan.nb; a.rc = plan.rc; a.slots = plan.slots;
    a.sub = plan.sub; a.p_shift = plan.p_shift;
    if (p->batch_order) {
        int32_t* dev_order = reinterpret_cast<int32_t*>(ctx->ws + o_ord);
        e = cudaMemcpyAsync(dev_order, p->batch_order, sizeof(int32_t) * (size_t)T, cudaMemcpyHostToDevice, ctx->stream);
        if (e != cudaSuccess) return cuda_status(e);
        a.order = dev_order;
    }
    void* params[] = {&a};
    e = cudaLaunchKernelExC(&cfg, kernel, params);
    if (e != cudaSuccess) return cuda_status(e);
    ctx->launches += 1;
    ctx->last_engine = ZIPML_ENGINE_CLUSTER;
    return ZIPML_OK;
}

}  // namespace zipml
