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
#include <stdlib.h>
#include <string.h>

#include "int_digits.cuh"
#include "sgd_common.cuh"

namespace zipml {

constexpr int kCluThreads = 512;
constexpr int kCluWarps = kCluThreads / 32;
constexpr int kCluMaxSlots = 8;
constexpr int kCluCols = 4;                       // integer phase B: 16-byte tile columns per warp (half of it for 2-bit codes)
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
    float* model_out;            // null or n: the model the last executed step's gradient saw
    const int32_t* order;        // device copy of the batch order, or null
    unsigned long long* trace;
    DeviceStatus* status;
    int64_t m, batch, first_step, num_steps;
    uint64_t seed;
    uint32_t epoch;
    float lr;
    int reg;                     // ZIPML_REG_* and its fp32 constant
    float reg_cst;
    int n, bits, row_words, words;   // words = ceil(n / codes per word) <= row_words
    int pitch;                       // words between consecutive rows of a tile in shared memory (>= row_words)
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
    float fmax[kCluWarps];       // per-warp maxima (|w| of the word stage, then |residual|)
    uint4 zero16;                // sixteen zero bytes: the unused columns of the digit operands point here
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
    // (a phase that is complete already -- a tile copied steps ahead -- answers the non-blocking test at once)
    {
        uint32_t done;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(done) : "r"(smem_u32(bar)), "r"(parity) : "memory");
        if (done) return;
    }
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
//   uniform: wv[Fp]  w = step * x~ by feature;  los[Fp], steps[Fp]  lo and step by feature
//   table:   tab[L*Fp] level * x~ and lev[L*Fp] levels, both [code][slot i][word q]
//   xs[Fs]           the model this step sees (all-gather destination)
//   gpart[Fs]        this CTA's part of the gradient (reduce-scatter source)
//   gbuf[nb][sub]    the nb parts of the owned features (reduce-scatter destination)
//   xpub[sub], xown[sub], gsub[sub]   staging of the published slice, master model, gradient of the step
//   res[2*rc]        residuals (r1, r2) per row;   bsm[rc]  labels of the step's rows
//   gred[256*FPW]    cross-group sums of phase B (parts narrower than the CTA)
//   ring[slots][2][rc][row_words]  code tiles
template <int CB, bool TABLE, bool IMMA>
__global__ void __launch_bounds__(kCluThreads, 1) sgd_cluster_kernel(const ClusterArgs a) {
    static_assert(!(TABLE && IMMA), "level tables use the fp32 look-up path");
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
    constexpr int NG = IntPath<CB>::NG, NS = IntPath<CB>::NS;
    constexpr float QMAXF = (float)IntPath<CB>::QMAX;
    const int pitch = a.pitch;
    const int nks = (nw + 7) >> 3;                       // k-slabs of 8 words (32 bytes of codes)
    const int ncol = (nw + 3) >> 2;                      // 16-byte columns of the tile
    uint32_t* wdig = reinterpret_cast<uint32_t*>(steps + Fp);            // [k-slab][group][digit][8 words]
    unsigned char* rdig = reinterpret_cast<unsigned char*>(wdig + (size_t)((rw + 7) >> 3) * NG * NS * 8);   // [32 rows][r1, r2][digit][32 B]
    int* dacc = reinterpret_cast<int*>(rdig + (size_t)((a.rc + 31) / 32) * 256);                        // [row][plane][digit]
    float* gred = TABLE ? lev + (size_t)L * Fp : steps + Fp;             // fp32 paths
    float* xs = IMMA ? reinterpret_cast<float*>(dacc + ((a.rc + 15) & ~15) * 8) : gred + kCluThreads * FPW;
    float* gpart = xs + Fs;
    float* gbuf = gpart + Fs;
    float* xpub = gbuf + Fs;
    float* xown = xpub + sub;
    float* gsub = xown + sub;
    float* res = gsub + sub;
    float* bsm = res + ((2 * a.rc + 3) & ~3);
    uint32_t* ring = reinterpret_cast<uint32_t*>(
        (reinterpret_cast<uintptr_t>(bsm + ((a.rc + 3) & ~3)) + 127) & ~(uintptr_t)127);
    const size_t slot_words = (size_t)2 * a.rc * pitch;

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
    // the tile of step `it` into `slot`, issued by one whole warp: one contiguous piece per plane, or, when the
    // rows are padded apart in shared memory, one piece per row (the lanes share them)
    auto issue_tile = [&](int64_t it, int slot) {
        int64_t r0; int bt, rcnt;
        step_rows(it, r0, bt, rcnt);
        uint64_t* full = reinterpret_cast<uint64_t*>(sh->full + slot);
        const uint32_t bytes = (uint32_t)rcnt * (uint32_t)rw * 4u;
        if (lane == 0) mbar_arrive_expect_tx(full, 2u * bytes);
        __syncwarp();
        uint32_t* dst = ring + (size_t)slot * slot_words;
        const size_t src = (size_t)(r0 + k0) * rw;
        if (pitch == rw) {
            if (lane < 2 && rcnt > 0) bulk_copy_g2s(dst + (size_t)lane * a.rc * pitch, (lane ? a.p2 : a.p1) + src, bytes, full);
        } else {
            for (int i = lane; i < 2 * rcnt; i += 32) {
                const int pl = i & 1, r = i >> 1;
                bulk_copy_g2s(dst + (size_t)(pl * a.rc + r) * pitch, (pl ? a.p2 : a.p1) + src + (size_t)r * rw, (uint32_t)rw * 4u, full);
            }
        }
    };

    // the same for padded rows, called by every warp: lane 0 of warp w issues pieces w, w + 16, ...
    auto issue_tile_rows = [&](int64_t it, int slot) {
        int64_t r0; int bt, rcnt;
        step_rows(it, r0, bt, rcnt);
        uint64_t* full = reinterpret_cast<uint64_t*>(sh->full + slot);
        if (lane != 0) return;
        // (bytes that land before the count is armed are held against it: the phase cannot complete earlier)
        if (warp == kCluWarps - 1) mbar_arrive_expect_tx(full, 2u * (uint32_t)rcnt * (uint32_t)rw * 4u);
        uint32_t* dst = ring + (size_t)slot * slot_words;
        const size_t src = (size_t)(r0 + k0) * rw;
        for (int i = warp; i < 2 * rcnt; i += kCluWarps) {
            const int pl = i & 1, r = i >> 1;
            bulk_copy_g2s(dst + (size_t)(pl * a.rc + r) * pitch, (pl ? a.p2 : a.p1) + src + (size_t)r * rw, (uint32_t)rw * 4u, full);
        }
    };

    if (tid == 0) {
        for (int s = 0; s < a.slots; ++s) mbar_init(reinterpret_cast<uint64_t*>(sh->full + s), 1);
        mbar_init(reinterpret_cast<uint64_t*>(&sh->rs_bar), 1);
        mbar_init(reinterpret_cast<uint64_t*>(&sh->ag_bar), 1);
        mbar_init(reinterpret_cast<uint64_t*>(&sh->gn_bar), 1);
        mbar_init(reinterpret_cast<uint64_t*>(&sh->xn_bar), 1);
        sh->abort_flag = 0;
        sh->zero16 = make_uint4(0u, 0u, 0u, 0u);
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
    if constexpr (IMMA)
        for (int i = tid; i < ((a.rc + 15) & ~15) * 8; i += kCluThreads) dacc[i] = 0;
    for (int k = tid; k < sub; k += kCluThreads) xown[k] = (bi * sub + k < n) ? a.x[bi * sub + k] : 0.0f;
    __syncthreads();
    if (warp == 0)
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
    double delta_w = 0.0;                                          // one fixed-point unit of w, renewed with the model

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
            const uint32_t* t2 = t1 + (size_t)a.rc * pitch;
            clu_mark(a, it, 1);

            if constexpr (IMMA) {
                // ------------------------------------------------------ phase A: digit sums of the dots
                // A k-slab is 8 words (32 bytes of codes) of a row; a warp takes every kCluWarps-th slab for
                // each block of 16 rows and both planes: the code bytes come as A fragments straight from the
                // tile (ldmatrix), each code group of the bytes meets its own digit vectors of w (B
                // fragments), all in the same accumulators.  The warps' sums meet in dacc (integer sums: the
                // order of the atomics does not matter).  Rows past the CTA's last one are read (clamped to
                // the tile) and dropped; bytes past the row's last code meet zero digits.
                const int gl = lane >> 2, tl = lane & 3, lm = lane >> 3, l8 = lane & 7;
                const uint32_t wdig_addr = smem_u32(wdig), rdig_addr = smem_u32(rdig), zero_addr = smem_u32(&sh->zero16);
                const uint32_t tile_addr = smem_u32(t1);
                const uint32_t plane_bytes = (uint32_t)a.rc * (uint32_t)pitch * 4u;
                const int nrb = (rcnt + 15) >> 4;
#pragma unroll 1
                for (int rb0 = 0; rb0 < nrb && warp < nks; rb0 += 4) {     // four blocks of 16 rows per pass
                    int c[2][4][4];                                // [plane][row block][fragment]
#pragma unroll
                    for (int pl = 0; pl < 2; ++pl)
#pragma unroll
                        for (int rb = 0; rb < 4; ++rb)
#pragma unroll
                            for (int e = 0; e < 4; ++e) c[pl][rb][e] = 0;
#pragma unroll 1
                    for (int ks = warp; ks < nks; ks += kCluWarps) {
                        uint32_t bf[NG][2];
#pragma unroll
                        for (int g = 0; g < NG; ++g)
                            ldsm_x2(bf[g][0], bf[g][1],
                                    l8 < NS ? wdig_addr + (uint32_t)(((ks * NG + g) * NS + l8) * 32 + (lm & 1) * 16) : zero_addr);
#pragma unroll
                        for (int rb = 0; rb < 4; ++rb) {
                            if (rb0 + rb < nrb) {
                                const uint32_t row = (uint32_t)min((rb0 + rb) * 16 + l8 + (lm & 1) * 8, a.rc - 1);
                                const uint32_t addr = tile_addr + row * (uint32_t)pitch * 4u + (uint32_t)ks * 32u + (lm >> 1) * 16u;
                                uint32_t a1[4], a2[4];
                                ldsm_x4(a1, addr);
                                ldsm_x4(a2, addr + plane_bytes);
#pragma unroll
                                for (int g = 0; g < NG; ++g) {
                                    mma_u8s8(c[0][rb], group_bytes<CB>(a1[0], g), group_bytes<CB>(a1[1], g), group_bytes<CB>(a1[2], g),
                                             group_bytes<CB>(a1[3], g), bf[g][0], bf[g][1]);
                                    mma_u8s8(c[1][rb], group_bytes<CB>(a2[0], g), group_bytes<CB>(a2[1], g), group_bytes<CB>(a2[2], g),
                                             group_bytes<CB>(a2[3], g), bf[g][0], bf[g][1]);
                                }
                            }
                        }
                    }
                    if (tl < 2) {                                  // columns 2t, 2t+1 are digits; dacc is [row][plane][digit]
#pragma unroll
                        for (int rb = 0; rb < 4; ++rb) {
                            if (rb0 + rb < nrb) {
                                int* d = dacc + ((rb0 + rb) * 16 + gl) * 8 + 2 * tl;
#pragma unroll
                                for (int pl = 0; pl < 2; ++pl) {
                                    atomicAdd(d + pl * 4, c[pl][rb][0]); atomicAdd(d + pl * 4 + 1, c[pl][rb][1]);
                                    atomicAdd(d + 64 + pl * 4, c[pl][rb][2]); atomicAdd(d + 64 + pl * 4 + 1, c[pl][rb][3]);
                                }
                            }
                        }
                    }
                }
                __syncthreads();
                // residuals, one thread per (row, plane); the sums are taken and cleared
                double base = 0.0;                                 // lo^T x~
#pragma unroll
                for (int w = 0; w < kCluWarps; ++w) base += sh->wbase[w];
                double srow = 0.0;
                float rmax = 0.0f;
#pragma unroll 1
                for (int idx = tid; idx < 32 * nrb; idx += kCluThreads) {
                    const int4 dv = *reinterpret_cast<const int4*>(dacc + idx * 4);
                    *reinterpret_cast<int4*>(dacc + idx * 4) = make_int4(0, 0, 0, 0);
                    const int r = idx >> 1;
                    if (r < rcnt) {
                        const int dd[NS] = {dv.x, dv.y, dv.z, dv.w};
                        const float rv = (float)((double)combine_digits<NS>(dd) * delta_w + base - (double)bsm[r]);
                        res[idx] = rv;
                        srow += (double)rv;
                        rmax = fmaxf(rmax, fabsf(rv));
                    }
                }
                srow = warp_sum(srow);
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) rmax = fmaxf(rmax, __shfl_xor_sync(0xffffffffu, rmax, o));
                if (lane == 0) { sh->ssum[warp] = srow; sh->fmax[warp] = rmax; }
                __syncthreads();
                clu_mark(a, it, 2);
                double S = 0.0;                                    // sum of r1 + r2 over the CTA's rows
                float rho = 0.0f;
#pragma unroll
                for (int w = 0; w < kCluWarps; ++w) { S += sh->ssum[w]; rho = fmaxf(rho, sh->fmax[w]); }
                const float inv_r = rho > 0.0f ? QMAXF / rho : 0.0f;
                const float delta_rf = (float)((double)rho / (double)QMAXF), Sf = (float)S;
                // digits of the residuals as B operands of phase B: per 32 rows and residual, per digit, 32 bytes
                // in the row order the transposed code fragments come in (k = 16h + 4t + e <-> row 16h + 2t +
                // (e & 1) + 8 (e >> 1)); rows past the CTA's last one count as zero
                const int nslab = (rcnt + 31) >> 5;
                for (int kk = tid; kk < 8 * nslab; kk += kCluThreads) {
                    const int rbase = (kk >> 3) * 32 + ((kk >> 2) & 1) * 16 + 2 * (kk & 3);
                    float v1[4], v2[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const int k = rbase + (e & 1) + 8 * (e >> 1);
                        v1[e] = k < rcnt ? res[2 * k] : 0.0f;
                        v2[e] = k < rcnt ? res[2 * k + 1] : 0.0f;
                    }
                    const uint4 o1 = digit_words<NS>(v1, inv_r), o2 = digit_words<NS>(v2, inv_r);
                    uint32_t* d1 = reinterpret_cast<uint32_t*>(rdig) + (size_t)((kk >> 3) * 2 * NS) * 8 + (kk & 7);
                    d1[0] = o1.x; d1[8] = o1.y; d1[16] = o1.z; d1[24] = o1.w;
                    d1[32] = o2.x; d1[40] = o2.y; d1[48] = o2.z; d1[56] = o2.w;
                }
                __syncthreads();

                // ------------------------------------------------------ phase B: the rows' part of the gradient
                // A task is a 16-byte column of the tile over 32 rows.  A transposing ldmatrix hands each lane the
                // bytes {2g, 2g+1} of rows {2t, 2t+1} of the four 8-row groups; two permutes per half turn them
                // into A fragments "byte 2g (or 2g+1) of the column, four rows", i.e. features x rows in the row
                // order of the residual digits.  Each code group of the bytes meets the residual digits (plane 1
                // those of r2, plane 2 those of r1) in its own accumulators.
                constexpr int TI = (CB == 2) ? kCluCols / 2 : kCluCols;
#pragma unroll 1
                for (int col0 = 0; col0 < ncol; col0 += kCluWarps * TI) {      // the tile stays: wide rows take several passes
                int acc[TI][NG][4];
#pragma unroll
                for (int ti = 0; ti < TI; ++ti)
#pragma unroll
                    for (int g = 0; g < NG; ++g)
#pragma unroll
                        for (int e = 0; e < 4; ++e) acc[ti][g][e] = 0;
#pragma unroll 1
                for (int slab = 0; slab < nslab; ++slab) {
#pragma unroll
                    for (int pl = 0; pl < 2; ++pl) {
                        uint32_t b0, b1;
                        ldsm_x2(b0, b1, l8 < NS ? rdig_addr + (uint32_t)(((slab * 2 + (1 - pl)) * NS + l8) * 32 + (lm & 1) * 16) : zero_addr);
                        const uint32_t row_addr = tile_addr + pl * plane_bytes + (uint32_t)min(slab * 32 + lane, a.rc - 1) * (uint32_t)pitch * 4u;
#pragma unroll
                        for (int ti = 0; ti < TI; ++ti) {
                            const int col = col0 + warp + ti * kCluWarps;
                            if (col < ncol) {
                                uint32_t r4[4];
                                ldsm_x4_trans(r4, row_addr + (uint32_t)col * 16u);
                                const uint32_t pel = __byte_perm(r4[0], r4[1], 0x6420), pol = __byte_perm(r4[0], r4[1], 0x7531);
                                const uint32_t peh = __byte_perm(r4[2], r4[3], 0x6420), poh = __byte_perm(r4[2], r4[3], 0x7531);
#pragma unroll
                                for (int g = 0; g < NG; ++g)
                                    mma_u8s8(acc[ti][g], group_bytes<CB>(pel, g), group_bytes<CB>(pol, g), group_bytes<CB>(peh, g),
                                             group_bytes<CB>(poh, g), b0, b1);
                            }
                        }
                    }
                }
                // columns 2t, 2t+1 of lane t < 2 are digits 2t, 2t+1 (the pair in double, exact; the other pair
                // comes from lane t+1); accumulator rows g, g+8 are bytes 2g, 2g+1 of the column
#pragma unroll
                for (int ti = 0; ti < TI; ++ti) {
                    const int col = col0 + warp + ti * kCluWarps;
                    if (col < ncol) {
#pragma unroll
                        for (int g = 0; g < NG; ++g) {
#pragma unroll
                            for (int odd = 0; odd < 2; ++odd) {
                                // (the digit sums meet in 64-bit integers and are converted once: conversions to and
                                // from double run at a sixteenth of the FMA rate and made up most of this epilogue)
                                const long long pair = (long long)acc[ti][g][2 * odd] + 128ll * (long long)acc[ti][g][2 * odd + 1];
                                const long long upper = __shfl_down_sync(0xffffffffu, pair, 1);
                                const int byte_in_row = col * 16 + 2 * gl + odd;
                                const int f = (byte_in_row >> 2) * FPW + (byte_in_row & 3) * NG + g;
                                if (tl == 0 && f < n)
                                    gpart[f] = fmaf(steps[f], (float)(pair + 16384ll * upper) * delta_rf, los[f] * Sf);
                            }
                        }
                    }
                }
                }
            } else {
                // ---------------------------------------------------------- phase A: dots and residuals
                double base = 0.0;                                     // lo^T x~ (uniform grids)
                if constexpr (!TABLE) {
#pragma unroll
                    for (int w = 0; w < kCluWarps; ++w) base += sh->wbase[w];
                }
                double srow = 0.0;
#pragma unroll 1
                for (int r = warp; r < rcnt; r += kCluWarps) {
                    const uint32_t* row1 = t1 + (size_t)r * pitch;
                    const uint32_t* row2 = t2 + (size_t)r * pitch;
                    float acc1 = 0.0f, acc2 = 0.0f;
#pragma unroll 2
                    for (int q = lane; q < nw; q += 32) {
                        const uint32_t u1 = row1[q], u2 = row2[q];
                        if constexpr (!TABLE) {
                            float c1[FPW], c2[FPW];
                            unpack_word<CB>(u1, c1);
                            unpack_word<CB>(u2, c2);
                            // the word's FPW entries of w lie together: 16-byte loads, a quarter of the load instructions
                            const float4* wq = reinterpret_cast<const float4*>(wv) + (size_t)q * (FPW / 4);
#pragma unroll
                            for (int i4 = 0; i4 < FPW / 4; ++i4) {
                                const float4 w4 = wq[i4];
                                acc1 = fmaf(c1[4 * i4], w4.x, acc1); acc2 = fmaf(c2[4 * i4], w4.x, acc2);
                                acc1 = fmaf(c1[4 * i4 + 1], w4.y, acc1); acc2 = fmaf(c2[4 * i4 + 1], w4.y, acc2);
                                acc1 = fmaf(c1[4 * i4 + 2], w4.z, acc1); acc2 = fmaf(c2[4 * i4 + 2], w4.z, acc2);
                                acc1 = fmaf(c1[4 * i4 + 3], w4.w, acc1); acc2 = fmaf(c2[4 * i4 + 3], w4.w, acc2);
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
                const float Sf = (float)S;
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
                            const uint32_t u1 = t1[(size_t)r * pitch + q], u2 = t2[(size_t)r * pitch + q];
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
                            if constexpr (!TABLE) v = fmaf(steps[f], v, los[f] * Sf);      // (fp32: conversions are slow)
                            gpart[f] = v;
                        }
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
            // (row-by-row tiles: the warps share the rows, since one warp issues its copies one after the other
            // and a whole tile from one warp held the CTA's next barrier back by thousands of cycles)
            if (it + a.slots < step_end) {
                if (pitch == rw) { if (warp == kCluWarps - 1) issue_tile(it + a.slots, slot); }
                else issue_tile_rows(it + a.slots, slot);
            }
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
                if (a.model_out && it + 2 == step_end && f < n) a.model_out[f] = xt;
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
        float wm = 0.0f;
#pragma unroll 1
        for (int idx = tid; idx < Fp; idx += kCluThreads) {
            // level tables: consecutive threads take consecutive word columns of one feature slot, so that the L
            // table rows they read and write are contiguous (feature-major threads hit one bank eight times when
            // the row has a multiple of 32 words: 2 k cycles per step on 64-word rows)
            const int q = TABLE ? idx % rw : idx >> LOGF, i = TABLE ? idx / rw : idx & (FPW - 1);
            const int f = TABLE ? q * FPW + i : idx;
            const float xt = (f < n) ? xs[f] : 0.0f;
            if constexpr (IMMA) {
                const float w = steps[f] * xt;
                wv[f] = w;
                wm = fmaxf(wm, fabsf(w));
                bpart += (double)los[f] * (double)xt;
            } else if constexpr (!TABLE) {
                wv[f] = steps[f] * xt;
                bpart += (double)los[f] * (double)xt;
            } else {
                for (int c = 0; c < L; ++c) tab[(c * FPW + i) * rw + q] = lev[(c * FPW + i) * rw + q] * xt;
            }
        }
        if constexpr (!TABLE) {
            bpart = warp_sum(bpart);
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) wm = fmaxf(wm, __shfl_xor_sync(0xffffffffu, wm, o));
            if (lane == 0) { sh->wbase[warp] = bpart; sh->fmax[warp] = wm; }
        }
        if (tid < rcnt) bsm[tid] = breg;
        for (int r = tid + kCluThreads; r < rcnt; r += kCluThreads) bsm[r] = __ldg(a.b + r0 + k0 + r);
        if constexpr (IMMA) {
            // digits of w as B operands of phase A, scaled by the largest |w| of the whole vector: per k-slab
            // (8 words), code group and digit a 32-byte k vector
            __syncthreads();
            float wmax = 0.0f;
#pragma unroll
            for (int w = 0; w < kCluWarps; ++w) wmax = fmaxf(wmax, sh->fmax[w]);
            const float inv_w = wmax > 0.0f ? QMAXF / wmax : 0.0f;
            delta_w = (double)wmax / (double)QMAXF;
#pragma unroll 1
            for (int item = tid; item < 8 * ((rw + 7) >> 3) * NG; item += kCluThreads) {
                const int q = item / NG, g = item - q * NG;
                uint4 o = make_uint4(0u, 0u, 0u, 0u);
                if (q < rw) {
                    const float v4[4] = {wv[q * FPW + g], wv[q * FPW + NG + g], wv[q * FPW + 2 * NG + g], wv[q * FPW + 3 * NG + g]};
                    o = digit_words<NS>(v4, inv_w);
                }
                uint32_t* dst = wdig + (size_t)(((q >> 3) * NG + g) * NS) * 8 + (q & 7);
                dst[0] = o.x; dst[8] = o.y; dst[16] = o.z; dst[24] = o.w;
            }
        }
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
    int nb, rc, slots, sub, p_shift, pitch;
    bool imma;                   // uniform grids: int8 tensor-core contraction instead of fp32 FMA
    size_t smem;
};

// Rows of a tile lie `pitch` words apart in shared memory.  The integer path loads fragments of 8 rows x 16
// bytes; they fall into 8 different bank groups when the pitch is an odd number of 16-byte units.
static int cluster_pitch(bool imma, int row_words) { return (!imma || ((row_words / 4) & 1)) ? row_words : row_words + 4; }

static size_t cluster_smem_bytes(int cb, bool table, bool imma, int row_words, int bits, int nb, int sub, int rc, int slots) {
    const size_t fpw = 32 / cb, Fp = (size_t)row_words * fpw, L = (size_t)1 << bits, Fs = (size_t)nb * sub;
    size_t bytes = (sizeof(ClusterShared) + 15) & ~(size_t)15;
    if (imma) bytes += sizeof(float) * 3 * Fp + (size_t)((row_words + 7) / 8) * (8 / cb) * 4 * 32 + (size_t)((rc + 31) / 32) * 256 +
                       sizeof(int) * (size_t)((rc + 15) & ~15) * 8;
    else bytes += sizeof(float) * ((table ? 2 * L * Fp : 3 * Fp) + (size_t)kCluThreads * fpw);
    bytes += sizeof(float) * (3 * Fs + 3 * (size_t)sub + (size_t)((2 * rc + 3) & ~3) + (size_t)((rc + 3) & ~3));
    bytes += 128 + 64;                                              // slack to align the ring, and past its last row
    bytes += sizeof(uint32_t) * (size_t)slots * 2 * rc * cluster_pitch(imma, row_words);
    return bytes;
}

static const void* cluster_kernel_ptr(int cb, bool table, bool imma) {
    if (cb == 2) return table ? (const void*)sgd_cluster_kernel<2, true, false> : imma ? (const void*)sgd_cluster_kernel<2, false, true> : (const void*)sgd_cluster_kernel<2, false, false>;
    if (cb == 4) return table ? (const void*)sgd_cluster_kernel<4, true, false> : imma ? (const void*)sgd_cluster_kernel<4, false, true> : (const void*)sgd_cluster_kernel<4, false, false>;
    return imma ? (const void*)sgd_cluster_kernel<8, false, true> : (const void*)sgd_cluster_kernel<8, false, false>;
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
    // the caller may fix the contraction for uniform grids (tests, tuning): 1 = fp32, 2 = int8 tensor cores
    const int force_int8 = p->cluster_contraction == 1 ? 0 : p->cluster_contraction == 2 ? 1 : -1;
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
        // the integer contraction pays its per-step digit conversions back on tiles of 24 KiB per plane and more
        // (measured: 16 rows x 1 KB 6.6 vs 5.5 us per step in fp32; 64 rows x 512 B 17.3 vs 21.6 us)
        r.imma = !table && (int64_t)r.rc * d->row_bytes >= 24 * 1024;
        if (!table && force_int8 >= 0) r.imma = force_int8 != 0;
        r.pitch = cluster_pitch(r.imma, (int)row_words);
        int slots = kCluMaxSlots;
        while (slots >= 2 && cluster_smem_bytes(cb, table, r.imma, (int)row_words, d->bits, r.nb, r.sub, r.rc, slots) > cap) --slots;
        if (slots < 2) continue;
        r.slots = slots;
        r.smem = cluster_smem_bytes(cb, table, r.imma, (int)row_words, d->bits, r.nb, r.sub, r.rc, slots);
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
    const void* kernel = cluster_kernel_ptr(cb, table, plan.imma);
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
    a.b = b; a.x = x; a.grad_out = grad_out; a.model_out = p->model_out;
    a.trace = reinterpret_cast<unsigned long long*>(p->trace);
    a.trace_steps = p->trace ? p->trace_steps : 0;
    a.status = ctx->d_status;
    a.m = d->m; a.batch = p->batch < d->m ? p->batch : d->m;
    a.first_step = first_step; a.num_steps = num_steps;
    a.seed = p->seed; a.epoch = (uint32_t)p->epoch; a.lr = p->lr; a.reg = p->reg; a.reg_cst = reg_constant(p);
    a.n = (int)d->n; a.bits = d->bits; a.row_words = (int)(d->row_bytes / 4);
    a.words = (int)((d->n + fpw - 1) / fpw);
    a.model_bits = p->model_bits; a.grad_bits = p->grad_bits;
    a.nb = plan.nb; a.rc = plan.rc; a.slots = plan.slots;
    a.sub = plan.sub; a.p_shift = plan.p_shift; a.pitch = plan.pitch;
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
