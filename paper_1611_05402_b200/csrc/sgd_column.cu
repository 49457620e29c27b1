// Column engine of zipml_sgd_epoch: large minibatch tiles on uniform grids, fp32 model and gradient,
// every code byte read from HBM exactly once per step.
//
// A step of the double-sampled minibatch SGD (paper Eq. (double) in its symmetrised form, footnote of
// "Double Sampling"; update in full precision, "End-to-end Quantization") needs the step's code tile
// twice: for the dots q1^T x, q2^T x of every row, and, once the residuals r = dot - b are known, for
// the gradient 1/(2B) sum_k [q1_k r2_k + q2_k r1_k].  Here the features are partitioned: CTA j owns
// the 128-byte column block j of the packed rows (1024 / CB features) for all rows and the whole
// launch, so its slice of the model, of w = step * x and of the gradient never leave the CTA, and the
// only thing CTAs exchange is the rows' dots.  Rows travel in chunks of R rows (both planes, R x 128
// bytes each, one 2-D tensor copy per plane with the 128-byte swizzle) through a ring of shared-memory
// slots, and a chunk stays in its slot until both of its uses are over:
//
//   producer  (1 warp)   tensor copies of the coming chunks, across step boundaries (codes do not depend
//                        on the model); publishes "this CTA's dots of chunk q are added" to a counter
//   A warps   (8)        partial dots of the chunk from shared memory on the int8 tensor cores
//                        (mma.sync m16n8k32, u8 codes x s8 digits of w), converted to a fixed-point unit
//                        common to all CTAs and added to dots[row] with 64-bit integer atomics
//   R warps   (4)        wait until all CTAs' parts of the chunk have arrived (counter), read the chunk's
//                        dots and labels, turn the residuals into eight balanced base-128 int8 digits
//   B warps   (8)        gradient of the CTA's own features from the same slot (transposing ldmatrix,
//                        residual digits as the other operand), accumulated in registers over the step;
//                        at the step's end: update of the own slice of x, digits of the next w
//
// There is no grid-wide barrier: while the exchange of chunk q settles (about one L2 round trip plus
// the slowest CTA's lag) the CTA streams and processes the chunks behind it.  At a step's end the
// pipeline drains (the next dots need the whole new w of the CTA), while the producer keeps filling
// free slots with the next step's first chunks.
//
// Fixed point.  w of the own features: four digits relative to the CTA's own max |w| (27 bits).  Dots:
// each CTA rounds its part (own part of lo^T x + delta * digit sums) to a multiple of U = 2^e / 2^61
// where 2^e >= D, and D bounds every |dot| of the step: D(0) = sum_j |x_j| amax_j from the caller's
// model, D(t+1) = grow * D(t) + lr * rmax(t) * sum_j amax_j^2 (amax_j the largest |value| of feature
// j, rmax(t) the step's largest |residual|, which every CTA reads off the same dots): every CTA
// derives the same U without asking anyone, 64-bit sums of multiples of U are exact and order-free,
// and the bound may be loose by 2^30 before 2^-31 relative precision is touched.  Residuals: eight
// digits (55 bits) relative to D(t) + max |b| of the step, for the same reason; all eight columns of
// the tensor-core tile carry a digit.  Results do not depend on timing: every sum is an integer sum or
// has a fixed order.
#include <cuda.h>
#include <string.h>

#include "int_digits.cuh"
#include "sgd_common.cuh"

namespace zipml {

constexpr int kColAWarps = 8, kColBWarps = 8, kColRWarps = 4;
constexpr int kColWarpA0 = 1, kColWarpB0 = kColWarpA0 + kColAWarps, kColWarpR0 = kColWarpB0 + kColBWarps;
constexpr int kColThreads = 32 * (kColWarpR0 + kColRWarps);
constexpr int kColRThreads = 32 * kColRWarps;
constexpr int kColBThreads = 32 * kColBWarps;
constexpr int kColBlockBytes = 128;         // bytes of a packed row that a CTA owns
constexpr int kColMaxBatch = 8192;
constexpr int kColMaxSlots = 8;
constexpr int kColRDigits = 8;              // digits of a residual
constexpr long long kColQmaxR = 35000000000000000LL;     // below 63 * (128^8 - 1) / 127
constexpr long long kColWaitCycles = 6000000000LL;       // a wait gives up after about three seconds
constexpr int kColNamedR = 1, kColNamedB = 2;            // named barriers of the R and B warps

struct ColumnArgs {
    int64_t m, batch, first_step, num_steps;
    const int32_t* order;
    const float* lo;
    const float* step;
    const float* b;
    float* x;
    float* grad_out;
    int n, bits;
    int R;                   // rows of a chunk (multiple of 32)
    int slots;               // ring slots
    int bpad;                // rows of a dots buffer: chunks of the largest step * R
    int ring;                // entries of the counter ring (a power of two)
    float lr;
    int reg;
    float reg_cst;
    long long* dots;         // [3][2][bpad] fixed-point dots (three steps in rotation), zeroed before the launch
    unsigned* count;         // [ring][32] one counter per chunk in flight (128 bytes apart), zeroed before the launch
    DeviceStatus* status;
    unsigned long long* trace;
    int trace_steps;
};

struct ColStepParams {       // by step parity
    double U, invU;          // fixed-point unit of the dots                     (R warps -> A, R warps)
    double delta_w, base;    // unit of the w digits, own part of lo^T x        (B warps -> A warps)
    double inv_r, delta_r;   // fixed point of the residuals                     (R warps -> B warps)
    double rsum;             // sum of all fixed-point residuals of the step     (R warps -> B warps)
};

struct ColShared {
    unsigned long long full[kColMaxSlots];     // the slot's tensor copies have landed
    unsigned long long empty[kColMaxSlots];    // the B warps are done with the slot
    unsigned long long adone[kColMaxSlots];    // the A warps have added the slot's dots
    unsigned long long rfull[2], rempty[2];    // residual digits of a chunk: written / consumed
    unsigned long long wready;                 // digits of the next w are in place
    ColStepParams sp[2];
    double red_d[2][32];
    float red_f[2][32];
    long long red_l[2][kColRWarps];
    int abort_flag;
};

__device__ __forceinline__ bool col_aborted(const ColShared* sh) { return *reinterpret_cast<const volatile int*>(&sh->abort_flag) != 0; }

__device__ __forceinline__ bool mbar_test_wait(unsigned long long* bar, uint32_t parity) {
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done) : "r"(smem_u32(bar)), "r"(parity) : "memory");
    return done != 0;
}

// Bounded wait on a local mbarrier phase.  False once this CTA has given up anywhere.
__device__ __forceinline__ bool col_wait(unsigned long long* bar, uint32_t parity, ColShared* sh, DeviceStatus* status, int where) {
    if (mbar_test_wait(bar, parity)) return true;
    if (col_aborted(sh)) return false;
    const long long t0 = clock64();
#pragma unroll 1
    for (int spin = 0;; ++spin) {
        if (mbar_try_wait(reinterpret_cast<uint64_t*>(bar), parity)) return true;
        if ((spin & 15) == 15) {
            if (col_aborted(sh)) return false;
            if (clock64() - t0 > kColWaitCycles) break;
        }
    }
    sh->abort_flag = 1;
    set_status(status, ZIPML_ERR_TIMEOUT, where);
    return false;
}

__device__ __forceinline__ void named_barrier(int id, int threads) { asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory"); }

__device__ __forceinline__ void tensor_load_2d(void* dst_smem, const CUtensorMap* tm, int x, int y, unsigned long long* bar) {
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                 ::"r"(smem_u32(dst_smem)), "l"(tm), "r"(x), "r"(y), "r"(smem_u32(bar)) : "memory");
}

__device__ __forceinline__ void col_mark(const ColumnArgs& a, int64_t t_rel, int k) {
    if (a.trace && blockIdx.x == 0 && t_rel < a.trace_steps) a.trace[t_rel * 8 + k] = (unsigned long long)clock64();
}

// Rows of step position `it`.
struct ColStep {
    int64_t row0;
    int bt, nch;
};
__device__ __forceinline__ ColStep col_step(const ColumnArgs& a, int64_t it) {
    ColStep s;
    const int64_t t = a.order ? (int64_t)a.order[it] : it;
    s.row0 = t * a.batch;
    s.bt = (int)min(a.batch, a.m - s.row0);
    s.nch = (s.bt + a.R - 1) / a.R;
    return s;
}

template <int CB>
__global__ void __launch_bounds__(kColThreads, 1) sgd_column_kernel(const ColumnArgs a, const __grid_constant__ CUtensorMap tm1,
                                                                    const __grid_constant__ CUtensorMap tm2) {
    constexpr int NG = 8 / CB;                         // codes per byte = code groups
    constexpr int NS = IntPath<CB>::NS;                // digits of w
    constexpr int QMAXW = IntPath<CB>::QMAX;
    constexpr int NF = (2 * NG + 3) / 4;               // own features per B-warp lane
    constexpr int NRD = kColRDigits;
    static_assert(NS == 4, "four digits of w");
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    // [slots][2 planes][R rows][128 B] (1024-byte aligned), then the digit operands, then the bookkeeping
    unsigned char* tiles = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const int R = a.R;
    const uint32_t plane_bytes = (uint32_t)R * kColBlockBytes, slot_bytes = 2u * plane_bytes;
    const int rstride = R + 32;                        // bytes between the residual digit vectors
    signed char* rdig = reinterpret_cast<signed char*>(tiles + (size_t)a.slots * slot_bytes);     // [2 buffers][2 operands][8 digits][rstride]
    signed char* wdig = rdig + (size_t)2 * 2 * NRD * rstride;                                      // [NG][4 k-blocks][4 digits][32 B]
    ColShared* sh = reinterpret_cast<ColShared*>((reinterpret_cast<uintptr_t>(wdig + NG * 4 * NS * 32) + 15) & ~(uintptr_t)15);

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, gl = lane >> 2, tl = lane & 3;
    const int cta = blockIdx.x, G = gridDim.x;
    const int n = a.n;
    const int64_t steps = a.num_steps;
    const int64_t byte0 = (int64_t)cta * kColBlockBytes;          // first byte of the own column block

    if (tid == 0) {
        for (int s = 0; s < a.slots; ++s) {
            mbar_init(reinterpret_cast<uint64_t*>(sh->full + s), 1);
            mbar_init(reinterpret_cast<uint64_t*>(sh->empty + s), kColBWarps);
            mbar_init(reinterpret_cast<uint64_t*>(sh->adone + s), kColAWarps);
        }
        for (int s = 0; s < 2; ++s) {
            mbar_init(reinterpret_cast<uint64_t*>(sh->rfull + s), kColRWarps);
            mbar_init(reinterpret_cast<uint64_t*>(sh->rempty + s), kColBWarps);
        }
        mbar_init(reinterpret_cast<uint64_t*>(&sh->wready), kColBWarps);
        sh->abort_flag = 0;
        mbar_fence_init();
    }
    // ---- every CTA scans the model once, with the same arithmetic: the bound of the dots and its growth rate
    const float smax = (float)((1 << a.bits) - 1);
    double dsum = 0.0, csum = 0.0;
    for (int j = tid; j < n; j += kColThreads) {
        const float l = a.lo[j], s = a.step[j];
        const double am = (double)fmaxf(fabsf(l), fabsf(l + s * smax));
        dsum += am * (double)fabsf(a.x[j]);
        csum += am * am;
    }
    dsum = warp_sum(dsum);
    csum = warp_sum(csum);
    if (lane == 0) { sh->red_d[0][warp] = dsum; sh->red_d[1][warp] = csum; }
    __syncthreads();
    double dbound = 0.0, c2 = 0.0;
    for (int w = 0; w < kColThreads / 32; ++w) { dbound += sh->red_d[0][w]; c2 += sh->red_d[1][w]; }
    dbound *= 1.0001;
    auto unit_of = [](double bound, double& U, double& invU) {
        int ex = 0;
        if (bound > 0.0) (void)frexp(bound, &ex);        // bound <= 2^ex
        U = ldexp(1.0, ex - 61);
        invU = ldexp(1.0, 61 - ex);
    };
    if (tid == 0) unit_of(dbound, sh->sp[0].U, sh->sp[0].invU);
    __syncthreads();                                      // barriers initialised, sums read, U(0) in place

    // =================================================================================== producer
    if (warp == 0) {
        if (lane == 0) {
            int64_t tL = 0, tP = 0;                       // steps of the next chunk to load / to publish
            int cL = 0, cP = 0;
            int64_t qL = 0, qP = 0;                       // their positions in the launch's chunk sequence
            ColStep sL = col_step(a, a.first_step), sP = sL;
            long long idle0 = clock64();
            bool ok = true;
            while (tP < steps && ok) {
                bool progress = false;
                if (tL < steps) {
                    const int slot = (int)(qL % a.slots);
                    const int64_t use = qL / a.slots;
                    if (use == 0 || mbar_test_wait(sh->empty + slot, (uint32_t)((use - 1) & 1))) {
                        unsigned char* dst = tiles + (size_t)slot * slot_bytes;
                        mbar_arrive_expect_tx(reinterpret_cast<uint64_t*>(sh->full + slot), slot_bytes);
                        const int y = (int)(sL.row0 + (int64_t)cL * R);
                        tensor_load_2d(dst, &tm1, (int)byte0, y, sh->full + slot);
                        tensor_load_2d(dst + plane_bytes, &tm2, (int)byte0, y, sh->full + slot);
                        ++qL;
                        if (++cL == sL.nch) { cL = 0; if (++tL < steps) sL = col_step(a, a.first_step + tL); }
                        progress = true;
                    }
                }
                if (qP < qL) {
                    const int slot = (int)(qP % a.slots);
                    if (mbar_test_wait(sh->adone + slot, (uint32_t)((qP / a.slots) & 1))) {
                        // every A warp's additions come before its arrival, this thread's fence after its wait:
                        // whoever sees the count sees the sums
                        __threadfence();
                        atomicAdd(a.count + (size_t)(qP & (a.ring - 1)) * 32, 1u);
                        ++qP;
                        if (++cP == sP.nch) {
                            if (blockIdx.x == 0 && a.trace && tP < a.trace_steps) a.trace[tP * 8 + 6] = (unsigned long long)clock64();
                            cP = 0;
                            if (++tP < steps) sP = col_step(a, a.first_step + tP);
                        }
                        progress = true;
                    }
                }
                if (progress) idle0 = clock64();
                else {
                    if (col_aborted(sh)) ok = false;
                    else if (clock64() - idle0 > kColWaitCycles) { sh->abort_flag = 1; set_status(a.status, ZIPML_ERR_TIMEOUT, 70); ok = false; }
                }
            }
            if (!ok) {
                // leaving early: the copies in flight must land before the CTA's shared memory goes away
                for (int64_t q = (qL > a.slots ? qL - a.slots : 0); q < qL; ++q) {
                    const long long t0 = clock64();
                    while (!mbar_test_wait(sh->full + (q % a.slots), (uint32_t)((q / a.slots) & 1)) && clock64() - t0 < kColWaitCycles) {}
                }
            }
        }
    }
    // =================================================================================== A warps: dots
    else if (warp < kColWarpB0) {
        const int aw = warp - kColWarpA0;
        int64_t q = 0;
        constexpr uint32_t kLow = CB == 8 ? 0xFFFFFFFFu : CB == 4 ? 0x0F0F0F0Fu : 0x03030303u;
        // ldmatrix row addresses: lane l gives row (l & 7) + 8 * ((l >> 3) & 1) of the 16-row block and the
        // 16-byte piece (l >> 4) of a 32-byte k-block; the 128-byte swizzle moves piece c of row r to c ^ (r & 7)
        const uint32_t a_row = (uint32_t)((lane & 7) + 8 * ((lane >> 3) & 1)), a_piece = (uint32_t)(lane >> 4), a_x = (uint32_t)(lane & 7);
        const uint32_t wdig_lane = smem_u32(wdig) + (uint32_t)(gl * 32 + tl * 8);          // lanes with gl < 4 read digit gl
        bool ok = true;
        for (int64_t t_rel = 0; t_rel < steps && ok; ++t_rel) {
            const ColStep st = col_step(a, a.first_step + t_rel);
            ok = __all_sync(0xffffffffu, col_wait(&sh->wready, (uint32_t)(t_rel & 1), sh, a.status, 71));     // (the warp acts as one)
            if (!ok) break;
            if (aw == 0 && lane == 0) col_mark(a, t_rel, 0);
            const ColStepParams& sp = sh->sp[t_rel & 1];
            const double invU = sp.invU, delta_w = sp.delta_w, base = sp.base;
            long long* dots = a.dots + (size_t)(t_rel % 3) * 2 * a.bpad;
            for (int c = 0; c < st.nch; ++c, ++q) {
                const int slot = (int)(q % a.slots);
                ok = __all_sync(0xffffffffu, col_wait(sh->full + slot, (uint32_t)((q / a.slots) & 1), sh, a.status, 72));
                if (!ok) break;
                const uint32_t tile = smem_u32(tiles) + (uint32_t)slot * slot_bytes;
                for (int rb = aw; rb < R / 16; rb += kColAWarps) {
                    const int k0 = c * R + rb * 16;                      // first row of the block within the step
                    if (k0 >= st.bt) break;
                    int c1[NG][4], c2[NG][4];
#pragma unroll
                    for (int g = 0; g < NG; ++g)
#pragma unroll
                        for (int e = 0; e < 4; ++e) { c1[g][e] = 0; c2[g][e] = 0; }
                    const uint32_t row_addr = tile + (uint32_t)(rb * 16 + a_row) * kColBlockBytes;
#pragma unroll
                    for (int kb = 0; kb < 4; ++kb) {
                        uint32_t f1[4], f2[4];
                        const uint32_t off = row_addr + (((uint32_t)(2 * kb) + a_piece) ^ a_x) * 16u;
                        ldsm_x4(f1, off);
                        ldsm_x4(f2, off + plane_bytes);
#pragma unroll
                        for (int g = 0; g < NG; ++g) {
                            uint32_t b0 = 0u, b1 = 0u;
                            if (gl < NS) asm volatile("ld.shared.v2.u32 {%0, %1}, [%2];" : "=r"(b0), "=r"(b1) : "r"(wdig_lane + (uint32_t)((g * 4 + kb) * NS * 32)));
                            // group g's codes stay where they are in the byte: its sums come out 2^(g CB) times too large
                            const uint32_t mk = kLow << (g * CB);
                            mma_u8s8(c1[g], f1[0] & mk, f1[1] & mk, f1[2] & mk, f1[3] & mk, b0, b1);
                            mma_u8s8(c2[g], f2[0] & mk, f2[1] & mk, f2[2] & mk, f2[3] & mk, b0, b1);
                        }
                    }
                    // lane t < 2 holds digits 2t, 2t+1 of rows g (c[0], c[1]) and g+8 (c[2], c[3])
#pragma unroll
                    for (int e = 0; e < 2; ++e) {
                        long long q1 = 0, q2 = 0;
#pragma unroll
                        for (int g = 0; g < NG; ++g) {                   // exact: the sums are multiples of 2^(g CB)
                            q1 += (long long)(c1[g][2 * e] >> (g * CB)) + 128ll * (long long)(c1[g][2 * e + 1] >> (g * CB));
                            q2 += (long long)(c2[g][2 * e] >> (g * CB)) + 128ll * (long long)(c2[g][2 * e + 1] >> (g * CB));
                        }
                        const long long v1 = q1 + 16384ll * __shfl_down_sync(0xffffffffu, q1, 1);
                        const long long v2 = q2 + 16384ll * __shfl_down_sync(0xffffffffu, q2, 1);
                        const int k = k0 + gl + 8 * e;
                        if (tl == 0 && k < st.bt) {
                            // this CTA's part of the dot, as a multiple of the unit every CTA uses this step
                            const long long P1 = __double2ll_rn(((double)v1 * delta_w + base) * invU);
                            const long long P2 = __double2ll_rn(((double)v2 * delta_w + base) * invU);
                            atomicAdd(reinterpret_cast<unsigned long long*>(dots + k), (unsigned long long)P1);
                            atomicAdd(reinterpret_cast<unsigned long long*>(dots + a.bpad + k), (unsigned long long)P2);
                        }
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(reinterpret_cast<uint64_t*>(sh->adone + slot));
            }
            if (aw == 0 && lane == 0) col_mark(a, t_rel, 1);
        }
    }
    // =================================================================================== B warps: gradient, update
    else if (warp < kColWarpR0) {
        const int p = warp - kColWarpB0;                 // the warp's 16-byte piece of the column block
        const int btid = tid - 32 * kColWarpB0;
        // own features: (byte 2g + h of the piece, code group gi), fi = h * NG + gi = tl + 4e
        float xo[NF], lo_o[NF], st_o[NF];
        int64_t jo[NF];
        bool have[NF];
#pragma unroll
        for (int e = 0; e < NF; ++e) {
            const int fi = tl + 4 * e, h = fi / NG, gi = fi - h * NG;
            have[e] = fi < 2 * NG;
            jo[e] = (byte0 + 16 * p + 2 * gl + h) * NG + gi;
            have[e] = have[e] && jo[e] < n;
            xo[e] = have[e] ? a.x[jo[e]] : 0.0f;
            lo_o[e] = have[e] ? a.lo[jo[e]] : 0.0f;
            st_o[e] = have[e] ? a.step[jo[e]] : 0.0f;
        }
        // digits of w = step * x of the own features for the step at parity `par`, and the own part of lo^T x
        auto publish_w = [&](int par) {
            float wm = 0.0f;
            double bs = 0.0;
#pragma unroll
            for (int e = 0; e < NF; ++e) { wm = fmaxf(wm, fabsf(st_o[e] * xo[e])); bs += (double)lo_o[e] * (double)xo[e]; }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) wm = fmaxf(wm, __shfl_xor_sync(0xffffffffu, wm, o));
            bs = warp_sum(bs);
            if (lane == 0) { sh->red_f[0][p] = wm; sh->red_d[0][p] = bs; }
            named_barrier(kColNamedB, kColBThreads);
            float wmax = 0.0f;
            double bsum = 0.0;
#pragma unroll
            for (int w = 0; w < kColBWarps; ++w) { wmax = fmaxf(wmax, sh->red_f[0][w]); bsum += sh->red_d[0][w]; }
            const float inv = wmax > 0.0f ? (float)QMAXW / wmax : 0.0f;
            if (btid == 0) { sh->sp[par].delta_w = (double)wmax / (double)QMAXW; sh->sp[par].base = bsum; }
#pragma unroll
            for (int e = 0; e < NF; ++e) {
                const int fi = tl + 4 * e, h = fi / NG, gi = fi - h * NG;
                if (fi < 2 * NG) {
                    const int byte = 16 * p + 2 * gl + h, kb = byte >> 5, bb = byte & 31;
                    int d[NS];
                    balanced_digits<NS>(have[e] ? max(-QMAXW, min(QMAXW, __float2int_rn(st_o[e] * xo[e] * inv))) : 0, d);
                    signed char* dst = wdig + (size_t)((gi * 4 + kb) * NS) * 32 + ((bb & 15) >> 2) * 8 + (bb >> 4) * 4 + (bb & 3);
#pragma unroll
                    for (int s = 0; s < NS; ++s) dst[s * 32] = (signed char)d[s];
                }
            }
            named_barrier(kColNamedB, kColBThreads);     // (also: nobody re-enters with red_* still being read)
            __syncwarp();
            if (lane == 0) mbar_arrive(reinterpret_cast<uint64_t*>(&sh->wready));
        };
        publish_w(0);

        const uint32_t b_x = (uint32_t)(lane & 7);
        const uint32_t b_off = (uint32_t)lane * kColBlockBytes + (((uint32_t)p ^ b_x) << 4);
        const uint32_t rdig_lane = smem_u32(rdig) + (uint32_t)(gl * rstride + tl * 8);
        int64_t q = 0;
        // After a wait has given up the warp stays in step with the others (the named barriers below need every
        // B thread) but waits for nothing and skips the arithmetic.
        bool ok = true;
        for (int64_t t_rel = 0; t_rel < steps; ++t_rel) {
            const ColStep st = col_step(a, a.first_step + t_rel);
            const bool last = t_rel + 1 == steps;
            int acc[NG][4];
#pragma unroll
            for (int g = 0; g < NG; ++g)
#pragma unroll
                for (int e = 0; e < 4; ++e) acc[g][e] = 0;
            for (int c = 0; c < st.nch; ++c, ++q) {
                const int slot = (int)(q % a.slots), rbuf = (int)(q & 1);
                ok = ok && col_wait(sh->rfull + rbuf, (uint32_t)((q >> 1) & 1), sh, a.status, 73);
                ok = ok && col_wait(sh->full + slot, (uint32_t)((q / a.slots) & 1), sh, a.status, 74);     // (landed long ago: makes the copy's bytes visible here)
                ok = __all_sync(0xffffffffu, ok);                      // the warp acts as one
                const uint32_t tile = smem_u32(tiles) + (uint32_t)slot * slot_bytes + b_off;
                const int nrb = ok ? (min(R, st.bt - c * R) + 31) >> 5 : 0;
#pragma unroll 1
                for (int rb = 0; rb < nrb; ++rb) {
#pragma unroll
                    for (int pl = 0; pl < 2; ++pl) {
                        uint32_t r4[4], b0, b1;
                        ldsm_x4_trans(r4, tile + (uint32_t)pl * plane_bytes + (uint32_t)rb * 32u * kColBlockBytes);
                        asm volatile("ld.shared.v2.u32 {%0, %1}, [%2];" : "=r"(b0), "=r"(b1)
                                     : "r"(rdig_lane + (uint32_t)(((rbuf * 2 + pl) * NRD) * rstride + rb * 32)));
                        // bytes {2g, 2g+1} of rows {2t, 2t+1} of the four 8-row groups -> byte 2g (and 2g+1) of rows
                        // {2t, 2t+1, 8+2t, 9+2t} (+16): features x rows, in the row order of the residual digits
                        const uint32_t e0 = __byte_perm(r4[0], r4[1], 0x6420), o0 = __byte_perm(r4[0], r4[1], 0x7531);
                        const uint32_t e1 = __byte_perm(r4[2], r4[3], 0x6420), o1 = __byte_perm(r4[2], r4[3], 0x7531);
#pragma unroll
                        for (int g = 0; g < NG; ++g) {
                            // All groups of a byte meet the same residual digits, so the sums may nest: accumulator g
                            // takes the byte with the groups below g cleared (g = 0: the byte as it is), i.e.
                            // sum_{h >= g} 2^(h CB) code_h; group g is the difference of two neighbours.
                            const uint32_t mk = 0x01010101u * (uint32_t)((0xFFu << (g * CB)) & 0xFFu);
                            mma_u8s8(acc[g], e0 & mk, o0 & mk, e1 & mk, o1 & mk, b0, b1);
                        }
                    }
                }
                __syncwarp();
                if (lane == 0) {
                    mbar_arrive(reinterpret_cast<uint64_t*>(sh->empty + slot));
                    mbar_arrive(reinterpret_cast<uint64_t*>(sh->rempty + rbuf));
                }
            }
            if (p == 0 && lane == 0) col_mark(a, t_rel, 4);
            // ---- the step's gradient of the own features; update; digits of the next w
            // lane (g, t): acc[gi][0..1] = digits 2t, 2t+1 of byte 2g, acc[gi][2..3] of byte 2g+1
            const ColStepParams& sp = sh->sp[t_rel & 1];
            const double delta_r = sp.delta_r, lo_term = sp.delta_r * sp.rsum, scale = 1.0 / (2.0 * (double)st.bt);
            const double w0 = (tl == 0) ? 1.0 : (tl == 1) ? 16384.0 : (tl == 2) ? 268435456.0 : 4398046511104.0;     // 128^(2t)
            double Sf[NF];
#pragma unroll
            for (int e = 0; e < NF; ++e) Sf[e] = 0.0;
#pragma unroll
            for (int fi = 0; fi < 2 * NG; ++fi) {
                const int h = fi / NG, gi = fi - h * NG;
                const int lo_d = acc[gi][2 * h] - (gi + 1 < NG ? acc[gi + 1 < NG ? gi + 1 : gi][2 * h] : 0);
                const int hi_d = acc[gi][2 * h + 1] - (gi + 1 < NG ? acc[gi + 1 < NG ? gi + 1 : gi][2 * h + 1] : 0);
                // (exact: the differences are 2^(gi CB) times the group's digit sums)
                double v = ((double)(lo_d >> (gi * CB)) + 128.0 * (double)(hi_d >> (gi * CB))) * w0;
                v += __shfl_xor_sync(0xffffffffu, v, 1);
                v += __shfl_xor_sync(0xffffffffu, v, 2);
                if ((fi & 3) == tl) Sf[fi >> 2] = v;
            }
#pragma unroll
            for (int e = 0; e < NF; ++e) {
                if (have[e]) {
                    const float g = (float)(((double)lo_o[e] * lo_term + (double)st_o[e] * (delta_r * Sf[e])) * scale);
                    if (last && a.grad_out) { a.grad_out[jo[e]] = g; a.grad_out[n + jo[e]] = g; }
                    xo[e] = regularise(fmaf(-a.lr, g, xo[e]), xo[e], a.reg, a.reg_cst);
                    if (last) a.x[jo[e]] = xo[e];
                }
            }
            if (last) break;
            publish_w((int)((t_rel + 1) & 1));
            if (p == 0 && lane == 0) col_mark(a, t_rel, 5);
        }
    }
    // =================================================================================== R warps: residual digits
    else {
        const int rt = tid - 32 * kColWarpR0, rw = rt >> 5;
        int64_t q = 0;
        bool ok = true;                                  // (after a failure: as for the B warps)
        const double grow = a.reg == ZIPML_REG_LSSVM ? fmax(1.0, fabs(1.0 - (double)a.reg_cst)) : 1.0;
        const int zper = (a.bpad + G - 1) / G;           // rows of a dots buffer that this CTA clears
        for (int64_t t_rel = 0; t_rel < steps; ++t_rel) {
            const ColStep st = col_step(a, a.first_step + t_rel);
            const ColStepParams& sp = sh->sp[t_rel & 1];
            const long long* dots = a.dots + (size_t)(t_rel % 3) * 2 * a.bpad;
            // the step's largest |label| completes the bound of its residuals
            float bm = 0.0f;
            for (int k = rt; k < st.bt; k += kColRThreads) bm = fmaxf(bm, fabsf(__ldg(a.b + st.row0 + k)));
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) bm = fmaxf(bm, __shfl_xor_sync(0xffffffffu, bm, o));
            if (lane == 0) sh->red_f[1][rw] = bm;
            named_barrier(kColNamedR, kColRThreads);
            bm = fmaxf(fmaxf(sh->red_f[1][0], sh->red_f[1][1]), fmaxf(sh->red_f[1][2], sh->red_f[1][3]));
            const double rbound = (dbound + (double)bm) * 1.0001;
            const double inv_r = rbound > 0.0 ? (double)kColQmaxR / rbound : 0.0;
            const double U = sp.U;
            double rmax = 0.0;
            long long rs_hi = 0, rs_lo = 0;              // sum of the fixed-point residuals: high parts and low 28 bits
            for (int c = 0; c < st.nch; ++c, ++q) {
                const int rbuf = (int)(q & 1);
                // ---- all CTAs' parts of the chunk's dots have arrived
                if (rt == 0 && ok) {
                    const unsigned* cnt = a.count + (size_t)(q & (a.ring - 1)) * 32;
                    const unsigned target = (unsigned)((q / a.ring + 1) * G);
                    const long long t0 = clock64();
                    for (int spin = 0;; ++spin) {
                        unsigned v;
                        asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(cnt) : "memory");
                        if (v >= target) break;
                        if ((spin & 31) == 31) {
                            if (col_aborted(sh) || *reinterpret_cast<volatile int*>(&a.status->code) != 0) { sh->abort_flag = 1; break; }
                            if (clock64() - t0 > kColWaitCycles) { sh->abort_flag = 1; set_status(a.status, ZIPML_ERR_TIMEOUT, 75); break; }
                        }
                    }
                    if (c == 0) col_mark(a, t_rel, 7);
                    if (c == st.nch - 1) col_mark(a, t_rel, 2);
                }
                named_barrier(kColNamedR, kColRThreads);
                ok = ok && !col_aborted(sh);
                // every CTA has left step t - 1 behind: its dots buffer is cleared for step t + 2 (this CTA's
                // share; the stores precede this CTA's counter arrivals of step t + 1, which every adder waits for)
                if (c == 0 && ok) {
                    long long* z = a.dots + (size_t)((t_rel + 2) % 3) * 2 * a.bpad;
                    const int z0 = cta * zper, z1 = min(a.bpad, z0 + zper);
                    for (int i = z0 + rt; i < z1; i += kColRThreads) { z[i] = 0; z[a.bpad + i] = 0; }
                }
                if (ok && q >= 2) ok = col_wait(sh->rempty + rbuf, (uint32_t)(((q >> 1) - 1) & 1), sh, a.status, 76);
                signed char* rd = rdig + (size_t)rbuf * 2 * NRD * rstride;
                for (int kk = rt; kk < R && ok; kk += kColRThreads) {
                    const int k = c * R + kk;
                    long long R1 = 0, R2 = 0;
                    if (k < st.bt) {
                        const double bk = (double)__ldg(a.b + st.row0 + k);
                        const double r1 = (double)__ldcg(dots + k) * U - bk, r2 = (double)__ldcg(dots + a.bpad + k) * U - bk;
                        rmax = fmax(rmax, fmax(fabs(r1), fabs(r2)));
                        R1 = max(-kColQmaxR, min(kColQmaxR, __double2ll_rn(r1 * inv_r)));
                        R2 = max(-kColQmaxR, min(kColQmaxR, __double2ll_rn(r2 * inv_r)));
                        rs_hi += (R1 >> 28) + (R2 >> 28);
                        rs_lo += (R1 & 0xFFFFFFFll) + (R2 & 0xFFFFFFFll);
                    }
                    // row rho of a 32-row block sits where the transposed code fragments look for it:
                    // k index 4t + i <-> row 2t + (i & 1) + 8 (i >> 1), second half 16 rows further
                    const int rho = kk & 31, r16 = rho & 15;
                    signed char* dst = rd + (kk >> 5) * 32 + ((r16 & 7) >> 1) * 8 + (rho >> 4) * 4 + (r16 & 1) + 2 * (r16 >> 3);
                    long long W1 = R1, W2 = R2;
#pragma unroll
                    for (int s = 0; s < NRD; ++s) {
                        int d1, d2;
                        if (s < NRD - 1) {
                            d1 = (int)((W1 + 64) & 127) - 64; W1 = (W1 - d1) >> 7;
                            d2 = (int)((W2 + 64) & 127) - 64; W2 = (W2 - d2) >> 7;
                        } else { d1 = (int)W1; d2 = (int)W2; }
                        dst[(size_t)s * rstride] = (signed char)d2;                    // plane 1 meets r2
                        dst[(size_t)(NRD + s) * rstride] = (signed char)d1;            // plane 2 meets r1
                    }
                }
                if (c == st.nch - 1) {
                    // ---- the step's residuals are all known: their sum for the B warps, the next step's bound and unit
                    rmax = fmax(rmax, __shfl_xor_sync(0xffffffffu, rmax, 16));
#pragma unroll
                    for (int o = 8; o > 0; o >>= 1) rmax = fmax(rmax, __shfl_xor_sync(0xffffffffu, rmax, o));
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1) { rs_hi += __shfl_xor_sync(0xffffffffu, rs_hi, o); rs_lo += __shfl_xor_sync(0xffffffffu, rs_lo, o); }
                    if (lane == 0) { sh->red_d[1][rw] = rmax; sh->red_l[0][rw] = rs_hi; sh->red_l[1][rw] = rs_lo; }
                    named_barrier(kColNamedR, kColRThreads);
                    double rm = 0.0;
                    long long hi = 0, lo = 0;
#pragma unroll
                    for (int w = 0; w < kColRWarps; ++w) { rm = fmax(rm, sh->red_d[1][w]); hi += sh->red_l[0][w]; lo += sh->red_l[1][w]; }
                    dbound = (dbound * grow + fabs((double)a.lr) * rm * c2) * 1.0001;
                    if (rt == 0) {
                        ColStepParams& cur = sh->sp[t_rel & 1];
                        cur.inv_r = inv_r;
                        cur.delta_r = rbound / (double)kColQmaxR;
                        cur.rsum = (double)hi * 268435456.0 + (double)lo;
                        unit_of(dbound, sh->sp[(t_rel + 1) & 1].U, sh->sp[(t_rel + 1) & 1].invU);
                    }
                    named_barrier(kColNamedR, kColRThreads);       // (red_* free again; the parameters precede the arrivals)
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(reinterpret_cast<uint64_t*>(sh->rfull + rbuf));
                if (rt == 0 && c == st.nch - 1) col_mark(a, t_rel, 3);
            }
        }
    }
    __syncthreads();
}

// ---------------------------------------------------------------------------------------------
// Host side
// ---------------------------------------------------------------------------------------------
static const void* column_kernel_ptr(int cb) {
    if (cb == 2) return reinterpret_cast<const void*>(&sgd_column_kernel<2>);
    if (cb == 4) return reinterpret_cast<const void*>(&sgd_column_kernel<4>);
    return reinterpret_cast<const void*>(&sgd_column_kernel<8>);
}

// Tensor maps over the two planes as m x row_bytes byte matrices: boxes of 128 bytes x R rows with the
// 128-byte swizzle, bytes past the row or the last row read as zero.  The encoder is a driver entry
// point looked up through the runtime (no link against the driver library).
static int encode_column_maps(zipml_ctx* ctx, const zipml_dataset* d, int R, CUtensorMap* out) {
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
    const cuuint64_t gdim[2] = {(cuuint64_t)d->row_bytes, (cuuint64_t)d->m};
    const cuuint64_t gstride[1] = {(cuuint64_t)d->row_bytes};
    const cuuint32_t box[2] = {(cuuint32_t)kColBlockBytes, (cuuint32_t)R};
    const cuuint32_t estr[2] = {1, 1};
    const void* planes[2] = {d->plane1, d->plane2};
    for (int i = 0; i < 2; ++i) {
        const CUresult r = reinterpret_cast<EncodeFn>(ctx->tmap_encode)(
            &out[i], CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(planes[i]), gdim, gstride, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) return ZIPML_ERR_CUDA;
    }
    return ZIPML_OK;
}

int launch_sgd_column(zipml_ctx* ctx, const zipml_dataset* d, const float* b, float* x, const zipml_sgd_params* p,
                      int64_t first_step, int64_t num_steps, float* grad_out, bool only_if_profitable) {
    if (!ctx->cooperative) return ZIPML_ERR_WORKSPACE;
    if (d->level_mode != ZIPML_LEVELS_UNIFORM || p->model_bits != 0 || p->grad_bits != 0 || p->model_out) return ZIPML_ERR_WORKSPACE;
    if (d->m > 0x7fffffffLL || d->row_bytes < kColBlockBytes) return ZIPML_ERR_WORKSPACE;
    const int cb = container_bits(d->bits);
    const int ng = 8 / cb;
    const int64_t T = (d->m + p->batch - 1) / p->batch;
    const int64_t B = p->batch < d->m ? p->batch : d->m;
    if (B > kColMaxBatch) return ZIPML_ERR_WORKSPACE;
    const int64_t G = (d->row_bytes + kColBlockBytes - 1) / kColBlockBytes;
    if (G > ctx->sm_count) return ZIPML_ERR_WORKSPACE;                 // one CTA per SM, all resident at once
    // worth it where the rows occupy most of the device and a step holds several chunks
    if (only_if_profitable && (G < ctx->sm_count / 2 || B < 256)) return ZIPML_ERR_WORKSPACE;
    int R = p->column_chunk_rows > 0 ? p->column_chunk_rows : 128;
    if (R > (B + 31) / 32 * 32) R = (int)((B + 31) / 32 * 32);
    const int nch_max = (int)((B + R - 1) / R);
    const int bpad = nch_max * R;
    int ring = 16;
    while (ring < 2 * nch_max + 2 * kColMaxSlots) ring *= 2;

    const size_t slot_bytes = (size_t)2 * R * kColBlockBytes;
    const size_t fixed = 1024 + (size_t)2 * 2 * kColRDigits * (R + 32) + (size_t)ng * 4 * 4 * 32 + 16 + sizeof(ColShared);
    if (fixed + 2 * slot_bytes > (size_t)ctx->smem_optin) return ZIPML_ERR_WORKSPACE;
    int slots = (int)(((size_t)ctx->smem_optin - fixed) / slot_bytes);
    if (slots > kColMaxSlots) slots = kColMaxSlots;
    const size_t smem = fixed + (size_t)slots * slot_bytes;
    const void* kernel = column_kernel_ptr(cb);
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return cuda_status(e);
    int per_sm = 0;
    e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, kColThreads, smem);
    if (e != cudaSuccess) return cuda_status(e);
    if (per_sm < 1 || G > (int64_t)per_sm * ctx->sm_count) return ZIPML_ERR_WORKSPACE;

    CUtensorMap tmaps[2];
    int rc = encode_column_maps(ctx, d, R, tmaps);
    if (rc != ZIPML_OK) return rc;

    size_t off = 0;
    auto piece = [&](size_t bytes) { const size_t o = off; off += carve_size(bytes); return o; };
    const size_t o_count = piece(sizeof(unsigned) * 32 * (size_t)ring);
    const size_t o_dots = piece(sizeof(long long) * 3 * 2 * (size_t)bpad);
    const size_t zero_bytes = off;
    const size_t o_ord = piece(sizeof(int32_t) * (size_t)(p->batch_order ? T : 0));
    rc = ws_reserve(ctx, off);
    if (rc != ZIPML_OK) return rc;

    ColumnArgs a;
    memset(&a, 0, sizeof(a));
    a.m = d->m; a.batch = B; a.lo = d->feat_lo; a.step = d->feat_step; a.b = b; a.x = x; a.grad_out = grad_out;
    a.n = (int)d->n; a.bits = d->bits; a.R = R; a.slots = slots; a.bpad = bpad; a.ring = ring;
    a.lr = p->lr; a.reg = p->reg; a.reg_cst = reg_constant(p);
    a.count = reinterpret_cast<unsigned*>(ctx->ws + o_count);
    a.dots = reinterpret_cast<long long*>(ctx->ws + o_dots);
    a.status = ctx->d_status;
    a.trace = reinterpret_cast<unsigned long long*>(p->trace);
    a.trace_steps = p->trace ? p->trace_steps : 0;
    if (p->batch_order) {
        int32_t* dev_order = reinterpret_cast<int32_t*>(ctx->ws + o_ord);
        e = cudaMemcpyAsync(dev_order, p->batch_order, sizeof(int32_t) * (size_t)T, cudaMemcpyHostToDevice, ctx->stream);
        if (e != cudaSuccess) return cuda_status(e);
        a.order = dev_order;
    }
    // the chunk counters are 32-bit: (chunks of a launch / ring + 1) * G must stay below 2^31
    const int64_t max_steps = ((int64_t)(0x7fffffff / G) - 2) * ring / nch_max;
    for (int64_t s0 = first_step; s0 < first_step + num_steps; s0 += max_steps) {
        e = cudaMemsetAsync(ctx->ws, 0, zero_bytes, ctx->stream);
        if (e != cudaSuccess) return cuda_status(e);
        ColumnArgs chunk = a;
        chunk.first_step = s0;
        chunk.num_steps = (first_step + num_steps - s0 < max_steps) ? first_step + num_steps - s0 : max_steps;
        if (s0 + chunk.num_steps < first_step + num_steps) chunk.grad_out = nullptr;
        if (s0 > first_step) { chunk.trace = nullptr; chunk.trace_steps = 0; }
        void* params[] = {&chunk, &tmaps[0], &tmaps[1]};
        e = cudaLaunchCooperativeKernel(kernel, dim3((unsigned)G), dim3(kColThreads), params, smem, ctx->stream);
        if (e != cudaSuccess) return cuda_status(e);
        ctx->launches += 1;
    }
    ctx->last_engine = ZIPML_ENGINE_COLUMN;
    return ZIPML_OK;
}

}  // namespace zipml
