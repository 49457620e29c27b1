// Column engine of zipml_sgd_epoch: large minibatch tiles on uniform grids, fp32 model and gradient,
// every code byte read from HBM exactly once per step, no grid-wide barrier.
//
// A step of the double-sampled minibatch SGD (paper Eq. (double) in its symmetrised form, footnote of
// "Double Sampling"; update in full precision, "End-to-end Quantization") needs the step's code tile
// twice: for the dots q1^T x, q2^T x of every row, and, once the residuals r = dot - b are known, for
// the gradient 1/(2B) sum_k [q1_k r2_k + q2_k r1_k].  Here the features are partitioned: CTA j owns
// the 128-byte column block j of the packed rows (1024 / CB features) for all rows and the whole
// launch, so its slice of the model, of w = step * x and of the gradient never leave the CTA, and the
// only thing CTAs exchange is the rows' dots.  Rows travel in chunks of R rows (both planes, R x 128
// bytes each, one 2-D tensor copy per plane with the 128-byte swizzle).  A chunk comes into shared memory
// twice: from HBM for its dots, and again -- out of L2, where the first copy left it a few microseconds
// earlier -- when its residuals are known.  Between the two visits it occupies no shared memory, so the
// exchange of its dots (several L2 round trips under load) may take as long as it likes without holding
// the stream up:
//
//   service   (2 warps)  lane 0 of each: tensor copies into a ring of slots, "A" (first visit, ahead of the A
//                        warps, across step boundaries: codes do not depend on the model) for warp 0, "B"
//                        (second visit, in the same order, as far ahead of the B warps as that ring allows) for
//                        the last warp; each sleeps on its ring's barrier
//   A warps   (8)        partial dots of the chunk on the int8 tensor cores (mma.sync m16n8k32, u8 codes x
//                        s8 digits of w), converted to a fixed-point unit common to all CTAs and added to
//                        the row's word with one 64-bit integer atomic, whose low byte counts the CTAs
//   R warps   (4)        poll a chunk's words until their counts are complete, read the labels, turn the
//                        residuals into eight balanced base-256 int8 digits; each warp takes every fourth
//                        chunk, so four exchanges are in flight at a time
//   B warps   (8)        gradient of the CTA's own features (transposing ldmatrix, residual digits as the
//                        other operand), accumulated in registers over the step; at the step's end: update
//                        of the own slice of x, digits of the next w
//
// A word is its own flag (sum in the upper 56 bits, count below), so there is no counter and no barrier
// between CTAs.  At a step's end the pipeline drains (the next dots need the whole new w of the CTA) while
// the A ring fills with the next step's first chunks.  The CTAs may be split into groups with a word each per
// row (same-address atomics are served one after the other), but one word for all measured fastest.
//
// Fixed point.  Dots: every CTA adds its part as a multiple of U = 2^e / 2^52 where 2^e > D, and D bounds
// every |dot| of the step: D(0) = sum_j |x_j| amax_j from the caller's model, D(t+1) = grow * D(t) +
// lr * rmax(t) * sum_j amax_j^2 (amax_j the largest |value| of feature j, rmax(t) the step's largest
// |residual|, which every CTA reads off the same words): every CTA derives the same U without asking
// anyone, sums of multiples of U are exact and order-free, and the bound may be loose by 2^21 before 2^-31
// relative precision is touched.  w of the own features: four digits (27 bits) whose unit is U times a power
// of two, at most twice what the CTA's own max |w| needs, so that a digit sum becomes a multiple of U by a
// shift; the own part of lo^T x is rounded to a multiple of U once per step: the path from the tensor-core
// sums to the atomic is integer arithmetic only.  Residuals: eight digits (55 bits) whose unit is a power of two
// as well, at most twice what D(t) + max |b| of the step needs, so that a dot becomes a residual by a shift and
// the label's fixed-point value (one conversion per row); all eight columns of the tensor-core tile carry a digit.  Digits are balanced
// and found without a carry chain: with half the base added to every digit the number is plain base 128 (w,
// -64..63) or plain base 256 (residuals, -128..127: the digits are the number's own bytes, xor 0x80).
// Results do not depend on timing: every sum is an integer sum or has a fixed order.
//
// The machine code is kept small on purpose (four roles share the instruction cache): 32-bit counters kept up
// step by step instead of 64-bit divisions, waits as functions with one copy, loops unrolled only where
// registers demand it.  Measured on 65,536 x 32,768 4-bit rows, B = 2,048: 23.0 us per step (stream engine:
// 29.8), DRAM reads 1.00 x the packed bytes.  Not HBM bounds it but the chain of a step: the first chunk's dots
// have to cross L2 and become digits before pass B can start, pass B (about 1.2 k cycles per chunk on its own, 2 k
// while pass A runs beside it) ends about 9 k cycles after pass A, and the next step's first dots come 5 k cycles
// after the last chunk's gradient.  The SM issues about two instructions per cycle in every variant tried, so a
// role given more warps slows the others by as much; what helped was taking instructions and tests out of the
// loops and keeping the R warps from waiting for pass B (two digit buffers each).
//
// Memory order.  A buffer of dot words serves every third step and is cleared in between by the R warp that
// has seen the first chunk of step t complete (then every CTA has left step t-1, the buffer's last use,
// behind: hence its fence before the stores), once that chunk's digits are out; the A warps fence once per step before their first
// addition, so that whoever sees a CTA's additions of step t+1 -- which every adder of step t+2 has -- also
// sees its cleared share.
#include <cuda.h>
#include <string.h>

#include <type_traits>

#include "int_digits.cuh"
#include "sgd_common.cuh"

namespace zipml {

constexpr int kColAWarps = 8, kColBWarps = 8, kColRWarps = 4;
// Digit buffers: two per R warp (chunk q goes to buffer q mod kColRBufs), so that a warp can write its next chunk's
// digits while pass B still reads its previous ones.
constexpr int kColRBufs = 2 * kColRWarps, kColRBufShift = 3;                        // (kColRBufs = 2^kColRBufShift)
constexpr int kColWarpA0 = 1, kColWarpB0 = kColWarpA0 + kColAWarps, kColWarpR0 = kColWarpB0 + kColBWarps;
constexpr int kColWarpS2 = kColWarpR0 + kColRWarps;             // the second service warp (second visits)
constexpr int kColThreads = 32 * (kColWarpS2 + 1);
constexpr int kColRThreads = 32 * kColRWarps;
constexpr int kColBThreads = 32 * kColBWarps;
constexpr int kColBlockBytes = 128;         // bytes of a packed row that a CTA owns
constexpr int kColMaxBatch = 8192;
constexpr int kColMaxSlots = 16;            // per ring
constexpr int kColMaxChunkRows = 128;       // a lane of an R warp takes four rows of a chunk
constexpr int kColMaxGroups = 4;            // words per row and plane
constexpr int kColRDigits = 8;              // digits of a residual
constexpr long long kColQmaxR = 35000000000000000LL;     // below 2^55: eight balanced base-256 digits hold it with room
// Residual digits are balanced base-256 digits (-128..127), found without a carry chain: with 128 added to every digit
// the number is plain base 256, i.e. the bytes of R + bias; a byte xor 0x80 is the digit as a signed byte.
constexpr unsigned long long kColBiasR = 0x8080808080808080ull;
constexpr int kColBiasW = 64 * 2113665;                      // 64 * (128^4 - 1) / 127
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
    int slots_a, slots_b;    // slots of the two rings
    int bpad;                // rows of a buffer of dot words: chunks of the largest step * R
    int ngrp, gsize;         // groups of CTAs with a dot word each per row and plane; CTAs per group
    int blocked;             // the planes are in the column-block layout: a CTA's pieces of consecutive rows are contiguous
    float lr;
    int reg;
    float reg_cst;
    long long* dots;         // [3][ngrp][2][bpad] three steps in rotation, zeroed before the launch; a word holds the
                             // fixed-point sum in its upper 56 bits and the number of CTAs that added in its low byte
    DeviceStatus* status;
    unsigned long long* trace;
    int trace_steps;
};

struct ColStepParams {       // by step parity
    double U, invU;          // fixed-point unit of the dots                     (R warps -> A, R warps)
    long long bint;          // own part of lo^T x in units of U                 (B warps -> A warps)
    int kshift;              // the unit of the own w digits is U * 2^kshift     (B warps -> A warps)
    double inv_r, delta_r;   // fixed point of the residuals                     (R warps -> B warps)
    double rsum;             // sum of all fixed-point residuals of the step     (R warps -> B warps)
};

struct ColShared {
    unsigned long long full_a[kColMaxSlots], empty_a[kColMaxSlots];     // A ring: copies landed / the A warps are done
    unsigned long long full_b[kColMaxSlots], empty_b[kColMaxSlots];     // B ring: copies landed / the B warps are done
    unsigned long long rfull[kColRBufs], rempty[kColRBufs];     // residual digits of a chunk (buffer q mod kColRBufs): written / consumed
    int w_version;                             // steps (+1) whose digits of w are in place
    ColStepParams sp[2];
    double red_d[2][32];
    float red_f[2][32];
    long long red_l[2][kColRWarps];
    int abort_flag;
    int qa_issued;                             // chunks whose first copy has been issued
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

// try_wait that lets the hardware park the thread for up to about a microsecond: a warp that waits should not
// take issue slots from the warps that work.
__device__ __forceinline__ bool mbar_try_wait_parked(unsigned long long* bar, uint32_t parity) {
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done) : "r"(smem_u32(bar)), "r"(parity), "r"(1000u) : "memory");
    return done != 0;
}

// Bounded wait on a local mbarrier phase.  False once this CTA has given up anywhere.  (Not inlined: one copy.)
__device__ __noinline__ bool col_wait(unsigned long long* bar, uint32_t parity, ColShared* sh, DeviceStatus* status, int where) {
    if (mbar_test_wait(bar, parity)) return true;
    if (col_aborted(sh)) return false;
    const long long t0 = clock64();
#pragma unroll 1
    for (int spin = 0;; ++spin) {
        if (mbar_try_wait_parked(bar, parity)) return true;
        if (spin >= 4) __nanosleep(spin < 16 ? 200 : 800);       // a warp that waits long should stay out of the others' way
        if ((spin & 15) == 15) {
            if (col_aborted(sh)) return false;
            if (clock64() - t0 > kColWaitCycles) break;
        }
    }
    sh->abort_flag = 1;
    set_status(status, ZIPML_ERR_TIMEOUT, where);
    return false;
}

// Addition to a word in global memory that returns nothing: fire and forget.  (atomicAdd on a generic pointer
// compiled to an atomic that brings the old value back, and the warp waited an L2 round trip for a register
// it never read: 5.6 k cycles per 32-row task instead of a few hundred.)
__device__ __forceinline__ void red_add_u64(long long* p, unsigned long long v) {
    asm volatile("red.relaxed.gpu.global.add.u64 [%0], %1;" ::"l"(__cvta_generic_to_global(p)), "l"(v) : "memory");
}

// Polling load of two neighbouring words straight from L2 (16-byte aligned).
__device__ __forceinline__ void ld_l2_v2(const long long* p, long long& v0, long long& v1) {
    asm volatile("ld.global.cg.v2.s64 {%0, %1}, [%2];" : "=l"(v0), "=l"(v1) : "l"(p) : "memory");
}

__device__ __forceinline__ void st_release_cta(int* p, int v) {
    asm volatile("st.release.cta.shared.s32 [%0], %1;" ::"r"(smem_u32(p)), "r"(v) : "memory");
}
__device__ __forceinline__ int ld_acquire_cta(const int* p) {
    int v;
    asm volatile("ld.acquire.cta.shared.s32 %0, [%1];" : "=r"(v) : "r"(smem_u32(p)) : "memory");
    return v;
}

// Bounded wait until a version count in shared memory has reached `want`.
__device__ __noinline__ bool col_wait_version(const int* version, int want, ColShared* sh, DeviceStatus* status, int where) {
    const long long t0 = clock64();
#pragma unroll 1
    for (int spin = 0; ld_acquire_cta(version) < want; ++spin) {
        __nanosleep(400);
        if ((spin & 15) == 15) {
            if (col_aborted(sh)) return false;
            if (clock64() - t0 > kColWaitCycles) { sh->abort_flag = 1; set_status(status, ZIPML_ERR_TIMEOUT, where); return false; }
        }
    }
    return true;
}

// Powers of two by their exponent fields (no library call: the code must stay small).
__device__ __forceinline__ int col_exponent(double v) { return (int)((__double_as_longlong(v) >> 52) & 0x7FF) - 1023; }     // v < 2^(e + 1)
__device__ __forceinline__ double col_pow2(int e) { return __longlong_as_double((long long)(min(1000, max(-1000, e)) + 1023) << 52); }

// The fixed-point unit of the dots for a bound of their size: 2^e / 2^52 with bound < 2^e.
__device__ __forceinline__ void col_unit_of(double bound, double& U, double& invU) {
    const int ex = max(-900, min(900, col_exponent(bound) + 1));
    U = col_pow2(ex - 52);
    invU = col_pow2(52 - ex);
}

__device__ __forceinline__ void named_barrier(int id, int threads) { asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory"); }

__device__ __forceinline__ void tensor_load_2d(void* dst_smem, const CUtensorMap* tm, int x, int y, unsigned long long* bar) {
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                 ::"r"(smem_u32(dst_smem)), "l"(tm), "r"(x), "r"(y), "r"(smem_u32(bar)) : "memory");
}
// The same with an L2 eviction policy for the lines it reads.
__device__ __forceinline__ void tensor_load_2d_hint(void* dst_smem, const CUtensorMap* tm, int x, int y, unsigned long long* bar, uint64_t policy) {
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%2, %3}], [%4], %5;"
                 ::"r"(smem_u32(dst_smem)), "l"(tm), "r"(x), "r"(y), "r"(smem_u32(bar)), "l"(policy) : "memory");
}

__device__ __forceinline__ void col_mark(const ColumnArgs& a, int64_t t_rel, int k) {
    if (a.trace && blockIdx.x == 0 && t_rel < a.trace_steps) a.trace[t_rel * 8 + k] = (unsigned long long)clock64();
}
// Adds `cycles` to slot k of the step's trace record (one writer per slot).
__device__ __forceinline__ void col_tally(const ColumnArgs& a, int64_t t_rel, int k, long long cycles) {
    if (a.trace && blockIdx.x == 0 && t_rel < a.trace_steps) a.trace[t_rel * 8 + k] += (unsigned long long)cycles;
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

// A position in a ring of slots: slot index and the parity of the number of times the ring has wrapped.
struct ColRing {
    int slot;
    uint32_t phase;
    __device__ __forceinline__ void next(int slots) { if (++slot == slots) { slot = 0; phase ^= 1u; } }
};

// The kernel's machine code must stay small: four roles run side by side, and once their loops do not fit the
// instruction cache together every warp waits for its next instructions (a first version of 96 KB spent more
// time there than anywhere else).  Hence: 32-bit counters kept up step by step instead of 64-bit divisions,
// waits and helpers as functions with one copy, loops unrolled only where registers demand it.
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
    // [A slots + B slots][2 planes][R rows][128 B] (1024-byte aligned), then the digit operands, then the bookkeeping
    unsigned char* tiles = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const int R = a.R;
    const uint32_t plane_bytes = (uint32_t)R * kColBlockBytes, slot_bytes = 2u * plane_bytes;
    unsigned char* tiles_b = tiles + (size_t)a.slots_a * slot_bytes;
    const int rstride = R + 32;                        // bytes between the residual digit vectors
    signed char* rdig = reinterpret_cast<signed char*>(tiles_b + (size_t)a.slots_b * slot_bytes);  // [R warps][2 operands][8 digits][rstride]
    signed char* wdig = rdig + (size_t)kColRBufs * 2 * NRD * rstride;                             // [NG][4 k-blocks][8 columns: 4 digits, 4 x zero][32 B]
    // the A warps' hand-over of a task's digit sums from the lanes that hold them to a lane per row ([A warps][2 planes][32 rows][2])
    int* ascr = reinterpret_cast<int*>((reinterpret_cast<uintptr_t>(wdig + NG * 4 * 8 * 32) + 15) & ~(uintptr_t)15);
    ColShared* sh = reinterpret_cast<ColShared*>(ascr + (size_t)kColAWarps * 2 * 32 * 2);

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, gl = lane >> 2, tl = lane & 3;
    const int cta = blockIdx.x, G = gridDim.x;
    const int n = a.n;
    const int steps = (int)a.num_steps;
    const int64_t byte0 = (int64_t)cta * kColBlockBytes;          // first byte of the own column block
    // tensor-copy coordinates of row 0 of the own block (rows past the step's last one come along and meet zero digits)
    const int x_own = a.blocked ? 0 : (int)byte0;
    const int64_t y_own = a.blocked ? (int64_t)cta * a.m : 0;

    for (int i = tid; i < NG * 4 * 8 * 32 / 4; i += kColThreads) reinterpret_cast<uint32_t*>(wdig)[i] = 0u;     // (digit columns 4..7 stay zero)
    if (tid == 0) {
        for (int s = 0; s < kColMaxSlots; ++s) {
            mbar_init(reinterpret_cast<uint64_t*>(sh->full_a + s), 1);
            mbar_init(reinterpret_cast<uint64_t*>(sh->empty_a + s), a.R / 32);     // one arrival per 32-row task
            mbar_init(reinterpret_cast<uint64_t*>(sh->full_b + s), 1);
            mbar_init(reinterpret_cast<uint64_t*>(sh->empty_b + s), kColBWarps);
        }
        for (int s = 0; s < kColRBufs; ++s) {
            mbar_init(reinterpret_cast<uint64_t*>(sh->rfull + s), 1);
            mbar_init(reinterpret_cast<uint64_t*>(sh->rempty + s), kColBWarps);
        }
        sh->w_version = 0;
        sh->abort_flag = 0;
        sh->qa_issued = 0;
        mbar_fence_init();
    }
    // ---- every CTA scans the model once, with the same arithmetic: the bound of the dots and its growth rate
    const float smax = (float)((1 << a.bits) - 1);
    double dsum = 0.0, csum = 0.0;
#pragma unroll 1
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
#pragma unroll 1
    for (int w = 0; w < kColThreads / 32; ++w) { dbound += sh->red_d[0][w]; c2 += sh->red_d[1][w]; }
    dbound *= 1.0001;
    if (tid == 0) col_unit_of(dbound, sh->sp[0].U, sh->sp[0].invU);
    __syncthreads();                                      // barriers initialised, sums read, U(0) in place

    // =================================================================================== service warps
    // One lane each.  Warp 0, first visits: the next chunk as soon as a slot of the A ring is free.  The last warp, second
    // visits: the next chunk that has had its first copy issued (it is in L2 or on its way there), as soon as a slot of
    // the B ring is free.  Each sleeps on its ring's barrier and is woken by the release itself: a shared loop that
    // looked at both rings in turn, with pauses, let a freed slot wait several hundred cycles for its next copy.
    if (warp == 0 || warp == kColWarpS2) {
        if (lane == 0) {
            const bool first_visit = warp == 0;
            unsigned long long* full = first_visit ? sh->full_a : sh->full_b;
            unsigned long long* empty = first_visit ? sh->empty_a : sh->empty_b;
            unsigned char* base = first_visit ? tiles : tiles_b;
            const int nslots = first_visit ? a.slots_a : a.slots_b;
            int q = 0, t = 0, c = 0;
            ColRing ring{0, 0u};
            ColStep st = col_step(a, a.first_step);
            uint64_t evict_first;
            asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(evict_first));
            bool ok = true;
#pragma unroll 1
            while (ok && t < steps) {
                if (q >= nslots) ok = col_wait(empty + ring.slot, ring.phase ^ 1u, sh, a.status, 70);
                if (ok && !first_visit) {
                    const long long t0 = clock64();
#pragma unroll 1
                    for (int spin = 0; *reinterpret_cast<volatile int*>(&sh->qa_issued) <= q; ++spin) {
                        __nanosleep(50);
                        if ((spin & 63) == 63 && (col_aborted(sh) || clock64() - t0 > kColWaitCycles)) {
                            if (!col_aborted(sh)) { sh->abort_flag = 1; set_status(a.status, ZIPML_ERR_TIMEOUT, 78); }
                            ok = false;
                            break;
                        }
                    }
                }
                if (!ok) break;
                unsigned char* dst = base + (size_t)ring.slot * slot_bytes;
                mbar_arrive_expect_tx(reinterpret_cast<uint64_t*>(full + ring.slot), slot_bytes);
                const int y = (int)(y_own + st.row0 + (int64_t)c * R);
                if (first_visit) {
                    tensor_load_2d(dst, &tm1, x_own, y, full + ring.slot);
                    tensor_load_2d(dst + plane_bytes, &tm2, x_own, y, full + ring.slot);
                    *reinterpret_cast<volatile int*>(&sh->qa_issued) = q + 1;
                } else {
                    // (nobody reads these lines again this epoch: they may leave L2 ahead of the rest)
                    tensor_load_2d_hint(dst, &tm1, x_own, y, full + ring.slot, evict_first);
                    tensor_load_2d_hint(dst + plane_bytes, &tm2, x_own, y, full + ring.slot, evict_first);
                }
                ++q;
                ring.next(nslots);
                if (++c == st.nch) { c = 0; if (++t < steps) st = col_step(a, a.first_step + t); }
            }
            if (!ok) {
                // leaving early: the copies in flight must land before the CTA's shared memory goes away
                const long long t0 = clock64();
#pragma unroll 1
                for (int s = 0; s < kColMaxSlots; ++s) {
                    if (s < nslots && s < q) {
                        const uint32_t par = (uint32_t)((((q - 1 - ((q - 1 - s + nslots) % nslots)) / nslots)) & 1);
                        while (!mbar_test_wait(full + s, par) && clock64() - t0 < kColWaitCycles) {}
                    }
                }
            }
        }
    }
    // =================================================================================== A warps: dots
    else if (warp < kColWarpB0) {
        // A task is 32 rows of a chunk (two 16-row tiles, interleaved); the tasks of the launch's chunk sequence are
        // dealt to the eight warps in turn, so that several chunks are worked on at a time.
        const int aw = warp - kColWarpA0;
        constexpr uint32_t kLow = CB == 8 ? 0xFFFFFFFFu : CB == 4 ? 0x0F0F0F0Fu : 0x03030303u;
        // ldmatrix row addresses: lane l gives row (l & 7) + 8 * ((l >> 3) & 1) of the 16-row block and the
        // 16-byte piece (l >> 4) of a 32-byte k-block; the 128-byte swizzle moves piece c of row r to c ^ (r & 7)
        const uint32_t a_row = (uint32_t)((lane & 7) + 8 * ((lane >> 3) & 1)), a_piece = (uint32_t)(lane >> 4), a_x = (uint32_t)(lane & 7);
        const uint32_t wdig_lane = smem_u32(wdig) + (uint32_t)(gl * 32 + tl * 8);          // lanes with gl < 4 read digit gl
        const int grp = cta / a.gsize;
        const int tpc = R / 32;                          // tasks per chunk
        int t_rel = 0, c = 0, j = aw;                    // the current task: step, chunk of the step, task of the chunk
        ColRing ring{0, 0u};                             // the chunk's slot
        ColStep st = col_step(a, a.first_step);
        bool fresh = true, ok = true;                    // fresh: the step's parameters are still to be fetched
        int kshift = 0;
        long long bint = 0;
        long long* dots = a.dots;
#pragma unroll 1
        while (ok) {
#pragma unroll 1
            while (j >= tpc && t_rel < steps) {          // on to the task's chunk
                j -= tpc;
                ring.next(a.slots_a);
                if (++c == st.nch) {
                    c = 0;
                    fresh = true;
                    if (++t_rel < steps) st = col_step(a, a.first_step + t_rel);
                }
            }
            if (t_rel >= steps) break;
            if (fresh) {
                // the digits of this step's w (a version count, not a phase: a warp without a task in some step
                // never looks at that step's digits)
                ok = __all_sync(0xffffffffu, col_wait_version(&sh->w_version, t_rel + 1, sh, a.status, 71));     // (the warp acts as one)
                if (!ok) break;
                __threadfence();        // (see "Memory order" above: the cleared words before this step's additions)
                const ColStepParams& sp = sh->sp[t_rel & 1];
                kshift = sp.kshift; bint = sp.bint;
                dots = a.dots + ((size_t)(t_rel % 3) * a.ngrp + grp) * 2 * a.bpad;
                fresh = false;
                if (lane == 0 && c == 0 && j == 0) col_mark(a, t_rel, 0);
            }
            const long long w0c = (a.trace && aw == 0) ? clock64() : 0;
            if (!__all_sync(0xffffffffu, mbar_test_wait(sh->full_a + ring.slot, ring.phase))) {      // (usually there already)
                ok = __all_sync(0xffffffffu, col_wait(sh->full_a + ring.slot, ring.phase, sh, a.status, 72));
                if (!ok) break;
            }
            if (a.trace && aw == 0 && lane == 0) col_tally(a, t_rel, 1, clock64() - w0c);
            const uint32_t tile = smem_u32(tiles) + (uint32_t)ring.slot * slot_bytes;
            const int k0 = c * R + j * 32;                                // first row of the task within the step
            if (k0 < st.bt) {
                int c1[2][NG][4], c2[2][NG][4];                          // [tile][group][fragment]: plane 1, plane 2
                const uint32_t row_addr = tile + (uint32_t)(j * 32 + a_row) * kColBlockBytes;
                // one 32-byte k-block of the two tiles and planes; the first one starts the sums (no cleared registers)
                auto kblock = [&](int kb, auto first) {
                    uint32_t f1[2][4], f2[2][4];
                    const uint32_t off = row_addr + (((uint32_t)(2 * kb) + a_piece) ^ a_x) * 16u;
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        ldsm_x4(f1[h], off + (uint32_t)h * 16u * kColBlockBytes);
                        ldsm_x4(f2[h], off + (uint32_t)h * 16u * kColBlockBytes + plane_bytes);
                    }
#pragma unroll
                    for (int g = 0; g < NG; ++g) {
                        uint32_t b0, b1;                         // (columns 4..7 of the operand are zeros that stay in place)
                        asm volatile("ld.shared.v2.u32 {%0, %1}, [%2];" : "=r"(b0), "=r"(b1) : "r"(wdig_lane + (uint32_t)((g * 4 + kb) * 8 * 32)));
                        // group g's codes stay where they are in the byte: its sums come out 2^(g CB) times too large
                        const uint32_t mk = kLow << (g * CB);
#pragma unroll
                        for (int h = 0; h < 2; ++h) {
                            if constexpr (decltype(first)::value) {
                                mma_u8s8_first(c1[h][g], f1[h][0] & mk, f1[h][1] & mk, f1[h][2] & mk, f1[h][3] & mk, b0, b1);
                                mma_u8s8_first(c2[h][g], f2[h][0] & mk, f2[h][1] & mk, f2[h][2] & mk, f2[h][3] & mk, b0, b1);
                            } else {
                                mma_u8s8(c1[h][g], f1[h][0] & mk, f1[h][1] & mk, f1[h][2] & mk, f1[h][3] & mk, b0, b1);
                                mma_u8s8(c2[h][g], f2[h][0] & mk, f2[h][1] & mk, f2[h][2] & mk, f2[h][3] & mk, b0, b1);
                            }
                        }
                    }
                };
                kblock(0, std::true_type{});
#pragma unroll 1
                for (int kb = 1; kb < 4; ++kb) kblock(kb, std::false_type{});      // (unrolled it was no faster: more machine code)
                // lane t < 2 holds digits 2t, 2t+1 of rows g (c[0], c[1]) and g+8 (c[2], c[3]) of each tile.  Integers all
                // the way: the groups' sums (multiples of 2^(g CB), shifted back exactly) and two digits per lane in
                // 32 bits; through a few words of shared memory every lane then takes one row: the two lanes' pairs
                // in 64 bits, the shift into the dots' unit, the own part of lo^T x, and one addition per plane whose
                // 32 lanes cover 256 consecutive bytes (the fewer and wider the requests, the sooner L2 is through
                // with a chunk's additions).
                int* as = ascr + (size_t)aw * 2 * 32 * 2;
#pragma unroll
                for (int h = 0; h < 2; ++h)
#pragma unroll
                    for (int e = 0; e < 2; ++e) {
                        int x10 = 0, x11 = 0, x20 = 0, x21 = 0;
#pragma unroll
                        for (int g = 0; g < NG; ++g) {
                            x10 += c1[h][g][2 * e] >> (g * CB); x11 += c1[h][g][2 * e + 1] >> (g * CB);
                            x20 += c2[h][g][2 * e] >> (g * CB); x21 += c2[h][g][2 * e + 1] >> (g * CB);
                        }
                        if (tl < 2) {
                            const int row = 16 * h + 8 * e + gl;
                            as[row * 2 + tl] = x10 + (x11 << 7);
                            as[64 + row * 2 + tl] = x20 + (x21 << 7);
                        }
                    }
                __syncwarp();
                {
                    const int2 p1 = *reinterpret_cast<const int2*>(as + 2 * lane), p2 = *reinterpret_cast<const int2*>(as + 64 + 2 * lane);
                    const long long v1 = (long long)p1.x + ((long long)p1.y << 14), v2 = (long long)p2.x + ((long long)p2.y << 14);
                    const int k = k0 + lane;
                    if (k < st.bt) {
                        // the word's upper 56 bits take the sum, its low byte counts this CTA in
                        red_add_u64(dots + k, ((unsigned long long)((v1 << kshift) + bint) << 8) + 1ull);
                        red_add_u64(dots + a.bpad + k, ((unsigned long long)((v2 << kshift) + bint) << 8) + 1ull);
                    }
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(reinterpret_cast<uint64_t*>(sh->empty_a + ring.slot));
            j += kColAWarps;
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
        const uint32_t b_x = (uint32_t)(lane & 7);
        const uint32_t b_off = (uint32_t)lane * kColBlockBytes + (((uint32_t)p ^ b_x) << 4);
        const uint32_t rdig_lane = smem_u32(rdig) + (uint32_t)(gl * rstride + tl * 8);
        int q = 0;                                       // chunks so far
        ColRing ring{0, 0u};
        // After a wait has given up the warp stays in step with the others (the named barriers below need every
        // B thread) but waits for nothing and skips the arithmetic.
        bool ok = true;
#pragma unroll 1
        for (int t_rel = 0; t_rel < steps; ++t_rel) {
            const ColStep st = col_step(a, a.first_step + t_rel);
            const bool last = t_rel + 1 == steps;
            // ---- digits of w = step * x of the own features for this step, and the own part of lo^T x
            {
                const int par = t_rel & 1;
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
                // the unit of the digits is the dots' unit times a power of two (at most twice what max |w| needs), so
                // that a digit sum turns into the dots' unit by a shift
                const double U = sh->sp[par].U, need = (double)wmax * (1.0 / (double)QMAXW);
                const int eu = col_exponent(U);                           // U = 2^eu
                const int ks = need > U ? col_exponent(need) + 1 - eu : 0;   // need < U * 2^ks
                const float inv = (float)col_pow2(-(eu + ks));
                if (btid == 0) { sh->sp[par].kshift = ks; sh->sp[par].bint = __double2ll_rn(bsum * sh->sp[par].invU); }
#pragma unroll
                for (int e = 0; e < NF; ++e) {
                    const int fi = tl + 4 * e, h = fi / NG, gi = fi - h * NG;
                    if (fi < 2 * NG) {
                        const int byte = 16 * p + 2 * gl + h, kb = byte >> 5, bb = byte & 31;
                        // balanced digits without a carry chain: with 64 added to every digit the number is plain base 128
                        const uint32_t u = (uint32_t)((have[e] ? max(-QMAXW, min(QMAXW, __float2int_rn(st_o[e] * xo[e] * inv))) : 0) + kColBiasW);
                        signed char* dst = wdig + (size_t)((gi * 4 + kb) * 8) * 32 + ((bb & 15) >> 2) * 8 + (bb >> 4) * 4 + (bb & 3);
#pragma unroll
                        for (int s = 0; s < NS; ++s) dst[s * 32] = (signed char)((int)((u >> (7 * s)) & 127u) - 64);
                    }
                }
                named_barrier(kColNamedB, kColBThreads);     // every digit is written (also: red_* may be reused)
                if (btid == 0) st_release_cta(&sh->w_version, t_rel + 1);
                if (t_rel > 0 && p == 0 && lane == 0) col_mark(a, t_rel - 1, 7);
            }
            int acc2[2][NG][4];                                  // two sets, for alternate 32-row blocks: shorter dependency chains
#pragma unroll
            for (int h = 0; h < 2; ++h)
#pragma unroll
                for (int g = 0; g < NG; ++g)
#pragma unroll
                    for (int e = 0; e < 4; ++e) acc2[h][g][e] = 0;
#pragma unroll 1
            for (int c = 0; c < st.nch; ++c, ++q) {
                const int rbuf = q & (kColRBufs - 1);
                const long long w0c = (a.trace && p == 0) ? clock64() : 0;
                long long w1c = w0c;
                // both are usually there already: one look at each, side by side, before the waiting routine is called
                const bool have_r = mbar_test_wait(sh->rfull + rbuf, (uint32_t)((q >> kColRBufShift) & 1));
                const bool have_c = mbar_test_wait(sh->full_b + ring.slot, ring.phase);
                if (!__all_sync(0xffffffffu, ok && have_r && have_c)) {
                    ok = ok && col_wait(sh->rfull + rbuf, (uint32_t)((q >> kColRBufShift) & 1), sh, a.status, 73);
                    w1c = (a.trace && p == 0) ? clock64() : 0;
                    ok = ok && col_wait(sh->full_b + ring.slot, ring.phase, sh, a.status, 74);
                    ok = __all_sync(0xffffffffu, ok);                  // the warp acts as one
                }
                if (a.trace && p == 0 && lane == 0) { col_tally(a, t_rel, 4, w1c - w0c); col_tally(a, t_rel, 5, clock64() - w1c); }
                const uint32_t tile = smem_u32(tiles_b) + (uint32_t)ring.slot * slot_bytes + b_off;
                // Rows past the step's last one carry zero digits, so whole chunks are contracted: all R / 32 blocks, and
                // for the usual R = 128 without a test per block.
                const int nrb = ok ? R >> 5 : 0;
                auto blocks = [&](auto whole) {
#pragma unroll
                for (int rb2 = 0; rb2 < kColMaxChunkRows / 32; rb2 += 2) {
                    // the four operand pairs of two 32-row blocks are fetched together, then used: one wait for shared
                    // memory per pair of blocks instead of one per block and plane
                    uint32_t r4[2][2][4], b0[2][2], b1[2][2];
#pragma unroll
                    for (int h = 0; h < 2; ++h)
#pragma unroll
                        for (int pl = 0; pl < 2; ++pl) {
                            const int rb = rb2 + h;
                            if (decltype(whole)::value || rb < nrb) {
                                ldsm_x4_trans(r4[h][pl], tile + (uint32_t)pl * plane_bytes + (uint32_t)rb * 32u * kColBlockBytes);
                                asm volatile("ld.shared.v2.u32 {%0, %1}, [%2];" : "=r"(b0[h][pl]), "=r"(b1[h][pl])
                                             : "r"(rdig_lane + (uint32_t)(((rbuf * 2 + pl) * NRD) * rstride + rb * 32)));
                            }
                        }
#pragma unroll
                    for (int pl = 0; pl < 2; ++pl)                   // (neighbouring MMAs go to different accumulators)
#pragma unroll
                        for (int h = 0; h < 2; ++h) {
                            if (decltype(whole)::value || rb2 + h < nrb) {
                                // bytes {2g, 2g+1} of rows {2t, 2t+1} of the four 8-row groups -> byte 2g (and 2g+1) of rows
                                // {2t, 2t+1, 8+2t, 9+2t} (+16): features x rows, in the row order of the residual digits
                                const uint32_t* r = r4[h][pl];
                                const uint32_t e0 = __byte_perm(r[0], r[1], 0x6420), o0 = __byte_perm(r[0], r[1], 0x7531);
                                const uint32_t e1 = __byte_perm(r[2], r[3], 0x6420), o1 = __byte_perm(r[2], r[3], 0x7531);
#pragma unroll
                                for (int g = 0; g < NG; ++g) {
                                    // All groups of a byte meet the same residual digits, so the sums may nest: accumulator g
                                    // takes the byte with the groups below g cleared (g = 0: the byte as it is), i.e.
                                    // sum_{h >= g} 2^(h CB) code_h; group g is the difference of two neighbours.
                                    const uint32_t mk = 0x01010101u * (uint32_t)((0xFFu << (g * CB)) & 0xFFu);
                                    mma_u8s8(acc2[h][g], e0 & mk, o0 & mk, e1 & mk, o1 & mk, b0[h][pl], b1[h][pl]);
                                }
                            }
                        }
                }
                };
                if (nrb == kColMaxChunkRows / 32) blocks(std::true_type{});
                else blocks(std::false_type{});
                __syncwarp();
                if (lane == 0) {
                    mbar_arrive(reinterpret_cast<uint64_t*>(sh->empty_b + ring.slot));
                    mbar_arrive(reinterpret_cast<uint64_t*>(sh->rempty + rbuf));
                }
                ring.next(a.slots_b);
            }
            const long long u0c = (a.trace && p == 0) ? clock64() : 0;
            // ---- the step's gradient of the own features; update
            // lane (g, t): acc[gi][0..1] = digits 2t, 2t+1 of byte 2g, acc[gi][2..3] of byte 2g+1
            int acc[NG][4];
#pragma unroll
            for (int g = 0; g < NG; ++g)
#pragma unroll
                for (int e = 0; e < 4; ++e) acc[g][e] = acc2[0][g][e] + acc2[1][g][e];
            const ColStepParams& sp = sh->sp[t_rel & 1];
            const double delta_r = sp.delta_r, lo_term = sp.delta_r * sp.rsum, scale = 1.0 / (2.0 * (double)st.bt);
            const double w0 = (tl == 0) ? 1.0 : (tl == 1) ? 65536.0 : (tl == 2) ? 4294967296.0 : 281474976710656.0;  // 256^(2t)
            double Sf[NF];
#pragma unroll
            for (int e = 0; e < NF; ++e) Sf[e] = 0.0;
#pragma unroll
            for (int fi = 0; fi < 2 * NG; ++fi) {
                const int h = fi / NG, gi = fi - h * NG;
                const int lo_d = acc[gi][2 * h] - (gi + 1 < NG ? acc[gi + 1 < NG ? gi + 1 : gi][2 * h] : 0);
                const int hi_d = acc[gi][2 * h + 1] - (gi + 1 < NG ? acc[gi + 1 < NG ? gi + 1 : gi][2 * h + 1] : 0);
                // (exact: the differences are 2^(gi CB) times the group's digit sums)
                double v = ((double)(lo_d >> (gi * CB)) + 256.0 * (double)(hi_d >> (gi * CB))) * w0;
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
            if (p == 0 && lane == 0) col_tally(a, t_rel, 6, clock64() - u0c);
        }
    }
    // =================================================================================== R warps: residual digits
    else if (warp < kColWarpS2) {
        // Each R warp works alone on the chunks q = rw (mod kColRWarps) of the launch's sequence, with a digit buffer
        // of its own: that many exchanges are in flight at a time.  The warps meet twice per step: for the largest
        // |label| and for the step's sums.
        const int rt = tid - 32 * kColWarpR0, rw = rt >> 5;
        int q0 = 0;                                      // the step's first chunk in the launch's sequence
        bool ok = true;                                  // (after a failure: as for the B warps)
        const double grow = a.reg == ZIPML_REG_LSSVM ? fmax(1.0, fabs(1.0 - (double)a.reg_cst)) : 1.0;
        const int zper = (a.bpad + G - 1) / G;           // rows of a buffer of dot words that this CTA clears
        const int ngrp = a.ngrp;
        const int last_size = G - (ngrp - 1) * a.gsize;  // CTAs of the last group
#pragma unroll 1
        for (int t_rel = 0; t_rel < steps; ++t_rel) {
            const ColStep st = col_step(a, a.first_step + t_rel);
            const ColStepParams& sp = sh->sp[t_rel & 1];
            const long long* dots = a.dots + (size_t)(t_rel % 3) * ngrp * 2 * a.bpad;
            // the step's largest |label| completes the bound of its residuals
            float bm = 0.0f;
#pragma unroll 1
            for (int k = rt; k < st.bt; k += kColRThreads) bm = fmaxf(bm, fabsf(__ldg(a.b + st.row0 + k)));
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) bm = fmaxf(bm, __shfl_xor_sync(0xffffffffu, bm, o));
            if (lane == 0) sh->red_f[1][rw] = bm;
            named_barrier(kColNamedR, kColRThreads);
            bm = 0.0f;
#pragma unroll
            for (int w = 0; w < kColRWarps; ++w) bm = fmaxf(bm, sh->red_f[1][w]);
            const double rbound = (dbound + (double)bm) * 1.0001;
            // The residuals' unit is a power of two as well (at most twice what the bound needs), so that a dot becomes
            // a residual by a shift and the label's own fixed-point value: integers only on the way to the digits.
            const int ed = rbound > 0.0 ? max(-900, min(900, col_exponent(rbound * (1.0 / (double)kColQmaxR)) + 1)) : 0;
            const double delta_r = col_pow2(ed), inv_delta = col_pow2(-ed);
            const int sft = col_exponent(sp.U) - ed;     // dot unit over residual unit: 2^sft (at most 2^4 by construction)
            const int lsh = max(0, min(sft, 8)), rsh = min(63, max(0, -sft));
            const long long half = rsh > 0 ? (1ll << (rsh - 1)) : 0;
            long long amax = 0;                          // largest |fixed-point residual| of the lane
            long long rs_hi = 0, rs_lo = 0;              // sum of the fixed-point residuals: high parts and low 28 bits
            const int c_last = st.nch - 1;
            bool behind = false;                         // (a step's first chunks are never complete yet)
#pragma unroll 1
            for (int c = (rw - q0) & (kColRWarps - 1); c < st.nch; c += kColRWarps) {
                const int q = q0 + c, rbuf = q & (kColRBufs - 1);
                signed char* rd = rdig + (size_t)rbuf * 2 * NRD * rstride;
                // A lane takes the four rows whose digits make one 32-bit word of pass B's operand: rows 2t, 2t+1, 8+2t,
                // 9+2t of half `hf` of the 32-row block `blk` (k index 4t + i <-> row 2t + (i & 1) + 8 (i >> 1)).
                const int blk = lane >> 3, hf = (lane >> 2) & 1;
                const int kkA = blk * 32 + 16 * hf + 2 * tl;           // the first of them within the chunk
                const int kA = c * R + kkA;                              // and within the step
                const bool mine = kkA < R && kA < st.bt;
                float bk[4];                                             // the labels wait for nobody
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int k = kA + (i & 1) + 8 * (i >> 1);
                    bk[i] = (mine && k < st.bt) ? __ldg(a.b + st.row0 + k) : 0.0f;
                }
                // ---- the chunk's dots.  First a few lanes watch the last row of each 32-row task and group (one request
                // per look, with a pause: five hundred warps looking at L2 as fast as it answers would take a good part
                // of its bandwidth), then every lane reads its own rows' words until their counts are complete too.
                // A warp that found its previous chunk complete at the first look is behind pass A: it skips the watch
                // (a round trip to L2) and reads the words at once.
                const long long t0 = clock64();
                bool first_look = true;
                if (lane < 4 * ngrp && ok && !behind) {
                    const int g = lane >> 2, first = c * R + 32 * (lane & 3);
                    if (first < st.bt && 32 * (lane & 3) < R) {
                        const long long* wl = dots + ((size_t)g * 2 + 1) * a.bpad + min(st.bt, first + 32) - 1;
                        const int want = g == ngrp - 1 ? last_size : a.gsize;
#pragma unroll 1
                        for (int spin = 0;; ++spin) {
                            long long v0;
                            asm volatile("ld.global.cg.s64 %0, [%1];" : "=l"(v0) : "l"(wl) : "memory");
                            if ((int)(v0 & 0xFF) >= want) break;
                            first_look = false;
                            if ((spin & 15) == 15) {
                                if (col_aborted(sh) || *reinterpret_cast<volatile int*>(&a.status->code) != 0) { sh->abort_flag = 1; break; }
                                if (clock64() - t0 > kColWaitCycles) { sh->abort_flag = 1; set_status(a.status, ZIPML_ERR_TIMEOUT, 75); break; }
                            }
                            __nanosleep(400);
                        }
                    }
                }
                __syncwarp();
                ok = __all_sync(0xffffffffu, ok && !col_aborted(sh));          // (the warp acts as one)
                if (a.trace && rw == 0 && lane == 0) col_tally(a, t_rel, 2, clock64() - t0);
                long long D1[4], D2[4];                                  // the rows' dots: sums over the groups' words
#pragma unroll 1
                for (int spin = 0;; ++spin) {
                    bool done = true;
#pragma unroll
                    for (int i = 0; i < 4; ++i) { D1[i] = 0; D2[i] = 0; }
                    if (mine && ok) {
#pragma unroll 1
                        for (int g = 0; g < ngrp; ++g) {
                            const long long* s1 = dots + (size_t)g * 2 * a.bpad + kA;
                            const int want = g == ngrp - 1 ? last_size : a.gsize;
                            long long w1[4], w2[4];
                            ld_l2_v2(s1, w1[0], w1[1]);
                            ld_l2_v2(s1 + 8, w1[2], w1[3]);
                            ld_l2_v2(s1 + a.bpad, w2[0], w2[1]);
                            ld_l2_v2(s1 + a.bpad + 8, w2[2], w2[3]);
#pragma unroll
                            for (int i = 0; i < 4; ++i) {
                                if (kA + (i & 1) + 8 * (i >> 1) < st.bt) done = done && (int)(w1[i] & 0xFF) >= want && (int)(w2[i] & 0xFF) >= want;
                                D1[i] += w1[i] >> 8;
                                D2[i] += w2[i] >> 8;
                            }
                        }
                    }
                    if (__all_sync(0xffffffffu, done) || !ok) break;
                    first_look = false;
                    __nanosleep(200);
                    if ((spin & 7) == 7) {
                        bool give_up = col_aborted(sh) || *reinterpret_cast<volatile int*>(&a.status->code) != 0;
                        if (clock64() - t0 > kColWaitCycles) { set_status(a.status, ZIPML_ERR_TIMEOUT, 77); give_up = true; }
                        if (__any_sync(0xffffffffu, give_up)) { sh->abort_flag = 1; ok = false; }
                    }
                }
                behind = __all_sync(0xffffffffu, first_look);
                const long long e0c = (a.trace && rw == 0) ? clock64() : 0;
                if (ok && q >= kColRBufs) ok = col_wait(sh->rempty + rbuf, (uint32_t)(((q >> kColRBufShift) - 1) & 1), sh, a.status, 76);
                ok = __all_sync(0xffffffffu, ok);
                if (a.trace && rw == 0 && lane == 0) col_tally(a, t_rel, 3, clock64() - e0c);
                if (kkA < R && ok) {
                    // residuals r = U * dot - label in fixed point, then their digits: with 64 added to every digit the
                    // number is plain base 256 (no carry chain); four rows' digits make a word
                    unsigned long long u1[4], u2[4];
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        long long R1 = 0, R2 = 0;
                        if (kA + (i & 1) + 8 * (i >> 1) < st.bt) {
                            const long long bfix = __double2ll_rn((double)bk[i] * inv_delta);
                            R1 = max(-kColQmaxR, min(kColQmaxR, (((D1[i] + half) >> rsh) << lsh) - bfix));
                            R2 = max(-kColQmaxR, min(kColQmaxR, (((D2[i] + half) >> rsh) << lsh) - bfix));
                            amax = max(amax, max(llabs(R1), llabs(R2)));
                            rs_hi += (R1 >> 28) + (R2 >> 28);
                            rs_lo += (R1 & 0xFFFFFFFll) + (R2 & 0xFFFFFFFll);
                        }
                        u1[i] = ((unsigned long long)R1 + kColBiasR) ^ kColBiasR;      // eight digits as signed bytes
                        u2[i] = ((unsigned long long)R2 + kColBiasR) ^ kColBiasR;
                    }
                    // the four rows' words (four digits each) are transposed into one word per digit
                    signed char* dst = rd + blk * 32 + tl * 8 + hf * 4;
#pragma unroll
                    for (int h = 0; h < 4; ++h) {                        // digits 0..3, 4..7 of r2 (meets plane 1), then of r1
                        uint32_t e[4];
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            const unsigned long long u = h < 2 ? u2[i] : u1[i];
                            e[i] = (h & 1) ? (uint32_t)(u >> 32) : (uint32_t)u;
                        }
                        const uint32_t t0 = __byte_perm(e[0], e[1], 0x5140), t1 = __byte_perm(e[2], e[3], 0x5140);
                        const uint32_t t2 = __byte_perm(e[0], e[1], 0x7362), t3 = __byte_perm(e[2], e[3], 0x7362);
                        *reinterpret_cast<uint32_t*>(dst + (size_t)(4 * h + 0) * rstride) = __byte_perm(t0, t1, 0x5410);
                        *reinterpret_cast<uint32_t*>(dst + (size_t)(4 * h + 1) * rstride) = __byte_perm(t0, t1, 0x7632);
                        *reinterpret_cast<uint32_t*>(dst + (size_t)(4 * h + 2) * rstride) = __byte_perm(t2, t3, 0x5410);
                        *reinterpret_cast<uint32_t*>(dst + (size_t)(4 * h + 3) * rstride) = __byte_perm(t2, t3, 0x7632);
                    }
                }
                if (c != c_last) {                       // (the step's last chunk is released below, after the step's sums)
                    __syncwarp();
                    if (lane == 0) mbar_arrive(reinterpret_cast<uint64_t*>(sh->rfull + rbuf));
                }
                // (off the chunk's path) every CTA has left step t - 1 behind, as chunk 0's complete dots showed: its buffer of dot words is cleared for step t + 2 (this CTA's share)
                if (c == 0 && ok) {
                    __threadfence();        // (see "Memory order" above: the others' reads of that buffer before these stores)
                    long long* z = a.dots + (size_t)((t_rel + 2) % 3) * ngrp * 2 * a.bpad;
                    const int z0 = cta * zper, z1 = min(a.bpad, z0 + zper);
#pragma unroll 1
                    for (int g = 0; g < 2 * ngrp; ++g)
#pragma unroll 1
                        for (int i = z0 + lane; i < z1; i += 32) z[(size_t)g * a.bpad + i] = 0;
                }
            }
            // ---- the step's residuals are all known: their sum for the B warps, the next step's bound and unit
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                amax = max(amax, __shfl_xor_sync(0xffffffffu, amax, o));
                rs_hi += __shfl_xor_sync(0xffffffffu, rs_hi, o);
                rs_lo += __shfl_xor_sync(0xffffffffu, rs_lo, o);
            }
            if (lane == 0) { sh->red_d[1][rw] = (double)amax * delta_r; sh->red_l[0][rw] = rs_hi; sh->red_l[1][rw] = rs_lo; }
            named_barrier(kColNamedR, kColRThreads);     // (the next step's barrier keeps these slots from being rewritten early)
            double rm = 0.0;
            long long hi = 0, lo = 0;
#pragma unroll
            for (int w = 0; w < kColRWarps; ++w) { rm = fmax(rm, sh->red_d[1][w]); hi += sh->red_l[0][w]; lo += sh->red_l[1][w]; }
            dbound = (dbound * grow + fabs((double)a.lr) * rm * c2) * 1.0001;
            if (((q0 + c_last) & (kColRWarps - 1)) == rw) {      // the warp that holds the step's last chunk
                if (lane == 0) {
                    ColStepParams& cur = sh->sp[t_rel & 1];
                    cur.inv_r = inv_delta;
                    cur.delta_r = delta_r;
                    cur.rsum = (double)hi * 268435456.0 + (double)lo;
                    col_unit_of(dbound, sh->sp[(t_rel + 1) & 1].U, sh->sp[(t_rel + 1) & 1].invU);
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(reinterpret_cast<uint64_t*>(sh->rfull + ((q0 + c_last) & (kColRBufs - 1))));
            }
            q0 += st.nch;
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

// Tensor maps over the two planes as byte matrices: boxes of 128 bytes x R rows with the 128-byte swizzle,
// bytes past the row or the matrix's last row read as zero.  The encoder is a driver entry
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
    // row-major: m x row_bytes; column blocks: (blocks * m) pieces of 128 bytes, a CTA's rows one after the other
    const bool blocks = d->layout == ZIPML_LAYOUT_COLUMN_BLOCKS;
    const cuuint64_t nblk = (cuuint64_t)((d->row_bytes + kColBlockBytes - 1) / kColBlockBytes);
    const cuuint64_t gdim[2] = {blocks ? (cuuint64_t)kColBlockBytes : (cuuint64_t)d->row_bytes, blocks ? nblk * (cuuint64_t)d->m : (cuuint64_t)d->m};
    const cuuint64_t gstride[1] = {blocks ? (cuuint64_t)kColBlockBytes : (cuuint64_t)d->row_bytes};
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
    if ((d->row_bytes + kColBlockBytes - 1) / kColBlockBytes * d->m > 0x7fffffffLL) return ZIPML_ERR_WORKSPACE;     // (32-bit copy coordinates)
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
    if (R > kColMaxChunkRows) R = kColMaxChunkRows;
    if (R > (B + 31) / 32 * 32) R = (int)((B + 31) / 32 * 32);
    const int nch_max = (int)((B + R - 1) / R);
    const int bpad = nch_max * R;
    // One dot word per row and plane for all CTAs (tuning: grid_feature_parts = words, each shared by a group of
    // CTAs).  Same-address atomics are served one after the other, but more words cost the readers more than the
    // shorter queues give back: measured on 128 CTAs, 16 KB rows: 26.3 / 27.8 / 30.8 us per step with 1 / 2 / 4 words.
    int ngrp = p->grid_feature_parts > 0 ? p->grid_feature_parts : 1;
    if (ngrp > kColMaxGroups) ngrp = kColMaxGroups;
    if (ngrp > G) ngrp = (int)G;
    int gsize = (int)((G + ngrp - 1) / ngrp);
    while (ngrp > 1 && (int64_t)(ngrp - 1) * gsize >= G) --ngrp;       // no empty group

    const size_t slot_bytes = (size_t)2 * R * kColBlockBytes;
    const size_t fixed = 1024 + (size_t)kColRBufs * 2 * kColRDigits * (R + 32) + (size_t)ng * 4 * 8 * 32 + 16 +
                         (size_t)kColAWarps * 2 * 32 * 2 * sizeof(int) + sizeof(ColShared);
    if (fixed + 4 * slot_bytes > (size_t)ctx->smem_optin) return ZIPML_ERR_WORKSPACE;
    int slots = (int)(((size_t)ctx->smem_optin - fixed) / slot_bytes);
    if (slots > 2 * kColMaxSlots) slots = 2 * kColMaxSlots;
    // the first visits come from HBM and need the deeper ring (tuning: grid_row_parts = slots of the B ring)
    int slots_b = p->grid_row_parts > 0 ? p->grid_row_parts : slots / 3;
    if (slots_b < 2) slots_b = 2;
    if (slots_b > slots - 2) slots_b = slots - 2;
    if (slots_b > kColMaxSlots) slots_b = kColMaxSlots;
    int slots_a = slots - slots_b;
    if (slots_a > kColMaxSlots) slots_a = kColMaxSlots;
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
    const size_t o_dots = piece(sizeof(long long) * 3 * 2 * (size_t)bpad * ngrp);
    const size_t zero_bytes = off;
    const size_t o_ord = piece(sizeof(int32_t) * (size_t)(p->batch_order ? T : 0));
    rc = ws_reserve(ctx, off);
    if (rc != ZIPML_OK) return rc;

    ColumnArgs a;
    memset(&a, 0, sizeof(a));
    a.m = d->m; a.batch = B; a.lo = d->feat_lo; a.step = d->feat_step; a.b = b; a.x = x; a.grad_out = grad_out;
    a.n = (int)d->n; a.bits = d->bits; a.R = R; a.slots_a = slots_a; a.slots_b = slots_b; a.bpad = bpad;
    a.ngrp = ngrp; a.gsize = gsize; a.blocked = d->layout == ZIPML_LAYOUT_COLUMN_BLOCKS;
    a.lr = p->lr; a.reg = p->reg; a.reg_cst = reg_constant(p);
    a.dots = reinterpret_cast<long long*>(ctx->ws + o_dots);
    a.status = ctx->d_status;
    a.trace = reinterpret_cast<unsigned long long*>(p->trace);
    a.trace_steps = p->trace ? p->trace_steps : 0;
    a.first_step = first_step;
    a.num_steps = num_steps;
    if (p->batch_order) {
        int32_t* dev_order = reinterpret_cast<int32_t*>(ctx->ws + o_ord);
        e = cudaMemcpyAsync(dev_order, p->batch_order, sizeof(int32_t) * (size_t)T, cudaMemcpyHostToDevice, ctx->stream);
        if (e != cudaSuccess) return cuda_status(e);
        a.order = dev_order;
    }
    e = cudaMemsetAsync(ctx->ws, 0, zero_bytes, ctx->stream);
    if (e != cudaSuccess) return cuda_status(e);
    void* params[] = {&a, &tmaps[0], &tmaps[1]};
    e = cudaLaunchCooperativeKernel(kernel, dim3((unsigned)G), dim3(kColThreads), params, smem, ctx->stream);
    if (e != cudaSuccess) return cuda_status(e);
    ctx->launches += 1;
    ctx->last_engine = ZIPML_ENGINE_COLUMN;
    return ZIPML_OK;
}

}  // namespace zipml
