// Device-side pieces shared by the SGD engines: the argument block, mbarrier / bulk-copy wrappers,
// the bounded grid barrier and the row-scaled vector quantizer.
#pragma once

#include "common.cuh"
#include "internal.h"

namespace zipml {

constexpr int kSgdThreads = 256;
constexpr int kSgdWarps = kSgdThreads / 32;
constexpr int kMaxStages = 4;
constexpr long long kBarrierSpinLimit = 1ll << 21;
constexpr long long kCopySpinLimit = 1ll << 24;

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
    float* model_out;       // null or n: the model the last executed step's gradient saw (Q3(x) or x)
    int64_t batch, first_step, num_steps;
    const int32_t* order;   // device copy of the batch order, or null
    float lr;
    int reg;                // ZIPML_REG_* and its fp32 constant
    float reg_cst;
    int model_bits, grad_bits, vector_norm;
    uint64_t seed;
    uint32_t epoch;
    int na, nb;             // feature parts, row parts
    int wc;                 // words per feature part (multiple of 32)
    int rc;                 // rows per row part
    int stages;             // shared-memory stages of the code ring (STAGED kernels)
    int cr;                 // ring engine: rows per chunk (one ring slot holds cr rows of both planes)
    int sub;                // ring engine: features of a part that one row-part CTA reduces and updates
    int pitch;              // ring engine: words between consecutive rows of a chunk in shared memory (>= wc)
    // ring engine: exchange buffers of 8-byte packets {fp32 value, step tag}, zeroed before a launch
    unsigned long long* ll_pd;   // [2][nb][na][rc][4]   partial dots (hi, lo of two doubles); only na > 1
    unsigned long long* ll_rs;   // [na][nb][nb][sub+2]  partial gradients per (owner, writer) + residual sum
    unsigned long long* ll_gn;   // [2][G][2]            partial squared gradient norms (hi, lo)
    unsigned long long* ll_ag;   // [na*wc*FPW] model the next step sees, then [2][G][2] partial squared model norms
    double* pd;             // [2][na][batch][2]   partial dots
    float* pg;              // [2][nb][na*wc*FPW]  partial code gradients (table mode: value gradients)
    double* ps;             // [2][nb]             partial sums of r1 + r2
    unsigned* barrier;      // grid barrier counter (zeroed before a persistent launch)
    DeviceStatus* status;
    unsigned long long* trace;   // ring engine: optional timestamps, 8 per step for the first trace_steps steps
    int trace_steps;
    int use_tmap;           // ring engine: chunks arrive as 2-D tensor copies
    int phases;             // mask of kPhase*
    int persistent;
};

// ---------------------------------------------------------------------------------------------
// mbarrier + bulk copy wrappers (shared::cta addresses are passed as 32-bit shared pointers)
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, int count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_fence_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
    return ok != 0;
}
// Global -> shared bulk copy; both addresses 16-byte aligned, bytes a multiple of 16.
__device__ __forceinline__ void bulk_copy_g2s(void* dst_smem, const void* src_gmem, uint32_t bytes, uint64_t* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_u32(dst_smem)), "l"(src_gmem), "r"(bytes), "r"(smem_u32(bar)) : "memory");
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

// The scale M(v) of a vector in shared memory: ||v||_2, or max |v_i| for ZIPML_NORM_LINF.
__device__ __forceinline__ float l2_norm_smem(const float* v, int count, double* red);
__device__ __forceinline__ float vector_scale_smem(const float* v, int count, double* red, int norm) {
    if (norm == ZIPML_NORM_L2) return l2_norm_smem(v, count, red);
    double mx = 0.0;
    for (int i = threadIdx.x; i < count; i += kSgdThreads) mx = fmax(mx, (double)fabsf(v[i]));
    return (float)block_max(mx, red);
}

__device__ __forceinline__ float l2_norm_smem(const float* v, int count, double* red) {
    double ss = 0.0;
    for (int i = threadIdx.x; i < count; i += kSgdThreads) ss += (double)v[i] * (double)v[i];
    return (float)sqrt(block_sum(ss, red));
}

}  // namespace zipml
