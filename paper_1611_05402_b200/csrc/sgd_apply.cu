// zipml_sgd_apply_gradient: the owner stage of a step on its own -- Q4 of a gradient that the caller holds (paper
// "End-to-end Quantization": g -> Q4(g), the l2-scaled sign-magnitude quantizer of Supplement Eq. (quant2)) and the
// update x <- R(x - lr * Q4(g)) (Eq. (proxupdate); LS-SVM term of the Supplement) -- for callers that form the
// gradient of a minibatch from several devices' rows: every device applies the same sum with the same random draws
// (keyed by seed, epoch, step and coordinate), so the replicas of x stay identical.
#include "sgd_common.cuh"

namespace zipml {

constexpr int kApplyThreads = 1024;

// One block: the norm of g in a fixed order (double), then every coordinate.  The payload is n floats once per step
// beside a collective: launch latency, not bandwidth, is what it costs.
__global__ void __launch_bounds__(kApplyThreads) sgd_apply_kernel(float* __restrict__ x, const float* __restrict__ g, int64_t n,
                                                                  float lr, int grad_bits, uint64_t seed, uint32_t epoch,
                                                                  uint32_t step, int reg, float reg_cst, int vector_norm,
                                                                  float* __restrict__ applied_out) {
    __shared__ double red[40];
    VecQuant q4{0.0f, 1, seed, epoch, step, 4u};
    if (grad_bits > 0) {
        if (vector_norm == ZIPML_NORM_LINF) {
            double mx = 0.0;
            for (int64_t j = threadIdx.x; j < n; j += kApplyThreads) mx = fmax(mx, (double)fabsf(g[j]));
            q4.M = (float)block_max(mx, red);
        } else {
            double ss = 0.0;
            for (int64_t j = threadIdx.x; j < n; j += kApplyThreads) ss += (double)g[j] * (double)g[j];
            q4.M = (float)sqrt(block_sum(ss, red));
        }
        q4.sm = (1 << (grad_bits - 1)) - 1;
    }
    for (int64_t j = threadIdx.x; j < n; j += kApplyThreads) {
        float gj = g[j];
        if (grad_bits > 0) gj = q4.apply(gj, (uint32_t)j);
        if (applied_out) applied_out[j] = gj;
        x[j] = regularise(fmaf(-lr, gj, x[j]), x[j], reg, reg_cst);
    }
}

int launch_sgd_apply(zipml_ctx* ctx, float* x, const float* g, int64_t n, const zipml_sgd_params* p, int64_t step,
                     float* applied_out) {
    sgd_apply_kernel<<<1, kApplyThreads, 0, ctx->stream>>>(x, g, n, p->lr, p->grad_bits, p->seed, (uint32_t)p->epoch,
                                                           (uint32_t)step, p->reg, reg_constant(p), p->vector_norm, applied_out);
    ++ctx->launches;
    return cuda_status(cudaGetLastError());
}

}  // namespace zipml

