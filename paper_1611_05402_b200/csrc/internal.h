// Host-side internals of the library: the context and the kernel launchers that the C-ABI entry
// points call.  Not part of the public interface.
#pragma once

#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "../../include/zipml.h"

namespace zipml {
struct DeviceStatus;
}

struct zipml_ctx {
    int device = 0;
    cudaStream_t stream = nullptr;
    int sm_count = 0;
    int smem_optin = 0;             // max dynamic shared memory per block (opt-in), bytes
    int cooperative = 0;            // device supports cooperative launch
    unsigned char* ws = nullptr;    // general workspace
    size_t ws_bytes = 0;
    zipml::DeviceStatus* d_status = nullptr;
    // staging buffers of zipml_train_host (grown on demand)
    unsigned char* stage = nullptr;
    size_t stage_bytes = 0;
    int64_t launches = 0;           // kernels launched so far (diagnostics)
    int last_engine = 0;            // engine of the latest zipml_sgd_epoch call (diagnostics)
    void* tmap_encode = nullptr;    // cuTensorMapEncodeTiled, resolved on first use
};

namespace zipml {

// Argument checks shared by every entry point that takes a dataset: ZIPML_OK, or the status to return.
int check_dataset(const zipml_dataset* d);

// Status helpers -------------------------------------------------------------------------------
int cuda_status(cudaError_t e);                       // ZIPML_OK or ZIPML_ERR_CUDA (clears the sticky error)
int ws_reserve(zipml_ctx* ctx, size_t bytes);         // grow ctx->ws to at least `bytes`
int stage_reserve(zipml_ctx* ctx, size_t bytes);

// The fp32 constant of zipml_sgd_params' regulariser for step length lr (see regularise() in common.cuh).
inline float reg_constant(const zipml_sgd_params* p) {
    if (p->reg == ZIPML_REG_L2) return (float)(1.0 / (1.0 + (double)p->lr * (double)p->reg_param));
    if (p->reg == ZIPML_REG_L1 || p->reg == ZIPML_REG_LSSVM) return (float)((double)p->lr * (double)p->reg_param);
    return 0.0f;
}

// Simple bump carving of the workspace: 256-byte aligned pieces.
struct Carver {
    unsigned char* base;
    size_t off = 0;
    explicit Carver(unsigned char* b) : base(b) {}
    template <typename T>
    T* take(size_t count) {
        T* p = reinterpret_cast<T*>(base + off);
        off += (count * sizeof(T) + 255) / 256 * 256;
        return p;
    }
};
inline size_t carve_size(size_t bytes) { return (bytes + 255) / 256 * 256; }

// Launchers (each enqueues on ctx->stream and returns a status) -------------------------------
// Column range: lo/hi per feature, inv = s/(hi-lo) and step = (hi-lo)/s for a grid of s intervals.
// Any of hi_out, inv_out, step_out may be null.  Sets NONFINITE in the device status.
int launch_column_range(zipml_ctx* ctx, const float* A, int64_t m, int64_t n, int64_t lda, int s, bool symmetric,
                        uint32_t* key_scratch /* 2n */, float* lo_out, float* hi_out, float* inv_out,
                        float* step_out);

int launch_quantize(zipml_ctx* ctx, const float* A, int64_t m, int64_t n, int64_t lda, int bits, int level_mode,
                    const float* lo, const float* inv, const float* levels, uint64_t seed, uint32_t draw, uint8_t* plane1,
                    uint8_t* plane2, int64_t row_bytes);
int launch_code_weights(zipml_ctx* ctx, const zipml_dataset* d, const float* x, float* wtab, double* base);
int launch_poly_rows(zipml_ctx* ctx, const zipml_dataset* d, const uint8_t* const* planes, int degree, const double* coef,
                     const float* wtab, const double* base, const float* scale, double* rows_out);
int plane_mean_chunks(const zipml_ctx* ctx, int64_t m);
int launch_plane_mean(zipml_ctx* ctx, const zipml_dataset* d, const uint8_t* plane, const double* c, double* partial,
                      float* g_out);

int launch_histogram(zipml_ctx* ctx, const float* A, int64_t m, int64_t n, int64_t lda, int bins,
                     const float* lo, const float* inv, uint32_t* counts /* n x bins, zeroed here */);

int launch_levels_dp(zipml_ctx* ctx, const uint32_t* counts, int64_t n, int bins, int s, const float* lo,
                     const float* hi, float* levels_out, uint64_t* objective_out);

int launch_loss_dense(zipml_ctx* ctx, const float* A, int64_t m, int64_t n, int64_t lda, const float* b,
                      const float* x, double* partials, int max_partials, double* loss_out);

int launch_loss_codes(zipml_ctx* ctx, const zipml_dataset* d, const float* b, const float* x, double* partials,
                      int max_partials, double* loss_out);

int launch_sgd_ring(zipml_ctx* ctx, const zipml_dataset* d, const float* b, float* x, const zipml_sgd_params* p,
                    int64_t first_step, int64_t num_steps, float* grad_out, bool probe_only);
int launch_sgd_lean(zipml_ctx* ctx, const zipml_dataset* d, const float* b, float* x, const zipml_sgd_params* p,
                    int64_t first_step, int64_t num_steps, float* grad_out);
int launch_sgd_cluster(zipml_ctx* ctx, const zipml_dataset* d, const float* b, float* x, const zipml_sgd_params* p,
                       int64_t first_step, int64_t num_steps, float* grad_out);
// Stream engine (uniform grids, fp32 model and gradient).  With only_if_profitable it declines
// (ZIPML_ERR_WORKSPACE) shapes whose steps are too narrow or too short for it.
int launch_sgd_stream(zipml_ctx* ctx, const zipml_dataset* d, const float* b, float* x, const zipml_sgd_params* p,
                      int64_t first_step, int64_t num_steps, float* grad_out, bool only_if_profitable);
// Column engine (uniform grids, fp32 model and gradient, rows of at most 128 bytes per SM).
int launch_sgd_apply(zipml_ctx* ctx, float* x, const float* g, int64_t n, const zipml_sgd_params* p, int64_t step,
                     float* applied_out);
int launch_sgd_column(zipml_ctx* ctx, const zipml_dataset* d, const float* b, float* x, const zipml_sgd_params* p,
                      int64_t first_step, int64_t num_steps, float* grad_out, bool only_if_profitable);
// Both planes of d into the other layout (see ZIPML_LAYOUT_* in zipml.h).
int launch_convert_layout(zipml_ctx* ctx, const zipml_dataset* d, int to_layout, uint8_t* out1, uint8_t* out2);
int launch_barrier_latency(zipml_ctx* ctx, int ctas, int floats, int iterations, unsigned long long* ns_out_dev);
int launch_sgd_epoch(zipml_ctx* ctx, const zipml_dataset* d, const float* b, float* x, const zipml_sgd_params* p,
                     int64_t first_step, int64_t num_steps, float* grad_out);

}  // namespace zipml
