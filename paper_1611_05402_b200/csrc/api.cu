// C-ABI entry points: argument validation, workspace management and the order of kernel launches.
#include <new>

#include "common.cuh"
#include "internal.h"

namespace zipml {

int cuda_status(cudaError_t e) {
    if (e == cudaSuccess) return ZIPML_OK;
    (void)cudaGetLastError();
    return ZIPML_ERR_CUDA;
}

static int grow(unsigned char** buf, size_t* have, size_t want, cudaStream_t stream) {
    if (want <= *have) return ZIPML_OK;
    // earlier work on the stream may still use the old buffer
    cudaError_t e = cudaStreamSynchronize(stream);
    if (e != cudaSuccess) return cuda_status(e);
    if (*buf) { e = cudaFree(*buf); *buf = nullptr; *have = 0; if (e != cudaSuccess) return cuda_status(e); }
    const size_t bytes = (want + (1u << 20) - 1) >> 20 << 20;
    e = cudaMalloc(reinterpret_cast<void**>(buf), bytes);
    if (e != cudaSuccess) { *buf = nullptr; return cuda_status(e); }
    *have = bytes;
    return ZIPML_OK;
}

int ws_reserve(zipml_ctx* ctx, size_t bytes) { return grow(&ctx->ws, &ctx->ws_bytes, bytes, ctx->stream); }
int stage_reserve(zipml_ctx* ctx, size_t bytes) { return grow(&ctx->stage, &ctx->stage_bytes, bytes, ctx->stream); }

static bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

struct DeviceGuard {
    int prev = -1;
    bool ok = false;
    explicit DeviceGuard(int device) {
        if (cudaGetDevice(&prev) != cudaSuccess) { (void)cudaGetLastError(); prev = -1; }
        ok = cudaSetDevice(device) == cudaSuccess;
        if (!ok) (void)cudaGetLastError();
    }
    ~DeviceGuard() { if (prev >= 0) (void)cudaSetDevice(prev); }
};

int check_dataset(const zipml_dataset* d) {
    if (!d || d->struct_size != sizeof(zipml_dataset)) return ZIPML_ERR_INVALID_ARG;
    const int cb = container_bits(d->bits);
    if (cb == 0) return ZIPML_ERR_UNSUPPORTED;
    if (d->level_mode != ZIPML_LEVELS_UNIFORM && d->level_mode != ZIPML_LEVELS_TABLE) return ZIPML_ERR_INVALID_ARG;
    if (d->layout != ZIPML_LAYOUT_ROWS && d->layout != ZIPML_LAYOUT_COLUMN_BLOCKS) return ZIPML_ERR_INVALID_ARG;
    if (d->level_mode == ZIPML_LEVELS_TABLE && d->bits > 4) return ZIPML_ERR_UNSUPPORTED;
    if (d->m <= 0 || d->n <= 0) return ZIPML_ERR_INVALID_ARG;
    if (d->n > 0x7fffffffLL / 8) return ZIPML_ERR_WORKSPACE;
    if (!d->plane1 || !d->plane2 || !aligned16(d->plane1) || !aligned16(d->plane2)) return ZIPML_ERR_INVALID_ARG;
    if (d->row_bytes % 16 != 0 || d->row_bytes < zipml_row_bytes(d->n, d->bits)) return ZIPML_ERR_INVALID_ARG;
    if (d->level_mode == ZIPML_LEVELS_UNIFORM && (!d->feat_lo || !d->feat_step)) return ZIPML_ERR_INVALID_ARG;
    if (d->level_mode == ZIPML_LEVELS_TABLE && !d->levels) return ZIPML_ERR_INVALID_ARG;
    return ZIPML_OK;
}

constexpr int kLossPartials = 4096;

}  // namespace zipml

using namespace zipml;

namespace zipml {
// A wait that cannot succeed, bounded like the engines' waits: lane 0 polls a zero flag `limit` times with an
// acquire load and a pause now and then, then records the time-out (see zipml_wait_probe).
__global__ void wait_probe_kernel(const unsigned* flag, long long limit, DeviceStatus* status) {
    if (threadIdx.x != 0) return;
    for (long long it = 0; it < limit; ++it) {
        unsigned v;
        asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(flag) : "memory");
        if (v != 0) return;
        if ((it & 1023) == 1023) __nanosleep(200);
    }
    set_status(status, ZIPML_ERR_TIMEOUT, 90);
}
}  // namespace zipml

extern "C" {

const char* zipml_strerror(int status) {
    switch (status) {
        case ZIPML_OK: return "ok";
        case ZIPML_ERR_INVALID_ARG: return "invalid argument";
        case ZIPML_ERR_UNSUPPORTED: return "unsupported configuration";
        case ZIPML_ERR_NONFINITE: return "non-finite value in the input";
        case ZIPML_ERR_CUDA: return "CUDA runtime error (no device, out of memory or failed launch)";
        case ZIPML_ERR_TIMEOUT: return "a device-side wait gave up";
        case ZIPML_ERR_WORKSPACE: return "problem does not fit the kernels' shared memory or scratch limits";
        default: return "unknown status";
    }
}

int64_t zipml_column_blocks_bytes(int64_t m, int64_t row_bytes) {
    if (m <= 0 || row_bytes <= 0) return 0;
    return (row_bytes + 127) / 128 * m * 128;
}

int zipml_convert_layout(zipml_ctx* ctx, const zipml_dataset* data, int32_t to_layout, uint8_t* out1, uint8_t* out2) {
    if (!ctx) return ZIPML_ERR_INVALID_ARG;
    int rc = check_dataset(data);
    if (rc != ZIPML_OK) return rc;
    if (to_layout != ZIPML_LAYOUT_ROWS && to_layout != ZIPML_LAYOUT_COLUMN_BLOCKS) return ZIPML_ERR_INVALID_ARG;
    if (to_layout == data->layout) return ZIPML_ERR_INVALID_ARG;
    if (!out1 || !out2 || !aligned16(out1) || !aligned16(out2)) return ZIPML_ERR_INVALID_ARG;
    if (out1 == data->plane1 || out1 == data->plane2 || out2 == data->plane1 || out2 == data->plane2 || out1 == out2)
        return ZIPML_ERR_INVALID_ARG;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return ZIPML_ERR_CUDA;
    return launch_convert_layout(ctx, data, to_layout, out1, out2);
}

int64_t zipml_row_bytes(int64_t n, int32_t bits) {
    const int cb = container_bits(bits);
    if (cb == 0 || n <= 0) return 0;
    return ((n * cb + 7) / 8 + 15) / 16 * 16;
}

int zipml_create(zipml_ctx** ctx_out, int device, void* cuda_stream) {
    if (!ctx_out) return ZIPML_ERR_INVALID_ARG;
    *ctx_out = nullptr;
    int count = 0;
    if (cudaGetDeviceCount(&count) != cudaSuccess || device < 0 || device >= count) {
        (void)cudaGetLastError();
        return ZIPML_ERR_CUDA;
    }
    DeviceGuard guard(device);
    if (!guard.ok) return ZIPML_ERR_CUDA;
    zipml_ctx* ctx = new (std::nothrow) zipml_ctx();
    if (!ctx) return ZIPML_ERR_CUDA;
    ctx->device = device;
    ctx->stream = reinterpret_cast<cudaStream_t>(cuda_stream);
    cudaError_t e = cudaDeviceGetAttribute(&ctx->sm_count, cudaDevAttrMultiProcessorCount, device);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&ctx->smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, device);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&ctx->cooperative, cudaDevAttrCooperativeLaunch, device);
    if (e == cudaSuccess) e = cudaMalloc(reinterpret_cast<void**>(&ctx->d_status), sizeof(DeviceStatus));
    if (e == cudaSuccess) e = cudaMemsetAsync(ctx->d_status, 0, sizeof(DeviceStatus), ctx->stream);
    if (e != cudaSuccess) { if (ctx->d_status) (void)cudaFree(ctx->d_status); delete ctx; return cuda_status(e); }
    *ctx_out = ctx;
    return ZIPML_OK;
}

int zipml_destroy(zipml_ctx* ctx) {
    if (!ctx) return ZIPML_OK;
    DeviceGuard guard(ctx->device);
    (void)cudaStreamSynchronize(ctx->stream);
    if (ctx->ws) (void)cudaFree(ctx->ws);
    if (ctx->stage) (void)cudaFree(ctx->stage);
    if (ctx->d_status) (void)cudaFree(ctx->d_status);
    (void)cudaGetLastError();
    delete ctx;
    return ZIPML_OK;
}

int64_t zipml_kernel_launches(const zipml_ctx* ctx) { return ctx ? ctx->launches : 0; }

int32_t zipml_last_engine(const zipml_ctx* ctx) { return ctx ? ctx->last_engine : 0; }

int zipml_sync(zipml_ctx* ctx) {
    if (!ctx) return ZIPML_ERR_INVALID_ARG;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return ZIPML_ERR_CUDA;
    DeviceStatus host{0, 0};
    cudaError_t e = cudaMemcpyAsync(&host, ctx->d_status, sizeof(host), cudaMemcpyDeviceToHost, ctx->stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize(ctx->stream);
    if (e != cudaSuccess) return cuda_status(e);
    if (host.code != 0) {
        e = cudaMemsetAsync(ctx->d_status, 0, sizeof(DeviceStatus), ctx->stream);
        if (e != cudaSuccess) return cuda_status(e);
    }
    return host.code;
}

int zipml_quantize(zipml_ctx* ctx, const float* A, int64_t m, int64_t n, int64_t lda, int32_t bits,
                   int32_t level_mode, const float* levels, uint64_t seed, uint8_t* plane1, uint8_t* plane2,
                   int64_t row_bytes, float* feat_lo, float* feat_step) {
    return zipml_quantize_draw(ctx, A, m, n, lda, bits, level_mode, levels, seed, 0u, ZIPML_GRID_RANGE, plane1, plane2, row_bytes, feat_lo,
                               feat_step);
}

int zipml_quantize_draw(zipml_ctx* ctx, const float* A, int64_t m, int64_t n, int64_t lda, int32_t bits,
                        int32_t level_mode, const float* levels, uint64_t seed, uint32_t draw, int32_t grid, uint8_t* plane1,
                        uint8_t* plane2, int64_t row_bytes, float* feat_lo, float* feat_step) {
    if (!ctx) return ZIPML_ERR_INVALID_ARG;
    if (grid != ZIPML_GRID_RANGE && grid != ZIPML_GRID_SYMMETRIC) return ZIPML_ERR_INVALID_ARG;
    if (grid == ZIPML_GRID_SYMMETRIC && level_mode != ZIPML_LEVELS_UNIFORM) return ZIPML_ERR_INVALID_ARG;
    const int cb = container_bits(bits);
    if (cb == 0) return ZIPML_ERR_UNSUPPORTED;
    if (level_mode != ZIPML_LEVELS_UNIFORM && level_mode != ZIPML_LEVELS_TABLE) return ZIPML_ERR_INVALID_ARG;
    if (level_mode == ZIPML_LEVELS_TABLE && bits > 4) return ZIPML_ERR_UNSUPPORTED;
    if (!A || !plane1 || !plane2 || !feat_lo || m <= 0 || n <= 0 || lda < n) return ZIPML_ERR_INVALID_ARG;
    if (level_mode == ZIPML_LEVELS_TABLE && !levels) return ZIPML_ERR_INVALID_ARG;
    if (level_mode == ZIPML_LEVELS_UNIFORM && !feat_step) return ZIPML_ERR_INVALID_ARG;
    if (row_bytes % 16 != 0 || row_bytes < zipml_row_bytes(n, bits)) return ZIPML_ERR_INVALID_ARG;
    if (!aligned16(plane1) || !aligned16(plane2)) return ZIPML_ERR_INVALID_ARG;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return ZIPML_ERR_CUDA;
    const int s = (1 << bits) - 1;
    int rc = ws_reserve(ctx, carve_size(sizeof(uint32_t) * 2 * (size_t)n) + 2 * carve_size(sizeof(float) * (size_t)n));
    if (rc != ZIPML_OK) return rc;
    Carver cv(ctx->ws);
    uint32_t* keys = cv.take<uint32_t>(2 * (size_t)n);
    float* inv = cv.take<float>((size_t)n);
    float* step_tmp = cv.take<float>((size_t)n);
    rc = launch_column_range(ctx, A, m, n, lda, s, grid == ZIPML_GRID_SYMMETRIC, keys, feat_lo, nullptr, inv,
                             feat_step ? feat_step : step_tmp);
    if (rc != ZIPML_OK) return rc;
    return launch_quantize(ctx, A, m, n, lda, bits, level_mode, feat_lo, inv, levels, seed, draw, plane1, plane2, row_bytes);
}

int zipml_optimal_levels(zipml_ctx* ctx, const float* A, int64_t m, int64_t n, int64_t lda, int32_t bits,
                         int32_t hist_bins, float* levels_out, uint64_t* objective_out) {
    if (!ctx) return ZIPML_ERR_INVALID_ARG;
    if (bits != 2 && bits != 3 && bits != 4) return ZIPML_ERR_UNSUPPORTED;
    const int s = (1 << bits) - 1;
    if (!A || !levels_out || m <= 0 || n <= 0 || lda < n) return ZIPML_ERR_INVALID_ARG;
    if (hist_bins < s || hist_bins > 1024 || m > 1000000000LL) return ZIPML_ERR_UNSUPPORTED;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return ZIPML_ERR_CUDA;
    int rc = ws_reserve(ctx, carve_size(sizeof(uint32_t) * 2 * (size_t)n) + 3 * carve_size(sizeof(float) * (size_t)n) +
                                 carve_size(sizeof(uint32_t) * (size_t)n * hist_bins));
    if (rc != ZIPML_OK) return rc;
    Carver cv(ctx->ws);
    uint32_t* keys = cv.take<uint32_t>(2 * (size_t)n);
    float* lo = cv.take<float>((size_t)n);
    float* hi = cv.take<float>((size_t)n);
    float* inv = cv.take<float>((size_t)n);
    uint32_t* counts = cv.take<uint32_t>((size_t)n * hist_bins);
    rc = launch_column_range(ctx, A, m, n, lda, hist_bins, false, keys, lo, hi, inv, nullptr);
    if (rc != ZIPML_OK) return rc;
    rc = launch_histogram(ctx, A, m, n, lda, hist_bins, lo, inv, counts);
    if (rc != ZIPML_OK) return rc;
    return launch_levels_dp(ctx, counts, n, hist_bins, s, lo, hi, levels_out, objective_out);
}

int zipml_sgd_epoch(zipml_ctx* ctx, const zipml_dataset* data, const float* b, float* x,
                    const zipml_sgd_params* params, float* grad_out) {
    if (!ctx || !params || params->struct_size != sizeof(zipml_sgd_params)) return ZIPML_ERR_INVALID_ARG;
    int rc = check_dataset(data);
    if (rc != ZIPML_OK) return rc;
    if (!b || !x || params->batch <= 0) return ZIPML_ERR_INVALID_ARG;
    if (params->model_bits != 0 && (params->model_bits < 2 || params->model_bits > 8)) return ZIPML_ERR_UNSUPPORTED;
    if (params->grad_bits != 0 && (params->grad_bits < 2 || params->grad_bits > 8)) return ZIPML_ERR_UNSUPPORTED;
    if (params->engine < ZIPML_ENGINE_AUTO || params->engine > ZIPML_ENGINE_COLUMN) return ZIPML_ERR_INVALID_ARG;
    if (params->epoch < 0 || params->epoch > 0xffffffffLL) return ZIPML_ERR_INVALID_ARG;
    if (params->reg < ZIPML_REG_NONE || params->reg > ZIPML_REG_LSSVM) return ZIPML_ERR_INVALID_ARG;
    if (params->reg != ZIPML_REG_NONE && params->reg != ZIPML_REG_NONNEG && !(params->reg_param >= 0.0f)) return ZIPML_ERR_INVALID_ARG;
    if (params->cluster_contraction < 0 || params->cluster_contraction > 2) return ZIPML_ERR_INVALID_ARG;
    if (params->stream_prefetch < 0 || params->stream_prefetch > 9) return ZIPML_ERR_INVALID_ARG;
    if (params->column_chunk_rows < 0 || params->column_chunk_rows > 256 || params->column_chunk_rows % 32 != 0) return ZIPML_ERR_INVALID_ARG;
    if (params->vector_norm != ZIPML_NORM_L2 && params->vector_norm != ZIPML_NORM_LINF) return ZIPML_ERR_INVALID_ARG;
    // the other scaling of Q3/Q4 lives in the first-generation engine only
    const bool linf = params->vector_norm == ZIPML_NORM_LINF && (params->model_bits > 0 || params->grad_bits > 0);
    if (linf && params->engine != ZIPML_ENGINE_AUTO && params->engine != ZIPML_ENGINE_STEPWISE && params->engine != ZIPML_ENGINE_PERSISTENT)
        return ZIPML_ERR_UNSUPPORTED;
    const int64_t T = (data->m + params->batch - 1) / params->batch;
    const int64_t first = params->first_step;
    const int64_t count = params->num_steps < 0 ? T - first : params->num_steps;
    if (first < 0 || first > T || count < 0 || first + count > T) return ZIPML_ERR_INVALID_ARG;
    if (params->batch_order)
        for (int64_t i = 0; i < T; ++i)
            if (params->batch_order[i] < 0 || params->batch_order[i] >= T) return ZIPML_ERR_INVALID_ARG;
    if (count == 0) return ZIPML_OK;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return ZIPML_ERR_CUDA;
    if (linf && data->layout == ZIPML_LAYOUT_COLUMN_BLOCKS) return ZIPML_ERR_UNSUPPORTED;
    if (data->layout == ZIPML_LAYOUT_COLUMN_BLOCKS) {                 // the column engine's own layout
        if (params->engine != ZIPML_ENGINE_AUTO && params->engine != ZIPML_ENGINE_COLUMN) return ZIPML_ERR_UNSUPPORTED;
        rc = launch_sgd_column(ctx, data, b, x, params, first, count, grad_out, false);
        return rc == ZIPML_ERR_WORKSPACE ? ZIPML_ERR_UNSUPPORTED : rc;
    }
    if (params->engine == ZIPML_ENGINE_RING) return launch_sgd_ring(ctx, data, b, x, params, first, count, grad_out, false);
    if (params->engine == ZIPML_ENGINE_LEAN) return launch_sgd_lean(ctx, data, b, x, params, first, count, grad_out);
    if (params->engine == ZIPML_ENGINE_CLUSTER) return launch_sgd_cluster(ctx, data, b, x, params, first, count, grad_out);
    if (params->engine == ZIPML_ENGINE_STREAM) return launch_sgd_stream(ctx, data, b, x, params, first, count, grad_out, false);
    if (params->engine == ZIPML_ENGINE_COLUMN) return launch_sgd_column(ctx, data, b, x, params, first, count, grad_out, false);
    if (params->engine == ZIPML_ENGINE_AUTO && !linf) {
        // Small minibatch tiles are bound by the step-to-step chain, not by HBM: one cluster whose CTAs
        // exchange through shared memory, else row parts exchanging through L2.  Larger tiles go to the
        // column engine (codes read once per step), the stream engine, then the ring engine.  Each engine
        // answers ZIPML_ERR_WORKSPACE when the shape does not fit it.
        const int64_t B = params->batch < data->m ? params->batch : data->m;
        const int64_t step_bytes = 2 * B * data->row_bytes;
        if (step_bytes <= (2ll << 20)) {
            rc = launch_sgd_cluster(ctx, data, b, x, params, first, count, grad_out);
            if (rc != ZIPML_ERR_WORKSPACE) return rc;
            rc = launch_sgd_lean(ctx, data, b, x, params, first, count, grad_out);
            if (rc != ZIPML_ERR_WORKSPACE) return rc;
        }
        // (also for small steps on rows too wide for the two above)
        rc = launch_sgd_column(ctx, data, b, x, params, first, count, grad_out, true);
        if (rc != ZIPML_ERR_WORKSPACE) return rc;
        rc = launch_sgd_stream(ctx, data, b, x, params, first, count, grad_out, true);
        if (rc != ZIPML_ERR_WORKSPACE) return rc;
        rc = launch_sgd_ring(ctx, data, b, x, params, first, count, grad_out, false);
        if (rc != ZIPML_ERR_WORKSPACE) return rc;
    }
    return launch_sgd_epoch(ctx, data, b, x, params, first, count, grad_out);
}

int zipml_sgd_apply_gradient(zipml_ctx* ctx, float* x, const float* g, int64_t n, const zipml_sgd_params* params,
                             int64_t step, float* applied_out) {
    if (!ctx || !params || params->struct_size != sizeof(zipml_sgd_params)) return ZIPML_ERR_INVALID_ARG;
    if (!x || !g || n <= 0 || n > 0x7fffffffLL || step < 0 || step > 0xffffffffLL) return ZIPML_ERR_INVALID_ARG;
    if (params->grad_bits != 0 && (params->grad_bits < 2 || params->grad_bits > 8)) return ZIPML_ERR_UNSUPPORTED;
    if (params->epoch < 0 || params->epoch > 0xffffffffLL) return ZIPML_ERR_INVALID_ARG;
    if (params->reg < ZIPML_REG_NONE || params->reg > ZIPML_REG_LSSVM) return ZIPML_ERR_INVALID_ARG;
    if (params->reg != ZIPML_REG_NONE && params->reg != ZIPML_REG_NONNEG && !(params->reg_param >= 0.0f)) return ZIPML_ERR_INVALID_ARG;
    if (params->vector_norm != ZIPML_NORM_L2 && params->vector_norm != ZIPML_NORM_LINF) return ZIPML_ERR_INVALID_ARG;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return ZIPML_ERR_CUDA;
    return launch_sgd_apply(ctx, x, g, n, params, step, applied_out);
}

int zipml_barrier_latency(zipml_ctx* ctx, int32_t ctas, int32_t floats_per_cta, int32_t iterations, uint64_t* ns_out) {
    if (!ctx || !ns_out || ctas < 1 || floats_per_cta < 0 || floats_per_cta % 4 != 0 || iterations < 1 || iterations > (1 << 20))
        return ZIPML_ERR_INVALID_ARG;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return ZIPML_ERR_CUDA;
    return launch_barrier_latency(ctx, ctas, floats_per_cta, iterations, reinterpret_cast<unsigned long long*>(ns_out));
}

int zipml_poly_rows(zipml_ctx* ctx, const zipml_dataset* grid, const uint8_t* const* planes, int32_t degree,
                    const double* coef, const float* x, const float* scale, double* rows_out) {
    if (!ctx || !coef || !x || !rows_out || degree < 0 || degree > ZIPML_POLY_MAX_DEGREE) return ZIPML_ERR_INVALID_ARG;
    int rc = check_dataset(grid);
    if (rc != ZIPML_OK) return rc;
    if (grid->layout != ZIPML_LAYOUT_ROWS) return ZIPML_ERR_UNSUPPORTED;
    if (degree > 0 && !planes) return ZIPML_ERR_INVALID_ARG;
    for (int i = 0; i < degree; ++i)
        if (!planes[i] || !aligned16(planes[i])) return ZIPML_ERR_INVALID_ARG;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return ZIPML_ERR_CUDA;
    const bool table = grid->level_mode == ZIPML_LEVELS_TABLE;
    const size_t wcount = (size_t)grid->n * (table ? ((size_t)1 << grid->bits) : 1);
    rc = ws_reserve(ctx, carve_size(sizeof(float) * wcount) + carve_size(sizeof(double)));
    if (rc != ZIPML_OK) return rc;
    Carver cv(ctx->ws);
    float* wtab = cv.take<float>(wcount);
    double* base = cv.take<double>(1);
    rc = launch_code_weights(ctx, grid, x, wtab, base);
    if (rc != ZIPML_OK) return rc;
    return launch_poly_rows(ctx, grid, planes, degree, coef, wtab, base, scale, rows_out);
}

int zipml_weighted_plane_mean(zipml_ctx* ctx, const zipml_dataset* grid, const uint8_t* plane, const double* c, float* g_out) {
    if (!ctx || !plane || !c || !g_out || !aligned16(plane)) return ZIPML_ERR_INVALID_ARG;
    int rc = check_dataset(grid);
    if (rc != ZIPML_OK) return rc;
    if (grid->layout != ZIPML_LAYOUT_ROWS) return ZIPML_ERR_UNSUPPORTED;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return ZIPML_ERR_CUDA;
    const size_t count = (size_t)plane_mean_chunks(ctx, grid->m) * ((size_t)grid->n + 1);
    rc = ws_reserve(ctx, carve_size(sizeof(double) * count));
    if (rc != ZIPML_OK) return rc;
    return launch_plane_mean(ctx, grid, plane, c, reinterpret_cast<double*>(ctx->ws), g_out);
}

int zipml_wait_probe(zipml_ctx* ctx, int64_t spin_limit) {
    if (!ctx || spin_limit < 1 || spin_limit > (1 << 24)) return ZIPML_ERR_INVALID_ARG;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return ZIPML_ERR_CUDA;
    int rc = ws_reserve(ctx, 256);
    if (rc != ZIPML_OK) return rc;
    cudaError_t e = cudaMemsetAsync(ctx->ws, 0, 256, ctx->stream);
    if (e != cudaSuccess) return cuda_status(e);
    wait_probe_kernel<<<1, 32, 0, ctx->stream>>>(reinterpret_cast<const unsigned*>(ctx->ws), spin_limit, ctx->d_status);
    ctx->launches += 1;
    return cuda_status(cudaGetLastError());
}

int zipml_loss(zipml_ctx* ctx, int32_t mode, const float* A, int64_t m, int64_t n, int64_t lda,
               const zipml_dataset* data, const float* b, const float* x, double* loss_out) {
    if (!ctx || !b || !x || !loss_out) return ZIPML_ERR_INVALID_ARG;
    if (mode != ZIPML_LOSS_DENSE && mode != ZIPML_LOSS_CODES) return ZIPML_ERR_INVALID_ARG;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return ZIPML_ERR_CUDA;
    if (mode == ZIPML_LOSS_DENSE) {
        if (!A || m <= 0 || n <= 0 || lda < n) return ZIPML_ERR_INVALID_ARG;
        int rc = ws_reserve(ctx, carve_size(sizeof(double) * kLossPartials));
        if (rc != ZIPML_OK) return rc;
        return launch_loss_dense(ctx, A, m, n, lda, b, x, reinterpret_cast<double*>(ctx->ws), kLossPartials, loss_out);
    }
    int rc = check_dataset(data);
    if (rc != ZIPML_OK) return rc;
    if (data->layout != ZIPML_LAYOUT_ROWS) return ZIPML_ERR_UNSUPPORTED;
    // behind the partials: the level * x table, or (uniform grids) the digit vectors of step * x, which follow the
    // packed row byte for byte and so take their size from the stride, not from n
    const size_t tab = data->level_mode == ZIPML_LEVELS_TABLE
                           ? sizeof(float) * ((size_t)1 << data->bits) * (size_t)data->n
                           : (size_t)(8 / container_bits(data->bits)) * 4 * (((size_t)data->row_bytes + 63) / 64 * 64);
    rc = ws_reserve(ctx, carve_size(sizeof(double) * (kLossPartials + 2) + tab + 256));
    if (rc != ZIPML_OK) return rc;
    return launch_loss_codes(ctx, data, b, x, reinterpret_cast<double*>(ctx->ws), kLossPartials, loss_out);
}

int zipml_train_host(zipml_ctx* ctx, const float* A_host, int64_t m, int64_t n, int64_t lda, const float* b_host,
                     float* x_host, int32_t bits, int32_t optimal_levels, int32_t hist_bins, uint64_t quantize_seed,
                     const zipml_sgd_params* params, int32_t epochs, int32_t lr_decay, double* loss_out_host) {
    if (!ctx || !params || params->struct_size != sizeof(zipml_sgd_params)) return ZIPML_ERR_INVALID_ARG;
    if (!A_host || !b_host || !x_host || !loss_out_host || m <= 0 || n <= 0 || lda < n || epochs < 0)
        return ZIPML_ERR_INVALID_ARG;
    const int64_t rb = zipml_row_bytes(n, bits);
    if (rb == 0) return ZIPML_ERR_UNSUPPORTED;
    if (optimal_levels && (bits < 2 || bits > 4)) return ZIPML_ERR_UNSUPPORTED;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return ZIPML_ERR_CUDA;
    const size_t L = (size_t)1 << bits;
    size_t total = 0;
    auto piece = [&](size_t bytes) { const size_t off = total; total += carve_size(bytes); return off; };
    const size_t oA = piece(sizeof(float) * (size_t)m * n), ob = piece(sizeof(float) * (size_t)m);
    const size_t ox = piece(sizeof(float) * (size_t)n), op1 = piece((size_t)m * rb), op2 = piece((size_t)m * rb);
    const size_t olo = piece(sizeof(float) * (size_t)n), ostep = piece(sizeof(float) * (size_t)n);
    const size_t olev = piece(sizeof(float) * (size_t)n * L), oloss = piece(sizeof(double));
    int rc = stage_reserve(ctx, total);
    if (rc != ZIPML_OK) return rc;
    unsigned char* s = ctx->stage;
    float* dA = reinterpret_cast<float*>(s + oA);
    float* db = reinterpret_cast<float*>(s + ob);
    float* dx = reinterpret_cast<float*>(s + ox);
    float* dlev = reinterpret_cast<float*>(s + olev);
    double* dloss = reinterpret_cast<double*>(s + oloss);
    // (contiguous rows travel as one linear copy: a pitched copy of many short rows is much slower)
    cudaError_t e = lda == n ? cudaMemcpyAsync(dA, A_host, sizeof(float) * (size_t)m * n, cudaMemcpyHostToDevice, ctx->stream)
                             : cudaMemcpy2DAsync(dA, sizeof(float) * n, A_host, sizeof(float) * lda, sizeof(float) * n, (size_t)m,
                                                 cudaMemcpyHostToDevice, ctx->stream);
    if (e == cudaSuccess) e = cudaMemcpyAsync(db, b_host, sizeof(float) * m, cudaMemcpyHostToDevice, ctx->stream);
    if (e == cudaSuccess) e = cudaMemcpyAsync(dx, x_host, sizeof(float) * n, cudaMemcpyHostToDevice, ctx->stream);
    if (e != cudaSuccess) return cuda_status(e);

    zipml_dataset d{};
    d.struct_size = sizeof(zipml_dataset);
    d.bits = bits; d.m = m; d.n = n; d.row_bytes = rb;
    d.plane1 = s + op1; d.plane2 = s + op2;
    d.feat_lo = reinterpret_cast<float*>(s + olo);
    d.feat_step = reinterpret_cast<float*>(s + ostep);
    d.levels = nullptr;
    d.level_mode = optimal_levels ? ZIPML_LEVELS_TABLE : ZIPML_LEVELS_UNIFORM;
    if (optimal_levels) {
        rc = zipml_optimal_levels(ctx, dA, m, n, n, bits, hist_bins, dlev, nullptr);
        if (rc != ZIPML_OK) return rc;
        d.levels = dlev;
    }
    rc = zipml_quantize(ctx, dA, m, n, n, bits, d.level_mode, d.levels, quantize_seed, s + op1, s + op2, rb,
                        reinterpret_cast<float*>(s + olo), reinterpret_cast<float*>(s + ostep));
    if (rc != ZIPML_OK) return rc;
    zipml_sgd_params p = *params;
    for (int32_t ep = 0; ep < epochs; ++ep) {
        p.epoch = ep; p.first_step = 0; p.num_steps = -1;
        p.lr = lr_decay ? params->lr / (float)(ep + 1) : params->lr;
        rc = zipml_sgd_epoch(ctx, &d, db, dx, &p, nullptr);
        if (rc != ZIPML_OK) return rc;
    }
    rc = zipml_loss(ctx, ZIPML_LOSS_DENSE, dA, m, n, n, nullptr, db, dx, dloss);
    if (rc != ZIPML_OK) return rc;
    e = cudaMemcpyAsync(x_host, dx, sizeof(float) * n, cudaMemcpyDeviceToHost, ctx->stream);
    if (e == cudaSuccess) e = cudaMemcpyAsync(loss_out_host, dloss, sizeof(double), cudaMemcpyDeviceToHost, ctx->stream);
    if (e != cudaSuccess) return cuda_status(e);
    return zipml_sync(ctx);
}

}  // extern "C"
