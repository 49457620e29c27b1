// Shared-base storage of the two samples (paper Section 2.2, "Overhead of Storing Samples"): the two
// quantizations of a value can only be the lower or the upper end of one interval of levels, so the
// smaller code is stored once (the base plane, an ordinary plane) and each sample keeps one bit per
// value ("up" planes: feature j at bit j of its row, low bits first): bits + 2 instead of 2 * bits per
// value.  Here: the conversion both ways (bit for bit) and the code-plane loss computed straight from
// the three planes, q_c^T x = lo^T x + base^T w + up_c^T w with w = step * x.
#include "common.cuh"
#include "internal.h"

namespace zipml {

// One thread per 32 features of a row (one 32-bit word of an up plane, CB words of a code plane).
template <int CB, bool ENCODE>
__global__ void __launch_bounds__(256) shared_base_kernel(const uint32_t* __restrict__ in_a, const uint32_t* __restrict__ in_b,
                                                          const uint32_t* __restrict__ in_c, uint32_t* __restrict__ out_a,
                                                          uint32_t* __restrict__ out_b, uint32_t* __restrict__ out_c, int64_t m,
                                                          int64_t row_words, int64_t up_words, DeviceStatus* status) {
    // ENCODE: in_a, in_b = planes 1, 2 -> out_a = base, out_b, out_c = up 1, up 2
    // decode: in_a = base, in_b, in_c = up 1, up 2 -> out_a, out_b = planes 1, 2
    constexpr uint32_t kMask = (1u << CB) - 1u;
    constexpr int PER = 32 / CB;                          // codes of a 32-bit word
    const int64_t total = m * up_words;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
        const int64_t row = i / up_words, uw = i - row * up_words;
        uint32_t u1 = ENCODE ? 0u : in_b[i], u2 = ENCODE ? 0u : in_c[i];
        bool bad = false;
#pragma unroll
        for (int q = 0; q < CB; ++q) {
            const int64_t w = uw * CB + q;                // word of the code planes' row
            if (w < row_words) {
                const int64_t idx = row * row_words + w;
                if (ENCODE) {
                    const uint32_t a = in_a[idx], b = in_b[idx];
                    uint32_t base = 0u;
#pragma unroll
                    for (int k = 0; k < PER; ++k) {
                        const uint32_t c1 = (a >> (k * CB)) & kMask, c2 = (b >> (k * CB)) & kMask;
                        const uint32_t lower = min(c1, c2);
                        bad = bad || c1 - lower > 1u || c2 - lower > 1u;
                        base |= lower << (k * CB);
                        u1 |= (c1 - lower) << (q * PER + k);
                        u2 |= (c2 - lower) << (q * PER + k);
                    }
                    out_a[idx] = base;
                } else {
                    const uint32_t base = in_a[idx];
                    uint32_t p1 = 0u, p2 = 0u;
#pragma unroll
                    for (int k = 0; k < PER; ++k) {
                        const uint32_t lower = (base >> (k * CB)) & kMask;
                        p1 |= ((lower + ((u1 >> (q * PER + k)) & 1u)) & kMask) << (k * CB);
                        p2 |= ((lower + ((u2 >> (q * PER + k)) & 1u)) & kMask) << (k * CB);
                    }
                    out_a[idx] = p1;
                    out_b[idx] = p2;
                }
            }
        }
        if (ENCODE) {
            out_b[i] = u1;
            out_c[i] = u2;
            if (bad) set_status(status, ZIPML_ERR_INVALID_ARG, 60);     // codes two levels apart: not two samples of one value
        }
    }
}

__global__ void shared_base_prepare_kernel(const float* __restrict__ lo, const float* __restrict__ step,
                                           const float* __restrict__ x, int64_t n, float* __restrict__ w, double* __restrict__ base_out) {
    __shared__ double red[40];
    double base = 0.0;
    for (int64_t j = threadIdx.x; j < n; j += blockDim.x) {
        const float xv = x[j];
        w[j] = step[j] * xv;
        base += (double)lo[j] * (double)xv;
    }
    base = block_sum(base, red);
    if (threadIdx.x == 0) *base_out = base;
}

// A warp per row; a lane takes 32 features at a time (one word of each up plane, CB words of the base plane).
template <int CB>
__global__ void __launch_bounds__(256) shared_base_loss_kernel(const uint32_t* __restrict__ base, const uint32_t* __restrict__ up1,
                                                               const uint32_t* __restrict__ up2, int64_t row_words, int64_t up_words,
                                                               int64_t m, int64_t n, const float* __restrict__ w,
                                                               const double* __restrict__ base_in, const float* __restrict__ b,
                                                               double* __restrict__ partials) {
    constexpr uint32_t kMask = (1u << CB) - 1u;
    constexpr int PER = 32 / CB;
    __shared__ double red[40];
    const int lane = threadIdx.x & 31;
    const int64_t warp_global = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int64_t nwarps = ((int64_t)gridDim.x * blockDim.x) >> 5;
    const double lox = *base_in;
    const int64_t groups = (n + 31) / 32;
    double total = 0.0;
    for (int64_t k = warp_global; k < m; k += nwarps) {
        double db = 0.0, d1 = 0.0, d2 = 0.0;
        for (int64_t g = lane; g < groups; g += 32) {
            const uint32_t u1 = __ldg(up1 + k * up_words + g), u2 = __ldg(up2 + k * up_words + g);
            float ab = 0.0f, a1 = 0.0f, a2 = 0.0f;
#pragma unroll
            for (int q = 0; q < CB; ++q) {
                const int64_t wd = g * CB + q;
                const uint32_t cw = wd < row_words ? __ldg(base + k * row_words + wd) : 0u;
#pragma unroll
                for (int i = 0; i < PER; ++i) {
                    const int64_t j = g * 32 + q * PER + i;
                    const float wv = j < n ? __ldg(w + j) : 0.0f;
                    ab = fmaf((float)((cw >> (i * CB)) & kMask), wv, ab);
                    a1 += ((u1 >> (q * PER + i)) & 1u) ? wv : 0.0f;
                    a2 += ((u2 >> (q * PER + i)) & 1u) ? wv : 0.0f;
                }
            }
            db += (double)ab; d1 += (double)a1; d2 += (double)a2;
        }
        db = warp_sum(db); d1 = warp_sum(d1); d2 = warp_sum(d2);
        const double bk = (double)__ldg(b + k);
        if (lane == 0) total += (lox + db + d1 - bk) * (lox + db + d2 - bk);
    }
    total = block_sum(total, red);
    if (threadIdx.x == 0) partials[blockIdx.x] = total;
}

__global__ void shared_base_finish_kernel(const double* __restrict__ partials, int count, double scale, double* out) {
    __shared__ double red[40];
    double v = 0.0;
    for (int i = threadIdx.x; i < count; i += blockDim.x) v += partials[i];
    v = block_sum(v, red);
    if (threadIdx.x == 0) *out = v * scale;
}

static int check_shared_base(const zipml_shared_base* d) {
    if (!d || d->struct_size != sizeof(zipml_shared_base)) return ZIPML_ERR_INVALID_ARG;
    if (container_bits(d->bits) == 0) return ZIPML_ERR_UNSUPPORTED;
    if (d->m <= 0 || d->n <= 0 || d->n > 0x7fffffffLL / 8) return ZIPML_ERR_INVALID_ARG;
    if (!d->base || !d->up1 || !d->up2) return ZIPML_ERR_INVALID_ARG;
    if (((uintptr_t)d->base | (uintptr_t)d->up1 | (uintptr_t)d->up2) & 15) return ZIPML_ERR_INVALID_ARG;
    if (d->row_bytes % 16 != 0 || d->row_bytes < zipml_row_bytes(d->n, d->bits)) return ZIPML_ERR_INVALID_ARG;
    if (d->up_row_bytes % 16 != 0 || d->up_row_bytes < zipml_up_row_bytes(d->n)) return ZIPML_ERR_INVALID_ARG;
    return ZIPML_OK;
}

static int blocks_for(const zipml_ctx* ctx, int64_t units) {
    int64_t blocks = (units + 255) / 256;
    if (blocks > (int64_t)ctx->sm_count * 32) blocks = (int64_t)ctx->sm_count * 32;
    return (int)(blocks < 1 ? 1 : blocks);
}

}  // namespace zipml

using namespace zipml;

extern "C" {

int64_t zipml_up_row_bytes(int64_t n) {
    if (n <= 0) return 0;
    return ((n + 7) / 8 + 15) / 16 * 16;
}

int zipml_shared_base_encode(zipml_ctx* ctx, const zipml_dataset* data, const zipml_shared_base* out) {
    if (!ctx) return ZIPML_ERR_INVALID_ARG;
    int rc = check_dataset(data);
    if (rc != ZIPML_OK) return rc;
    if (data->layout != ZIPML_LAYOUT_ROWS) return ZIPML_ERR_UNSUPPORTED;
    rc = check_shared_base(out);
    if (rc != ZIPML_OK) return rc;
    if (out->bits != data->bits || out->m != data->m || out->n != data->n || out->row_bytes != data->row_bytes) return ZIPML_ERR_INVALID_ARG;
    int prev = -1;
    if (cudaGetDevice(&prev) != cudaSuccess || cudaSetDevice(ctx->device) != cudaSuccess) return cuda_status(cudaGetLastError());
    const int cb = container_bits(data->bits);
    const int64_t rw = data->row_bytes / 4, uw = out->up_row_bytes / 4;
    const uint32_t* p1 = reinterpret_cast<const uint32_t*>(data->plane1);
    const uint32_t* p2 = reinterpret_cast<const uint32_t*>(data->plane2);
    uint32_t* ob = reinterpret_cast<uint32_t*>(const_cast<uint8_t*>(out->base));
    uint32_t* o1 = reinterpret_cast<uint32_t*>(const_cast<uint8_t*>(out->up1));
    uint32_t* o2 = reinterpret_cast<uint32_t*>(const_cast<uint8_t*>(out->up2));
    const int blocks = blocks_for(ctx, data->m * uw);
    if (cb == 2) shared_base_kernel<2, true><<<blocks, 256, 0, ctx->stream>>>(p1, p2, nullptr, ob, o1, o2, data->m, rw, uw, ctx->d_status);
    else if (cb == 4) shared_base_kernel<4, true><<<blocks, 256, 0, ctx->stream>>>(p1, p2, nullptr, ob, o1, o2, data->m, rw, uw, ctx->d_status);
    else shared_base_kernel<8, true><<<blocks, 256, 0, ctx->stream>>>(p1, p2, nullptr, ob, o1, o2, data->m, rw, uw, ctx->d_status);
    ctx->launches += 1;
    rc = cuda_status(cudaGetLastError());
    (void)cudaSetDevice(prev);
    return rc;
}

int zipml_shared_base_decode(zipml_ctx* ctx, const zipml_shared_base* data, uint8_t* plane1, uint8_t* plane2) {
    if (!ctx || !plane1 || !plane2 || (((uintptr_t)plane1 | (uintptr_t)plane2) & 15)) return ZIPML_ERR_INVALID_ARG;
    int rc = check_shared_base(data);
    if (rc != ZIPML_OK) return rc;
    int prev = -1;
    if (cudaGetDevice(&prev) != cudaSuccess || cudaSetDevice(ctx->device) != cudaSuccess) return cuda_status(cudaGetLastError());
    const int cb = container_bits(data->bits);
    const int64_t rw = data->row_bytes / 4, uw = data->up_row_bytes / 4;
    const uint32_t* ib = reinterpret_cast<const uint32_t*>(data->base);
    const uint32_t* i1 = reinterpret_cast<const uint32_t*>(data->up1);
    const uint32_t* i2 = reinterpret_cast<const uint32_t*>(data->up2);
    uint32_t* o1 = reinterpret_cast<uint32_t*>(plane1);
    uint32_t* o2 = reinterpret_cast<uint32_t*>(plane2);
    const int blocks = blocks_for(ctx, data->m * uw);
    if (cb == 2) shared_base_kernel<2, false><<<blocks, 256, 0, ctx->stream>>>(ib, i1, i2, o1, o2, nullptr, data->m, rw, uw, ctx->d_status);
    else if (cb == 4) shared_base_kernel<4, false><<<blocks, 256, 0, ctx->stream>>>(ib, i1, i2, o1, o2, nullptr, data->m, rw, uw, ctx->d_status);
    else shared_base_kernel<8, false><<<blocks, 256, 0, ctx->stream>>>(ib, i1, i2, o1, o2, nullptr, data->m, rw, uw, ctx->d_status);
    ctx->launches += 1;
    rc = cuda_status(cudaGetLastError());
    (void)cudaSetDevice(prev);
    return rc;
}

int zipml_loss_shared_base(zipml_ctx* ctx, const zipml_shared_base* data, const float* b, const float* x, double* loss_out) {
    if (!ctx || !b || !x || !loss_out) return ZIPML_ERR_INVALID_ARG;
    int rc = check_shared_base(data);
    if (rc != ZIPML_OK) return rc;
    if (!data->feat_lo || !data->feat_step) return ZIPML_ERR_INVALID_ARG;
    int prev = -1;
    if (cudaGetDevice(&prev) != cudaSuccess || cudaSetDevice(ctx->device) != cudaSuccess) return cuda_status(cudaGetLastError());
    constexpr int kPartials = 4096;
    rc = ws_reserve(ctx, carve_size(sizeof(double) * (kPartials + 2)) + carve_size(sizeof(float) * (size_t)data->n));
    if (rc == ZIPML_OK) {
        Carver cv(ctx->ws);
        double* partials = cv.take<double>(kPartials + 2);
        float* w = cv.take<float>((size_t)data->n);
        double* lox = partials + kPartials;
        shared_base_prepare_kernel<<<1, 1024, 0, ctx->stream>>>(data->feat_lo, data->feat_step, x, data->n, w, lox);
        int blocks = ctx->sm_count * 8;
        if (blocks > kPartials) blocks = kPartials;
        const int64_t need = (data->m + 7) / 8;
        if (blocks > need) blocks = (int)need;
        const int cb = container_bits(data->bits);
        const int64_t rw = data->row_bytes / 4, uw = data->up_row_bytes / 4;
        const uint32_t* ib = reinterpret_cast<const uint32_t*>(data->base);
        const uint32_t* i1 = reinterpret_cast<const uint32_t*>(data->up1);
        const uint32_t* i2 = reinterpret_cast<const uint32_t*>(data->up2);
        if (cb == 2) shared_base_loss_kernel<2><<<blocks, 256, 0, ctx->stream>>>(ib, i1, i2, rw, uw, data->m, data->n, w, lox, b, partials);
        else if (cb == 4) shared_base_loss_kernel<4><<<blocks, 256, 0, ctx->stream>>>(ib, i1, i2, rw, uw, data->m, data->n, w, lox, b, partials);
        else shared_base_loss_kernel<8><<<blocks, 256, 0, ctx->stream>>>(ib, i1, i2, rw, uw, data->m, data->n, w, lox, b, partials);
        shared_base_finish_kernel<<<1, 256, 0, ctx->stream>>>(partials, blocks, 1.0 / (2.0 * (double)data->m), loss_out);
        ctx->launches += 3;
        rc = cuda_status(cudaGetLastError());
    }
    (void)cudaSetDevice(prev);
    return rc;
}

int zipml_sgd_epoch_shared_base(zipml_ctx* ctx, const zipml_shared_base* data, const float* b, float* x,
                                const zipml_sgd_params* params, float* grad_out) {
    if (!ctx) return ZIPML_ERR_INVALID_ARG;
    int rc = check_shared_base(data);
    if (rc != ZIPML_OK) return rc;
    if (!data->feat_lo || !data->feat_step) return ZIPML_ERR_INVALID_ARG;
    // the epoch engines read two planes: they are rebuilt in the context's staging buffer (kept until the next call)
    const size_t plane_bytes = (size_t)data->m * (size_t)data->row_bytes;
    rc = stage_reserve(ctx, 2 * carve_size(plane_bytes));
    if (rc != ZIPML_OK) return rc;
    uint8_t* p1 = ctx->stage;
    uint8_t* p2 = ctx->stage + carve_size(plane_bytes);
    rc = zipml_shared_base_decode(ctx, data, p1, p2);
    if (rc != ZIPML_OK) return rc;
    zipml_dataset d{};
    d.struct_size = sizeof(zipml_dataset);
    d.bits = data->bits; d.level_mode = ZIPML_LEVELS_UNIFORM; d.layout = ZIPML_LAYOUT_ROWS;
    d.m = data->m; d.n = data->n; d.row_bytes = data->row_bytes;
    d.plane1 = p1; d.plane2 = p2; d.feat_lo = data->feat_lo; d.feat_step = data->feat_step; d.levels = nullptr;
    return zipml_sgd_epoch(ctx, &d, b, x, params, grad_out);
}

}  // extern "C"
