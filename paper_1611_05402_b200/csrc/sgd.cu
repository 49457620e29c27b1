// Mini-batch SGD over double-sampled packed codes (Supplement "Double Sampling", footnote form;
// "End-to-end Quantization").
//
// Decomposition.  A minibatch tile (B rows x n features, two planes) is cut into na feature
// parts x nb row parts; CTA (ai, bi) owns one piece for the whole call and keeps its slice of the
// model in shared memory.  Per step:
//   phase A  partial dots of the CTA's rows over its features, both planes.  With na == 1 the dots
//            are complete and become residuals on the spot; otherwise they go to pd (global) and
//            a grid barrier follows.
//   phase B  residuals of its rows; partial gradient of its features over its rows -> pg, ps (global)
//   barrier  (only if more than one CTA)
//   phase C  every CTA sums the row parts of its own features in a fixed order, applies the
//            optional gradient quantizer and updates its model slice.  CTAs that share a feature
//            part do this redundantly and reach bit-identical slices, so no model exchange and no
//            further barrier is needed.
// For a uniform grid value = lo_j + code * step_j, so with w_j = step_j * x_j
//   q^T x = sum_j lo_j x_j + sum_j code_j w_j,
//   g_j   = [ lo_j * sum_k (r1_k + r2_k) + step_j * sum_k (c1_kj r2_k + c2_kj r1_k) ] / (2 B_t),
// i.e. both phases contract raw integer codes with an fp32 vector.  Level tables use lookups into
// per-step tables level*x (phase A) and level (phase B) laid out [code][slot][word] so that a warp
// reading consecutive words is bank-conflict free.
//
// Staging.  The codes a step needs do not depend on the model, only the arithmetic does.  When a
// CTA's tile fits, a ring of shared-memory stages is filled by bulk asynchronous copies
// (cp.async.bulk, completion on an mbarrier) several steps ahead, so that the HBM latency is off
// the step-to-step dependency chain and phase B re-reads the tile from shared memory.
//
// Accuracy: fp32 lane partials over short runs, combined in double across lanes, warps and CTAs.
// Determinism: every reduction has a fixed order; no floating-point atomics.
//
// The same kernel runs "stepwise" (one launch per phase, kernel boundaries as barriers, model in
// global memory) or "persistent" (one cooperative launch, bounded-spin grid barriers).
#include "sgd_common.cuh"

namespace zipml {

// Diagnostic: `iterations` grid barriers back to back, each preceded by a small exchange through L2
// (every CTA publishes `floats` floats and reads one float4 of every other CTA's), which is the
// communication skeleton of one SGD step.  CTA 0 records the elapsed nanoseconds.
__global__ void __launch_bounds__(kSgdThreads) barrier_latency_kernel(unsigned* counter, float* scratch, int floats,
                                                                      int iterations, DeviceStatus* status,
                                                                      unsigned long long* ns_out) {
    const int G = gridDim.x;
    unsigned long long t0 = 0;
    if (blockIdx.x == 0 && threadIdx.x == 0) asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t0));
    float sink = 0.0f;
    for (int it = 0; it < iterations; ++it) {
        float* mine = scratch + ((size_t)(it & 1) * G + blockIdx.x) * floats;
        for (int i = threadIdx.x; i < floats; i += kSgdThreads) __stcg(mine + i, (float)(it + i));
        if (!grid_barrier(counter, (unsigned)G * (unsigned)(it + 1), status, 4)) return;
        if (floats >= 4)
            for (int p = threadIdx.x; p < G; p += kSgdThreads)
                sink += __ldcg(reinterpret_cast<const float4*>(scratch + ((size_t)(it & 1) * G + p) * floats)).x;
    }
    if (sink == -1.0f) scratch[0] = sink;
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        unsigned long long t1;
        asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t1));
        *ns_out = t1 - t0;
    }
}

int launch_barrier_latency(zipml_ctx* ctx, int ctas, int floats, int iterations, unsigned long long* ns_out_dev) {
    const size_t bytes = carve_size(sizeof(unsigned) * 4) + carve_size(sizeof(float) * 2 * (size_t)ctas * (floats > 0 ? floats : 1));
    int rc = ws_reserve(ctx, bytes);
    if (rc != ZIPML_OK) return rc;
    unsigned* counter = reinterpret_cast<unsigned*>(ctx->ws);
    float* scratch = reinterpret_cast<float*>(ctx->ws + carve_size(sizeof(unsigned) * 4));
    int per_sm = 0;
    cudaError_t e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, barrier_latency_kernel, kSgdThreads, 0);
    if (e != cudaSuccess) return cuda_status(e);
    if (!ctx->cooperative || ctas > per_sm * ctx->sm_count) return ZIPML_ERR_WORKSPACE;
    e = cudaMemsetAsync(counter, 0, sizeof(unsigned) * 4, ctx->stream);
    if (e != cudaSuccess) return cuda_status(e);
    DeviceStatus* status = ctx->d_status;
    void* params[] = {&counter, &scratch, &floats, &iterations, &status, &ns_out_dev};
    e = cudaLaunchCooperativeKernel((const void*)barrier_latency_kernel, dim3((unsigned)ctas), dim3(kSgdThreads), params, 0,
                                    ctx->stream);
    if (e != cudaSuccess) return cuda_status(e);
    ctx->launches += 1;
    return ZIPML_OK;
}

// Shared memory plan, F = wc * FPW features per CTA:
//   red[40] double            block reductions
//   dpart[2*kSgdWarps] double per-(row, segment) partial dots when a row is split over warps
//   mbar[kMaxStages] u64      "stage filled" barriers
//   xs[F] float               model slice
//   tab float                 uniform: w[F], layout [u][word][4] (u-th float4 of a word);
//                             table: WL[L*F] = level*x then LV[L*F] = level, layout [code][slot][word];
//                             tab[0..F) doubles as the gradient slice in phase C
//   gred[kSgdThreads*FPW]     cross-group reduction of phase B
//   res[2*rc]                 residuals r1, r2 of the CTA's rows
//   tiles[stages][2][rc][wc]  u32, STAGED only
template <int CB, bool TABLE, bool STAGED>
__global__ void __launch_bounds__(kSgdThreads) sgd_kernel(const SgdArgs a) {
    constexpr int FPW = 32 / CB;
    extern __shared__ __align__(16) unsigned char s_raw[];
    const int L = 1 << a.bits;
    const int F = a.wc * FPW;
    double* red = reinterpret_cast<double*>(s_raw);
    double* dpart = red + 40;
    uint64_t* mbar = reinterpret_cast<uint64_t*>(dpart + 2 * kSgdWarps);
    float* xs = reinterpret_cast<float*>(mbar + kMaxStages);
    float* tab = xs + F;
    float* gred = tab + (TABLE ? 2 * L * F : F);
    float* res = gred + kSgdThreads * FPW;
    uint32_t* tiles = reinterpret_cast<uint32_t*>(res + ((2 * a.rc + 3) & ~3));
    float* gs = tab;

    const int ai = blockIdx.x % a.na, bi = blockIdx.x / a.na;
    const int G = a.na * a.nb;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t words_needed = (a.n + FPW - 1) / FPW;
    const int64_t w0 = (int64_t)ai * a.wc;                        // first word of this feature part
    const int wcnt = (int)max((int64_t)0, min((int64_t)a.wc, words_needed - w0));
    const int wcopy = (wcnt + 3) & ~3;                            // words copied per row: 16-byte multiples
    const int64_t j0 = w0 * FPW;                                  // first feature
    const int fcnt = (int)max((int64_t)0, min((int64_t)F, a.n - j0));
    const int64_t npad = (int64_t)a.na * F;
    const int k0 = bi * a.rc;                                     // first batch-local row of this CTA
    unsigned barriers_done = 0;
    const size_t stage_words = (size_t)2 * a.rc * a.wc;

    // rows of the CTA in the step at position `it`
    auto step_rows = [&](int64_t it, int64_t& r0, int& bt, int& rcnt) {
        const int64_t t = a.order ? (int64_t)a.order[it] : it;
        r0 = t * a.batch;
        bt = (int)min(a.batch, a.m - r0);
        rcnt = max(0, min(a.rc, bt - k0));
    };
    // warp 0 starts the copies of one step's tile into its stage
    auto issue_copies = [&](int64_t it) {
        if constexpr (STAGED) {
            const int sl = (int)(it - a.first_step);
            uint64_t* bar = mbar + (sl % a.stages);
            uint32_t* dst = tiles + (size_t)(sl % a.stages) * stage_words;
            int64_t r0; int bt, rcnt;
            step_rows(it, r0, bt, rcnt);
            const uint32_t row_bytes = (uint32_t)wcopy * 4u;
            if (lane == 0) {
                if (rcnt > 0 && wcopy > 0) mbar_arrive_expect_tx(bar, 2u * (uint32_t)rcnt * row_bytes);
                else mbar_arrive(bar);
            }
            __syncwarp();
            if (rcnt > 0 && wcopy > 0) {
                const bool contiguous = (a.row_words == a.wc) && (wcopy == a.wc);
                if (contiguous) {
                    if (lane < 2) {
                        const uint32_t* src = (lane == 0 ? a.p1 : a.p2) + (r0 + k0) * a.row_words;
                        bulk_copy_g2s(dst + (size_t)lane * a.rc * a.wc, src, (uint32_t)rcnt * row_bytes, bar);
                    }
                } else {
                    for (int i = lane; i < 2 * rcnt; i += 32) {
                        const int plane = i & 1, r = i >> 1;
                        const uint32_t* src = (plane == 0 ? a.p1 : a.p2) + (r0 + k0 + r) * a.row_words + w0;
                        bulk_copy_g2s(dst + ((size_t)plane * a.rc + r) * a.wc, src, row_bytes, bar);
                    }
                }
            }
        }
    };

    if constexpr (STAGED) {
        if (threadIdx.x == 0) {
            for (int s = 0; s < a.stages; ++s) mbar_init(mbar + s, 1);
            mbar_fence_init();
        }
    }
    if (a.persistent || (a.phases & (kPhaseA | kPhaseC))) {
        for (int f = threadIdx.x; f < F; f += kSgdThreads) xs[f] = (f < fcnt) ? a.x[j0 + f] : 0.0f;
    }
    if (TABLE && (a.persistent || (a.phases & kPhaseB))) {
        float* LV = tab + L * F;
        for (int idx = threadIdx.x; idx < L * F; idx += kSgdThreads) {
            const int q = idx % a.wc, ci = idx / a.wc, i = ci % FPW, c = ci / FPW;
            const int f = q * FPW + i;
            LV[idx] = (f < fcnt) ? __ldg(a.levels + (j0 + f) * L + c) : 0.0f;
        }
    }
    __syncthreads();
    if constexpr (STAGED) {
        if (warp == 0)
            for (int64_t it = a.first_step; it < a.first_step + min((int64_t)(a.stages - 1), a.num_steps); ++it) issue_copies(it);
    }

    for (int64_t it = a.first_step; it < a.first_step + a.num_steps; ++it) {
        int64_t r0; int bt, rcnt;
        step_rows(it, r0, bt, rcnt);
        const int par = (int)(it & 1);
        double* pd = a.pd + (size_t)par * a.na * a.batch * 2;
        float* pg = a.pg + (size_t)par * a.nb * npad;
        double* ps = a.ps + (size_t)par * a.nb;
        const bool last = (it == a.first_step + a.num_steps - 1);
        const int sl = (int)(it - a.first_step);
        const uint32_t* tile1 = nullptr;
        const uint32_t* tile2 = nullptr;
        if constexpr (STAGED) {
            // the stage freed by the previous step takes the tile of step it + stages - 1
            if (warp == 0 && it + a.stages - 1 < a.first_step + a.num_steps) issue_copies(it + a.stages - 1);
            tile1 = tiles + (size_t)(sl % a.stages) * stage_words;
            tile2 = tile1 + (size_t)a.rc * a.wc;
        }
        auto row_of = [&](int plane, int r) -> const uint32_t* {
            if constexpr (STAGED) return (plane == 0 ? tile1 : tile2) + (size_t)r * a.wc;
            else return (plane == 0 ? a.p1 : a.p2) + (r0 + k0 + r) * a.row_words + w0;
        };
        auto load_code = [&](const uint32_t* p) -> uint32_t {
            if constexpr (STAGED) return *p;
            else return __ldg(p);
        };
        const bool dots_local = (a.na == 1 && a.phases == kPhaseAll);

        // ------------------------------------------------------------------ phase A: dots
        if (a.phases & kPhaseA) {
            VecQuant q3{0.0f, 1, a.seed, a.epoch, (uint32_t)it, 3u};
            if (a.model_bits > 0) { q3.M = vector_scale_smem(xs, F, red, a.vector_norm); q3.sm = (1 << (a.model_bits - 1)) - 1; }
            double base = 0.0;
            if constexpr (!TABLE) {
                for (int q = threadIdx.x; q < a.wc; q += kSgdThreads) {
#pragma unroll
                    for (int i = 0; i < FPW; ++i) {
                        const int f = q * FPW + i;
                        float xv = xs[f];
                        if (a.model_bits > 0) xv = q3.apply(xv, (uint32_t)(j0 + f));
                        if (a.model_out && last && bi == 0 && f < fcnt) a.model_out[j0 + f] = xv;
                        float sv = 0.0f, lv = 0.0f;
                        if (f < fcnt) { sv = __ldg(a.step + j0 + f); lv = __ldg(a.lo + j0 + f); }
                        tab[((i >> 2) * a.wc + q) * 4 + (i & 3)] = sv * xv;
                        base += (double)lv * (double)xv;
                    }
                }
                base = block_sum(base, red);   // ends with a barrier: w is complete
            } else {
                for (int f = threadIdx.x; f < F; f += kSgdThreads) {
                    float xv = xs[f];
                    if (a.model_bits > 0) xv = q3.apply(xv, (uint32_t)(j0 + f));
                    if (a.model_out && last && bi == 0 && f < fcnt) a.model_out[j0 + f] = xv;
                    const int q = f / FPW, i = f % FPW;
                    for (int c = 0; c < L; ++c) {
                        const float lv = (f < fcnt) ? __ldg(a.levels + (j0 + f) * L + c) : 0.0f;
                        tab[(c * FPW + i) * a.wc + q] = lv * xv;
                    }
                }
                __syncthreads();
            }
            if constexpr (STAGED) {
                // wait for this step's tile (bounded)
                const uint32_t parity = (uint32_t)((sl / a.stages) & 1);
                bool got = false;
                for (long long spin = 0; spin < kCopySpinLimit; ++spin)
                    if (mbar_try_wait(mbar + (sl % a.stages), parity)) { got = true; break; }
                if (__syncthreads_or(!got)) {
                    if (threadIdx.x == 0) set_status(a.status, ZIPML_ERR_TIMEOUT, 3);
                    return;
                }
            }

            // tasks = rows x segments; a row is split over S warps when the CTA has fewer rows than warps
            const int chunks = (wcnt + 31) / 32;
            int S = 1;
            if (rcnt > 0 && rcnt < kSgdWarps) S = max(1, min(chunks, kSgdWarps / rcnt));
            const int cps = (chunks + S - 1) / S;
            const int ntasks = rcnt * S;
            for (int task = warp; task < ntasks; task += kSgdWarps) {
                const int r = task / S, seg = task - r * S;
                const uint32_t* row1 = row_of(0, r);
                const uint32_t* row2 = row_of(1, r);
                float acc1[2] = {0.0f, 0.0f}, acc2[2] = {0.0f, 0.0f};
                const int c_end = min(chunks, (seg + 1) * cps);
#pragma unroll 4
                for (int c = seg * cps; c < c_end; ++c) {
                    const int q = c * 32 + lane;
                    if (q < wcnt) {
                        const uint32_t u1 = load_code(row1 + q), u2 = load_code(row2 + q);
                        if constexpr (!TABLE) {
                            float c1[FPW], c2[FPW];
                            unpack_word<CB>(u1, c1);
                            unpack_word<CB>(u2, c2);
#pragma unroll
                            for (int u = 0; u < FPW / 4; ++u) {
                                const float4 wv = *reinterpret_cast<const float4*>(tab + (u * a.wc + q) * 4);
                                acc1[u & 1] = fmaf(c1[4 * u + 0], wv.x, acc1[u & 1]);
                                acc1[u & 1] = fmaf(c1[4 * u + 1], wv.y, acc1[u & 1]);
                                acc1[u & 1] = fmaf(c1[4 * u + 2], wv.z, acc1[u & 1]);
                                acc1[u & 1] = fmaf(c1[4 * u + 3], wv.w, acc1[u & 1]);
                                acc2[u & 1] = fmaf(c2[4 * u + 0], wv.x, acc2[u & 1]);
                                acc2[u & 1] = fmaf(c2[4 * u + 1], wv.y, acc2[u & 1]);
                                acc2[u & 1] = fmaf(c2[4 * u + 2], wv.z, acc2[u & 1]);
                                acc2[u & 1] = fmaf(c2[4 * u + 3], wv.w, acc2[u & 1]);
                            }
                        } else {
#pragma unroll
                            for (int i = 0; i < FPW; ++i) {
                                acc1[i & 1] += tab[(code_at<CB>(u1, i) * FPW + i) * a.wc + q];
                                acc2[i & 1] += tab[(code_at<CB>(u2, i) * FPW + i) * a.wc + q];
                            }
                        }
                    }
                }
                const double d1 = warp_sum((double)acc1[0] + (double)acc1[1]);
                const double d2 = warp_sum((double)acc2[0] + (double)acc2[1]);
                if (lane == 0) {
                    if (S > 1) {
                        dpart[2 * task] = d1;
                        dpart[2 * task + 1] = d2;
                    } else if (dots_local) {
                        const double bk = (double)__ldg(a.b + r0 + k0 + r);
                        res[2 * r] = (float)(d1 + base - bk);
                        res[2 * r + 1] = (float)(d2 + base - bk);
                    } else {
                        __stcg(pd + ((size_t)ai * a.batch + k0 + r) * 2 + 0, d1 + base);
                        __stcg(pd + ((size_t)ai * a.batch + k0 + r) * 2 + 1, d2 + base);
                    }
                }
            }
            if (S > 1) {
                __syncthreads();
                if (threadIdx.x < rcnt) {
                    const int r = threadIdx.x;
                    double d1 = base, d2 = base;
                    for (int sg = 0; sg < S; ++sg) { d1 += dpart[2 * (r * S + sg)]; d2 += dpart[2 * (r * S + sg) + 1]; }
                    if (dots_local) {
                        const double bk = (double)__ldg(a.b + r0 + k0 + r);
                        res[2 * r] = (float)(d1 - bk);
                        res[2 * r + 1] = (float)(d2 - bk);
                    } else {
                        __stcg(pd + ((size_t)ai * a.batch + k0 + r) * 2 + 0, d1);
                        __stcg(pd + ((size_t)ai * a.batch + k0 + r) * 2 + 1, d2);
                    }
                }
            }
        }
        if (a.persistent && a.na > 1) {
            ++barriers_done;
            if (!grid_barrier(a.barrier, (unsigned)G * barriers_done, a.status, 1)) return;
        } else {
            __syncthreads();
        }

        // ------------------------------------------------------------------ phase B: gradient
        if (a.phases & kPhaseB) {
            double ssum = 0.0;
            for (int r = threadIdx.x; r < rcnt; r += kSgdThreads) {
                float r1, r2;
                if (dots_local) {
                    r1 = res[2 * r];
                    r2 = res[2 * r + 1];
                } else {
                    double d1 = 0.0, d2 = 0.0;
                    for (int p = 0; p < a.na; ++p) {
                        d1 += __ldcg(pd + ((size_t)p * a.batch + k0 + r) * 2 + 0);
                        d2 += __ldcg(pd + ((size_t)p * a.batch + k0 + r) * 2 + 1);
                    }
                    const double bk = (double)__ldg(a.b + r0 + k0 + r);
                    r1 = (float)(d1 - bk);
                    r2 = (float)(d2 - bk);
                    res[2 * r] = r1;
                    res[2 * r + 1] = r2;
                }
                ssum += (double)r1 + (double)r2;
            }
            ssum = block_sum(ssum, red);       // ends with a barrier: residuals are complete
            if (threadIdx.x == 0 && ai == 0) __stcg(ps + bi, ssum);

            const int lanes_q = min(kSgdThreads, ((wcnt + 31) / 32) * 32);
            const int ngroups = lanes_q > 0 ? kSgdThreads / lanes_q : 1;
            const int group = lanes_q > 0 ? threadIdx.x / lanes_q : 0;
            const int ql = lanes_q > 0 ? threadIdx.x % lanes_q : 0;
            const float* LV = tab + L * F;
            for (int qb = 0; qb < wcnt; qb += lanes_q) {
                const int q = qb + ql;
                const bool active = (group < ngroups) && (q < wcnt);
                float acc[FPW];
#pragma unroll
                for (int i = 0; i < FPW; ++i) acc[i] = 0.0f;
                if (active) {
                    const uint32_t* col1 = row_of(0, 0) + q;
                    const uint32_t* col2 = row_of(1, 0) + q;
                    const int64_t pitch = STAGED ? (int64_t)a.wc : a.row_words;
#pragma unroll 4
                    for (int r = group; r < rcnt; r += ngroups) {
                        const uint32_t u1 = load_code(col1 + (int64_t)r * pitch);
                        const uint32_t u2 = load_code(col2 + (int64_t)r * pitch);
                        const float r1 = res[2 * r], r2 = res[2 * r + 1];
                        if constexpr (!TABLE) {
                            float c1[FPW], c2[FPW];
                            unpack_word<CB>(u1, c1);
                            unpack_word<CB>(u2, c2);
#pragma unroll
                            for (int i = 0; i < FPW; ++i) acc[i] = fmaf(c1[i], r2, fmaf(c2[i], r1, acc[i]));
                        } else {
#pragma unroll
                            for (int i = 0; i < FPW; ++i) {
                                const float l1 = LV[(code_at<CB>(u1, i) * FPW + i) * a.wc + q];
                                const float l2 = LV[(code_at<CB>(u2, i) * FPW + i) * a.wc + q];
                                acc[i] = fmaf(l1, r2, fmaf(l2, r1, acc[i]));
                            }
                        }
                    }
                }
                if (ngroups > 1) {
                    __syncthreads();
                    if (active) {
#pragma unroll
                        for (int i = 0; i < FPW; ++i) gred[(group * FPW + i) * lanes_q + ql] = acc[i];
                    }
                    __syncthreads();
                    if (active && group == 0) {
#pragma unroll
                        for (int i = 0; i < FPW; ++i) {
                            float tsum = gred[i * lanes_q + ql];
                            for (int gidx = 1; gidx < ngroups; ++gidx) tsum += gred[(gidx * FPW + i) * lanes_q + ql];
                            acc[i] = tsum;
                        }
                    }
                }
                if (active && group == 0) {
                    float4* dst = reinterpret_cast<float4*>(pg + (size_t)bi * npad + (size_t)(w0 + q) * FPW);
#pragma unroll
                    for (int u = 0; u < FPW / 4; ++u) __stcg(dst + u, make_float4(acc[4 * u], acc[4 * u + 1], acc[4 * u + 2], acc[4 * u + 3]));
                }
            }
        }
        if (a.persistent && G > 1) {
            ++barriers_done;
            if (!grid_barrier(a.barrier, (unsigned)G * barriers_done, a.status, 2)) return;
        } else {
            __syncthreads();
        }

        // ------------------------------------------------------------------ phase C: reduce, update
        if (a.phases & kPhaseC) {
            double ssum = 0.0;
            if constexpr (!TABLE) {
                for (int p = 0; p < a.nb; ++p) ssum += __ldcg(ps + p);
            }
            const double scale = 1.0 / (2.0 * (double)bt);
            for (int f4 = threadIdx.x; f4 < F / 4; f4 += kSgdThreads) {
                const int f = 4 * f4;
                float g[4] = {0.0f, 0.0f, 0.0f, 0.0f};
                if (f < fcnt) {
                    double acc[4] = {0.0, 0.0, 0.0, 0.0};
                    const float4* src = reinterpret_cast<const float4*>(pg + j0 + f);
#pragma unroll 8
                    for (int p = 0; p < a.nb; ++p) {
                        const float4 v = __ldcg(src + (size_t)p * (npad / 4));
                        acc[0] += (double)v.x; acc[1] += (double)v.y; acc[2] += (double)v.z; acc[3] += (double)v.w;
                    }
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        if (f + e < fcnt) {
                            double v = acc[e];
                            if constexpr (!TABLE) v = (double)__ldg(a.lo + j0 + f + e) * ssum + (double)__ldg(a.step + j0 + f + e) * v;
                            g[e] = (float)(v * scale);
                            if (last && a.grad_out && bi == 0) a.grad_out[j0 + f + e] = g[e];
                        }
                    }
                }
                *reinterpret_cast<float4*>(gs + f) = make_float4(g[0], g[1], g[2], g[3]);
            }
            __syncthreads();
            VecQuant q4{0.0f, 1, a.seed, a.epoch, (uint32_t)it, 4u};
            if (a.grad_bits > 0) { q4.M = vector_scale_smem(gs, F, red, a.vector_norm); q4.sm = (1 << (a.grad_bits - 1)) - 1; }
            for (int f = threadIdx.x; f < fcnt; f += kSgdThreads) {
                float g = gs[f];
                if (a.grad_bits > 0) g = q4.apply(g, (uint32_t)(j0 + f));
                if (last && a.grad_out && bi == 0) a.grad_out[a.n + j0 + f] = g;
                xs[f] = regularise(fmaf(-a.lr, g, xs[f]), xs[f], a.reg, a.reg_cst);
            }
            __syncthreads();
            if (!a.persistent && bi == 0)
                for (int f = threadIdx.x; f < fcnt; f += kSgdThreads) a.x[j0 + f] = xs[f];
        }
    }
    if (a.persistent && bi == 0)
        for (int f = threadIdx.x; f < fcnt; f += kSgdThreads) a.x[j0 + f] = xs[f];
}

// ---------------------------------------------------------------------------------------------
// Host side: partition plan, workspace, launches
// ---------------------------------------------------------------------------------------------
struct SgdPlan {
    int na, nb, wc, rc;
    int stages;             // 0: codes are read straight from global memory
    size_t smem;
};

static size_t sgd_smem_bytes(int cb, bool table, int wc, int rc, int bits, int stages) {
    const int fpw = 32 / cb;
    const size_t F = (size_t)wc * fpw, L = (size_t)1 << bits;
    size_t bytes = sizeof(double) * (40 + 2 * kSgdWarps) + sizeof(uint64_t) * kMaxStages;
    bytes += sizeof(float) * (F + (table ? 2 * L * F : F) + (size_t)kSgdThreads * fpw + (size_t)((2 * rc + 3) & ~3));
    bytes += sizeof(uint32_t) * (size_t)stages * 2 * rc * wc;
    return bytes;
}

template <bool STAGED>
static const void* sgd_kernel_ptr(int cb, bool table) {
    if (cb == 2) return table ? (const void*)sgd_kernel<2, true, STAGED> : (const void*)sgd_kernel<2, false, STAGED>;
    if (cb == 4) return table ? (const void*)sgd_kernel<4, true, STAGED> : (const void*)sgd_kernel<4, false, STAGED>;
    return (const void*)sgd_kernel<8, false, STAGED>;
}

static int round_up(int v, int q) { return (v + q - 1) / q * q; }

// Chooses the CTA grid.  Feature parts are the fewest that fit shared memory unless the exchange
// volume (na * 2B doubles of dots + nb * n floats of gradient per step) says otherwise; row parts
// fill the remaining CTAs while every CTA keeps at least a warp's worth of rows.  If a CTA's tile
// fits shared memory at least twice, the codes are staged through a ring of up to kMaxStages.
static int make_plan(const zipml_ctx* ctx, const zipml_dataset* d, const zipml_sgd_params* p, bool stepwise, SgdPlan* plan) {
    const int cb = container_bits(d->bits);
    const bool table = d->level_mode == ZIPML_LEVELS_TABLE;
    const int fpw = 32 / cb;
    const int64_t words = (d->n + fpw - 1) / fpw;
    const int64_t B = p->batch < d->m ? p->batch : d->m;
    const size_t smem_cap = (size_t)ctx->smem_optin;
    const bool need_full = p->model_bits > 0 || p->grad_bits > 0;
    const int sms = ctx->sm_count > 0 ? ctx->sm_count : 1;

    auto fits = [&](int na, int nb, int* wc_out, int* rc_out, size_t* smem_out) {
        const int wc = round_up((int)((words + na - 1) / na), 32);
        const int rc = (int)((B + nb - 1) / nb);
        const size_t s = sgd_smem_bytes(cb, table, wc, rc, d->bits, 0);
        *wc_out = wc; *rc_out = rc; *smem_out = s;
        return s <= smem_cap;
    };
    int best_na = 0, best_nb = 0;
    if (p->grid_feature_parts > 0 || p->grid_row_parts > 0) {
        best_na = p->grid_feature_parts > 0 ? p->grid_feature_parts : 1;
        best_nb = p->grid_row_parts > 0 ? p->grid_row_parts : 1;
        if ((int64_t)best_na * 32 > round_up((int)words, 32)) best_na = (int)((words + 31) / 32);
        if (best_nb > B) best_nb = (int)B;
    } else {
        double best_cost = 0.0;
        const int na_max = (int)((words + 31) / 32);
        for (int na = 1; na <= na_max && na <= sms; ++na) {
            if (need_full && na > 1) break;
            int nb = sms / na;
            const int64_t nb_rows = (B + kSgdWarps - 1) / kSgdWarps;     // at least a warp's worth of rows each
            if (nb > nb_rows) nb = (int)nb_rows;
            if (nb < 1) nb = 1;
            int wc, rc; size_t s;
            if (!fits(na, nb, &wc, &rc, &s)) continue;
            // per-step critical path model: streamed bytes per CTA + exchanged bytes + barrier count
            const double tile = 2.0 * (double)rc * wc * 4.0;
            const double exch = (na > 1 ? (double)na * 2.0 * (double)B * 8.0 : 0.0) + (double)nb * (double)d->n * 4.0 / na;
            const double cost = tile + 0.25 * exch + (na > 1 ? 65536.0 : 0.0);
            if (best_na == 0 || cost < best_cost) { best_cost = cost; best_na = na; best_nb = nb; }
        }
        if (best_na == 0) return ZIPML_ERR_WORKSPACE;
    }
    if (need_full && best_na > 1) return ZIPML_ERR_WORKSPACE;
    int wc, rc; size_t s;
    if (!fits(best_na, best_nb, &wc, &rc, &s)) return ZIPML_ERR_WORKSPACE;
    plan->na = best_na; plan->nb = best_nb; plan->wc = wc; plan->rc = rc; plan->smem = s; plan->stages = 0;
    if (!stepwise) {
        // mbarrier transaction counts stay below 2^20 bytes per stage
        const size_t stage_bytes = sizeof(uint32_t) * 2 * (size_t)rc * wc;
        for (int st = kMaxStages; st >= 2; --st) {
            const size_t total = sgd_smem_bytes(cb, table, wc, rc, d->bits, st);
            if (total <= smem_cap && stage_bytes < (1u << 20)) { plan->stages = st; plan->smem = total; break; }
        }
    }
    return ZIPML_OK;
}

struct SgdScratch {
    size_t pd_off, pg_off, ps_off, bar_off, order_off, total;
};

static SgdScratch sgd_scratch(const zipml_dataset* d, const zipml_sgd_params* p, const SgdPlan& plan, int64_t T) {
    const int fpw = 32 / container_bits(d->bits);
    const int64_t B = p->batch < d->m ? p->batch : d->m;
    SgdScratch s;
    size_t off = 0;
    s.pd_off = off; off += carve_size(sizeof(double) * 2 * (size_t)plan.na * (size_t)B * 2);
    s.pg_off = off; off += carve_size(sizeof(float) * 2 * (size_t)plan.nb * (size_t)plan.na * plan.wc * fpw);
    s.ps_off = off; off += carve_size(sizeof(double) * 2 * (size_t)plan.nb);
    s.bar_off = off; off += carve_size(sizeof(unsigned) * 4);
    s.order_off = off; off += carve_size(sizeof(int32_t) * (size_t)(p->batch_order ? T : 0));
    s.total = off;
    return s;
}

int launch_sgd_epoch(zipml_ctx* ctx, const zipml_dataset* d, const float* b, float* x, const zipml_sgd_params* p,
                     int64_t first_step, int64_t num_steps, float* grad_out) {
    const int cb = container_bits(d->bits);
    const bool table = d->level_mode == ZIPML_LEVELS_TABLE;
    const int64_t T = (d->m + p->batch - 1) / p->batch;

    // decide the engine: persistent needs every CTA of the grid resident at once
    SgdPlan plan;
    int engine = p->engine;
    int rc = make_plan(ctx, d, p, engine == ZIPML_ENGINE_STEPWISE, &plan);
    if (rc != ZIPML_OK) return rc;
    const void* kernel = plan.stages > 0 ? sgd_kernel_ptr<true>(cb, table) : sgd_kernel_ptr<false>(cb, table);
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)plan.smem);
    if (e != cudaSuccess) return cuda_status(e);
    int G = plan.na * plan.nb;
    if (engine != ZIPML_ENGINE_STEPWISE) {
        int per_sm = 0;
        e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, kSgdThreads, plan.smem);
        if (e != cudaSuccess) return cuda_status(e);
        const bool can_persist = ctx->cooperative && per_sm > 0 && G <= per_sm * ctx->sm_count;
        if (!can_persist) {
            if (engine == ZIPML_ENGINE_PERSISTENT) return ZIPML_ERR_WORKSPACE;
            engine = ZIPML_ENGINE_STEPWISE;
            rc = make_plan(ctx, d, p, true, &plan);
            if (rc != ZIPML_OK) return rc;
            kernel = sgd_kernel_ptr<false>(cb, table);
            e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)plan.smem);
            if (e != cudaSuccess) return cuda_status(e);
            G = plan.na * plan.nb;
        } else {
            engine = ZIPML_ENGINE_PERSISTENT;
        }
    }
    const SgdScratch sc = sgd_scratch(d, p, plan, T);
    rc = ws_reserve(ctx, sc.total);
    if (rc != ZIPML_OK) return rc;

    SgdArgs a;
    a.p1 = reinterpret_cast<const uint32_t*>(d->plane1);
    a.p2 = reinterpret_cast<const uint32_t*>(d->plane2);
    a.row_words = d->row_bytes / 4;
    a.m = d->m; a.n = d->n; a.bits = d->bits;
    a.lo = d->feat_lo; a.step = d->feat_step; a.levels = d->levels;
    a.b = b; a.x = x; a.grad_out = grad_out; a.model_out = p->model_out;
    a.batch = p->batch < d->m ? p->batch : d->m;
    a.first_step = first_step; a.num_steps = num_steps;
    a.lr = p->lr; a.reg = p->reg; a.reg_cst = reg_constant(p); a.model_bits = p->model_bits; a.grad_bits = p->grad_bits; a.vector_norm = p->vector_norm;
    a.seed = p->seed; a.epoch = (uint32_t)p->epoch;
    a.na = plan.na; a.nb = plan.nb; a.wc = plan.wc; a.rc = plan.rc; a.stages = plan.stages;
    a.pd = reinterpret_cast<double*>(ctx->ws + sc.pd_off);
    a.pg = reinterpret_cast<float*>(ctx->ws + sc.pg_off);
    a.ps = reinterpret_cast<double*>(ctx->ws + sc.ps_off);
    a.barrier = reinterpret_cast<unsigned*>(ctx->ws + sc.bar_off);
    a.status = ctx->d_status;
    a.order = nullptr;
    a.phases = kPhaseAll; a.persistent = 0;
    a.trace = nullptr; a.trace_steps = 0; a.use_tmap = 0;
    if (p->batch_order) {
        int32_t* dev_order = reinterpret_cast<int32_t*>(ctx->ws + sc.order_off);
        e = cudaMemcpyAsync(dev_order, p->batch_order, sizeof(int32_t) * (size_t)T, cudaMemcpyHostToDevice, ctx->stream);
        if (e != cudaSuccess) return cuda_status(e);
        a.order = dev_order;
    }

    if (engine == ZIPML_ENGINE_PERSISTENT) {
        // barrier targets are 32-bit: at most 2 barriers per step and G arrivals per barrier
        const int64_t max_steps = (int64_t)(0x7fffffffLL / (2LL * G));
        for (int64_t s0 = first_step; s0 < first_step + num_steps; s0 += max_steps) {
            e = cudaMemsetAsync(a.barrier, 0, sizeof(unsigned) * 4, ctx->stream);
            if (e != cudaSuccess) return cuda_status(e);
            SgdArgs chunk = a;
            chunk.first_step = s0;
            chunk.num_steps = (first_step + num_steps - s0 < max_steps) ? first_step + num_steps - s0 : max_steps;
            chunk.phases = kPhaseAll; chunk.persistent = 1;
            if (s0 + chunk.num_steps < first_step + num_steps) { chunk.grad_out = nullptr; chunk.model_out = nullptr; }
            void* params[] = {&chunk};
            e = cudaLaunchCooperativeKernel(kernel, dim3((unsigned)G), dim3(kSgdThreads), params, plan.smem, ctx->stream);
            if (e != cudaSuccess) return cuda_status(e);
            ctx->launches += 1;
        }
        ctx->last_engine = ZIPML_ENGINE_PERSISTENT;
        return ZIPML_OK;
    }

    for (int64_t s = first_step; s < first_step + num_steps; ++s) {
        SgdArgs step_args = a;
        step_args.first_step = s; step_args.num_steps = 1;
        if (s != first_step + num_steps - 1) { step_args.grad_out = nullptr; step_args.model_out = nullptr; }
        for (int ph : {kPhaseA, kPhaseB, kPhaseC}) {
            step_args.phases = ph;
            void* params[] = {&step_args};
            e = cudaLaunchKernel(kernel, dim3((unsigned)G), dim3(kSgdThreads), params, plan.smem, ctx->stream);
            if (e != cudaSuccess) return cuda_status(e);
            ctx->launches += 1;
        }
    }
    ctx->last_engine = ZIPML_ENGINE_STEPWISE;
    return ZIPML_OK;
}

}  // namespace zipml
