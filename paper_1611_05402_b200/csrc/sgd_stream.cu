// Stream engine of zipml_sgd_epoch: large minibatch tiles on uniform grids, fp32 model and gradient.
//
// A step of the double-sampled minibatch SGD (paper Eq. (double) in its symmetrised form, footnote
// of "Double Sampling"; update in full precision, "End-to-end Quantization") is two passes over the
// step's code tile: the dots q1^T x, q2^T x of every row (pass A), then the gradient
// 1/(2B) sum_k [q1_k r2_k + q2_k r1_k] (pass B), with r = dot - b between them.  Here both passes
// read the codes straight from global memory into int8 tensor-core fragments (no shared-memory
// staging): pass A streams the tile from HBM and leaves it in L2, pass B re-reads it from L2.
//
//   pass A   a warp takes 16 rows x a run of 64-byte spans; code bytes are the A operand of
//            mma.sync m16n8k32 (u8 x s8), the four balanced base-128 digits of w = step * x the B
//            operand's columns; digit sums are exact integers, combined in 64 bits and added to
//            dots[plane][row] with integer atomics (order-free).
//   barrier  one grid barrier per step: every dot is complete.
//   resid.   every CTA computes all residuals (2B values), their common fixed-point scale and digits
//            (shared memory), redundantly and identically.
//   pass B   a CTA owns whole column blocks (CW bytes of the row = CW * 8 / CB features) for all rows
//            of the step, so its gradient entries never leave it.  The contraction runs over rows:
//            a lane loads LB bytes of 8 rows, transposes 4 x 4 byte blocks with byte permutes and
//            feeds (features x rows) fragments; the residual digits are the B operand.
//   update   the owner updates its features of x, turns w = step * x into digits for the next
//            step and raises a per-block flag; pass A of the next step waits only for the flags of
//            the blocks it reads (no second grid barrier).
//
// The digit scale of w must be known to writers and readers without another exchange: it is a bound,
// |w_j(t+1)| <= max|w(t)| + lr * max_j(step_j * max|a_j|) * max_k|r_k(t)|, whose pieces every CTA
// already holds after the step's barrier (owners publish their part of max|w| and of lo^T x with
// the flags).  The bound costs a few of the 27 fixed-point bits while the model is still near zero.
#include <string.h>

#include "int_digits.cuh"
#include "sgd_common.cuh"

namespace zipml {

constexpr int kStreamThreads = 512;
constexpr int kStreamWarps = kStreamThreads / 32;
constexpr int kStreamMaxBatch = 8192;      // residual digits of a step live in shared memory
constexpr int kStreamMaxOwn = 4;           // column blocks per CTA

struct StreamArgs {
    const unsigned char* p1;
    const unsigned char* p2;
    int64_t row_bytes, m;
    int n, bits;
    const float* lo;
    const float* step;
    const float* b;
    float* x;
    float* grad_out;
    int64_t batch, first_step, num_steps;
    const int32_t* order;
    float lr;
    int ca;                  // pass A: column parts per 16-row block
    int spans;               // 64-byte spans of a row
    int ncb;                 // pass B: column blocks of the row
    int bpc;                 // column blocks per CTA
    int bpad;                // batch rounded up to 32
    int64_t vec_bytes;       // bytes of one digit vector (row_bytes rounded up to 128)
    signed char* wdig;       // [NG][NS][vec_bytes] digits of w, in the byte order of the codes
    unsigned* ready;         // [ncb] number of digit versions published for the block
    long long* dots;         // [3][2][bpad] fixed-point dots of the step (three steps in rotation)
    float* wmax_part;        // [2][G] owners' max |w| (by step parity)
    double* base_part;       // [2][G] owners' part of lo^T x
    unsigned* barrier;
    DeviceStatus* status;
    unsigned long long* trace;
    int trace_steps;
};

__device__ __forceinline__ void stream_mark(const StreamArgs& a, int64_t t_rel, int k) {
    if (a.trace && blockIdx.x == 0 && threadIdx.x == 0 && t_rel < a.trace_steps) a.trace[t_rel * 8 + k] = (unsigned long long)clock64();
}

__device__ __forceinline__ unsigned ld_acquire_u32(const unsigned* p) {
    unsigned v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_release_u32(unsigned* p, unsigned v) {
    asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}

// Max over the block; every thread gets it.  `sh` holds 33 floats.  Ends with the block synchronised.
__device__ __forceinline__ float block_max(float v, float* sh) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    __syncthreads();
    if ((threadIdx.x & 31) == 0) sh[threadIdx.x >> 5] = v;
    __syncthreads();
    if (threadIdx.x == 0) {
        float t = 0.0f;
        for (int w = 0; w < (int)(blockDim.x >> 5); ++w) t = fmaxf(t, sh[w]);
        sh[32] = t;
    }
    __syncthreads();
    return sh[32];
}

__device__ __forceinline__ int fixed_point(float v, float inv) {
    int W = __float2int_rn(v * inv);
    return max(-IntPath<8>::QMAX, min(IntPath<8>::QMAX, W));
}

template <int LB>
struct LaneBytes;
template <>
struct LaneBytes<16> {
    using T = uint4;
    static __device__ __forceinline__ T zero() { return make_uint4(0u, 0u, 0u, 0u); }
    static __device__ __forceinline__ uint32_t word(const T& v, int i) { return i == 0 ? v.x : i == 1 ? v.y : i == 2 ? v.z : v.w; }
};
template <>
struct LaneBytes<8> {
    using T = uint2;
    static __device__ __forceinline__ T zero() { return make_uint2(0u, 0u); }
    static __device__ __forceinline__ uint32_t word(const T& v, int i) { return i == 0 ? v.x : v.y; }
};

template <int CB, int LB>
__global__ void __launch_bounds__(kStreamThreads, 1) sgd_stream_kernel(const StreamArgs a) {
    constexpr int NG = IntPath<CB>::NG, NS = IntPath<CB>::NS, FPW = 32 / CB;
    constexpr int CW = 8 * LB, WPL = LB / 4;
    constexpr int QMAX = IntPath<CB>::QMAX;
    using Vec = typename LaneBytes<LB>::T;
    static_assert(NS == 4, "four digits");
    extern __shared__ __align__(16) unsigned char smem[];
    signed char* rdig = reinterpret_cast<signed char*>(smem);                    // [2][NS][bpad]
    int* gacc = reinterpret_cast<int*>(smem + (size_t)2 * NS * a.bpad);          // [bpc][NG][CW][NS]
    __shared__ double red[40];
    __shared__ float fsh[40];

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, gl = lane >> 2, tl = lane & 3;
    const int cta = blockIdx.x, G = gridDim.x;
    const int n = a.n;
    const int64_t rb = a.row_bytes, vb = a.vec_bytes;
    const int cb0 = min(a.ncb, cta * a.bpc), cb1 = min(a.ncb, cb0 + a.bpc);
    const int own_bytes = (cb1 - cb0) * CW;
    const float smax = (float)((1 << a.bits) - 1);

    // ---- set-up: every CTA scans the model once (identical arithmetic everywhere)
    float cmax = 0.0f, wm = 0.0f;
    double base = 0.0;
    for (int j = tid; j < n; j += kStreamThreads) {
        const float l = a.lo[j], s = a.step[j], xv = a.x[j];
        cmax = fmaxf(cmax, fabsf(s) * fmaxf(fabsf(l), fabsf(l + s * smax)));
        wm = fmaxf(wm, fabsf(s * xv));
        base += (double)l * (double)xv;
    }
    cmax = block_max(cmax, fsh);
    wm = block_max(wm, fsh);
    base = block_sum(base, red);
    float bound = wm;                      // digit scale of the w that the coming step reads

    // digits of w for the first step, from the caller's model
    {
        const float inv = bound > 0.0f ? (float)QMAX / bound : 0.0f;
        for (int idx = tid; idx < own_bytes * NG; idx += kStreamThreads) {
            const int bl = idx / NG, grp = idx - bl * NG;
            const int64_t byte = (int64_t)cb0 * CW + bl;
            if (byte >= vb) continue;
            const int64_t j = (byte >> 2) * FPW + (byte & 3) * NG + grp;
            int d[NS];
            balanced_digits<NS>(j < n ? fixed_point(a.step[j] * a.x[j], inv) : 0, d);
#pragma unroll
            for (int s = 0; s < NS; ++s) a.wdig[((int64_t)grp * NS + s) * vb + byte] = (signed char)d[s];
        }
        __syncthreads();
        if (tid == 0) {
            __threadfence();
            for (int c = cb0; c < cb1; ++c) st_release_u32(a.ready + c, 1u);
        }
    }

    for (int64_t t_rel = 0; t_rel < a.num_steps; ++t_rel) {
        const int64_t it = a.first_step + t_rel;
        const bool last = t_rel + 1 == a.num_steps;
        const int64_t bt_idx = a.order ? (int64_t)a.order[it] : it;
        const int64_t row0 = bt_idx * a.batch;
        const int bt = (int)min(a.batch, a.m - row0);
        const unsigned char* t1 = a.p1 + row0 * rb;
        const unsigned char* t2 = a.p2 + row0 * rb;
        long long* dots = a.dots + (size_t)(t_rel % 3) * 2 * a.bpad;
        stream_mark(a, t_rel, 0);

        // ------------------------------------------------------------------ pass A: dots
        {
            const int nrb = (bt + 15) >> 4;
            const int ntasks = nrb * a.ca;
            for (int q = cta * kStreamWarps + warp; q < ntasks; q += G * kStreamWarps) {
                const int rblk = q / a.ca, part = q - rblk * a.ca;
                const int s0 = (int)((int64_t)part * a.spans / a.ca), s1 = (int)((int64_t)(part + 1) * a.spans / a.ca);
                // digits of this column part present?
                {
                    const int f0 = (s0 * 64) / CW, f1 = min(a.ncb, (s1 * 64 + CW - 1) / CW);
                    const unsigned want = (unsigned)(t_rel + 1);
                    for (int f = f0 + lane; f < f1; f += 32) {
                        long long spin = 0;
                        while (ld_acquire_u32(a.ready + f) < want) {
                            if (++spin > kBarrierSpinLimit) { set_status(a.status, ZIPML_ERR_TIMEOUT, 20); break; }
                            if ((spin & 63) == 63) {
                                if (*reinterpret_cast<volatile int*>(&a.status->code) != 0) break;
                                __nanosleep(100);
                            }
                        }
                    }
                    __syncwarp();
                    __threadfence();
                }
                const int ra = min(rblk * 16 + gl, bt - 1), rh = min(rblk * 16 + gl + 8, bt - 1);
                const unsigned char* a1 = t1 + ra * rb + 16 * tl;
                const unsigned char* h1 = t1 + rh * rb + 16 * tl;
                const unsigned char* a2 = t2 + ra * rb + 16 * tl;
                const unsigned char* h2 = t2 + rh * rb + 16 * tl;
                int c1[4] = {0, 0, 0, 0}, c2[4] = {0, 0, 0, 0};
#pragma unroll 2
                for (int sp = s0; sp < s1; ++sp) {
                    const int64_t off = (int64_t)sp * 64;
                    uint4 ua = make_uint4(0u, 0u, 0u, 0u), uh = ua, va = ua, vh = ua;
                    const bool in = off + 16 * tl < rb;
                    if (in) {
                        ua = __ldcg(reinterpret_cast<const uint4*>(a1 + off));
                        uh = __ldcg(reinterpret_cast<const uint4*>(h1 + off));
                        va = __ldcg(reinterpret_cast<const uint4*>(a2 + off));
                        vh = __ldcg(reinterpret_cast<const uint4*>(h2 + off));
                    }
#pragma unroll
                    for (int g = 0; g < NG; ++g) {
                        uint4 bd = make_uint4(0u, 0u, 0u, 0u);
                        if (gl < NS && in) bd = __ldcg(reinterpret_cast<const uint4*>(a.wdig + ((int64_t)g * NS + gl) * vb + off + 16 * tl));
                        mma_u8s8(c1, group_bytes<CB>(ua.x, g), group_bytes<CB>(uh.x, g), group_bytes<CB>(ua.y, g), group_bytes<CB>(uh.y, g), bd.x, bd.y);
                        mma_u8s8(c1, group_bytes<CB>(ua.z, g), group_bytes<CB>(uh.z, g), group_bytes<CB>(ua.w, g), group_bytes<CB>(uh.w, g), bd.z, bd.w);
                        mma_u8s8(c2, group_bytes<CB>(va.x, g), group_bytes<CB>(vh.x, g), group_bytes<CB>(va.y, g), group_bytes<CB>(vh.y, g), bd.x, bd.y);
                        mma_u8s8(c2, group_bytes<CB>(va.z, g), group_bytes<CB>(vh.z, g), group_bytes<CB>(va.w, g), group_bytes<CB>(vh.w, g), bd.z, bd.w);
                    }
                }
                // lane t < 2 holds digits 2t, 2t+1 of rows g (c[0], c[1]) and g+8 (c[2], c[3])
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    const long long q1 = (long long)c1[2 * e] + 128ll * (long long)c1[2 * e + 1];
                    const long long q2 = (long long)c2[2 * e] + 128ll * (long long)c2[2 * e + 1];
                    const long long v1 = q1 + 16384ll * __shfl_down_sync(0xffffffffu, q1, 1);
                    const long long v2 = q2 + 16384ll * __shfl_down_sync(0xffffffffu, q2, 1);
                    const int k = rblk * 16 + gl + 8 * e;
                    if (tl == 0 && k < bt) {
                        atomicAdd(reinterpret_cast<unsigned long long*>(dots + k), (unsigned long long)v1);
                        atomicAdd(reinterpret_cast<unsigned long long*>(dots + a.bpad + k), (unsigned long long)v2);
                    }
                }
            }
        }
        stream_mark(a, t_rel, 1);
        if (!grid_barrier(a.barrier, (unsigned)((t_rel + 1) * G), a.status, 21)) return;
        stream_mark(a, t_rel, 2);

        // ------------------------------------------------------------------ residuals (every CTA, all rows)
        // clear the dots two steps ahead (its last readers passed the previous barrier)
        {
            long long* z = a.dots + (size_t)((t_rel + 2) % 3) * 2 * a.bpad;
            for (int i = cta * kStreamThreads + tid; i < 2 * a.bpad; i += G * kStreamThreads) z[i] = 0;
        }
        if (t_rel > 0) {                   // max |w| and lo^T x of the model this step saw
            const size_t par = (size_t)(t_rel & 1) * G;
            float pm = 0.0f;
            double pb = 0.0;
            for (int i = tid; i < G; i += kStreamThreads) { pm = fmaxf(pm, __ldcg(a.wmax_part + par + i)); pb += __ldcg(a.base_part + par + i); }
            wm = block_max(pm, fsh);
            base = block_sum(pb, red);
        }
        const double delta_w = (double)bound / (double)QMAX;
        float rmax = 0.0f;
        for (int k = tid; k < bt; k += kStreamThreads) {
            const double bk = (double)a.b[row0 + k];
            const float r1 = (float)((double)__ldcg(dots + k) * delta_w + base - bk);
            const float r2 = (float)((double)__ldcg(dots + a.bpad + k) * delta_w + base - bk);
            rmax = fmaxf(rmax, fmaxf(fabsf(r1), fabsf(r2)));
        }
        rmax = block_max(rmax, fsh);
        const float inv_r = rmax > 0.0f ? (float)QMAX / rmax : 0.0f;
        const double delta_r = (double)rmax / (double)QMAX;
        double rsum = 0.0;                 // sum of all fixed-point residuals (exact in double)
        for (int k = tid; k < a.bpad; k += kStreamThreads) {
            int R1 = 0, R2 = 0;
            if (k < bt) {
                const double bk = (double)a.b[row0 + k];
                R1 = fixed_point((float)((double)__ldcg(dots + k) * delta_w + base - bk), inv_r);
                R2 = fixed_point((float)((double)__ldcg(dots + a.bpad + k) * delta_w + base - bk), inv_r);
            }
            rsum += (double)R1 + (double)R2;
            int d1[NS], d2[NS];
            balanced_digits<NS>(R1, d1);
            balanced_digits<NS>(R2, d2);
#pragma unroll
            for (int s = 0; s < NS; ++s) {
                rdig[(size_t)s * a.bpad + k] = (signed char)d2[s];                 // plane 1 meets r2
                rdig[(size_t)(NS + s) * a.bpad + k] = (signed char)d1[s];          // plane 2 meets r1
            }
        }
        for (int i = tid; i < (cb1 - cb0) * NG * CW * NS; i += kStreamThreads) gacc[i] = 0;
        rsum = block_sum(rsum, red);       // its barriers publish rdig and the cleared gacc
        // scale of the next model's digits: a bound that writers and readers both know now
        const float bound_next = (wm + fabsf(a.lr) * cmax * rmax) * 1.0001f;
        stream_mark(a, t_rel, 3);

        // ------------------------------------------------------------------ pass B: gradient of the own blocks
        {
            const int nrb = (bt + 31) >> 5;
            for (int c = cb0; c < cb1; ++c) {
                const int64_t coff = (int64_t)c * CW + gl * LB;
                const bool in = coff < rb;
                int acc[NG][WPL][2][4];
#pragma unroll
                for (int g = 0; g < NG; ++g)
#pragma unroll
                    for (int w = 0; w < WPL; ++w)
#pragma unroll
                        for (int u = 0; u < 2; ++u)
#pragma unroll
                            for (int e = 0; e < 4; ++e) acc[g][w][u][e] = 0;
                bool any = false;
                // newest rows first: they are the likeliest to be still in L2
#pragma unroll 1
                for (int rblk = nrb - 1 - warp; rblk >= 0; rblk -= kStreamWarps) {
                    any = true;
                    const int r0 = rblk * 32;
#pragma unroll
                    for (int pl = 0; pl < 2; ++pl) {
                        const unsigned char* tp = pl == 0 ? t1 : t2;
                        Vec lo4[4], hi4[4];
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            lo4[i] = LaneBytes<LB>::zero();
                            hi4[i] = LaneBytes<LB>::zero();
                            if (in) {
                                const int ka = min(r0 + 4 * tl + i, bt - 1), kh = min(r0 + 16 + 4 * tl + i, bt - 1);
                                lo4[i] = __ldcs(reinterpret_cast<const Vec*>(tp + ka * rb + coff));
                                hi4[i] = __ldcs(reinterpret_cast<const Vec*>(tp + kh * rb + coff));
                            }
                        }
                        uint32_t b0 = 0u, b1 = 0u;
                        if (gl < NS) {
                            const signed char* rd = rdig + (size_t)(pl * NS + gl) * a.bpad + r0 + 4 * tl;
                            b0 = *reinterpret_cast<const uint32_t*>(rd);
                            b1 = *reinterpret_cast<const uint32_t*>(rd + 16);
                        }
#pragma unroll
                        for (int w = 0; w < WPL; ++w) {
                            uint32_t ta[4], th[4];
                            transpose4x4(LaneBytes<LB>::word(lo4[0], w), LaneBytes<LB>::word(lo4[1], w), LaneBytes<LB>::word(lo4[2], w),
                                         LaneBytes<LB>::word(lo4[3], w), ta);
                            transpose4x4(LaneBytes<LB>::word(hi4[0], w), LaneBytes<LB>::word(hi4[1], w), LaneBytes<LB>::word(hi4[2], w),
                                         LaneBytes<LB>::word(hi4[3], w), th);
#pragma unroll
                            for (int g = 0; g < NG; ++g)
#pragma unroll
                                for (int u = 0; u < 2; ++u)
                                    mma_u8s8(acc[g][w][u], group_bytes<CB>(ta[2 * u], g), group_bytes<CB>(ta[2 * u + 1], g),
                                             group_bytes<CB>(th[2 * u], g), group_bytes<CB>(th[2 * u + 1], g), b0, b1);
                        }
                    }
                }
                // lane t < 2: acc[g][w][u][0..1] = digits 2t, 2t+1 of byte 4w+2u of the lane's bytes, [2..3] of byte 4w+2u+1
                if (any && tl < 2) {
                    int* dst = gacc + (size_t)(c - cb0) * NG * CW * NS;
#pragma unroll
                    for (int g = 0; g < NG; ++g)
#pragma unroll
                        for (int w = 0; w < WPL; ++w)
#pragma unroll
                            for (int u = 0; u < 2; ++u) {
                                const int byte = gl * LB + 4 * w + 2 * u;
                                int* p = dst + ((size_t)g * CW + byte) * NS + 2 * tl;
                                atomicAdd(p, acc[g][w][u][0]);
                                atomicAdd(p + 1, acc[g][w][u][1]);
                                atomicAdd(p + NS, acc[g][w][u][2]);
                                atomicAdd(p + NS + 1, acc[g][w][u][3]);
                            }
                }
            }
        }
        __syncthreads();
        stream_mark(a, t_rel, 4);

        // ------------------------------------------------------------------ update of the own features, digits of the next w
        {
            const double scale = 1.0 / (2.0 * (double)bt);
            const double lo_term = delta_r * rsum;
            const float inv = bound_next > 0.0f ? (float)QMAX / bound_next : 0.0f;
            float pm = 0.0f;
            double pb = 0.0;
            for (int idx = tid; idx < own_bytes * NG; idx += kStreamThreads) {
                const int bl = idx / NG, grp = idx - bl * NG;
                const int64_t byte = (int64_t)cb0 * CW + bl;
                if (byte >= vb) continue;
                const int64_t j = (byte >> 2) * FPW + (byte & 3) * NG + grp;
                int W = 0;
                if (j < n) {
                    const int cl = bl / CW, bb = bl - cl * CW;
                    const int* src = gacc + (((size_t)cl * NG + grp) * CW + bb) * NS;
                    const int sv[NS] = {src[0], src[1], src[2], src[3]};
                    const long long S = combine_digits<NS>(sv);
                    const float l = a.lo[j], s = a.step[j];
                    const float g = (float)(((double)l * lo_term + (double)s * (delta_r * (double)S)) * scale);
                    if (last && a.grad_out) { a.grad_out[j] = g; a.grad_out[n + j] = g; }
                    const float xn = fmaf(-a.lr, g, a.x[j]);
                    a.x[j] = xn;
                    const float w = s * xn;
                    pm = fmaxf(pm, fabsf(w));
                    pb += (double)l * (double)xn;
                    W = fixed_point(w, inv);
                }
                if (!last) {
                    int d[NS];
                    balanced_digits<NS>(W, d);
#pragma unroll
                    for (int s = 0; s < NS; ++s) a.wdig[((int64_t)grp * NS + s) * vb + byte] = (signed char)d[s];
                }
            }
            if (last) break;
            pm = block_max(pm, fsh);
            pb = block_sum(pb, red);       // ends with a barrier: every digit store of the CTA is issued
            if (tid == 0) {
                const size_t par = (size_t)((t_rel + 1) & 1) * G;
                a.wmax_part[par + cta] = pm;
                a.base_part[par + cta] = pb;
                __threadfence();
                for (int c = cb0; c < cb1; ++c) st_release_u32(a.ready + c, (unsigned)(t_rel + 2));
            }
            bound = bound_next;
        }
        stream_mark(a, t_rel, 5);
    }
}

// ---------------------------------------------------------------------------------------------
// Host side
// ---------------------------------------------------------------------------------------------
static const void* stream_kernel_ptr(int cb) {
    if (cb == 2) return reinterpret_cast<const void*>(&sgd_stream_kernel<2, 8>);
    if (cb == 4) return reinterpret_cast<const void*>(&sgd_stream_kernel<4, 8>);
    return reinterpret_cast<const void*>(&sgd_stream_kernel<8, 16>);
}

int launch_sgd_stream(zipml_ctx* ctx, const zipml_dataset* d, const float* b, float* x, const zipml_sgd_params* p,
                      int64_t first_step, int64_t num_steps, float* grad_out, bool only_if_profitable) {
    if (!ctx->cooperative) return ZIPML_ERR_WORKSPACE;
    if (d->level_mode != ZIPML_LEVELS_UNIFORM || p->model_bits != 0 || p->grad_bits != 0) return ZIPML_ERR_WORKSPACE;
    if (d->n > (1 << 30) / 8) return ZIPML_ERR_WORKSPACE;
    const int cb = container_bits(d->bits);
    const int lb = cb == 8 ? 16 : 8, cw = 8 * lb, ng = 8 / cb;
    const int64_t T = (d->m + p->batch - 1) / p->batch;
    const int64_t B = p->batch < d->m ? p->batch : d->m;
    if (B > kStreamMaxBatch) return ZIPML_ERR_WORKSPACE;
    const int bpad = (int)((B + 31) / 32 * 32);
    const int64_t rb = d->row_bytes;
    const int64_t ncb64 = (rb + cw - 1) / cw;
    int G = ctx->sm_count;
    if (p->grid_row_parts > 0 && p->grid_row_parts < G) G = p->grid_row_parts;      // tuning: fewer CTAs
    int64_t bpc = (ncb64 + G - 1) / G;
    if (bpc > kStreamMaxOwn) {             // the hint does not fit: plan for the whole device
        G = ctx->sm_count;
        bpc = (ncb64 + G - 1) / G;
    }
    if (bpc > kStreamMaxOwn) return ZIPML_ERR_WORKSPACE;
    G = (int)((ncb64 + bpc - 1) / bpc);
    // worth it only where a step is wide enough to occupy the device and long enough to hide the barrier
    if (only_if_profitable && (G < ctx->sm_count / 2 || B < 256)) return ZIPML_ERR_WORKSPACE;
    const int spans = (int)((rb + 63) / 64);
    const int64_t nrb16 = (B + 15) / 16;
    int64_t ca = ((int64_t)G * kStreamWarps) / nrb16;
    if (ca < 1) ca = 1;
    if (ca > spans) ca = spans;
    // a task's digit sums must stay within 32 bits: at most 255 * 64 * codes per group
    while ((int64_t)(spans + ca - 1) / ca * 64 > 65536) ++ca;
    const int64_t vec_bytes = (rb + 127) / 128 * 128;

    const size_t smem = (size_t)2 * 4 * bpad + sizeof(int) * (size_t)bpc * ng * cw * 4;
    const void* kernel = stream_kernel_ptr(cb);
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return cuda_status(e);
    int per_sm = 0;
    e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, kStreamThreads, smem);
    if (e != cudaSuccess) return cuda_status(e);
    if (per_sm < 1 || G > per_sm * ctx->sm_count) return ZIPML_ERR_WORKSPACE;

    size_t off = 0;
    auto piece = [&](size_t bytes) { const size_t o = off; off += carve_size(bytes); return o; };
    // zeroed before a launch: barrier counter, flags, dots
    const size_t o_bar = piece(sizeof(unsigned) * 64);
    const size_t o_ready = piece(sizeof(unsigned) * (size_t)ncb64);
    const size_t o_dots = piece(sizeof(long long) * 3 * 2 * (size_t)bpad);
    const size_t zero_bytes = off;
    const size_t o_wdig = piece((size_t)ng * 4 * vec_bytes);
    const size_t o_wmax = piece(sizeof(float) * 2 * (size_t)G);
    const size_t o_base = piece(sizeof(double) * 2 * (size_t)G);
    const size_t o_ord = piece(sizeof(int32_t) * (size_t)(p->batch_order ? T : 0));
    int rc = ws_reserve(ctx, off);
    if (rc != ZIPML_OK) return rc;

    StreamArgs a;
    memset(&a, 0, sizeof(a));
    a.p1 = d->plane1; a.p2 = d->plane2; a.row_bytes = rb; a.m = d->m; a.n = (int)d->n; a.bits = d->bits;
    a.lo = d->feat_lo; a.step = d->feat_step; a.b = b; a.x = x; a.grad_out = grad_out;
    a.batch = B; a.lr = p->lr;
    a.ca = (int)ca; a.spans = spans; a.ncb = (int)ncb64; a.bpc = (int)bpc; a.bpad = bpad; a.vec_bytes = vec_bytes;
    a.barrier = reinterpret_cast<unsigned*>(ctx->ws + o_bar);
    a.ready = reinterpret_cast<unsigned*>(ctx->ws + o_ready);
    a.dots = reinterpret_cast<long long*>(ctx->ws + o_dots);
    a.wdig = reinterpret_cast<signed char*>(ctx->ws + o_wdig);
    a.wmax_part = reinterpret_cast<float*>(ctx->ws + o_wmax);
    a.base_part = reinterpret_cast<double*>(ctx->ws + o_base);
    a.status = ctx->d_status;
    a.trace = reinterpret_cast<unsigned long long*>(p->trace);
    a.trace_steps = p->trace ? p->trace_steps : 0;
    if (p->batch_order) {
        int32_t* dev_order = reinterpret_cast<int32_t*>(ctx->ws + o_ord);
        e = cudaMemcpyAsync(dev_order, p->batch_order, sizeof(int32_t) * (size_t)T, cudaMemcpyHostToDevice, ctx->stream);
        if (e != cudaSuccess) return cuda_status(e);
        a.order = dev_order;
    }
    // the barrier counter and the flag versions are 32-bit step counts
    const int64_t max_steps = (int64_t)(0x7fffffff / G) - 2;
    for (int64_t s0 = first_step; s0 < first_step + num_steps; s0 += max_steps) {
        e = cudaMemsetAsync(ctx->ws, 0, zero_bytes, ctx->stream);
        if (e != cudaSuccess) return cuda_status(e);
        StreamArgs chunk = a;
        chunk.first_step = s0;
        chunk.num_steps = (first_step + num_steps - s0 < max_steps) ? first_step + num_steps - s0 : max_steps;
        if (s0 + chunk.num_steps < first_step + num_steps) chunk.grad_out = nullptr;
        if (s0 > first_step) { chunk.trace = nullptr; chunk.trace_steps = 0; }
        void* params[] = {&chunk};
        e = cudaLaunchCooperativeKernel(kernel, dim3((unsigned)G), dim3(kStreamThreads), params, smem, ctx->stream);
        if (e != cudaSuccess) return cuda_status(e);
        ctx->launches += 1;
    }
    ctx->last_engine = ZIPML_ENGINE_STREAM;
    return ZIPML_OK;
}

}  // namespace zipml
