// Column range scan and the quantize + pack kernel (paper Section 2.1; Supplement "Randomized
// Quantization" and "Column Scaling"): two independent unbiased stochastic roundings of every
// sample element onto its feature's level grid, written as two bit-packed planes.
#include "common.cuh"
#include "internal.h"

namespace zipml {

// ---------------------------------------------------------------------------------------------
// Column range.  A tile is 32*VEC columns wide; blockDim = (32, 8): x walks the columns (one VEC-wide
// load per thread, a warp reads 128*VEC contiguous bytes of a row), y walks rows.  Row chunks are
// spread over gridDim.y; results meet in order-preserving integer atomics (min/max are exact and
// order independent).
// ---------------------------------------------------------------------------------------------
__global__ void range_init_kernel(uint32_t* lo_key, uint32_t* hi_key, int64_t n) {
    const int64_t j = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (j < n) { lo_key[j] = 0xffffffffu; hi_key[j] = 0u; }
}

template <int VEC>
__global__ void __launch_bounds__(256) range_scan_kernel(const float* __restrict__ A, int64_t m, int64_t n,
                                                         int64_t lda, int64_t rows_per_block, uint32_t* lo_key,
                                                         uint32_t* hi_key, DeviceStatus* status) {
    __shared__ float s_lo[8][32 * VEC];
    __shared__ float s_hi[8][32 * VEC];
    const int64_t j0 = ((int64_t)blockIdx.x * 32 + threadIdx.x) * VEC;
    const int64_t r0 = (int64_t)blockIdx.y * rows_per_block;
    const int64_t r1 = min(m, r0 + rows_per_block);
    float lo[VEC], hi[VEC];
    bool bad = false;
#pragma unroll
    for (int v = 0; v < VEC; ++v) { lo[v] = INFINITY; hi[v] = -INFINITY; }
    if (j0 < n) {
        for (int64_t r = r0 + threadIdx.y; r < r1; r += 8) {
            float val[VEC];
            bool have[VEC];
            if constexpr (VEC == 4) {
                if (j0 + 3 < n) {
                    const float4 q = __ldg(reinterpret_cast<const float4*>(A + r * lda + j0));
                    val[0] = q.x; val[1] = q.y; val[2] = q.z; val[3] = q.w;
                    have[0] = have[1] = have[2] = have[3] = true;
                } else {
#pragma unroll
                    for (int v = 0; v < VEC; ++v) {
                        have[v] = j0 + v < n;
                        val[v] = have[v] ? __ldg(A + r * lda + j0 + v) : 0.0f;
                    }
                }
            } else {
                val[0] = __ldg(A + r * lda + j0);
                have[0] = true;
            }
#pragma unroll
            for (int v = 0; v < VEC; ++v) {
                if (!have[v]) continue;
                bad |= !(fabsf(val[v]) <= 3.402823466e+38f);
                lo[v] = fminf(lo[v], val[v]);
                hi[v] = fmaxf(hi[v], val[v]);
            }
        }
    }
#pragma unroll
    for (int v = 0; v < VEC; ++v) { s_lo[threadIdx.y][threadIdx.x * VEC + v] = lo[v]; s_hi[threadIdx.y][threadIdx.x * VEC + v] = hi[v]; }
    if (bad) set_status(status, ZIPML_ERR_NONFINITE, 1);
    __syncthreads();
    const int t = threadIdx.y * 32 + threadIdx.x;
    if (t < 32 * VEC) {
        const int64_t j = (int64_t)blockIdx.x * 32 * VEC + t;
        if (j < n) {
            float a = s_lo[0][t], b = s_hi[0][t];
#pragma unroll
            for (int y = 1; y < 8; ++y) { a = fminf(a, s_lo[y][t]); b = fmaxf(b, s_hi[y][t]); }
            if (a <= b) {  // at least one row seen
                atomicMin(lo_key + j, float_order_key(a));
                atomicMax(hi_key + j, float_order_key(b));
            }
        }
    }
}

// The same scan for wide matrices: a block reads 4 KB of consecutive columns of a row at a time (256 threads x
// float4; the narrow kernel's 512-byte pieces waste DRAM pages on rows of tens of kilobytes), a thread keeps its
// four columns for all rows of the block's chunk, four rows' loads in flight; no meeting in shared memory.
__global__ void __launch_bounds__(256) range_scan_wide_kernel(const float* __restrict__ A, int64_t m, int64_t n, int64_t lda,
                                                              int64_t rows_per_block, uint32_t* lo_key, uint32_t* hi_key,
                                                              DeviceStatus* status) {
    const int64_t j0 = ((int64_t)blockIdx.x * 256 + threadIdx.x) * 4;
    if (j0 >= n) return;
    const int64_t r0 = (int64_t)blockIdx.y * rows_per_block;
    const int64_t r1 = min(m, r0 + rows_per_block);
    const int nv = (int)min((int64_t)4, n - j0);
    float lo[4], hi[4];
#pragma unroll
    for (int v = 0; v < 4; ++v) { lo[v] = INFINITY; hi[v] = -INFINITY; }
    bool bad = false;
    const float* col = A + j0;
    if (nv == 4) {
#pragma unroll 4
        for (int64_t r = r0; r < r1; ++r) {
            const float4 q = __ldg(reinterpret_cast<const float4*>(col + r * lda));
            const float val[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
            for (int v = 0; v < 4; ++v) {
                bad |= !(fabsf(val[v]) <= 3.402823466e+38f);
                lo[v] = fminf(lo[v], val[v]);
                hi[v] = fmaxf(hi[v], val[v]);
            }
        }
    } else {
        for (int64_t r = r0; r < r1; ++r)
            for (int v = 0; v < nv; ++v) {
                const float val = __ldg(col + r * lda + v);
                bad |= !(fabsf(val) <= 3.402823466e+38f);
                lo[v] = fminf(lo[v], val);
                hi[v] = fmaxf(hi[v], val);
            }
    }
    if (bad) set_status(status, ZIPML_ERR_NONFINITE, 1);
    for (int v = 0; v < nv; ++v)
        if (lo[v] <= hi[v]) {  // at least one row seen
            atomicMin(lo_key + j0 + v, float_order_key(lo[v]));
            atomicMax(hi_key + j0 + v, float_order_key(hi[v]));
        }
}

__global__ void range_finalize_kernel(const uint32_t* lo_key, const uint32_t* hi_key, int64_t n, int s, bool symmetric,
                                      float* lo_out, float* hi_out, float* inv_out, float* step_out) {
    const int64_t j = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= n) return;
    float lo = float_from_order_key(lo_key[j]), hi = float_from_order_key(hi_key[j]);
    if (symmetric) {                     // the grid [-M_j, M_j], M_j = max |value| (Supplement "Column Scaling")
        hi = fmaxf(fabsf(lo), fabsf(hi));
        lo = -hi;
    }
    const float range = __fsub_rn(hi, lo);
    lo_out[j] = lo;
    if (hi_out) hi_out[j] = hi;
    if (inv_out) inv_out[j] = range > 0.0f ? __fdiv_rn((float)s, range) : 0.0f;
    if (step_out) step_out[j] = __fdiv_rn(range, (float)s);
}

int launch_column_range(zipml_ctx* ctx, const float* A, int64_t m, int64_t n, int64_t lda, int s, bool symmetric,
                        uint32_t* key_scratch, float* lo_out, float* hi_out, float* inv_out, float* step_out) {
    uint32_t* lo_key = key_scratch;
    uint32_t* hi_key = key_scratch + n;
    const unsigned nb = (unsigned)((n + 255) / 256);
    range_init_kernel<<<nb, 256, 0, ctx->stream>>>(lo_key, hi_key, n);
    const bool vec = (lda % 4 == 0) && ((reinterpret_cast<uintptr_t>(A) & 15) == 0);
    if (vec && n >= 2048) {
        const int64_t col_tiles = (n + 1023) / 1024;
        int64_t chunks = (int64_t)ctx->sm_count * 8 / col_tiles;
        chunks = chunks < 1 ? 1 : chunks;
        int64_t rows_per_block = (m + chunks - 1) / chunks;
        rows_per_block = rows_per_block < 64 ? 64 : rows_per_block;
        chunks = (m + rows_per_block - 1) / rows_per_block;
        if (chunks > 65535) { rows_per_block = (m + 65534) / 65535; chunks = (m + rows_per_block - 1) / rows_per_block; }
        range_scan_wide_kernel<<<dim3((unsigned)col_tiles, (unsigned)chunks), 256, 0, ctx->stream>>>(A, m, n, lda, rows_per_block, lo_key,
                                                                                                   hi_key, ctx->d_status);
        range_finalize_kernel<<<nb, 256, 0, ctx->stream>>>(lo_key, hi_key, n, s, symmetric, lo_out, hi_out, inv_out, step_out);
        ctx->launches += 3;
        return cuda_status(cudaGetLastError());
    }
    const int width = vec ? 128 : 32;
    const int64_t col_tiles = (n + width - 1) / width;
    // enough row chunks to give every SM a few blocks, at least 64 rows each
    int64_t chunks = (int64_t)ctx->sm_count * 8 / col_tiles;
    chunks = chunks < 1 ? 1 : chunks;
    int64_t rows_per_block = (m + chunks - 1) / chunks;
    rows_per_block = rows_per_block < 64 ? 64 : rows_per_block;
    chunks = (m + rows_per_block - 1) / rows_per_block;
    if (chunks > 65535) { rows_per_block = (m + 65534) / 65535; chunks = (m + rows_per_block - 1) / rows_per_block; }
    const dim3 grid((unsigned)col_tiles, (unsigned)chunks), block(32, 8);
    if (vec) range_scan_kernel<4><<<grid, block, 0, ctx->stream>>>(A, m, n, lda, rows_per_block, lo_key, hi_key, ctx->d_status);
    else range_scan_kernel<1><<<grid, block, 0, ctx->stream>>>(A, m, n, lda, rows_per_block, lo_key, hi_key, ctx->d_status);
    range_finalize_kernel<<<nb, 256, 0, ctx->stream>>>(lo_key, hi_key, n, s, symmetric, lo_out, hi_out, inv_out, step_out);
    ctx->launches += 3;
    return cuda_status(cudaGetLastError());
}

// ---------------------------------------------------------------------------------------------
// Quantize + pack.  A thread owns one 32-bit word column of the planes (FPW = 32/CB consecutive
// features) for kQuantRows consecutive rows: the features' lo and inv are loaded once, the rows'
// Philox chains are independent and overlap.  Per row it reads the FPW samples as float4s when the
// row is 16-byte aligned, decides cell and up-probability in pinned fp32 arithmetic, draws one
// Philox block per feature pair (four words = two features x two copies) and writes the two
// words.  A pair whose up-probabilities are all 0 or 1 (values on a level: the zeros of sparse
// rows, the column extremes) needs no random numbers -- the comparison u * 2^-24 < p is decided
// without them -- and skips its Philox block; the codes are the same.  Words past the last
// feature are written as zero so that the planes are fully defined.
// Level tables: the block's tables are staged in shared memory as [level][feature slot of the
// word][word column], so that the lanes of a warp (consecutive word columns) read consecutive
// addresses; read from global memory, where the tables of neighbouring lanes lie FPW * L floats
// apart, every look-up took 32 cache lines per warp and the kernel ran at a tenth of this rate.
// ---------------------------------------------------------------------------------------------
constexpr int kQuantRows = 4;          // rows per thread and pass
constexpr int kQuantTableCols = 64;    // word columns per block with level tables (shared memory: L * FPW * 64 floats)

template <int CB, bool TABLE>
__global__ void __launch_bounds__(256) quantize_kernel(const float* __restrict__ A, int64_t m, int64_t n, int64_t lda,
                                                       int bits, const float* __restrict__ lo,
                                                       const float* __restrict__ inv, const float* __restrict__ levels,
                                                       uint64_t seed, uint32_t draw, uint32_t* __restrict__ plane1,
                                                       uint32_t* __restrict__ plane2, int64_t row_words, bool vec_ok,
                                                       int passes) {
    constexpr int FPW = 32 / CB;
    extern __shared__ float lev_s[];                               // TABLE: [L][FPW][blockDim.x]
    // blockDim = (word columns, row groups); blockIdx.x runs over the rows, blockIdx.y over the columns
    const int64_t q = (int64_t)blockIdx.y * blockDim.x + threadIdx.x;
    const int L = 1 << bits, s = L - 1;
    if constexpr (TABLE) {
        const int tx = blockDim.x, nthreads = blockDim.x * blockDim.y, tid = threadIdx.y * blockDim.x + threadIdx.x;
        const int64_t jb = (int64_t)blockIdx.y * tx * FPW;         // first feature of the block
        // consecutive threads read consecutive floats of the n x L table
        for (int idx = tid; idx < tx * FPW * L; idx += nthreads) {
            const int f = idx / L, k = idx - f * L;                // feature within the block, level
            const float val = (jb + f < n) ? __ldg(levels + (jb + f) * L + k) : 0.0f;
            lev_s[(k * FPW + (f % FPW)) * tx + f / FPW] = val;
        }
        __syncthreads();
    }
    if (q >= row_words) return;
    const int64_t j0 = q * FPW;
    const int nf = (int)min((int64_t)FPW, n - j0);                 // real features of this word (<= 0: padding only)
    float flo[TABLE ? 1 : FPW], finv[TABLE ? 1 : FPW];
    if constexpr (!TABLE) {
#pragma unroll
        for (int i = 0; i < FPW; ++i) {
            flo[i] = i < nf ? __ldg(lo + j0 + i) : 0.0f;
            finv[i] = i < nf ? __ldg(inv + j0 + i) : 0.0f;
        }
    }
    const bool vec = vec_ok && nf == FPW;
    const int64_t row_first = ((int64_t)blockIdx.x * blockDim.y + threadIdx.y) * kQuantRows * passes;
#pragma unroll 2
    for (int rr = 0; rr < kQuantRows * passes; ++rr) {
        const int64_t row = row_first + rr;
        if (row >= m) break;
        uint32_t w1 = 0u, w2 = 0u;
        if (nf > 0) {
            float v[FPW];
            const float* src = A + row * lda + j0;
            if (vec) {
#pragma unroll
                for (int i = 0; i < FPW / 4; ++i) {
                    const float4 t = __ldg(reinterpret_cast<const float4*>(src) + i);
                    v[4 * i] = t.x; v[4 * i + 1] = t.y; v[4 * i + 2] = t.z; v[4 * i + 3] = t.w;
                }
            } else {
#pragma unroll
                for (int i = 0; i < FPW; ++i) v[i] = (i < nf) ? __ldg(src + i) : 0.0f;
            }
            if constexpr (FPW <= 8) {
                // pass 1: cells and thresholds of all features; a threshold strictly between 0 and 2^24 needs a draw
                uint32_t thr[FPW];
                uint32_t need = 0u;                                     // pairs with at least one such feature
    #pragma unroll
                for (int i = 0; i < FPW; ++i) {
                    thr[i] = 0u;
                    if (i >= nf) continue;
                    uint32_t cell;
                    float p;
                    if constexpr (!TABLE) {
                        uniform_cell(v[i], flo[i], finv[i], s, cell, p);
                    } else {
                        const float* lev = lev_s + i * blockDim.x + threadIdx.x;       // level k at lev[k * FPW * blockDim.x]
                        const int ls = FPW * blockDim.x;
                        int l = 0;
                        for (int k = 1; k <= s - 1; ++k) l = (lev[k * ls] <= v[i]) ? k : l;
                        const float base = lev[l * ls];
                        const float width = __fsub_rn(lev[(l + 1) * ls], base);
                        cell = (uint32_t)l;
                        p = width > 0.0f ? __fdiv_rn(__fsub_rn(v[i], base), width) : 0.0f;
                    }
                    const uint32_t t = up_threshold(p);
                    const bool open = t > 0u && t < 16777216u;
                    // decided without a draw: threshold 0 never up, 2^24 and more always up
                    const uint32_t c = cell + (t >= 16777216u ? 1u : 0u);
                    w1 |= c << (i * CB);
                    w2 |= c << (i * CB);
                    thr[i] = open ? t : 0u;                             // 0: this feature adds nothing in pass 2
                    need |= open ? 1u << (i >> 1) : 0u;
                }
                // pass 2: one Philox block per pair that needs one.  Where every lane needs every pair (dense continuous
                // data) the pairs run as independent unrolled chains; otherwise every lane walks its own short list, so
                // a warp runs as many rounds as its busiest lane has pairs (sparse rows: about two of four).
                auto apply = [&](int pr, const Philox4& rnd) {
    #pragma unroll
                    for (int i = 0; i < FPW / 2; ++i)
                        if (i == pr) {
                            w1 += ((rnd.v[0] >> 8) < thr[2 * i] ? 1u : 0u) << (2 * i * CB);
                            w2 += ((rnd.v[1] >> 8) < thr[2 * i] ? 1u : 0u) << (2 * i * CB);
                            w1 += ((rnd.v[2] >> 8) < thr[2 * i + 1] ? 1u : 0u) << ((2 * i + 1) * CB);
                            w2 += ((rnd.v[3] >> 8) < thr[2 * i + 1] ? 1u : 0u) << ((2 * i + 1) * CB);
                        }
                };
                constexpr uint32_t kAllPairs = (1u << (FPW / 2)) - 1u;
                if (__all_sync(__activemask(), need == kAllPairs)) {
    #pragma unroll
                    for (int pr = 0; pr < FPW / 2; ++pr) apply(pr, sample_block(seed, (uint64_t)row, (uint32_t)((j0 >> 1) + pr), draw));
                } else {
                    while (need) {
                        const int pr = __ffs(need) - 1;
                        need &= need - 1u;
                        apply(pr, sample_block(seed, (uint64_t)row, (uint32_t)((j0 >> 1) + pr), draw));
                    }
                }
        
            } else {
                // sixteen features per word: the thresholds of a whole word would not fit the registers; pair by pair
#pragma unroll
                for (int pr = 0; pr < FPW / 2; ++pr) {
                    if (2 * pr >= nf) break;
                    uint32_t cell[2] = {0u, 0u}, t[2] = {0u, 0u};
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        const int i = 2 * pr + h;
                        if (i >= nf) break;
                        float p;
                        if constexpr (!TABLE) {
                            uniform_cell(v[i], flo[i], finv[i], s, cell[h], p);
                        } else {
                            const float* lev = lev_s + i * blockDim.x + threadIdx.x;
                            const int ls = FPW * blockDim.x;
                            int l = 0;
                            for (int k = 1; k <= s - 1; ++k) l = (lev[k * ls] <= v[i]) ? k : l;
                            const float base = lev[l * ls];
                            const float width = __fsub_rn(lev[(l + 1) * ls], base);
                            cell[h] = (uint32_t)l;
                            p = width > 0.0f ? __fdiv_rn(__fsub_rn(v[i], base), width) : 0.0f;
                        }
                        t[h] = up_threshold(p);
                    }
                    const bool random = (t[0] > 0u && t[0] < 16777216u) || (t[1] > 0u && t[1] < 16777216u);
                    Philox4 rnd;
                    if (random) rnd = sample_block(seed, (uint64_t)row, (uint32_t)((j0 >> 1) + pr), draw);
                    else rnd.v[0] = rnd.v[1] = rnd.v[2] = rnd.v[3] = 0u;    // decided without them: 0 never up, 2^24 always up
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        const int i = 2 * pr + h;
                        if (i >= nf) break;
                        w1 |= round_up_if(cell[h], t[h], rnd.v[2 * h]) << (i * CB);
                        w2 |= round_up_if(cell[h], t[h], rnd.v[2 * h + 1]) << (i * CB);
                    }
                }
            }
        }
        plane1[row * row_words + q] = w1;
        plane2[row * row_words + q] = w2;
    }
}

int launch_quantize(zipml_ctx* ctx, const float* A, int64_t m, int64_t n, int64_t lda, int bits, int level_mode,
                    const float* lo, const float* inv, const float* levels, uint64_t seed, uint32_t draw, uint8_t* plane1,
                    uint8_t* plane2, int64_t row_bytes) {
    const int cb = container_bits(bits);
    const int64_t row_words = row_bytes / 4;
    const bool table = level_mode == ZIPML_LEVELS_TABLE;
    // 256 threads: as many word columns as the row has (a power of two from 8 to 256; 64 with level tables),
    // the rest row groups; with level tables a thread makes four passes, so that staging the tables pays
    int tx = 8;
    while (tx < (table ? kQuantTableCols : 256) && tx < row_words) tx *= 2;
    const int ty = 256 / tx;
    const int passes = table ? 4 : 1;
    const size_t smem = table ? sizeof(float) * ((size_t)1 << bits) * (32 / cb) * tx : 0;
    const int64_t rows_per_block = (int64_t)ty * kQuantRows * passes;
    const int64_t row_blocks = (m + rows_per_block - 1) / rows_per_block;
    const int64_t col_blocks = (row_words + tx - 1) / tx;
    if (row_blocks > 0x7fffffffLL || col_blocks > 65535) return ZIPML_ERR_WORKSPACE;
    const dim3 grid((unsigned)row_blocks, (unsigned)col_blocks), block((unsigned)tx, (unsigned)ty);
    const bool vec_ok = (lda % 4 == 0) && ((reinterpret_cast<uintptr_t>(A) & 15) == 0);
    uint32_t* p1 = reinterpret_cast<uint32_t*>(plane1);
    uint32_t* p2 = reinterpret_cast<uint32_t*>(plane2);
#define ZIPML_LAUNCH_Q(CB_, T_) \
    quantize_kernel<CB_, T_><<<grid, block, smem, ctx->stream>>>(A, m, n, lda, bits, lo, inv, levels, seed, draw, p1, p2, row_words, vec_ok, passes)
    if (cb == 2) { if (table) ZIPML_LAUNCH_Q(2, true); else ZIPML_LAUNCH_Q(2, false); }
    else if (cb == 4) { if (table) ZIPML_LAUNCH_Q(4, true); else ZIPML_LAUNCH_Q(4, false); }
    else { ZIPML_LAUNCH_Q(8, false); }
#undef ZIPML_LAUNCH_Q
    ctx->launches += 1;
    return cuda_status(cudaGetLastError());
}

// ---------------------------------------------------------------------------------------------
// Layout conversion: row-major planes <-> 128-byte column blocks ([block][row][128 B]).  One thread moves
// 16 bytes; a warp covers four 128-byte pieces (four consecutive rows of one block): 512 contiguous bytes
// on the blocked side, four runs of 128 bytes on the row-major side.  Bytes of a block past the end of
// the row are written as zero (to blocks) or skipped (to rows).
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) convert_layout_kernel(const uint4* __restrict__ in1, const uint4* __restrict__ in2,
                                                             uint4* __restrict__ out1, uint4* __restrict__ out2, int64_t m,
                                                             int64_t row_bytes, int64_t nblk, bool to_blocks) {
    const int64_t pieces = nblk * m;                      // 128-byte pieces of a plane
    const int64_t row16 = row_bytes / 16;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < pieces * 8; i += (int64_t)gridDim.x * blockDim.x) {
        const int64_t piece = i >> 3, blk = piece / m, row = piece - blk * m;
        const int64_t c16 = blk * 8 + (i & 7);            // 16-byte column of the row
        const bool inside = c16 < row16;
        const int64_t r_idx = row * row16 + c16;
        if (to_blocks) {
            const uint4 z = make_uint4(0u, 0u, 0u, 0u);
            out1[i] = inside ? __ldg(in1 + r_idx) : z;
            out2[i] = inside ? __ldg(in2 + r_idx) : z;
        } else if (inside) {
            out1[r_idx] = __ldg(in1 + i);
            out2[r_idx] = __ldg(in2 + i);
        }
    }
}

int launch_convert_layout(zipml_ctx* ctx, const zipml_dataset* d, int to_layout, uint8_t* out1, uint8_t* out2) {
    const int64_t nblk = (d->row_bytes + 127) / 128;
    const int64_t units = nblk * d->m * 8;
    int64_t blocks = (units + 255) / 256;
    if (blocks > (int64_t)ctx->sm_count * 32) blocks = (int64_t)ctx->sm_count * 32;
    convert_layout_kernel<<<(unsigned)blocks, 256, 0, ctx->stream>>>(
        reinterpret_cast<const uint4*>(d->plane1), reinterpret_cast<const uint4*>(d->plane2), reinterpret_cast<uint4*>(out1),
        reinterpret_cast<uint4*>(out2), d->m, d->row_bytes, nblk, to_layout == ZIPML_LAYOUT_COLUMN_BLOCKS);
    ctx->launches += 1;
    return cuda_status(cudaGetLastError());
}

}  // namespace zipml
