// ZipML oracle: a plain, slow, single-threaded CPU statement of what the double-sampled
// low-precision SGD path computes.  TEST INFRASTRUCTURE ONLY: it is imported by the tests, by the
// smoke check and by the benchmark's cpu-baseline leg, never by the product path, and it shares no
// code with the CUDA library.  Accumulation is in double; every operation that decides an integer
// (a code, a bin, a level index) is an individually rounded IEEE fp32 operation (build with
// -ffp-contract=off and without fast-math), because both sides must take that decision in the same
// precision.
//
// Paper passages followed (arxiv 1611.05402):
//   * stochastic quantization Q(v, s): Section 2.1 and Supplement "Randomized Quantization"
//     (the definition with l = floor(s |v| / M) and p(x, s) = x s - l);
//   * column scaling for samples, row (l2) scaling for model and gradient: Supplement
//     "Column Scaling", "Row Scaling", "Choice between Row Scaling and Column Scaling";
//   * double sampling, Eq. (double), and the symmetrised form of the Supplement's footnote in
//     "Double Sampling";
//   * end-to-end quantization: Supplement "End-to-end Quantization" (Q4(Q1(a)(Q2(a)^T Q3(x) - b)),
//     update in full precision);
//   * variance-optimal levels: Section 3 (problem statement, Lemma on endpoints, the recursion
//     T(k, m) = min_j T(k-1, j) + V(j, m), "Dynamic Programming with Candidate Points");
//   * objective: Eq. (leastsquares) with l = a^T x - b, i.e. 1/(2K) sum (a_k^T x - b_k)^2;
//   * shared-base storage of the two samples (base code + one bit per sample): Section 2.2,
//     "Overhead of Storing Samples".
//
// Readings taken where the paper is silent (all listed in the design notes):
//   samples use L = 2^bits unsigned levels on the per-feature range [lo_j, hi_j] (s = L-1
//   intervals); model/gradient use sign-magnitude codes with s_m = 2^(bits-1) - 1; the sign
//   convention is a^T x - b; a minibatch gradient is the mean over its rows; codes are drawn once
//   and reused by every epoch; the random numbers come from Philox4x32-10 (Salmon et al., SC'11)
//   used as a pure function of (seed, row, feature, copy) resp. (seed, epoch, step, coordinate,
//   stream).
//
// Pins (tests marked "not gpu"): Philox known-answer vectors; unbiasedness and per-coordinate
// variance over 10^6 draws; the l2-scaled variance bound; naive-estimator bias in closed form;
// zero bias of the double-sampled forms; pack/unpack round trip; on-grid data reduces the
// minibatch gradient to the textbook least-squares gradient; DP against brute force over all level
// subsets; convergence to the normal-equation solution; frozen-code fixed point in closed form;
// shared-base encoding: a hand-written example, exhaustive code pairs, round trip on quantized data.
// Parity partly unpinned by nature: Q3/Q4 trajectories (a sub-ulp difference may flip a stochastic
// rounding); see the design notes.

#include <cmath>
#include <cstdint>
#include <cstdlib>
#include <cstring>
#include <limits>
#include <vector>

extern "C" {

enum { ORC_OK = 0, ORC_ERR_INVALID_ARG = -1, ORC_ERR_UNSUPPORTED = -2, ORC_ERR_NONFINITE = -3 };
enum { ORC_LEVELS_UNIFORM = 0, ORC_LEVELS_TABLE = 1 };

// ---------------------------------------------------------------------------------------------
// Philox4x32-10, from its published definition (Salmon, Moraes, Dror, Shaw: "Parallel random
// numbers: as easy as 1, 2, 3", SC'11): ten rounds of
//   (c0, c1, c2, c3) <- (hi(M1*c2) ^ c1 ^ k0, lo(M1*c2), hi(M0*c0) ^ c3 ^ k1, lo(M0*c0))
// with the key bumped by the Weyl constants between rounds.
// ---------------------------------------------------------------------------------------------
void orc_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]) {
    const uint32_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u, W0 = 0x9E3779B9u, W1 = 0xBB67AE85u;
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int round = 0; round < 10; ++round) {
        if (round > 0) { k0 += W0; k1 += W1; }
        const uint64_t p0 = (uint64_t)M0 * c0;
        const uint64_t p1 = (uint64_t)M1 * c2;
        const uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
        const uint32_t n1 = (uint32_t)p1;
        const uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
        const uint32_t n3 = (uint32_t)p0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

// 24-bit uniform integer for sample element (row, feature), copy in {1, 2}.  One Philox block
// serves the feature pair (2f, 2f+1): counter (row_lo, row_hi, feature >> 1, 0), key = seed,
// output word 2*(feature & 1) + (copy - 1); the top 24 bits of the word are used.
uint32_t orc_u24_sample_pair(uint64_t seed, uint64_t row, uint32_t feature, uint32_t copy, uint32_t pair);
uint32_t orc_u24_sample(uint64_t seed, uint64_t row, uint32_t feature, uint32_t copy) {
    return orc_u24_sample_pair(seed, row, feature, copy, 0u);
}

// The same for further, independent pairs of quantizations of the same sample (Section 4.1 "Quantizing
// Polynomials" uses d of them): pair q differs in the counter's last word, (row_lo, row_hi, feature >> 1, q).
uint32_t orc_u24_sample_pair(uint64_t seed, uint64_t row, uint32_t feature, uint32_t copy, uint32_t pair) {
    const uint32_t ctr[4] = {(uint32_t)row, (uint32_t)(row >> 32), feature >> 1, pair};
    const uint32_t key[2] = {(uint32_t)seed, (uint32_t)(seed >> 32)};
    uint32_t out[4];
    orc_philox4x32_10(ctr, key, out);
    return out[2u * (feature & 1u) + (copy - 1u)] >> 8;
}

// 24-bit uniform integer for coordinate `coord` of the model (stream 3) or gradient (stream 4)
// quantizer at (epoch, step): counter (coord >> 2, step, epoch, stream), output word coord & 3.
uint32_t orc_u24_vector(uint64_t seed, uint32_t epoch, uint32_t step, uint32_t coord, uint32_t stream) {
    const uint32_t ctr[4] = {coord >> 2, step, epoch, stream};
    const uint32_t key[2] = {(uint32_t)seed, (uint32_t)(seed >> 32)};
    uint32_t out[4];
    orc_philox4x32_10(ctr, key, out);
    return out[coord & 3u] >> 8;
}

// ---------------------------------------------------------------------------------------------
// Layout helpers (canonical packed layout): a plane is row-major with `row_bytes` per row;
// feature j occupies `cb` bits at bit position j*cb of the row, low bits first; cb = 2, 4, 4, 8
// for bits = 2, 3, 4, 8 (3-bit codes sit in 4-bit containers).
// ---------------------------------------------------------------------------------------------
int orc_container_bits(int bits) {
    switch (bits) { case 1: case 2: return 2; case 3: case 4: return 4; case 5: case 6: case 7: case 8: return 8; default: return 0; }
}

int64_t orc_row_bytes(int64_t n, int bits) {
    const int cb = orc_container_bits(bits);
    if (cb == 0 || n <= 0) return 0;
    const int64_t raw = (n * cb + 7) / 8;
    return (raw + 15) / 16 * 16;
}

static inline void put_code(uint8_t* row, int64_t j, int cb, uint32_t code) {
    const int64_t bit = j * cb;
    row[bit >> 3] = (uint8_t)(row[bit >> 3] | (code << (bit & 7)));
}

static inline uint32_t get_code(const uint8_t* row, int64_t j, int cb) {
    const int64_t bit = j * cb;
    return ((uint32_t)row[bit >> 3] >> (bit & 7)) & ((1u << cb) - 1u);
}

void orc_pack_codes(const uint8_t* codes, int64_t n, int bits, uint8_t* row_out, int64_t row_bytes) {
    const int cb = orc_container_bits(bits);
    std::memset(row_out, 0, (size_t)row_bytes);
    for (int64_t j = 0; j < n; ++j) put_code(row_out, j, cb, codes[j]);
}

void orc_unpack_codes(const uint8_t* row, int64_t n, int bits, uint8_t* codes_out) {
    const int cb = orc_container_bits(bits);
    for (int64_t j = 0; j < n; ++j) codes_out[j] = (uint8_t)get_code(row, j, cb);
}

// ---------------------------------------------------------------------------------------------
// Shared-base storage of the two samples (Section 2.2, "Overhead of Storing Samples"): the two
// quantizations of a value land on the same interval of levels, so they can only be its lower or
// its upper end.  It is enough to store the smaller of the two codes once (the base, `bits` wide)
// and one bit per sample saying whether that sample lies one level higher: bits + 2 instead of
// 2 * bits per value.  Layout: the base plane is an ordinary plane (container width cb); an "up"
// plane holds one bit per feature, feature j at bit j of its row, low bits first, row stride
// orc_up_row_bytes(n) = ceil(n / 8) rounded up to 16.  Decoding gives back exactly the two codes.
// Returns ORC_ERR_INVALID_ARG if the two codes of a value differ by more than one level (then they
// are not two samples of one value).
// ---------------------------------------------------------------------------------------------
int64_t orc_up_row_bytes(int64_t n) {
    if (n <= 0) return 0;
    return ((n + 7) / 8 + 15) / 16 * 16;
}

int orc_shared_base_encode(const uint8_t* plane1, const uint8_t* plane2, int64_t row_bytes, int64_t m, int64_t n, int bits,
                           uint8_t* base, uint8_t* up1, uint8_t* up2, int64_t up_row_bytes) {
    const int cb = orc_container_bits(bits);
    if (cb == 0) return ORC_ERR_UNSUPPORTED;
    if (!plane1 || !plane2 || !base || !up1 || !up2 || m <= 0 || n <= 0) return ORC_ERR_INVALID_ARG;
    if (row_bytes < orc_row_bytes(n, bits) || up_row_bytes < orc_up_row_bytes(n)) return ORC_ERR_INVALID_ARG;
    std::memset(base, 0, (size_t)(m * row_bytes));
    std::memset(up1, 0, (size_t)(m * up_row_bytes));
    std::memset(up2, 0, (size_t)(m * up_row_bytes));
    for (int64_t k = 0; k < m; ++k)
        for (int64_t j = 0; j < n; ++j) {
            const uint32_t c1 = get_code(plane1 + k * row_bytes, j, cb), c2 = get_code(plane2 + k * row_bytes, j, cb);
            const uint32_t lower = c1 < c2 ? c1 : c2;
            if (c1 - lower > 1u || c2 - lower > 1u) return ORC_ERR_INVALID_ARG;
            put_code(base + k * row_bytes, j, cb, lower);
            put_code(up1 + k * up_row_bytes, j, 1, c1 - lower);
            put_code(up2 + k * up_row_bytes, j, 1, c2 - lower);
        }
    return ORC_OK;
}

int orc_shared_base_decode(const uint8_t* base, const uint8_t* up1, const uint8_t* up2, int64_t row_bytes,
                           int64_t up_row_bytes, int64_t m, int64_t n, int bits, uint8_t* plane1, uint8_t* plane2) {
    const int cb = orc_container_bits(bits);
    if (cb == 0) return ORC_ERR_UNSUPPORTED;
    if (!plane1 || !plane2 || !base || !up1 || !up2 || m <= 0 || n <= 0) return ORC_ERR_INVALID_ARG;
    if (row_bytes < orc_row_bytes(n, bits) || up_row_bytes < orc_up_row_bytes(n)) return ORC_ERR_INVALID_ARG;
    std::memset(plane1, 0, (size_t)(m * row_bytes));
    std::memset(plane2, 0, (size_t)(m * row_bytes));
    for (int64_t k = 0; k < m; ++k)
        for (int64_t j = 0; j < n; ++j) {
            const uint32_t lower = get_code(base + k * row_bytes, j, cb);
            put_code(plane1 + k * row_bytes, j, cb, lower + get_code(up1 + k * up_row_bytes, j, 1));
            put_code(plane2 + k * row_bytes, j, cb, lower + get_code(up2 + k * up_row_bytes, j, 1));
        }
    return ORC_OK;
}

// ---------------------------------------------------------------------------------------------
// Column scaling: per-feature range over all rows (Supplement, "Column Scaling").
// ---------------------------------------------------------------------------------------------
int orc_column_range(const float* A, int64_t m, int64_t n, int64_t lda, float* lo, float* hi) {
    if (!A || !lo || !hi || m <= 0 || n <= 0 || lda < n) return ORC_ERR_INVALID_ARG;
    for (int64_t j = 0; j < n; ++j) { lo[j] = std::numeric_limits<float>::infinity(); hi[j] = -lo[j]; }
    for (int64_t k = 0; k < m; ++k)
        for (int64_t j = 0; j < n; ++j) {
            const float v = A[k * lda + j];
            if (!std::isfinite(v)) return ORC_ERR_NONFINITE;
            if (v < lo[j]) lo[j] = v;
            if (v > hi[j]) hi[j] = v;
        }
    return ORC_OK;
}

// ---------------------------------------------------------------------------------------------
// One stochastic rounding decision.  The value lies in cell l = [level_l, level_{l+1}] and moves
// up with probability p = (v - level_l) / (level_{l+1} - level_l), which makes E[Q(v)] = v
// (Section 2.1).  u24 * 2^-24 < p is evaluated in fp32 (u24 is exact there).
// ---------------------------------------------------------------------------------------------
static inline uint32_t round_up_if(uint32_t cell, float p, uint32_t u24) {
    const float u = (float)u24 * 5.9604644775390625e-08f;  // 2^-24, exact
    return cell + (u < p ? 1u : 0u);
}

// Uniform grid: inv = s / (hi - lo) (0 for a constant feature), t = (v - lo) * inv,
// l = clamp(floor(t), 0, s-1), p = t - l.  v = hi gives l = s-1, p = 1: always the top code.
static inline void uniform_cell(float v, float lo, float inv, int s, uint32_t* cell, float* p) {
    const float d = v - lo;
    const float t = d * inv;
    float fl = floorf(t);
    if (fl < 0.0f) fl = 0.0f;
    if (fl > (float)(s - 1)) fl = (float)(s - 1);
    *cell = (uint32_t)fl;
    *p = t - fl;
}

// Table grid: l = the largest index <= s-1 whose level is <= v; p by IEEE sub, sub, div.
static inline void table_cell(float v, const float* lev, int s, uint32_t* cell, float* p) {
    int l = 0;
    for (int i = 1; i <= s - 1; ++i)
        if (lev[i] <= v) l = i;
    const float w = lev[l + 1] - lev[l];
    const float d = v - lev[l];
    *cell = (uint32_t)l;
    *p = (w > 0.0f) ? d / w : 0.0f;
}

// Two independent unbiased quantizations of every sample, bit-packed (double sampling, Eq. (double)).
// Out: plane1, plane2 (m * row_bytes each), feat_lo (n), feat_step (n; uniform grid only: (hi-lo)/s).
// For ORC_LEVELS_TABLE `levels` is n x L ascending fp32 with levels[j][0] <= every value <= levels[j][s].
int orc_quantize_pair(const float* A, int64_t m, int64_t n, int64_t lda, int bits, int level_mode,
                      const float* levels, uint64_t seed, uint32_t pair, int symmetric, uint8_t* plane1, uint8_t* plane2,
                      int64_t row_bytes, float* feat_lo, float* feat_step);
int orc_quantize(const float* A, int64_t m, int64_t n, int64_t lda, int bits, int level_mode,
                 const float* levels, uint64_t seed, uint8_t* plane1, uint8_t* plane2,
                 int64_t row_bytes, float* feat_lo, float* feat_step) {
    return orc_quantize_pair(A, m, n, lda, bits, level_mode, levels, seed, 0u, 0, plane1, plane2, row_bytes, feat_lo, feat_step);
}

// Pair `pair` of quantizations of the same samples on the same grid: planes 2 pair + 1 and 2 pair + 2 of the
// sequence Q_1, Q_2, ... (pair 0 is orc_quantize).  symmetric != 0 (uniform levels only): the grid of the Supplement's
// "Column Scaling", [-M_j, M_j] with M_j the feature's largest |value|, instead of the feature's own range.
int orc_quantize_pair(const float* A, int64_t m, int64_t n, int64_t lda, int bits, int level_mode,
                      const float* levels, uint64_t seed, uint32_t pair, int symmetric, uint8_t* plane1, uint8_t* plane2,
                      int64_t row_bytes, float* feat_lo, float* feat_step) {
    if (symmetric && level_mode != ORC_LEVELS_UNIFORM) return ORC_ERR_INVALID_ARG;
    const int cb = orc_container_bits(bits);
    if (cb == 0) return ORC_ERR_UNSUPPORTED;
    if (level_mode == ORC_LEVELS_TABLE && bits > 4) return ORC_ERR_UNSUPPORTED;
    if (!A || !plane1 || !plane2 || !feat_lo || m <= 0 || n <= 0 || lda < n) return ORC_ERR_INVALID_ARG;
    if (row_bytes < orc_row_bytes(n, bits) || row_bytes % 16 != 0) return ORC_ERR_INVALID_ARG;
    if (level_mode == ORC_LEVELS_TABLE && !levels) return ORC_ERR_INVALID_ARG;
    if (level_mode == ORC_LEVELS_UNIFORM && !feat_step) return ORC_ERR_INVALID_ARG;
    const int L = 1 << bits, s = L - 1;

    std::vector<float> lo((size_t)n), hi((size_t)n), inv((size_t)n);
    const int rc = orc_column_range(A, m, n, lda, lo.data(), hi.data());
    if (rc != ORC_OK) return rc;
    for (int64_t j = 0; j < n; ++j) {
        if (symmetric) {
            hi[j] = std::fmax(std::fabs(lo[j]), std::fabs(hi[j]));
            lo[j] = -hi[j];
        }
        feat_lo[j] = lo[j];
        const float range = hi[j] - lo[j];
        inv[j] = (range > 0.0f) ? (float)s / range : 0.0f;
        if (level_mode == ORC_LEVELS_UNIFORM) feat_step[j] = range / (float)s;
    }
    std::memset(plane1, 0, (size_t)(m * row_bytes));
    std::memset(plane2, 0, (size_t)(m * row_bytes));
    for (int64_t k = 0; k < m; ++k) {
        uint8_t* r1 = plane1 + k * row_bytes;
        uint8_t* r2 = plane2 + k * row_bytes;
        for (int64_t j = 0; j < n; ++j) {
            const float v = A[k * lda + j];
            uint32_t cell; float p;
            if (level_mode == ORC_LEVELS_UNIFORM) uniform_cell(v, lo[j], inv[j], s, &cell, &p);
            else table_cell(v, levels + j * L, s, &cell, &p);
            put_code(r1, j, cb, round_up_if(cell, p, orc_u24_sample_pair(seed, (uint64_t)k, (uint32_t)j, 1, pair)));
            put_code(r2, j, cb, round_up_if(cell, p, orc_u24_sample_pair(seed, (uint64_t)k, (uint32_t)j, 2, pair)));
        }
    }
    return ORC_OK;
}

// Value a stored code stands for.
static inline double dequant(uint32_t code, int64_t j, int level_mode, int L, const float* feat_lo,
                             const float* feat_step, const float* levels) {
    if (level_mode == ORC_LEVELS_UNIFORM) return (double)feat_lo[j] + (double)code * (double)feat_step[j];
    return (double)levels[j * L + code];
}

void orc_dequantize_row(const uint8_t* row, int64_t n, int bits, int level_mode, const float* feat_lo,
                        const float* feat_step, const float* levels, double* out) {
    const int cb = orc_container_bits(bits), L = 1 << bits;
    for (int64_t j = 0; j < n; ++j)
        out[j] = dequant(get_code(row, j, cb), j, level_mode, L, feat_lo, feat_step, levels);
}

// ---------------------------------------------------------------------------------------------
// Row-scaled (l2) stochastic quantization of a vector (model Q3, gradient Q4): Supplement Eq.
// (quant2) with M(v) = ||v||_2.  Sign-magnitude, s_m = 2^(bits-1) - 1 magnitude intervals.
// M = (float) sqrt(sum in double of v_i^2); a = |v_i| / M; t = a * s_m; l = min(floor(t), s_m-1);
// p = t - l; Q_i = sgn(v_i) * M * ((l + up) / s_m), each op rounded to fp32.  Q(0) = 0.
// ---------------------------------------------------------------------------------------------
void orc_quantize_vector_norm(const float* v, int64_t n, int bits, uint64_t seed, uint32_t epoch, uint32_t step,
                              uint32_t stream, int norm, float* out, int32_t* codes_out_or_null);
void orc_quantize_vector(const float* v, int64_t n, int bits, uint64_t seed, uint32_t epoch,
                         uint32_t step, uint32_t stream, float* out, int32_t* codes_out_or_null) {
    orc_quantize_vector_norm(v, n, bits, seed, epoch, step, stream, 0, out, codes_out_or_null);
}

// The scaling function M(v) of Eq. (quant2) is left general by the Supplement ("Randomized Quantization"): norm 0 is
// the paper's choice ||v||_2, norm 1 is max |v_i| (every |v_i| / M still lies in [0, 1]; the largest entry is exact).
void orc_quantize_vector_norm(const float* v, int64_t n, int bits, uint64_t seed, uint32_t epoch, uint32_t step,
                              uint32_t stream, int norm, float* out, int32_t* codes_out_or_null) {
    const int sm = (1 << (bits - 1)) - 1;
    float M = 0.0f;
    if (norm == 1) {
        for (int64_t i = 0; i < n; ++i) M = fmaxf(M, fabsf(v[i]));
    } else {
        double ss = 0.0;
        for (int64_t i = 0; i < n; ++i) ss += (double)v[i] * (double)v[i];
        M = (float)std::sqrt(ss);
    }
    for (int64_t i = 0; i < n; ++i) {
        if (!(M > 0.0f)) { out[i] = 0.0f; if (codes_out_or_null) codes_out_or_null[i] = 0; continue; }
        const float a = fabsf(v[i]) / M;
        const float t = a * (float)sm;
        float fl = floorf(t);
        if (fl > (float)(sm - 1)) fl = (float)(sm - 1);
        const float p = t - fl;
        const uint32_t mag = round_up_if((uint32_t)fl, p, orc_u24_vector(seed, epoch, step, (uint32_t)i, stream));
        const float mu = (float)mag / (float)sm;
        const float q = M * mu;
        out[i] = (v[i] < 0.0f) ? -q : q;
        if (codes_out_or_null) codes_out_or_null[i] = (v[i] < 0.0f) ? -(int32_t)mag : (int32_t)mag;
    }
}

// ---------------------------------------------------------------------------------------------
// Mini-batch SGD over the stored double samples (Supplement "Double Sampling", footnote form):
//   g = 1/(2 B_t) sum_{k in batch} [ Q1(a_k) (Q2(a_k)^T x~ - b_k) + Q2(a_k) (Q1(a_k)^T x~ - b_k) ]
// with x~ = Q3(x) if model_bits > 0 else x, g^ = Q4(g) if grad_bits > 0 else g, and the update
// x <- x - lr * g^ in full precision.  Batch t holds rows [t*batch, min(m, (t+1)*batch)); the
// steps executed are batch_order[first_step .. first_step+num_steps) (identity order if null).
// grad_out_or_null (2n): the last executed step's gradient before and after Q4.
//
// Regulariser (main text Eq. (proxupdate): x <- prox_{lr R}(x - lr g^), the proximal operator
// being argmin_z 1/2 ||z - y||^2 + lr R(z)), applied coordinate by coordinate to y = x - lr g^:
//   reg 0  R = 0                          z = y
//   reg 1  R = c/2 ||x||_2^2              z = y * shrink,  shrink = fp32(1 / (1 + lr c))
//   reg 2  R = lambda ||x||_1             z = sign(y) max(|y| - thr, 0),  thr = fp32(lr lambda)
//   reg 3  R = indicator of x >= 0        z = max(y, 0)
//   reg 4  least-squares SVM (Supplement "Least Squares Support Vector Machines": the gradient
//          gains the term c x, kept in full precision):  z = y - fp32(lr c) * x_old
// The constants are rounded to fp32 once per call and the coordinate arithmetic is fp32 products
// and differences of fp32 values, evaluated in double and rounded once.
// ---------------------------------------------------------------------------------------------
static float orc_regularise(float y, float x_old, int reg, float cst) {
    if (reg == 1) return (float)((double)y * (double)cst);
    if (reg == 2) {
        const float mag = (float)((double)std::fabs(y) - (double)cst);
        return mag > 0.0f ? (y < 0.0f ? -mag : mag) : 0.0f;
    }
    if (reg == 3) return y > 0.0f ? y : 0.0f;
    if (reg == 4) return (float)((double)y - (double)cst * (double)x_old);
    return y;
}

int orc_sgd_epoch(const uint8_t* plane1, const uint8_t* plane2, int64_t row_bytes, int64_t m, int64_t n,
                  int bits, int level_mode, const float* feat_lo, const float* feat_step,
                  const float* levels, const float* b, float* x, int64_t batch, float lr,
                  int model_bits, int grad_bits, uint64_t seed, int64_t epoch, int64_t first_step,
                  int64_t num_steps, const int32_t* batch_order, float* grad_out_or_null, int reg, float reg_param,
                  int vector_norm) {
    if (vector_norm != 0 && vector_norm != 1) return ORC_ERR_INVALID_ARG;
    const int cb = orc_container_bits(bits);
    if (cb == 0) return ORC_ERR_UNSUPPORTED;
    if (reg < 0 || reg > 4 || (reg != 0 && reg != 3 && !(reg_param >= 0.0f))) return ORC_ERR_INVALID_ARG;
    float reg_cst = 0.0f;
    if (reg == 1) reg_cst = (float)(1.0 / (1.0 + (double)lr * (double)reg_param));
    if (reg == 2 || reg == 4) reg_cst = (float)((double)lr * (double)reg_param);
    if (level_mode == ORC_LEVELS_TABLE && bits > 4) return ORC_ERR_UNSUPPORTED;
    if (model_bits != 0 && (model_bits < 2 || model_bits > 8)) return ORC_ERR_UNSUPPORTED;
    if (grad_bits != 0 && (grad_bits < 2 || grad_bits > 8)) return ORC_ERR_UNSUPPORTED;
    if (!plane1 || !plane2 || !b || !x || m <= 0 || n <= 0 || batch <= 0) return ORC_ERR_INVALID_ARG;
    const int64_t T = (m + batch - 1) / batch;
    if (first_step < 0 || num_steps < 0 || first_step + num_steps > T) return ORC_ERR_INVALID_ARG;
    std::vector<float> xt((size_t)n), g((size_t)n), gq((size_t)n);
    std::vector<double> q1((size_t)n), q2((size_t)n), gacc((size_t)n);

    for (int64_t it = first_step; it < first_step + num_steps; ++it) {
        const int64_t t = batch_order ? (int64_t)batch_order[it] : it;
        if (t < 0 || t >= T) return ORC_ERR_INVALID_ARG;
        const int64_t r0 = t * batch, r1 = (r0 + batch < m) ? r0 + batch : m;
        if (model_bits > 0) orc_quantize_vector_norm(x, n, model_bits, seed, (uint32_t)epoch, (uint32_t)it, 3, vector_norm, xt.data(), nullptr);
        else std::memcpy(xt.data(), x, sizeof(float) * (size_t)n);
        for (int64_t j = 0; j < n; ++j) gacc[j] = 0.0;
        for (int64_t k = r0; k < r1; ++k) {
            orc_dequantize_row(plane1 + k * row_bytes, n, bits, level_mode, feat_lo, feat_step, levels, q1.data());
            orc_dequantize_row(plane2 + k * row_bytes, n, bits, level_mode, feat_lo, feat_step, levels, q2.data());
            double d1 = 0.0, d2 = 0.0;
            for (int64_t j = 0; j < n; ++j) { d1 += q1[j] * (double)xt[j]; d2 += q2[j] * (double)xt[j]; }
            const double res1 = d1 - (double)b[k], res2 = d2 - (double)b[k];
            for (int64_t j = 0; j < n; ++j) gacc[j] += q1[j] * res2 + q2[j] * res1;
        }
        const double scale = 1.0 / (2.0 * (double)(r1 - r0));
        for (int64_t j = 0; j < n; ++j) g[j] = (float)(gacc[j] * scale);
        const float* gu = g.data();
        if (grad_bits > 0) {
            orc_quantize_vector_norm(g.data(), n, grad_bits, seed, (uint32_t)epoch, (uint32_t)it, 4, vector_norm, gq.data(), nullptr);
            gu = gq.data();
        }
        for (int64_t j = 0; j < n; ++j) {
            const float y = (float)((double)x[j] - (double)lr * (double)gu[j]);
            x[j] = orc_regularise(y, x[j], reg, reg_cst);
        }
        if (grad_out_or_null && it == first_step + num_steps - 1) {
            std::memcpy(grad_out_or_null, g.data(), sizeof(float) * (size_t)n);
            std::memcpy(grad_out_or_null + n, gu, sizeof(float) * (size_t)n);
        }
    }
    return ORC_OK;
}

// The same step with the naive single-sample estimator Q(a)(Q(a)^T x - b) (Section 2.2; biased) and
// with the one-sided double-sampled estimator Q1(a)(Q2(a)^T x - b) (Eq. (double)); diagnostics that
// pin the bias statements.  which: 0 naive on plane1, 1 one-sided, 2 symmetrised.  Mean over all
// m rows at fixed x, written to g_out (n doubles).
int orc_estimator_mean(const uint8_t* plane1, const uint8_t* plane2, int64_t row_bytes, int64_t m, int64_t n,
                       int bits, int level_mode, const float* feat_lo, const float* feat_step,
                       const float* levels, const float* b, const float* x, int which, double* g_out) {
    std::vector<double> q1((size_t)n), q2((size_t)n);
    for (int64_t j = 0; j < n; ++j) g_out[j] = 0.0;
    for (int64_t k = 0; k < m; ++k) {
        orc_dequantize_row(plane1 + k * row_bytes, n, bits, level_mode, feat_lo, feat_step, levels, q1.data());
        orc_dequantize_row(plane2 + k * row_bytes, n, bits, level_mode, feat_lo, feat_step, levels, q2.data());
        double d1 = 0.0, d2 = 0.0;
        for (int64_t j = 0; j < n; ++j) { d1 += q1[j] * (double)x[j]; d2 += q2[j] * (double)x[j]; }
        const double res1 = d1 - (double)b[k], res2 = d2 - (double)b[k];
        for (int64_t j = 0; j < n; ++j) {
            if (which == 0) g_out[j] += q1[j] * res1;
            else if (which == 1) g_out[j] += q1[j] * res2;
            else g_out[j] += 0.5 * (q1[j] * res2 + q2[j] * res1);
        }
    }
    for (int64_t j = 0; j < n; ++j) g_out[j] /= (double)m;
    return ORC_OK;
}

// ---------------------------------------------------------------------------------------------
// Loss, Eq. (leastsquares): 1/(2m) sum (a_k^T x - b_k)^2 on the original samples, or its unbiased
// estimate from the two planes, 1/(2m) sum (Q1(a_k)^T x - b_k)(Q2(a_k)^T x - b_k) (the two factors
// are independent given a_k, the argument of Section 2.2).
// ---------------------------------------------------------------------------------------------
int orc_loss_dense(const float* A, int64_t m, int64_t n, int64_t lda, const float* b, const float* x, double* loss_out) {
    if (!A || !b || !x || !loss_out || m <= 0 || n <= 0 || lda < n) return ORC_ERR_INVALID_ARG;
    double acc = 0.0;
    for (int64_t k = 0; k < m; ++k) {
        double d = 0.0;
        for (int64_t j = 0; j < n; ++j) d += (double)A[k * lda + j] * (double)x[j];
        const double r = d - (double)b[k];
        acc += r * r;
    }
    *loss_out = acc / (2.0 * (double)m);
    return ORC_OK;
}

int orc_loss_codes(const uint8_t* plane1, const uint8_t* plane2, int64_t row_bytes, int64_t m, int64_t n, int bits,
                   int level_mode, const float* feat_lo, const float* feat_step, const float* levels,
                   const float* b, const float* x, double* loss_out) {
    if (orc_container_bits(bits) == 0) return ORC_ERR_UNSUPPORTED;
    if (!plane1 || !plane2 || !b || !x || !loss_out || m <= 0 || n <= 0) return ORC_ERR_INVALID_ARG;
    std::vector<double> q1((size_t)n), q2((size_t)n);
    double acc = 0.0;
    for (int64_t k = 0; k < m; ++k) {
        orc_dequantize_row(plane1 + k * row_bytes, n, bits, level_mode, feat_lo, feat_step, levels, q1.data());
        orc_dequantize_row(plane2 + k * row_bytes, n, bits, level_mode, feat_lo, feat_step, levels, q2.data());
        double d1 = 0.0, d2 = 0.0;
        for (int64_t j = 0; j < n; ++j) { d1 += q1[j] * (double)x[j]; d2 += q2[j] * (double)x[j]; }
        acc += (d1 - (double)b[k]) * (d2 - (double)b[k]);
    }
    *loss_out = acc / (2.0 * (double)m);
    return ORC_OK;
}

// Section 4.1 "Quantizing Polynomials": with d independent quantizations Q_1 .. Q_d of a sample a, the estimate
// of P(a^T x) for P(z) = sum_{i=0}^{d} coef_i z^i is  Q(P) = sum_i coef_i prod_{j <= i} Q_j(a)^T x  (unbiased: the
// factors of a product are independent).  planes[j] is Q_{j+1} (m x row_bytes, all on one grid).  rows_out[k] is
// Q(P) of sample k, times scale_or_null[k] where that is given (the label b_k of Section 4.2's protocol).
int orc_poly_rows(const uint8_t* const* planes, int d, int64_t row_bytes, int64_t m, int64_t n, int bits, int level_mode,
                  const float* feat_lo, const float* feat_step, const float* levels, const float* x,
                  const double* coef, const float* scale_or_null, double* rows_out) {
    if (orc_container_bits(bits) == 0) return ORC_ERR_UNSUPPORTED;
    if (!planes || d < 0 || !x || !coef || !rows_out || m <= 0 || n <= 0) return ORC_ERR_INVALID_ARG;
    std::vector<double> q((size_t)n);
    for (int64_t k = 0; k < m; ++k) {
        double value = coef[0], prod = 1.0;
        for (int i = 1; i <= d; ++i) {
            orc_dequantize_row(planes[i - 1] + k * row_bytes, n, bits, level_mode, feat_lo, feat_step, levels, q.data());
            double z = 0.0;
            for (int64_t j = 0; j < n; ++j) z += q[j] * (double)x[j];
            prod *= z;
            value += coef[i] * prod;
        }
        rows_out[k] = scale_or_null ? (double)scale_or_null[k] * value : value;
    }
    return ORC_OK;
}

// The gradient of Section 4.2's protocol for given per-sample factors c_k (there: b_k Q(P)_k): the mean of
// c_k Q_{d+1}(a_k) over the samples, with `plane` holding Q_{d+1}.
int orc_weighted_plane_mean(const uint8_t* plane, int64_t row_bytes, int64_t m, int64_t n, int bits, int level_mode,
                            const float* feat_lo, const float* feat_step, const float* levels, const double* c,
                            double* g_out) {
    if (orc_container_bits(bits) == 0) return ORC_ERR_UNSUPPORTED;
    if (!plane || !c || !g_out || m <= 0 || n <= 0) return ORC_ERR_INVALID_ARG;
    std::vector<double> q((size_t)n);
    for (int64_t j = 0; j < n; ++j) g_out[j] = 0.0;
    for (int64_t k = 0; k < m; ++k) {
        orc_dequantize_row(plane + k * row_bytes, n, bits, level_mode, feat_lo, feat_step, levels, q.data());
        for (int64_t j = 0; j < n; ++j) g_out[j] += c[k] * q[j];
    }
    for (int64_t j = 0; j < n; ++j) g_out[j] /= (double)m;
    return ORC_OK;
}

// ---------------------------------------------------------------------------------------------
// Variance-optimal levels (Section 3).  The feature is normalised to [0, 1]; the candidate
// endpoints are the M+1 edges d_i = i/M of M equal bins ("Discretization"); only bin counts are
// kept and every point stands at its bin centre, so with positions in units of 1/(2M)
//   4 M^2 V(j, m) = sum_{i=j}^{m-1} cnt_i (2m - (2i+1)) ((2i+1) - 2j)
// is an exact integer: err(x, [a, b]) = (b - x)(x - a) summed over the points of [d_j, d_m].
// ---------------------------------------------------------------------------------------------

// Bin of a value: the uniform-grid cell with s = M (same pinned fp32 arithmetic).
int orc_histogram(const float* A, int64_t m, int64_t n, int64_t lda, int M, const float* lo, const float* hi,
                  uint32_t* counts /* n x M, zeroed here */) {
    if (!A || !lo || !hi || !counts || m <= 0 || n <= 0 || M < 1 || lda < n) return ORC_ERR_INVALID_ARG;
    std::memset(counts, 0, sizeof(uint32_t) * (size_t)(n * M));
    for (int64_t j = 0; j < n; ++j) {
        const float range = hi[j] - lo[j];
        const float inv = (range > 0.0f) ? (float)M / range : 0.0f;
        for (int64_t k = 0; k < m; ++k) {
            uint32_t cell; float p;
            uniform_cell(A[k * lda + j], lo[j], inv, M, &cell, &p);
            counts[j * M + cell] += 1u;
        }
    }
    return ORC_OK;
}

// V(j, m) straight from the definition: a sum over the bins of [d_j, d_m].
uint64_t orc_interval_cost(const uint32_t* cnt, int j, int m) {
    uint64_t v = 0;
    for (int i = j; i < m; ++i)
        v += (uint64_t)cnt[i] * (uint64_t)(2 * m - (2 * i + 1)) * (uint64_t)((2 * i + 1) - 2 * j);
    return v;
}

// The same V(j, m) in O(1) from prefix sums over the bins: with x_i = 2i+1, a = 2j, b = 2m,
//   sum c_i (b - x_i)(x_i - a) = (a + b) S1 - S2 - a b S0,   S_p = sum_{i=j}^{m-1} c_i x_i^p.
// Every term is an exact integer below 2^63 for N <= 10^9 points and M <= 1024 bins.
struct PrefixSums {
    std::vector<uint64_t> p0, p1, p2;
    PrefixSums(const uint32_t* cnt, int M) : p0((size_t)M + 1, 0), p1((size_t)M + 1, 0), p2((size_t)M + 1, 0) {
        for (int i = 0; i < M; ++i) {
            const uint64_t x = (uint64_t)(2 * i + 1), c = cnt[i];
            p0[i + 1] = p0[i] + c; p1[i + 1] = p1[i] + c * x; p2[i + 1] = p2[i] + c * x * x;
        }
    }
    uint64_t cost(int j, int m) const {
        const uint64_t a = (uint64_t)(2 * j), b = (uint64_t)(2 * m);
        return (a + b) * (p1[m] - p1[j]) - (p2[m] - p2[j]) - a * b * (p0[m] - p0[j]);
    }
};

uint64_t orc_interval_cost_prefix(const uint32_t* cnt, int M, int j, int m) {
    return PrefixSums(cnt, M).cost(j, m);
}

// The recursion T(k, m) = min_{j in [k-1, m-1]} T(k-1, j) + V(j, m) with T(1, m) = V(0, m),
// ties to the smallest j; the answer is T(s, M) and the chosen edges idx[0] = 0 < ... < idx[s] = M.
// Needs s <= M.
int orc_levels_dp(const uint32_t* cnt, int M, int s, int32_t* idx_out /* s+1 */, uint64_t* objective_out) {
    if (!cnt || !idx_out || M < 1 || s < 1 || s > M) return ORC_ERR_INVALID_ARG;
    const uint64_t INF = std::numeric_limits<uint64_t>::max();
    const PrefixSums V(cnt, M);
    std::vector<uint64_t> T((size_t)(s + 1) * (size_t)(M + 1), INF);
    std::vector<int32_t> arg((size_t)(s + 1) * (size_t)(M + 1), -1);
    for (int mm = 1; mm <= M; ++mm) { T[(size_t)1 * (M + 1) + mm] = V.cost(0, mm); arg[(size_t)1 * (M + 1) + mm] = 0; }
    for (int k = 2; k <= s; ++k)
        for (int mm = k; mm <= M; ++mm) {
            uint64_t best = INF; int32_t bj = -1;
            for (int j = k - 1; j <= mm - 1; ++j) {
                const uint64_t c = T[(size_t)(k - 1) * (M + 1) + j] + V.cost(j, mm);
                if (c < best) { best = c; bj = j; }
            }
            T[(size_t)k * (M + 1) + mm] = best; arg[(size_t)k * (M + 1) + mm] = bj;
        }
    if (objective_out) *objective_out = T[(size_t)s * (M + 1) + M];
    int mm = M;
    for (int k = s; k >= 1; --k) { idx_out[k] = mm; mm = arg[(size_t)k * (M + 1) + mm]; }
    idx_out[0] = 0;
    return ORC_OK;
}

// The plain definition: try every set of s-1 interior edges, keep the cheapest (first in
// lexicographic order among equals).  Tiny grids only.
int orc_levels_bruteforce(const uint32_t* cnt, int M, int s, int32_t* idx_out, uint64_t* objective_out) {
    if (!cnt || !idx_out || M < 1 || s < 1 || s > M) return ORC_ERR_INVALID_ARG;
    std::vector<int32_t> cur((size_t)s + 1), best((size_t)s + 1);
    uint64_t best_cost = std::numeric_limits<uint64_t>::max();
    cur[0] = 0; cur[s] = M;
    for (int i = 1; i < s; ++i) cur[i] = i;
    for (;;) {
        uint64_t c = 0;
        for (int i = 0; i < s; ++i) c += orc_interval_cost(cnt, cur[i], cur[i + 1]);
        if (c < best_cost) { best_cost = c; best = cur; }
        int pos = s - 1;
        while (pos >= 1 && cur[pos] == M - (s - pos)) --pos;
        if (pos < 1) break;
        ++cur[pos];
        for (int i = pos + 1; i < s; ++i) cur[i] = cur[i - 1] + 1;
    }
    for (int i = 0; i <= s; ++i) idx_out[i] = best[i];
    if (objective_out) *objective_out = best_cost;
    return ORC_OK;
}

// Exact problem on raw points (Section 3.1): total variance sum err(x, I) in double for a given
// ascending set of endpoints e[0..s] covering all points; used to pin the Lemma that optimal
// endpoints can be taken at data points.
double orc_total_variance(const double* pts, int64_t N, const double* e, int s) {
    double tot = 0.0;
    for (int64_t i = 0; i < N; ++i) {
        int c = 0;
        while (c < s - 1 && pts[i] > e[c + 1]) ++c;
        tot += (e[c + 1] - pts[i]) * (pts[i] - e[c]);
    }
    return tot;
}

// Levels of one feature from its chosen edges: lo + (hi - lo) * (idx / M), each op rounded to
// fp32, first and last forced to lo and hi.
void orc_levels_from_idx(const int32_t* idx, int s, int M, float lo, float hi, float* lev_out) {
    const float range = hi - lo;
    for (int i = 0; i <= s; ++i) {
        const float frac = (float)idx[i] / (float)M;
        const float off = range * frac;
        lev_out[i] = lo + off;
    }
    lev_out[0] = lo; lev_out[s] = hi;
}

// Whole call: ranges, one histogram pass, DP per feature.  levels_out is n x L (L = 2^bits),
// objective_out_or_null (n) holds 4 M^2 * N * MV of the chosen levels in normalised units.
// A constant feature (hi == lo) puts every point in bin 0 and still returns increasing edges.
int orc_optimal_levels(const float* A, int64_t m, int64_t n, int64_t lda, int bits, int M,
                       float* levels_out, uint64_t* objective_out_or_null) {
    if (bits != 2 && bits != 3 && bits != 4) return ORC_ERR_UNSUPPORTED;
    const int L = 1 << bits, s = L - 1;
    if (!A || !levels_out || m <= 0 || n <= 0 || lda < n || M < s) return ORC_ERR_INVALID_ARG;
    std::vector<float> lo((size_t)n), hi((size_t)n);
    int rc = orc_column_range(A, m, n, lda, lo.data(), hi.data());
    if (rc != ORC_OK) return rc;
    std::vector<uint32_t> counts((size_t)(n * M));
    rc = orc_histogram(A, m, n, lda, M, lo.data(), hi.data(), counts.data());
    if (rc != ORC_OK) return rc;
    std::vector<int32_t> idx((size_t)s + 1);
    for (int64_t j = 0; j < n; ++j) {
        uint64_t obj = 0;
        rc = orc_levels_dp(counts.data() + j * M, M, s, idx.data(), &obj);
        if (rc != ORC_OK) return rc;
        orc_levels_from_idx(idx.data(), s, M, lo[j], hi[j], levels_out + j * L);
        if (objective_out_or_null) objective_out_or_null[j] = obj;
    }
    return ORC_OK;
}

}  // extern "C"
