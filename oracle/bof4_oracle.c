/*
 * CPU oracle for block-wise 4-bit optimal-float quantisation (BOF4 / BOF4-S / OPQ).
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain definition of what the CUDA library
 * must compute.  It shares no code, header, table or helper with the CUDA path and must never
 * be linked into or called from the product.  Only the test-suite, the smoke check and the
 * benchmark's CPU-baseline leg may load it.
 *
 * Build: gcc -O2 -std=c11 -fno-fast-math -ffp-contract=off -fopenmp -shared -fPIC
 * All fp32 operations are IEEE round-to-nearest-even, never contracted into FMAs, subnormals
 * kept.  Sums that the paper defines without an order are taken in index order inside fixed
 * chunks of ORC_CHUNK blocks, the chunk partials then added in chunk order, so the result does
 * not depend on the number of threads.
 *
 * Notation follows the paper: block size I, B = n/I blocks, block constant m = w_b^max,
 * normalised weight x, 16 reconstruction levels xhat[0..15] ascending (0-based index = the
 * paper's l-1), 15 decision thresholds xi[0..14].
 *
 * Readings where the paper is silent (each is also listed in the design notes):
 *  - thresholds are the midpoints of adjacent levels (nearest-neighbour rule, Sec. 3.2 /
 *    App. B.2), a tie x == xi goes to the upper level (half-open regions [xi(l-1), xi(l)));
 *  - signed block maximum with several elements of maximal magnitude: the lowest index wins;
 *  - an all-zero block has m = 0 and x = 0 for every element;
 *  - a region whose weight sum is zero keeps its level;
 *  - the weighted median returned is the minimiser of the stated MAE objective, i.e. the
 *    first sorted sample whose cumulative weight reaches half of the total;
 *  - OPQ block statistics are the two-pass formulas of App. E in fp32 with a balanced binary
 *    summation tree over the block;
 *  - quantise / dequantise / OPQ accept n that is not a multiple of I: the last block is simply
 *    shorter (its own maximum, its own mean and deviation over its own length; for the tree
 *    sums it is padded with zeros to the next power of two; a code byte that has only one
 *    weight carries 0 in its low nibble).  The EM functions need whole blocks.
 *
 * Parity pins: every function here is pinned by tests/test_oracle_pins.py (printed codebooks
 * of Tab. 6-8 as fixed points, exact DP optimum on tiny inputs, library k-means / medians in
 * the equal-constant special case, numerical integration of the Gaussian centroid formula,
 * closed forms and invariants).  Absolute error values on real LLM weights (Tab. 1, 9) are
 * "parity unpinned": the weights are not available.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define L 16
#define ORC_CHUNK 4096 /* blocks per summation chunk */

/* ---------------------------------------------------------------- helpers ------------- */

static float bf16_bits_to_f32(uint16_t h)
{
    uint32_t u = (uint32_t)h << 16;
    float f;
    memcpy(&f, &u, 4);
    return f;
}

/* fp32 -> bfloat16, round to nearest, ties to even (finite inputs). */
static uint16_t f32_to_bf16_rne(float f)
{
    uint32_t u;
    memcpy(&u, &f, 4);
    if ((u & 0x7f800000u) == 0x7f800000u) /* inf / nan: truncate, keep nan-ness */
        return (uint16_t)((u >> 16) | ((u & 0xffffu) ? 0x40u : 0u));
    uint32_t lower = u & 0xffffu;
    uint32_t upper = u >> 16;
    if (lower > 0x8000u || (lower == 0x8000u && (upper & 1u)))
        upper += 1u;
    return (uint16_t)upper;
}

void orc_f32_to_bf16(const float *in, int64_t n, uint16_t *out)
{
    for (int64_t i = 0; i < n; ++i)
        out[i] = f32_to_bf16_rne(in[i]);
}

void orc_bf16_to_f32(const uint16_t *in, int64_t n, float *out)
{
    for (int64_t i = 0; i < n; ++i)
        out[i] = bf16_bits_to_f32(in[i]);
}

/* Block constant: Eq. 1 (norm = 0, absolute maximum) or Eq. 4 (norm = 1, the element of
 * largest magnitude with its sign; lowest index on ties). */
static float block_constant(const float *w, int I, int norm)
{
    float best_abs = 0.0f;
    int best_j = -1;
    for (int i = 0; i < I; ++i) {
        float a = fabsf(w[i]);
        if (a > best_abs) {
            best_abs = a;
            best_j = i;
        }
    }
    if (best_j < 0)
        return 0.0f; /* all-zero block */
    return norm ? w[best_j] : best_abs;
}

/* Eq. 2, with the 0/0 reading x = 0. */
static float normalise(float w, float m)
{
    return (m == 0.0f) ? 0.0f : w / m;
}

/* Decision thresholds: midpoints of adjacent levels (fp32 add, then exact halving). */
void orc_thresholds(const float *xhat, float *xi)
{
    for (int j = 0; j < L - 1; ++j)
        xi[j] = (xhat[j] + xhat[j + 1]) * 0.5f;
}

/* Region index of x: the number of thresholds that are <= x (Sec. 3.2, regions
 * [xi(l-1), xi(l)) with xi(0) = -inf, xi(16) = +inf). */
static int region_of(float x, const float *xi)
{
    int c = 0;
    for (int j = 0; j < L - 1; ++j)
        c += (xi[j] <= x) ? 1 : 0;
    return c;
}

/* Length of block b of a tensor of n weights: I, or the remainder for a ragged last block. */
static int block_len(int64_t n, int I, int64_t b)
{
    int64_t left = n - b * I;
    return (int)(left < I ? left : I);
}

/* The blocks of a list of tensors laid out one after the other: every tensor is cut into blocks
 * of I weights from its own start, its last block being shorter when its length is not a multiple
 * of I (a block never spans two tensors).  Returns the number of blocks; off[b] is the position
 * of block b in the concatenated data, len[b] its length. */
static int64_t build_blocks(const int64_t *seg, int n_seg, int I, int64_t **off, int **len)
{
    int64_t B = 0;
    for (int s = 0; s < n_seg; ++s)
        B += (seg[s] + I - 1) / I;
    *off = malloc(sizeof(int64_t) * (size_t)(B > 0 ? B : 1));
    *len = malloc(sizeof(int) * (size_t)(B > 0 ? B : 1));
    int64_t b = 0, pos = 0;
    for (int s = 0; s < n_seg; ++s) {
        int64_t nb = (seg[s] + I - 1) / I;
        for (int64_t k = 0; k < nb; ++k, ++b) {
            (*off)[b] = pos + k * I;
            (*len)[b] = block_len(seg[s], I, k);
        }
        pos += seg[s];
    }
    return B;
}

void orc_block_constants(const float *w, int64_t n, int I, int norm, float *m_out)
{
    int64_t B = (n + I - 1) / I;
#pragma omp parallel for schedule(static)
    for (int64_t b = 0; b < B; ++b)
        m_out[b] = block_constant(w + b * I, block_len(n, I, b), norm);
}

/* ---------------------------------------------------------------- quantise ------------ */

/* Sec. 2.1: per block, constant m, normalise, nearest level; stored as one 4-bit code per
 * weight (even element in the high nibble of its byte) plus m per block. */
void orc_quantize(const float *w, int64_t n, int I, int norm, const float *xhat,
                  uint8_t *codes, float *scales)
{
    float xi[L - 1];
    orc_thresholds(xhat, xi);
    int64_t B = (n + I - 1) / I;
#pragma omp parallel for schedule(static)
    for (int64_t b = 0; b < B; ++b) {
        const float *wb = w + b * I;
        int len = block_len(n, I, b);
        float m = block_constant(wb, len, norm);
        scales[b] = m;
        for (int i = 0; i < len; i += 2) {
            int c0 = region_of(normalise(wb[i], m), xi);
            int c1 = (i + 1 < len) ? region_of(normalise(wb[i + 1], m), xi) : 0;
            codes[(b * I + i) / 2] = (uint8_t)((c0 << 4) | c1);
        }
    }
}

/* Eq. 3: Q_b(w) = m * xhat(code), one fp32 multiplication. */
void orc_dequantize(const uint8_t *codes, const float *scales, int64_t n, int I,
                    const float *xhat, float *out)
{
    int64_t B = (n + I - 1) / I;
#pragma omp parallel for schedule(static)
    for (int64_t b = 0; b < B; ++b) {
        float m = scales[b];
        int len = block_len(n, I, b);
        for (int i = 0; i < len; ++i) {
            int64_t k = b * I + i;
            uint8_t byte = codes[k / 2];
            int c = (k & 1) ? (byte & 15) : (byte >> 4);
            out[k] = m * xhat[c];
        }
    }
}

/* ---------------------------------------------------------------- EM, MSE ------------- */

/* One expectation + accumulation pass with the levels held fixed (Eq. 6 and the first line
 * of the un-normalised-domain error, App. B.3):
 *   s1[l] = sum m^2 x,  s0[l] = sum m^2,  cnt[l] = K_l,  err = sum (w - m xhat(l))^2. */
static void em_accumulate_mse_impl(const float *w, const int64_t *seg, int n_seg, int I, int norm,
                                   const float *xhat, int unit, double *s1, double *s0, uint64_t *cnt,
                                   double *err);

void orc_em_accumulate_mse(const float *w, int64_t n, int I, int norm, const float *xhat,
                           double *s1, double *s0, uint64_t *cnt, double *err)
{
    em_accumulate_mse_impl(w, &n, 1, I, norm, xhat, 0, s1, s0, cnt, err);
}

/* The same over a list of n_seg tensors of seg[] weights each, stored one after the other. */
void orc_em_accumulate_mse_seg(const float *w, const int64_t *seg, int n_seg, int I, int norm,
                               const float *xhat, int unit, double *s1, double *s0, uint64_t *cnt,
                               double *err)
{
    em_accumulate_mse_impl(w, seg, n_seg, I, norm, xhat, unit, s1, s0, cnt, err);
}

/* The same pass for the quantisation error of the NORMALISED weights (App. D, the plain-mean
 * centroid): every sample has weight 1, s1[l] = sum x, s0[l] = K_l, err = sum (x - xhat(l))^2. */
void orc_em_accumulate_mse_normdom(const float *w, int64_t n, int I, int norm, const float *xhat,
                                   double *s1, double *s0, uint64_t *cnt, double *err)
{
    em_accumulate_mse_impl(w, &n, 1, I, norm, xhat, 1, s1, s0, cnt, err);
}

static void em_accumulate_mse_impl(const float *w, const int64_t *seg, int n_seg, int I, int norm,
                                   const float *xhat, int unit, double *s1, double *s0, uint64_t *cnt,
                                   double *err)
{
    float xi[L - 1];
    orc_thresholds(xhat, xi);
    int64_t *boff;
    int *blen;
    int64_t B = build_blocks(seg, n_seg, I, &boff, &blen);
    int64_t nchunk = (B + ORC_CHUNK - 1) / ORC_CHUNK;
    double *p1 = calloc((size_t)nchunk * L, sizeof(double));
    double *p0 = calloc((size_t)nchunk * L, sizeof(double));
    uint64_t *pc = calloc((size_t)nchunk * L, sizeof(uint64_t));
    double *pe = calloc((size_t)nchunk, sizeof(double));
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t ch = 0; ch < nchunk; ++ch) {
        int64_t b0 = ch * ORC_CHUNK, b1 = b0 + ORC_CHUNK;
        if (b1 > B)
            b1 = B;
        double *a1 = p1 + ch * L, *a0 = p0 + ch * L;
        uint64_t *ac = pc + ch * L;
        double e = 0.0;
        for (int64_t b = b0; b < b1; ++b) {
            const float *wb = w + boff[b];
            const int Ib = blen[b];
            float m = block_constant(wb, Ib, norm);
            double md = (double)m;
            for (int i = 0; i < Ib; ++i) {
                float x = normalise(wb[i], m);
                int c = region_of(x, xi);
                if (unit) {
                    a1[c] += (double)x;
                    a0[c] += 1.0;
                    ac[c] += 1;
                    double d = (double)x - (double)xhat[c];
                    e += d * d;
                } else {
                    a1[c] += md * md * (double)x;
                    a0[c] += md * md;
                    ac[c] += 1;
                    double d = (double)wb[i] - md * (double)xhat[c];
                    e += d * d;
                }
            }
        }
        pe[ch] = e;
    }
    for (int l = 0; l < L; ++l) {
        s1[l] = 0.0;
        s0[l] = 0.0;
        cnt[l] = 0;
    }
    *err = 0.0;
    for (int64_t ch = 0; ch < nchunk; ++ch) {
        for (int l = 0; l < L; ++l) {
            s1[l] += p1[ch * L + l];
            s0[l] += p0[ch * L + l];
            cnt[l] += pc[ch * L + l];
        }
        *err += pe[ch];
    }
    free(p1);
    free(p0);
    free(pc);
    free(pe);
    free(boff);
    free(blen);
}

/* ---------------------------------------------------------------- EM, MAE ------------- */

typedef struct {
    float x; /* normalised weight */
    float a; /* |m| of its block: the weight of the weighted median (Eq. 8, App. B.3) */
} member_t;

static int cmp_member(const void *p, const void *q)
{
    float a = ((const member_t *)p)->x, b = ((const member_t *)q)->x;
    return (a > b) - (a < b);
}

/* One pass for the MAE criterion.  For every region the members are sorted ascending and the
 * weighted median is the first sample whose cumulative weight reaches half the total weight:
 * the minimiser of f(xh) = sum a_k |x_k - xh| (objective of App. B.3, "MAE Optimization").
 *   med[l]  = that sample (unchanged input level when the region's total weight is 0),
 *   wsum[l] = total weight of the region, cnt[l] = K_l, err = sum |w - m xhat(l)|. */
static void em_accumulate_mae_impl(const float *w, const int64_t *seg, int n_seg, int I, int norm,
                                   const float *xhat, int unit, float *med, double *wsum, uint64_t *cnt,
                                   double *err);

void orc_em_accumulate_mae(const float *w, int64_t n, int I, int norm, const float *xhat,
                           float *med, double *wsum, uint64_t *cnt, double *err)
{
    em_accumulate_mae_impl(w, &n, 1, I, norm, xhat, 0, med, wsum, cnt, err);
}

/* The same over a list of n_seg tensors of seg[] weights each, stored one after the other. */
void orc_em_accumulate_mae_seg(const float *w, const int64_t *seg, int n_seg, int I, int norm,
                               const float *xhat, int unit, float *med, double *wsum, uint64_t *cnt,
                               double *err)
{
    em_accumulate_mae_impl(w, seg, n_seg, I, norm, xhat, unit, med, wsum, cnt, err);
}

/* Normalised-domain variant (App. D, the plain median): all weights 1, err = sum |x - xhat(l)|. */
void orc_em_accumulate_mae_normdom(const float *w, int64_t n, int I, int norm, const float *xhat,
                                   float *med, double *wsum, uint64_t *cnt, double *err)
{
    em_accumulate_mae_impl(w, &n, 1, I, norm, xhat, 1, med, wsum, cnt, err);
}

static void em_accumulate_mae_impl(const float *w, const int64_t *seg, int n_seg, int I, int norm,
                                   const float *xhat, int unit, float *med, double *wsum, uint64_t *cnt,
                                   double *err)
{
    float xi[L - 1];
    orc_thresholds(xhat, xi);
    int64_t n = 0;
    for (int s = 0; s < n_seg; ++s)
        n += seg[s];
    int64_t *boff;
    int *blen;
    int64_t B = build_blocks(seg, n_seg, I, &boff, &blen);
    uint8_t *code = malloc((size_t)(n > 0 ? n : 1));
    float *xs = malloc(sizeof(float) * (size_t)(n > 0 ? n : 1));
    float *ms = malloc(sizeof(float) * (size_t)(n > 0 ? n : 1)); /* |m| of the block of every weight */
    double e = 0.0;
    for (int l = 0; l < L; ++l)
        cnt[l] = 0;
    for (int64_t b = 0; b < B; ++b) {
        const float *wb = w + boff[b];
        const int Ib = blen[b];
        float m = block_constant(wb, Ib, norm);
        for (int i = 0; i < Ib; ++i) {
            float x = normalise(wb[i], m);
            int c = region_of(x, xi);
            xs[boff[b] + i] = x;
            ms[boff[b] + i] = fabsf(m);
            code[boff[b] + i] = (uint8_t)c;
            cnt[c] += 1;
            e += unit ? fabs((double)x - (double)xhat[c])
                      : fabs((double)wb[i] - (double)m * (double)xhat[c]);
        }
    }
    *err = e;
#pragma omp parallel for schedule(dynamic, 1)
    for (int l = 0; l < L; ++l) {
        med[l] = xhat[l];
        wsum[l] = 0.0;
        if (cnt[l] == 0)
            continue;
        member_t *mem = malloc(sizeof(member_t) * (size_t)cnt[l]);
        int64_t k = 0;
        for (int64_t j = 0; j < n; ++j)
            if (code[j] == l) {
                mem[k].x = xs[j];
                mem[k].a = unit ? 1.0f : ms[j];
                ++k;
            }
        qsort(mem, (size_t)k, sizeof(member_t), cmp_member);
        double total = 0.0;
        for (int64_t j = 0; j < k; ++j)
            total += (double)mem[j].a;
        wsum[l] = total;
        if (total > 0.0) {
            double half = total * 0.5, c = 0.0;
            for (int64_t j = 0; j < k; ++j) {
                c += (double)mem[j].a;
                if (c >= half) {
                    med[l] = mem[j].x;
                    break;
                }
            }
        }
        free(mem);
    }
    free(code);
    free(xs);
    free(ms);
    free(boff);
    free(blen);
}

/* ---------------------------------------------------------------- EM loop ------------- */

/* Lloyd iteration of Sec. 3.2: `iters` times { thresholds from the current levels, assign,
 * recompute every level that is not fixed (bit l of fixed_mask) }.  err_log[t] is the mean
 * error (MSE or MAE over all n weights, un-normalised domain) of the levels that ENTER
 * iteration t.  metric: 0 = MSE (Eq. 6), 1 = MAE (Eq. 8); 2 / 3 = the same criteria on the
 * normalised weights (App. D: plain mean / plain median, error measured on x). */
void orc_fit_seg(const float *w, const int64_t *seg, int n_seg, int I, int norm, int metric,
                 float *xhat, uint32_t fixed_mask, int iters, double *err_log);

void orc_fit(const float *w, int64_t n, int I, int norm, int metric, float *xhat,
             uint32_t fixed_mask, int iters, double *err_log)
{
    orc_fit_seg(w, &n, 1, I, norm, metric, xhat, fixed_mask, iters, err_log);
}

/* The same over a list of tensors (every tensor cut into blocks from its own start; a tensor
 * whose length is not a multiple of I ends in a shorter block with its own constant). */
void orc_fit_seg(const float *w, const int64_t *seg, int n_seg, int I, int norm, int metric,
                 float *xhat, uint32_t fixed_mask, int iters, double *err_log)
{
    int64_t n = 0;
    for (int s = 0; s < n_seg; ++s)
        n += seg[s];
    for (int t = 0; t < iters; ++t) {
        uint64_t cnt[L];
        double err;
        if (metric == 0 || metric == 2) {
            double s1[L], s0[L];
            em_accumulate_mse_impl(w, seg, n_seg, I, norm, xhat, metric == 2, s1, s0, cnt, &err);
            for (int l = 0; l < L; ++l)
                if (!((fixed_mask >> l) & 1u) && s0[l] > 0.0)
                    xhat[l] = (float)(s1[l] / s0[l]);
        } else {
            float med[L];
            double ws[L];
            em_accumulate_mae_impl(w, seg, n_seg, I, norm, xhat, metric == 3, med, ws, cnt, &err);
            for (int l = 0; l < L; ++l)
                if (!((fixed_mask >> l) & 1u) && ws[l] > 0.0)
                    xhat[l] = med[l];
        }
        if (err_log)
            err_log[t] = (n > 0) ? err / (double)n : 0.0;
    }
}

/* Mean error of a codebook on a weight set: (MSE, MAE) of Q(W) against W, App. B.3. */
void orc_quant_error(const float *w, int64_t n, int I, int norm, const float *xhat,
                     double *mse, double *mae)
{
    float xi[L - 1];
    orc_thresholds(xhat, xi);
    int64_t B = n / I;
    double s2 = 0.0, s1 = 0.0;
#pragma omp parallel for schedule(static) reduction(+ : s2, s1)
    for (int64_t b = 0; b < B; ++b) {
        const float *wb = w + b * I;
        float m = block_constant(wb, I, norm);
        for (int i = 0; i < I; ++i) {
            int c = region_of(normalise(wb[i], m), xi);
            double d = (double)wb[i] - (double)m * (double)xhat[c];
            s2 += d * d;
            s1 += fabs(d);
        }
    }
    *mse = n ? s2 / (double)n : 0.0;
    *mae = n ? s1 / (double)n : 0.0;
}

/* ---------------------------------------------------------------- OPQ ----------------- */

/* Balanced binary summation tree over v[0..len), len a power of two: neighbours first, then
 * pairs of pairs.  Overwrites v. */
static float tree_sum(float *v, int len)
{
    for (int step = 1; step < len; step *= 2)
        for (int i = 0; i < len; i += 2 * step)
            v[i] = v[i] + v[i + step];
    return v[0];
}

/* Corrected sample standard deviation of one block of len weights (App. E, the sigma_b
 * equation): two-pass, fp32, tree-ordered sums.  A ragged block (len not a power of two) is
 * padded with zeros for the two tree sums only; mean and variance divide by its own length.
 * A block of one weight gives 0/0 = NaN, and no weight compares greater than NaN. */
static float block_sigma(const float *w, int len)
{
    float tmp[4096]; /* largest supported block */
    int P = 1;
    while (P < len)
        P *= 2;
    for (int i = 0; i < P; ++i)
        tmp[i] = (i < len) ? w[i] : 0.0f;
    float mean = tree_sum(tmp, P) / (float)len;
    for (int i = 0; i < P; ++i) {
        float d = (i < len) ? w[i] - mean : 0.0f;
        tmp[i] = d * d;
    }
    float ss = tree_sum(tmp, P);
    return sqrtf(ss / (float)(len - 1));
}

void orc_block_sigmas(const float *w, int64_t n, int I, float *sigma)
{
    int64_t B = (n + I - 1) / I;
    for (int64_t b = 0; b < B; ++b)
        sigma[b] = block_sigma(w + b * I, block_len(n, I, b));
}

/* Outlier split of Sec. 3.3 / Eq. 9: |w| > sigma_b * tau with tau = F_M^{-1}(q).  Outliers are
 * listed in ascending flattened index with their value rounded to bfloat16, and replaced by
 * zero in w_clean.  Returns the number of outliers; at most `cap` are written. */
int64_t orc_opq_split(const float *w, int64_t n, int I, float tau, float *w_clean,
                      int64_t *idx, uint16_t *val, int64_t cap)
{
    int64_t B = (n + I - 1) / I, count = 0;
    for (int64_t b = 0; b < B; ++b) {
        const float *wb = w + b * I;
        int len = block_len(n, I, b);
        float thr = block_sigma(wb, len) * tau;
        for (int i = 0; i < len; ++i) {
            int64_t k = b * I + i;
            if (fabsf(wb[i]) > thr) {
                if (count < cap) {
                    idx[count] = k;
                    val[count] = f32_to_bf16_rne(wb[i]);
                }
                ++count;
                if (w_clean)
                    w_clean[k] = 0.0f;
            } else if (w_clean) {
                w_clean[k] = wb[i];
            }
        }
    }
    return count;
}

/* Write the stored outliers back over a dequantised tensor (Sec. 3.3, decoding side). */
void orc_opq_restore(float *out, const int64_t *idx, const uint16_t *val, int64_t n_out)
{
    for (int64_t k = 0; k < n_out; ++k)
        out[idx[k]] = bf16_bits_to_f32(val[k]);
}
