// Data-free codebook design (Sec. 3.2 Eq. 5 and Eq. 7), for Gaussian weights in closed form and,
// further down, for any tabulated symmetric density.  Gaussian weights (Sec. 3.2 Eq. 5 and Eq. 7; App. B.2, "Simplified
// Solution for Gaussian Network Weights" and "MAE Optimization"): Lloyd iterations whose
// centroids are ratios (MSE) or roots (MAE) of one-dimensional integrals over the absolute
// block maximum m, evaluated by Simpson quadrature in fp64.
//
// With g, G the pdf / cdf of N(0,1), the block maximum has density proportional to
// (2G(m)-1)^(I-1) g(m) and, given m, the other normalised weights have cdf
// (G(m x) - G(-m)) / (2G(m)-1) on (-1, 1).  For a region (lo, hi) inside [-1, 1]:
//   MSE centroid = - INT m [g(m hi) - g(m lo)] c(m) dm / INT m^2 [G(m hi) - G(m lo)] c(m) dm,
//   MAE centroid = the x with INT m [G(m x) - G(m lo)] c(m) dm = 1/2 INT m [G(m hi) - G(m lo)] c(m) dm,
// c(m) = (2G(m)-1)^(I-2) g(m).  (The printed boxed MSE formula has lost the leading minus sign of
// the two equations it is derived from; it is restored here.)  The outermost regions carry the
// point mass of the block maximum itself, so their levels must be fixed (-1 and 1 for absolute,
// 1 for signed normalisation).
#include <math.h>

#include "common.cuh"

namespace bof4 {

constexpr int kThThreads = 512;
constexpr int kThIntervals = 8192;  // Simpson intervals on m in [0, kThMax]
constexpr double kThMax = 12.0;     // g(12) ~ 1e-32: the tail is far below fp64 resolution

__device__ __forceinline__ double gauss_pdf(double x) { return 0.3989422804014326779 * exp(-0.5 * x * x); }
// G(b) - G(a)
__device__ __forceinline__ double gauss_mass(double a, double b)
{
    return 0.5 * (erf(b * 0.70710678118654752440) - erf(a * 0.70710678118654752440));
}

// Sum over the CTA, result in every thread.
__device__ __forceinline__ double cta_sum(double v, double* s_red)
{
#pragma unroll
    for (int off = 16; off; off >>= 1) v += __shfl_xor_sync(kFull, v, off);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) s_red[threadIdx.x >> 5] = v;
    __syncthreads();
    double t = 0.0;
    for (int k = 0; k < kThThreads / 32; ++k) t += s_red[k];
    return t;
}

// Simpson weight of node q (0 .. kThIntervals) times the step, and its abscissa.
__device__ __forceinline__ void node(int q, double& m, double& wq)
{
    const double h = kThMax / kThIntervals;
    m = q * h;
    wq = (q == 0 || q == kThIntervals) ? h / 3.0 : ((q & 1) ? 4.0 * h / 3.0 : 2.0 * h / 3.0);
}

// Problems of one batched call: block size, metric and fixed levels of each (kernel parameter).
constexpr int kThMaxBatch = 128;
struct TheoryBatch {
    int I[kThMaxBatch];
    int metric[kThMaxBatch];
    uint32_t fixed_mask[kThMaxBatch];
};

// One Lloyd iteration of every problem: CTA (l, p) recomputes level l of problem p from the
// thresholds of its current levels.  Problem p keeps two sets of 16 fp64 levels in the workspace
// (32 doubles); `flip` tells which of the two is current.
__global__ void __launch_bounds__(kThThreads)
theory_step_kernel(double* __restrict__ state, int flip, const TheoryBatch B)
{
    __shared__ double s_red[kThThreads / 32];
    const int l = blockIdx.x, p = blockIdx.y;
    const double* levels_in = state + (size_t)p * 2 * kLevels + (flip ? kLevels : 0);
    double* levels_out = state + (size_t)p * 2 * kLevels + (flip ? 0 : kLevels);
    const int I = B.I[p], metric = B.metric[p];
    const uint32_t fixed_mask = B.fixed_mask[p];
    const double cur = levels_in[l];
    if ((fixed_mask >> l) & 1u) {
        if (threadIdx.x == 0) levels_out[l] = cur;
        return;
    }
    double lo = (l > 0) ? 0.5 * (levels_in[l - 1] + cur) : -1.0;
    double hi = (l < kLevels - 1) ? 0.5 * (cur + levels_in[l + 1]) : 1.0;
    lo = fmin(fmax(lo, -1.0), 1.0);
    hi = fmin(fmax(hi, -1.0), 1.0);
    const double expo = (double)(I - 2);
    if (metric == BOF4_METRIC_MSE) {
        double num = 0.0, den = 0.0;
        for (int q = threadIdx.x; q <= kThIntervals; q += kThThreads) {
            double m, wq;
            node(q, m, wq);
            const double c = pow(erf(m * 0.70710678118654752440), expo) * gauss_pdf(m) * wq;
            num -= m * (gauss_pdf(m * hi) - gauss_pdf(m * lo)) * c;
            den += m * m * gauss_mass(m * lo, m * hi) * c;
        }
        num = cta_sum(num, s_red);
        den = cta_sum(den, s_red);
        if (threadIdx.x == 0) levels_out[l] = (den > 0.0) ? num / den : cur;
    } else {
        // weights m c(m) of the nodes this thread owns stay in registers during the bisection
        constexpr int PER = kThIntervals / kThThreads + 1;
        double mm[PER], wc[PER];
        double full = 0.0;
#pragma unroll
        for (int k = 0; k < PER; ++k) {
            const int q = threadIdx.x + k * kThThreads;
            double m = 0.0, wq = 0.0;
            if (q <= kThIntervals) node(q, m, wq);
            mm[k] = m;
            wc[k] = (q <= kThIntervals) ? m * pow(erf(m * 0.70710678118654752440), expo) * gauss_pdf(m) * wq : 0.0;
            full += wc[k] * gauss_mass(m * lo, m * hi);
        }
        const double half = 0.5 * cta_sum(full, s_red);
        double a = lo, b = hi;
        for (int it = 0; it < 60; ++it) {  // the mass below x grows with x: bisection
            const double x = 0.5 * (a + b);
            double part = 0.0;
#pragma unroll
            for (int k = 0; k < PER; ++k) part += wc[k] * gauss_mass(mm[k] * lo, mm[k] * x);
            if (cta_sum(part, s_red) < half)
                a = x;
            else
                b = x;
        }
        if (threadIdx.x == 0) levels_out[l] = (half > 0.0) ? 0.5 * (a + b) : cur;
    }
}

// ---------------------------------------------------------------- any symmetric weight density
//
// Eq. 5 and Eq. 7 before the Gaussian simplification (App. B.1: cdf of X given M = m, density of
// M; App. B.2: centroid as a ratio of integrals over m, conditional expectation of X for fixed m).
// The density p_W is given as samples on the uniform grid w_j = j h, j = 0 .. n-1 (w >= 0; p_W is
// symmetric).  With Fc(w) = INT_0^w p_W (so F_W = 1/2 + Fc, odd) and H(w) = INT_0^w u p_W(u) du
// (even), M has density 2I (2 Fc(m))^(I-1) p_W(m), INT_R m x p_W(m x) dx = [H(m x)]_R / m, and
//   MSE centroid = INT m [H(m x)]_lo^hi c(m) dm / INT m^2 [Fc(m x)]_lo^hi c(m) dm,
//   MAE centroid = the x with INT m [Fc(m x)]_lo^x c(m) dm = 1/2 INT m [Fc(m x)]_lo^hi c(m) dm,
// c(m) = (2 Fc(m))^(I-2) p_W(m).  Fc and H are cumulative trapezoid sums on the grid (after
// scaling the samples to total mass 1), read between nodes by linear interpolation; the
// integrals over m are trapezoid sums on the same grid.

struct DensityTable {
    const double* fc;    // [n] Fc(w_j)
    const double* hh;    // [n] H(w_j)
    const double* core;  // [n] c(w_j) times the trapezoid weight of node j
    int n;
    double h, inv_h;
};

// Tables from the samples: one CTA.  ws: [n] fc, [n] hh, [n] core.
__global__ void __launch_bounds__(kThThreads)
theory_table_kernel(const double* __restrict__ pdf, int n, double h, int I, double* __restrict__ fc,
                    double* __restrict__ hh, double* __restrict__ core)
{
    __shared__ double s_red[kThThreads / 32];
    double part = 0.0;
    for (int j = threadIdx.x; j < n; j += kThThreads) part += ((j == 0 || j == n - 1) ? 0.5 : 1.0) * pdf[j];
    const double half_mass = cta_sum(part, s_red) * h;  // INT_0^wmax p
    const double scale = (half_mass > 0.0) ? 0.5 / half_mass : 0.0;
    if (threadIdx.x == 0) {  // cumulative sums in grid order
        double a = 0.0;
        fc[0] = 0.0;
        for (int j = 1; j < n; ++j) {
            a += 0.5 * (pdf[j] + pdf[j - 1]) * scale * h;
            fc[j] = a;
        }
    }
    if (threadIdx.x == 32) {
        double a = 0.0;
        hh[0] = 0.0;
        for (int j = 1; j < n; ++j) {
            a += 0.5 * (j * h * pdf[j] + (j - 1) * h * pdf[j - 1]) * scale * h;
            hh[j] = a;
        }
    }
    __syncthreads();
    for (int j = threadIdx.x; j < n; j += kThThreads)
        core[j] = pow(2.0 * fc[j], (double)(I - 2)) * pdf[j] * scale * ((j == 0 || j == n - 1) ? 0.5 * h : h);
}

__device__ __forceinline__ double table_at(const double* __restrict__ t, const DensityTable& D, double w_abs)
{
    const double a = w_abs * D.inv_h;
    int j = (int)a;
    j = min(max(j, 0), D.n - 2);
    const double lo = t[j];
    return lo + (a - (double)j) * (t[j + 1] - lo);
}
__device__ __forceinline__ double fc_at(const DensityTable& D, double w)  // odd
{
    const double v = table_at(D.fc, D, fabs(w));
    return w < 0.0 ? -v : v;
}

__global__ void __launch_bounds__(kThThreads)
theory_general_step_kernel(double* __restrict__ state, int flip, int metric, uint32_t fixed_mask, const DensityTable D)
{
    __shared__ double s_red[kThThreads / 32];
    const int l = blockIdx.x;
    const double* levels_in = state + (flip ? kLevels : 0);
    double* levels_out = state + (flip ? 0 : kLevels);
    const double cur = levels_in[l];
    if ((fixed_mask >> l) & 1u) {
        if (threadIdx.x == 0) levels_out[l] = cur;
        return;
    }
    double lo = (l > 0) ? 0.5 * (levels_in[l - 1] + cur) : -1.0;
    double hi = (l < kLevels - 1) ? 0.5 * (cur + levels_in[l + 1]) : 1.0;
    lo = fmin(fmax(lo, -1.0), 1.0);
    hi = fmin(fmax(hi, -1.0), 1.0);
    if (metric == BOF4_METRIC_MSE) {
        double num = 0.0, den = 0.0;
        for (int q = threadIdx.x; q < D.n; q += kThThreads) {
            const double m = q * D.h, c = D.core[q];
            num += m * (table_at(D.hh, D, fabs(m * hi)) - table_at(D.hh, D, fabs(m * lo))) * c;
            den += m * m * (fc_at(D, m * hi) - fc_at(D, m * lo)) * c;
        }
        num = cta_sum(num, s_red);
        den = cta_sum(den, s_red);
        if (threadIdx.x == 0) levels_out[l] = (den > 0.0) ? num / den : cur;
    } else {
        auto mass = [&](double x) {
            double part = 0.0;
            for (int q = threadIdx.x; q < D.n; q += kThThreads) {
                const double m = q * D.h;
                part += m * (fc_at(D, m * x) - fc_at(D, m * lo)) * D.core[q];
            }
            return cta_sum(part, s_red);
        };
        const double half = 0.5 * mass(hi);
        double a = lo, b = hi;
        for (int it = 0; it < 60; ++it) {
            const double x = 0.5 * (a + b);
            if (mass(x) < half)
                a = x;
            else
                b = x;
        }
        if (threadIdx.x == 0) levels_out[l] = (half > 0.0) ? 0.5 * (a + b) : cur;
    }
}

// levels of problem p: codebooks[p][16] (fp32) <-> the current set of the fp64 state
__global__ void theory_load_kernel(const float* __restrict__ codebooks, double* __restrict__ state)
{
    const int p = blockIdx.x;
    if (threadIdx.x < kLevels) state[(size_t)p * 2 * kLevels + threadIdx.x] = (double)codebooks[p * kLevels + threadIdx.x];
}
__global__ void theory_store_kernel(const double* __restrict__ state, int flip, float* __restrict__ codebooks)
{
    const int p = blockIdx.x;
    if (threadIdx.x < kLevels)
        codebooks[p * kLevels + threadIdx.x] = (float)state[(size_t)p * 2 * kLevels + (flip ? kLevels : 0) + threadIdx.x];
}

static int check_theory_problem(const char* fn, int block_size, int norm, int metric, uint32_t fixed_mask)
{
    if (block_size < 2 || block_size > (1 << 20)) {
        set_error("%s: block_size must be in 2 ... 2^20", fn);
        return BOF4_ERR_SHAPE;
    }
    if ((norm != BOF4_NORM_ABS && norm != BOF4_NORM_SIGNED) ||
        (metric != BOF4_METRIC_MSE && metric != BOF4_METRIC_MAE)) {
        set_error("%s: bad norm or metric", fn);
        return BOF4_ERR_INVALID_ARG;
    }
    if (!((fixed_mask >> 15) & 1u) || (norm == BOF4_NORM_ABS && !(fixed_mask & 1u))) {
        set_error("%s: the outermost levels (1, and -1 for absolute normalisation) "
                  "carry the point mass of the block maximum and must be fixed", fn);
        return BOF4_ERR_INVALID_ARG;
    }
    return BOF4_OK;
}

static int run_theory(const char* fn, int n, const TheoryBatch& B, float* d_codebooks, int iters, void* d_ws,
                      size_t ws_bytes, void* stream)
{
    if (iters < 0 || !d_codebooks) {
        set_error("%s: negative iteration count or NULL codebook", fn);
        return BOF4_ERR_INVALID_ARG;
    }
    if (!d_ws || ((uintptr_t)d_ws & 255u) || ws_bytes < (size_t)256 * n) {
        set_error("%s: workspace NULL, not 256-byte aligned, or smaller than 256 bytes per problem", fn);
        return BOF4_ERR_WORKSPACE;
    }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    double* state = static_cast<double*>(d_ws);
    theory_load_kernel<<<n, 32, 0, st>>>(d_codebooks, state);
    BOF4_CUDA_TRY(cudaGetLastError());
    int flip = 0;
    for (int t = 0; t < iters; ++t) {
        theory_step_kernel<<<dim3(kLevels, n), kThThreads, 0, st>>>(state, flip, B);
        BOF4_CUDA_TRY(cudaGetLastError());
        flip ^= 1;
    }
    theory_store_kernel<<<n, 32, 0, st>>>(state, flip, d_codebooks);
    BOF4_CUDA_TRY(cudaGetLastError());
    return BOF4_OK;
}

}  // namespace bof4

extern "C" int bof4_theoretical_codebook(int block_size, int norm, int metric, float* d_codebook,
                                         uint32_t fixed_mask, int iters, void* d_ws, size_t ws_bytes,
                                         void* stream)
{
    using namespace bof4;
    const int rc = check_theory_problem("bof4_theoretical_codebook", block_size, norm, metric, fixed_mask);
    if (rc) return rc;
    TheoryBatch B{};
    B.I[0] = block_size;
    B.metric[0] = metric;
    B.fixed_mask[0] = fixed_mask;
    return run_theory("bof4_theoretical_codebook", 1, B, d_codebook, iters, d_ws, ws_bytes, stream);
}

extern "C" int bof4_theoretical_codebook_batch(int n_problems, const int* h_block_size, const int* h_norm,
                                               const int* h_metric, const uint32_t* h_fixed_mask,
                                               float* d_codebooks, int iters, void* d_ws, size_t ws_bytes,
                                               void* stream)
{
    using namespace bof4;
    if (n_problems < 0 || n_problems > kThMaxBatch) {
        set_error("bof4_theoretical_codebook_batch: n_problems must be in 0 ... %d", kThMaxBatch);
        return BOF4_ERR_SHAPE;
    }
    if (n_problems == 0) return BOF4_OK;
    if (!h_block_size || !h_norm || !h_metric || !h_fixed_mask) {
        set_error("bof4_theoretical_codebook_batch: NULL parameter array");
        return BOF4_ERR_INVALID_ARG;
    }
    TheoryBatch B{};
    for (int p = 0; p < n_problems; ++p) {
        const int rc = check_theory_problem("bof4_theoretical_codebook_batch", h_block_size[p], h_norm[p],
                                            h_metric[p], h_fixed_mask[p]);
        if (rc) return rc;
        B.I[p] = h_block_size[p];
        B.metric[p] = h_metric[p];
        B.fixed_mask[p] = h_fixed_mask[p];
    }
    return run_theory("bof4_theoretical_codebook_batch", n_problems, B, d_codebooks, iters, d_ws, ws_bytes, stream);
}

extern "C" int bof4_theoretical_codebook_general(int block_size, int norm, int metric, const double* d_pdf,
                                                 int n_grid, double w_max, float* d_codebook,
                                                 uint32_t fixed_mask, int iters, void* d_ws, size_t ws_bytes,
                                                 void* stream)
{
    using namespace bof4;
    const char* fn = "bof4_theoretical_codebook_general";
    const int rc = check_theory_problem(fn, block_size, norm, metric, fixed_mask);
    if (rc) return rc;
    if (!d_pdf || n_grid < 3 || n_grid > (1 << 20) || !(w_max > 0.0) || iters < 0 || !d_codebook) {
        set_error("%s: NULL pointer, n_grid outside 3 ... 2^20, w_max <= 0 or negative iteration count", fn);
        return BOF4_ERR_INVALID_ARG;
    }
    const size_t need = 256 + (size_t)3 * n_grid * sizeof(double);
    if (!d_ws || ((uintptr_t)d_ws & 255u) || ws_bytes < need) {
        set_error("%s: workspace NULL, not 256-byte aligned, or smaller than 256 + 24 * n_grid bytes", fn);
        return BOF4_ERR_WORKSPACE;
    }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    double* state = static_cast<double*>(d_ws);
    double* fc = state + 32;
    double* hh = fc + n_grid;
    double* core = hh + n_grid;
    const double h = w_max / (double)(n_grid - 1);
    theory_table_kernel<<<1, kThThreads, 0, st>>>(d_pdf, n_grid, h, block_size, fc, hh, core);
    BOF4_CUDA_TRY(cudaGetLastError());
    theory_load_kernel<<<1, 32, 0, st>>>(d_codebook, state);
    BOF4_CUDA_TRY(cudaGetLastError());
    const DensityTable D{fc, hh, core, n_grid, h, 1.0 / h};
    int flip = 0;
    for (int t = 0; t < iters; ++t) {
        theory_general_step_kernel<<<kLevels, kThThreads, 0, st>>>(state, flip, metric, fixed_mask, D);
        BOF4_CUDA_TRY(cudaGetLastError());
        flip ^= 1;
    }
    theory_store_kernel<<<1, 32, 0, st>>>(state, flip, d_codebook);
    BOF4_CUDA_TRY(cudaGetLastError());
    return BOF4_OK;
}
