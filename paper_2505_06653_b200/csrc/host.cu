// Host-only parts of the C ABI: error strings, the OPQ threshold, the default starting codebook.
#include <math.h>
#include <stdarg.h>
#include <stdio.h>

#include "common.cuh"
#include "layout.h"

namespace bof4 {

static thread_local char g_err[512] = "";

void set_error(const char* fmt, ...)
{
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof(g_err), fmt, ap);
    va_end(ap);
}

int cuda_fail(cudaError_t e, const char* what)
{
    set_error("CUDA error %d (%s) in %s", (int)e, cudaGetErrorString(e), what);
    return BOF4_ERR_CUDA;
}

}  // namespace bof4

extern "C" {

const char* bof4_last_error(void) { return bof4::g_err; }

size_t bof4_workspace_bytes(int op, int64_t n_max, int block_size, int metric)
{
    if (n_max < 0 || !bof4::valid_block_size(block_size)) return 0;
    if (op == BOF4_OP_EM) {
        if (metric < BOF4_METRIC_MSE || metric > BOF4_METRIC_MAE_NORMALIZED) return 0;
        return bof4::em_workspace_bytes_for(n_max);
    }
    if (op == BOF4_OP_OPQ) return bof4::opq_layout(n_max).total;
    return 0;
}

// The synchronising half of the two-call pattern: the outlier-producing calls only leave the true
// count on the device; this reads it back and turns an overflow into an error code.
int bof4_outlier_count(const int64_t* d_n_out, int64_t capacity, int64_t* h_n_out, void* stream)
{
    if (!d_n_out || capacity < 0) {
        bof4::set_error("bof4_outlier_count: NULL count pointer or negative capacity");
        return BOF4_ERR_INVALID_ARG;
    }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int64_t count = 0;
    BOF4_CUDA_TRY(cudaMemcpyAsync(&count, d_n_out, sizeof(count), cudaMemcpyDeviceToHost, st));
    BOF4_CUDA_TRY(cudaStreamSynchronize(st));
    if (h_n_out) *h_n_out = count;
    if (count > capacity) {
        bof4::set_error("outlier list overflow: %lld outliers found, capacity %lld (only the first %lld were "
                        "stored; call again with capacity >= %lld)",
                        (long long)count, (long long)capacity, (long long)capacity, (long long)count);
        return BOF4_ERR_CAPACITY;
    }
    return BOF4_OK;
}

// tau with G(tau) = (1 + q^(1/I)) / 2  <=>  erfc(tau / sqrt 2) = 1 - q^(1/I) = -expm1(ln q / I).
// erfc is strictly decreasing, so bisection on [0, 40] converges to the last bit.
double bof4_opq_threshold(double q, int block_size)
{
    if (!(q > 0.0 && q < 1.0) || block_size < 1) return NAN;
    const double target = -expm1(log(q) / (double)block_size);
    double lo = 0.0, hi = 40.0;
    for (int it = 0; it < 200; ++it) {
        const double mid = 0.5 * (lo + hi);
        if (erfc(mid * M_SQRT1_2) > target)
            lo = mid;
        else
            hi = mid;
    }
    return 0.5 * (lo + hi);
}

int bof4_default_init(int norm, float h_levels[BOF4_LEVELS], uint32_t* h_fixed_mask)
{
    if (!h_levels || (norm != BOF4_NORM_ABS && norm != BOF4_NORM_SIGNED)) {
        bof4::set_error("bof4_default_init: bad argument");
        return BOF4_ERR_INVALID_ARG;
    }
    for (int k = 0; k < 7; ++k) h_levels[k] = (float)(-1.0 + (double)k / 7.0);
    h_levels[7] = 0.0f;
    for (int k = 1; k <= 8; ++k) h_levels[7 + k] = (float)((double)k / 8.0);
    if (h_fixed_mask)
        *h_fixed_mask = (norm == BOF4_NORM_ABS) ? ((1u << 0) | (1u << 7) | (1u << 15))
                                                : ((1u << 7) | (1u << 15));
    return BOF4_OK;
}

}  // extern "C"
