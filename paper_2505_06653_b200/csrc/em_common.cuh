// Pieces shared by the MSE and MAE passes of the codebook fit: the per-launch tensor table,
// the host-side argument record and its validation.
#pragma once

#include "common.cuh"
#include "layout.h"

namespace bof4 {

constexpr int kEmMaxTensors = 64;  // tensors per launch (kernel parameter table)

struct EmTensors {
    const void* ptr[kEmMaxTensors];
    int64_t n[kEmMaxTensors];
    int64_t row_end[kEmMaxTensors];  // cumulative number of CTA rows up to and including tensor t
    int count;
    int accumulate;  // 0: this launch overwrites the partial records, 1: adds to them
    int last;        // 1: no further launch of this pass follows
    int unit;        // 1: normalised-domain variant (App. D): all sample weights are 1, errors on x
};

struct EmArgs {
    const void* const* h_w;
    const int64_t* h_n;
    int n_tensors, w_dtype, block_size, norm, metric;
    int64_t n_total;
};

// Validates the common arguments of bof4_em_step / bof4_fit_codebook; fills a.n_total.
int check_em(const char* fn, EmArgs& a, const void* d_codebook, void* d_ws, size_t ws_bytes);

// Calls fire(T) for the non-empty tensors of the list, kEmMaxTensors per call, with row_end
// computed for CTA rows of `row` weights; T.accumulate is 0 for the first call only.
// Returns the number of calls through *n_calls.
template <class Fire>
int for_each_tensor_chunk(const EmArgs& a, int row, Fire fire, int* n_calls)
{
    EmTensors T;
    T.count = 0;
    T.accumulate = 0;
    T.unit = (a.metric >= 2) ? 1 : 0;
    int64_t rows = 0;
    int calls = 0, nonempty = 0;
    for (int t = 0; t < a.n_tensors; ++t) nonempty += a.h_n[t] > 0;
    const int total_calls = (nonempty + kEmMaxTensors - 1) / kEmMaxTensors;
    for (int t = 0; t <= a.n_tensors; ++t) {
        if (t < a.n_tensors) {
            if (a.h_n[t] == 0) continue;
            rows += (a.h_n[t] + row - 1) / row;
            T.ptr[T.count] = a.h_w[t];
            T.n[T.count] = a.h_n[t];
            T.row_end[T.count] = rows;
            ++T.count;
        }
        if (T.count == kEmMaxTensors || (t == a.n_tensors && T.count > 0)) {
            T.last = (calls + 1 == total_calls) ? 1 : 0;
            const int rc = fire(T);
            if (rc) return rc;
            ++calls;
            T.count = 0;
            T.accumulate = 1;
            rows = 0;
        }
    }
    *n_calls = calls;
    return BOF4_OK;
}

// MAE (Eq. 8) side, implemented in em_mae.cu.  mae_prepare runs once per call (largest
// |w| of the data, needed for the fixed-point weights); mae_iteration enqueues one
// iteration: selection passes, then the level update / statistics.
int mae_prepare(const EmArgs& a, void* d_ws, size_t ws_bytes, cudaStream_t st);
int mae_iteration(const EmArgs& a, const float* d_levels_in, float* d_levels_out, uint32_t skip_mask,
                  bof4_em_stats* d_stats, double* d_err_slot, void* d_ws, size_t ws_bytes, cudaStream_t st);

}  // namespace bof4
