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

// Short last blocks (tensors whose length is not a multiple of the block size): each is a block
// of its own with its own constant (Eq. 1 / Eq. 4).  They are few and small, so one small CTA
// per launch adds their contribution to the same records, histograms and lists as the whole
// blocks; it is enqueued before the streaming kernel of the same pass.
constexpr int kEmTailThreads = 512;
struct EmTails {
    const void* ptr[kEmMaxTensors];  // first weight of the short block
    int len[kEmMaxTensors];          // its length, 1 ... block_size - 1
    int count;
    int accumulate;  // 0: this launch overwrites the record, 1: adds to it
    int unit;
};

template <class DT>
__device__ __forceinline__ float short_block_elem(const void* p, int i);
template <>
__device__ __forceinline__ float short_block_elem<F32>(const void* p, int i)
{
    return static_cast<const float*>(p)[i];
}
template <>
__device__ __forceinline__ float short_block_elem<BF16>(const void* p, int i)
{
    return __uint_as_float((uint32_t)static_cast<const uint16_t*>(p)[i] << 16);
}

// Copies a short block into s_w and returns its constant: the element of largest magnitude
// (lowest index on ties), with its sign if SIGNED; 0 for an all-zero block.  Called by all
// kEmTailThreads threads; s_red holds one word per warp.
template <class DT, bool SIGNED>
__device__ __forceinline__ float load_short_block(const void* p, int len, float* s_w, unsigned long long* s_red)
{
    const int tid = threadIdx.x;
    unsigned long long best = 0ull;
    for (int i = tid; i < len; i += kEmTailThreads) {
        const float v = short_block_elem<DT>(p, i);
        s_w[i] = v;
        const float a = fabsf(v);
        if (a > 0.0f)  // false for a NaN, which never is the maximum
            best = max(best, ((unsigned long long)__float_as_uint(a) << 32) | (0xffffffffu - (uint32_t)i));
    }
#pragma unroll
    for (int off = 16; off; off >>= 1) best = max(best, __shfl_xor_sync(kFull, best, off));
    __syncthreads();  // s_red may still be read from the previous block
    if ((tid & 31) == 0) s_red[tid >> 5] = best;
    __syncthreads();
    for (int k = 0; k < kEmTailThreads / 32; ++k) best = max(best, s_red[k]);
    if (best == 0ull) return 0.0f;
    const float v = s_w[0xffffffffu - (uint32_t)best];
    return SIGNED ? v : fabsf(v);
}

// Validates the common arguments of bof4_em_step / bof4_fit_codebook; fills a.n_total.
int check_em(const char* fn, EmArgs& a, const void* d_codebook, void* d_ws, size_t ws_bytes);

// Calls fire(Q) for the short last blocks of the list, kEmMaxTensors per call; Q.accumulate is 0
// for the first call only.
template <class Fire>
int for_each_tail_chunk(const EmArgs& a, Fire fire)
{
    EmTails Q;
    Q.count = 0;
    Q.accumulate = 0;
    Q.unit = (a.metric >= 2) ? 1 : 0;
    const size_t esize = a.w_dtype == BOF4_F32 ? 4 : 2;
    for (int t = 0; t <= a.n_tensors; ++t) {
        if (t < a.n_tensors) {
            const int r = (int)(a.h_n[t] % a.block_size);
            if (r == 0) continue;
            Q.ptr[Q.count] = static_cast<const char*>(a.h_w[t]) + (size_t)(a.h_n[t] - r) * esize;
            Q.len[Q.count] = r;
            ++Q.count;
        }
        if (Q.count == kEmMaxTensors || (t == a.n_tensors && Q.count > 0)) {
            const int rc = fire(Q);
            if (rc) return rc;
            Q.count = 0;
            Q.accumulate = 1;
        }
    }
    return BOF4_OK;
}
inline bool has_tails(const EmArgs& a)
{
    for (int t = 0; t < a.n_tensors; ++t)
        if (a.h_n[t] % a.block_size) return true;
    return false;
}
inline bool has_whole_blocks(const EmArgs& a)
{
    for (int t = 0; t < a.n_tensors; ++t)
        if (a.h_n[t] >= a.block_size) return true;
    return false;
}

// Calls fire(T) for the whole blocks of the non-empty tensors of the list, kEmMaxTensors per call, with row_end
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
    for (int t = 0; t < a.n_tensors; ++t) nonempty += a.h_n[t] >= a.block_size;
    const int total_calls = (nonempty + kEmMaxTensors - 1) / kEmMaxTensors;
    for (int t = 0; t <= a.n_tensors; ++t) {
        if (t < a.n_tensors) {
            const int64_t n_whole = a.h_n[t] - a.h_n[t] % a.block_size;  // the short last block goes to the tail kernel
            if (n_whole == 0) continue;
            rows += (n_whole + row - 1) / row;
            T.ptr[T.count] = a.h_w[t];
            T.n[T.count] = n_whole;
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
