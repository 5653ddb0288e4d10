// MAE variant of the codebook fit (Eq. 8, App. B.3): every free level becomes the weighted
// median of the normalised weights of its region, the weight of a sample being |m| of its block.
//
// The weighted median is found by radix selection on an order-preserving integer key of x.
// All members of region l have keys in [key(xi[l-1]), key(xi[l])), so only the B_l low bits of
// rel = key - key(xi[l-1]) differ; each data pass histograms the next (up to) 9 of those bits for
// the samples that match the digits chosen so far, and a single-CTA kernel picks the bin in
// which the cumulative weight first reaches half of the region's total.  After ceil(B_l / 9)
// digits the key, hence the sample, is known exactly.  The second data pass also copies the
// samples that match the first digit (about 1/512 of the region) into a candidate list; when
// that list fits (64 Ki samples per level) the remaining digits are resolved from the list by
// one CTA and no further data pass is needed.  Otherwise (very large or degenerate inputs) the
// third and fourth data passes finish the selection; they return at once when nothing is left.
// In every pass after the first only the samples that carry the digits chosen so far matter:
// the pass finds them with one table read and two comparisons per weight (the table bins hold
// the range of normalised weights that can still take part) and queues them in shared memory;
// the queue is worked off by all threads once the data has been read.
//
// Weights enter the histograms as 31-bit fixed-point integers relative to the largest |w| of
// the data (exact whenever |m| is within 2^-7 of it for fp32 input, 2^-23 for bf16 input), so
// every sum is an integer sum: independent of the order of the atomics, bit-reproducible, and
// equal to the exact real-number sums that define the median.
#include <cooperative_groups.h>

#include "common.cuh"
#include "em_common.cuh"
#include "lane32.cuh"
#include "layout.h"

namespace bof4 {

constexpr int kMaeThreads = 1024;
constexpr int kMaeRow = kMaeThreads * kLaneW;
constexpr int kMaeStage = 256;  // candidates staged per CTA and level in the collecting pass
constexpr size_t kMaeSmem = (size_t)kLutBytes + 3u * kLevels * kMaeBins * 4u  // table; lo, hi, count
                            + (size_t)kLevels * kMaeStage * 8u;                // staged candidates

struct MaeState {
    unsigned long long before[kLevels];  // weight below the current candidate range
    unsigned long long total[kLevels];   // total weight of the region (after the first pass)
    unsigned long long count[kLevels];   // members of the region (after the first pass)
    uint32_t base[kLevels];              // key of the region's lower edge
    uint32_t prefix[kLevels];            // digits chosen so far
    int top[kLevels];                    // key bits still unresolved (0: done)
    uint32_t limit[kLevels];             // largest relative key that can still take part (bound of the range)
    uint32_t cand_count[kLevels];        // samples offered to the candidate list of level l
    uint32_t active;                     // bit l: level l takes part in the selection
    uint32_t max_bits;                   // bits of the largest |w| of the data
    uint32_t ticket;                     // CTAs of a pass with a fused selection that have finished
};
static_assert(sizeof(MaeState) <= kEmMaeStateBytes, "state must fit its slot");

struct MaeWs {
    double* partials;
    MaeState* state;
    unsigned long long* hist;   // [16][kMaeBins] weight
    unsigned long long* chist;  // [16][kMaeBins] count
    uint2* cand;                // [16][cand_cap] {rel key, fixed-point weight}
    uint32_t cand_cap;          // entries per level (from the workspace size)
};

__host__ __device__ inline MaeWs mae_ws(void* d_ws, size_t ws_bytes)
{
    char* p = static_cast<char*>(d_ws) + kEmMaeOffset;
    return MaeWs{static_cast<double*>(d_ws), reinterpret_cast<MaeState*>(p),
                 reinterpret_cast<unsigned long long*>(p + kEmMaeStateBytes),
                 reinterpret_cast<unsigned long long*>(p + kEmMaeStateBytes + kEmMaeHistBytes),
                 reinterpret_cast<uint2*>(p + kEmMaeStateBytes + 2 * kEmMaeHistBytes), mae_cand_capacity(ws_bytes)};
}

// Order-preserving key: x <= y  <=>  key(x) <= key(y); -0 and +0 share a key.
__device__ __forceinline__ uint32_t order_key(float x)
{
    const uint32_t u = __float_as_uint(x + 0.0f);
    return u ^ ((uint32_t)((int32_t)u >> 31) | 0x80000000u);  // negative: all bits flip, else only the sign
}
__device__ __forceinline__ float key_to_float(uint32_t k)
{
    return __uint_as_float((k & 0x80000000u) ? (k & 0x7fffffffu) : ~k);
}

// |m| as a 31-bit fixed-point integer relative to the largest magnitude of the data.
__device__ __forceinline__ uint32_t fixed_weight(float m, uint32_t max_bits)
{
    const uint32_t b = __float_as_uint(fabsf(m));
    const int e = max((int)(b >> 23), 1), emax = max((int)(max_bits >> 23), 1);
    const uint32_t mant = (b & 0x7fffffu) | ((b >> 23) ? 0x800000u : 0u);
    const int sh = e - emax + 7;
    if (sh >= 0) return mant << min(sh, 7);
    return (-sh >= 32) ? 0u : (mant >> (-sh));
}

// ---------------------------------------------------------------- largest |w|

template <class DT>
__global__ void __launch_bounds__(kMaeThreads, 1)
mae_absmax_kernel(const EmTensors T, MaeState* __restrict__ state)
{
    __shared__ uint32_t s_max[kMaeThreads / 32];
    const int tid = threadIdx.x;
    const int64_t total_rows = T.row_end[T.count - 1];
    float a = 0.0f;
    int t_cur = 0;
    for (int64_t g = blockIdx.x; g < total_rows; g += gridDim.x) {
        while (g >= T.row_end[t_cur]) ++t_cur;
        const int64_t r = g - (t_cur ? T.row_end[t_cur - 1] : 0);
        const int64_t idx = (r * kMaeThreads + tid) * kLaneW;
        if (idx < T.n[t_cur]) {
            float v[kLaneW];
            widen(load_raw<DT>(T.ptr[t_cur], idx), v);
#pragma unroll
            for (int k = 0; k < kLaneW; ++k) a = fmaxf(a, fabsf(v[k]));
        }
    }
    uint32_t b = __float_as_uint(a);
#pragma unroll
    for (int off = 16; off; off >>= 1) b = max(b, __shfl_xor_sync(kFull, b, off));
    if ((tid & 31) == 0) s_max[tid >> 5] = b;
    __syncthreads();
    if (tid == 0) {
        for (int k = 1; k < kMaeThreads / 32; ++k) b = max(b, s_max[k]);
        atomicMax(&state->max_bits, b);  // non-negative floats order like their bits
    }
}

// ---------------------------------------------------------------- per-iteration setup

// Region key ranges from the current levels, selection state reset, histograms cleared.
__global__ void __launch_bounds__(kMaeBins)
mae_init_kernel(const float* __restrict__ levels, uint32_t skip_mask, MaeWs W)
{
    __shared__ float s_xi[kLevels], s_lv[kLevels];
    make_thresholds(levels, s_xi, s_lv, threadIdx.x);
    __syncthreads();
    if (threadIdx.x < kLevels) {
        const int l = threadIdx.x;
        // members of region l lie in [lo, hi] with lo, hi clipped to [-1, 1]
        const float lo = (l == 0) ? -1.0f : fminf(fmaxf(s_xi[l - 1], -1.0f), 1.0f);
        const float hi = (l == kLevels - 1) ? 1.0f : fminf(fmaxf(s_xi[l], -1.0f), 1.0f);
        const uint32_t klo = order_key(lo), khi = order_key(hi);
        const uint32_t range = (khi > klo) ? khi - klo : 0u;
        const int bits = 32 - __clz(range | 1u);
        const bool on = !((skip_mask >> l) & 1u);
        W.state->base[l] = klo;
        W.state->prefix[l] = 0u;
        W.state->top[l] = on ? bits : 0;
        W.state->before[l] = 0ull;
        W.state->total[l] = 0ull;
        W.state->count[l] = 0ull;
        W.state->cand_count[l] = 0u;
        W.state->limit[l] = 0xffffffffu;
    }
    if (threadIdx.x == 0) W.state->active = ~skip_mask & 0xffffu;
    for (int k = threadIdx.x; k < kFineSlots; k += blockDim.x) {  // covers the 16 x kMaeBins digit bins as well
        W.hist[k] = 0ull;
        W.chist[k] = 0ull;
    }
}

// ---------------------------------------------------------------- bin selection

// Block-wide step of the selection, one thread per bin (threads beyond the bins pass 0): given this thread's bin weight `mine`,
// finds the first bin j with 2 (before + cumulative(j)) >= total.  Returns through the shared
// result the bin and the cumulative weight below it.  *all_out = sum of all bins.
struct PickResult {
    int bin;
    unsigned long long excl;
};

template <int NT = kMaeBins>
__device__ __forceinline__ PickResult pick_bin(unsigned long long mine, unsigned long long before,
                                               unsigned long long total, bool total_is_sum,
                                               unsigned long long* s_wsum, PickResult* s_res,
                                               unsigned long long* all_out)
{
    const int j = threadIdx.x, lane = j & 31, warp = j >> 5;
    unsigned long long incl = mine;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const unsigned long long t = __shfl_up_sync(kFull, incl, off);
        if (lane >= off) incl += t;
    }
    __syncthreads();  // s_wsum / s_res may still be read from a previous call
    if (lane == 31) s_wsum[warp] = incl;
    __syncthreads();
    unsigned long long carry = 0ull, all = 0ull;
    for (int k = 0; k < NT / 32; ++k) {
        if (k < warp) carry += s_wsum[k];
        all += s_wsum[k];
    }
    incl += carry;
    if (total_is_sum) total = all;
    const unsigned long long excl = incl - mine;
    const bool reached = 2ull * (before + incl) >= total;
    const bool prev_reached = (j > 0) && (2ull * (before + excl) >= total);
    if (reached && !prev_reached) *s_res = PickResult{j, excl};  // exactly one thread: monotone
    __syncthreads();
    *all_out = all;
    return *s_res;
}

// The next digit of level l after a pass that was not the first: the bin of the global
// histogram (cleared on the way) in which the cumulative weight reaches half of the region's
// total.  Called by all NT threads of a CTA; threads beyond the bins only take part in the scan.
template <int NT>
__device__ __forceinline__ void select_body(const MaeWs& W, int l, unsigned long long* s_wsum, PickResult* s_res)
{
    MaeState* S = W.state;
    const int j = threadIdx.x;
    const int top = S->top[l];
    if (top <= 0) return;  // uniform over the CTA
    unsigned long long mine = 0ull;
    if (j < kMaeBins) {
        mine = __ldcg(&W.hist[l * kMaeBins + j]);
        W.hist[l * kMaeBins + j] = 0ull;
    }
    const unsigned long long before = S->before[l];
    unsigned long long all;
    const PickResult r = pick_bin<NT>(mine, before, S->total[l], false, s_wsum, s_res, &all);
    if (j == 0) {
        const int sh = max(top - kMaeDigitBits, 0);
        S->before[l] = before + r.excl;
        S->prefix[l] = (S->prefix[l] << (top - sh)) | (uint32_t)r.bin;
        S->top[l] = sh;
    }
}

// What the level update needs beside the selection state.
struct MaeFinal {
    int enabled;  // the pass that carries this is the iteration's last launch and ends with the update
    int n_records;
    int64_t n_total;
    const float* levels_in;
    float* levels_out;
    uint32_t skip_mask;
    bof4_em_stats* stats;
    double* err_slot;
    int unit;
};

// Level update and statistics of one iteration, by all threads of one CTA (s_part: one double per warp).
__device__ __forceinline__ void finalize_body(const MaeWs& W, const MaeFinal& F, double* s_part)
{
    const MaeState* S = W.state;
    double e = 0.0;
    for (int r = threadIdx.x; r < F.n_records; r += blockDim.x) e += __ldcg(&W.partials[(size_t)r * kEmRecordDoubles]);
#pragma unroll
    for (int off = 16; off; off >>= 1) e += __shfl_xor_sync(kFull, e, off);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) s_part[threadIdx.x >> 5] = e;
    __syncthreads();
    if (threadIdx.x < kLevels) {
        const int l = threadIdx.x;
        const float old = F.levels_in[l];
        const bool on = !((F.skip_mask >> l) & 1u);
        const unsigned long long total = S->total[l];
        const float med = (on && total > 0ull) ? key_to_float(S->base[l] + S->prefix[l]) : old;
        if (F.stats) {
            const int emax = max((int)(S->max_bits >> 23), 1);
            F.stats->s1[l] = 0.0;
            F.stats->s0[l] = F.unit ? (double)total : ldexp((double)total, emax - 157);  // undo the fixed-point scale
            F.stats->count[l] = S->count[l];
            F.stats->median[l] = med;
        }
        if (F.levels_out && on) F.levels_out[l] = med;
    }
    if (threadIdx.x == 0) {
        double err = 0.0;
        for (int k = 0; k < (int)(blockDim.x >> 5); ++k) err += s_part[k];  // warp order: fixed
        if (F.stats) {
            F.stats->err_sum = err;
            F.stats->n_total = F.n_total;
        }
        if (F.err_slot) *F.err_slot = (F.n_total > 0) ? err / (double)F.n_total : 0.0;
    }
}

// ---------------------------------------------------------------- data pass

// FIRST: every member of an active level takes part; also accumulates sum |w - m xhat[c]| (one
// partial record per CTA) and, with COUNT, the member counts.
// Later passes return at once when no level has bits left.  Only about one sample in 500 still
// takes part in them (those whose key carries the digits chosen so far), so their loop over the
// data does no more than find these: the 257-bin table of the region search holds, instead of
// thresholds, the hull [lo, hi] of the normalised weights that can still take part in each bin
// (one 8-byte read and two comparisons per weight), and a hit is appended to a queue in shared
// memory.  The queue is worked off by all threads after the loop (region search, digit,
// histogram, candidate list), so that the rare, long path does not run with one lane in 32.
// COLLECT (second pass): every participating sample is also appended to its level's list.
constexpr int kMaeQueue = kLevels * kMaeBins * 4 / 8;  // entries {x, weight} in the count histogram's space
constexpr int kLaterQueue = kLevels * kMaeBins * 4 / 16;  // entries {address, block constant, weight} (bf16 later passes)

// TAIL (a later pass without a candidate list): the CTA that finishes last, found by an atomic
// ticket so that nobody waits, also selects the next digit of every level and, if F.enabled,
// updates the levels: one launch instead of three.  When nothing is left the whole grid
// returns at once and CTA 0 does the update.
template <class DT, int I, bool SIGNED, bool FIRST, bool COUNT, bool COLLECT, bool TAIL>
__global__ void __launch_bounds__(kMaeThreads, 1)
mae_pass_kernel(const EmTensors T, const float* __restrict__ levels, MaeWs W, const MaeFinal F)
{
    extern __shared__ __align__(16) unsigned char s_raw[];
    unsigned char* s_lut = s_raw;
    uint32_t* s_lo = reinterpret_cast<uint32_t*>(s_raw + kLutBytes);
    uint32_t* s_hi = s_lo + kLevels * kMaeBins;
    uint32_t* s_cn = s_hi + kLevels * kMaeBins;
    uint2* s_queue = reinterpret_cast<uint2*>(s_cn);  // later passes (which keep no counts)
    uint2* s_cand = reinterpret_cast<uint2*>(s_cn + kLevels * kMaeBins);  // [16][kMaeStage] (COLLECT)
    __shared__ uint32_t s_ncand[kLevels], s_gbase[kLevels];
    __shared__ volatile uint32_t s_over[kLevels];  // level's global list is known to have overflowed
    __shared__ float s_xi[kLevels], s_lv[kLevels];
    __shared__ int s_multi;
    __shared__ WideScratch s_wide;
    __shared__ uint4 s_lvl[kLevels];  // {base, prefix, top | shift << 8 | mask << 16, on}
    // first pass: {base, shift | on << 31, level, -}, one column per lane of a quarter warp (the unit
    // a 16-byte shared-memory read is served in), so that the read never meets a bank conflict
    __shared__ uint4 s_lvl1[kLevels * 8];
    __shared__ uint2 s_iv[kLutBins];  // later passes: bits of {lo, hi} per table bin (lo > hi: nothing)
    __shared__ float2 s_span[kLevels];
    __shared__ uint32_t s_qn;
    __shared__ double s_err[kMaeThreads / 32];
    __shared__ const void* s_ptr[kEmMaxTensors];
    __shared__ int64_t s_n[kEmMaxTensors], s_row_end[kEmMaxTensors];

    __shared__ unsigned long long s_wsum[kMaeThreads / 32];
    __shared__ PickResult s_res;
    __shared__ int s_last;
    if (!FIRST) {  // nothing left to resolve: uniform over the grid
        int any = 0;
        for (int l = 0; l < kLevels; ++l) any |= W.state->top[l];
        if (any <= 0) {
            if (TAIL && F.enabled && T.last && blockIdx.x == 0) finalize_body(W, F, s_err);
            return;
        }
    }
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    make_thresholds(levels, s_xi, s_lv, tid);
    if (tid < kLevels) {
        const int top = W.state->top[tid];
        const int sh = max(top - kMaeDigitBits, 0);
        const uint32_t mask = (1u << (top - sh)) - 1u;
        s_lvl[tid] = make_uint4(W.state->base[tid], W.state->prefix[tid],
                                (uint32_t)top | ((uint32_t)sh << 8) | (mask << 16), top > 0 ? 1u : 0u);
        for (int q = 0; q < 8; ++q)
            s_lvl1[tid * 8 + q] = make_uint4(W.state->base[tid], (uint32_t)sh | (top > 0 ? 0x80000000u : 0u),
                                             __float_as_uint(levels[tid]), 0u);
    }
    if (tid < T.count) {
        s_ptr[tid] = T.ptr[tid];
        s_n[tid] = T.n[tid];
        s_row_end[tid] = T.row_end[tid];
    }
    for (int k = tid; k < (FIRST ? 3 : 2) * kLevels * kMaeBins; k += kMaeThreads) s_lo[k] = 0u;
    if (tid < kLevels) {
        s_ncand[tid] = 0u;
        s_over[tid] = 0u;
    }
    if (tid == 0) s_qn = 0u;
    const uint32_t max_bits = W.state->max_bits;
    __syncthreads();
    bool lut_ok = true;
    if (FIRST) {
        build_lut(s_xi, s_lut, &s_multi, [](int base) { return (uint32_t)base; });
        __syncthreads();
        lut_ok = s_multi == 0;
    } else {
        // Participants of level l have keys in [base + (prefix << top), base + ((prefix + 1) << top));
        // keys and normalised weights are ordered alike, so they lie between the weights of the
        // two end keys (clipped to [-1, 1]), and so do their table bins.
        if (tid < kLevels) {
            const uint4 L = s_lvl[tid];
            const int top = (int)(L.z & 0xffu);
            float2 span = make_float2(2.0f, -2.0f);
            if (L.w) {
                const uint32_t kmin = order_key(-1.0f), kmax = order_key(1.0f);
                const unsigned long long lo64 = (unsigned long long)L.x + ((unsigned long long)L.y << top);
                const unsigned long long hi64 = lo64 + ((1ull << top) - 1ull);
                const uint32_t klo = max(lo64 > kmax ? kmax : (uint32_t)lo64, kmin);
                const uint32_t khi = max(hi64 > kmax ? kmax : (uint32_t)hi64, kmin);
                span = make_float2(key_to_float(klo), key_to_float(khi));
            }
            s_span[tid] = span;
        }
        __syncthreads();
        for (int b = tid; b < kLutBins; b += kMaeThreads) {
            float2 iv = make_float2(2.0f, -2.0f);
            for (int l = 0; l < kLevels; ++l) {
                const float2 sp = s_span[l];
                if (sp.x > sp.y) continue;
                const int blo = (int)(__float_as_uint(lut_key(sp.x)) - kLutMagicBits);
                const int bhi = (int)(__float_as_uint(lut_key(sp.y)) - kLutMagicBits);
                if (b >= blo && b <= bhi) iv = make_float2(fminf(iv.x, sp.x), fmaxf(iv.y, sp.y));
            }
            s_iv[b] = make_uint2(__float_as_uint(iv.x), __float_as_uint(iv.y));
        }
        __syncthreads();
        for (int k = tid; k < kLutBins * 32; k += kMaeThreads)  // one column per lane, as in the region table
            *reinterpret_cast<uint2*>(s_lut + k * 8) = s_iv[k >> 5];
        __syncthreads();
    }

    // One participating sample of a later pass: digit histogram and (COLLECT) candidate list.
    auto later_sample = [&](float xk, uint32_t a) {
        const uint32_t c = (uint32_t)region_of(xk, s_xi);
        const uint4 L = s_lvl[c];
        const uint32_t rel = order_key(xk) - L.x;
        const uint32_t top = L.z & 0xffu, sh = (L.z >> 8) & 0xffu, mask = L.z >> 16;
        if (!(L.w && (uint32_t)((unsigned long long)rel >> top) == L.y)) return;
        const uint32_t bin = c * kMaeBins + ((rel >> sh) & mask);
        const uint32_t old = atomicAdd(&s_lo[bin], a);
        if (old + a < old) atomicAdd(&s_hi[bin], 1u);
        if (COLLECT) {
            // staged per CTA and level; the rare overflow of a slot goes straight to the
            // global list (whose count only needs to stay above the capacity once full)
            const uint32_t slot = atomicAdd(&s_ncand[c], 1u);
            if (slot < (uint32_t)kMaeStage) {
                s_cand[c * kMaeStage + slot] = make_uint2(rel, a);
            } else if (!s_over[c]) {
                uint32_t* cnt = &W.state->cand_count[c];
                if (*reinterpret_cast<volatile uint32_t*>(cnt) <= W.cand_cap) {
                    const uint32_t gslot = atomicAdd(cnt, 1u);
                    if (gslot < W.cand_cap) W.cand[(size_t)c * W.cand_cap + gslot] = make_uint2(rel, a);
                } else {
                    s_over[c] = 1u;  // remembered per CTA: later samples of this level skip the look-up
                }
            }
        }
    };

    const int64_t total_rows = T.row_end[T.count - 1];
    const uint32_t lut_base = lut_lane_base(s_lut, lane);
    double err = 0.0;
    int t_cur = 0;
    // row g of the concatenated tensors: this thread's 16 weights, or zeros past the end (ok = false)
    auto fetch = [&](int64_t g, bool& ok) -> RawRow<DT> {
        ok = false;
        if (g >= total_rows) return zero_raw<DT>();
        while (g >= s_row_end[t_cur]) ++t_cur;
        const int64_t r = g - (t_cur ? s_row_end[t_cur - 1] : 0);
        const int64_t idx = (r * kMaeThreads + tid) * kLaneW;
        ok = idx < s_n[t_cur];
        return ok ? load_raw<DT>(s_ptr[t_cur], idx) : zero_raw<DT>();
    };
    bool ok, ok_next;
    RawRow<DT> raw = fetch(blockIdx.x, ok);
    for (int64_t g = blockIdx.x; g < total_rows; g += gridDim.x, ok = ok_next) {
        const RawRow<DT> next = fetch(g + gridDim.x, ok_next);  // in flight while this row is processed
        float v[kLaneW];
        widen(raw, v);
        raw = next;
        float gmax;
        const float m = block_constant<I, SIGNED>(v, gmax, &s_wide);
        const bool safe = row_is_safe(gmax, ok);
        float x[kLaneW];
        normalise16<false>(v, m, safe && DT::code == BF16::code, x);
        if (!ok) continue;
        const uint32_t a = T.unit ? 1u : fixed_weight(m, max_bits);  // App. D variant: plain median
        if (FIRST) {
            const bool use_lut = lut_ok && safe;
            float e = 0.0f;
            // error of a weight: |v - m xhat|; the normalised-domain variant measures |x - xhat|
            float scale = m;
            if (T.unit) {
                scale = 1.0f;
#pragma unroll
                for (int k = 0; k < kLaneW; ++k) v[k] = x[k];
            }
#pragma unroll
            for (int k = 0; k < kLaneW; k += 2) {
                const float2 key = lut_key2(make_float2(x[k], x[k + 1]));
                const float kk[2] = {key.x, key.y};
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    const float xk = x[k + h];
                    uint32_t c;
                    if (use_lut) {
                        const uint2 ent = lut_probe(kk[h], lut_base);
                        c = ent.y + ((xk >= __uint_as_float(ent.x)) ? 1u : 0u);
                    } else {
                        c = (uint32_t)region_of(xk, s_xi);
                    }
                    const uint4 L = s_lvl1[c * 8 + (lane & 7)];
                    e += fabsf(fmaf(-scale, __uint_as_float(L.z), v[k + h]));
                    if ((int32_t)L.y < 0) {
                        // a member's rel is below 2^top, so its digit is rel >> (top - 9) as it stands; the
                        // constant mask only keeps a non-finite input's garbage inside the level's bins.
                        // The funnel shift takes the shift count from the low five bits of L.y.
                        const uint32_t rel = order_key(xk) - L.x;
                        const uint32_t bin = c * kMaeBins + (__funnelshift_r(rel, 0u, L.y) & (kMaeBins - 1u));
                        const uint32_t old = atomicAdd(&s_lo[bin], a);
                        if (old + a < old) atomicAdd(&s_hi[bin], 1u);
                        if (COUNT) atomicAdd(&s_cn[bin], 1u);
                    }
                }
            }
            err += (double)e;
        } else {
            // A weight inside its bin's hull may take part and is queued.  A row that cannot use the
            // table (a non-finite or extreme block constant makes its quotients unfit as table
            // keys) offers all 16.
#pragma unroll
            for (int k = 0; k < kLaneW; k += 2) {
                const float2 key = lut_key2(make_float2(x[k], x[k + 1]));
                const float kk[2] = {key.x, key.y};
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    bool hit = true;
                    if (safe) {
                        const uint2 iv = lut_probe(kk[h], lut_base);
                        hit = x[k + h] >= __uint_as_float(iv.x) && x[k + h] <= __uint_as_float(iv.y);
                    }
                    if (hit) {
                        const uint32_t slot = atomicAdd(&s_qn, 1u);
                        if (slot < (uint32_t)kMaeQueue)
                            s_queue[slot] = make_uint2(__float_as_uint(x[k + h]), a);
                        else
                            later_sample(x[k + h], a);  // queue full: handled on the spot
                    }
                }
            }
        }
    }
    __syncthreads();
    if (!FIRST) {
        const uint32_t q = min(s_qn, (uint32_t)kMaeQueue);
        for (uint32_t i = tid; i < q; i += kMaeThreads) {
            const uint2 ent = s_queue[i];
            later_sample(__uint_as_float(ent.x), ent.y);
        }
        __syncthreads();
    }
    for (int k = tid; k < kLevels * kMaeBins; k += kMaeThreads) {
        const unsigned long long wsum = ((unsigned long long)s_hi[k] << 32) + s_lo[k];
        if (wsum) atomicAdd(&W.hist[k], wsum);
        if (FIRST && COUNT && s_cn[k]) atomicAdd(&W.chist[k], (unsigned long long)s_cn[k]);
    }
    if (COLLECT) {
        // one reservation per CTA and level, then a plain copy of the staged samples
        if (tid < kLevels) {
            const uint32_t k = min(s_ncand[tid], (uint32_t)kMaeStage);
            s_gbase[tid] = k ? atomicAdd(&W.state->cand_count[tid], k) : 0u;
        }
        __syncthreads();
        for (int k = tid; k < kLevels * kMaeStage; k += kMaeThreads) {
            const int l = k / kMaeStage, i = k % kMaeStage;
            const uint32_t dst = s_gbase[l] + (uint32_t)i;
            if ((uint32_t)i < min(s_ncand[l], (uint32_t)kMaeStage) && dst < W.cand_cap)
                W.cand[(size_t)l * W.cand_cap + dst] = s_cand[k];
        }
    }
    if (FIRST) {
#pragma unroll
        for (int off = 16; off; off >>= 1) err += __shfl_xor_sync(kFull, err, off);
        if (lane == 0) s_err[warp] = err;
        __syncthreads();
        if (tid == 0) {
            double t = 0.0;
            for (int k = 0; k < kMaeThreads / 32; ++k) t += s_err[k];
            double* rec = W.partials + (size_t)blockIdx.x * kEmRecordDoubles;
            rec[0] = T.accumulate ? rec[0] + t : t;
        }
    }
    if (TAIL && T.last) {
        // every thread's histogram atomics are ordered before the ticket of its CTA
        __threadfence();
        __syncthreads();
        if (tid == 0) s_last = (atomicAdd(&W.state->ticket, 1u) == gridDim.x - 1) ? 1 : 0;
        __syncthreads();
        if (s_last) {
            __threadfence();
            for (int l = 0; l < kLevels; ++l) select_body<kMaeThreads>(W, l, s_wsum, &s_res);
            if (tid == 0) W.state->ticket = 0u;
            if (F.enabled) {
                __threadfence();
                __syncthreads();  // the state written by thread 0 is read by the update
                finalize_body(W, F, s_err);
            }
        }
    }
}

// ---------------------------------------------------------------- later passes, bf16 weights
//
// The passes after the first on the 64-byte-per-lane front end: the same set-up, queue, digit
// histogram, candidate lists and fused selection as mae_pass_kernel without its first-pass
// parts; only the streaming loop differs (32 weights per lane, packed min/max, two row buffers
// used in turn).

// What a participating sample of a later pass does (digit histogram, candidate list), out of
// line: the streaming loop only queues samples, and its thirty-two unrolled copies must stay small
// enough for the instruction cache.
struct LaterCtx {
    const float* xi;
    const uint4* lvl;
    const uint32_t* limit;
    uint32_t *lo, *hi, *ncand;
    uint2* cand;
    volatile uint32_t* over;
    MaeState* state;
    uint2* gcand;
    uint32_t cap;
};
// marked |= bit if lo <= x <= hi (iv = bits of {lo, hi}); two predicate operations and a predicated OR.
__device__ __forceinline__ void mark_if_inside(uint32_t& marked, float x, uint2 iv, uint32_t bit)
{
    asm("{\n\t.reg .pred p;\n\tsetp.ge.f32 p, %1, %2;\n\tsetp.le.and.f32 p, %1, %3, p;\n\t@p or.b32 %0, %0, %4;\n\t}"
        : "+r"(marked)
        : "f"(x), "f"(__uint_as_float(iv.x)), "f"(__uint_as_float(iv.y)), "r"(bit));
}

template <bool COLLECT>
__device__ __noinline__ void later_sample_fn(const LaterCtx* C, float xk, uint32_t a)
{
    const uint32_t c = (uint32_t)region_of(xk, C->xi);
    const uint4 L = C->lvl[c];
    const uint32_t rel = order_key(xk) - L.x;
    const uint32_t top = L.z & 0xffu, sh = (L.z >> 8) & 0xffu, mask = L.z >> 16;
    if (!(L.w && (uint32_t)((unsigned long long)rel >> top) == L.y && rel <= C->limit[c])) return;
    const uint32_t bin = c * kMaeBins + ((rel >> sh) & mask);
    const uint32_t old = atomicAdd(&C->lo[bin], a);
    if (old + a < old) atomicAdd(&C->hi[bin], 1u);
    if (COLLECT) {
        // staged per CTA and level; the rare overflow of a slot goes straight to the
        // global list (whose count only needs to stay above the capacity once full)
        const uint32_t slot = atomicAdd(&C->ncand[c], 1u);
        if (slot < (uint32_t)kMaeStage) {
            C->cand[c * kMaeStage + slot] = make_uint2(rel, a);
        } else if (!C->over[c]) {
            uint32_t* cnt = &C->state->cand_count[c];
            if (*reinterpret_cast<volatile uint32_t*>(cnt) <= C->cap) {
                const uint32_t gslot = atomicAdd(cnt, 1u);
                if (gslot < C->cap) C->gcand[(size_t)c * C->cap + gslot] = make_uint2(rel, a);
            } else {
                C->over[c] = 1u;  // remembered per CTA: later samples of this level skip the look-up
            }
        }
    }
}

template <int I, bool SIGNED, bool COLLECT, bool TAIL>
__global__ void __launch_bounds__(kMaeThreads, 1)
mae_later32_kernel(const EmTensors T, const float* __restrict__ levels, MaeWs W, const MaeFinal F)
{
    constexpr bool FIRST = false, COUNT = false;
    extern __shared__ __align__(16) unsigned char s_raw[];
    unsigned char* s_lut = s_raw;
    uint32_t* s_lo = reinterpret_cast<uint32_t*>(s_raw + kLutBytes);
    uint32_t* s_hi = s_lo + kLevels * kMaeBins;
    uint32_t* s_cn = s_hi + kLevels * kMaeBins;
    uint4* s_queue = reinterpret_cast<uint4*>(s_cn);  // kLaterQueue entries in the count histogram's space
    uint2* s_cand = reinterpret_cast<uint2*>(s_cn + kLevels * kMaeBins);  // [16][kMaeStage] (COLLECT)
    __shared__ uint32_t s_ncand[kLevels], s_gbase[kLevels];
    __shared__ volatile uint32_t s_over[kLevels];  // level's global list is known to have overflowed
    __shared__ float s_xi[kLevels], s_lv[kLevels];
    __shared__ int s_multi;
    __shared__ WideScratch s_wide;
    __shared__ uint4 s_lvl[kLevels];  // {base, prefix, top | shift << 8 | mask << 16, on}
    __shared__ uint32_t s_limit[kLevels];  // largest relative key of the level's range
    // first pass: {base, shift | on << 31, level, -}, one column per lane of a quarter warp (the unit
    // a 16-byte shared-memory read is served in), so that the read never meets a bank conflict
    __shared__ uint4 s_lvl1[kLevels * 8];
    __shared__ uint2 s_iv[kLutBins];  // later passes: bits of {lo, hi} per table bin (lo > hi: nothing)
    __shared__ float2 s_span[kLevels];
    __shared__ uint32_t s_qn;
    __shared__ double s_err[kMaeThreads / 32];
    __shared__ const void* s_ptr[kEmMaxTensors];
    __shared__ int64_t s_n[kEmMaxTensors], s_row_end[kEmMaxTensors];

    __shared__ unsigned long long s_wsum[kMaeThreads / 32];
    __shared__ PickResult s_res;
    __shared__ int s_last;
    if (!FIRST) {  // nothing left to resolve: uniform over the grid
        int any = 0;
        for (int l = 0; l < kLevels; ++l) any |= W.state->top[l];
        if (any <= 0) {
            if (TAIL && F.enabled && T.last && blockIdx.x == 0) finalize_body(W, F, s_err);
            return;
        }
    }
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    make_thresholds(levels, s_xi, s_lv, tid);
    if (tid < kLevels) {
        const int top = W.state->top[tid];
        const int sh = max(top - kMaeDigitBits, 0);
        const uint32_t mask = (1u << (top - sh)) - 1u;
        s_lvl[tid] = make_uint4(W.state->base[tid], W.state->prefix[tid],
                                (uint32_t)top | ((uint32_t)sh << 8) | (mask << 16), top > 0 ? 1u : 0u);
        s_limit[tid] = W.state->limit[tid];
        for (int q = 0; q < 8; ++q)
            s_lvl1[tid * 8 + q] = make_uint4(W.state->base[tid], (uint32_t)sh | (top > 0 ? 0x80000000u : 0u),
                                             __float_as_uint(levels[tid]), 0u);
    }
    if (tid < T.count) {
        s_ptr[tid] = T.ptr[tid];
        s_n[tid] = T.n[tid];
        s_row_end[tid] = T.row_end[tid];
    }
    for (int k = tid; k < (FIRST ? 3 : 2) * kLevels * kMaeBins; k += kMaeThreads) s_lo[k] = 0u;
    if (tid < kLevels) {
        s_ncand[tid] = 0u;
        s_over[tid] = 0u;
    }
    if (tid == 0) s_qn = 0u;
    const uint32_t max_bits = W.state->max_bits;
    __syncthreads();
    bool lut_ok = true;
    if (FIRST) {
        build_lut(s_xi, s_lut, &s_multi, [](int base) { return (uint32_t)base; });
        __syncthreads();
        lut_ok = s_multi == 0;
    } else {
        // Participants of level l have keys in [base + (prefix << top), base + ((prefix + 1) << top));
        // keys and normalised weights are ordered alike, so they lie between the weights of the
        // two end keys (clipped to [-1, 1]), and so do their table bins.
        if (tid < kLevels) {
            const uint4 L = s_lvl[tid];
            const int top = (int)(L.z & 0xffu);
            float2 span = make_float2(2.0f, -2.0f);
            if (L.w) {
                const uint32_t kmin = order_key(-1.0f), kmax = order_key(1.0f);
                const unsigned long long lo64 = (unsigned long long)L.x + ((unsigned long long)L.y << top);
                unsigned long long hi64 = lo64 + ((1ull << top) - 1ull);
                const unsigned long long cap64 = (unsigned long long)L.x + W.state->limit[tid];
                if (hi64 > cap64) hi64 = cap64;
                const uint32_t klo = max(lo64 > kmax ? kmax : (uint32_t)lo64, kmin);
                const uint32_t khi = max(hi64 > kmax ? kmax : (uint32_t)hi64, kmin);
                span = make_float2(key_to_float(klo), key_to_float(khi));
                // The streaming loop tests the one-multiplication estimate x~ = RN(w RN(1/m)) of the
                // quotient, which lies within 1.5 * 2^-23 (relative) of it: the span is widened by
                // four times that, and what it lets through is tested again with the true quotient.
                span.x -= fabsf(span.x) * 0x1p-21f + 1e-30f;
                span.y += fabsf(span.y) * 0x1p-21f + 1e-30f;
            }
            s_span[tid] = span;
        }
        __syncthreads();
        for (int b = tid; b < kLutBins; b += kMaeThreads) {
            float2 iv = make_float2(2.0f, -2.0f);
            for (int l = 0; l < kLevels; ++l) {
                const float2 sp = s_span[l];
                if (sp.x > sp.y) continue;
                const int blo = (int)(__float_as_uint(lut_key(sp.x)) - kLutMagicBits);
                const int bhi = (int)(__float_as_uint(lut_key(sp.y)) - kLutMagicBits);
                if (b >= blo && b <= bhi) iv = make_float2(fminf(iv.x, sp.x), fmaxf(iv.y, sp.y));
            }
            s_iv[b] = make_uint2(__float_as_uint(iv.x), __float_as_uint(iv.y));
        }
        __syncthreads();
        for (int k = tid; k < kLutBins * 32; k += kMaeThreads)  // one column per lane, as in the region table
            *reinterpret_cast<uint2*>(s_lut + k * 8) = s_iv[k >> 5];
        __syncthreads();
    }

    // One participating sample of a later pass: digit histogram and (COLLECT) candidate list.
    __shared__ LaterCtx s_ctx;
    if (tid == 0)
        s_ctx = LaterCtx{s_xi, s_lvl, s_limit, s_lo, s_hi, s_ncand, s_cand, s_over, W.state, W.cand, W.cand_cap};
    __syncthreads();
    auto later_sample = [&](float xk, uint32_t a) { later_sample_fn<COLLECT>(&s_ctx, xk, a); };

    const int64_t total_rows = T.row_end[T.count - 1];
    const uint32_t lut_base = lut_lane_base(s_lut, lane);
    double err = 0.0;
    int t_cur = 0;
    // row g of the concatenated tensors: this thread's 32 weights, or zeros past the end (ok = false);
    // src: where they came from (a participating weight is read again by its index)
    auto fetch = [&](int64_t g, bool& ok, const uint16_t*& src) -> Raw32 {
        ok = false;
        if (g < total_rows) {
            while (g >= s_row_end[t_cur]) ++t_cur;
            const int64_t r = g - (t_cur ? s_row_end[t_cur - 1] : 0);
            const int64_t idx = (r * kMaeThreads + tid) * kLW;
            ok = idx < s_n[t_cur];
            if (ok) {
                src = static_cast<const uint16_t*>(s_ptr[t_cur]) + idx;
                return load_raw32(s_ptr[t_cur], idx);
            }
        }
        return zero_raw32();
    };
    // A weight that may take part is queued as {address, block constant}: the streaming loop only
    // notes where it is (a few instructions with one lane active); the division, the region search
    // and the rest are done when the queue is worked off, with all lanes busy.  A full queue makes
    // the lane handle its weight on the spot.
    auto quotient = [&](float v, float m) {
        if (div_safe(fabsf(m))) {  // the reciprocal sequence of the streaming loop, one weight
            const float r = __frcp_rn(m), q0 = __fmul_rn(v, r);
            return fmaf(fmaf(q0, -m, v), r, q0);
        }
        return normalise(v, m);
    };
    // A weight inside its table bin's hull may take part.  The streaming loop only marks such
    // weights in a bit mask (two comparisons and one predicated OR per weight); the few marked ones
    // (about one in 200) are queued by address.  A row that cannot use the table (a zero, non-finite
    // or extreme block constant) offers all its weights.
    auto row = [&](const Raw32& raw, bool ok, const uint16_t* src) {
        uint32_t u[16];
        words_of(raw, u);
        float mx, mn, g;
        lane_minmax32(u, mx, mn);
        const float m = block_constant32<I, SIGNED>(u, mx, mn, g, &s_wide);
        const uint32_t a = T.unit ? 1u : fixed_weight(m, max_bits);
        const bool table = __all_sync(kFull, ok && div_safe(g));
        const bool recip = div_safe(fabsf(m));
        const float r = recip ? __frcp_rn(m) : 0.0f;
        const float2 rr = make_float2(r, r);
        uint32_t marked = ok ? 0xffffffffu : 0u;
        if (table) {
            marked = 0u;
#pragma unroll
            for (int k = 0; k < 16; ++k) {
                const float2 v = make_float2(bf_lo(u[k]), bf_hi(u[k]));
                const float2 x = __fmul2_rn(v, rr);  // estimates of the quotients (see the widened spans)
                const float2 key = lut_key2(x);
                const uint2 i0 = lut_probe(key.x, lut_base), i1 = lut_probe(key.y, lut_base);
                mark_if_inside(marked, x.x, i0, 1u << (2 * k));
                mark_if_inside(marked, x.y, i1, 2u << (2 * k));
            }
        }
        if (marked) {
            const uint32_t cnt = (uint32_t)__popc(marked);
            uint32_t slot = atomicAdd(&s_qn, cnt);
            while (marked) {
                const int j = __ffs(marked) - 1;
                marked &= marked - 1u;
                if (slot < (uint32_t)kLaterQueue) {
                    const unsigned long long p = (unsigned long long)(src + j);
                    s_queue[slot] = make_uint4((uint32_t)p, (uint32_t)(p >> 32), __float_as_uint(m), a);
                } else {
                    later_sample(quotient(__uint_as_float((uint32_t)__ldg(src + j) << 16), m), a);
                }
                ++slot;
            }
        }
    };
    // The queue is worked off by all threads: region search, digit, histogram; with COLLECT the
    // candidates staged meanwhile go to the global lists (one reservation per level).  Called by
    // the whole CTA every kDrainRows rows, so that neither the queue nor the staging slots fill up
    // however many rows a CTA streams.
    auto drain = [&]() {
        __syncthreads();
        const uint32_t q = min(s_qn, (uint32_t)kLaterQueue);
        for (uint32_t i = tid; i < q; i += kMaeThreads) {
            const uint4 ent = s_queue[i];
            const uint16_t* p = reinterpret_cast<const uint16_t*>(((unsigned long long)ent.y << 32) | ent.x);
            const float m = __uint_as_float(ent.z);
            later_sample(quotient(__uint_as_float((uint32_t)__ldg(p) << 16), m), ent.w);
        }
        __syncthreads();
        if (tid == 0) s_qn = 0u;
        if (COLLECT) {
            if (tid < kLevels) {
                const uint32_t k = min(s_ncand[tid], (uint32_t)kMaeStage);
                s_gbase[tid] = k ? atomicAdd(&W.state->cand_count[tid], k) : 0u;
            }
            __syncthreads();
            for (int k = tid; k < kLevels * kMaeStage; k += kMaeThreads) {
                const int l = k / kMaeStage, i = k % kMaeStage;
                const uint32_t dst = s_gbase[l] + (uint32_t)i;
                if ((uint32_t)i < min(s_ncand[l], (uint32_t)kMaeStage) && dst < W.cand_cap)
                    W.cand[(size_t)l * W.cand_cap + dst] = s_cand[k];
            }
            __syncthreads();
            if (tid < kLevels) s_ncand[tid] = 0u;
        }
        __syncthreads();
    };
    // after a first pass on the fine grid about 130 samples per row are queued, up to a sixth of
    // them for one of the central levels (whose staging slot holds kMaeStage)
    constexpr int kDrainRows = 8;
    {
        bool ok_a, ok_b;
        const uint16_t *src_a = nullptr, *src_b = nullptr;
        int64_t g = blockIdx.x;
        const int64_t GS = gridDim.x;
        Raw32 ra = fetch(g, ok_a, src_a), rb;
        int since = 0;
        if (g < total_rows) {
            while (true) {  // g and the trip count are the same for all threads of the CTA
                rb = fetch(g + GS, ok_b, src_b);
                row(ra, ok_a, src_a);
                g += GS;
                if (g >= total_rows) break;
                ra = fetch(g + GS, ok_a, src_a);
                row(rb, ok_b, src_b);
                g += GS;
                if (g >= total_rows) break;
                since += 2;
                if (since >= kDrainRows) {
                    since = 0;
                    drain();
                }
            }
        }
    }
    drain();
    for (int k = tid; k < kLevels * kMaeBins; k += kMaeThreads) {
        const unsigned long long wsum = ((unsigned long long)s_hi[k] << 32) + s_lo[k];
        if (wsum) atomicAdd(&W.hist[k], wsum);
        if (FIRST && COUNT && s_cn[k]) atomicAdd(&W.chist[k], (unsigned long long)s_cn[k]);
    }
    if (FIRST) {
#pragma unroll
        for (int off = 16; off; off >>= 1) err += __shfl_xor_sync(kFull, err, off);
        if (lane == 0) s_err[warp] = err;
        __syncthreads();
        if (tid == 0) {
            double t = 0.0;
            for (int k = 0; k < kMaeThreads / 32; ++k) t += s_err[k];
            double* rec = W.partials + (size_t)blockIdx.x * kEmRecordDoubles;
            rec[0] = T.accumulate ? rec[0] + t : t;
        }
    }
    if (TAIL && T.last) {
        // every thread's histogram atomics are ordered before the ticket of its CTA
        __threadfence();
        __syncthreads();
        if (tid == 0) s_last = (atomicAdd(&W.state->ticket, 1u) == gridDim.x - 1) ? 1 : 0;
        __syncthreads();
        if (s_last) {
            __threadfence();
            for (int l = 0; l < kLevels; ++l) select_body<kMaeThreads>(W, l, s_wsum, &s_res);
            if (tid == 0) W.state->ticket = 0u;
            if (F.enabled) {
                __threadfence();
                __syncthreads();  // the state written by thread 0 is read by the update
                finalize_body(W, F, s_err);
            }
        }
    }
}

// One CTA per level, one thread per bin.  For a level with bits left: the bin in which the
// cumulative weight first reaches half of the total becomes the next digit.  After the first
// pass the totals (and counts) are those of the whole region.
__global__ void __launch_bounds__(kMaeBins)
mae_select_kernel(MaeWs W, int first)
{
    __shared__ unsigned long long s_wsum[kMaeBins / 32], s_csum[kMaeBins / 32];
    __shared__ PickResult s_res;
    MaeState* S = W.state;
    const int l = blockIdx.x, j = threadIdx.x, lane = j & 31, warp = j >> 5;
    const int top = S->top[l];
    if (top <= 0) return;  // uniform over the CTA
    const unsigned long long mine = W.hist[l * kMaeBins + j];
    W.hist[l * kMaeBins + j] = 0ull;
    unsigned long long c = 0ull;
    if (first) {
        c = W.chist[l * kMaeBins + j];
        W.chist[l * kMaeBins + j] = 0ull;
#pragma unroll
        for (int off = 16; off; off >>= 1) c += __shfl_xor_sync(kFull, c, off);
        if (lane == 0) s_csum[warp] = c;
    }
    const unsigned long long before = S->before[l];
    unsigned long long all;
    const PickResult r = pick_bin(mine, before, first ? 0ull : S->total[l], first != 0, s_wsum, &s_res, &all);
    if (j == 0) {
        const int sh = max(top - kMaeDigitBits, 0);
        S->before[l] = before + r.excl;
        S->prefix[l] = (S->prefix[l] << (top - sh)) | (uint32_t)r.bin;
        S->top[l] = sh;
        if (first) {
            unsigned long long count = 0ull;
            for (int k = 0; k < kMaeBins / 32; ++k) count += s_csum[k];
            S->total[l] = all;
            S->count[l] = count;
        }
    }
}

// After the collecting (second) pass.  A level whose candidate list holds every sample that
// matched the first digit is finished here: the remaining digits are selected from the list.
// A level whose list overflowed takes the ordinary histogram step and goes on to the later
// passes.  The lists reach millions of entries, so a cluster of kResolveCtas CTAs shares one
// level: each reads its part of the list into its own histogram, the histograms are summed
// through distributed shared memory, and every CTA takes the same (deterministic) decision.
constexpr int kResolveCtas = 8;

__global__ void __cluster_dims__(kResolveCtas, 1, 1) __launch_bounds__(kMaeThreads)
mae_resolve_kernel(MaeWs W)
{
    namespace cg = cooperative_groups;
    cg::cluster_group cluster = cg::this_cluster();
    const unsigned rank = cluster.block_rank();
    __shared__ unsigned long long s_wsum[kMaeThreads / 32];
    __shared__ uint32_t s_lo[kMaeBins], s_hi[kMaeBins];  // 64-bit bins as two words: native 32-bit atomics
    __shared__ PickResult s_res;
    MaeState* S = W.state;
    const int l = blockIdx.x / kResolveCtas, j = threadIdx.x;
    const bool has_bin = j < kMaeBins;  // one thread per bin; all threads read the list
    int top = S->top[l];
    if (top <= 0) return;  // the same for all CTAs of the cluster
    const uint32_t m = S->cand_count[l];
    unsigned long long before = S->before[l];
    const unsigned long long total = S->total[l];
    uint32_t prefix = S->prefix[l];
    unsigned long long all;
    // the digit of this pass, from the global histogram (cleared once every CTA has read it)
    {
        const unsigned long long mine = has_bin ? __ldcg(&W.hist[l * kMaeBins + j]) : 0ull;
        cluster.sync();  // also orders the reads of the state above before the write at the end
        if (rank == 0 && has_bin) W.hist[l * kMaeBins + j] = 0ull;
        const PickResult r = pick_bin<kMaeThreads>(mine, before, total, false, s_wsum, &s_res, &all);
        const int sh = max(top - kMaeDigitBits, 0);
        before += r.excl;
        prefix = (prefix << (top - sh)) | (uint32_t)r.bin;
        top = sh;
    }
    if (m <= W.cand_cap) {
        const uint2* cand = W.cand + (size_t)l * W.cand_cap;
        constexpr int kInFlight = 16;  // independent loads per thread
        constexpr uint32_t kChunk = kInFlight * kMaeThreads;
        while (top > 0) {
            const int sh = max(top - kMaeDigitBits, 0);
            const uint32_t mask = (1u << (top - sh)) - 1u;
            if (has_bin) {
                s_lo[j] = 0u;
                s_hi[j] = 0u;
            }
            __syncthreads();
            for (uint32_t i0 = rank * kChunk; i0 < m; i0 += kResolveCtas * kChunk) {
                uint2 c[kInFlight];
#pragma unroll
                for (int u = 0; u < kInFlight; ++u) {
                    const uint32_t i = i0 + u * kMaeThreads + j;
                    c[u] = (i < m) ? __ldcg(&cand[i]) : make_uint2(0xffffffffu, 0u);
                }
#pragma unroll
                for (int u = 0; u < kInFlight; ++u)
                    if (c[u].y != 0u && (c[u].x >> top) == prefix) {
                        const uint32_t bin = (c[u].x >> sh) & mask;
                        const uint32_t old = atomicAdd(&s_lo[bin], c[u].y);
                        if (old + c[u].y < old) atomicAdd(&s_hi[bin], 1u);
                    }
            }
            cluster.sync();  // every CTA's histogram is complete
            unsigned long long mine = 0ull;
            if (has_bin) {
                for (unsigned r = 0; r < kResolveCtas; ++r) {  // fixed order; integer sums anyway
                    const uint32_t* rlo = cluster.map_shared_rank(s_lo, r);
                    const uint32_t* rhi = cluster.map_shared_rank(s_hi, r);
                    mine += ((unsigned long long)rhi[j] << 32) + rlo[j];
                }
            }
            cluster.sync();  // nobody clears its histogram while another CTA still reads it
            const PickResult r = pick_bin<kMaeThreads>(mine, before, total, false, s_wsum, &s_res, &all);
            before += r.excl;
            prefix = (prefix << (top - sh)) | (uint32_t)r.bin;
            top = sh;
        }
    }
    if (rank == 0 && j == 0) {
        S->before[l] = before;
        S->prefix[l] = prefix;
        S->top[l] = top;
    }
}

// ---------------------------------------------------------------- first pass, bf16 weights
//
// With the 64-byte-per-lane front end the first data pass bins every normalised weight on ONE
// uniform grid instead of on a grid per region: fine bin f = RN(2048 x) + 2048 (a single packed
// multiply-add for two weights), and the slot of a sample of region c is (f, c & 1).  Regions are
// intervals of x, so a fine bin holds samples of consecutive regions; as long as no fine bin holds
// two thresholds, these are at most two regions of different parity and every slot belongs to one
// region.  Inside a region slots follow the order of x, so the selection walks the region's fine
// bins in ascending order; no per-region key arithmetic is needed per weight (the former first
// pass spent a third of its instructions on it).  The selected fine bin becomes the key range
// [base, base + 2^top) that the later passes refine digit by digit, exactly as after a first
// digit.  A codebook with two thresholds in one fine bin (levels closer than 1/2048) is
// "degenerate": the pass then bins per region on the first nine bits of the region-relative
// key, like the generic first pass, and the selection kernel does that pass's selection.

constexpr float kFineMagic = 12582912.0f + (float)kFineScale;  // 1.5 * 2^23 + 2048
__device__ __forceinline__ float2 fine_key2(float2 x)
{
    return __ffma2_rn(x, make_float2((float)kFineScale, (float)kFineScale), make_float2(kFineMagic, kFineMagic));
}
// Fine bin of x, clamped to the grid (x outside [-1, 1] only occurs for non-finite input).
__device__ __forceinline__ int fine_bin(float x)
{
    const float c = fminf(fmaxf(x, -1.0f), 1.0f);
    return (int)(__float_as_uint(fmaf(c, (float)kFineScale, kFineMagic)) - kLutMagicBits);
}
// Two thresholds share a fine bin.
__device__ __forceinline__ bool degenerate_codebook(const float* s_xi)
{
    bool d = false;
    for (int j = 0; j + 1 < kLevels - 1; ++j) d = d || fine_bin(s_xi[j]) == fine_bin(s_xi[j + 1]);
    return d;
}

// Slot sums in shared memory: 64-bit bins kept as two words (native 32-bit atomics with carry;
// addresses fall on random banks, so every atomic costs several wavefronts and a scheme with more,
// carry-free partial words per slot measured slower).
constexpr int kMae1Words = 2;
constexpr size_t kMae1Smem(bool count) { return (size_t)kLutBytes + (size_t)kFineSlots * 4u * (kMae1Words + (count ? 1u : 0u)); }
static_assert(kFineSlots >= kLevels * kMaeBins, "the per-region bins of the degenerate case fit the slot arrays");

struct Mae1Shared {
    float xi[kLevels], lv[kLevels];
    uint2 lvrep[kLevels * 32];  // {level l, byte offset of its parity half of the slots} for lane q at [l * 32 + q]
    uint32_t base[kLevels];     // degenerate case: key of each region's lower edge and digit shift
    int shift[kLevels];
    int multi, degenerate;
    WideScratch wide;
    double err[kMaeThreads / 32];
    const void* ptr[kEmMaxTensors];
    int64_t n[kEmMaxTensors], row_end[kEmMaxTensors];
};

// One sample into its slot.  The streaming loop addresses the slot arrays and the level table
// through explicit shared-window addresses (32-bit), like the table probe.
__device__ __forceinline__ void red_shared_add(uint32_t addr, uint32_t v)
{
    asm volatile("red.shared.add.u32 [%0], %1;" ::"r"(addr), "r"(v) : "memory");
}
template <int OFF>
__device__ __forceinline__ void red_shared_add_off(uint32_t addr, uint32_t v)
{
    asm volatile("red.shared.add.u32 [%0+%2], %1;" ::"r"(addr), "r"(v), "n"(OFF) : "memory");
}
__device__ __forceinline__ uint2 ld_shared_v2(uint32_t addr)
{
    uint2 v;
    asm("ld.shared.v2.u32 {%0, %1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"(addr));
    return v;
}
__device__ __forceinline__ uint32_t atom_shared_add(uint32_t addr, uint32_t v)
{
    uint32_t old;
    asm volatile("atom.shared.add.u32 %0, [%1], %2;" : "=r"(old) : "r"(addr), "r"(v) : "memory");
    return old;
}
// addr: shared-window address of the slot's low word (word arrays are kFineSlots * 4 bytes apart).
template <bool COUNT>
__device__ __forceinline__ void slot_add_at(uint32_t addr, uint32_t a)
{
    const uint32_t old = atom_shared_add(addr, a);
    if (old + a < old) red_shared_add_off<kFineSlots * 4>(addr, 1u);
    if (COUNT) red_shared_add_off<2 * kFineSlots * 4>(addr, 1u);
}
template <bool COUNT>
__device__ __forceinline__ void slot_add(uint32_t* s_lo, int slot, uint32_t a)
{
    slot_add_at<COUNT>((uint32_t)__cvta_generic_to_shared(s_lo) + (uint32_t)slot * 4u, a);
}

// A row outside the common case (a zero, extreme or non-finite block constant, a codebook the
// region table cannot serve, a degenerate codebook): true quotients, binary search.  Out of
// line.  Returns the row's error sum.
template <bool COUNT>
__device__ __noinline__ float mae1_row_slow(Raw32 raw, float m, uint32_t a, bool unit, const Mae1Shared* S, uint32_t* s_lo)
{
    uint32_t u[16];
    words_of(raw, u);
    const bool recip = div_safe(fabsf(m));
    const float r = recip ? __frcp_rn(m) : 0.0f;
    float e = 0.0f;
#pragma unroll 1
    for (int k = 0; k < 16; ++k) {
        const float2 v = make_float2(bf_lo(u[k]), bf_hi(u[k]));
        float2 x;
        if (recip) {  // the same quotient as the common path (reciprocal sequence, no guard)
            const float2 rr = make_float2(r, r), nm = make_float2(-m, -m);
            const float2 q0 = __fmul2_rn(v, rr);
            x = __ffma2_rn(__ffma2_rn(q0, nm, v), rr, q0);
        } else {
            x = make_float2(normalise(v.x, m), normalise(v.y, m));
        }
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const float xh = h ? x.y : x.x, vh = h ? v.y : v.x;
            const int c = region_of(xh, S->xi);
            e += unit ? fabsf(xh - S->lv[c]) : fabsf(fmaf(-m, S->lv[c], vh));
            if (S->degenerate) {
                const uint32_t rel = order_key(xh) - S->base[c];
                slot_add<COUNT>(s_lo, c * kMaeBins + (int)((rel >> S->shift[c]) & (uint32_t)(kMaeBins - 1)), a);
            } else if (xh == xh) {  // a NaN has no place on the grid
                slot_add<COUNT>(s_lo, fine_bin(xh) + (c & 1) * kFineStride, a);
            }
        }
    }
    return e;
}

template <int I, bool SIGNED, bool COUNT>
__global__ void __launch_bounds__(kMaeThreads, 1)
mae_pass1_32_kernel(const EmTensors T, const float* __restrict__ levels, MaeWs W)
{
    extern __shared__ __align__(16) unsigned char s_raw[];
    unsigned char* s_lut = s_raw;
    uint32_t* s_lo = reinterpret_cast<uint32_t*>(s_raw + kLutBytes);  // lo [kFineSlots], hi, (count)
    __shared__ Mae1Shared S;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    make_thresholds(levels, S.xi, S.lv, tid);
    if (tid < T.count) {
        S.ptr[tid] = T.ptr[tid];
        S.n[tid] = T.n[tid];
        S.row_end[tid] = T.row_end[tid];
    }
    if (tid < kLevels) {
        const int top = W.state->top[tid];
        S.base[tid] = W.state->base[tid];
        S.shift[tid] = max(top - kMaeDigitBits, 0);
    }
    for (int k = tid; k < kFineSlots * (kMae1Words + (COUNT ? 1 : 0)); k += kMaeThreads) s_lo[k] = 0u;
    if (tid < kLevels * 32)
        S.lvrep[tid] = make_uint2(__float_as_uint(levels[tid >> 5]), (uint32_t)((tid >> 5) & 1) * (uint32_t)(kFineStride * 4));
    const uint32_t max_bits = W.state->max_bits;
    __syncthreads();
    if (tid == 0) S.degenerate = degenerate_codebook(S.xi) ? 1 : 0;
    // table payload: byte offset of the region's row in the level table
    build_lut(S.xi, s_lut, &S.multi, [](int base) { return (uint32_t)base * 256u; });
    __syncthreads();
    const bool table_ok = S.multi == 0 && S.degenerate == 0;
    const bool unit = T.unit != 0;

    const int64_t total_rows = T.row_end[T.count - 1];
    double err = 0.0;
    int t_cur = 0;
    auto fetch = [&](int64_t g, bool& ok) -> Raw32 {
        ok = false;
        if (g < total_rows) {
            while (g >= S.row_end[t_cur]) ++t_cur;
            const int64_t r = g - (t_cur ? S.row_end[t_cur - 1] : 0);
            const int64_t idx = (r * kMaeThreads + tid) * kLW;
            ok = idx < S.n[t_cur];
            if (ok) return load_raw32(S.ptr[t_cur], idx);
        }
        return zero_raw32();
    };
    const uint32_t lut_base = lut_lane_base(s_lut, lane);
    const uint32_t lv_base = (uint32_t)__cvta_generic_to_shared(S.lvrep) + (uint32_t)lane * 8u;
    // slot address of a sample from the bits of its fine key: (bits - magic) * 4 + start of the slot array
    const uint32_t slot_base = (uint32_t)__cvta_generic_to_shared(s_lo) - kLutMagicBits * 4u;

    auto row = [&](const Raw32& raw, bool ok) {
        uint32_t u[16];
        words_of(raw, u);
        float mx, mn, g;
        lane_minmax32(u, mx, mn);
        const float m = block_constant32<I, SIGNED>(u, mx, mn, g, &S.wide);
        const uint32_t a = unit ? 1u : fixed_weight(m, max_bits);
        float e = 0.0f;
        if (table_ok && __all_sync(kFull, ok && div_safe(g))) {
            // true quotients (reciprocal sequence), region by the one-probe table, fine bin
            const float r = __frcp_rn(m), scale = unit ? 1.0f : m;
            const float2 rr = make_float2(r, r), nm = make_float2(-m, -m);
#pragma unroll
            for (int k = 0; k < 16; ++k) {
                const float2 v = make_float2(bf_lo(u[k]), bf_hi(u[k]));
                const float2 q0 = __fmul2_rn(v, rr);
                const float2 x = __ffma2_rn(__ffma2_rn(q0, nm, v), rr, q0);
                const float2 key = lut_key2(x), fk = fine_key2(x);
                const float2 vv = unit ? x : v;
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    const float xh = h ? x.y : x.x, vh = h ? vv.y : vv.x;
                    const uint2 ent = lut_probe(h ? key.y : key.x, lut_base);
                    const uint2 lv = ld_shared_v2(ent.y + ((xh >= __uint_as_float(ent.x)) ? 256u : 0u) + lv_base);
                    e += fabsf(fmaf(-scale, __uint_as_float(lv.x), vh));
                    slot_add_at<COUNT>(__float_as_uint(h ? fk.y : fk.x) * 4u + slot_base + lv.y, a);
                }
            }
        } else if (ok) {
            e = mae1_row_slow<COUNT>(raw, m, a, unit, &S, s_lo);
        }
        err += (double)e;
    };

    bool ok_a, ok_b;
    int64_t g = blockIdx.x;
    const int64_t GS = gridDim.x;
    Raw32 ra = fetch(g, ok_a), rb;
    if (g < total_rows) {
        while (true) {
            rb = fetch(g + GS, ok_b);
            row(ra, ok_a);
            g += GS;
            if (g >= total_rows) break;
            ra = fetch(g + GS, ok_a);
            row(rb, ok_b);
            g += GS;
            if (g >= total_rows) break;
        }
    }
    __syncthreads();
    for (int k = tid; k < kFineSlots; k += kMaeThreads) {
        const unsigned long long wsum = ((unsigned long long)s_lo[kFineSlots + k] << 32) + s_lo[k];
        if (wsum) atomicAdd(&W.hist[k], wsum);
        if (COUNT && s_lo[2 * kFineSlots + k]) atomicAdd(&W.chist[k], (unsigned long long)s_lo[2 * kFineSlots + k]);
    }
#pragma unroll
    for (int off = 16; off; off >>= 1) err += __shfl_xor_sync(kFull, err, off);
    if (lane == 0) S.err[warp] = err;
    __syncthreads();
    if (tid == 0) {
        double t = 0.0;
        for (int k = 0; k < kMaeThreads / 32; ++k) t += S.err[k];
        double* rec = W.partials + (size_t)blockIdx.x * kEmRecordDoubles;
        rec[0] = T.accumulate ? rec[0] + t : t;
    }
}

// Selection after the bf16 first pass: one CTA per level walks the level's slots in ascending
// order of x (thread t owns a run of consecutive fine bins), finds the fine bin in which the
// cumulative weight reaches half of the region's total, and turns it into the key range of the
// later passes: base = key of the smallest candidate, top = bits of the range.  Also records the
// region's total weight and member count and clears the slots it read.  For a degenerate
// codebook it performs the generic first selection on the per-region bins instead.
__global__ void __launch_bounds__(1024)
mae_select1_kernel(const float* __restrict__ levels, MaeWs W)
{
    __shared__ float s_xi[kLevels], s_lv[kLevels];
    __shared__ unsigned long long s_wsum[32], s_csum[32];
    __shared__ PickResult s_res;
    __shared__ int s_pick;
    __shared__ unsigned long long s_excl;
    MaeState* S = W.state;
    const int l = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    make_thresholds(levels, s_xi, s_lv, tid);
    if (tid == 0) s_pick = -1;
    __syncthreads();
    const int top0 = S->top[l];  // from the set-up kernel: bits of the region's key range, 0 for a level that does not take part
    if (degenerate_codebook(s_xi)) {
        unsigned long long mine = 0ull, c = 0ull;
        if (tid < kMaeBins) {
            mine = __ldcg(&W.hist[l * kMaeBins + tid]);
            W.hist[l * kMaeBins + tid] = 0ull;
            c = __ldcg(&W.chist[l * kMaeBins + tid]);
            W.chist[l * kMaeBins + tid] = 0ull;
        }
#pragma unroll
        for (int off = 16; off; off >>= 1) c += __shfl_xor_sync(kFull, c, off);
        if (lane == 0) s_csum[warp] = c;
        unsigned long long all;
        const PickResult r = pick_bin<1024>(mine, 0ull, 0ull, true, s_wsum, &s_res, &all);
        if (tid == 0) {
            unsigned long long count = 0ull;
            for (int k = 0; k < 32; ++k) count += s_csum[k];
            S->total[l] = all;
            S->count[l] = count;
            if (top0 > 0) {
                const int sh = max(top0 - kMaeDigitBits, 0);
                S->before[l] = r.excl;
                S->prefix[l] = (uint32_t)r.bin;
                S->top[l] = sh;
            }
        }
        return;
    }
    // the region's closed range of fine bins
    const float lo_x = (l == 0) ? -1.0f : fminf(fmaxf(s_xi[l - 1], -1.0f), 1.0f);
    const float hi_x = (l == kLevels - 1) ? 1.0f : fminf(fmaxf(s_xi[l], -1.0f), 1.0f);
    const int f_lo = fine_bin(lo_x), f_hi = fine_bin(hi_x);
    const int span = f_hi - f_lo + 1, per = (span + 1023) / 1024;  // at most 5 bins per thread
    const int half = (l & 1) * kFineStride;
    unsigned long long mine = 0ull, cmine = 0ull;
    unsigned long long vals[5];
#pragma unroll
    for (int q = 0; q < 5; ++q) {
        const int f = f_lo + tid * per + q;
        unsigned long long v = 0ull;
        if (q < per && f <= f_hi) {
            v = __ldcg(&W.hist[half + f]);
            W.hist[half + f] = 0ull;
            cmine += __ldcg(&W.chist[half + f]);
            W.chist[half + f] = 0ull;
        }
        vals[q] = v;
        mine += v;
    }
    unsigned long long incl = mine;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const unsigned long long t = __shfl_up_sync(kFull, incl, off);
        if (lane >= off) incl += t;
    }
    unsigned long long csum = cmine;
#pragma unroll
    for (int off = 16; off; off >>= 1) csum += __shfl_xor_sync(kFull, csum, off);
    if (lane == 31) s_wsum[warp] = incl;
    if (lane == 0) s_csum[warp] = csum;
    __syncthreads();
    unsigned long long carry = 0ull, total = 0ull, count = 0ull;
    for (int k = 0; k < 32; ++k) {
        if (k < warp) carry += s_wsum[k];
        total += s_wsum[k];
        count += s_csum[k];
    }
    incl += carry;
    const unsigned long long excl = incl - mine;
    if (top0 > 0 && total > 0ull && 2ull * incl >= total && 2ull * excl < total) {
        unsigned long long run = excl;  // the crossing lies in this thread's run of bins
#pragma unroll
        for (int q = 0; q < 5; ++q) {
            if (2ull * (run + vals[q]) >= total) {
                s_pick = f_lo + tid * per + q;
                s_excl = run;
                break;
            }
            run += vals[q];
        }
    }
    __syncthreads();
    if (tid == 0) {
        S->total[l] = total;
        S->count[l] = count;
        S->prefix[l] = 0u;
        S->before[l] = 0ull;
        S->top[l] = 0;
        S->base[l] = order_key(lo_x);
        if (s_pick >= 0) {
            const int f = s_pick;
            const uint32_t kmin = order_key(-1.0f), kmax = order_key(1.0f);
            // smallest x of fine bin f: start a few steps below its lower edge and walk up
            uint32_t kl = order_key(((float)(f - kFineScale) - 0.5f) * (1.0f / (float)kFineScale));
            kl = (f == 0 || kl < kmin + 4u) ? kmin : kl - 4u;
            while (kl < kmax && fine_bin(key_to_float(kl)) < f) ++kl;
            // largest x of the bin, generously (keys above it only add samples beyond the median)
            uint32_t kh = order_key(((float)(f - kFineScale) + 0.5f) * (1.0f / (float)kFineScale));
            kh = (kh > kmax - 4u) ? kmax : kh + 4u;
            // inside the region
            const uint32_t rl = order_key(lo_x), rh = order_key(hi_x);
            if (kl < rl) kl = rl;
            if (kh > rh) kh = rh;
            if (kh < kl) kh = kl;
            const uint32_t range = kh - kl;
            S->base[l] = kl;
            S->limit[l] = range;
            S->before[l] = s_excl;
            S->top[l] = range ? 32 - __clz(range) : 0;  // key bits still unresolved
        }
    }
}

// ---------------------------------------------------------------- short last blocks
//
// The short last blocks of ragged tensors take part in every data pass through one small CTA
// that is enqueued before the pass's streaming kernel and adds to the same global histograms,
// candidate lists and error records (integer sums: the order of the additions does not
// matter).  mode selects what the pass needs of them.
enum : int {
    kTailAbsmax = 0,     // largest |w| (fixed-point reference of the weights)
    kTailFirst = 1,      // first pass, per-region digit bins (fp32 weights)
    kTailFirstFine = 2,  // first pass, uniform fine grid (bf16 weights)
    kTailLater = 3       // later passes
};

template <class DT, bool SIGNED>
__global__ void __launch_bounds__(kEmTailThreads)
mae_tail_kernel(const EmTails Q, const float* __restrict__ levels, MaeWs W, int mode, int count, int collect,
                int record)
{
    __shared__ float s_w[4096];
    __shared__ float s_xi[kLevels], s_lv[kLevels];
    __shared__ unsigned long long s_red[kEmTailThreads / 32];
    __shared__ double s_err[kEmTailThreads / 32];
    MaeState* S = W.state;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (mode == kTailAbsmax) {
        uint32_t b = 0u;
        for (int q = 0; q < Q.count; ++q)
            for (int i = tid; i < Q.len[q]; i += kEmTailThreads)
                b = max(b, __float_as_uint(fmaxf(0.0f, fabsf(short_block_elem<DT>(Q.ptr[q], i)))));  // fmaxf drops a NaN
#pragma unroll
        for (int off = 16; off; off >>= 1) b = max(b, __shfl_xor_sync(kFull, b, off));
        if (lane == 0 && b) atomicMax(&S->max_bits, b);
        return;
    }
    if (mode == kTailLater) {  // nothing left to resolve: uniform over the CTA
        int any = 0;
        for (int l = 0; l < kLevels; ++l) any |= S->top[l];
        if (any <= 0) return;
    }
    make_thresholds(levels, s_xi, s_lv, tid);
    __syncthreads();
    const bool fine = mode == kTailFirstFine && !degenerate_codebook(s_xi);
    const uint32_t max_bits = S->max_bits;
    double err = 0.0;
    for (int q = 0; q < Q.count; ++q) {
        const int len = Q.len[q];
        const float m = load_short_block<DT, SIGNED>(Q.ptr[q], len, s_w, s_red);
        const uint32_t a = Q.unit ? 1u : fixed_weight(m, max_bits);
        for (int i = tid; i < len; i += kEmTailThreads) {
            const float w = s_w[i], x = normalise(w, m);
            const int c = region_of(x, s_xi);
            const uint32_t rel = order_key(x) - S->base[c];
            const int top = S->top[c];
            const int sh = max(top - kMaeDigitBits, 0);
            if (mode == kTailLater) {
                const uint32_t mask = (1u << (top - sh)) - 1u;
                if (!(top > 0 && (uint32_t)((unsigned long long)rel >> top) == S->prefix[c] && rel <= S->limit[c])) continue;
                atomicAdd(&W.hist[c * kMaeBins + ((rel >> sh) & mask)], (unsigned long long)a);
                if (collect) {
                    const uint32_t gslot = atomicAdd(&S->cand_count[c], 1u);
                    if (gslot < W.cand_cap) W.cand[(size_t)c * W.cand_cap + gslot] = make_uint2(rel, a);
                }
                continue;
            }
            err += (double)(Q.unit ? fabsf(x - s_lv[c]) : fabsf(fmaf(-m, s_lv[c], w)));
            int slot = -1;
            if (fine) {
                if (x == x) slot = fine_bin(x) + (c & 1) * kFineStride;  // a NaN has no place on the grid
            } else if (mode == kTailFirstFine || top > 0) {  // per-region digit bins (degenerate codebook, fp32 weights)
                slot = c * kMaeBins + (int)((rel >> sh) & (uint32_t)(kMaeBins - 1));
            }
            if (slot >= 0) {
                atomicAdd(&W.hist[slot], (unsigned long long)a);
                if (count) atomicAdd(&W.chist[slot], 1ull);
            }
        }
        __syncthreads();  // before the next block overwrites s_w
    }
    if (mode == kTailLater) return;
#pragma unroll
    for (int off = 16; off; off >>= 1) err += __shfl_xor_sync(kFull, err, off);
    if (lane == 0) s_err[warp] = err;
    __syncthreads();
    if (tid == 0) {
        double t = 0.0;
        for (int k = 0; k < kEmTailThreads / 32; ++k) t += s_err[k];
        double* rec = W.partials + (size_t)record * kEmRecordDoubles;
        rec[0] = Q.accumulate ? rec[0] + t : t;
    }
}

// ---------------------------------------------------------------- level update

__global__ void __launch_bounds__(256)
mae_finalize_kernel(MaeWs W, const MaeFinal F)
{
    __shared__ double s_part[8];
    finalize_body(W, F, s_part);
}

// ================================================================= host side

namespace {

template <class DT, int I, bool SG>
int launch_pass(const EmTensors& T, const float* d_levels, const MaeWs& W, int pass, bool collect,
                bool count, const MaeFinal* tail, cudaStream_t st)
{
    const MaeFinal F = tail ? *tail : MaeFinal{};
#define BOF4_MAE_GO(FIRST_, COUNT_, COLLECT_, TAIL_)                                                    \
    {                                                                                                   \
        constexpr auto kern = mae_pass_kernel<DT, I, SG, FIRST_, COUNT_, COLLECT_, TAIL_>;              \
        if (const int rc_ = ensure_dynamic_smem<kern>((int)kMaeSmem)) return rc_;                       \
        kern<<<kEmGrid, kMaeThreads, kMaeSmem, st>>>(T, d_levels, W, F);                                \
    }
    if (pass == 0 && count) BOF4_MAE_GO(true, true, false, false)
    else if (pass == 0) BOF4_MAE_GO(true, false, false, false)
    else if (collect) BOF4_MAE_GO(false, false, true, false)
    else if (tail) BOF4_MAE_GO(false, false, false, true)
    else BOF4_MAE_GO(false, false, false, false)
#undef BOF4_MAE_GO
    BOF4_CUDA_TRY(cudaGetLastError());
    return BOF4_OK;
}

template <int I, bool SG>
int launch_pass1_32(const EmTensors& T, const float* d_levels, const MaeWs& W, bool count, cudaStream_t st)
{
    if (count) {
        constexpr auto kern = mae_pass1_32_kernel<I, SG, true>;
        if (const int rc = ensure_dynamic_smem<kern>((int)kMae1Smem(true))) return rc;
        kern<<<kEmGrid, kMaeThreads, kMae1Smem(true), st>>>(T, d_levels, W);
    } else {
        constexpr auto kern = mae_pass1_32_kernel<I, SG, false>;
        if (const int rc = ensure_dynamic_smem<kern>((int)kMae1Smem(false))) return rc;
        kern<<<kEmGrid, kMaeThreads, kMae1Smem(false), st>>>(T, d_levels, W);
    }
    BOF4_CUDA_TRY(cudaGetLastError());
    return BOF4_OK;
}

template <int I, bool SG>
int launch_later32(const EmTensors& T, const float* d_levels, const MaeWs& W, bool collect, const MaeFinal* tail,
                   cudaStream_t st)
{
    const MaeFinal F = tail ? *tail : MaeFinal{};
#define BOF4_MAE_L32(COLLECT_, TAIL_)                                                           \
    {                                                                                           \
        constexpr auto kern = mae_later32_kernel<I, SG, COLLECT_, TAIL_>;                       \
        if (const int rc_ = ensure_dynamic_smem<kern>((int)kMaeSmem)) return rc_;               \
        kern<<<kEmGrid, kMaeThreads, kMaeSmem, st>>>(T, d_levels, W, F);                        \
    }
    if (collect) BOF4_MAE_L32(true, false)
    else if (tail) BOF4_MAE_L32(false, true)
    else BOF4_MAE_L32(false, false)
#undef BOF4_MAE_L32
    BOF4_CUDA_TRY(cudaGetLastError());
    return BOF4_OK;
}

int dispatch_later32(const EmArgs& a, const EmTensors& T, const float* d_levels, const MaeWs& W, bool collect,
                     const MaeFinal* tail, cudaStream_t st)
{
    const bool sg = a.norm == BOF4_NORM_SIGNED;
#define BOF4_MAEL_I(I_) return sg ? launch_later32<I_, true>(T, d_levels, W, collect, tail, st) \
                                  : launch_later32<I_, false>(T, d_levels, W, collect, tail, st);
    switch (a.block_size) {
        case 32: BOF4_MAEL_I(32)
        case 64: BOF4_MAEL_I(64)
        case 128: BOF4_MAEL_I(128)
        case 256: BOF4_MAEL_I(256)
        case 512: BOF4_MAEL_I(512)
        case 1024: BOF4_MAEL_I(1024)
        case 2048: BOF4_MAEL_I(2048)
        default: BOF4_MAEL_I(4096)
    }
#undef BOF4_MAEL_I
}

int dispatch_pass1_32(const EmArgs& a, const EmTensors& T, const float* d_levels, const MaeWs& W, bool count,
                      cudaStream_t st)
{
    const bool sg = a.norm == BOF4_NORM_SIGNED;
#define BOF4_MAE1_I(I_) return sg ? launch_pass1_32<I_, true>(T, d_levels, W, count, st) \
                                  : launch_pass1_32<I_, false>(T, d_levels, W, count, st);
    switch (a.block_size) {
        case 32: BOF4_MAE1_I(32)
        case 64: BOF4_MAE1_I(64)
        case 128: BOF4_MAE1_I(128)
        case 256: BOF4_MAE1_I(256)
        case 512: BOF4_MAE1_I(512)
        case 1024: BOF4_MAE1_I(1024)
        case 2048: BOF4_MAE1_I(2048)
        default: BOF4_MAE1_I(4096)
    }
#undef BOF4_MAE1_I
}

int dispatch_pass(const EmArgs& a, const EmTensors& T, const float* d_levels, const MaeWs& W, int pass,
                  bool collect, bool count, const MaeFinal* tail, cudaStream_t st)
{
    const bool sg = a.norm == BOF4_NORM_SIGNED;
#define BOF4_MAE_I(DT_, I_)                                                             \
    return sg ? launch_pass<DT_, I_, true>(T, d_levels, W, pass, collect, count, tail, st)   \
              : launch_pass<DT_, I_, false>(T, d_levels, W, pass, collect, count, tail, st);
#define BOF4_MAE_DT(DT_)                         \
    switch (a.block_size) {                      \
        case 32: BOF4_MAE_I(DT_, 32)             \
        case 64: BOF4_MAE_I(DT_, 64)             \
        case 128: BOF4_MAE_I(DT_, 128)           \
        case 256: BOF4_MAE_I(DT_, 256)           \
        case 512: BOF4_MAE_I(DT_, 512)           \
        case 1024: BOF4_MAE_I(DT_, 1024)         \
        case 2048: BOF4_MAE_I(DT_, 2048)         \
        default: BOF4_MAE_I(DT_, 4096)           \
    }
    if (a.w_dtype == BOF4_F32) { BOF4_MAE_DT(F32) } else { BOF4_MAE_DT(BF16) }
#undef BOF4_MAE_DT
#undef BOF4_MAE_I
}

}  // namespace

namespace {
// The short last blocks' part of a pass (see mae_tail_kernel).
int enqueue_tails(const EmArgs& a, const float* d_levels, const MaeWs& W, int mode, bool count, bool collect,
                  cudaStream_t st)
{
    const bool sg = a.norm == BOF4_NORM_SIGNED;
    return for_each_tail_chunk(a, [&](const EmTails& Q) -> int {
        if (a.w_dtype == BOF4_F32) {
            if (sg) mae_tail_kernel<F32, true><<<1, kEmTailThreads, 0, st>>>(Q, d_levels, W, mode, count, collect, kEmGrid);
            else mae_tail_kernel<F32, false><<<1, kEmTailThreads, 0, st>>>(Q, d_levels, W, mode, count, collect, kEmGrid);
        } else {
            if (sg) mae_tail_kernel<BF16, true><<<1, kEmTailThreads, 0, st>>>(Q, d_levels, W, mode, count, collect, kEmGrid);
            else mae_tail_kernel<BF16, false><<<1, kEmTailThreads, 0, st>>>(Q, d_levels, W, mode, count, collect, kEmGrid);
        }
        BOF4_CUDA_TRY(cudaGetLastError());
        return BOF4_OK;
    });
}
}  // namespace

int mae_prepare(const EmArgs& a, void* d_ws, size_t ws_bytes, cudaStream_t st)
{
    const MaeWs W = mae_ws(d_ws, ws_bytes);
    BOF4_CUDA_TRY(cudaMemsetAsync(W.state, 0, sizeof(MaeState), st));
    if (const int rc = enqueue_tails(a, nullptr, W, kTailAbsmax, false, false, st)) return rc;
    auto fire = [&](const EmTensors& T) -> int {
        if (a.w_dtype == BOF4_F32)
            mae_absmax_kernel<F32><<<kEmGrid, kMaeThreads, 0, st>>>(T, W.state);
        else
            mae_absmax_kernel<BF16><<<kEmGrid, kMaeThreads, 0, st>>>(T, W.state);
        BOF4_CUDA_TRY(cudaGetLastError());
        return BOF4_OK;
    };
    int calls = 0;
    return for_each_tensor_chunk(a, kMaeRow, fire, &calls);
}

int mae_iteration(const EmArgs& a, const float* d_levels_in, float* d_levels_out, uint32_t skip_mask,
                  bof4_em_stats* d_stats, double* d_err_slot, void* d_ws, size_t ws_bytes, cudaStream_t st)
{
    const MaeWs W = mae_ws(d_ws, ws_bytes);
    mae_init_kernel<<<1, kMaeBins, 0, st>>>(d_levels_in, skip_mask, W);
    BOF4_CUDA_TRY(cudaGetLastError());
    // The candidate lists are filled by the first pass after which a region's candidates
    // (about 1/512 of them survive each digit) are expected to fit: the second pass up to
    // 2^29 weights, the third beyond.
    // (The bf16 first pass narrows a region to one of its 140 ... 400 fine bins rather than to one
    // of 512 digit bins; a list that overflows all the same is finished by the later passes.)
    const bool bf16 = a.w_dtype == BOF4_BF16;
    // fp32 first pass: one of 512 digit bins per region; bf16: one of its 140 ... 400 fine bins.
    const int64_t expected = bf16 ? a.n_total / 1024 : a.n_total / kLevels / kMaeBins * 8;
    const int collect_pass = (expected <= (int64_t)W.cand_cap) ? 1 : 2;
    MaeFinal fin{};
    const bool tails = has_tails(a);
    fin.n_records = kEmGrid + (tails ? 1 : 0);
    fin.n_total = a.n_total;
    fin.levels_in = d_levels_in;
    fin.levels_out = d_levels_out;
    fin.skip_mask = skip_mask;
    fin.stats = d_stats;
    fin.err_slot = d_err_slot;
    fin.unit = a.metric >= 2 ? 1 : 0;
    bool updated = false;
    for (int p = 0; p < kMaeMaxPasses; ++p) {
        const bool first = p == 0;
        // From the third pass on (they usually find nothing left to do) the selection and, in the
        // last pass, the level update ride in the pass kernel itself.
        const bool fused = p >= 2 && p != collect_pass;
        fin.enabled = (fused && p == kMaeMaxPasses - 1) ? 1 : 0;
        const bool first32 = first && bf16;  // bf16 weights: first pass on the uniform grid
        auto fire = [&](const EmTensors& T) -> int {
            if (first32) return dispatch_pass1_32(a, T, d_levels_in, W, d_stats != nullptr, st);
            if (bf16) return dispatch_later32(a, T, d_levels_in, W, p == collect_pass, fused ? &fin : nullptr, st);
            return dispatch_pass(a, T, d_levels_in, W, p, p == collect_pass, first && d_stats != nullptr,
                                 fused ? &fin : nullptr, st);
        };
        if (first && !has_whole_blocks(a)) BOF4_CUDA_TRY(cudaMemsetAsync(W.partials, 0, kEmPartialBytes, st));
        if (tails) {
            const int mode = first ? (bf16 ? kTailFirstFine : kTailFirst) : kTailLater;
            if (const int rc = enqueue_tails(a, d_levels_in, W, mode, first && d_stats != nullptr, p == collect_pass, st))
                return rc;
        }
        int calls = 0;
        const int rc = for_each_tensor_chunk(a, bf16 ? kMaeThreads * kLW : kMaeRow, fire, &calls);
        if (rc) return rc;
        if (first32) {
            mae_select1_kernel<<<kLevels, 1024, 0, st>>>(d_levels_in, W);
            BOF4_CUDA_TRY(cudaGetLastError());
            continue;
        }
        if (fused && calls > 0) {
            updated = fin.enabled != 0;
            continue;
        }
        if (p == collect_pass)
            mae_resolve_kernel<<<kLevels * kResolveCtas, kMaeThreads, 0, st>>>(W);
        else
            mae_select_kernel<<<kLevels, kMaeBins, 0, st>>>(W, first ? 1 : 0);
        BOF4_CUDA_TRY(cudaGetLastError());
    }
    if (!updated) {
        fin.enabled = 1;
        mae_finalize_kernel<<<1, 256, 0, st>>>(W, fin);
        BOF4_CUDA_TRY(cudaGetLastError());
    }
    return BOF4_OK;
}

}  // namespace bof4
