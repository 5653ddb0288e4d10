// Data-driven EM / Lloyd codebook fit (Sec. 3.2, App. B.3): one streaming pass per iteration.
//
// MSE pass (Eq. 6): every lane owns 16 consecutive weights, a block is a group of I/16 lanes.
// Per weight: x = w / m, region c by the one-probe table search, then
//     s1[c] += m^2 x,   s0[c] += m^2            (one packed read-modify-write)
// and, per lane, w2 += w^2.  The error of App. B.3 follows in the combine step from
//     sum (w - m xhat[c])^2 = w2 - sum_l xhat[l] (2 s1[l] - xhat[l] s0[l]),
// evaluated in fp64.  The level-indexed sums live in shared memory as one private column per
// thread (no atomics, no bank conflicts: the bank is the lane), are folded into fp64 per-CTA
// totals in a fixed order, written as one partial record per CTA, and combined by a single-CTA
// kernel that also updates the free levels.  Nothing depends on scheduling, so results are
// bit-reproducible.  The COUNT variant also keeps the member count of every region.
#include "common.cuh"
#include "em_common.cuh"
#include "lane32.cuh"
#include "layout.h"

namespace bof4 {

constexpr int kEmFlushIters = 64;  // loop iterations (16 weights per lane each) between fp32 -> fp64 folds

// Both variants run 1024 threads per CTA, one CTA per SM.  The COUNT variant also keeps a 16-bit
// member counter per level and thread (folded before it can overflow) and, to make room for it,
// shares each table column between two lanes.
template <bool COUNT>
struct EmGeo {
    static constexpr int threads = 1024;
    static constexpr int row = threads * kLaneW;            // weights per CTA row
    static constexpr uint32_t acc_row_bytes = threads * 8;  // one level's float2 columns
    static constexpr int lut_rep = COUNT ? 16 : 32;
    static constexpr size_t smem =
        (size_t)lut_bytes(lut_rep) + (size_t)kLevels * threads * (COUNT ? 10 : 8);
};
static_assert(kEmFlushIters * kLaneW < 65536, "16-bit member counters must not overflow between folds");

// Record layout in doubles: [0,16) s1, [16,32) s0, [32,48) count (uint64 bits), [48] sum w^2.
constexpr int kRecS1 = 0, kRecS0 = 16, kRecCnt = 32, kRecW2 = 48;

// What the last accumulation CTA (or the stand-alone combine kernel) does with the records.
//   stats    != NULL: receives the combined record
//   codebook != NULL: every free level with s0 > 0 becomes (float)(s1 / s0)      (Eq. 6)
//   err_slot != NULL: receives err_sum / n_total
// err_sum = w2 - sum_l xhat[l] (2 s1[l] - xhat[l] s0[l]) with the levels that produced the sums.
struct MseTail {
    int enabled;            // the last CTA to arrive combines the records (fused M step)
    int n_records;
    int64_t n_total;
    const float* levels_in;
    bof4_em_stats* stats;
    float* codebook;
    uint32_t fixed_mask;
    double* err_slot;
    unsigned int* ticket;   // arrival counter, zero before the pass and reset by the last CTA
};

// Combines the per-CTA records in a fixed order (the order does not depend on which CTA runs
// this) and performs the M step.  Called by all threads of one CTA.
__device__ __forceinline__ void mse_combine(const double* partials, const MseTail& t, double* s_q,
                                            double* s_corr, unsigned long long* s_stage)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    constexpr int NQ = kRecW2 + 1;            // quantities per record
    constexpr int PER = (kEmRecords + 31) / 32;  // records per lane
    // Stage all records in shared memory first: coalesced, independent loads (every thread has
    // several in flight), instead of a chain of dependent L2 round trips per quantity.
    const int total = t.n_records * NQ;
    for (int i0 = 0; i0 < total; i0 += 8 * (int)blockDim.x) {
        unsigned long long raw[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const int i = i0 + u * (int)blockDim.x + (int)threadIdx.x;
            raw[u] = (i < total) ? __ldcg(reinterpret_cast<const unsigned long long*>(partials) +
                                          (size_t)(i / NQ) * kEmRecordDoubles + (i % NQ))
                                 : 0ull;
        }
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const int i = i0 + u * (int)blockDim.x + (int)threadIdx.x;
            if (i < total) s_stage[i] = raw[u];
        }
    }
    __syncthreads();
    for (int q = warp; q < NQ; q += nwarps) {
        const bool is_count = q >= kRecCnt && q < kRecW2;
        double a = 0.0;
        unsigned long long c = 0;
#pragma unroll
        for (int k = 0; k < PER; ++k) {  // fixed order: lane-strided, then the butterfly
            const int r = lane + 32 * k;
            const unsigned long long raw = (r < t.n_records) ? s_stage[r * NQ + q] : 0ull;  // zero bits = +0.0
            if (is_count)
                c += raw;
            else
                a += __longlong_as_double((long long)raw);
        }
#pragma unroll
        for (int off = 16; off; off >>= 1) {
            a += __shfl_xor_sync(kFull, a, off);
            c += __shfl_xor_sync(kFull, c, off);
        }
        if (lane == 0) {
            if (is_count)
                reinterpret_cast<unsigned long long*>(s_q)[q] = c;
            else
                s_q[q] = a;
        }
    }
    __syncthreads();
    if (threadIdx.x < kLevels) {
        const int l = threadIdx.x;
        const double s1 = s_q[kRecS1 + l], s0 = s_q[kRecS0 + l];
        const float old = t.levels_in[l];
        const float cen = (s0 > 0.0) ? (float)(s1 / s0) : old;
        s_corr[l] = (double)old * (2.0 * s1 - (double)old * s0);
        if (t.stats) {
            t.stats->s1[l] = s1;
            t.stats->s0[l] = s0;
            t.stats->count[l] = reinterpret_cast<unsigned long long*>(s_q)[kRecCnt + l];
            t.stats->median[l] = cen;
        }
        if (t.codebook && !((t.fixed_mask >> l) & 1u)) t.codebook[l] = cen;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        double corr = 0.0;
        for (int l = 0; l < kLevels; ++l) corr += s_corr[l];
        double err = s_q[kRecW2] - corr;
        if (err < 0.0) err = 0.0;
        if (t.stats) {
            t.stats->err_sum = err;
            t.stats->n_total = t.n_total;
        }
        if (t.err_slot) *t.err_slot = (t.n_total > 0) ? err / (double)t.n_total : 0.0;
    }
}

// Stand-alone combine, used when a pass launched no accumulation kernel at all: the records are
// all zero then and one of them stands for the sum.
__global__ void __launch_bounds__(1024)
em_mse_finalize_kernel(const double* partials, const MseTail t)
{
    __shared__ double s_q[kRecW2 + 1], s_corr[kLevels];
    __shared__ unsigned long long s_stage[kRecW2 + 1];  // the launcher passes a single (zero) record
    mse_combine(partials, t, s_q, s_corr, s_stage);
}

// M step from E-step records that were produced by separate calls (one per GPU of a joint fit,
// gathered in rank order): sums them in index order in fp64 and updates the free levels (Eq. 6).
// One warp; lane l owns level l.
__global__ void __launch_bounds__(32)
m_step_kernel(const bof4_em_stats* __restrict__ stats, int n_records, float* __restrict__ codebook,
              uint32_t fixed_mask, double* __restrict__ err_slot, bof4_em_stats* __restrict__ total)
{
    const int l = threadIdx.x;
    double s1 = 0.0, s0 = 0.0, err = 0.0;
    unsigned long long cnt = 0ull;
    long long n = 0;
    for (int r = 0; r < n_records; ++r) {
        if (l < kLevels) {
            s1 += stats[r].s1[l];
            s0 += stats[r].s0[l];
            cnt += stats[r].count[l];
        }
        err += stats[r].err_sum;
        n += stats[r].n_total;
    }
    if (l < kLevels) {
        const float old = codebook[l];
        const float cen = (s0 > 0.0) ? (float)(s1 / s0) : old;
        if (total) {
            total->s1[l] = s1;
            total->s0[l] = s0;
            total->count[l] = cnt;
            total->median[l] = cen;
        }
        if (!((fixed_mask >> l) & 1u)) codebook[l] = cen;
    }
    if (l == 0) {
        if (total) {
            total->err_sum = err;
            total->n_total = n;
        }
        if (err_slot) *err_slot = (n > 0) ? err / (double)n : 0.0;
    }
}

// The short last blocks of ragged tensors: one CTA, block after block.  Warp l sums the members
// of region l (lane-strided, then the butterfly: a fixed order), in fp64 throughout, and the
// result goes to a record of its own.
template <class DT, bool SIGNED>
__global__ void __launch_bounds__(kEmTailThreads)
em_mse_tail_kernel(const EmTails Q, const float* __restrict__ levels, double* __restrict__ rec)
{
    __shared__ float s_w[4096], s_x[4096];
    __shared__ unsigned char s_c[4096];
    __shared__ float s_xi[kLevels], s_lv[kLevels];
    __shared__ unsigned long long s_red[kEmTailThreads / 32];
    __shared__ double s_w2[kLevels];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    static_assert(kEmTailThreads / 32 == kLevels, "one warp per level");
    make_thresholds(levels, s_xi, s_lv, tid);
    double a1 = 0.0, a0 = 0.0, aw = 0.0;
    unsigned long long cnt = 0ull;
    for (int q = 0; q < Q.count; ++q) {
        const int len = Q.len[q];
        const float m = load_short_block<DT, SIGNED>(Q.ptr[q], len, s_w, s_red);  // orders s_xi as well
        for (int i = tid; i < len; i += kEmTailThreads) {
            const float x = normalise(s_w[i], m);
            s_x[i] = x;
            s_c[i] = (unsigned char)region_of(x, s_xi);
        }
        __syncthreads();
        const double md = (double)m, m2 = md * md;
        for (int i = lane; i < len; i += 32) {
            if (s_c[i] != warp) continue;
            const double x = (double)s_x[i], w = (double)s_w[i];
            if (Q.unit) {  // normalised-domain variant (App. D): unit weights, error on x
                a1 += x;
                a0 += 1.0;
                aw += x * x;
            } else {
                a1 += m2 * x;
                a0 += m2;
                aw += w * w;
            }
            ++cnt;
        }
        __syncthreads();  // before the next block overwrites the arrays
    }
#pragma unroll
    for (int off = 16; off; off >>= 1) {
        a1 += __shfl_xor_sync(kFull, a1, off);
        a0 += __shfl_xor_sync(kFull, a0, off);
        aw += __shfl_xor_sync(kFull, aw, off);
        cnt += __shfl_xor_sync(kFull, cnt, off);
    }
    if (lane == 0) {
        unsigned long long* rc = reinterpret_cast<unsigned long long*>(rec);
        if (Q.accumulate) {
            rec[kRecS1 + warp] += a1;
            rec[kRecS0 + warp] += a0;
            rc[kRecCnt + warp] += cnt;
        } else {
            rec[kRecS1 + warp] = a1;
            rec[kRecS0 + warp] = a0;
            rc[kRecCnt + warp] = cnt;
        }
        s_w2[warp] = aw;
    }
    __syncthreads();
    if (tid == 0) {
        double e = 0.0;
        for (int l = 0; l < kLevels; ++l) e += s_w2[l];
        rec[kRecW2] = Q.accumulate ? rec[kRecW2] + e : e;
    }
}

template <class DT, int I, bool SIGNED, bool COUNT>
__global__ void __launch_bounds__(EmGeo<COUNT>::threads, 1)
em_mse_kernel(const EmTensors T, const float* levels, double* partials, const MseTail tail)
{
    using G = EmGeo<COUNT>;
    constexpr int NT = G::threads, NW = NT / 32, NSEG = NW / kLevels;
    extern __shared__ __align__(16) unsigned char s_raw[];
    unsigned char* s_lut = s_raw;
    unsigned char* s_acc = s_raw + lut_bytes(G::lut_rep);               // float2 [16][NT]
    unsigned char* s_cnt = s_acc + (size_t)kLevels * G::acc_row_bytes;  // uint16 [16][NT] (COUNT)
    __shared__ float s_xi[kLevels], s_lv[kLevels];
    __shared__ int s_multi;
    __shared__ WideScratch s_wide;
    __shared__ double s_part[NSEG][3][kLevels];
    __shared__ double s_tot[3 * kLevels];  // s1, s0, count (as uint64 bits)
    __shared__ double s_w2[NW];
    __shared__ const void* s_ptr[kEmMaxTensors];
    __shared__ int64_t s_n[kEmMaxTensors], s_row_end[kEmMaxTensors];

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    make_thresholds(levels, s_xi, s_lv, tid);
    if (tid < 3 * kLevels) s_tot[tid] = 0.0;  // all-zero bits are also uint64 zero
    if (tid < T.count) {
        s_ptr[tid] = T.ptr[tid];
        s_n[tid] = T.n[tid];
        s_row_end[tid] = T.row_end[tid];
    }
#pragma unroll
    for (int l = 0; l < kLevels; ++l) {
        *reinterpret_cast<float2*>(s_acc + l * G::acc_row_bytes + tid * 8) = make_float2(0.0f, 0.0f);
        if (COUNT) *reinterpret_cast<uint16_t*>(s_cnt + l * (G::acc_row_bytes / 4) + tid * 2) = 0;
    }
    __syncthreads();
    build_lut<G::lut_rep>(s_xi, s_lut, &s_multi, [](int base) { return (uint32_t)base * G::acc_row_bytes; });
    __syncthreads();
    const bool lut_ok = s_multi == 0;

    const int64_t total_rows = T.row_end[T.count - 1];
    const bool unit = T.unit != 0;
    const uint32_t lut_base = lut_lane_base<G::lut_rep>(s_lut, lane), tid_off = tid * 8;
    double w2sum = 0.0;
    int t_cur = 0;
    int since_flush = 0;

    // Folds the private fp32 columns into the fp64 CTA totals (fixed order) and clears them.
    auto flush = [&]() {
        __syncthreads();
        {
            const int l = warp & (kLevels - 1), seg = warp >> 4;
            double a1 = 0.0, a0 = 0.0;
            unsigned long long ac = 0;
            constexpr int PER = NT / NSEG / 32;  // columns per lane
#pragma unroll 4
            for (int k = 0; k < PER; ++k) {
                const int col = seg * (NT / NSEG) + k * 32 + lane;
                float2* pa = reinterpret_cast<float2*>(s_acc + l * G::acc_row_bytes + col * 8);
                const float2 a = *pa;
                a1 += (double)a.x;
                a0 += (double)a.y;
                *pa = make_float2(0.0f, 0.0f);
                if (COUNT) {
                    uint16_t* pc = reinterpret_cast<uint16_t*>(s_cnt + l * (G::acc_row_bytes / 4) + col * 2);
                    ac += *pc;
                    *pc = 0;
                }
            }
#pragma unroll
            for (int off = 16; off; off >>= 1) {
                a1 += __shfl_xor_sync(kFull, a1, off);
                a0 += __shfl_xor_sync(kFull, a0, off);
                if (COUNT) ac += __shfl_xor_sync(kFull, ac, off);
            }
            if (lane == 0) {
                s_part[seg][0][l] = a1;
                s_part[seg][1][l] = a0;
                s_part[seg][2][l] = __longlong_as_double((long long)ac);
            }
        }
        __syncthreads();
        if (tid < 3 * kLevels) {
            const int q = tid / kLevels, l = tid % kLevels;
            if (q < 2) {
                double a = s_tot[tid];
                for (int sg = 0; sg < NSEG; ++sg) a += s_part[sg][q][l];
                s_tot[tid] = a;
            } else {
                unsigned long long a = (unsigned long long)__double_as_longlong(s_tot[tid]);
                for (int sg = 0; sg < NSEG; ++sg)
                    a += (unsigned long long)__double_as_longlong(s_part[sg][2][l]);
                s_tot[tid] = __longlong_as_double((long long)a);
            }
        }
        __syncthreads();
    };

    // Loads the lane's 16 weights of global row g (zeros beyond the end of the row's tensor).
    auto fetch = [&](int64_t g, bool& ok) -> RawRow<DT> {
        ok = false;
        if (g < total_rows) {
            while (g >= s_row_end[t_cur]) ++t_cur;
            const int64_t r = g - (t_cur ? s_row_end[t_cur - 1] : 0);
            const int64_t idx = (r * NT + tid) * kLaneW;
            ok = idx < s_n[t_cur];
            if (ok) return load_raw<DT>(s_ptr[t_cur], idx);
        }
        return zero_raw<DT>();
    };

    bool ok;
    RawRow<DT> raw = fetch(blockIdx.x, ok);
    for (int64_t g = blockIdx.x; g < total_rows; g += gridDim.x) {
        bool ok_next;
        const RawRow<DT> next = fetch(g + gridDim.x, ok_next);
        float v[kLaneW];
        widen(raw, v);
        float gmax;
        const float m = block_constant<I, SIGNED>(v, gmax, &s_wide);
        const bool safe = row_is_safe(gmax, ok);
        float x[kLaneW];
        normalise16<false>(v, m, safe && DT::code == BF16::code, x);
        float2 sq = make_float2(0.0f, 0.0f);
        if (unit) {  // App. D variant: the error is measured on x
#pragma unroll
            for (int k = 0; k < kLaneW / 2; ++k) {
                const float2 vv = make_float2(x[2 * k], x[2 * k + 1]);
                sq = __ffma2_rn(vv, vv, sq);
            }
        } else {
#pragma unroll
            for (int k = 0; k < kLaneW / 2; ++k) {
                const float2 vv = make_float2(v[2 * k], v[2 * k + 1]);
                sq = __ffma2_rn(vv, vv, sq);
            }
        }
        if (ok) w2sum += (double)(sq.x + sq.y);
        if (ok) {
            const float m2 = unit ? 1.0f : m * m;
            const float2 mm = make_float2(m2, m2);
            if (lut_ok && safe) {
#pragma unroll
                for (int k = 0; k < kLaneW / 2; ++k) {
                    const float2 key = lut_key2(make_float2(x[2 * k], x[2 * k + 1]));
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        const float xv = x[2 * k + h];
                        const uint2 ent = lut_probe<G::lut_rep>(h ? key.y : key.x, lut_base);
                        const uint32_t off =
                            ent.y + ((xv >= __uint_as_float(ent.x)) ? G::acc_row_bytes : 0u) + tid_off;
                        float2* pa = reinterpret_cast<float2*>(s_acc + off);
                        *pa = __ffma2_rn(mm, make_float2(xv, 1.0f), *pa);
                        if (COUNT) *reinterpret_cast<uint16_t*>(s_cnt + (off >> 2)) += 1;
                    }
                }
            } else {
#pragma unroll
                for (int k = 0; k < kLaneW; ++k) {
                    const uint32_t off = (uint32_t)region_of(x[k], s_xi) * G::acc_row_bytes + tid_off;
                    float2* pa = reinterpret_cast<float2*>(s_acc + off);
                    *pa = __ffma2_rn(mm, make_float2(x[k], 1.0f), *pa);
                    if (COUNT) *reinterpret_cast<uint16_t*>(s_cnt + (off >> 2)) += 1;
                }
            }
        }
        raw = next;
        ok = ok_next;
        if (++since_flush == kEmFlushIters) {
            flush();
            since_flush = 0;
        }
    }
    flush();

    // sum of squares: fixed-order fold over the CTA
#pragma unroll
    for (int off = 16; off; off >>= 1) w2sum += __shfl_xor_sync(kFull, w2sum, off);
    if (lane == 0) s_w2[warp] = w2sum;
    __syncthreads();
    double* rec = partials + (size_t)blockIdx.x * kEmRecordDoubles;
    if (tid < kLevels) {
        unsigned long long* rc = reinterpret_cast<unsigned long long*>(rec);
        const unsigned long long cnt = (unsigned long long)__double_as_longlong(s_tot[2 * kLevels + tid]);
        if (T.accumulate) {
            rec[kRecS1 + tid] += s_tot[tid];
            rec[kRecS0 + tid] += s_tot[kLevels + tid];
            rc[kRecCnt + tid] += cnt;
        } else {
            rec[kRecS1 + tid] = s_tot[tid];
            rec[kRecS0 + tid] = s_tot[kLevels + tid];
            rc[kRecCnt + tid] = cnt;
        }
    }
    if (tid == 0) {
        double e = 0.0;
        for (int k = 0; k < NW; ++k) e += s_w2[k];
        rec[kRecW2] = T.accumulate ? rec[kRecW2] + e : e;
    }
    // Fused M step: the CTA that arrives last (no CTA ever waits for another) combines all
    // records; the fences order every CTA's record writes before its arrival.
    if (tail.enabled) {
        __shared__ int s_last;
        __shared__ double s_q[kRecW2 + 1], s_corr[kLevels];
        __threadfence();
        __syncthreads();
        if (tid == 0) s_last = (atomicAdd(tail.ticket, 1u) == gridDim.x - 1) ? 1 : 0;
        __syncthreads();
        if (s_last) {
            __threadfence();
            // the accumulator columns are folded and no longer needed: reuse them as the staging area
            mse_combine(partials, tail, s_q, s_corr, reinterpret_cast<unsigned long long*>(s_acc));
            if (tid == 0) *tail.ticket = 0u;
        }
    }
}

// ---------------------------------------------------------------- MSE pass, bf16 weights
//
// The same pass with the 64-byte-per-lane front end (lane32.cuh): 32 weights per lane, packed
// min/max, the reciprocal FAST path (x~ = w RN(1/m); the region it falls into is the region of
// the true quotient whenever the block constant's significand is not marked "near", so member
// counts stay exact, and the sums only see the last-place difference of x~).  Rows outside the
// common case go to an out-of-line version that divides exactly.

template <bool COUNT>
struct EmGeo32 {
    static constexpr int threads = 1024;
    static constexpr int row = threads * kLW;               // weights per CTA row
    static constexpr uint32_t acc_row_bytes = threads * 8;  // one level's float2 columns
    static constexpr int lut_rep = COUNT ? 16 : 32;
    static constexpr int flush_rows = 32;                   // 1024 weights per thread between folds
    static constexpr size_t smem =
        (size_t)lut_bytes(lut_rep) + (size_t)kLevels * threads * (COUNT ? 10 : 8);
};

// s1[c] += mm x, s0[c] += mm in the thread's private column of level c (byte offset `off`).
template <bool COUNT>
__device__ __forceinline__ void em_add(unsigned char* s_acc, unsigned char* s_cnt, uint32_t off, float mm, float x)
{
    float2* pa = reinterpret_cast<float2*>(s_acc + off);
    float2 a = *pa;
    a.x = fmaf(mm, x, a.x);
    a.y += mm;
    *pa = a;
    if (COUNT) *reinterpret_cast<uint16_t*>(s_cnt + (off >> 2)) += 1;
}

// One row of a lane the slow way (true quotients, binary search against the true thresholds).
// Out of line.
template <bool COUNT>
__device__ __noinline__ float em_row32_slow(Raw32 raw, float m, float mm, bool unit, const float* s_xi,
                                            unsigned char* s_acc, unsigned char* s_cnt, uint32_t tid_off,
                                            uint32_t row_bytes)
{
    uint32_t u[16];
    words_of(raw, u);
    const bool recip = div_safe(fabsf(m));
    const float r = recip ? __frcp_rn(m) : 0.0f;
    float2 sq = make_float2(0.0f, 0.0f);
#pragma unroll 4
    for (int k = 0; k < 16; ++k) {
        const float2 v = make_float2(bf_lo(u[k]), bf_hi(u[k]));
        const float2 x = exact_quotient2(v, m, r, recip);
        sq = unit ? __ffma2_rn(x, x, sq) : __ffma2_rn(v, v, sq);
        em_add<COUNT>(s_acc, s_cnt, (uint32_t)region_of(x.x, s_xi) * row_bytes + tid_off, mm, x.x);
        em_add<COUNT>(s_acc, s_cnt, (uint32_t)region_of(x.y, s_xi) * row_bytes + tid_off, mm, x.y);
    }
    return sq.x + sq.y;
}

template <int I, bool SIGNED, bool COUNT>
__global__ void __launch_bounds__(EmGeo32<COUNT>::threads, 1)
em_mse32_kernel(const EmTensors T, const float* levels, double* partials, const MseTail tail)
{
    using G = EmGeo32<COUNT>;
    constexpr int NT = G::threads, NW = NT / 32, NSEG = NW / kLevels;
    extern __shared__ __align__(16) unsigned char s_raw[];
    unsigned char* s_lut = s_raw;
    unsigned char* s_acc = s_raw + lut_bytes(G::lut_rep);               // float2 [16][NT]
    unsigned char* s_cnt = s_acc + (size_t)kLevels * G::acc_row_bytes;  // uint16 [16][NT] (COUNT)
    __shared__ float s_xi[kLevels], s_lv[kLevels];
    __shared__ FastInfo s_info;
    __shared__ WideScratch s_wide;
    __shared__ double s_part[NSEG][3][kLevels];
    __shared__ double s_tot[3 * kLevels];  // s1, s0, count (as uint64 bits)
    __shared__ double s_w2[NW];
    __shared__ const void* s_ptr[kEmMaxTensors];
    __shared__ int64_t s_n[kEmMaxTensors], s_row_end[kEmMaxTensors];

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (tid < 3 * kLevels) s_tot[tid] = 0.0;  // all-zero bits are also uint64 zero
    if (tid < T.count) {
        s_ptr[tid] = T.ptr[tid];
        s_n[tid] = T.n[tid];
        s_row_end[tid] = T.row_end[tid];
    }
#pragma unroll
    for (int l = 0; l < kLevels; ++l) {
        *reinterpret_cast<float2*>(s_acc + l * G::acc_row_bytes + tid * 8) = make_float2(0.0f, 0.0f);
        if (COUNT) *reinterpret_cast<uint16_t*>(s_cnt + l * (G::acc_row_bytes / 4) + tid * 2) = 0;
    }
    const bool lut_ok = build_tables32<G::lut_rep>(levels, s_xi, s_lv, s_lut, &s_info,
                                                   [](int base) { return (uint32_t)base * G::acc_row_bytes; });
    const bool fast_ok = lut_ok && !s_info.tiny;

    const int64_t total_rows = T.row_end[T.count - 1];
    const bool unit = T.unit != 0;
    const uint32_t lut_base = lut_lane_base<G::lut_rep>(s_lut, lane), tid_off = tid * 8;
    double w2sum = 0.0;
    int t_cur = 0;
    int since_flush = 0;

    // Folds the private fp32 columns into the fp64 CTA totals (fixed order) and clears them.
    auto flush = [&]() {
        __syncthreads();
        {
            const int l = warp & (kLevels - 1), seg = warp >> 4;
            double a1 = 0.0, a0 = 0.0;
            unsigned long long ac = 0;
            constexpr int PER = NT / NSEG / 32;  // columns per lane
#pragma unroll 4
            for (int k = 0; k < PER; ++k) {
                const int col = seg * (NT / NSEG) + k * 32 + lane;
                float2* pa = reinterpret_cast<float2*>(s_acc + l * G::acc_row_bytes + col * 8);
                const float2 a = *pa;
                a1 += (double)a.x;
                a0 += (double)a.y;
                *pa = make_float2(0.0f, 0.0f);
                if (COUNT) {
                    uint16_t* pc = reinterpret_cast<uint16_t*>(s_cnt + l * (G::acc_row_bytes / 4) + col * 2);
                    ac += *pc;
                    *pc = 0;
                }
            }
#pragma unroll
            for (int off = 16; off; off >>= 1) {
                a1 += __shfl_xor_sync(kFull, a1, off);
                a0 += __shfl_xor_sync(kFull, a0, off);
                if (COUNT) ac += __shfl_xor_sync(kFull, ac, off);
            }
            if (lane == 0) {
                s_part[seg][0][l] = a1;
                s_part[seg][1][l] = a0;
                s_part[seg][2][l] = __longlong_as_double((long long)ac);
            }
        }
        __syncthreads();
        if (tid < 3 * kLevels) {
            const int q = tid / kLevels, l = tid % kLevels;
            if (q < 2) {
                double a = s_tot[tid];
                for (int sg = 0; sg < NSEG; ++sg) a += s_part[sg][q][l];
                s_tot[tid] = a;
            } else {
                unsigned long long a = (unsigned long long)__double_as_longlong(s_tot[tid]);
                for (int sg = 0; sg < NSEG; ++sg)
                    a += (unsigned long long)__double_as_longlong(s_part[sg][2][l]);
                s_tot[tid] = __longlong_as_double((long long)a);
            }
        }
        __syncthreads();
    };

    // Loads the lane's 32 weights of global row g (zeros beyond the end of the row's tensor or of
    // the data); rows are fetched in ascending order.
    auto fetch = [&](int64_t g, bool& ok) -> Raw32 {
        ok = false;
        if (g < total_rows) {
            while (g >= s_row_end[t_cur]) ++t_cur;
            const int64_t r = g - (t_cur ? s_row_end[t_cur - 1] : 0);
            const int64_t idx = (r * NT + tid) * kLW;
            ok = idx < s_n[t_cur];
            if (ok) return load_raw32(s_ptr[t_cur], idx);
        }
        return zero_raw32();
    };

    auto row = [&](const Raw32& raw, bool ok) {
        uint32_t u[16];
        words_of(raw, u);
        float mx, mn, g;
        lane_minmax32(u, mx, mn);
        const float m = block_constant32<I, SIGNED>(u, mx, mn, g, &s_wide);
        const float mm = unit ? 1.0f : m * m;
        float sq;
        if (row_is_fast(g, m, ok, fast_ok, &s_info)) {
            const float r = __frcp_rn(m);
            const float2 rr = make_float2(r, r);
            float2 sq2 = make_float2(0.0f, 0.0f);
#pragma unroll
            for (int k = 0; k < 16; ++k) {
                const float2 v = make_float2(bf_lo(u[k]), bf_hi(u[k]));
                const float2 x = __fmul2_rn(v, rr);
                const float2 key = lut_key2(x);
                sq2 = unit ? __ffma2_rn(x, x, sq2) : __ffma2_rn(v, v, sq2);
                const uint2 e0 = lut_probe<G::lut_rep>(key.x, lut_base), e1 = lut_probe<G::lut_rep>(key.y, lut_base);
                em_add<COUNT>(s_acc, s_cnt, e0.y + ((x.x >= __uint_as_float(e0.x)) ? G::acc_row_bytes : 0u) + tid_off, mm, x.x);
                em_add<COUNT>(s_acc, s_cnt, e1.y + ((x.y >= __uint_as_float(e1.x)) ? G::acc_row_bytes : 0u) + tid_off, mm, x.y);
            }
            sq = sq2.x + sq2.y;
        } else {
            sq = ok ? em_row32_slow<COUNT>(raw, m, mm, unit, s_xi, s_acc, s_cnt, tid_off, G::acc_row_bytes) : 0.0f;
        }
        w2sum += (double)sq;
        if (++since_flush == G::flush_rows) {
            flush();
            since_flush = 0;
        }
    };

    bool ok_a, ok_b;
    int64_t g = blockIdx.x;
    const int64_t GS = gridDim.x;
    Raw32 a = fetch(g, ok_a), b;
    if (g < total_rows) {
        while (true) {
            b = fetch(g + GS, ok_b);
            row(a, ok_a);
            g += GS;
            if (g >= total_rows) break;
            a = fetch(g + GS, ok_a);
            row(b, ok_b);
            g += GS;
            if (g >= total_rows) break;
        }
    }
    flush();

    // sum of squares: fixed-order fold over the CTA
#pragma unroll
    for (int off = 16; off; off >>= 1) w2sum += __shfl_xor_sync(kFull, w2sum, off);
    if (lane == 0) s_w2[warp] = w2sum;
    __syncthreads();
    double* rec = partials + (size_t)blockIdx.x * kEmRecordDoubles;
    if (tid < kLevels) {
        unsigned long long* rc = reinterpret_cast<unsigned long long*>(rec);
        const unsigned long long cnt = (unsigned long long)__double_as_longlong(s_tot[2 * kLevels + tid]);
        if (T.accumulate) {
            rec[kRecS1 + tid] += s_tot[tid];
            rec[kRecS0 + tid] += s_tot[kLevels + tid];
            rc[kRecCnt + tid] += cnt;
        } else {
            rec[kRecS1 + tid] = s_tot[tid];
            rec[kRecS0 + tid] = s_tot[kLevels + tid];
            rc[kRecCnt + tid] = cnt;
        }
    }
    if (tid == 0) {
        double e = 0.0;
        for (int k = 0; k < NW; ++k) e += s_w2[k];
        rec[kRecW2] = T.accumulate ? rec[kRecW2] + e : e;
    }
    if (tail.enabled) {
        __shared__ int s_last;
        __shared__ double s_q[kRecW2 + 1], s_corr[kLevels];
        __threadfence();
        __syncthreads();
        if (tid == 0) s_last = (atomicAdd(tail.ticket, 1u) == gridDim.x - 1) ? 1 : 0;
        __syncthreads();
        if (s_last) {
            __threadfence();
            mse_combine(partials, tail, s_q, s_corr, reinterpret_cast<unsigned long long*>(s_acc));
            if (tid == 0) *tail.ticket = 0u;
        }
    }
}

}  // namespace bof4

// ================================================================= launchers (C ABI)

namespace bof4 {

int check_em(const char* fn, EmArgs& a, const void* d_codebook, void* d_ws, size_t ws_bytes)
{
    if (a.n_tensors < 0 || (a.n_tensors > 0 && (!a.h_w || !a.h_n))) {
        set_error("%s: bad tensor list", fn);
        return BOF4_ERR_INVALID_ARG;
    }
    if (!valid_block_size(a.block_size)) {
        set_error("%s: block_size %d is not a power of two in 32 ... 4096", fn, a.block_size);
        return BOF4_ERR_SHAPE;
    }
    if (a.w_dtype != BOF4_F32 && a.w_dtype != BOF4_BF16) {
        set_error("%s: unknown weight dtype %d", fn, a.w_dtype);
        return BOF4_ERR_DTYPE;
    }
    if ((a.norm != BOF4_NORM_ABS && a.norm != BOF4_NORM_SIGNED) ||
        a.metric < BOF4_METRIC_MSE || a.metric > BOF4_METRIC_MAE_NORMALIZED) {
        set_error("%s: bad norm or metric", fn);
        return BOF4_ERR_INVALID_ARG;
    }
    int64_t tot = 0;
    for (int t = 0; t < a.n_tensors; ++t) {
        if (a.h_n[t] < 0 || (a.h_n[t] > 0 && !a.h_w[t])) {
            set_error("%s: tensor %d has a negative size or a NULL pointer", fn, t);
            return BOF4_ERR_INVALID_ARG;
        }
        if (a.h_n[t] > 0 && !aligned32(a.h_w[t])) {
            set_error("%s: tensor %d is not 32-byte aligned", fn, t);
            return BOF4_ERR_INVALID_ARG;
        }
        tot += a.h_n[t];
    }
    if (!d_codebook) {
        set_error("%s: NULL codebook", fn);
        return BOF4_ERR_INVALID_ARG;
    }
    if (!d_ws || ((uintptr_t)d_ws & 255u) || ws_bytes < em_workspace_bytes()) {
        set_error("%s: workspace NULL, not 256-byte aligned, or smaller than %zu bytes", fn,
                  em_workspace_bytes());
        return BOF4_ERR_WORKSPACE;
    }
    a.n_total = tot;
    return BOF4_OK;
}

}  // namespace bof4

namespace {

using namespace bof4;

template <class DT, int I, bool SG, bool COUNT>
int launch_mse_chunk(const EmTensors& T, const float* d_codebook, double* partials, MseTail tail,
                     cudaStream_t st)
{
    tail.enabled = T.last;
    if constexpr (DT::code == BOF4_BF16) {
        using G = EmGeo32<COUNT>;
        constexpr auto kern = em_mse32_kernel<I, SG, COUNT>;
        if (const int rc = ensure_dynamic_smem<kern>((int)G::smem)) return rc;
        kern<<<kEmGrid, G::threads, G::smem, st>>>(T, d_codebook, partials, tail);
    } else {
        using G = EmGeo<COUNT>;
        constexpr auto kern = em_mse_kernel<DT, I, SG, COUNT>;
        if (const int rc = ensure_dynamic_smem<kern>((int)G::smem)) return rc;
        kern<<<kEmGrid, G::threads, G::smem, st>>>(T, d_codebook, partials, tail);
    }
    BOF4_CUDA_TRY(cudaGetLastError());
    return BOF4_OK;
}

// Enqueues one MSE pass over all tensors (non-empty ones, in list order, kEmMaxTensors per
// launch); the last launch also combines the records and performs what `tail` asks for.  With
// no weights at all the records are zeroed and a stand-alone combine runs.
template <bool COUNT>
int enqueue_mse_pass(const EmArgs& a, const float* d_codebook, double* partials, MseTail tail,
                     cudaStream_t st)
{
    // Short last blocks first, into a record of their own (the only record when no tensor holds a
    // whole block).
    const bool tails = has_tails(a), whole = has_whole_blocks(a);
    if (!whole) BOF4_CUDA_TRY(cudaMemsetAsync(partials, 0, kEmPartialBytes, st));
    if (tails) {
        double* rec = partials + (size_t)(whole ? kEmGrid : 0) * kEmRecordDoubles;
        const bool sgn = a.norm == BOF4_NORM_SIGNED;
        const int rc = for_each_tail_chunk(a, [&](const EmTails& Q) -> int {
            if (a.w_dtype == BOF4_F32) {
                if (sgn) em_mse_tail_kernel<F32, true><<<1, kEmTailThreads, 0, st>>>(Q, d_codebook, rec);
                else em_mse_tail_kernel<F32, false><<<1, kEmTailThreads, 0, st>>>(Q, d_codebook, rec);
            } else {
                if (sgn) em_mse_tail_kernel<BF16, true><<<1, kEmTailThreads, 0, st>>>(Q, d_codebook, rec);
                else em_mse_tail_kernel<BF16, false><<<1, kEmTailThreads, 0, st>>>(Q, d_codebook, rec);
            }
            BOF4_CUDA_TRY(cudaGetLastError());
            return BOF4_OK;
        });
        if (rc) return rc;
    }
    tail.n_records = kEmGrid + (tails ? 1 : 0);
    tail.n_total = a.n_total;
    tail.levels_in = d_codebook;
    tail.ticket = reinterpret_cast<unsigned int*>(reinterpret_cast<char*>(partials) + kEmTicketOffset);
    const bool sg = a.norm == BOF4_NORM_SIGNED;
    auto fire = [&](const EmTensors& T) -> int {
#define BOF4_EM_CASE(DT_, I_)                                                                        \
    case I_: return sg ? launch_mse_chunk<DT_, I_, true, COUNT>(T, d_codebook, partials, tail, st)   \
                       : launch_mse_chunk<DT_, I_, false, COUNT>(T, d_codebook, partials, tail, st);
#define BOF4_EM_GO(DT_)                                                                              \
    switch (a.block_size) {                                                                          \
        BOF4_EM_CASE(DT_, 32) BOF4_EM_CASE(DT_, 64) BOF4_EM_CASE(DT_, 128) BOF4_EM_CASE(DT_, 256)    \
        BOF4_EM_CASE(DT_, 512) BOF4_EM_CASE(DT_, 1024) BOF4_EM_CASE(DT_, 2048)                       \
        default: return sg ? launch_mse_chunk<DT_, 4096, true, COUNT>(T, d_codebook, partials, tail, st)  \
                           : launch_mse_chunk<DT_, 4096, false, COUNT>(T, d_codebook, partials, tail, st); \
    }
        if (a.w_dtype == BOF4_F32) { BOF4_EM_GO(F32) } else { BOF4_EM_GO(BF16) }
#undef BOF4_EM_CASE
#undef BOF4_EM_GO
    };
    int calls = 0;
    const int rc = for_each_tensor_chunk(a, a.w_dtype == BOF4_BF16 ? EmGeo32<COUNT>::row : EmGeo<COUNT>::row, fire,
                                         &calls);
    if (rc) return rc;
    if (calls == 0) {  // records zeroed above; record 0 holds the short blocks' sums, if any
        tail.enabled = 0;
        tail.n_records = 1;
        em_mse_finalize_kernel<<<1, 1024, 0, st>>>(partials, tail);
        BOF4_CUDA_TRY(cudaGetLastError());
    }
    return BOF4_OK;
}

int reset_ticket(double* partials, cudaStream_t st)
{
    BOF4_CUDA_TRY(cudaMemsetAsync(reinterpret_cast<char*>(partials) + kEmTicketOffset, 0, 4, st));
    return BOF4_OK;
}

}  // namespace

extern "C" int bof4_em_step(const void* const* h_w, const int64_t* h_n, int n_tensors, int w_dtype,
                            int block_size, int norm, int metric, const float* d_codebook,
                            bof4_em_stats* d_stats, void* d_ws, size_t ws_bytes, void* stream)
{
    EmArgs a{h_w, h_n, n_tensors, w_dtype, block_size, norm, metric, 0};
    int rc = check_em("bof4_em_step", a, d_codebook, d_ws, ws_bytes);
    if (rc) return rc;
    if (!d_stats) {
        set_error("bof4_em_step: NULL stats");
        return BOF4_ERR_INVALID_ARG;
    }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    double* partials = static_cast<double*>(d_ws);
    if (metric == BOF4_METRIC_MSE || metric == BOF4_METRIC_MSE_NORMALIZED) {
        if ((rc = reset_ticket(partials, st))) return rc;
        MseTail tail{};
        tail.stats = d_stats;
        return enqueue_mse_pass<true>(a, d_codebook, partials, tail, st);
    }
    rc = mae_prepare(a, d_ws, ws_bytes, st);
    if (rc) return rc;
    return mae_iteration(a, d_codebook, nullptr, 0u, d_stats, nullptr, d_ws, ws_bytes, st);
}

extern "C" int bof4_fit_codebook(const void* const* h_w, const int64_t* h_n, int n_tensors,
                                 int w_dtype, int block_size, int norm, int metric,
                                 float* d_codebook, uint32_t fixed_mask, int iters,
                                 double* d_err_log, void* d_ws, size_t ws_bytes, void* stream)
{
    EmArgs a{h_w, h_n, n_tensors, w_dtype, block_size, norm, metric, 0};
    int rc = check_em("bof4_fit_codebook", a, d_codebook, d_ws, ws_bytes);
    if (rc) return rc;
    if (iters < 0) {
        set_error("bof4_fit_codebook: negative iteration count");
        return BOF4_ERR_INVALID_ARG;
    }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    double* partials = static_cast<double*>(d_ws);
    if (metric == BOF4_METRIC_MSE || metric == BOF4_METRIC_MSE_NORMALIZED) {
        if (iters > 0 && (rc = reset_ticket(partials, st))) return rc;
        for (int t = 0; t < iters; ++t) {
            MseTail tail{};
            tail.codebook = d_codebook;
            tail.fixed_mask = fixed_mask;
            tail.err_slot = d_err_log ? d_err_log + t : nullptr;
            rc = enqueue_mse_pass<false>(a, d_codebook, partials, tail, st);
            if (rc) return rc;
        }
        return BOF4_OK;
    }
    if (iters > 0) {
        rc = mae_prepare(a, d_ws, ws_bytes, st);
        if (rc) return rc;
    }
    for (int t = 0; t < iters; ++t) {
        rc = mae_iteration(a, d_codebook, d_codebook, fixed_mask, nullptr,
                           d_err_log ? d_err_log + t : nullptr, d_ws, ws_bytes, st);
        if (rc) return rc;
    }
    return BOF4_OK;
}

extern "C" int bof4_m_step(const bof4_em_stats* d_stats, int n_records, int metric, float* d_codebook,
                           uint32_t fixed_mask, double* d_err_slot, bof4_em_stats* d_total, void* stream)
{
    if (!d_stats || n_records < 1 || !d_codebook) {
        set_error("bof4_m_step: NULL pointer or no records");
        return BOF4_ERR_INVALID_ARG;
    }
    if (metric != BOF4_METRIC_MSE && metric != BOF4_METRIC_MSE_NORMALIZED) {
        set_error("bof4_m_step: only the MSE centroids are sums that can be merged from separate records "
                  "(a weighted median of a union needs the histograms of every selection pass)");
        return BOF4_ERR_INVALID_ARG;
    }
    m_step_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(d_stats, n_records, d_codebook, fixed_mask,
                                                                   d_err_slot, d_total);
    BOF4_CUDA_TRY(cudaGetLastError());
    return BOF4_OK;
}
