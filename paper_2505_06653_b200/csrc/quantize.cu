// Block-wise quantiser and dequantiser (Sec. 2.1 Eq. 1-3, Sec. 3.1 Eq. 4) and the OPQ outlier
// split (Sec. 3.3, App. E): streaming kernels.
//
// quantize: one lane owns 16 consecutive weights (32-byte load), a block is a group of I/16
// lanes; shuffle butterfly for the block constant, exact division (reciprocal sequence for
// bf16, IEEE divide otherwise), one-probe table search of the region, 16 codes packed into one
// 64-bit store per lane (256 contiguous bytes per warp).  The next row's load is issued before
// the current row is processed.
// dequantize: one lane owns 16 outputs (8 code bytes in, 32 or 64 bytes out).
#include <mutex>

#include "common.cuh"
#include "lane32.cuh"
#include "layout.h"

namespace bof4 {

constexpr int kQThreads = 512;              // quantise / OPQ pass 1
constexpr int kQRow = kQThreads * kLaneW;   // weights per CTA row
constexpr int kQCtasPerSm = 2;              // two CTAs, each with its own region table
constexpr int kDThreads = 512;              // dequantise
constexpr int kDCtasPerSm = 3;              // each with its own 64 KiB level-pair table
constexpr int kDTableBytes = 256 * 32 * 8;  // [code byte][lane] pairs of levels
constexpr int kDLaneW = 32;                 // outputs per lane and row (16 code bytes in)
constexpr int kDRow = kDThreads * kDLaneW;  // outputs per CTA row (dequantise)

template <class ST>
__device__ __forceinline__ void store_scale(void* scales, int64_t b, float m);
template <>
__device__ __forceinline__ void store_scale<F32>(void* scales, int64_t b, float m)
{
    static_cast<float*>(scales)[b] = m;
}
template <>
__device__ __forceinline__ void store_scale<BF16>(void* scales, int64_t b, float m)
{
    static_cast<uint16_t*>(scales)[b] = (uint16_t)(__float_as_uint(m) >> 16);  // exact: m is a bf16 value
}

// Region setup shared by the quantising kernels: thresholds, levels and the one-probe table.
struct QuantTables {
    float* xi;
    unsigned char* lut;
    bool lut_ok;
};

__device__ __forceinline__ QuantTables setup_tables(const float* __restrict__ levels, float* s_xi,
                                                    float* s_lv, unsigned char* s_lut, int* s_multi)
{
    make_thresholds(levels, s_xi, s_lv, threadIdx.x);
    __syncthreads();
    build_lut(s_xi, s_lut, s_multi, [](int base) { return (uint32_t)base; });
    __syncthreads();
    return QuantTables{s_xi, s_lut, *s_multi == 0};
}

// Codes of the 16 normalised weights of a lane packed as 8 bytes (two words), even element in
// the high nibble of its byte.  Each word is built by Horner steps w = 16 w + code over its 8
// codes in the order 6 7 4 5 2 3 0 1, which leaves byte k = (code[2k] << 4) | code[2k+1].
// use_lut (warp-uniform) requires finite x in [-1, 1].
__device__ __forceinline__ void encode16(const float (&x)[kLaneW], const QuantTables& T, bool use_lut,
                                         uint32_t lut_base, uint32_t& w0, uint32_t& w1)
{
    uint32_t word[2];
    if (use_lut) {
        float key[kLaneW];
#pragma unroll
        for (int k = 0; k < kLaneW / 2; ++k) {
            const float2 kk = lut_key2(make_float2(x[2 * k], x[2 * k + 1]));
            key[2 * k] = kk.x;
            key[2 * k + 1] = kk.y;
        }
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            uint32_t w = 0u;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const int k = 8 * h + (6 - 2 * (j >> 1)) + (j & 1);
                const uint2 e = lut_probe(key[k], lut_base);
                w = w * 16u + e.y;
                if (x[k] >= __uint_as_float(e.x)) w += 1u;
            }
            word[h] = w;
        }
    } else {
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            uint32_t w = 0u;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const int k = 8 * h + (6 - 2 * (j >> 1)) + (j & 1);
                w = w * 16u + (uint32_t)region_of(x[k], T.xi);
            }
            word[h] = w;
        }
    }
    w0 = word[0];
    w1 = word[1];
}

// Block constant, normalisation, codes and stores for one lane-row of (cleaned) weights.
template <class DT, int I, bool SIGNED, class ST>
__device__ __forceinline__ void quantize_row(const float (&v)[kLaneW], float mx, float mn, int64_t idx,
                                             bool ok, const QuantTables& T, uint32_t lut_base, int lane,
                                             uint8_t* __restrict__ codes, void* __restrict__ scales,
                                             WideScratch* ws)
{
    float g;
    const float m = block_constant<I, SIGNED>(v, mx, mn, g, ws);
    const bool safe = row_is_safe(g, ok);
    float x[kLaneW];
    normalise16<true>(v, m, safe && DT::code == BF16::code, x);
    uint32_t w0, w1;
    encode16(x, T, safe && T.lut_ok, lut_base, w0, w1);
    if (ok) {
        st_stream64(codes + idx / 2, w0, w1);
        if ((idx & (I - 1)) == 0) store_scale<ST>(scales, idx / I, m);  // the block's first lane
    }
}

template <class DT, int I, bool SIGNED, class ST>
__global__ void __launch_bounds__(kQThreads, kQCtasPerSm)
quantize_kernel(const void* __restrict__ w, int64_t n, const float* __restrict__ levels,
                uint8_t* __restrict__ codes, void* __restrict__ scales)
{
    extern __shared__ __align__(16) unsigned char s_lut[];
    __shared__ float s_xi[kLevels], s_lv[kLevels];
    __shared__ int s_multi;
    __shared__ WideScratch s_wide;
    const QuantTables T = setup_tables(levels, s_xi, s_lv, s_lut, &s_multi);
    const int lane = threadIdx.x & 31;
    const uint32_t lut_base = lut_lane_base(s_lut, lane);  // table base of this lane
    const RowMap map(n, kQRow, threadIdx.x);
    int r = blockIdx.x;
    if (r >= map.rows) return;
    RawRow<DT> raw = map.ok(r) ? load_raw<DT>(w, map.idx(r)) : zero_raw<DT>();
    for (; r < map.rows; r += gridDim.x) {
        const int rn = r + gridDim.x;
        const RawRow<DT> next = map.ok(rn) ? load_raw<DT>(w, map.idx(rn)) : zero_raw<DT>();
        float v[kLaneW], mx, mn;
        widen(raw, v);
        lane_minmax(v, mx, mn);
        quantize_row<DT, I, SIGNED, ST>(v, mx, mn, map.idx(r), map.ok(r), T, lut_base, lane, codes, scales,
                                        &s_wide);
        raw = next;
    }
}

// ---------------------------------------------------------------- quantise, bf16 weights
//
// 32 weights per lane (lane32.cuh); two row buffers used in turn, so that the load of the row
// after next is issued before a row is processed and no register is copied between iterations.

constexpr int kQRow32 = kQThreads * kLW;  // weights per CTA row

struct QuantShared32 {
    float xi[kLevels], lv[kLevels];
    int multi;
    WideScratch wide;
    FastInfo info;
};

// Block constant, codes and stores for the lane's 32 (cleaned) weights of one row.
template <int I, bool SIGNED, class ST>
__device__ __forceinline__ void quantize_row32(const uint32_t (&u)[16], float mx, float mn, int64_t idx, bool ok,
                                               bool fast_ok, uint32_t lut_base, QuantShared32* S,
                                               uint8_t* __restrict__ codes, void* __restrict__ scales)
{
    float g;
    const float m = block_constant32<I, SIGNED>(u, mx, mn, g, &S->wide);
    uint32_t cw[4];
    if (row_is_fast(g, m, ok, fast_ok, &S->info))
        encode32_fast(u, m, lut_base, cw);
    else
        encode32_slow(u, m, S->xi, cw);
    if (ok) {
        st_stream128(codes + idx / 2, cw[0], cw[1], cw[2], cw[3]);
        if ((idx & (I - 1)) == 0) store_scale<ST>(scales, idx / I, m);  // the block's first lane
    }
}

// The same for one row outside the common case (a block constant that is zero, extreme, not
// finite or of a "near" significand; a codebook the table cannot serve; the partial last row of
// a tensor), kept out of line so that it costs the streaming loop no registers.  Blocks within
// a warp only (the wide-block kernel below calls quantize_row32 itself).
template <int I, bool SIGNED, class ST>
__device__ __noinline__ void quantize_row32_generic(Raw32 raw, int64_t idx, bool ok, bool fast_ok, uint32_t lut_base,
                                                    QuantShared32* S, uint8_t* __restrict__ codes,
                                                    void* __restrict__ scales)
{
    uint32_t u[16];
    words_of(raw, u);
    float mx, mn;
    lane_minmax32(u, mx, mn);
    quantize_row32<I, SIGNED, ST>(u, mx, mn, idx, ok, fast_ok, lut_base, S, codes, scales);
}

// The rows r, r + G, r + 2G, ... of one tensor (G = CTAs of the grid), `first` being row r already
// on its way.  Called by all threads of the CTA with the tables in place.
template <int I, bool SIGNED, class ST>
__device__ __forceinline__ void quantize32_rows(const void* __restrict__ w, int64_t n, uint8_t* __restrict__ codes,
                                                void* __restrict__ scales, const int r0, const Raw32& first,
                                                const bool fast_ok, const uint32_t lut_base, QuantShared32* S)
{
    const RowMap32 map(n, kQRow32, threadIdx.x);
    const int G = gridDim.x;
    int r = r0;
    auto fetch = [&](int rr) { return map.ok(rr) ? load_raw32(w, map.idx(rr)) : zero_raw32(); };
    if constexpr (Geo32<I>::WPB > 1) {
        // blocks of several warps: every thread of the CTA takes every step (barriers inside)
        Raw32 a = first;
        for (; r < map.rows; r += G) {
            const Raw32 next = fetch(r + G);
            uint32_t u[16];
            words_of(a, u);
            float mx, mn;
            lane_minmax32(u, mx, mn);
            quantize_row32<I, SIGNED, ST>(u, mx, mn, map.idx(r), map.ok(r), fast_ok, lut_base, S, codes, scales);
            a = next;
        }
    } else {
        // Whole rows: unconditional loads into two buffers used in turn; a row all of whose block
        // constants are ordinary is encoded here, any other goes to the out-of-line version.
        auto row = [&](const Raw32& raw, int rr) {
            uint32_t u[16];
            words_of(raw, u);
            float mx, mn, g;
            lane_minmax32(u, mx, mn);
            const float m = block_constant32<I, SIGNED>(u, mx, mn, g, nullptr);
            const int64_t idx = map.idx(rr);
            if (row_is_fast(g, m, true, fast_ok, &S->info)) {
                uint32_t cw[4];
                encode32_fast(u, m, lut_base, cw);
                st_stream128(codes + idx / 2, cw[0], cw[1], cw[2], cw[3]);
                if ((idx & (I - 1)) == 0) store_scale<ST>(scales, idx / I, m);
            } else {
                quantize_row32_generic<I, SIGNED, ST>(raw, idx, true, fast_ok, lut_base, S, codes, scales);
            }
        };
        const int full = map.rows_full;
        if (r < full) {
            Raw32 a = first, b = first;
            while (true) {
                int rn = r + G;
                if (rn < full) b = load_raw32(w, map.idx(rn));
                row(a, r);
                if (rn >= full) break;
                r = rn;
                rn = r + G;
                if (rn < full) a = load_raw32(w, map.idx(rn));
                row(b, r);
                if (rn >= full) break;
                r = rn;
            }
        }
        // the partial last row of the tensor, by the CTA whose turn it is
        if (map.rows > full && full >= r0 && (full - r0) % G == 0)
            quantize_row32_generic<I, SIGNED, ST>(full == r0 ? first : fetch(full), map.idx(full), map.ok(full),
                                                  fast_ok, lut_base, S, codes, scales);
    }
}

template <int I, bool SIGNED, class ST>
__global__ void __launch_bounds__(kQThreads, kQCtasPerSm)
quantize32_kernel(const void* __restrict__ w, int64_t n, const float* __restrict__ levels,
                  uint8_t* __restrict__ codes, void* __restrict__ scales)
{
    extern __shared__ __align__(16) unsigned char s_lut[];
    __shared__ QuantShared32 S;
    const RowMap32 map(n, kQRow32, threadIdx.x);
    const int r = blockIdx.x;
    if (r >= map.rows) return;
    const Raw32 first = map.ok(r) ? load_raw32(w, map.idx(r)) : zero_raw32();  // on its way while the tables are built
    const bool lut_ok = build_tables32(levels, S.xi, S.lv, s_lut, &S.info, [](int base) { return (uint32_t)base; });
    const bool fast_ok = lut_ok && !S.info.tiny;
    const uint32_t lut_base = lut_lane_base(s_lut, threadIdx.x & 31);
    quantize32_rows<I, SIGNED, ST>(w, n, codes, scales, r, first, fast_ok, lut_base, &S);
}

// Several tensors in one launch: the tables are built once per CTA, and the rows of all tensors
// are dealt round-robin over the CTAs as if they were one tensor (tensor t starts with the CTA
// that follows the last row of tensor t - 1), so that small tensors neither pay for a launch and
// a table build each nor leave part of the grid idle.
constexpr int kQBatch = 64;  // tensors per launch (kernel parameter table)
struct QuantBatch {
    const void* w[kQBatch];
    uint8_t* codes[kQBatch];
    void* scales[kQBatch];
    int64_t n[kQBatch];
    int start[kQBatch];  // CTA that takes the tensor's first row
    int count;
};

template <int I, bool SIGNED, class ST>
__global__ void __launch_bounds__(kQThreads, kQCtasPerSm)
quantize32_batch_kernel(const QuantBatch B, const float* __restrict__ levels)
{
    extern __shared__ __align__(16) unsigned char s_lut[];
    __shared__ QuantShared32 S;
    const int G = gridDim.x;
    const bool lut_ok = build_tables32(levels, S.xi, S.lv, s_lut, &S.info, [](int base) { return (uint32_t)base; });
    const bool fast_ok = lut_ok && !S.info.tiny;
    const uint32_t lut_base = lut_lane_base(s_lut, threadIdx.x & 31);
    for (int t = 0; t < B.count; ++t) {
        const int64_t n = B.n[t];
        const RowMap32 map(n, kQRow32, threadIdx.x);
        const int r0 = ((int)blockIdx.x + G - B.start[t]) % G;
        if (r0 >= map.rows) continue;  // uniform over the CTA
        const void* w = B.w[t];
        const Raw32 first = map.ok(r0) ? load_raw32(w, map.idx(r0)) : zero_raw32();
        quantize32_rows<I, SIGNED, ST>(w, n, B.codes[t], B.scales[t], r0, first, fast_ok, lut_base, &S);
    }
}

// ---------------------------------------------------------------- dequantise

template <class ST>
__device__ __forceinline__ float load_scale(const void* scales, int64_t b);
template <>
__device__ __forceinline__ float load_scale<F32>(const void* scales, int64_t b)
{
    return __ldg(static_cast<const float*>(scales) + b);
}
template <>
__device__ __forceinline__ float load_scale<BF16>(const void* scales, int64_t b)
{
    return __uint_as_float((uint32_t)__ldg(static_cast<const uint16_t*>(scales) + b) << 16);
}

// Two fp32 values to one packed pair of bf16 (round to nearest even): lo -> bits 0..15.
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi)
{
    uint32_t d;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
    return d;
}

// One code byte holds two weights, so the levels are tabulated per byte: entry b is the pair
// (xhat[b >> 4], xhat[b & 15]); one 8-byte shared-memory read and one packed multiplication by
// the block constant give both products (Eq. 3).  The table is kept once per lane ([byte][lane],
// 64 KiB): the code bytes of the 32 lanes are unrelated, and a shared table of 256 entries made
// every read a three-fold bank conflict on average, which bound the kernel; with a column per
// lane the bank only depends on the lane.
__device__ __forceinline__ void build_pair_table(const float* __restrict__ levels, unsigned char* s_tab)
{
    for (int e = threadIdx.x; e < 256 * 32; e += blockDim.x) {
        const int b = e >> 5;
        *reinterpret_cast<float2*>(s_tab + (size_t)e * 8) = make_float2(levels[b >> 4], levels[b & 15]);
    }
    __syncthreads();
}

template <class ST, class OT, int I>
__device__ __forceinline__ void dequantize_rows(const uint8_t* __restrict__ codes, const void* __restrict__ scales,
                                                int64_t n, void* __restrict__ out, const unsigned char* s_tab, const int r0)
{
    const int64_t rows = (n + kDRow - 1) / kDRow;
    int64_t r = r0;
    if (r >= rows) return;
    const uint32_t lane8 = (threadIdx.x & 31u) * 8u;
    // n is a multiple of 32, so a lane's 32 outputs are all inside the tensor or all outside
    auto fetch = [&](int64_t row, int64_t& idx, uint4& cc, float& m) {
        idx = (row * kDThreads + threadIdx.x) * kDLaneW;
        cc = make_uint4(0u, 0u, 0u, 0u);
        m = 0.0f;
        if (idx < n) {
            asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                         : "=r"(cc.x), "=r"(cc.y), "=r"(cc.z), "=r"(cc.w)
                         : "l"(codes + idx / 2));
            m = load_scale<ST>(scales, idx / I);
        }
    };
    int64_t idx, idx_next;
    uint4 cc, cc_next;
    float m, m_next;
    fetch(r, idx, cc, m);
    for (; r < rows; r += gridDim.x) {
        fetch(r + gridDim.x, idx_next, cc_next, m_next);
        if (idx < n) {
            const float2 mm = make_float2(m, m);
            const uint32_t word[4] = {cc.x, cc.y, cc.z, cc.w};
#pragma unroll
            for (int h = 0; h < 2; ++h) {  // 16 outputs at a time
                float2 o[8];
#pragma unroll
                for (int k = 0; k < 8; ++k) {
                    // byte offset of this lane's entry of the code byte: byte * 256 + lane * 8, one permute
                    const uint32_t off = __byte_perm(word[2 * h + (k >> 2)], lane8, 0x5504u | ((uint32_t)(k & 3) << 4));
                    o[k] = __fmul2_rn(mm, *reinterpret_cast<const float2*>(s_tab + off));
                }
                if (OT::code == BF16::code) {
                    Raw8 p;
#pragma unroll
                    for (int k = 0; k < 8; ++k) p.u[k] = pack_bf16x2(o[k].x, o[k].y);
                    st_stream256(static_cast<uint16_t*>(out) + idx + 16 * h, p);
                } else {
                    Raw8 p, q;
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        p.u[2 * k] = __float_as_uint(o[k].x);
                        p.u[2 * k + 1] = __float_as_uint(o[k].y);
                        q.u[2 * k] = __float_as_uint(o[4 + k].x);
                        q.u[2 * k + 1] = __float_as_uint(o[4 + k].y);
                    }
                    st_stream256(static_cast<float*>(out) + idx + 16 * h, p);
                    st_stream256(static_cast<float*>(out) + idx + 16 * h + 8, q);
                }
            }
        }
        idx = idx_next;
        cc = cc_next;
        m = m_next;
    }
}

template <class ST, class OT, int I>
__global__ void __launch_bounds__(kDThreads, kDCtasPerSm)
dequantize_kernel(const uint8_t* __restrict__ codes, const void* __restrict__ scales, int64_t n,
                  const float* __restrict__ levels, void* __restrict__ out)
{
    extern __shared__ __align__(16) unsigned char s_tab[];
    build_pair_table(levels, s_tab);
    dequantize_rows<ST, OT, I>(codes, scales, n, out, s_tab, (int)blockIdx.x);
}

// Several tensors in one launch, their rows dealt round-robin over the CTAs as in
// quantize32_batch_kernel.
struct DequantBatch {
    const uint8_t* codes[kQBatch];
    const void* scales[kQBatch];
    void* out[kQBatch];
    int64_t n[kQBatch];
    int start[kQBatch];
    int count;
};

template <class ST, class OT, int I>
__global__ void __launch_bounds__(kDThreads, kDCtasPerSm)
dequantize_batch_kernel(const DequantBatch B, const float* __restrict__ levels)
{
    extern __shared__ __align__(16) unsigned char s_tab[];
    build_pair_table(levels, s_tab);
    const int G = gridDim.x;
    for (int t = 0; t < B.count; ++t)
        dequantize_rows<ST, OT, I>(B.codes[t], B.scales[t], B.n[t], B.out[t], s_tab,
                                   ((int)blockIdx.x + G - B.start[t]) % G);
}

// Outliers written back over the dequantised tensor (Sec. 3.3, decoding side).
template <class OT>
__global__ void scatter_outliers_kernel(const int32_t* __restrict__ idx, const uint16_t* __restrict__ val,
                                        const int64_t* __restrict__ n_out, int64_t capacity, int64_t n,
                                        void* __restrict__ out)
{
    int64_t k_end = *n_out;
    if (k_end > capacity) k_end = capacity;
    for (int64_t k = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; k < k_end;
         k += (int64_t)gridDim.x * blockDim.x) {
        const int64_t i = idx[k];
        if (i < 0 || i >= n) continue;
        if (OT::code == BF16::code)
            static_cast<uint16_t*>(out)[i] = val[k];
        else
            static_cast<float*>(out)[i] = __uint_as_float((uint32_t)val[k] << 16);
    }
}

// ---------------------------------------------------------------- OPQ (Sec. 3.3, App. E)

// Balanced binary summation tree over the block: neighbours first inside the lane, then the
// lane butterfly, then (blocks wider than a warp) the warps of the block pairwise in order.
// Every addition is a separate fp32 RN operation.
template <int I>
__device__ __forceinline__ float tree_sum(const float (&t)[kLaneW], float* slot)
{
    constexpr int LPB = BlockGeo<I>::LPB, WPB = BlockGeo<I>::WPB;
    float a[8];
#pragma unroll
    for (int k = 0; k < 8; ++k) a[k] = __fadd_rn(t[2 * k], t[2 * k + 1]);
    float s = __fadd_rn(__fadd_rn(__fadd_rn(a[0], a[1]), __fadd_rn(a[2], a[3])),
                        __fadd_rn(__fadd_rn(a[4], a[5]), __fadd_rn(a[6], a[7])));
#pragma unroll
    for (int off = 1; off < LPB; off <<= 1) s = __fadd_rn(s, __shfl_xor_sync(kFull, s, off));
    if constexpr (WPB > 1) s = across_warps<WPB>(s, slot, [](float p, float q) { return __fadd_rn(p, q); });
    return s;
}

// The outlier threshold of the lane's block: sigma_b * tau, sigma_b the corrected sample
// standard deviation (two-pass formula in fp32, tree-ordered sums).  For blocks wider than a
// warp every thread of the CTA must call it.
template <int I>
__device__ __forceinline__ float outlier_threshold(const float (&v)[kLaneW], float tau, WideScratch* ws)
{
    const float mean = __fmul_rn(tree_sum<I>(v, ws ? ws->a : nullptr), 1.0f / (float)I);  // exact: I = 2^k
    float q[kLaneW];
#pragma unroll
    for (int k = 0; k < kLaneW; ++k) {
        const float d = __fsub_rn(v[k], mean);
        q[k] = __fmul_rn(d, d);
    }
    const float sigma = __fsqrt_rn(__fdiv_rn(tree_sum<I>(q, ws ? ws->b : nullptr), (float)(I - 1)));
    return __fmul_rn(sigma, tau);
}

// Bit k of the result is set iff element k of this lane is an outlier: |w| > thr.
__device__ __forceinline__ unsigned outlier_bits(const float (&v)[kLaneW], float thr)
{
    unsigned o = 0;
#pragma unroll
    for (int k = 0; k < kLaneW; ++k) o |= (fabsf(v[k]) > thr) ? (1u << k) : 0u;
    return o;
}

// The outlier threshold of the block that contains tile `tile`, computed by ONE warp alone (the
// re-derivation of an overflowed tile in the gather kernel): a block wider than a warp is read
// tile by tile, twice, and its per-tile sums are combined in the same tree order.
template <class DT, int I>
__device__ __forceinline__ float outlier_threshold_one_warp(const void* __restrict__ w, int64_t tile, float tau,
                                                            int lane, const float (&v)[kLaneW])
{
    constexpr int WPB = BlockGeo<I>::WPB;
    if constexpr (WPB == 1) {
        return outlier_threshold<I>(v, tau, nullptr);
    } else {
        const int64_t first = (tile / WPB) * WPB;  // first tile of the block
        float part[WPB];
        float u[kLaneW];
#pragma unroll
        for (int t = 0; t < WPB; ++t) {
            widen(load_raw<DT>(w, (first + t) * kWarpW + lane * kLaneW), u);
            part[t] = tree_sum<kWarpW>(u, nullptr);
        }
#pragma unroll
        for (int step = 1; step < WPB; step <<= 1)
#pragma unroll
            for (int k = 0; k < WPB; k += 2 * step) part[k] = __fadd_rn(part[k], part[k + step]);
        const float mean = __fmul_rn(part[0], 1.0f / (float)I);
#pragma unroll
        for (int t = 0; t < WPB; ++t) {
            widen(load_raw<DT>(w, (first + t) * kWarpW + lane * kLaneW), u);
#pragma unroll
            for (int k = 0; k < kLaneW; ++k) {
                const float d = __fsub_rn(u[k], mean);
                u[k] = __fmul_rn(d, d);
            }
            part[t] = tree_sum<kWarpW>(u, nullptr);
        }
#pragma unroll
        for (int step = 1; step < WPB; step <<= 1)
#pragma unroll
            for (int k = 0; k < WPB; k += 2 * step) part[k] = __fadd_rn(part[k], part[k + step]);
        const float sigma = __fsqrt_rn(__fdiv_rn(part[0], (float)(I - 1)));
        return __fmul_rn(sigma, tau);
    }
}

// Exclusive prefix of a per-lane count over the warp, and the warp total.
__device__ __forceinline__ int warp_excl_scan(int cnt, int lane, int& total)
{
    int inc = cnt;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const int t = __shfl_up_sync(kFull, inc, off);
        if (lane >= off) inc += t;
    }
    total = __shfl_sync(kFull, inc, 31);
    return inc - cnt;
}

// The 16 (cleaned) weights of a lane back to their storage type (exact: values are the
// original ones or zero).
__device__ __forceinline__ void store_row(BF16, void* base, int64_t idx, const float (&v)[kLaneW])
{
    Raw8 p;
#pragma unroll
    for (int k = 0; k < 8; ++k)
        p.u[k] = (__float_as_uint(v[2 * k]) >> 16) | (__float_as_uint(v[2 * k + 1]) & 0xffff0000u);
    st_stream256(static_cast<uint16_t*>(base) + idx, p);
}
__device__ __forceinline__ void store_row(F32, void* base, int64_t idx, const float (&v)[kLaneW])
{
    Raw8 p, q;
#pragma unroll
    for (int k = 0; k < 8; ++k) {
        p.u[k] = __float_as_uint(v[k]);
        q.u[k] = __float_as_uint(v[8 + k]);
    }
    st_stream256(static_cast<float*>(base) + idx, p);
    st_stream256(static_cast<float*>(base) + idx + 8, q);
}

// Pass 1 of OPQ.  Each warp iteration is one tile of kOpqTile weights: outliers are detected,
// counted (counts[tile]) and the first kOpqStage of the tile staged in ascending index order;
// the cleaned weights are quantised (QUANT) or stored (w_clean != NULL).
template <class DT, int I, bool SIGNED, class ST, bool QUANT>
__global__ void __launch_bounds__(kQThreads, kQCtasPerSm)
opq_pass1_kernel(const void* __restrict__ w, int64_t n, const float* __restrict__ levels, float tau,
                 uint8_t* __restrict__ codes, void* __restrict__ scales, void* __restrict__ w_clean,
                 int32_t* __restrict__ counts, unsigned long long* __restrict__ chunk_sum,
                 int32_t* __restrict__ stage_idx, uint16_t* __restrict__ stage_val)
{
    static_assert(kOpqTile == kWarpW, "one tile per warp iteration");
    extern __shared__ __align__(16) unsigned char s_lut[];
    __shared__ float s_xi[kLevels], s_lv[kLevels];
    __shared__ int s_multi;
    __shared__ WideScratch s_wide;
    QuantTables T{s_xi, s_lut, false};
    if (QUANT) T = setup_tables(levels, s_xi, s_lv, s_lut, &s_multi);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint32_t lut_base = lut_lane_base(s_lut, lane);  // table base of this lane
    const RowMap map(n, kQRow, threadIdx.x);
    int r = blockIdx.x;
    if (r >= map.rows) return;
    RawRow<DT> raw = map.ok(r) ? load_raw<DT>(w, map.idx(r)) : zero_raw<DT>();
    for (; r < map.rows; r += gridDim.x) {
        const int rn = r + gridDim.x;
        const RawRow<DT> next = map.ok(rn) ? load_raw<DT>(w, map.idx(rn)) : zero_raw<DT>();
        const int64_t idx = map.idx(r);
        const bool ok = map.ok(r);
        const int64_t tile = (int64_t)r * (kQThreads / 32) + warp;
        const bool tile_ok = tile * kOpqTile < n;  // warp-uniform
        float v[kLaneW];
        widen(raw, v);
        // A lane can only hold an outlier if its largest magnitude exceeds the threshold, so the
        // per-element test runs only in warps where some lane does (a NaN maximum also enters).
        float mx, mn;
        lane_minmax(v, mx, mn);
        const float thr = outlier_threshold<I>(v, tau, &s_wide);
        const bool maybe = !(fmaxf(mx, -mn) <= thr);
        if (__any_sync(kFull, maybe)) {
            const unsigned o = outlier_bits(v, thr);
            const unsigned any = __ballot_sync(kFull, o != 0u);
            if (any) {
                int total;
                int pos = warp_excl_scan(__popc(o), lane, total);
#pragma unroll
                for (int k = 0; k < kLaneW; ++k)
                    if ((o >> k) & 1u) {
                        if (pos < kOpqStage) {
                            stage_idx[tile * kOpqStage + pos] = (int32_t)(idx + k);
                            stage_val[tile * kOpqStage + pos] = (uint16_t)bf16_rne(v[k]);
                        }
                        ++pos;
                        v[k] = 0.0f;
                    }
                if (lane == 0) {
                    counts[tile] = total;
                    atomicAdd(&chunk_sum[tile / kOpqChunk], (unsigned long long)total);  // integer: order-free
                }
                lane_minmax(v, mx, mn);  // of the cleaned weights
            } else if (lane == 0 && tile_ok) {
                counts[tile] = 0;
            }
        } else if (lane == 0 && tile_ok) {
            counts[tile] = 0;
        }
        if (QUANT) {
            quantize_row<DT, I, SIGNED, ST>(v, mx, mn, idx, ok, T, lut_base, lane, codes, scales, &s_wide);
        } else if (w_clean != nullptr && ok) {
            store_row(DT{}, w_clean, idx, v);
        }
        raw = next;
    }
}

// ---------------------------------------------------------------- OPQ pass 1, bf16 weights
//
// The same pass on the 64-byte-per-lane front end.  A warp iteration covers two tiles of
// kOpqTile weights (lanes 0-15 and lanes 16-31), so the tile counts, staging slots and the gather
// kernel are those of the generic pass.  The two tree sums of the block statistics (App. E) keep
// the balanced-tree order: neighbours first inside the lane (32 weights, five levels, the upper
// four on packed pairs), then the lane butterfly, then the warps of a wide block.

// Balanced tree sum of the lane's 32 values given as 16 pairs {even, odd}: every addition is a
// separate fp32 RN operation; levels two to five add two independent partial sums per instruction.
__device__ __forceinline__ float lane_tree_sum32(const float2 (&t)[16])
{
    float a[16];
#pragma unroll
    for (int k = 0; k < 16; ++k) a[k] = __fadd_rn(t[k].x, t[k].y);
    float2 b[4], c[2];
#pragma unroll
    for (int k = 0; k < 4; ++k)  // (a0 + a1, a2 + a3), (a4 + a5, a6 + a7), ...
        b[k] = __fadd2_rn(make_float2(a[4 * k], a[4 * k + 2]), make_float2(a[4 * k + 1], a[4 * k + 3]));
#pragma unroll
    for (int k = 0; k < 2; ++k)
        c[k] = __fadd2_rn(make_float2(b[2 * k].x, b[2 * k + 1].x), make_float2(b[2 * k].y, b[2 * k + 1].y));
    const float2 d = __fadd2_rn(make_float2(c[0].x, c[1].x), make_float2(c[0].y, c[1].y));
    return __fadd_rn(d.x, d.y);
}

template <int I>
__device__ __forceinline__ float block_tree_sum32(float s, float* slot)
{
    constexpr int LPB = Geo32<I>::LPB, WPB = Geo32<I>::WPB;
#pragma unroll
    for (int off = 1; off < LPB; off <<= 1) s = __fadd_rn(s, __shfl_xor_sync(kFull, s, off));
    if constexpr (WPB > 1) s = across_warps<WPB>(s, slot, [](float p, float q) { return __fadd_rn(p, q); });
    return s;
}

// sigma_b * tau of the lane's block (two-pass formula in fp32, tree-ordered sums).
template <int I>
__device__ __forceinline__ float outlier_threshold32(const uint32_t (&u)[16], float tau, WideScratch* ws)
{
    float2 v[16];
#pragma unroll
    for (int k = 0; k < 16; ++k) v[k] = make_float2(bf_lo(u[k]), bf_hi(u[k]));
    const float mean = __fmul_rn(block_tree_sum32<I>(lane_tree_sum32(v), ws->a), 1.0f / (float)I);  // exact: I = 2^k
    const float2 nm = make_float2(-mean, -mean);
#pragma unroll
    for (int k = 0; k < 16; ++k) {
        const float2 d = __fadd2_rn(v[k], nm);
        v[k] = __fmul2_rn(d, d);
    }
    const float sigma = __fsqrt_rn(__fdiv_rn(block_tree_sum32<I>(lane_tree_sum32(v), ws->b), (float)(I - 1)));
    return __fmul_rn(sigma, tau);
}

template <int I, bool SIGNED, class ST, bool QUANT>
__global__ void __launch_bounds__(kQThreads, kQCtasPerSm)
opq_pass1_32_kernel(const void* __restrict__ w, int64_t n, const float* __restrict__ levels, float tau,
                    uint8_t* __restrict__ codes, void* __restrict__ scales, void* __restrict__ w_clean,
                    int32_t* __restrict__ counts, unsigned long long* __restrict__ chunk_sum,
                    int32_t* __restrict__ stage_idx, uint16_t* __restrict__ stage_val)
{
    static_assert(2 * kOpqTile == kWarpW32, "two tiles per warp iteration");
    extern __shared__ __align__(16) unsigned char s_lut[];
    __shared__ QuantShared32 S;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const RowMap32 map(n, kQRow32, threadIdx.x);
    const int G = gridDim.x;
    int r = blockIdx.x;
    if (r >= map.rows) return;
    auto fetch = [&](int rr) { return map.ok(rr) ? load_raw32(w, map.idx(rr)) : zero_raw32(); };
    Raw32 a = fetch(r);
    bool fast_ok = false;
    uint32_t lut_base = 0u;
    if (QUANT) {
        const bool lut_ok = build_tables32(levels, S.xi, S.lv, s_lut, &S.info, [](int base) { return (uint32_t)base; });
        fast_ok = lut_ok && !S.info.tiny;
        lut_base = lut_lane_base(s_lut, lane);
    }
    for (; r < map.rows; r += G) {
        const Raw32 next = fetch(r + G);
        const int64_t idx = map.idx(r);
        const bool ok = map.ok(r);
        // this lane's tile: lanes 0-15 the first, lanes 16-31 the second tile of the warp row
        const int64_t tile = ((int64_t)r * (kQThreads / 32) + warp) * 2 + (lane >> 4);
        const bool tile_ok = tile * kOpqTile < n;  // uniform over the half warp
        uint32_t u[16];
        words_of(a, u);
        float mx, mn;
        lane_minmax32(u, mx, mn);
        const float thr = outlier_threshold32<I>(u, tau, &S.wide);
        // A lane can only hold an outlier if its largest magnitude exceeds the threshold, so the
        // per-element test runs only in warps where some lane does (a NaN maximum also enters).
        const bool maybe = !(fmaxf(mx, -mn) <= thr);
        int total_half = 0;
        if (__any_sync(kFull, maybe)) {
            unsigned o = 0u;
#pragma unroll
            for (int k = 0; k < 16; ++k) {
                o |= (fabsf(bf_lo(u[k])) > thr) ? (1u << (2 * k)) : 0u;
                o |= (fabsf(bf_hi(u[k])) > thr) ? (2u << (2 * k)) : 0u;
            }
            if (__any_sync(kFull, o != 0u)) {
                int total;
                int pos = warp_excl_scan(__popc(o), lane, total);
                const int lower = __shfl_sync(kFull, pos, 16);  // outliers of lanes 0-15
                total_half = (lane >> 4) ? total - lower : lower;
                if (lane >> 4) pos -= lower;
#pragma unroll
                for (int k = 0; k < 16; ++k) {
#pragma unroll
                    for (int h = 0; h < 2; ++h)
                        if ((o >> (2 * k + h)) & 1u) {
                            if (pos < kOpqStage) {
                                stage_idx[tile * kOpqStage + pos] = (int32_t)(idx + 2 * k + h);
                                stage_val[tile * kOpqStage + pos] = (uint16_t)(h ? (u[k] >> 16) : (u[k] & 0xffffu));
                            }
                            ++pos;
                            u[k] &= h ? 0x0000ffffu : 0xffff0000u;  // the outlier becomes +0
                        }
                }
                if ((lane & 15) == 0 && total_half > 0)
                    atomicAdd(&chunk_sum[tile / kOpqChunk], (unsigned long long)total_half);  // integer: order-free
                lane_minmax32(u, mx, mn);  // of the cleaned weights
            }
        }
        if ((lane & 15) == 0 && tile_ok) counts[tile] = total_half;
        if (QUANT) {
            quantize_row32<I, SIGNED, ST>(u, mx, mn, idx, ok, fast_ok, lut_base, &S, codes, scales);
        } else if (w_clean != nullptr && ok) {
            uint16_t* dst = static_cast<uint16_t*>(w_clean) + idx;
            st_stream256(dst, Raw8{{u[0], u[1], u[2], u[3], u[4], u[5], u[6], u[7]}});
            st_stream256(dst + 16, Raw8{{u[8], u[9], u[10], u[11], u[12], u[13], u[14], u[15]}});
        }
        a = next;
    }
}

// Pass 2: every tile's staged outliers are copied to their final, globally ascending position;
// a tile with more than kOpqStage outliers is re-derived from the weights by one warp.  Each
// CTA owns one chunk of tiles; its first output position is the sum of the earlier chunks'
// outlier counts (accumulated by pass 1), and the last chunk's CTA also reports the total.
template <class DT, int I>
__global__ void __launch_bounds__(256)
opq_gather_kernel(const void* __restrict__ w, int64_t n, float tau, const int32_t* __restrict__ counts,
                  int64_t tiles, const unsigned long long* __restrict__ chunk_sum,
                  const int32_t* __restrict__ stage_idx, const uint16_t* __restrict__ stage_val,
                  int32_t* __restrict__ out_idx, uint16_t* __restrict__ out_val, int64_t capacity,
                  int64_t* __restrict__ n_out)
{
    constexpr int PER = kOpqChunk / 256;  // consecutive tiles per thread
    __shared__ int64_t s_warp[8];
    __shared__ unsigned long long s_base[8];
    __shared__ int32_t s_ovf_tile[kOpqChunk];  // tile index relative to the chunk
    __shared__ int32_t s_ovf_off[kOpqChunk];   // offset relative to the chunk's first output
    __shared__ int s_novf;
    if (threadIdx.x == 0) s_novf = 0;
    __syncthreads();
    const int64_t t0 = (int64_t)blockIdx.x * kOpqChunk + (int64_t)threadIdx.x * PER;
    int c[PER];
    int local = 0;
#pragma unroll
    for (int k = 0; k < PER; ++k) {
        c[k] = (t0 + k < tiles) ? counts[t0 + k] : 0;
        local += c[k];
    }
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int wtotal;
    int excl = warp_excl_scan(local, lane, wtotal);
    if (lane == 0) s_warp[warp] = wtotal;
    __syncthreads();
    int rel = excl;
    for (int k = 0; k < warp; ++k) rel += (int)s_warp[k];
    // first output position of this chunk: outliers of all earlier chunks
    unsigned long long before = 0ull;
    for (int k = threadIdx.x; k < (int)blockIdx.x; k += 256) before += chunk_sum[k];
#pragma unroll
    for (int off = 16; off; off >>= 1) before += __shfl_xor_sync(kFull, before, off);
    if (lane == 0) s_base[warp] = before;
    __syncthreads();
    before = 0ull;
    for (int k = 0; k < 8; ++k) before += s_base[k];
    const int64_t base = (int64_t)before;
    if (blockIdx.x == gridDim.x - 1 && threadIdx.x == 0) *n_out = base + (int64_t)chunk_sum[blockIdx.x];
#pragma unroll
    for (int k = 0; k < PER; ++k) {
        if (c[k] > 0) {
            if (c[k] <= kOpqStage) {
                for (int j = 0; j < c[k]; ++j) {
                    const int64_t dst = base + rel + j;
                    if (dst < capacity) {
                        out_idx[dst] = stage_idx[(t0 + k) * kOpqStage + j];
                        out_val[dst] = stage_val[(t0 + k) * kOpqStage + j];
                    }
                }
            } else {
                const int slot = atomicAdd(&s_novf, 1);
                s_ovf_tile[slot] = threadIdx.x * PER + k;
                s_ovf_off[slot] = rel;
            }
        }
        rel += c[k];
    }
    __syncthreads();
    const int novf = s_novf;
    for (int s = warp; s < novf; s += 8) {
        const int64_t tile = (int64_t)blockIdx.x * kOpqChunk + s_ovf_tile[s];
        const int64_t idx = tile * kOpqTile + lane * kLaneW;
        float v[kLaneW];
        widen((idx < n) ? load_raw<DT>(w, idx) : zero_raw<DT>(), v);
        const unsigned o = outlier_bits(v, outlier_threshold_one_warp<DT, I>(w, tile, tau, lane, v));
        int total;
        int pos = warp_excl_scan(__popc(o), lane, total);
#pragma unroll
        for (int k = 0; k < kLaneW; ++k)
            if ((o >> k) & 1u) {
                const int64_t dst = base + s_ovf_off[s] + pos;
                if (dst < capacity) {
                    out_idx[dst] = (int32_t)(idx + k);
                    out_val[dst] = (uint16_t)bf16_rne(v[k]);
                }
                ++pos;
            }
    }
}

}  // namespace bof4

// ================================================================= launchers (C ABI)

namespace {

using namespace bof4;

// ================================================================= ragged last block
//
// A tensor whose size is not a multiple of the block size ends in a shorter block.  It is handled
// by one CTA with plain loops (fewer than 4096 weights): the same arithmetic as the streaming
// kernels, written out element by element.  The block is its own unit: its own maximum, its own
// mean and deviation over its own length; the two tree sums pad it with zeros to the next power
// of two (neighbours first, as everywhere); a code byte with a single weight has a zero low nibble.

constexpr int kTailThreads = 256;

template <class DT>
__device__ __forceinline__ float tail_load(const void* w, int64_t k);
template <>
__device__ __forceinline__ float tail_load<F32>(const void* w, int64_t k)
{
    return static_cast<const float*>(w)[k];
}
template <>
__device__ __forceinline__ float tail_load<BF16>(const void* w, int64_t k)
{
    return __uint_as_float((uint32_t)static_cast<const uint16_t*>(w)[k] << 16);
}
template <class DT>
__device__ __forceinline__ void tail_store(void* w, int64_t k, float v);  // v is exact in DT
template <>
__device__ __forceinline__ void tail_store<F32>(void* w, int64_t k, float v)
{
    static_cast<float*>(w)[k] = v;
}
template <>
__device__ __forceinline__ void tail_store<BF16>(void* w, int64_t k, float v)
{
    static_cast<uint16_t*>(w)[k] = (uint16_t)(__float_as_uint(v) >> 16);
}

// Balanced tree sum of s_t[0 .. P), P a power of two, neighbours first; result in s_t[0].
__device__ __forceinline__ void tail_tree_sum(float* s_t, int P)
{
    for (int step = 1; step < P; step <<= 1) {
        __syncthreads();
        for (int i = threadIdx.x * 2 * step; i < P; i += kTailThreads * 2 * step)
            s_t[i] = __fadd_rn(s_t[i], s_t[i + step]);
    }
    __syncthreads();
}

// OPQ: outlier split (Sec. 3.3) of the block, appended to the list after the whole blocks'
// outliers; QUANT: block constant, codes and scale.  first = flat index of the block's first
// weight (a multiple of the block size), len = its length.
template <class DT, bool SIGNED, class ST, bool QUANT, bool OPQ>
__global__ void __launch_bounds__(kTailThreads)
tail_block_kernel(const void* __restrict__ w, int64_t first, int len, const float* __restrict__ levels,
                  float tau, uint8_t* __restrict__ codes, void* __restrict__ scales, int64_t scale_index,
                  void* __restrict__ w_clean, int32_t* __restrict__ out_idx, uint16_t* __restrict__ out_val,
                  int64_t capacity, int64_t* __restrict__ n_out)
{
    __shared__ float s_w[4096], s_t[4096];
    __shared__ unsigned char s_c[4096];
    __shared__ float s_xi[kLevels], s_lv[kLevels];
    __shared__ float s_val;
    const int tid = threadIdx.x;
    for (int i = tid; i < len; i += kTailThreads) s_w[i] = tail_load<DT>(w, first + i);
    __syncthreads();
    if (OPQ) {
        int P = 1;
        while (P < len) P <<= 1;
        for (int i = tid; i < P; i += kTailThreads) s_t[i] = (i < len) ? s_w[i] : 0.0f;
        tail_tree_sum(s_t, P);
        if (tid == 0) s_val = __fdiv_rn(s_t[0], (float)len);
        __syncthreads();
        const float mean = s_val;
        __syncthreads();
        for (int i = tid; i < P; i += kTailThreads) {
            const float d = (i < len) ? __fsub_rn(s_w[i], mean) : 0.0f;
            s_t[i] = __fmul_rn(d, d);
        }
        tail_tree_sum(s_t, P);
        if (tid == 0) {
            // one weight: 0 / 0 = NaN, and nothing compares greater than NaN
            const float thr = __fmul_rn(__fsqrt_rn(__fdiv_rn(s_t[0], (float)(len - 1))), tau);
            int64_t k = *n_out;
            for (int i = 0; i < len; ++i) {
                if (fabsf(s_w[i]) > thr) {
                    if (k < capacity) {
                        out_idx[k] = (int32_t)(first + i);
                        out_val[k] = (uint16_t)bf16_rne(s_w[i]);
                    }
                    ++k;
                    s_w[i] = 0.0f;
                }
            }
            *n_out = k;
        }
        __syncthreads();
        if (w_clean)
            for (int i = tid; i < len; i += kTailThreads) tail_store<DT>(w_clean, first + i, s_w[i]);
    }
    if (QUANT) {
        make_thresholds(levels, s_xi, s_lv, tid);
        if (tid == 0) {
            float best = 0.0f, m = 0.0f;  // largest magnitude, lowest index on ties (Eq. 1 / Eq. 4)
            for (int i = 0; i < len; ++i) {
                const float a = fabsf(s_w[i]);
                if (a > best) {
                    best = a;
                    m = SIGNED ? s_w[i] : a;
                }
            }
            s_val = m;
            store_scale<ST>(scales, scale_index, m);
        }
        __syncthreads();
        const float m = s_val;
        for (int i = tid; i < len; i += kTailThreads) s_c[i] = (unsigned char)region_of(normalise(s_w[i], m), s_xi);
        __syncthreads();
        for (int k = tid; k < (len + 1) / 2; k += kTailThreads)
            codes[first / 2 + k] = (uint8_t)((s_c[2 * k] << 4) | ((2 * k + 1 < len) ? s_c[2 * k + 1] : 0));
    }
}

template <class ST, class OT>
__global__ void __launch_bounds__(kTailThreads)
tail_dequantize_kernel(const uint8_t* __restrict__ codes, const void* __restrict__ scales, int64_t first, int len,
                       int64_t scale_index, const float* __restrict__ levels, void* __restrict__ out)
{
    const float m = load_scale<ST>(scales, scale_index);
    for (int i = threadIdx.x; i < len; i += kTailThreads) {
        const int64_t k = first + i;
        const uint32_t byte = codes[k >> 1];
        const uint32_t c = (k & 1) ? (byte & 15u) : (byte >> 4);
        const float v = __fmul_rn(m, levels[c]);
        if (OT::code == BF16::code)
            static_cast<uint16_t*>(out)[k] = (uint16_t)bf16_rne(v);
        else
            static_cast<float*>(out)[k] = v;
    }
}


int grid_for(int64_t rows, int per_sm)
{
    const int64_t cap = (int64_t)kSMs * per_sm;
    return (int)(rows < 1 ? 1 : (rows < cap ? rows : cap));
}

int check_common(const char* fn, int64_t n, int block_size, bool ragged_ok)
{
    if (n < 0) {
        set_error("%s: n is negative", fn);
        return BOF4_ERR_INVALID_ARG;
    }
    if (!valid_block_size(block_size)) {
        set_error("%s: block_size %d is not a power of two in 32 ... 4096", fn, block_size);
        return BOF4_ERR_SHAPE;
    }
    if (!ragged_ok && n % block_size) {
        set_error("%s: n = %lld is not a multiple of block_size %d", fn, (long long)n, block_size);
        return BOF4_ERR_SHAPE;
    }
    return BOF4_OK;
}

int check_quant_dtypes(const char* fn, int w_dtype, int scale_dtype, int norm)
{
    if (norm != BOF4_NORM_ABS && norm != BOF4_NORM_SIGNED) {
        set_error("%s: norm must be BOF4_NORM_ABS or BOF4_NORM_SIGNED", fn);
        return BOF4_ERR_INVALID_ARG;
    }
    if (w_dtype != BOF4_F32 && w_dtype != BOF4_BF16) {
        set_error("%s: unknown weight dtype %d", fn, w_dtype);
        return BOF4_ERR_DTYPE;
    }
    if (scale_dtype != BOF4_F32 && scale_dtype != BOF4_BF16) {
        set_error("%s: unknown scale dtype %d", fn, scale_dtype);
        return BOF4_ERR_DTYPE;
    }
    if (w_dtype == BOF4_F32 && scale_dtype == BOF4_BF16) {
        set_error("%s: fp32 weights need fp32 scales (the block constant is stored exactly)", fn);
        return BOF4_ERR_DTYPE;
    }
    return BOF4_OK;
}

int check_aligned(const char* fn, const char* what, const void* p)
{
    if (!aligned32(p)) {
        set_error("%s: %s is not 32-byte aligned", fn, what);
        return BOF4_ERR_INVALID_ARG;
    }
    return BOF4_OK;
}

// Expand the body with I_, SG, DT, ST bound to the compile-time configuration.
#define BOF4_DISPATCH_I(I_VAL, ...)                    \
    switch (I_VAL) {                                   \
        case 32: { constexpr int I_ = 32; __VA_ARGS__; } break;   \
        case 64: { constexpr int I_ = 64; __VA_ARGS__; } break;   \
        case 128: { constexpr int I_ = 128; __VA_ARGS__; } break; \
        case 256: { constexpr int I_ = 256; __VA_ARGS__; } break; \
        case 512: { constexpr int I_ = 512; __VA_ARGS__; } break; \
        case 1024: { constexpr int I_ = 1024; __VA_ARGS__; } break; \
        case 2048: { constexpr int I_ = 2048; __VA_ARGS__; } break; \
        default: { constexpr int I_ = 4096; __VA_ARGS__; } break;  \
    }
#define BOF4_DISPATCH_BOOL(FLAG, NAME, ...)                \
    if (FLAG) { constexpr bool NAME = true; __VA_ARGS__; } \
    else { constexpr bool NAME = false; __VA_ARGS__; }
#define BOF4_DISPATCH_ST(SD, ...)                        \
    if ((SD) == BOF4_BF16) { using ST = BF16; __VA_ARGS__; } \
    else { using ST = F32; __VA_ARGS__; }
// (weight dtype, scale dtype) in {(f32,f32), (bf16,bf16), (bf16,f32)}
#define BOF4_DISPATCH_WS(WD, SD, ...)                                               \
    if ((WD) == BOF4_F32) { using DT = F32; using ST = F32; __VA_ARGS__; }          \
    else if ((SD) == BOF4_BF16) { using DT = BF16; using ST = BF16; __VA_ARGS__; }  \
    else { using DT = BF16; using ST = F32; __VA_ARGS__; }

}  // namespace

extern "C" int bof4_quantize(const void* d_w, int w_dtype, int64_t n, int block_size, int norm,
                             const float* d_codebook, uint8_t* d_codes, void* d_scales,
                             int scale_dtype, void* stream)
{
    int rc = check_common("bof4_quantize", n, block_size, true);
    if (rc) return rc;
    rc = check_quant_dtypes("bof4_quantize", w_dtype, scale_dtype, norm);
    if (rc) return rc;
    if (n == 0) return BOF4_OK;
    if (!d_w || !d_codebook || !d_codes || !d_scales) {
        set_error("bof4_quantize: NULL pointer");
        return BOF4_ERR_INVALID_ARG;
    }
    if ((rc = check_aligned("bof4_quantize", "d_w", d_w)) || (rc = check_aligned("bof4_quantize", "d_codes", d_codes)))
        return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int tail = (int)(n % block_size);  // a ragged last block goes to its own small kernel
    const int64_t n_whole = n - tail;
    n = n_whole;
    if (n > 0) {
        if (w_dtype == BOF4_BF16) {
            const int grid = grid_for((n + kQRow32 - 1) / kQRow32, kQCtasPerSm);
            BOF4_DISPATCH_ST(scale_dtype,
                BOF4_DISPATCH_I(block_size,
                    BOF4_DISPATCH_BOOL(norm == BOF4_NORM_SIGNED, SG,
                        { constexpr auto kern = quantize32_kernel<I_, SG, ST>;
                          if ((rc = ensure_dynamic_smem<kern>(kLutBytes))) return rc;
                          kern<<<grid, kQThreads, kLutBytes, st>>>(d_w, n, d_codebook, d_codes, d_scales); })));
        } else {
            const int grid = grid_for((n + kQRow - 1) / kQRow, kQCtasPerSm);
            BOF4_DISPATCH_I(block_size,
                BOF4_DISPATCH_BOOL(norm == BOF4_NORM_SIGNED, SG,
                    { constexpr auto kern = quantize_kernel<F32, I_, SG, F32>;
                      if ((rc = ensure_dynamic_smem<kern>(kLutBytes))) return rc;
                      kern<<<grid, kQThreads, kLutBytes, st>>>(d_w, n, d_codebook, d_codes, d_scales); }));
        }
        BOF4_CUDA_TRY(cudaGetLastError());
    }
    if (tail) {
        BOF4_DISPATCH_WS(w_dtype, scale_dtype,
            BOF4_DISPATCH_BOOL(norm == BOF4_NORM_SIGNED, SG,
                (tail_block_kernel<DT, SG, ST, true, false><<<1, kTailThreads, 0, st>>>(
                    d_w, n_whole, tail, d_codebook, 0.0f, d_codes, d_scales, n_whole / block_size, nullptr, nullptr,
                    nullptr, 0, nullptr))));
        BOF4_CUDA_TRY(cudaGetLastError());
    }
    return BOF4_OK;
}

extern "C" int bof4_dequantize(const uint8_t* d_codes, const void* d_scales, int scale_dtype,
                               int64_t n, int block_size, const float* d_codebook,
                               const int32_t* d_out_idx, const void* d_out_val,
                               const int64_t* d_n_out, int64_t capacity, void* d_out,
                               int out_dtype, void* stream)
{
    int rc = check_common("bof4_dequantize", n, block_size, true);
    if (rc) return rc;
    if ((scale_dtype != BOF4_F32 && scale_dtype != BOF4_BF16) ||
        (out_dtype != BOF4_F32 && out_dtype != BOF4_BF16)) {
        set_error("bof4_dequantize: unknown dtype");
        return BOF4_ERR_DTYPE;
    }
    const bool opq = d_out_idx != nullptr;
    if (opq && (!d_out_val || !d_n_out)) {
        set_error("bof4_dequantize: outlier list needs d_out_idx, d_out_val and d_n_out together");
        return BOF4_ERR_INVALID_ARG;
    }
    if (opq && capacity < 0) {
        set_error("bof4_dequantize: negative capacity");
        return BOF4_ERR_CAPACITY;
    }
    if (n == 0) return BOF4_OK;
    if (!d_codes || !d_scales || !d_codebook || !d_out) {
        set_error("bof4_dequantize: NULL pointer");
        return BOF4_ERR_INVALID_ARG;
    }
    if ((rc = check_aligned("bof4_dequantize", "d_codes", d_codes)) || (rc = check_aligned("bof4_dequantize", "d_out", d_out)))
        return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int tail = (int)(n % block_size);  // a ragged last block goes to its own small kernel
    const int64_t n_whole = n - tail;
    const int64_t rows = (n_whole + kDRow - 1) / kDRow;
    const int grid = grid_for(rows, kDCtasPerSm);
#define BOF4_DEQ(ST_, OT_)                                                                                   \
    {                                                                                                        \
        if (n_whole > 0)                                                                                     \
            BOF4_DISPATCH_I(block_size, {                                                                    \
                constexpr auto kern = dequantize_kernel<ST_, OT_, I_>;                                       \
                if ((rc = ensure_dynamic_smem<kern>(kDTableBytes))) return rc;                               \
                kern<<<grid, kDThreads, kDTableBytes, st>>>(d_codes, d_scales, n_whole, d_codebook, d_out); })  \
        if (tail)                                                                                            \
            tail_dequantize_kernel<ST_, OT_><<<1, kTailThreads, 0, st>>>(d_codes, d_scales, n_whole, tail,   \
                                                                         n_whole / block_size, d_codebook, d_out); \
    }
    if (scale_dtype == BOF4_F32 && out_dtype == BOF4_F32) { BOF4_DEQ(F32, F32) }
    else if (scale_dtype == BOF4_F32) { BOF4_DEQ(F32, BF16) }
    else if (out_dtype == BOF4_F32) { BOF4_DEQ(BF16, F32) }
    else { BOF4_DEQ(BF16, BF16) }
#undef BOF4_DEQ
    BOF4_CUDA_TRY(cudaGetLastError());
    if (opq && capacity > 0) {
        const uint16_t* val = static_cast<const uint16_t*>(d_out_val);
        if (out_dtype == BOF4_F32)
            scatter_outliers_kernel<F32><<<kSMs, 256, 0, st>>>(d_out_idx, val, d_n_out, capacity, n, d_out);
        else
            scatter_outliers_kernel<BF16><<<kSMs, 256, 0, st>>>(d_out_idx, val, d_n_out, capacity, n, d_out);
        BOF4_CUDA_TRY(cudaGetLastError());
    }
    return BOF4_OK;
}

// Many tensors per launch.  bf16 weights whose whole blocks go through the batch kernels, kQBatch
// tensors per launch; fp32 weights and short last blocks take the single-tensor path.
extern "C" int bof4_quantize_batch(const void* const* h_w, const int64_t* h_n, int n_tensors, int w_dtype,
                                   int block_size, int norm, const float* d_codebook, uint8_t* const* h_codes,
                                   void* const* h_scales, int scale_dtype, void* stream)
{
    const char* fn = "bof4_quantize_batch";
    if (n_tensors < 0 || (n_tensors > 0 && (!h_w || !h_n || !h_codes || !h_scales))) {
        set_error("%s: bad tensor list", fn);
        return BOF4_ERR_INVALID_ARG;
    }
    int rc = check_quant_dtypes(fn, w_dtype, scale_dtype, norm);
    if (rc) return rc;
    if (!d_codebook) {
        set_error("%s: NULL codebook", fn);
        return BOF4_ERR_INVALID_ARG;
    }
    for (int t = 0; t < n_tensors; ++t) {
        if ((rc = check_common(fn, h_n[t], block_size, true))) return rc;
        if (h_n[t] == 0) continue;
        if (!h_w[t] || !h_codes[t] || !h_scales[t]) {
            set_error("%s: tensor %d has a NULL pointer", fn, t);
            return BOF4_ERR_INVALID_ARG;
        }
        if ((rc = check_aligned(fn, "a weight tensor", h_w[t])) || (rc = check_aligned(fn, "a code array", h_codes[t])))
            return rc;
    }
    if (w_dtype != BOF4_BF16) {
        for (int t = 0; t < n_tensors; ++t)
            if ((rc = bof4_quantize(h_w[t], w_dtype, h_n[t], block_size, norm, d_codebook, h_codes[t], h_scales[t],
                                    scale_dtype, stream)))
                return rc;
        return BOF4_OK;
    }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    QuantBatch B;
    B.count = 0;
    int64_t rows = 0;
    const int G = kSMs * kQCtasPerSm;
    for (int t = 0; t <= n_tensors; ++t) {
        if (t < n_tensors) {
            const int64_t n_whole = h_n[t] - h_n[t] % block_size;
            if (n_whole > 0) {
                B.w[B.count] = h_w[t];
                B.codes[B.count] = h_codes[t];
                B.scales[B.count] = h_scales[t];
                B.n[B.count] = n_whole;
                B.start[B.count] = (int)(rows % G);
                rows += (n_whole + kQRow32 - 1) / kQRow32;
                ++B.count;
            }
        }
        if (B.count == kQBatch || (t == n_tensors && B.count > 0)) {
            BOF4_DISPATCH_ST(scale_dtype,
                BOF4_DISPATCH_I(block_size,
                    BOF4_DISPATCH_BOOL(norm == BOF4_NORM_SIGNED, SG,
                        { constexpr auto kern = quantize32_batch_kernel<I_, SG, ST>;
                          if ((rc = ensure_dynamic_smem<kern>(kLutBytes))) return rc;
                          kern<<<G, kQThreads, kLutBytes, st>>>(B, d_codebook); })));
            BOF4_CUDA_TRY(cudaGetLastError());
            B.count = 0;
        }
    }
    for (int t = 0; t < n_tensors; ++t) {
        const int tail = (int)(h_n[t] % block_size);
        if (!tail) continue;
        const int64_t n_whole = h_n[t] - tail;
        BOF4_DISPATCH_ST(scale_dtype,
            BOF4_DISPATCH_BOOL(norm == BOF4_NORM_SIGNED, SG,
                (tail_block_kernel<BF16, SG, ST, true, false><<<1, kTailThreads, 0, st>>>(
                    h_w[t], n_whole, tail, d_codebook, 0.0f, h_codes[t], h_scales[t], n_whole / block_size, nullptr,
                    nullptr, nullptr, 0, nullptr))));
        BOF4_CUDA_TRY(cudaGetLastError());
    }
    return BOF4_OK;
}

extern "C" int bof4_dequantize_batch(const uint8_t* const* h_codes, const void* const* h_scales, int scale_dtype,
                                     const int64_t* h_n, int n_tensors, int block_size, const float* d_codebook,
                                     void* const* h_out, int out_dtype, void* stream)
{
    const char* fn = "bof4_dequantize_batch";
    if (n_tensors < 0 || (n_tensors > 0 && (!h_codes || !h_scales || !h_n || !h_out))) {
        set_error("%s: bad tensor list", fn);
        return BOF4_ERR_INVALID_ARG;
    }
    if ((scale_dtype != BOF4_F32 && scale_dtype != BOF4_BF16) || (out_dtype != BOF4_F32 && out_dtype != BOF4_BF16)) {
        set_error("%s: unknown dtype", fn);
        return BOF4_ERR_DTYPE;
    }
    if (!d_codebook) {
        set_error("%s: NULL codebook", fn);
        return BOF4_ERR_INVALID_ARG;
    }
    int rc;
    for (int t = 0; t < n_tensors; ++t) {
        if ((rc = check_common(fn, h_n[t], block_size, true))) return rc;
        if (h_n[t] == 0) continue;
        if (!h_codes[t] || !h_scales[t] || !h_out[t]) {
            set_error("%s: tensor %d has a NULL pointer", fn, t);
            return BOF4_ERR_INVALID_ARG;
        }
        if ((rc = check_aligned(fn, "a code array", h_codes[t])) || (rc = check_aligned(fn, "an output tensor", h_out[t])))
            return rc;
    }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    DequantBatch B;
    B.count = 0;
    int64_t rows = 0;
    const int G = kSMs * kDCtasPerSm;
    for (int t = 0; t <= n_tensors; ++t) {
        if (t < n_tensors) {
            const int64_t n_whole = h_n[t] - h_n[t] % block_size;
            if (n_whole > 0) {
                B.codes[B.count] = h_codes[t];
                B.scales[B.count] = h_scales[t];
                B.out[B.count] = h_out[t];
                B.n[B.count] = n_whole;
                B.start[B.count] = (int)(rows % G);
                rows += (n_whole + kDRow - 1) / kDRow;
                ++B.count;
            }
        }
        if (B.count == kQBatch || (t == n_tensors && B.count > 0)) {
#define BOF4_DEQB(ST_, OT_) BOF4_DISPATCH_I(block_size, {                                  \
        constexpr auto kern = dequantize_batch_kernel<ST_, OT_, I_>;                       \
        if ((rc = ensure_dynamic_smem<kern>(kDTableBytes))) return rc;                     \
        kern<<<G, kDThreads, kDTableBytes, st>>>(B, d_codebook); })
            if (scale_dtype == BOF4_F32 && out_dtype == BOF4_F32) { BOF4_DEQB(F32, F32) }
            else if (scale_dtype == BOF4_F32) { BOF4_DEQB(F32, BF16) }
            else if (out_dtype == BOF4_F32) { BOF4_DEQB(BF16, F32) }
            else { BOF4_DEQB(BF16, BF16) }
#undef BOF4_DEQB
            BOF4_CUDA_TRY(cudaGetLastError());
            B.count = 0;
        }
    }
    for (int t = 0; t < n_tensors; ++t) {
        const int tail = (int)(h_n[t] % block_size);
        if (!tail) continue;
        const int64_t n_whole = h_n[t] - tail;
#define BOF4_DEQT(ST_, OT_) tail_dequantize_kernel<ST_, OT_><<<1, kTailThreads, 0, st>>>( \
        h_codes[t], h_scales[t], n_whole, tail, n_whole / block_size, d_codebook, h_out[t]);
        if (scale_dtype == BOF4_F32 && out_dtype == BOF4_F32) { BOF4_DEQT(F32, F32) }
        else if (scale_dtype == BOF4_F32) { BOF4_DEQT(F32, BF16) }
        else if (out_dtype == BOF4_F32) { BOF4_DEQT(BF16, F32) }
        else { BOF4_DEQT(BF16, BF16) }
#undef BOF4_DEQT
        BOF4_CUDA_TRY(cudaGetLastError());
    }
    return BOF4_OK;
}

namespace {

// Shared launcher of opq_split (QUANT = false) and bof4_quantize_opq (QUANT = true).
template <bool QUANT>
int launch_opq(const char* fn, const void* d_w, int w_dtype, int64_t n, int block_size, int norm,
               const float* d_codebook, float tau, uint8_t* d_codes, void* d_scales, int scale_dtype,
               void* d_w_clean, int32_t* d_out_idx, void* d_out_val, int64_t capacity,
               int64_t* d_n_out, void* d_ws, size_t ws_bytes, void* stream, bool ragged_ok = true)
{
    int rc = check_common(fn, n, block_size, ragged_ok);
    if (rc) return rc;
    rc = check_quant_dtypes(fn, w_dtype, scale_dtype, norm);
    if (rc) return rc;
    if (n >= ((int64_t)1 << 31)) {
        set_error("%s: n must be below 2^31 (int32 outlier indices)", fn);
        return BOF4_ERR_SHAPE;
    }
    if (capacity < 0 || capacity >= ((int64_t)1 << 31)) {
        set_error("%s: capacity out of range", fn);
        return BOF4_ERR_CAPACITY;
    }
    if (!(tau >= 0.0f)) {
        set_error("%s: tau must be a non-negative number", fn);
        return BOF4_ERR_INVALID_ARG;
    }
    if (!d_n_out || (capacity > 0 && (!d_out_idx || !d_out_val))) {
        set_error("%s: NULL outlier output", fn);
        return BOF4_ERR_INVALID_ARG;
    }
    const OpqLayout L = opq_layout(n);
    if (!d_ws || ((uintptr_t)d_ws & 255u) || ws_bytes < L.total) {
        set_error("%s: workspace NULL, not 256-byte aligned, or smaller than %zu bytes", fn, L.total);
        return BOF4_ERR_WORKSPACE;
    }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (n == 0) {
        BOF4_CUDA_TRY(cudaMemsetAsync(d_n_out, 0, sizeof(int64_t), st));
        return BOF4_OK;
    }
    if (!d_w || (QUANT && (!d_codebook || !d_codes || !d_scales))) {
        set_error("%s: NULL pointer", fn);
        return BOF4_ERR_INVALID_ARG;
    }
    if ((rc = check_aligned(fn, "d_w", d_w)) || (rc = check_aligned(fn, "d_codes", d_codes)) ||
        (rc = check_aligned(fn, "d_w_clean", d_w_clean)))
        return rc;
    char* ws = static_cast<char*>(d_ws);
    int32_t* counts = reinterpret_cast<int32_t*>(ws + L.counts);
    unsigned long long* chunk_sum = reinterpret_cast<unsigned long long*>(ws + L.chunk_off);
    int32_t* stage_idx = reinterpret_cast<int32_t*>(ws + L.stage_idx);
    uint16_t* stage_val = reinterpret_cast<uint16_t*>(ws + L.stage_val);
    uint16_t* out_val = static_cast<uint16_t*>(d_out_val);
    const int tail = (int)(n % block_size);  // a ragged last block goes to its own small kernel
    const int64_t n_whole = n - tail;
    if (n_whole == 0) {
        BOF4_CUDA_TRY(cudaMemsetAsync(d_n_out, 0, sizeof(int64_t), st));
    } else {
        const OpqLayout Lw = opq_layout(n_whole);  // never larger than the layout of n
        const int64_t rows = (n_whole + kQRow - 1) / kQRow;
        const int grid = grid_for(rows, kQCtasPerSm);
        const int smem = QUANT ? kLutBytes : 0;
        counts = reinterpret_cast<int32_t*>(ws + Lw.counts);
        chunk_sum = reinterpret_cast<unsigned long long*>(ws + Lw.chunk_off);
        stage_idx = reinterpret_cast<int32_t*>(ws + Lw.stage_idx);
        stage_val = reinterpret_cast<uint16_t*>(ws + Lw.stage_val);
        BOF4_CUDA_TRY(cudaMemsetAsync(chunk_sum, 0, (size_t)Lw.chunks * 8, st));
        if (w_dtype == BOF4_BF16) {
            const int grid32 = grid_for((n_whole + kQRow32 - 1) / kQRow32, kQCtasPerSm);
            BOF4_DISPATCH_ST(scale_dtype,
                BOF4_DISPATCH_I(block_size,
                    BOF4_DISPATCH_BOOL(norm == BOF4_NORM_SIGNED, SG,
                        { constexpr auto kern = opq_pass1_32_kernel<I_, SG, ST, QUANT>;
                          if ((rc = ensure_dynamic_smem<kern>(kLutBytes))) return rc;
                          kern<<<grid32, kQThreads, smem, st>>>(d_w, n_whole, d_codebook, tau, d_codes, d_scales,
                                                                d_w_clean, counts, chunk_sum, stage_idx, stage_val); })));
        } else {
            BOF4_DISPATCH_I(block_size,
                BOF4_DISPATCH_BOOL(norm == BOF4_NORM_SIGNED, SG,
                    { constexpr auto kern = opq_pass1_kernel<F32, I_, SG, F32, QUANT>;
                      if ((rc = ensure_dynamic_smem<kern>(kLutBytes))) return rc;
                      kern<<<grid, kQThreads, smem, st>>>(d_w, n_whole, d_codebook, tau, d_codes, d_scales, d_w_clean,
                                                          counts, chunk_sum, stage_idx, stage_val); }));
        }
        BOF4_CUDA_TRY(cudaGetLastError());
        if (w_dtype == BOF4_F32) {
            BOF4_DISPATCH_I(block_size, (opq_gather_kernel<F32, I_><<<(int)Lw.chunks, 256, 0, st>>>(
                d_w, n_whole, tau, counts, Lw.tiles, chunk_sum, stage_idx, stage_val, d_out_idx, out_val, capacity,
                d_n_out)));
        } else {
            BOF4_DISPATCH_I(block_size, (opq_gather_kernel<BF16, I_><<<(int)Lw.chunks, 256, 0, st>>>(
                d_w, n_whole, tau, counts, Lw.tiles, chunk_sum, stage_idx, stage_val, d_out_idx, out_val, capacity,
                d_n_out)));
        }
        BOF4_CUDA_TRY(cudaGetLastError());
    }
    if (tail) {  // after the gather kernel: its outliers follow those of the whole blocks
        BOF4_DISPATCH_WS(w_dtype, scale_dtype,
            BOF4_DISPATCH_BOOL(norm == BOF4_NORM_SIGNED, SG,
                (tail_block_kernel<DT, SG, ST, QUANT, true><<<1, kTailThreads, 0, st>>>(
                    d_w, n_whole, tail, d_codebook, tau, d_codes, d_scales, n_whole / block_size, d_w_clean, d_out_idx,
                    out_val, capacity, d_n_out))));
        BOF4_CUDA_TRY(cudaGetLastError());
    }
    return BOF4_OK;
}

}  // namespace

extern "C" int opq_split(const void* d_w, int w_dtype, int64_t n, int block_size, float tau,
                         void* d_w_clean, int32_t* d_out_idx, void* d_out_val, int64_t capacity,
                         int64_t* d_n_out, void* d_ws, size_t ws_bytes, void* stream)
{
    return launch_opq<false>("opq_split", d_w, w_dtype, n, block_size, BOF4_NORM_ABS, nullptr, tau,
                             nullptr, nullptr, w_dtype, d_w_clean, d_out_idx, d_out_val, capacity,
                             d_n_out, d_ws, ws_bytes, stream);
}

extern "C" int bof4_quantize_opq(const void* d_w, int w_dtype, int64_t n, int block_size, int norm,
                                 const float* d_codebook, float tau, uint8_t* d_codes,
                                 void* d_scales, int scale_dtype, int32_t* d_out_idx,
                                 void* d_out_val, int64_t capacity, int64_t* d_n_out, void* d_ws,
                                 size_t ws_bytes, void* stream)
{
    return launch_opq<true>("bof4_quantize_opq", d_w, w_dtype, n, block_size, norm, d_codebook, tau,
                            d_codes, d_scales, scale_dtype, nullptr, d_out_idx, d_out_val, capacity,
                            d_n_out, d_ws, ws_bytes, stream);
}

// ================================================================= allocation-free outlier split

namespace {

// Scratch of opq_split_static: the tile counts, chunk offsets and staging slots that opq_split
// otherwise takes from the caller's workspace.  It lives in the library image, so every GPU
// that loads the library holds these 4 MiB until the process exits.
constexpr int64_t kStaticMaxN = (int64_t)1 << 24;
constexpr size_t kStaticScratchBytes = (size_t)4 << 20;
static __device__ __align__(256) unsigned char g_opq_static_scratch[kStaticScratchBytes];

constexpr int kMaxDevices = 64;
std::mutex g_static_mutex;
void* g_static_ptr[kMaxDevices] = {};

// Device address of the scratch array on the current device.  The array's name is only a
// host-side handle; the address a kernel may use comes from cudaGetSymbolAddress, once per
// device, with that device current.
int static_scratch(void** out)
{
    int dev = -1;
    BOF4_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) {
        set_error("opq_split_static: device ordinal %d is outside 0..%d", dev, kMaxDevices - 1);
        return BOF4_ERR_INVALID_ARG;
    }
    std::lock_guard<std::mutex> lock(g_static_mutex);
    if (!g_static_ptr[dev]) {
        void* p = nullptr;
        BOF4_CUDA_TRY(cudaGetSymbolAddress(&p, g_opq_static_scratch));
        g_static_ptr[dev] = p;
    }
    *out = g_static_ptr[dev];
    return BOF4_OK;
}

}  // namespace

// Whole blocks only (n % block_size == 0); the remembered scratch address does not survive a
// cudaDeviceReset of its device.
extern "C" int opq_split_static(const void* d_w, int w_dtype, int64_t n, int block_size, float tau,
                                void* d_w_clean, int32_t* d_out_idx, void* d_out_val,
                                int64_t capacity, int64_t* d_n_out, void* stream)
{
    if (n > kStaticMaxN) {
        set_error("opq_split_static: n = %lld exceeds the built-in scratch (at most %lld weights per "
                  "call; use opq_split with a workspace for larger tensors)",
                  (long long)n, (long long)kStaticMaxN);
        return BOF4_ERR_SHAPE;
    }
    if (n >= 0 && opq_layout(n).total > kStaticScratchBytes) {
        set_error("opq_split_static: internal scratch too small for n = %lld", (long long)n);
        return BOF4_ERR_WORKSPACE;
    }
    void* scratch = nullptr;
    const int rc = static_scratch(&scratch);
    if (rc) return rc;
    return launch_opq<false>("opq_split_static", d_w, w_dtype, n, block_size, BOF4_NORM_ABS, nullptr, tau,
                             nullptr, nullptr, w_dtype, d_w_clean, d_out_idx, d_out_val, capacity,
                             d_n_out, scratch, kStaticScratchBytes, stream, false);
}
