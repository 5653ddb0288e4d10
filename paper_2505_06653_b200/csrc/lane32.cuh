// bfloat16 front end of the streaming kernels: 64 bytes per lane.
//
// For bf16 weights one lane owns kLW = 32 consecutive weights (two 32-byte loads), so a block of
// I <= 1024 weights is I / 32 neighbouring lanes of one warp (one lane for I = 32) and a block of
// 2048 / 4096 weights is 2 / 4 neighbouring warps; one warp iteration covers 1024 weights.  Twice
// the weights per lane halve everything that is paid per lane and row (block reduction,
// reciprocal, row bookkeeping, stores), which is what bounds these kernels.
//
// Three ways to the region of a weight (Sec. 2.1 Eq. 2 + Sec. 3.2), chosen per warp row:
//   FAST   x~ = RN(w * RN(1/m)), one packed multiplication per two weights, then the one-probe
//          table search.  x~ differs from the true quotient RN(w/m) by at most a few units in
//          the last place, which only matters if a decision threshold lies that close to a
//          quotient the data can take.  Both operands have 8-bit significands, so for a given
//          significand of m the possible quotients are a small set that can be enumerated: at
//          table-build time every (threshold, significand of m) pair is checked, and a block
//          whose constant has a significand marked "near" does not take this path
//          (near_mask).  Thresholds of magnitude below 2^-90 (zero included) switch the path off for the
//          whole launch, because then the rounding of subnormal quotients would matter.
//   EXACT  the reciprocal sequence of normalise16 (the IEEE quotient for every normal result),
//          its guard for tiny quotients, and the table search.
//   SLOW   IEEE division and binary search: rows with a zero, non-finite or extreme block
//          constant, and codebooks the table cannot serve.
// All three give the same codes: the code of RN(w/m) against the fp32 thresholds.
#pragma once

#include "common.cuh"

namespace bof4 {

constexpr int kLW = 32;              // bf16 weights per lane and row
constexpr int kWarpW32 = 32 * kLW;   // weights per warp iteration

struct Raw32 {
    Raw8 a, b;  // weights 0..15 and 16..31 of the lane, two per word, lower index in the low half
};

// idx = element index of the lane's first weight (a multiple of 32).
__device__ __forceinline__ Raw32 load_raw32(const void* base, int64_t idx)
{
    const uint16_t* p = static_cast<const uint16_t*>(base) + idx;
    return Raw32{ld_stream256(p), ld_stream256(p + 16)};
}
__device__ __forceinline__ Raw32 zero_raw32()
{
    Raw32 r;
#pragma unroll
    for (int k = 0; k < 8; ++k) r.a.u[k] = r.b.u[k] = 0u;
    return r;
}
__device__ __forceinline__ void words_of(const Raw32& r, uint32_t (&u)[16])
{
#pragma unroll
    for (int k = 0; k < 8; ++k) {
        u[k] = r.a.u[k];
        u[8 + k] = r.b.u[k];
    }
}
__device__ __forceinline__ float bf_lo(uint32_t u) { return __uint_as_float(u << 16); }
__device__ __forceinline__ float bf_hi(uint32_t u) { return __uint_as_float(u & 0xffff0000u); }

template <int I>
struct Geo32 {
    static constexpr int LPB = (I >= kWarpW32) ? 32 : I / kLW;   // lanes of a warp per block
    static constexpr int WPB = (I >= kWarpW32) ? I / kWarpW32 : 1;  // warps per block
};

__device__ __forceinline__ uint32_t max_nan_bf16x2(uint32_t a, uint32_t b)
{
    uint32_t d;
    asm("max.NaN.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}
__device__ __forceinline__ uint32_t min_bf16x2(uint32_t a, uint32_t b)
{
    uint32_t d;
    asm("min.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}

// Largest (NaN-propagating) and smallest of the lane's 32 weights, two at a time.
__device__ __forceinline__ void lane_minmax32(const uint32_t (&u)[16], float& mx, float& mn)
{
    uint32_t x2 = max_nan_bf16x2(u[0], u[1]), n2 = min_bf16x2(u[0], u[1]);
#pragma unroll
    for (int k = 2; k < 16; ++k) {
        x2 = max_nan_bf16x2(x2, u[k]);
        n2 = min_bf16x2(n2, u[k]);
    }
    mx = max2_nan(bf_lo(x2), bf_hi(x2));
    mn = fminf(bf_lo(n2), bf_hi(n2));
}

// The lane's first weight of magnitude g (0 if none), in index order.
__device__ __forceinline__ float first_of_magnitude(const uint32_t (&u)[16], float g)
{
    float first = 0.0f;
#pragma unroll
    for (int k = 15; k >= 0; --k) {
        first = (fabsf(bf_hi(u[k])) == g) ? bf_hi(u[k]) : first;
        first = (fabsf(bf_lo(u[k])) == g) ? bf_lo(u[k]) : first;
    }
    return first;
}

// Block constant (Eq. 1 / Eq. 4) of the lane group (or warp group) that owns the block; the same
// contract as block_constant: all 32 lanes call it (all threads of the CTA for blocks wider than
// a warp), g receives the block's largest magnitude or NaN, an all-zero block gives +0, and the
// signed constant takes the lowest index on ties.
template <int I, bool SIGNED>
__device__ __forceinline__ float block_constant32(const uint32_t (&u)[16], float mx, float mn, float& g,
                                                  WideScratch* ws)
{
    constexpr int LPB = Geo32<I>::LPB, WPB = Geo32<I>::WPB;
    float gx = mx, gn = mn;
#pragma unroll
    for (int off = 1; off < LPB; off <<= 1) {
        gx = max2_nan(gx, __shfl_xor_sync(kFull, gx, off));
        gn = fminf(gn, __shfl_xor_sync(kFull, gn, off));
    }
    if constexpr (WPB > 1) {
        gx = across_warps<WPB>(gx, ws->a, [](float p, float q) { return max2_nan(p, q); });
        gn = across_warps<WPB>(gn, ws->b, [](float p, float q) { return fminf(p, q); });
    }
    g = max2_nan(gx, -gn);
    if (!SIGNED) return g;
    float m = (gx > -gn) ? gx : gn;
    const bool tie = (gx == -gn) && (g != 0.0f);
    const int lane = threadIdx.x & 31;
    if constexpr (WPB == 1) {
        if (__any_sync(kFull, tie)) {
            const int base = lane & ~(LPB - 1);
            const unsigned gmask = (LPB == 32) ? kFull : (((1u << (LPB & 31)) - 1u) << base);
            const unsigned hp = __ballot_sync(kFull, mx == g) & gmask;   // lanes holding +g
            const unsigned hn = __ballot_sync(kFull, mn == -g) & gmask;  // lanes holding -g
            const int lp = __ffs(hp) - 1, ln = __ffs(hn) - 1;            // -1: none
            const float first = first_of_magnitude(u, g);
            const int src = (lp >= 0 && (ln < 0 || lp <= ln)) ? lp : ln;  // lane of the block's first +-g
            const float pick = __shfl_sync(kFull, first, src < 0 ? 0 : src);
            if (tie) m = pick;
        }
    } else {
        if (__syncthreads_or(tie ? 1 : 0)) {
            const float first = first_of_magnitude(u, g);
            const unsigned has = __ballot_sync(kFull, fmaxf(mx, -mn) == g);
            const int src = __ffs(has) - 1;  // -1: this warp holds no +-g
            const float val = __shfl_sync(kFull, first, src < 0 ? 0 : src);
            const int warp = threadIdx.x >> 5;
            if (lane == 0) {
                ws->pos[warp] = src;
                ws->a[warp] = val;
            }
            __syncthreads();
            const int base = warp & ~(WPB - 1);
            float pick = 0.0f;
#pragma unroll
            for (int k = WPB - 1; k >= 0; --k) pick = (ws->pos[base + k] >= 0) ? ws->a[base + k] : pick;
            __syncthreads();
            if (tie) m = pick;
        }
    }
    return (g == 0.0f) ? 0.0f : m;
}

// ---------------------------------------------------------------- which significands of m are "near"
//
// bf16 values are a * 2^e with an integer a < 256, so for a block constant with significand
// b (128..255) every quotient is (a / b) * 2^j.  A threshold xi is "near" for b when some a in
// 128..255 (any j) has | a / b - |xi| 2^-j | <= 2^-20 |xi| 2^-j: with X the 24-bit significand
// of |xi|, a 2^s = X b up to that tolerance, s being the shift that brings X b into [128, 256).
// x~ and RN(w/m) are both within 2^-23 (relative) of the true quotient, so outside this set no
// threshold separates them.  near_mask: bit (b - 128) of a 128-bit mask, four words.
struct FastInfo {
    uint32_t near_mask[4];
    int tiny;  // some threshold has magnitude below 2^-90 (zero included): FAST is off
};

// One bin of the near-significand test: threshold index j, significand b.
__device__ __forceinline__ void mark_if_near(const float* s_xi, int j, int b, FastInfo* s_info)
{
    const uint32_t xb = __float_as_uint(s_xi[j]) & 0x7fffffffu;
    if (xb >= 0x7f800000u || xb < 0x12800000u) return;  // not finite, or below 2^-90 (see tiny)
    const uint32_t X = (xb & 0x7fffffu) | 0x800000u;       // 24-bit significand
    const uint32_t P = X * (uint32_t)b;                    // < 2^32, >= 2^30
    const int s = (P >> 31) ? 24 : 23;                     // P >> s in [128, 256)
    const uint32_t frac = P & ((1u << s) - 1u), tol = 1u << (s - 12);   // 2^-20 relative, rounded up
    if (frac <= tol || frac >= (1u << s) - tol) atomicOr(&s_info->near_mask[(b - 128) >> 5], 1u << ((b - 128) & 31));
}

// Everything a quantising kernel derives from the codebook, in two barriers: thresholds and
// levels (s_xi, s_lv), the one-probe region table (s_lut, [bin][lane] replicated REP times;
// payload(base) beside every threshold) and the FAST-path information.  Every thread derives
// the thresholds and their table bins itself from the 16 levels, so that the table entries, the
// "two thresholds in one bin" test and the "tiny threshold" test need no exchange.  Returns
// whether the table can serve the codebook.  Call with all threads of the CTA (>= 257).
template <int REP = 32, class PayloadFn>
__device__ __forceinline__ bool build_tables32(const float* __restrict__ levels, float* s_xi, float* s_lv,
                                               unsigned char* s_lut, FastInfo* s_info, PayloadFn payload)
{
    __shared__ uint2 s_ent[kLutBins];
    const int tid = threadIdx.x;
    float lv[kLevels], xi[kLevels];
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        const float4 t = __ldg(reinterpret_cast<const float4*>(levels) + q);
        lv[4 * q] = t.x;
        lv[4 * q + 1] = t.y;
        lv[4 * q + 2] = t.z;
        lv[4 * q + 3] = t.w;
    }
    int bin[kLevels - 1];
    bool multi = false, tiny = false;
#pragma unroll
    for (int j = 0; j < kLevels - 1; ++j) {
        xi[j] = __fmul_rn(__fadd_rn(lv[j], lv[j + 1]), 0.5f);
        const int bj = (int)(__float_as_uint(lut_key(xi[j])) - kLutMagicBits);
        bin[j] = bj < 0 ? 0 : (bj > kLutBins - 1 ? kLutBins - 1 : bj);
        tiny = tiny || fabsf(xi[j]) < 0x1p-90f;
        if (j > 0) multi = multi || bin[j] == bin[j - 1];   // ascending thresholds: equal bins are adjacent
    }
    xi[kLevels - 1] = __int_as_float(0x7f800000);
    if (tid < kLutBins) {
        int base = 0;
#pragma unroll
        for (int j = 0; j < kLevels - 1; ++j) base += (bin[j] < tid) ? 1 : 0;
        float thr = xi[kLevels - 1];
#pragma unroll
        for (int j = kLevels - 2; j >= 0; --j) thr = (base == j) ? xi[j] : thr;
        s_ent[tid] = make_uint2(__float_as_uint(thr), payload(base));
    }
    if (tid < kLevels) {
        float a = xi[kLevels - 1], l = lv[kLevels - 1];
#pragma unroll
        for (int j = kLevels - 2; j >= 0; --j) {
            a = (tid == j) ? xi[j] : a;
            l = (tid == j) ? lv[j] : l;
        }
        s_xi[tid] = a;
        s_lv[tid] = l;
    }
    if (tid < 4) s_info->near_mask[tid] = 0u;
    if (tid == 4) s_info->tiny = tiny ? 1 : 0;
    __syncthreads();
    for (int k = tid; k < kLutBins * REP; k += blockDim.x)
        *reinterpret_cast<uint2*>(s_lut + k * 8) = s_ent[k / REP];
    for (int t = tid; t < (kLevels - 1) * 128; t += blockDim.x) mark_if_near(s_xi, t >> 7, 128 + (t & 127), s_info);
    __syncthreads();
    return !multi;
}

// The significand of the block constant m is one for which FAST could disagree with the quotient.
__device__ __forceinline__ bool near_significand(float m, const FastInfo* s_info)
{
    const uint32_t b = (__float_as_uint(m) >> 16) & 127u;
    return (s_info->near_mask[b >> 5] >> (b & 31)) & 1u;
}

// ---------------------------------------------------------------- codes of a lane's 32 weights
//
// Each of the four result words packs eight codes, even element in the high nibble of its byte:
// Horner steps w = 16 w + code over the weights 6 7 4 5 2 3 0 1 of the word.

// wd = 16 wd + base + (x >= thr): one multiply-add, one comparison, one predicated increment.
__device__ __forceinline__ uint32_t horner_code(uint32_t wd, float x, uint2 entry)
{
    asm("{\n\t.reg .pred p;\n\t"
        "mad.lo.u32 %0, %0, 16, %2;\n\t"
        "setp.ge.f32 p, %1, %3;\n\t"
        "@p add.u32 %0, %0, 1;\n\t}"
        : "+r"(wd)
        : "f"(x), "r"(entry.y), "f"(__uint_as_float(entry.x)));
    return wd;
}

template <bool REFINE>
__device__ __forceinline__ void encode32_lut(const uint32_t (&u)[16], float m, uint32_t lut_base, uint32_t (&cw)[4])
{
    const float r = __frcp_rn(m);  // m != 0: the caller passes 1 for lanes without data
    const float2 rr = make_float2(r, r), nm = make_float2(-m, -m);
#pragma unroll
    for (int h = 0; h < 4; ++h) {
        uint32_t wd = 0u;
#pragma unroll
        for (int j = 3; j >= 0; --j) {
            const uint32_t uu = u[4 * h + j];
            const float2 v = make_float2(bf_lo(uu), bf_hi(uu));
            float2 x = __fmul2_rn(v, rr);
            if (REFINE) {
                const float2 e = __ffma2_rn(x, nm, v);
                x = __ffma2_rn(e, rr, x);
                // quotients below 2^-100: one rounding of the subnormal result
                if (fabsf(x.x) < 0x1p-100f && v.x != 0.0f) x.x = __fdiv_rn(v.x, m);
                if (fabsf(x.y) < 0x1p-100f && v.y != 0.0f) x.y = __fdiv_rn(v.y, m);
            }
            const float2 key = lut_key2(x);
            const uint2 e0 = lut_probe(key.x, lut_base), e1 = lut_probe(key.y, lut_base);
            wd = horner_code(wd, x.x, e0);
            wd = horner_code(wd, x.y, e1);
        }
        cw[h] = wd;
    }
}

// IEEE division and binary search; any input.  Kept out of line (the words travel by value) so
// that the rare path costs the common ones neither registers nor code size.
__device__ __noinline__ uint4 encode32_slow_words(uint4 q0, uint4 q1, uint4 q2, uint4 q3, float m, const float* s_xi)
{
    const uint32_t u[16] = {q0.x, q0.y, q0.z, q0.w, q1.x, q1.y, q1.z, q1.w,
                            q2.x, q2.y, q2.z, q2.w, q3.x, q3.y, q3.z, q3.w};
    uint32_t cw[4];
#pragma unroll
    for (int h = 0; h < 4; ++h) {
        uint32_t wd = 0u;
#pragma unroll
        for (int j = 3; j >= 0; --j) {
            const uint32_t uu = u[4 * h + j];
            wd = wd * 16u + (uint32_t)region_of(normalise(bf_lo(uu), m), s_xi);
            wd = wd * 16u + (uint32_t)region_of(normalise(bf_hi(uu), m), s_xi);
        }
        cw[h] = wd;
    }
    return make_uint4(cw[0], cw[1], cw[2], cw[3]);
}
__device__ __forceinline__ void encode32_slow(const uint32_t (&u)[16], float m, const float* s_xi, uint32_t (&cw)[4])
{
    const uint4 c = encode32_slow_words(make_uint4(u[0], u[1], u[2], u[3]), make_uint4(u[4], u[5], u[6], u[7]),
                                        make_uint4(u[8], u[9], u[10], u[11]), make_uint4(u[12], u[13], u[14], u[15]),
                                        m, s_xi);
    cw[0] = c.x;
    cw[1] = c.y;
    cw[2] = c.z;
    cw[3] = c.w;
}

// Which way a warp row takes (warp-uniform).  g: the lane's block maximum (or NaN); ok: the lane
// holds data (a lane without data must hold zeros and is encoded with m = 1); lut_ok: the
// codebook fits the one-probe table.  An all-zero block sends its row the slow way.
enum RowPath { kPathFast = 0, kPathExact = 1, kPathSlow = 2 };

__device__ __forceinline__ int row_path(float g, float m, bool ok, bool lut_ok, const FastInfo* s_info)
{
    const bool safe = div_safe(g) || !ok;
    if (!lut_ok || !__all_sync(kFull, safe)) return kPathSlow;
    if (s_info->tiny) return kPathExact;
    return __any_sync(kFull, ok && near_significand(m, s_info)) ? kPathExact : kPathFast;
}

// Rows of `row` consecutive weights over a tensor of n weights (n a multiple of 32); the calling
// thread owns 32 weights at offset tid * 32 of every row.  Only the last row can be partial.
struct RowMap32 {
    int rows, rows_full, row;
    int tid_off;
    bool tail_ok;
    __device__ __forceinline__ RowMap32(int64_t n, int row_, int tid)
        : rows((int)((n + row_ - 1) / row_)), rows_full((int)(n / row_)), row(row_), tid_off(tid * kLW),
          tail_ok((int64_t)(n / row_) * row_ + tid * kLW < n)
    {
    }
    __device__ __forceinline__ bool ok(int r) const { return r < rows_full || (r < rows && tail_ok); }
    __device__ __forceinline__ int64_t idx(int r) const { return (int64_t)r * row + tid_off; }
};

}  // namespace bof4
