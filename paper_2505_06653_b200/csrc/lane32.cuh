// bfloat16 front end of the streaming kernels: 64 bytes per lane.
//
// For bf16 weights one lane owns kLW = 32 consecutive weights (two 32-byte loads), so a block of
// I <= 1024 weights is I / 32 neighbouring lanes of one warp (one lane for I = 32) and a block of
// 2048 / 4096 weights is 2 / 4 neighbouring warps; one warp iteration covers 1024 weights.  Twice
// the weights per lane halve everything that is paid per lane and row (block reduction,
// reciprocal, row bookkeeping, stores), which is what bounds these kernels.
//
// Two ways to the region of a weight (Sec. 2.1 Eq. 2 + Sec. 3.2), chosen per warp row:
//   FAST   x~ = RN(w * RN(1/m)), one packed multiplication per two weights, then the one-probe
//          table search against thresholds LOWERED by three floating-point steps (xi' = the third
//          fp32 number below xi).  With q = w/m: x~ lies within 2.01 * 2^-24 (relative) of q, and
//          RN(q) >= xi  <=>  q >= xi up to rounding in the last place, so
//              q >= xi                   =>  x~ >= xi'      (x~ > xi (1 - 2.01 * 2^-24) > xi'),
//              q <  xi - 9 * 2^-24 |xi|  =>  x~ <  xi'  and  RN(q) < xi,
//          i.e. the comparison x~ >= xi' decides exactly like RN(w/m) >= xi unless q falls into
//          the narrow window just below xi (and a quotient less than half a step below xi rounds
//          to xi and has x~ >= xi' as well).  Both operands have 8-bit significands, so for a
//          given significand of m the quotients are a small set: at table-build time every
//          (threshold, significand of m) pair is checked, and a block whose constant has a
//          significand with a quotient in some window ("near") takes the other way.  A quotient
//          that equals a threshold, or whose fp32 rounding does (codebooks with dyadic or other
//          simple rational levels), is decided correctly here.
//          Thresholds of magnitude below 2^-90 (zero included) switch the path off for the whole
//          launch: the rounding of subnormal quotients would matter.
//   SLOW   the true quotient RN(w/m) (reciprocal sequence with its guard where it is proven,
//          IEEE division elsewhere) against the true thresholds by binary search: "near" rows,
//          rows with a zero, non-finite or extreme block constant, partial rows, and codebooks
//          the table cannot serve.
// Both give the same codes: the code of RN(w/m) against the fp32 thresholds.
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
// b (128..255) every quotient has magnitude (a / b) * 2^j.  With X the 24-bit significand of
// |xi|, P = X b = a_real * 2^s for the s that brings a_real into [128, 256); one unit of P is
// 1 / b of a unit in the last place of xi.  The quotient with numerator a = floor(a_real)
// (xi > 0: slightly smaller magnitude) or ceil(a_real) (xi < 0: slightly larger) lies
// dist = frac(P) resp. 2^s - frac(P) units of P below xi.  FAST decides like the true quotient
//   * for dist < b / 4: the quotient is less than a quarter step below xi, RN(q) = xi and
//     x~ > xi' (this is the case of codebooks with rational levels, whose thresholds are fp32
//     roundings of quotients the data takes);
//   * for dist > 9 * 2^-24 P: the quotient is more than 9 * 2^-24 |xi| below xi.
// In between the significand is marked (upper bound rounded up to 16 * 2^-24 P).
// near_mask: bit (b - 128) of a 128-bit mask.
struct FastInfo {
    uint32_t near_mask[4];
    int tiny;  // some threshold has magnitude below 2^-90 (zero included): FAST is off
};

// One bin of the near-significand test: threshold index j, significand b.
__device__ __forceinline__ void mark_if_near(const float* s_xi, int j, int b, FastInfo* s_info)
{
    const uint32_t bits = __float_as_uint(s_xi[j]), xb = bits & 0x7fffffffu;
    if (xb >= 0x7f800000u || xb < 0x12800000u) return;  // not finite, or below 2^-90 (see tiny)
    const uint32_t X = (xb & 0x7fffffu) | 0x800000u;       // 24-bit significand
    const uint32_t P = X * (uint32_t)b;                    // < 2^32, >= 2^30
    const int s = (P >> 31) ? 24 : 23;                     // P >> s in [128, 256)
    const uint32_t frac = P & ((1u << s) - 1u);
    const uint32_t dist = (bits >> 31) ? ((1u << s) - frac) & ((1u << s) - 1u) : frac;  // distance into the window side
    const bool near = 4u * dist >= (uint32_t)b && dist <= (P >> 20);
    if (near) atomicOr(&s_info->near_mask[(b - 128) >> 5], 1u << ((b - 128) & 31));
}

// The third fp32 number below x (finite, |x| >= 2^-90: no zero crossing).
__device__ __forceinline__ float three_steps_down(float x)
{
    const uint32_t u = __float_as_uint(x);
    return __uint_as_float((u >> 31) ? u + 3u : u - 3u);
}

// Everything a quantising kernel derives from the codebook, in two barriers: the true thresholds
// and the levels (s_xi, s_lv), the one-probe region table of the FAST path over the LOWERED
// thresholds (s_lut, [bin][lane] replicated REP times; payload(base) beside every threshold) and
// the FAST-path information.  Every thread derives
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
    float lo[kLevels];  // lowered thresholds (table side)
    int bin[kLevels - 1];
    bool multi = false, tiny = false;
#pragma unroll
    for (int j = 0; j < kLevels - 1; ++j) {
        xi[j] = __fmul_rn(__fadd_rn(lv[j], lv[j + 1]), 0.5f);
        const bool usable = fabsf(xi[j]) >= 0x1p-90f && fabsf(xi[j]) < __int_as_float(0x7f800000);
        tiny = tiny || !(fabsf(xi[j]) >= 0x1p-90f);
        lo[j] = usable ? three_steps_down(xi[j]) : xi[j];
        const int bj = (int)(__float_as_uint(lut_key(lo[j])) - kLutMagicBits);
        bin[j] = bj < 0 ? 0 : (bj > kLutBins - 1 ? kLutBins - 1 : bj);
        if (j > 0) multi = multi || bin[j] == bin[j - 1];   // ascending thresholds: equal bins are adjacent
    }
    xi[kLevels - 1] = lo[kLevels - 1] = __int_as_float(0x7f800000);
    if (tid < kLutBins) {
        int base = 0;
#pragma unroll
        for (int j = 0; j < kLevels - 1; ++j) base += (bin[j] < tid) ? 1 : 0;
        float thr = lo[kLevels - 1];
#pragma unroll
        for (int j = kLevels - 2; j >= 0; --j) thr = (base == j) ? lo[j] : thr;
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

// FAST path: m != 0, every |w| <= |m|, so every x~ is a finite number in [-1, 1].
__device__ __forceinline__ void encode32_fast(const uint32_t (&u)[16], float m, uint32_t lut_base, uint32_t (&cw)[4])
{
    const float r = __frcp_rn(m);
    const float2 rr = make_float2(r, r);
#pragma unroll
    for (int h = 0; h < 4; ++h) {
        uint32_t wd = 0u;
#pragma unroll
        for (int j = 3; j >= 0; --j) {
            const uint32_t uu = u[4 * h + j];
            const float2 x = __fmul2_rn(make_float2(bf_lo(uu), bf_hi(uu)), rr);
            const float2 key = lut_key2(x);
            const uint2 e0 = lut_probe(key.x, lut_base), e1 = lut_probe(key.y, lut_base);
            wd = horner_code(wd, x.x, e0);
            wd = horner_code(wd, x.y, e1);
        }
        cw[h] = wd;
    }
}

// The quotients RN(v / m) of two weights for the SLOW path: the reciprocal sequence of
// normalise16 with its guard where it is proven (recip: |m| in [2^-60, 2^60], r = RN(1/m)),
// IEEE division otherwise (x = 0 when m = 0).
__device__ __forceinline__ float2 exact_quotient2(float2 v, float m, float r, bool recip)
{
    if (!recip) return make_float2(normalise(v.x, m), normalise(v.y, m));
    const float2 rr = make_float2(r, r), nm = make_float2(-m, -m);
    float2 x = __fmul2_rn(v, rr);
    const float2 e = __ffma2_rn(x, nm, v);
    x = __ffma2_rn(e, rr, x);
    if (fabsf(x.x) < 0x1p-100f && v.x != 0.0f) x.x = __fdiv_rn(v.x, m);  // subnormal results: one rounding
    if (fabsf(x.y) < 0x1p-100f && v.y != 0.0f) x.y = __fdiv_rn(v.y, m);
    return x;
}

// SLOW path: true quotients against the true thresholds by binary search; any input.  Kept out
// of line (the words travel by value) so that it costs the common path neither registers nor
// code size.
static __device__ __noinline__ uint4 encode32_slow_words(uint4 q0, uint4 q1, uint4 q2, uint4 q3, float m, const float* s_xi)
{
    const uint32_t u[16] = {q0.x, q0.y, q0.z, q0.w, q1.x, q1.y, q1.z, q1.w,
                            q2.x, q2.y, q2.z, q2.w, q3.x, q3.y, q3.z, q3.w};
    const bool recip = div_safe(fabsf(m));
    const float r = recip ? __frcp_rn(m) : 0.0f;
    uint32_t cw[4];
#pragma unroll
    for (int h = 0; h < 4; ++h) {
        uint32_t wd = 0u;
#pragma unroll
        for (int j = 3; j >= 0; --j) {
            const uint32_t uu = u[4 * h + j];
            const float2 x = exact_quotient2(make_float2(bf_lo(uu), bf_hi(uu)), m, r, recip);
            wd = wd * 16u + (uint32_t)region_of(x.x, s_xi);
            wd = wd * 16u + (uint32_t)region_of(x.y, s_xi);
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

// Warp-uniform: the row takes the FAST path.  g: the lane's block maximum (or NaN), m its block
// constant; ok: the lane holds data; fast_ok: the table serves the codebook and no threshold is
// tiny.  A zero, extreme or non-finite block constant, a "near" significand or a lane without
// data send the row the slow way.
__device__ __forceinline__ bool row_is_fast(float g, float m, bool ok, bool fast_ok, const FastInfo* s_info)
{
    return fast_ok && __all_sync(kFull, ok && div_safe(g) && !near_significand(m, s_info));
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
