// Shared device helpers of the BOF4 kernels: 16-byte weight loads, block constant (Eq. 1 / Eq. 4),
// normalisation (Eq. 2), region search (Sec. 3.2), plus the host-side status plumbing.
//
// Work layout used by every streaming kernel: one lane owns 8 consecutive weights (one 16-byte
// load for bf16, two for fp32), so a block of I weights is owned by LPB = I / 8 neighbouring
// lanes of one warp (4, 8, 16 or 32 lanes) and every per-block reduction is a shuffle butterfly
// inside that lane group.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/bof4.h"

namespace bof4 {

constexpr int kLevels = 16;
constexpr unsigned kFull = 0xffffffffu;
constexpr int kSMs = 148;  // B200: grids are sized in multiples of this

// ---------------------------------------------------------------- host status plumbing

void set_error(const char* fmt, ...);
int cuda_fail(cudaError_t e, const char* what);

#define BOF4_CUDA_TRY(expr)                                         \
    do {                                                            \
        cudaError_t e__ = (expr);                                   \
        if (e__ != cudaSuccess) return ::bof4::cuda_fail(e__, #expr); \
    } while (0)

inline bool valid_block_size(int I) { return I == 32 || I == 64 || I == 128 || I == 256; }

// ---------------------------------------------------------------- loads

struct F32 {
    using scalar = float;
    static constexpr int code = BOF4_F32;
};
struct BF16 {
    using scalar = uint16_t;
    static constexpr int code = BOF4_BF16;
};

__device__ __forceinline__ uint4 ld_stream(const uint4* p)
{
    uint4 r;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w)
                 : "l"(p));
    return r;
}

// 8 consecutive weights starting at element index idx (idx a multiple of 8), widened to fp32.
template <class DT>
__device__ __forceinline__ void load8(const void* base, int64_t idx, float (&v)[8]);

template <>
__device__ __forceinline__ void load8<BF16>(const void* base, int64_t idx, float (&v)[8])
{
    const uint4 q = ld_stream(reinterpret_cast<const uint4*>(static_cast<const uint16_t*>(base) + idx));
    const uint32_t u[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        v[2 * k] = __uint_as_float(u[k] << 16);
        v[2 * k + 1] = __uint_as_float(u[k] & 0xffff0000u);
    }
}

template <>
__device__ __forceinline__ void load8<F32>(const void* base, int64_t idx, float (&v)[8])
{
    const uint4* p = reinterpret_cast<const uint4*>(static_cast<const float*>(base) + idx);
    const uint4 a = ld_stream(p), b = ld_stream(p + 1);
    v[0] = __uint_as_float(a.x); v[1] = __uint_as_float(a.y);
    v[2] = __uint_as_float(a.z); v[3] = __uint_as_float(a.w);
    v[4] = __uint_as_float(b.x); v[5] = __uint_as_float(b.y);
    v[6] = __uint_as_float(b.z); v[7] = __uint_as_float(b.w);
}

template <class DT>
__device__ __forceinline__ void zero8(float (&v)[8])
{
#pragma unroll
    for (int k = 0; k < 8; ++k) v[k] = 0.0f;
}

// fp32 -> bf16 bits, round to nearest even (finite inputs).
__device__ __forceinline__ uint32_t bf16_rne(float f)
{
    const uint32_t u = __float_as_uint(f);
    return (u + 0x7fffu + ((u >> 16) & 1u)) >> 16;
}

// ---------------------------------------------------------------- block constant

template <int LPB>
__device__ __forceinline__ float group_max(float a)
{
#pragma unroll
    for (int off = 1; off < LPB; off <<= 1) a = fmaxf(a, __shfl_xor_sync(kFull, a, off));
    return a;
}

// Block constant of the lane group that owns the block.  SIGNED = false: max |w| (Eq. 1).
// SIGNED = true: the element of largest magnitude with its sign, lowest index on ties (Eq. 4).
// An all-zero block gives +0.  Must be called by all 32 lanes.
template <int LPB, bool SIGNED>
__device__ __forceinline__ float block_constant(const float (&v)[8])
{
    float a = fmaxf(fmaxf(fmaxf(fabsf(v[0]), fabsf(v[1])), fmaxf(fabsf(v[2]), fabsf(v[3]))),
                    fmaxf(fmaxf(fabsf(v[4]), fabsf(v[5])), fmaxf(fabsf(v[6]), fabsf(v[7]))));
    const float g = group_max<LPB>(a);
    if (!SIGNED) return g;
    float cand = v[7];
#pragma unroll
    for (int j = 6; j >= 0; --j) cand = (fabsf(v[j]) == a) ? v[j] : cand;
    const unsigned hit = __ballot_sync(kFull, a == g);
    const int lane = threadIdx.x & 31;
    const int base = lane & ~(LPB - 1);
    const unsigned grp = (LPB == 32) ? hit : ((hit >> base) & ((1u << LPB) - 1u));
    const int src = base + __ffs(grp) - 1;
    const float m = __shfl_sync(kFull, cand, src);
    return (g == 0.0f) ? 0.0f : m;
}

// Eq. 2 with the 0/0 reading x = 0.  IEEE round-to-nearest division.
__device__ __forceinline__ float normalise(float w, float m)
{
    return (m == 0.0f) ? 0.0f : __fdiv_rn(w, m);
}

// ---------------------------------------------------------------- region search

// Decision thresholds from the levels: fp32 add, then exact halving; xi[15] = +inf pads the
// table so that the search never reads past it.
__device__ __forceinline__ void make_thresholds(const float* __restrict__ levels, float* s_xi,
                                                float* s_lv, int tid)
{
    if (tid < kLevels) {
        s_lv[tid] = levels[tid];
        s_xi[tid] = (tid < kLevels - 1) ? __fmul_rn(__fadd_rn(levels[tid], levels[tid + 1]), 0.5f)
                                        : __int_as_float(0x7f800000);
    }
}

// Number of thresholds <= x, by binary search over the ascending table (4 probes).
__device__ __forceinline__ int region_of(float x, const float* s_xi)
{
    int c = (x >= s_xi[7]) ? 8 : 0;
    c += (x >= s_xi[c + 3]) ? 4 : 0;
    c += (x >= s_xi[c + 1]) ? 2 : 0;
    c += (x >= s_xi[c]) ? 1 : 0;
    return c;
}

// ---------------------------------------------------------------- one-probe region search
//
// The interval [-1, 1] of normalised weights is cut into 257 bins by the monotone map
//     bin(x) = bits(fma(x, 128, 1.5 * 2^23 + 128)) - bits(1.5 * 2^23)  =  RN(128 x) + 128,
// and a table gives, per bin, base = the number of thresholds that fall into LOWER bins and
// thr = xi[base] (xi[15] = +inf).  Because bin() is monotone, every threshold in a lower bin
// is <= x and every threshold in a higher bin is > x, so when no bin holds two thresholds
//     region(x) = base + (x >= thr)
// exactly.  A codebook with two thresholds in one bin (levels closer than 1/128) makes the
// kernels fall back to the binary search.  Each table row is replicated for the 32 lanes
// ([bin][lane], 8 bytes each) so that the shared-memory bank only depends on the lane.
constexpr int kLutBins = 257;
constexpr uint32_t kLutMagicBits = 0x4B400000u;  // bits of 1.5 * 2^23
constexpr int kLutRowBytes = 32 * 8;
constexpr int kLutBytes = kLutBins * kLutRowBytes;

__device__ __forceinline__ float lut_key(float x) { return fmaf(x, 128.0f, 12583040.0f); }

// Byte offset of the lane's table entry for normalised weight x; key = lut_key(x).  The
// unsigned minimum also sends NaN / infinite keys (non-finite input) to the last row.
__device__ __forceinline__ uint32_t lut_offset(float key, uint32_t lane_off)
{
    const uint32_t b = min(__float_as_uint(key), kLutMagicBits + (uint32_t)(kLutBins - 1));
    return b * (uint32_t)kLutRowBytes + (lane_off - kLutMagicBits * (uint32_t)kLutRowBytes);
}

// Builds the table in shared memory from the thresholds; payload[base] is stored next to
// thr (a code, or a byte offset).  Returns through *s_multi whether some bin holds two
// thresholds.  Call with all threads of the CTA, then __syncthreads().
template <class PayloadFn>
__device__ __forceinline__ void build_lut(const float* s_xi, unsigned char* s_lut, int* s_multi,
                                          PayloadFn payload)
{
    if (threadIdx.x == 0) *s_multi = 0;
    __syncthreads();
    for (int b = threadIdx.x; b < kLutBins; b += blockDim.x) {
        int base = 0, inside = 0;
#pragma unroll
        for (int j = 0; j < kLevels - 1; ++j) {
            int bj = (int)(__float_as_uint(lut_key(s_xi[j])) - kLutMagicBits);
            bj = bj < 0 ? 0 : (bj > kLutBins - 1 ? kLutBins - 1 : bj);
            base += (bj < b) ? 1 : 0;
            inside += (bj == b) ? 1 : 0;
        }
        if (inside > 1) *s_multi = 1;
        const uint2 ent = make_uint2(__float_as_uint(s_xi[base]), payload(base));
        for (int l = 0; l < 32; ++l)
            *reinterpret_cast<uint2*>(s_lut + b * kLutRowBytes + l * 8) = ent;
    }
}

// ---------------------------------------------------------------- division for bf16 inputs
//
// For bfloat16 operands with 2^-60 <= |m| <= 2^60 the sequence
//     r = RN(1/m);  q0 = RN(w r);  e = fma(-q0, m, w);  q = fma(e, r, q0)
// returns exactly RN(w / m) whenever the quotient is a normal number (checked exhaustively
// over all operand pairs on the CPU by the test-suite).  It costs three (packed) operations
// per weight plus one reciprocal per block.
__device__ __forceinline__ bool div_safe(float m)
{
    const float a = fabsf(m);
    return a >= 0x1p-60f && a <= 0x1p60f;
}

__device__ __forceinline__ float2 fast_div2(float2 w, float m, float r)
{
    const float2 rr = make_float2(r, r), nm = make_float2(-m, -m);
    const float2 q0 = __fmul2_rn(w, rr);
    const float2 e = __ffma2_rn(q0, nm, w);
    return __ffma2_rn(e, rr, q0);
}

// x[k] = RN(v[k] / m) for the 8 weights of a lane (x = 0 when m = 0).  FAST selects the
// reciprocal sequence (bf16 operands only; the caller has checked div_safe for the whole
// warp).  With GUARD, quotients below 2^-100 in magnitude are recomputed by the IEEE
// division so that subnormal results are rounded once.
template <bool FAST, bool GUARD>
__device__ __forceinline__ void normalise8(const float (&v)[8], float m, float (&x)[8])
{
    if (FAST) {
        const float r = __frcp_rn(m);
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const float2 q = fast_div2(make_float2(v[2 * k], v[2 * k + 1]), m, r);
            x[2 * k] = q.x;
            x[2 * k + 1] = q.y;
        }
        if (GUARD) {
            const float lo = fminf(fminf(fminf(fabsf(x[0]), fabsf(x[1])), fminf(fabsf(x[2]), fabsf(x[3]))),
                                   fminf(fminf(fabsf(x[4]), fabsf(x[5])), fminf(fabsf(x[6]), fabsf(x[7]))));
            if (lo < 0x1p-100f) {
#pragma unroll
                for (int k = 0; k < 8; ++k)
                    if (fabsf(x[k]) < 0x1p-100f && v[k] != 0.0f) x[k] = normalise(v[k], m);
            }
        }
    } else {
#pragma unroll
        for (int k = 0; k < 8; ++k) x[k] = normalise(v[k], m);
    }
}

}  // namespace bof4
