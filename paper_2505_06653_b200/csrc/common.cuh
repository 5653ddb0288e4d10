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

}  // namespace bof4
