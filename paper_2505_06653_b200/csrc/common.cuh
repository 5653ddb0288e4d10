// Shared device helpers of the BOF4 kernels: 32-byte weight loads, block constant (Eq. 1 / Eq. 4),
// normalisation (Eq. 2), region search (Sec. 3.2), plus the host-side status plumbing.
//
// Work layout used by every streaming kernel: one lane owns kLaneW = 16 consecutive weights
// (one 32-byte load for bf16, two for fp32), so a block of I <= 512 weights is owned by
// LPB = I / 16 neighbouring lanes of one warp and every per-block reduction is a shuffle
// butterfly inside that lane group; a block of 1024 ... 4096 weights is owned by 2 ... 8
// neighbouring warps of one CTA, which exchange their per-warp results through shared memory.
// One warp iteration covers kWarpW = 512 consecutive weights.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>

#include "../../include/bof4.h"

namespace bof4 {

constexpr int kLevels = 16;
constexpr unsigned kFull = 0xffffffffu;
constexpr int kSMs = 148;  // B200: grids are sized in multiples of this
constexpr int kLaneW = 16;
constexpr int kWarpW = 32 * kLaneW;

// ---------------------------------------------------------------- host status plumbing

void set_error(const char* fmt, ...);
int cuda_fail(cudaError_t e, const char* what);

#define BOF4_CUDA_TRY(expr)                                         \
    do {                                                            \
        cudaError_t e__ = (expr);                                   \
        if (e__ != cudaSuccess) return ::bof4::cuda_fail(e__, #expr); \
    } while (0)

// Raises the dynamic shared-memory limit of kernel Kern to `bytes`, once per device and kernel
// instantiation (the attribute belongs to the function on the current device), so that the
// per-iteration launch path makes no attribute call.
template <auto Kern>
inline int ensure_dynamic_smem(int bytes)
{
    static std::atomic<unsigned long long> done{0ull};
    int dev = 0;
    BOF4_CUDA_TRY(cudaGetDevice(&dev));
    const unsigned long long bit = (dev >= 0 && dev < 64) ? (1ull << dev) : 0ull;
    if (bit && (done.load(std::memory_order_acquire) & bit)) return BOF4_OK;
    BOF4_CUDA_TRY(cudaFuncSetAttribute(Kern, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes));
    if (bit) done.fetch_or(bit, std::memory_order_release);
    return BOF4_OK;
}

inline bool valid_block_size(int I) { return I >= 32 && I <= 4096 && (I & (I - 1)) == 0; }
inline bool aligned32(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 31u) == 0; }

// ---------------------------------------------------------------- loads and stores

struct F32 {
    static constexpr int code = BOF4_F32;
};
struct BF16 {
    static constexpr int code = BOF4_BF16;
};

struct Raw8 {
    uint32_t u[8];
};

// 32 bytes, read once: no L1 allocation.
__device__ __forceinline__ Raw8 ld_stream256(const void* p)
{
    Raw8 r;
    asm volatile("ld.global.nc.L1::no_allocate.v8.u32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(r.u[0]), "=r"(r.u[1]), "=r"(r.u[2]), "=r"(r.u[3]), "=r"(r.u[4]), "=r"(r.u[5]),
                   "=r"(r.u[6]), "=r"(r.u[7])
                 : "l"(p));
    return r;
}
__device__ __forceinline__ void st_stream256(void* p, const Raw8& r)
{
    asm volatile("st.global.cs.v8.u32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"l"(p), "r"(r.u[0]), "r"(r.u[1]),
                 "r"(r.u[2]), "r"(r.u[3]), "r"(r.u[4]), "r"(r.u[5]), "r"(r.u[6]), "r"(r.u[7])
                 : "memory");
}
__device__ __forceinline__ void st_stream128(void* p, uint32_t a, uint32_t b, uint32_t c, uint32_t d)
{
    asm volatile("st.global.cs.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}
__device__ __forceinline__ void st_stream64(void* p, uint32_t a, uint32_t b)
{
    asm volatile("st.global.cs.v2.u32 [%0], {%1,%2};" ::"l"(p), "r"(a), "r"(b) : "memory");
}

// The raw bits of the 16 weights of a lane, as loaded (1 or 2 vectors of 32 bytes).
template <class DT>
struct RawRow;
template <>
struct RawRow<BF16> {
    Raw8 a;
};
template <>
struct RawRow<F32> {
    Raw8 a, b;
};

// idx = element index of the lane's first weight (a multiple of 16).
template <class DT>
__device__ __forceinline__ RawRow<DT> load_raw(const void* base, int64_t idx);
template <>
__device__ __forceinline__ RawRow<BF16> load_raw<BF16>(const void* base, int64_t idx)
{
    return RawRow<BF16>{ld_stream256(static_cast<const uint16_t*>(base) + idx)};
}
template <>
__device__ __forceinline__ RawRow<F32> load_raw<F32>(const void* base, int64_t idx)
{
    const float* p = static_cast<const float*>(base) + idx;
    return RawRow<F32>{ld_stream256(p), ld_stream256(p + 8)};
}

template <class DT>
__device__ __forceinline__ RawRow<DT> zero_raw()
{
    RawRow<DT> r;
#pragma unroll
    for (int k = 0; k < 8; ++k) r.a.u[k] = 0u;
    if constexpr (DT::code == BOF4_F32) {
#pragma unroll
        for (int k = 0; k < 8; ++k) r.b.u[k] = 0u;
    }
    return r;
}

// Widening to fp32 (exact).
__device__ __forceinline__ void widen(const RawRow<BF16>& r, float (&v)[kLaneW])
{
#pragma unroll
    for (int k = 0; k < 8; ++k) {
        v[2 * k] = __uint_as_float(r.a.u[k] << 16);
        v[2 * k + 1] = __uint_as_float(r.a.u[k] & 0xffff0000u);
    }
}
__device__ __forceinline__ void widen(const RawRow<F32>& r, float (&v)[kLaneW])
{
#pragma unroll
    for (int k = 0; k < 8; ++k) {
        v[k] = __uint_as_float(r.a.u[k]);
        v[8 + k] = __uint_as_float(r.b.u[k]);
    }
}

// Rows of `row` consecutive weights (one CTA iteration each) over a tensor of n weights; the
// calling thread owns kLaneW weights at offset tid * kLaneW of every row.  Row indices are
// 32-bit; only the last row can be partial (n is a multiple of the block size, hence of 16).
struct RowMap {
    int rows, rows_full, row;
    int tid_off;
    bool tail_ok;
    __device__ __forceinline__ RowMap(int64_t n, int row_, int tid)
        : rows((int)((n + row_ - 1) / row_)), rows_full((int)(n / row_)), row(row_), tid_off(tid * kLaneW),
          tail_ok((int64_t)(n / row_) * row_ + tid * kLaneW < n)
    {
    }
    __device__ __forceinline__ bool ok(int r) const { return r < rows_full || (r < rows && tail_ok); }
    __device__ __forceinline__ int64_t idx(int r) const { return (int64_t)r * row + tid_off; }
};

// fp32 -> bf16 bits, round to nearest even (finite inputs).
__device__ __forceinline__ uint32_t bf16_rne(float f)
{
    const uint32_t u = __float_as_uint(f);
    return (u + 0x7fffu + ((u >> 16) & 1u)) >> 16;
}

__device__ __forceinline__ float max3(float a, float b, float c)
{
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}
__device__ __forceinline__ float min3(float a, float b, float c)
{
    float d;
    asm("min.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}

// ---------------------------------------------------------------- block constant

__device__ __forceinline__ float max3_nan(float a, float b, float c)
{
    float d;
    asm("max.NaN.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}
__device__ __forceinline__ float max2_nan(float a, float b)
{
    float d;
    asm("max.NaN.f32 %0, %1, %2;" : "=f"(d) : "f"(a), "f"(b));
    return d;
}

// Block constant of the lane group that owns the block.  SIGNED = false: max |w| (Eq. 1).
// SIGNED = true: the element of largest magnitude with its sign, lowest index on ties (Eq. 4).
// An all-zero block gives +0.  Must be called by all 32 lanes.  `g` receives the largest
// magnitude of the block, or NaN if the block holds a NaN (the maximum chain propagates NaN),
// so that one range test on g tells whether every quotient w / m is a finite number in [-1, 1].
//
// The signed constant is found from the block's largest and smallest element: the larger
// magnitude wins.  Only when both +g and -g occur does the position matter; that case is
// settled by two ballots (which lane holds the first +g, which the first -g) and, where one
// lane holds both, by that lane's elements in index order.
// Largest (NaN-propagating) and smallest of the lane's 16 weights.
__device__ __forceinline__ void lane_minmax(const float (&v)[kLaneW], float& mx, float& mn)
{
    mx = max3_nan(v[0], v[1], v[2]);
    mn = min3(v[0], v[1], v[2]);
#pragma unroll
    for (int k = 3; k < 15; k += 2) {
        mx = max3_nan(mx, v[k], v[k + 1]);
        mn = min3(mn, v[k], v[k + 1]);
    }
    mx = max2_nan(mx, v[15]);
    mn = fminf(mn, v[15]);
}

// A block of I weights is LPB lanes of one warp (I <= 512) or WPB whole, neighbouring warps of
// one CTA (I = 1024 ... 4096; CTA rows are multiples of 8192 weights, so blocks never straddle
// CTA rows).  Blocks wider than a warp combine their per-warp results through shared memory.
template <int I>
struct BlockGeo {
    static constexpr int LPB = (I >= kWarpW) ? 32 : I / kLaneW;  // lanes of a warp per block
    static constexpr int WPB = (I >= kWarpW) ? I / kWarpW : 1;   // warps per block
};

// One slot per warp of the CTA for the cross-warp steps of wide blocks.
struct WideScratch {
    float a[32], b[32];
    int pos[32];
};

// Combines one value per warp over the WPB warps of a block, in warp order, with `op`; every
// thread of the CTA must call it.  Two barriers: publish, then protect the slots for reuse.
template <int WPB, class Op>
__device__ __forceinline__ float across_warps(float x, float* slot, Op op)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (lane == 0) slot[warp] = x;
    __syncthreads();
    const int base = warp & ~(WPB - 1);
    float t[WPB];
#pragma unroll
    for (int k = 0; k < WPB; ++k) t[k] = slot[base + k];
#pragma unroll
    for (int step = 1; step < WPB; step <<= 1)  // neighbours first: the order of a balanced tree
#pragma unroll
        for (int k = 0; k < WPB; k += 2 * step) t[k] = op(t[k], t[k + step]);
    __syncthreads();
    return t[0];
}

// Block constant from the lane's largest / smallest weight (lane_minmax).  `ws` is only used
// by blocks wider than a warp (then every thread of the CTA must take part).
template <int I, bool SIGNED>
__device__ __forceinline__ float block_constant(const float (&v)[kLaneW], float mx, float mn, float& g,
                                                WideScratch* ws)
{
    constexpr int LPB = BlockGeo<I>::LPB, WPB = BlockGeo<I>::WPB;
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
            float first = 0.0f;  // this lane's first element of magnitude g
#pragma unroll
            for (int k = kLaneW - 1; k >= 0; --k) first = (fabsf(v[k]) == g) ? v[k] : first;
            const int src = (lp >= 0 && (ln < 0 || lp <= ln)) ? lp : ln;  // lane of the block's first +-g
            const float pick = __shfl_sync(kFull, first, src < 0 ? 0 : src);
            if (tie) m = pick;
        }
    } else {
        if (__syncthreads_or(tie ? 1 : 0)) {
            // every warp reports the position and value of its first element of magnitude g
            float first = 0.0f;
#pragma unroll
            for (int k = kLaneW - 1; k >= 0; --k) first = (fabsf(v[k]) == g) ? v[k] : first;
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

template <int I, bool SIGNED>
__device__ __forceinline__ float block_constant(const float (&v)[kLaneW], float& g, WideScratch* ws)
{
    float mx, mn;
    lane_minmax(v, mx, mn);
    return block_constant<I, SIGNED>(v, mx, mn, g, ws);
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
//
// The table may only be indexed with finite x in [-1, 1]: callers use it for a warp row only
// when every block of the row has a finite, non-zero largest magnitude (row_is_safe), which
// makes every quotient such a number; all other rows take the binary search.
constexpr int kLutBins = 257;
constexpr uint32_t kLutMagicBits = 0x4B400000u;  // bits of 1.5 * 2^23
constexpr float kLutMagic = 12583040.0f;         // 1.5 * 2^23 + 128
// REP = number of lane columns per row: 32 (one per lane) or 16 (lanes L and L + 16 share a
// column; an 8-byte read is served half a warp at a time, so this is conflict-free as well and
// halves the table where shared memory is short).
__host__ __device__ constexpr int lut_row_bytes(int rep) { return rep * 8; }
__host__ __device__ constexpr int lut_bytes(int rep) { return kLutBins * rep * 8; }
constexpr int kLutRowBytes = lut_row_bytes(32);
constexpr int kLutBytes = lut_bytes(32);

__device__ __forceinline__ float lut_key(float x) { return fmaf(x, 128.0f, kLutMagic); }
__device__ __forceinline__ float2 lut_key2(float2 x)
{
    return __ffma2_rn(x, make_float2(128.0f, 128.0f), make_float2(kLutMagic, kLutMagic));
}

// The lane's table entry {thr bits, payload} for key = lut_key(x), whose bits are
// kLutMagicBits + bin.  lut_base = lut_lane_base(table, lane): a 32-bit shared-memory address
// with the magic folded in, so that the probe is one multiply-add and one 8-byte read.  The
// table is constant while it is probed, hence the read may be scheduled freely.
template <int REP = 32>
__device__ __forceinline__ uint32_t lut_lane_base(const unsigned char* s_lut, int lane)
{
    return (uint32_t)__cvta_generic_to_shared(s_lut) + (uint32_t)(lane & (REP - 1)) * 8u -
           kLutMagicBits * (uint32_t)lut_row_bytes(REP);
}
template <int REP = 32>
__device__ __forceinline__ uint2 lut_probe(float key, uint32_t lut_base)
{
    uint2 e;
    asm("ld.shared.v2.u32 {%0, %1}, [%2];"
        : "=r"(e.x), "=r"(e.y)
        : "r"(__float_as_uint(key) * (uint32_t)lut_row_bytes(REP) + lut_base));
    return e;
}

// Builds the table in shared memory from the thresholds; payload(base) is stored next to
// thr (a code, or a byte offset).  *s_multi tells whether some bin holds two thresholds.
// Call with all threads of the CTA, then __syncthreads().  The entries are first computed once
// per bin into the table's own first row slots and then replicated with one warp per row, so
// that the replicating stores of a warp fall into 32 different lanes' columns (no conflicts).
template <int REP = 32, class PayloadFn>
__device__ __forceinline__ void build_lut(const float* s_xi, unsigned char* s_lut, int* s_multi,
                                          PayloadFn payload)
{
    __shared__ uint2 s_ent[kLutBins];
    __shared__ int s_bin[kLevels];  // bin of every threshold
    if (threadIdx.x == 0) *s_multi = 0;
    if (threadIdx.x < kLevels - 1) {
        int bj = (int)(__float_as_uint(lut_key(s_xi[threadIdx.x])) - kLutMagicBits);
        s_bin[threadIdx.x] = bj < 0 ? 0 : (bj > kLutBins - 1 ? kLutBins - 1 : bj);
    }
    __syncthreads();
    for (int b = threadIdx.x; b < kLutBins; b += blockDim.x) {
        int base = 0, inside = 0;
#pragma unroll
        for (int j = 0; j < kLevels - 1; ++j) {
            const int bj = s_bin[j];
            base += (bj < b) ? 1 : 0;
            inside += (bj == b) ? 1 : 0;
        }
        if (inside > 1) *s_multi = 1;
        s_ent[b] = make_uint2(__float_as_uint(s_xi[base]), payload(base));
    }
    __syncthreads();
    for (int k = threadIdx.x; k < kLutBins * REP; k += blockDim.x)
        *reinterpret_cast<uint2*>(s_lut + k * 8) = s_ent[k / REP];
}

// ---------------------------------------------------------------- division for bf16 inputs
//
// For bfloat16 operands with 2^-60 <= |m| <= 2^60 the sequence
//     r = RN(1/m);  q0 = RN(w r);  e = fma(-q0, m, w);  q = fma(e, r, q0)
// returns exactly RN(w / m) whenever the quotient is a normal number (checked exhaustively
// over all operand pairs on the CPU by the test-suite).  It costs three packed operations
// per two weights plus one reciprocal per lane and block.
__device__ __forceinline__ bool div_safe(float g)
{
    return g >= 0x1p-60f && g <= 0x1p60f;  // false for NaN, infinity and zero
}

// Warp-uniform: every block of this warp row (lanes beyond the end of the data excepted) has a
// largest magnitude g inside the safe range.
__device__ __forceinline__ bool row_is_safe(float g, bool ok) { return __all_sync(kFull, div_safe(g) || !ok); }

// x[k] = RN(v[k] / m) for the 16 weights of a lane (x = 0 when m = 0).  `fast` (warp-uniform;
// only ever true for bf16 input whose block constants all pass div_safe) selects the
// reciprocal sequence.  With GUARD, quotients below 2^-100 in magnitude are recomputed by the
// IEEE division so that subnormal results are rounded once.
template <bool GUARD>
__device__ __forceinline__ void normalise16(const float (&v)[kLaneW], float m, bool fast,
                                            float (&x)[kLaneW])
{
    if (fast) {
        // lanes beyond the end of the data hold zeros and m = 0: give them x = 0, a valid table index
        const float r = (m == 0.0f) ? 0.0f : __frcp_rn(m);
        const float2 rr = make_float2(r, r), nm = make_float2(-m, -m);
#pragma unroll
        for (int k = 0; k < kLaneW / 2; ++k) {
            const float2 w = make_float2(v[2 * k], v[2 * k + 1]);
            const float2 q0 = __fmul2_rn(w, rr);
            const float2 e = __ffma2_rn(q0, nm, w);
            const float2 q = __ffma2_rn(e, rr, q0);
            x[2 * k] = q.x;
            x[2 * k + 1] = q.y;
        }
        if (GUARD) {
            float lo = min3(fabsf(x[0]), fabsf(x[1]), fabsf(x[2]));
#pragma unroll
            for (int k = 3; k < 15; k += 2) lo = min3(lo, fabsf(x[k]), fabsf(x[k + 1]));
            lo = fminf(lo, fabsf(x[15]));
            if (lo < 0x1p-100f) {
#pragma unroll
                for (int k = 0; k < kLaneW; ++k)
                    if (fabsf(x[k]) < 0x1p-100f && v[k] != 0.0f) x[k] = normalise(v[k], m);
            }
        }
    } else {
#pragma unroll
        for (int k = 0; k < kLaneW; ++k) x[k] = normalise(v[k], m);
    }
}

}  // namespace bof4
