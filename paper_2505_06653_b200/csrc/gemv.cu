// Decoding fused into its consumer: y = W_q x for a block-wise 4-bit matrix (Eq. 3 applied on the
// fly), with the OPQ outliers applied as a sparse correction (Sec. 3.3, decoding side).  This is
// the operation whose run time the paper reports for token generation (App. E.2); a matrix-vector
// product is bound by reading the weights once, here 0.5 byte per weight plus the block constants.
//
// Definition: y[r] = sum over the blocks b of row r of  scale_b * sum_i xhat[code_i] * x_i  in
// fp32 (no intermediate rounding of the dequantised weight to bf16), where an outlier position
// contributes val * x instead of its quantised value.
//
// Work layout: a CTA holds G row groups of S = ceil(cols / 1024) warps.  Warp s of a group owns
// the column stripe [1024 s, 1024 s + 1024) for every row the group visits, and lane l of it the
// 32 columns from 1024 s + 32 l, whose 32 values of x stay in registers as fp32 for the whole
// kernel.  Per row a lane reads its 16 code bytes with one load, looks the two levels of each byte
// up in a pair table in shared memory and multiplies with the matching pair of x (packed fp32x2
// FMA).  The table has one 8-byte column per lane ([byte][lane], 256 bytes per row), so that no
// two lanes ever meet in a bank, whatever their codes, and so that one byte permute builds the
// whole table offset: the code byte lands in bits 8..15 and the lane's column offset in bits
// 0..7.  The look-up is the busiest unit of this kernel: 8 bytes of shared memory per code byte
// against 128 bytes per clock and SM bound it to 16 code bytes per clock and SM, about two
// thirds of what HBM could deliver.
//
// A CTA of up to 16 warps (cols <= 16384) runs with 128 registers per thread and requests the
// next batch of kGvRows rows straight into registers before it uses the current one.  The
// 32-warp CTA of wider matrices has 64 registers per thread and no room for that: its codes
// travel global -> shared memory by asynchronous 16-byte copies into a ring that each warp owns
// (kGvStages batches); a lane later reads back exactly the 16 bytes it copied itself, so the
// ring needs no barrier and costs no registers.  The per-lane partial sums of a
// batch are reduced over the warp with a halving butterfly, then every kGvDefer batches over the
// stripes through shared memory in a fixed order.  Nothing is accumulated with atomics, so y is
// bit-reproducible.
#include "common.cuh"

namespace bof4 {

constexpr int kGvStripe = 1024;  // columns per warp
constexpr int kGvLane = 32;      // columns per lane = 16 code bytes

template <class ST>
__device__ __forceinline__ float gv_scale(const void* scales, int64_t b);
template <>
__device__ __forceinline__ float gv_scale<F32>(const void* scales, int64_t b)
{
    return __ldg(static_cast<const float*>(scales) + b);
}
template <>
__device__ __forceinline__ float gv_scale<BF16>(const void* scales, int64_t b)
{
    return __uint_as_float((uint32_t)__ldg(static_cast<const uint16_t*>(scales) + b) << 16);
}

template <class XT>
__device__ __forceinline__ float gv_x(const void* x, int64_t c);
template <>
__device__ __forceinline__ float gv_x<F32>(const void* x, int64_t c)
{
    return __ldg(static_cast<const float*>(x) + c);
}
template <>
__device__ __forceinline__ float gv_x<BF16>(const void* x, int64_t c)
{
    return __uint_as_float((uint32_t)__ldg(static_cast<const uint16_t*>(x) + c) << 16);
}

// Sums v[0 .. R) over the 32 lanes.  After the call lane (32 / R) * r holds in v[0] the total of
// row r; the exchange order is fixed, so the result is too.
template <int R>
__device__ __forceinline__ void reduce_rows(float (&v)[R], int lane)
{
    static_assert(R == 8 || R == 4 || R == 2, "halving butterfly written for 2, 4 or 8 rows");
    int off = 16;
#pragma unroll
    for (int h = R / 2; h >= 1; h >>= 1, off >>= 1) {
        const bool upper = (lane & off) != 0;
#pragma unroll
        for (int i = 0; i < h; ++i) {
            const float send = upper ? v[i] : v[i + h];
            const float keep = upper ? v[i + h] : v[i];
            v[i] = keep + __shfl_xor_sync(kFull, send, off);
        }
    }
    for (; off >= 1; off >>= 1) v[0] += __shfl_xor_sync(kFull, v[0], off);
}

constexpr int kGvRows = 4;    // rows per batch
constexpr int kGvStages = 2;  // batches in a warp's ring
constexpr int kGvDefer = 4;   // batches between two reductions over the stripes
constexpr int kGvTabBytes = 256 * 32 * 8;  // [byte][lane] pairs of levels
// dynamic shared memory of a CTA of `threads`: the table, then [warp][stage][row][lane] 16 bytes
constexpr int gv_smem(int threads) { return kGvTabBytes + (threads / 32) * kGvStages * kGvRows * 512; }

// Two fp32 in one 64-bit register, the operand form of the packed FMA.
__device__ __forceinline__ uint64_t pack2(float lo, float hi)
{
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ float sum2(uint64_t v)
{
    float lo, hi;
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
    return lo + hi;
}
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c)
{
    uint64_t d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}

// A lane's 32 values of x as packed fp32 pairs (bf16 is widened once, when the kernel starts).
template <class XT>
__device__ __forceinline__ void load_x(const void* x, int64_t c0, bool live, uint64_t (&v)[16]);
template <>
__device__ __forceinline__ void load_x<BF16>(const void* x, int64_t c0, bool live, uint64_t (&v)[16])
{
    const uint4* src = reinterpret_cast<const uint4*>(static_cast<const uint16_t*>(x) + c0);
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        const uint4 t = live ? __ldg(src + q) : make_uint4(0u, 0u, 0u, 0u);
        const uint32_t p[4] = {t.x, t.y, t.z, t.w};
#pragma unroll
        for (int k = 0; k < 4; ++k)
            v[4 * q + k] = pack2(__uint_as_float(p[k] << 16), __uint_as_float(p[k] & 0xffff0000u));
    }
}
template <>
__device__ __forceinline__ void load_x<F32>(const void* x, int64_t c0, bool live, uint64_t (&v)[16])
{
    const float4* src = reinterpret_cast<const float4*>(static_cast<const float*>(x) + c0);
#pragma unroll
    for (int q = 0; q < 8; ++q) {
        const float4 t = live ? __ldg(src + q) : make_float4(0.f, 0.f, 0.f, 0.f);
        v[2 * q] = pack2(t.x, t.y), v[2 * q + 1] = pack2(t.z, t.w);
    }
}

// MAXT = 512 (up to 16 stripes; 128 registers per thread keep many look-ups of a warp in flight,
// which measured faster than twice the warps) or 1024 (17 ... 32 stripes).  One CTA per SM.
constexpr bool kGvRing512 = false;  // the 512-thread variant prefetches into registers (measured 8 % faster)

template <class ST, class XT, int MAXT, bool RING>
__global__ void __launch_bounds__(MAXT, 1)
gemv_kernel(const uint8_t* __restrict__ codes, const void* __restrict__ scales, int64_t rows, int64_t cols,
            int block_shift, const float* __restrict__ levels, const void* __restrict__ x, float* __restrict__ y,
            int stripes, int groups)
{
    constexpr int R = kGvRows, K = kGvDefer, S = kGvStages;
    extern __shared__ __align__(256) unsigned char s_dyn[];  // table, then the rings
    unsigned char* const s_tab = s_dyn;
    __shared__ float s_part[2][K][R][32];  // groups * stripes <= 32
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int group = warp / stripes, stripe = warp - group * stripes;
    const int64_t c0 = (int64_t)stripe * kGvStripe + lane * kGvLane;  // this lane's first column
    const bool live = c0 < cols;  // cols is a multiple of 32: all of the lane's columns exist or none
    const uint32_t column = (uint32_t)lane * 8u;  // < 256: the low byte of every table offset
    const int64_t batches = (rows + R - 1) / R;
    const int64_t bstep = (int64_t)gridDim.x * groups;
    // this lane's 16 bytes of (stage 0, row 0); a row is 512 bytes, a stage R rows
    const uint32_t ring = (uint32_t)__cvta_generic_to_shared(s_dyn + kGvTabBytes) + (uint32_t)warp * (S * R * 512) +
                          (uint32_t)lane * 16u;
    const uint32_t row_bytes = (uint32_t)(cols >> 1);             // codes of one row
    const uint32_t row_blocks = (uint32_t)(cols >> block_shift);  // block constants of one row
    const int64_t step_bytes = bstep * R * (int64_t)row_bytes;    // from one of this warp's batches to the next
    const int64_t step_blocks = bstep * R * (int64_t)row_blocks;
    // Starts the copies of a batch into `stage`: `left` rows remain from its first row on, whose
    // codes for this lane start at src.  Nothing is copied for rows past the end or dead lanes:
    // whatever the slot then holds is multiplied by a zero block constant.
    auto issue = [&](const uint8_t* src, int64_t left, int stage) {
        if constexpr (RING) {
#pragma unroll
            for (int u = 0; u < R; ++u) {
                if (live && u < left)
                    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(ring +
                                                                                  (uint32_t)(stage * R + u) * 512u),
                                 "l"(src + u * row_bytes)
                                 : "memory");
            }
            asm volatile("cp.async.commit_group;" ::: "memory");
        }
    };
    // Without the ring: the same 16 bytes per row straight into registers (zeros past the end).
    auto fetch = [&](const uint8_t* src, int64_t left, uint4(&c)[R]) {
#pragma unroll
        for (int u = 0; u < R; ++u) {
            c[u] = make_uint4(0u, 0u, 0u, 0u);
            if (live && u < left)
                asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                             : "=r"(c[u].x), "=r"(c[u].y), "=r"(c[u].z), "=r"(c[u].w)
                             : "l"(src + u * row_bytes));
        }
    };
    // block constants of a batch; index = that of this lane's block in the batch's first row
    auto block_constants = [&](int64_t index, int64_t left, float(&m)[R]) {
#pragma unroll
        for (int u = 0; u < R; ++u) m[u] = (live && u < left) ? gv_scale<ST>(scales, index + u * row_blocks) : 0.0f;
    };

    int64_t b0 = (int64_t)blockIdx.x * groups;  // batch of group 0 in this iteration
    const int64_t r_first = (b0 + group) * R;    // first row of this warp's first batch
    int64_t left = rows - r_first;               // rows from the current batch's first row to the end (may be <= 0)
    const int64_t step_rows = bstep * R;
    const uint8_t* src = codes + ((r_first * cols + c0) >> 1);               // codes of the next batch to request
    int64_t blk = (r_first * cols + c0) >> block_shift;                      // block of the next batch's constants
    // The first codes, x and the levels are requested together: the cold misses overlap.
    uint4 cc[R];
    if (RING) {
#pragma unroll
        for (int sI = 0; sI < S - 1; ++sI) {
            issue(src, left - sI * step_rows, sI);
            src += step_bytes;
        }
    } else {
        fetch(src, left, cc);
        src += step_bytes;
    }
    float m[R];
    block_constants(blk, left, m);
    blk += step_blocks;
    uint64_t xr[16];
    load_x<XT>(x, c0, live, xr);
    {
        const float mine = levels[threadIdx.x & 15];  // level l sits in the lanes with (lane & 15) == l
        for (int e = threadIdx.x; e < 256 * 32; e += blockDim.x) {  // blockDim is a multiple of 32: e & 31 == lane
            const int byte = e >> 5;
            reinterpret_cast<float2*>(s_tab)[e] = make_float2(__shfl_sync(kFull, mine, byte >> 4),
                                                              __shfl_sync(kFull, mine, byte & 15));
        }
    }
    __syncthreads();
    int k = 0, buf = 0, stage = 0;
    for (; b0 < batches; b0 += bstep) {
        // refill the slot consumed in the previous iteration, then wait for this iteration's batch
        // (registers: request the next batch before this one is used)
        uint4 cn[R];
        if (RING)
            issue(src, left - (S - 1) * step_rows, stage == 0 ? S - 1 : stage - 1);
        else
            fetch(src, left - step_rows, cn);
        src += step_bytes;
        float mn[R];
        block_constants(blk, left - step_rows, mn);  // block constants run one batch ahead in registers
        blk += step_blocks;
        left -= step_rows;
        uint32_t word[R][4];
        if (RING) {
            asm volatile("cp.async.wait_group %0;" ::"n"(S - 1) : "memory");
#pragma unroll
            for (int u = 0; u < R; ++u)
                asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];"
                             : "=r"(word[u][0]), "=r"(word[u][1]), "=r"(word[u][2]), "=r"(word[u][3])
                             : "r"(ring + (uint32_t)(stage * R + u) * 512u));
        } else {
#pragma unroll
            for (int u = 0; u < R; ++u)
                word[u][0] = cc[u].x, word[u][1] = cc[u].y, word[u][2] = cc[u].z, word[u][3] = cc[u].w;
        }
        uint64_t a2[R];
#pragma unroll
        for (int u = 0; u < R; ++u) a2[u] = 0ull;
        // column pair j of all R rows before pair j + 1: R independent chains share one x register
#pragma unroll
        for (int j = 0; j < 16; ++j) {
#pragma unroll
            for (int u = 0; u < R; ++u) {
                // byte j holds the codes of columns 2j (high nibble) and 2j + 1 (low nibble);
                // offset = byte * 256 + lane * 8 in one permute
                const uint32_t off = __byte_perm(word[u][j >> 2], column, 0x5504u | ((uint32_t)(j & 3) << 4));
                a2[u] = fma2(*reinterpret_cast<const uint64_t*>(s_tab + off), xr[j], a2[u]);
            }
        }
        float part[R];
#pragma unroll
        for (int u = 0; u < R; ++u) part[u] = __fmul_rn(m[u], sum2(a2[u]));
        reduce_rows<R>(part, lane);
        if ((lane & (32 / R - 1)) == 0) s_part[buf][k][lane / (32 / R)][warp] = part[0];
        const bool last = b0 + bstep >= batches;
        if (k == K - 1 || last) {
            __syncthreads();
            // Sum over the stripes for the k + 1 batches since the last reduction.  Two buffers:
            // whoever writes this buffer again has passed the next barrier, which the readers
            // reach only after this read.
            const int per = groups * R;
            for (int t = threadIdx.x; t < (k + 1) * per; t += blockDim.x) {
                const int j = t / per, rem = t - j * per, g = rem / R, u = rem - g * R;
                const int64_t r = (b0 - (int64_t)(k - j) * bstep + g) * R + u;
                if (r < rows) {
                    float sum = 0.0f;
                    for (int sI = 0; sI < stripes; ++sI) sum += s_part[buf][j][u][g * stripes + sI];
                    y[r] = sum;
                }
            }
            buf ^= 1;
            k = 0;
        } else {
            ++k;
        }
        stage = (stage == S - 1) ? 0 : stage + 1;
#pragma unroll
        for (int u = 0; u < R; ++u) {
            m[u] = mn[u];
            if (!RING) cc[u] = cn[u];
        }
    }
    if (RING) asm volatile("cp.async.wait_group 0;" ::: "memory");  // nothing of this CTA is in flight when it ends
}

// Sparse correction: y[row] += sum over the row's outliers of (val - scale * xhat[code]) * x.
// Every thread computes the term of one outlier (independent loads); the thread that holds the
// first outlier of a row then adds that row's terms in list order (the list is ascending, so
// they are contiguous) and is the only writer of y[row]: no atomics, a fixed order.  Terms of
// the CTA's own chunk come from shared memory; a row that runs past the chunk is finished from
// global memory by the same thread.
template <class ST, class XT>
__global__ void __launch_bounds__(256)
gemv_outlier_kernel(const uint8_t* __restrict__ codes, const void* __restrict__ scales, int64_t rows,
                    int64_t cols, int block_shift, const float* __restrict__ levels, const void* __restrict__ x,
                    const int32_t* __restrict__ idx, const uint16_t* __restrict__ val,
                    const int64_t* __restrict__ n_out, int64_t capacity, float* __restrict__ y)
{
    __shared__ float s_term[256];
    __shared__ int s_row[256];
    int64_t k_end = *n_out;
    if (k_end > capacity) k_end = capacity;
    const int64_t n = rows * cols;
    // row of list entry k (-1 for an index outside the matrix) and its term
    auto row_of = [&](int64_t k) -> int {
        const int64_t i = idx[k];
        return (i < 0 || i >= n) ? -1 : (int)(i / cols);
    };
    auto term_of = [&](int64_t k, int r) -> float {
        const int64_t i = idx[k];
        const uint32_t byte = codes[i >> 1];
        const uint32_t c = (i & 1) ? (byte & 15u) : (byte >> 4);
        const float q = __fmul_rn(gv_scale<ST>(scales, i >> block_shift), __ldg(levels + c));
        return __fmul_rn(__uint_as_float((uint32_t)val[k] << 16) - q, gv_x<XT>(x, i - (int64_t)r * cols));
    };
    const int tid = threadIdx.x;
    for (int64_t base = (int64_t)blockIdx.x * 256; base < k_end; base += (int64_t)gridDim.x * 256) {
        const int64_t k = base + tid;
        const int r = (k < k_end) ? row_of(k) : -1;
        s_row[tid] = r;
        s_term[tid] = (r >= 0) ? term_of(k, r) : 0.0f;
        __syncthreads();
        if (r >= 0) {
            const int before = (tid > 0) ? s_row[tid - 1] : (k > 0 ? row_of(k - 1) : -1);
            if (before != r) {  // first outlier of its row
                float sum = 0.0f;
                int j = tid;
                while (j < 256 && s_row[j] == r) sum += s_term[j++];
                if (j == 256)
                    for (int64_t kk = base + 256; kk < k_end && row_of(kk) == r; ++kk) sum += term_of(kk, r);
                y[r] += sum;
            }
        }
        __syncthreads();
    }
}

template <class ST, class XT, int MAXT>
static int launch_gemv_kernel(const uint8_t* d_codes, const void* d_scales, int64_t rows, int64_t cols,
                              int block_size, const float* d_codebook, const void* d_x, float* d_y, int stripes,
                              cudaStream_t st)
{
    const int64_t batches = (rows + kGvRows - 1) / kGvRows;
    int groups = (MAXT / 32) / stripes;  // row groups per CTA, >= 1 by the caller's choice of MAXT
    if (groups > batches) groups = (int)batches;
    const int64_t want = (batches + groups - 1) / groups;
    const int grid = (int)(want < kSMs ? want : kSMs);  // one CTA per SM (its shared memory fills the SM)
    int block_shift = 0;
    while ((1 << block_shift) < block_size) ++block_shift;
    constexpr bool RING = MAXT > 512 || kGvRing512;
    constexpr int smem = RING ? gv_smem(MAXT) : kGvTabBytes;
    constexpr auto kern = gemv_kernel<ST, XT, MAXT, RING>;
    if (const int rc = ensure_dynamic_smem<kern>(smem)) return rc;
    kern<<<grid, 32 * stripes * groups, smem, st>>>(d_codes, d_scales, rows, cols, block_shift, d_codebook,
                                                             d_x, d_y, stripes, groups);
    BOF4_CUDA_TRY(cudaGetLastError());
    return BOF4_OK;
}

template <class ST, class XT>
static int launch_gemv(const uint8_t* d_codes, const void* d_scales, int64_t rows, int64_t cols, int block_size,
                       const float* d_codebook, const void* d_x, const int32_t* d_out_idx, const uint16_t* val,
                       const int64_t* d_n_out, int64_t capacity, bool opq, float* d_y, cudaStream_t st)
{
    const int stripes = (int)((cols + kGvStripe - 1) / kGvStripe);  // <= 32: cols <= 32768 was checked
    const int rc = (stripes <= 16) ? launch_gemv_kernel<ST, XT, 512>(d_codes, d_scales, rows, cols, block_size,
                                                                     d_codebook, d_x, d_y, stripes, st)
                                   : launch_gemv_kernel<ST, XT, 1024>(d_codes, d_scales, rows, cols, block_size,
                                                                      d_codebook, d_x, d_y, stripes, st);
    if (rc != BOF4_OK) return rc;
    if (opq && capacity > 0) {
        int block_shift = 0;
        while ((1 << block_shift) < block_size) ++block_shift;
        gemv_outlier_kernel<ST, XT><<<2 * kSMs, 256, 0, st>>>(d_codes, d_scales, rows, cols, block_shift, d_codebook,
                                                              d_x, d_out_idx, val, d_n_out, capacity, d_y);
        BOF4_CUDA_TRY(cudaGetLastError());
    }
    return BOF4_OK;
}

}  // namespace bof4

extern "C" int bof4_gemv(const uint8_t* d_codes, const void* d_scales, int scale_dtype, int64_t rows,
                         int64_t cols, int block_size, const float* d_codebook, const void* d_x, int x_dtype,
                         const int32_t* d_out_idx, const void* d_out_val, const int64_t* d_n_out,
                         int64_t capacity, float* d_y, void* stream)
{
    using namespace bof4;
    if (rows < 0 || cols < 0) {
        set_error("bof4_gemv: negative shape");
        return BOF4_ERR_INVALID_ARG;
    }
    if (!valid_block_size(block_size) || cols % block_size || cols > 32768) {
        set_error("bof4_gemv: block_size must be a power of two in 32 ... 4096 that divides cols, cols <= 32768");
        return BOF4_ERR_SHAPE;
    }
    if ((scale_dtype != BOF4_F32 && scale_dtype != BOF4_BF16) || (x_dtype != BOF4_F32 && x_dtype != BOF4_BF16)) {
        set_error("bof4_gemv: unknown dtype");
        return BOF4_ERR_DTYPE;
    }
    const bool opq = d_out_idx != nullptr;
    if (opq && (!d_out_val || !d_n_out)) {
        set_error("bof4_gemv: outlier list needs d_out_idx, d_out_val and d_n_out together");
        return BOF4_ERR_INVALID_ARG;
    }
    if (opq && capacity < 0) {
        set_error("bof4_gemv: negative capacity");
        return BOF4_ERR_CAPACITY;
    }
    if (opq && rows * cols > (int64_t)INT32_MAX) {
        set_error("bof4_gemv: outlier indices are 32-bit, rows * cols must not exceed 2^31 - 1");
        return BOF4_ERR_SHAPE;
    }
    if (rows == 0) return BOF4_OK;
    if (!d_y || (cols > 0 && (!d_codes || !d_scales || !d_codebook || !d_x))) {
        set_error("bof4_gemv: NULL pointer");
        return BOF4_ERR_INVALID_ARG;
    }
    if (!aligned32(d_codes) || (reinterpret_cast<uintptr_t>(d_x) & 15u)) {
        set_error("bof4_gemv: d_codes must be 32-byte aligned and d_x 16-byte aligned");
        return BOF4_ERR_INVALID_ARG;
    }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (cols == 0) {
        BOF4_CUDA_TRY(cudaMemsetAsync(d_y, 0, (size_t)rows * sizeof(float), st));
        return BOF4_OK;
    }
    const uint16_t* val = static_cast<const uint16_t*>(d_out_val);
    if (scale_dtype == BOF4_F32 && x_dtype == BOF4_F32)
        return launch_gemv<F32, F32>(d_codes, d_scales, rows, cols, block_size, d_codebook, d_x, d_out_idx, val,
                                     d_n_out, capacity, opq, d_y, st);
    if (scale_dtype == BOF4_F32)
        return launch_gemv<F32, BF16>(d_codes, d_scales, rows, cols, block_size, d_codebook, d_x, d_out_idx, val,
                                      d_n_out, capacity, opq, d_y, st);
    if (x_dtype == BOF4_F32)
        return launch_gemv<BF16, F32>(d_codes, d_scales, rows, cols, block_size, d_codebook, d_x, d_out_idx, val,
                                      d_n_out, capacity, opq, d_y, st);
    return launch_gemv<BF16, BF16>(d_codes, d_scales, rows, cols, block_size, d_codebook, d_x, d_out_idx, val,
                                   d_n_out, capacity, opq, d_y, st);
}
