// Decode fused into a batched consumer on the tensor cores: Y = W_q X^T for 16 ... 64 right-hand
// sides (App. E.2 times token generation; with several tokens or sequences in flight the
// matrix-vector product of gemv.cu becomes this small-N matrix product, and the decode of Eq. 3
// amortises over the batch).
//
// Reading (the paper gives no arithmetic for a fused consumer): the A operand is the dequantised
// weight rounded to bf16, bit for bit what bof4_dequantize writes (Eq. 3, then round to nearest
// even), X is bf16, products are exact and the sums are accumulated in fp32 by the tensor cores.
//
// One CTA owns 128 rows of W and a range of K.  Eight producer warps decode, per k-block of 64
// weights, the 128 x 64 tile (4 KiB of codes) into shared memory as bf16 in the K-major
// 128-byte-swizzled layout that the tcgen05 shared-memory descriptor names (8-row groups of 1024
// bytes, 16-byte chunk c of row r stored at chunk c ^ (r & 7)) and copy the matching 64 columns
// of X the same way; each warp then arrives on the stage's "full" mbarrier.  One thread of a ninth
// warp waits for a full stage and issues four tcgen05.mma (M = 128, N = batch, K = 16 each) that
// accumulate into tensor memory; its tcgen05.commit arrives on the stage's "empty" mbarrier when
// the tensor cores have read the stage, which the producers wait for before they overwrite it
// (three stages).  No CTA-wide barrier inside the loop.  Every wait is bounded: a time-out sets
// the status word, the issuing thread still commits and waits (bounded) for what it has issued,
// and the kernel frees its tensor memory and returns.  The epilogue reads the accumulator with
// tcgen05.ld (one row per thread) and writes fp32.
#include <cuda.h>

#include "common.cuh"

namespace bof4 {

constexpr int kTcProducerWarps = 8;
constexpr int kTcProducers = kTcProducerWarps * 32;  // threads that decode
constexpr int kTcThreads = 32 + kTcProducers;        // and one warp that issues the tensor-core instructions
constexpr int kTcM = 128;         // rows per CTA = tensor-memory lanes
constexpr int kTcK = 64;          // weights per k-block: one 128-byte swizzle row of bf16
constexpr int kTcStages = 3;
constexpr int kTcCtasPerSm = 2;   // 106 KiB of shared memory and 64 tensor-memory columns each
constexpr int kTcMaxN = 64;
constexpr int kTcTmemCols = 64;   // power of two >= 32 and >= N
constexpr int kTcABytes = kTcM * kTcK * 2;     // 16 KiB
constexpr int kTcBBytes = kTcMaxN * kTcK * 2;  // 8 KiB
constexpr int kTcTableBytes = 256 * 16 * 8;    // level pairs per code byte, one column per lane pair (L, L + 16)
constexpr int kTcSmem = kTcStages * (kTcABytes + kTcBBytes) + 1024 + kTcTableBytes;  // + slack to align to 1024 bytes
constexpr uint32_t kTcSpinLimit = 1u << 16;    // try_wait calls before a wait gives up (a k-block takes microseconds)

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

// Shared-memory matrix descriptor of a K-major tile in the 128-byte swizzled layout: start
// address and offsets in units of 16 bytes, leading offset 1 (unused for swizzled K-major), stride
// between 8-row groups 1024 bytes, descriptor version 1, layout type 2 (128-byte swizzle).
__device__ __forceinline__ uint64_t tc_smem_desc(uint32_t addr)
{
    uint64_t d = 0;
    d |= (uint64_t)((addr >> 4) & 0x3fffu);
    d |= (uint64_t)1 << 16;
    d |= (uint64_t)(1024 >> 4) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;
    return d;
}

// Instruction descriptor: fp32 accumulator, bf16 x bf16, both K-major, M = 128, N = n.
__host__ __device__ inline uint32_t tc_instr_desc(int n)
{
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(kTcM >> 4) << 24);
}

__device__ __forceinline__ bool tc_wait(uint32_t bar, uint32_t parity)
{
    for (uint32_t it = 0; it < kTcSpinLimit; ++it) {
        uint32_t ok;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(ok)
            : "r"(bar), "r"(parity)
            : "memory");
        if (ok) return true;
    }
    return false;
}

template <class ST>
__device__ __forceinline__ float tc_scale(const void* scales, int64_t b);
template <>
__device__ __forceinline__ float tc_scale<F32>(const void* scales, int64_t b)
{
    return __ldg(static_cast<const float*>(scales) + b);
}
template <>
__device__ __forceinline__ float tc_scale<BF16>(const void* scales, int64_t b)
{
    return __uint_as_float((uint32_t)__ldg(static_cast<const uint16_t*>(scales) + b) << 16);
}

template <class ST>
__global__ void __launch_bounds__(kTcThreads, kTcCtasPerSm)
gemm_tc_kernel(const uint8_t* __restrict__ codes, const void* __restrict__ scales, int64_t cols, int block_shift,
               const float* __restrict__ levels, const __grid_constant__ CUtensorMap x_map, int n_rhs,
               float* __restrict__ y, int kb_per_split, int* __restrict__ status)
{
    extern __shared__ unsigned char s_dyn[];
    // full[s]: the producers have filled stage s (one arrival per producer warp); empty[s]: the tensor
    // cores have read it (tcgen05.commit); done: every instruction of the CTA has completed
    __shared__ __align__(8) unsigned long long s_full[kTcStages], s_empty[kTcStages], s_done;
    __shared__ uint32_t s_tmem;
    __shared__ int s_fail;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t tiles = (smem_u32(s_dyn) + 1023u) & ~1023u;  // 1024-byte aligned: the swizzle atoms start here
    unsigned char* tiles_ptr = s_dyn + (tiles - smem_u32(s_dyn));
    const int64_t row0 = (int64_t)blockIdx.x * kTcM;
    // blockIdx.y selects a range of k-blocks (split along K so that matrices with few row tiles still
    // fill the machine); its partial product goes to slab blockIdx.y of y
    const int kblocks = kb_per_split, kb0 = (int)blockIdx.y * kb_per_split;
    y += (int64_t)blockIdx.y * ((int64_t)gridDim.x * kTcM) * n_rhs;

    // Level pairs of a code byte (Eq. 3's xhat for its two weights), one 8-byte column per pair of
    // lanes L and L + 16: an 8-byte read is served half a warp at a time, so the 16 lanes of a half
    // never share a bank whatever their code bytes are.
    unsigned char* tab_ptr = tiles_ptr + kTcStages * (kTcABytes + kTcBBytes);
    __shared__ float s_lv[kLevels];
    if (tid < kLevels) s_lv[tid] = levels[tid];
    __syncthreads();  // the table is filled from shared memory: no global read per entry
    for (int e = tid; e < 256 * 16; e += kTcThreads)
        reinterpret_cast<float2*>(tab_ptr)[e] = make_float2(s_lv[e >> 8], s_lv[(e >> 4) & 15]);
    const uint32_t tab = smem_u32(tab_ptr) + (uint32_t)(lane & 15) * 8u;
    if (tid == 0) {
        s_fail = 0;
        for (int s = 0; s < kTcStages; ++s) {
            asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(&s_full[s])), "r"(kTcProducerWarps + 1) : "memory");
            asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(&s_empty[s])), "r"(1) : "memory");
        }
        asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(&s_done)), "r"(1) : "memory");
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) {  // tensor memory for the 128 x N fp32 accumulator
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&s_tmem)),
                     "r"(kTcTmemCols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem = s_tmem;

    if (warp == 0) {
        // ---- the issuing warp: one thread waits for a full stage, issues its four instructions and
        // lets tcgen05.commit hand the stage back
        if (lane == 0) {
            const uint32_t idesc = tc_instr_desc(n_rhs);
            bool ok = true;
            for (int kb = 0; kb < kblocks && ok; ++kb) {
                const int s = kb % kTcStages;
                if (!tc_wait(smem_u32(&s_full[s]), (uint32_t)((kb / kTcStages) & 1))) {
                    ok = false;
                    break;
                }
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t sa = tiles + (uint32_t)s * (kTcABytes + kTcBBytes);
                const uint64_t da = tc_smem_desc(sa), db = tc_smem_desc(sa + kTcABytes);
#pragma unroll
                for (int kk = 0; kk < kTcK / 16; ++kk) {  // 32 bytes of K per instruction: +2 in the address field
                    const uint32_t acc = (kb > 0 || kk > 0) ? 1u : 0u;
                    asm volatile(
                        "{\n\t.reg .pred p;\n\t"
                        "setp.ne.b32 p, %4, 0;\n\t"
                        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, {%5, %5, %5, %5}, p;\n\t}"
                        :
                        : "r"(tmem), "l"(da + (uint64_t)(2 * kk)), "l"(db + (uint64_t)(2 * kk)), "r"(idesc), "r"(acc), "r"(0u)
                        : "memory");
                }
                asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(
                                 smem_u32(&s_empty[s]))
                             : "memory");
            }
            // whatever has been issued arrives on `done` when it has completed (also after a time-out)
            asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(
                             smem_u32(&s_done))
                         : "memory");
            if (!ok) s_fail = 1;
            if (!tc_wait(smem_u32(&s_done), 0u)) s_fail = 1;
        }
    } else {
        // ---- producer warps: thread t decodes half a row (32 weights = 16 code bytes = four 16-byte
        // chunks) of the 128 x 64 tile; the first of them also requests the X tile
        const int t = tid - 32;
        const int a_row = t >> 1, a_half = t & 1;
        const uint8_t* a_codes = codes + ((row0 + a_row) * cols) / 2 + a_half * 16;
        const int64_t a_first = (row0 + a_row) * cols + a_half * 32;  // flat index of its first weight in k-block 0
        const uint32_t a_off = (uint32_t)((a_row >> 3) * 1024 + (a_row & 7) * 128);
        struct Fetched {
            uint4 cc;
            float m;
        };
        auto fetch = [&](int kb) {  // what the thread reads from global memory for one k-block
            Fetched f;
            kb += kb0;
            // a row's codes are read 32 bytes per k-block (two threads); the hint brings the whole 128-byte
            // line into L2 at the first touch, so DRAM sees full lines instead of scattered sectors
            asm volatile("ld.global.nc.L2::128B.v4.u32 {%0, %1, %2, %3}, [%4];"
                         : "=r"(f.cc.x), "=r"(f.cc.y), "=r"(f.cc.z), "=r"(f.cc.w)
                         : "l"(a_codes + (int64_t)kb * (kTcK / 2)));
            f.m = tc_scale<ST>(scales, (a_first + (int64_t)kb * kTcK) >> block_shift);
            return f;
        };
        // One k-block: wait for the stage, request X, decode, publish.  false: a wait ran out.
        auto step = [&](int kb, const Fetched& cur) -> bool {
            const int s = kb % kTcStages;
            unsigned char* sa = tiles_ptr + s * (kTcABytes + kTcBBytes);
            unsigned char* sb = sa + kTcABytes;
            if (kb >= kTcStages) {  // the tensor cores must have read what the stage held (k-block kb - stages)
                int ok = 1;
                if (lane == 0) ok = tc_wait(smem_u32(&s_empty[s]), (uint32_t)(((kb / kTcStages) - 1) & 1)) ? 1 : 0;
                ok = __shfl_sync(kFull, ok, 0);
                if (!ok) {
                    if (lane == 0) s_fail = 1;
                    return false;
                }
            }
            if (t == 0) {
                // the X tile (n_rhs rows of 64 values) comes by TMA straight into the swizzled layout; its
                // bytes count towards the stage's "full" barrier together with the producer warps' arrivals
                const uint32_t bar = smem_u32(&s_full[s]);
                asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"((uint32_t)n_rhs * 128u)
                             : "memory");
                asm volatile(
                    "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
                    :
                    : "r"(smem_u32(sb)), "l"(reinterpret_cast<uint64_t>(&x_map)), "r"(bar), "r"((kb0 + kb) * kTcK), "r"(0)
                    : "memory");
            }
            const float2 mm = make_float2(cur.m, cur.m);
            const uint32_t word[4] = {cur.cc.x, cur.cc.y, cur.cc.z, cur.cc.w};
#pragma unroll
            for (int j = 0; j < 4; ++j) {  // chunk j of this half: weights 8j .. 8j+7 = code bytes 4j .. 4j+3
                uint32_t p[4];
#pragma unroll
                for (int b = 0; b < 4; ++b) {
                    // byte b of the word times 128 (the table's row size): one shift and one mask
                    const uint32_t off = ((b == 0) ? (word[j] << 7) : (word[j] >> (8 * b - 7))) & 0x7f80u;
                    float2 lv2;
                    asm("ld.shared.v2.f32 {%0, %1}, [%2];" : "=f"(lv2.x), "=f"(lv2.y) : "r"(tab + off));
                    const float2 w2 = __fmul2_rn(mm, lv2);  // Eq. 3 for the (even, odd) weight of the byte
                    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(p[b]) : "f"(w2.y), "f"(w2.x));  // even weight in the low half
                }
                const int chunk = a_half * 4 + j;
                *reinterpret_cast<uint4*>(sa + a_off + ((chunk ^ (a_row & 7)) * 16)) = make_uint4(p[0], p[1], p[2], p[3]);
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // generic-proxy writes -> tensor-core reads
            __syncwarp();
            if (lane == 0)
                asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(&s_full[s])) : "memory");
            return true;
        };
        // two fetch buffers used in turn (no register copies): the loads of k-block kb + 1 are in flight
        // while k-block kb is decoded
        {
            Fetched fa = fetch(0), fb = fa;
            int kb = 0;
            while (kb < kblocks) {
                if (kb + 1 < kblocks) fb = fetch(kb + 1);
                if (!step(kb, fa)) break;
                if (++kb >= kblocks) break;
                if (kb + 1 < kblocks) fa = fetch(kb + 1);
                if (!step(kb, fb)) break;
                ++kb;
            }
        }
    }
    // Every loop above is bounded, so every warp gets here.  After a time-out the issuing thread has
    // still committed and waited (bounded) for what it issued.
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const bool failed = s_fail != 0;
    if (!failed && warp < 4) {  // the accumulator, one row per thread (warp w reads lanes 32 w .. 32 w + 31)
        float* yrow = y + (row0 + warp * 32 + lane) * n_rhs;
        for (int c0 = 0; c0 < n_rhs; c0 += 8) {
            uint32_t v[8];
            asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                         : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7])
                         : "r"(tmem + ((uint32_t)(warp * 32) << 16) + (uint32_t)c0));
            asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
            for (int c = 0; c < 8; ++c) yrow[c0 + c] = __uint_as_float(v[c]);
        }
    }
    if (failed) {
        // a TMA copy requested before the time-out may still be writing this CTA's shared memory: it
        // takes microseconds; give it a bounded 100 before the CTA goes away
        if (tid == 0) atomicExch(status, 1);
        for (int i = 0; i < 100; ++i) __nanosleep(1000);
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 0)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTcTmemCols) : "memory");
}

// OPQ (Sec. 3.3, decoding side): an outlier position holds its stored bf16 value instead of the
// decoded weight, so Y[r][b] += (val - decoded) * X[b][c] for every outlier (r, c).  One warp per
// row: the row's outliers are a contiguous run of the ascending index list (two binary searches),
// each lane owns right-hand sides b = lane, lane + 32 and adds the row's terms in list order.
template <class ST>
__global__ void __launch_bounds__(256)
gemm_tc_outlier_kernel(const uint8_t* __restrict__ codes, const void* __restrict__ scales, int64_t rows, int64_t cols,
                       int block_shift, const float* __restrict__ levels, const uint16_t* __restrict__ x, int n_rhs,
                       const int32_t* __restrict__ idx, const uint16_t* __restrict__ val,
                       const int64_t* __restrict__ n_out, int64_t capacity, float* __restrict__ y)
{
    int64_t k_end = *n_out;
    if (k_end > capacity) k_end = capacity;
    if (k_end <= 0) return;
    auto lower_bound = [&](int64_t key) {  // first k with idx[k] >= key
        int64_t lo = 0, hi = k_end;
        while (lo < hi) {
            const int64_t mid = (lo + hi) >> 1;
            if ((int64_t)idx[mid] < key) lo = mid + 1; else hi = mid;
        }
        return lo;
    };
    const int lane = threadIdx.x & 31;
    const int64_t warps = (int64_t)gridDim.x * (blockDim.x >> 5);
    for (int64_t r = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5); r < rows; r += warps) {
        const int64_t lo = lower_bound(r * cols), hi = lower_bound((r + 1) * cols);
        if (lo == hi) continue;
        for (int b = lane; b < n_rhs; b += 32) {
            float acc = y[r * n_rhs + b];
            for (int64_t k = lo; k < hi; ++k) {
                const int64_t i = idx[k];
                const uint32_t byte = codes[i >> 1];
                const uint32_t c = (i & 1) ? (byte & 15u) : (byte >> 4);
                const float q32 = __fmul_rn(tc_scale<ST>(scales, i >> block_shift), __ldg(levels + c));
                uint32_t qb;
                asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(qb) : "f"(0.0f), "f"(q32));  // the operand the tile held
                const float delta = __uint_as_float((uint32_t)val[k] << 16) - __uint_as_float(qb << 16);
                const float xv = __uint_as_float((uint32_t)x[(int64_t)b * cols + (i - r * cols)] << 16);
                acc = __fadd_rn(acc, __fmul_rn(delta, xv));
            }
            y[r * n_rhs + b] = acc;
        }
    }
}

// Sum of the K-split partial products in slab order (fixed: the result does not depend on scheduling).
__global__ void gemm_tc_reduce_kernel(const float* __restrict__ part, int splits, int64_t total, float* __restrict__ y)
{
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
        float a = part[i];
        for (int s = 1; s < splits; ++s) a += part[(int64_t)s * total + i];
        y[i] = a;
    }
}

}  // namespace bof4

using namespace bof4;

namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// Tensor map of X (bf16 [n_rhs][cols]) with a box of 64 columns x n_rhs rows and the 128-byte swizzle:
// one TMA load per k-block lands in the layout the tcgen05 descriptor of the B operand names.
int make_x_map(const void* d_x, int64_t cols, int n_rhs, CUtensorMap* map)
{
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        BOF4_CUDA_TRY(cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q));
        if (!p || q != cudaDriverEntryPointSuccess) {
            set_error("bof4_gemm_tc: the driver does not provide cuTensorMapEncodeTiled");
            return BOF4_ERR_CUDA;
        }
        fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)n_rhs};
    const cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
    const cuuint32_t box[2] = {(cuuint32_t)kTcK, (cuuint32_t)n_rhs};
    const cuuint32_t estr[2] = {1, 1};
    const CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(d_x), dims, strides, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        set_error("bof4_gemm_tc: cuTensorMapEncodeTiled failed with code %d", (int)r);
        return BOF4_ERR_CUDA;
    }
    return BOF4_OK;
}

}  // namespace

extern "C" int bof4_gemm_tc(const uint8_t* d_codes, const void* d_scales, int scale_dtype, int64_t rows, int64_t cols,
                            int block_size, const float* d_codebook, const void* d_x, int n_rhs,
                            const int32_t* d_out_idx, const void* d_out_val, const int64_t* d_n_out, int64_t capacity,
                            float* d_y, int* d_status, void* d_ws, size_t ws_bytes, void* stream)
{
    const char* fn = "bof4_gemm_tc";
    if (!valid_block_size(block_size)) {
        set_error("%s: block_size %d is not a power of two in 32 ... 4096", fn, block_size);
        return BOF4_ERR_SHAPE;
    }
    if (scale_dtype != BOF4_F32 && scale_dtype != BOF4_BF16) {
        set_error("%s: unknown scale dtype %d", fn, scale_dtype);
        return BOF4_ERR_DTYPE;
    }
    if (rows < 0 || cols < 0 || rows % kTcM || cols % kTcK || cols % block_size || n_rhs < 16 || n_rhs > kTcMaxN ||
        n_rhs % 16) {
        set_error("%s: rows must be a multiple of 128, cols of 64 and of block_size, n_rhs one of 16, 32, 48, 64", fn);
        return BOF4_ERR_SHAPE;
    }
    const bool opq = d_out_idx != nullptr;
    if (opq && (!d_out_val || !d_n_out || capacity < 0)) {
        set_error("%s: outlier list needs d_out_idx, d_out_val and d_n_out together and a capacity >= 0", fn);
        return BOF4_ERR_INVALID_ARG;
    }
    if (opq && rows * cols > 0x7fffffffLL) {
        set_error("%s: outlier indices are 32-bit, rows * cols must not exceed 2^31 - 1", fn);
        return BOF4_ERR_SHAPE;
    }
    if (rows == 0) return BOF4_OK;
    if (!d_codes || !d_scales || !d_codebook || !d_x || !d_y || !d_status) {
        set_error("%s: NULL pointer", fn);
        return BOF4_ERR_INVALID_ARG;
    }
    if (((uintptr_t)d_codes & 15u) || ((uintptr_t)d_x & 15u)) {
        set_error("%s: d_codes and d_x must be 16-byte aligned", fn);
        return BOF4_ERR_INVALID_ARG;
    }
    if (rows / kTcM > 0x7fffffff) {
        set_error("%s: too many rows", fn);
        return BOF4_ERR_SHAPE;
    }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    BOF4_CUDA_TRY(cudaMemsetAsync(d_status, 0, sizeof(int), st));
    if (cols == 0) {
        BOF4_CUDA_TRY(cudaMemsetAsync(d_y, 0, (size_t)rows * n_rhs * sizeof(float), st));
        return BOF4_OK;
    }
    const int grid = (int)(rows / kTcM);
    // K split: enough CTAs to fill the SMs (kTcCtasPerSm each), a divisor of the number of k-blocks,
    // partial products in the workspace (none: no split).  Measured: more and shorter CTAs than
    // that cost more (table set-up, pipeline fill and drain, epilogue) than the fuller last wave gains.
    const int kblocks = (int)(cols / kTcK);
    int splits = 1;
    const size_t slab = (size_t)rows * n_rhs * sizeof(float);
    if (d_ws && !((uintptr_t)d_ws & 15u)) {
        for (int cand = 2; cand <= 8; ++cand)
            if (kblocks % cand == 0 && (size_t)cand * slab <= ws_bytes && (int64_t)grid * (cand - 1) < kSMs * 4)
                splits = cand;
    }
    float* out = splits > 1 ? static_cast<float*>(d_ws) : d_y;
    const dim3 g(grid, splits);
    const int per = kblocks / splits;
    int rc, block_shift = 0;
    while ((1 << block_shift) < block_size) ++block_shift;
    CUtensorMap x_map;
    if ((rc = make_x_map(d_x, cols, n_rhs, &x_map))) return rc;
    if (scale_dtype == BOF4_F32) {
        constexpr auto kern = gemm_tc_kernel<F32>;
        if ((rc = ensure_dynamic_smem<kern>(kTcSmem))) return rc;
        kern<<<g, kTcThreads, kTcSmem, st>>>(d_codes, d_scales, cols, block_shift, d_codebook, x_map, n_rhs, out, per,
                                             d_status);
    } else {
        constexpr auto kern = gemm_tc_kernel<BF16>;
        if ((rc = ensure_dynamic_smem<kern>(kTcSmem))) return rc;
        kern<<<g, kTcThreads, kTcSmem, st>>>(d_codes, d_scales, cols, block_shift, d_codebook, x_map, n_rhs, out, per,
                                             d_status);
    }
    BOF4_CUDA_TRY(cudaGetLastError());
    if (splits > 1) {
        gemm_tc_reduce_kernel<<<kSMs * 4, 256, 0, st>>>(out, splits, (int64_t)rows * n_rhs, d_y);
        BOF4_CUDA_TRY(cudaGetLastError());
    }
    if (opq && capacity > 0) {
        const uint16_t* val = static_cast<const uint16_t*>(d_out_val);
        const uint16_t* xb = static_cast<const uint16_t*>(d_x);
        if (scale_dtype == BOF4_F32)
            gemm_tc_outlier_kernel<F32><<<kSMs * 4, 256, 0, st>>>(d_codes, d_scales, rows, cols, block_shift, d_codebook, xb,
                                                                  n_rhs, d_out_idx, val, d_n_out, capacity, d_y);
        else
            gemm_tc_outlier_kernel<BF16><<<kSMs * 4, 256, 0, st>>>(d_codes, d_scales, rows, cols, block_shift, d_codebook, xb,
                                                                   n_rhs, d_out_idx, val, d_n_out, capacity, d_y);
        BOF4_CUDA_TRY(cudaGetLastError());
    }
    return BOF4_OK;
}
