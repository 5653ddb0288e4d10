// Double quantisation of the block constants (Limitations; App. F): the constants of 256
// consecutive blocks share one fp32 group constant g (their largest magnitude) and each keeps an
// 8-bit code q = round-half-even(|m| / (g / 255)); under signed normalisation (Sec. 3.1) the sign
// of every constant is kept in a bit array, so that the second quantiser only sees magnitudes.
// The decoder's constant is m^ = +-(g / 255) * q, all in fp32.  The weights' 4-bit codes are not
// touched: they were formed with the exact constant.
//
// Both directions are one small streaming pass over the constants (one or four bytes per block
// of weights, against block_size / 2 bytes of codes), one CTA of 256 threads per group.
#include "common.cuh"

namespace bof4 {

constexpr int kDqGroup = 256;

template <class ST>
__device__ __forceinline__ float read_constant(const void* scales, int64_t b);
template <>
__device__ __forceinline__ float read_constant<F32>(const void* scales, int64_t b)
{
    return static_cast<const float*>(scales)[b];
}
template <>
__device__ __forceinline__ float read_constant<BF16>(const void* scales, int64_t b)
{
    return __uint_as_float((uint32_t)static_cast<const uint16_t*>(scales)[b] << 16);
}

template <class ST>
__global__ void __launch_bounds__(kDqGroup)
scales_compress_kernel(const void* __restrict__ scales, int64_t n_blocks, uint8_t* __restrict__ q,
                       float* __restrict__ group, uint8_t* __restrict__ sign_bytes)
{
    __shared__ uint32_t s_max[kDqGroup / 32];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    for (int64_t k = blockIdx.x; k * kDqGroup < n_blocks; k += gridDim.x) {
        const int64_t b = k * kDqGroup + tid;
        const float m = (b < n_blocks) ? read_constant<ST>(scales, b) : 0.0f;
        const float a = fabsf(m);
        uint32_t bits = __float_as_uint(a);  // non-negative floats order like their bits
#pragma unroll
        for (int off = 16; off; off >>= 1) bits = max(bits, __shfl_xor_sync(kFull, bits, off));
        __syncthreads();  // s_max may still be read from the previous group
        if (lane == 0) s_max[warp] = bits;
        __syncthreads();
#pragma unroll
        for (int w = 0; w < kDqGroup / 32; ++w) bits = max(bits, s_max[w]);
        const float g = __uint_as_float(bits);
        const float t = __fdiv_rn(g, 255.0f);
        if (b < n_blocks) {
            const float r = (t == 0.0f) ? 0.0f : fminf(rintf(__fdiv_rn(a, t)), 255.0f);
            q[b] = (uint8_t)r;
        }
        if (tid == 0) group[k] = g;
        if (sign_bytes) {
            // bit (b mod 8) of byte (b div 8): a warp's 32 blocks are four bytes, written byte by byte
            // (the array's length need not be a multiple of four)
            const uint32_t word = __ballot_sync(kFull, m < 0.0f);
            const int64_t byte0 = (k * kDqGroup + warp * 32) / 8;
            if (lane < 4 && byte0 * 8 + lane * 8 < n_blocks) sign_bytes[byte0 + lane] = (uint8_t)(word >> (8 * lane));
        }
    }
}

__global__ void __launch_bounds__(kDqGroup)
scales_expand_kernel(const uint8_t* __restrict__ q, const float* __restrict__ group,
                     const uint8_t* __restrict__ sign_bytes, int64_t n_blocks, float* __restrict__ out)
{
    const int tid = threadIdx.x;
    for (int64_t k = blockIdx.x; k * kDqGroup < n_blocks; k += gridDim.x) {
        const int64_t b = k * kDqGroup + tid;
        if (b >= n_blocks) continue;
        const float t = __fdiv_rn(group[k], 255.0f);
        float m = __fmul_rn(t, (float)q[b]);
        if (sign_bytes && ((sign_bytes[b >> 3] >> (b & 7)) & 1)) m = -m;
        out[b] = m;
    }
}

}  // namespace bof4

using namespace bof4;

extern "C" int bof4_scales_compress(const void* d_scales, int scale_dtype, int64_t n_blocks, int norm,
                                    uint8_t* d_q, float* d_group, uint8_t* d_sign, void* stream)
{
    if (n_blocks < 0 || (norm != BOF4_NORM_ABS && norm != BOF4_NORM_SIGNED)) {
        set_error("bof4_scales_compress: negative block count or bad norm");
        return BOF4_ERR_INVALID_ARG;
    }
    if (scale_dtype != BOF4_F32 && scale_dtype != BOF4_BF16) {
        set_error("bof4_scales_compress: unknown scale dtype %d", scale_dtype);
        return BOF4_ERR_DTYPE;
    }
    if (n_blocks == 0) return BOF4_OK;
    if (!d_scales || !d_q || !d_group || (norm == BOF4_NORM_SIGNED && !d_sign)) {
        set_error("bof4_scales_compress: NULL pointer (signed normalisation needs d_sign)");
        return BOF4_ERR_INVALID_ARG;
    }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int64_t groups = (n_blocks + kDqGroup - 1) / kDqGroup;
    const int grid = (int)(groups < 148 * 8 ? groups : 148 * 8);
    uint8_t* sg = norm == BOF4_NORM_SIGNED ? d_sign : nullptr;
    if (scale_dtype == BOF4_F32)
        scales_compress_kernel<F32><<<grid, kDqGroup, 0, st>>>(d_scales, n_blocks, d_q, d_group, sg);
    else
        scales_compress_kernel<BF16><<<grid, kDqGroup, 0, st>>>(d_scales, n_blocks, d_q, d_group, sg);
    BOF4_CUDA_TRY(cudaGetLastError());
    return BOF4_OK;
}

extern "C" int bof4_scales_expand(const uint8_t* d_q, const float* d_group, const uint8_t* d_sign,
                                  int64_t n_blocks, float* d_scales_out, void* stream)
{
    if (n_blocks < 0) {
        set_error("bof4_scales_expand: negative block count");
        return BOF4_ERR_INVALID_ARG;
    }
    if (n_blocks == 0) return BOF4_OK;
    if (!d_q || !d_group || !d_scales_out) {
        set_error("bof4_scales_expand: NULL pointer");
        return BOF4_ERR_INVALID_ARG;
    }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int64_t groups = (n_blocks + kDqGroup - 1) / kDqGroup;
    const int grid = (int)(groups < 148 * 8 ? groups : 148 * 8);
    scales_expand_kernel<<<grid, kDqGroup, 0, st>>>(d_q, d_group, d_sign, n_blocks, d_scales_out);
    BOF4_CUDA_TRY(cudaGetLastError());
    return BOF4_OK;
}
