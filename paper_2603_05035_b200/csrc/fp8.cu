// E4M3 operands for the offloaded product (the paper's Limitations / Future Work list FP8 next to FP16; Eq. 2 is the
// product that runs on the untrusted accelerator, so that is the one whose operands are narrowed):
//   per-tensor quantiser   scale = max|x| / 448 (binary32),  code = nearest-even E4M3 of x / scale (binary32 division)
//   product                Y' = (s_U s_W) (U8 W8), fp32 accumulation on the tensor cores, stored in bf16
// The quantiser is three small launches: |x| maximum (integer atomic on the bit pattern, exact and order-free), the
// scale, the cast (16-byte loads, 8 codes per 8-byte store).
#include <cuda_fp8.h>

#include "common.cuh"

namespace gelo {

namespace {

__device__ __forceinline__ float widen8(const __nv_bfloat16* e, int j) { return __bfloat162float(e[j]); }
__device__ __forceinline__ float widen8(const __half* e, int j) { return __half2float(e[j]); }

template <typename T>
__global__ void __launch_bounds__(256) amax_kernel(const T* __restrict__ x, int rows, int cols, int ld, unsigned* __restrict__ amax_bits)
{
    constexpr int kVec = 16 / (int)sizeof(T);
    float m = 0.0f;
    const int groups = cols / kVec;                           // cols is a multiple of 8
    for (int r = blockIdx.y; r < rows; r += gridDim.y)
        for (int g = blockIdx.x * 256 + threadIdx.x; g < groups; g += gridDim.x * 256) {
            const uint4 raw = *reinterpret_cast<const uint4*>(x + (size_t)r * ld + g * kVec);
            if (sizeof(T) == 4) {
                const float* f = reinterpret_cast<const float*>(&raw);
#pragma unroll
                for (int j = 0; j < 4; ++j) m = fmaxf(m, fabsf(f[j]));
            } else {
                const T* e = reinterpret_cast<const T*>(&raw);
#pragma unroll
                for (int j = 0; j < kVec; ++j) m = fmaxf(m, fabsf(widen8(reinterpret_cast<const typename std::conditional<sizeof(T) == 4, __half, T>::type*>(e), j)));
            }
        }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, off));
    if ((threadIdx.x & 31) == 0 && m > 0.0f) atomicMax(amax_bits, __float_as_uint(m));   // non-negative floats order like their bits
}

__global__ void scale_kernel(const unsigned* __restrict__ amax_bits, float* __restrict__ scale)
{
    const float amax = __uint_as_float(*amax_bits);
    *scale = amax > 0.0f ? __fdiv_rn(amax, 448.0f) : 1.0f;
}

template <typename T>
__global__ void __launch_bounds__(256) cast_e4m3_kernel(const T* __restrict__ x, int rows, int cols, int ld, const float* __restrict__ scale,
                                                        uint8_t* __restrict__ out, int ldo)
{
    const float s = *scale;
    const int groups = cols / 8;
    for (int r = blockIdx.y; r < rows; r += gridDim.y)
        for (int g = blockIdx.x * 256 + threadIdx.x; g < groups; g += gridDim.x * 256) {
            float v[8];
            if (sizeof(T) == 4) {
                const float4 a = *reinterpret_cast<const float4*>(x + (size_t)r * ld + g * 8);
                const float4 b = *reinterpret_cast<const float4*>(x + (size_t)r * ld + g * 8 + 4);
                v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w; v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
            } else {
                const uint4 raw = *reinterpret_cast<const uint4*>(x + (size_t)r * ld + g * 8);
                const typename std::conditional<sizeof(T) == 4, __half, T>::type* e =
                    reinterpret_cast<const typename std::conditional<sizeof(T) == 4, __half, T>::type*>(&raw);
#pragma unroll
                for (int j = 0; j < 8; ++j) v[j] = widen8(e, j);
            }
            uint8_t c[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) c[j] = (uint8_t)__nv_cvt_float_to_fp8(__fdiv_rn(v[j], s), __NV_SATFINITE, __NV_E4M3);
            *reinterpret_cast<uint2*>(out + (size_t)r * ldo + g * 8) = *reinterpret_cast<const uint2*>(c);
        }
}

template <typename T>
int quantize_typed(gelo_ctx* ctx, const void* x, int rows, int cols, int ld, uint8_t* out, int ldo, float* scale, cudaStream_t st)
{
    unsigned* amax_bits = reinterpret_cast<unsigned*>(scale + 1);
    GELO_CUDA_OK(cudaMemsetAsync(amax_bits, 0, sizeof(unsigned), st));
    const int gx = ceil_div(cols / 8, 256) > 0 ? ceil_div(cols / 8, 256) : 1;
    int gy = ceil_div(4 * ctx->sm_count, gx);
    if (gy > rows) gy = rows;
    amax_kernel<T><<<dim3(gx, gy), 256, 0, st>>>(static_cast<const T*>(x), rows, cols, ld, amax_bits);
    GELO_TRY(after_launch(ctx));
    scale_kernel<<<1, 1, 0, st>>>(amax_bits, scale);
    GELO_TRY(after_launch(ctx));
    cast_e4m3_kernel<T><<<dim3(gx, gy), 256, 0, st>>>(static_cast<const T*>(x), rows, cols, ld, scale, out, ldo);
    return after_launch(ctx);
}

}  // namespace

// out (rows x cols E4M3 codes, row stride ldo bytes) and scale[0] from x (rows x cols of `dtype`, row stride ld);
// scale[1] is scratch for the maximum.  cols a multiple of 8, ld a multiple of 8 (4 for fp32 pairs of loads), ldo a multiple of 8.
int launch_quantize_e4m3(gelo_ctx* ctx, const void* x, int rows, int cols, int ld, int dtype, void* out, int ldo, float* scale,
                         cudaStream_t st)
{
    if (rows <= 0 || cols <= 0) return GELO_OK;
    if ((cols % 8) || (ld % 8) || (ldo % 8) || ld < cols || ldo < cols) return GELO_ERR_INVALID;
    if (dtype == GELO_BF16) return quantize_typed<__nv_bfloat16>(ctx, x, rows, cols, ld, static_cast<uint8_t*>(out), ldo, scale, st);
    if (dtype == GELO_F16) return quantize_typed<__half>(ctx, x, rows, cols, ld, static_cast<uint8_t*>(out), ldo, scale, st);
    return quantize_typed<float>(ctx, x, rows, cols, ld, static_cast<uint8_t*>(out), ldo, scale, st);
}

}  // namespace gelo
