// Element-type and layout conversions of the m x m mixing matrices: fp32 working
// copies to the stored type, and the transpose that serves as the inverse of an
// orthogonal A ("If A is orthogonal, A^-1 = A^T", paper Section 3.2 step 3).
#include "common.cuh"

namespace gelo {

namespace {

__device__ __forceinline__ void put(float* p, float v) { *p = v; }
__device__ __forceinline__ void put(__nv_bfloat16* p, float v) { *p = __float2bfloat16_rn(v); }
__device__ __forceinline__ float get(const float* p) { return *p; }
__device__ __forceinline__ float get(const __nv_bfloat16* p) { return __bfloat162float(*p); }

// dst = src (optionally column-signed); dstT = dst^T.  32 x 32 tiles through shared memory
// so that both the read and the two writes are coalesced.
template <typename T>
__global__ void __launch_bounds__(256) finish_mixing_kernel(int m, const float* __restrict__ src, int lds,
                                                            const float* __restrict__ sign_diag, int ldg,
                                                            T* __restrict__ dst, T* __restrict__ dstT, int ldd)
{
    __shared__ float tile[32][33];
    const int r0 = blockIdx.y * 32, c0 = blockIdx.x * 32;
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
    for (int i = ty; i < 32; i += 8) {
        const int r = r0 + i, c = c0 + tx;
        float v = 0.0f;
        if (r < m && c < m) {
            v = src[(size_t)r * lds + c];
            if (sign_diag && sign_diag[(size_t)c * ldg + c] < 0.0f) v = -v;
            put(dst + (size_t)r * ldd + c, v);
            v = get(dst + (size_t)r * ldd + c);      // the transpose holds the stored (rounded) value
        }
        tile[i][tx] = v;
    }
    __syncthreads();
    if (dstT) {
        for (int i = ty; i < 32; i += 8) {
            const int r = c0 + i, c = r0 + tx;       // transposed coordinates
            if (r < m && c < m) put(dstT + (size_t)r * ldd + c, tile[tx][i]);
        }
    }
}

template <typename TS, typename TD>
__global__ void __launch_bounds__(256) convert_kernel(int m, const TS* __restrict__ src, int lds, TD* __restrict__ dst, int ldd)
{
    const int c = blockIdx.x * blockDim.x + threadIdx.x;
    const int r = blockIdx.y;
    if (c < m) put(dst + (size_t)r * ldd + c, get(src + (size_t)r * lds + c));
}

// hi = bf16(x), lo = bf16(x - hi) for a rows x cols block (fp32, stride lds) -> bf16 pair (stride ldo);
// with T the pair is written transposed (cols x rows, stride ldo) through a shared-memory tile.
__global__ void __launch_bounds__(256) split_kernel(const float* __restrict__ src, int lds, int rows, int cols,
                                                    __nv_bfloat16* __restrict__ hi, __nv_bfloat16* __restrict__ lo, int ldo)
{
    const int c = blockIdx.x * 256 + threadIdx.x;
    const int r = blockIdx.y;
    if (c >= cols) return;
    const float x = src[(size_t)r * lds + c];
    const __nv_bfloat16 h = __float2bfloat16_rn(x);
    hi[(size_t)r * ldo + c] = h;
    lo[(size_t)r * ldo + c] = __float2bfloat16_rn(x - __bfloat162float(h));
}

__global__ void __launch_bounds__(256) split_transpose_kernel(const float* __restrict__ src, int lds, int rows, int cols,
                                                              __nv_bfloat16* __restrict__ hi, __nv_bfloat16* __restrict__ lo, int ldo)
{
    __shared__ float tile[32][33];
    const int r0 = blockIdx.y * 32, c0 = blockIdx.x * 32;
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
    for (int i = ty; i < 32; i += 8) {
        const int r = r0 + i, c = c0 + tx;
        tile[i][tx] = (r < rows && c < cols) ? src[(size_t)r * lds + c] : 0.0f;
    }
    __syncthreads();
    for (int i = ty; i < 32; i += 8) {
        const int c = c0 + i, r = r0 + tx;              // output row = source column
        if (c < cols && r < rows) {
            const float x = tile[tx][i];
            const __nv_bfloat16 h = __float2bfloat16_rn(x);
            hi[(size_t)c * ldo + r] = h;
            lo[(size_t)c * ldo + r] = __float2bfloat16_rn(x - __bfloat162float(h));
        }
    }
}

}  // namespace

int launch_split(gelo_ctx* ctx, const float* src, int lds, int rows, int cols, void* hi, void* lo, int ldo,
                 bool transpose, cudaStream_t st)
{
    if (rows <= 0 || cols <= 0) return GELO_OK;
    if (transpose) {
        dim3 grid(ceil_div(cols, 32), ceil_div(rows, 32));
        split_transpose_kernel<<<grid, 256, 0, st>>>(src, lds, rows, cols, static_cast<__nv_bfloat16*>(hi),
                                                     static_cast<__nv_bfloat16*>(lo), ldo);
    } else {
        dim3 grid(ceil_div(cols, 256), rows);
        split_kernel<<<grid, 256, 0, st>>>(src, lds, rows, cols, static_cast<__nv_bfloat16*>(hi),
                                           static_cast<__nv_bfloat16*>(lo), ldo);
    }
    return after_launch(ctx);
}

int launch_finish_mixing(gelo_ctx* ctx, int m, const float* src, int lds, const float* sign_diag, int ldg,
                         int dtype, void* dst, void* dstT, int ldd, cudaStream_t st)
{
    dim3 grid(ceil_div(m, 32), ceil_div(m, 32));
    if (dtype == GELO_BF16)
        finish_mixing_kernel<__nv_bfloat16><<<grid, 256, 0, st>>>(m, src, lds, sign_diag, ldg,
            static_cast<__nv_bfloat16*>(dst), static_cast<__nv_bfloat16*>(dstT), ldd);
    else
        finish_mixing_kernel<float><<<grid, 256, 0, st>>>(m, src, lds, sign_diag, ldg,
            static_cast<float*>(dst), static_cast<float*>(dstT), ldd);
    return after_launch(ctx);
}

int launch_widen(gelo_ctx* ctx, int m, const void* src, int lds, int dtype, float* dst, int ldd, cudaStream_t st)
{
    dim3 grid(ceil_div(m, 256), m);
    if (dtype == GELO_BF16)
        convert_kernel<__nv_bfloat16, float><<<grid, 256, 0, st>>>(m, static_cast<const __nv_bfloat16*>(src), lds, dst, ldd);
    else
        convert_kernel<float, float><<<grid, 256, 0, st>>>(m, static_cast<const float*>(src), lds, dst, ldd);
    return after_launch(ctx);
}

int launch_narrow(gelo_ctx* ctx, int m, const float* src, int lds, int dtype, void* dst, int ldd, cudaStream_t st)
{
    dim3 grid(ceil_div(m, 256), m);
    if (dtype == GELO_BF16)
        convert_kernel<float, __nv_bfloat16><<<grid, 256, 0, st>>>(m, src, lds, static_cast<__nv_bfloat16*>(dst), ldd);
    else
        convert_kernel<float, float><<<grid, 256, 0, st>>>(m, src, lds, static_cast<float*>(dst), ldd);
    return after_launch(ctx);
}

}  // namespace gelo
