// Element-type and layout conversions of the m x m mixing matrices: fp32 working
// copies to the stored type, and the transpose that serves as the inverse of an
// orthogonal A ("If A is orthogonal, A^-1 = A^T", paper Section 3.2 step 3).
#include "common.cuh"

namespace gelo {

namespace {

__device__ __forceinline__ void put(float* p, float v) { *p = v; }
__device__ __forceinline__ void put(__nv_bfloat16* p, float v) { *p = __float2bfloat16_rn(v); }
__device__ __forceinline__ void put(__half* p, float v) { *p = __float2half_rn(v); }
__device__ __forceinline__ float get(const __half* p) { return __half2float(*p); }
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

// dst = convert(src) for an m x m matrix, four consecutive columns per thread (rows start 16-byte aligned for the
// wider of the two types, which every row stride of this library guarantees); `back`, if given, receives the stored
// values widened again (what a later fp32 computation on the stored matrix must start from).
__device__ __forceinline__ void load4(const float* p, float (&x)[4])
{
    const float4 t = *reinterpret_cast<const float4*>(p);
    x[0] = t.x; x[1] = t.y; x[2] = t.z; x[3] = t.w;
}
__device__ __forceinline__ void store4(float* p, const float (&x)[4]) { *reinterpret_cast<float4*>(p) = make_float4(x[0], x[1], x[2], x[3]); }
__device__ __forceinline__ void store4(__nv_bfloat16* p, float (&x)[4])
{
    __nv_bfloat162 a = __floats2bfloat162_rn(x[0], x[1]), b = __floats2bfloat162_rn(x[2], x[3]);
    uint2 t;
    t.x = *reinterpret_cast<uint32_t*>(&a); t.y = *reinterpret_cast<uint32_t*>(&b);
    *reinterpret_cast<uint2*>(p) = t;
    const float2 fa = __bfloat1622float2(a), fb = __bfloat1622float2(b);
    x[0] = fa.x; x[1] = fa.y; x[2] = fb.x; x[3] = fb.y;       // the stored values
}

__device__ __forceinline__ void store4(__half* p, float (&x)[4])
{
    __half2 a = __floats2half2_rn(x[0], x[1]), b = __floats2half2_rn(x[2], x[3]);
    uint2 t;
    t.x = *reinterpret_cast<uint32_t*>(&a); t.y = *reinterpret_cast<uint32_t*>(&b);
    *reinterpret_cast<uint2*>(p) = t;
    const float2 fa = __half22float2(a), fb = __half22float2(b);
    x[0] = fa.x; x[1] = fa.y; x[2] = fb.x; x[3] = fb.y;       // the stored values
}

template <typename TS, typename TD>
__global__ void __launch_bounds__(256) convert_kernel(int m, const TS* __restrict__ src, int lds, TD* __restrict__ dst, int ldd,
                                                      float* __restrict__ back, int ldb)
{
    const int c4 = (blockIdx.x * blockDim.x + threadIdx.x) * 4;
    const int r = blockIdx.y;
    if (c4 >= m) return;
    if (c4 + 3 < m) {
        float x[4];
        load4(src + (size_t)r * lds + c4, x);
        store4(dst + (size_t)r * ldd + c4, x);
        if (back) *reinterpret_cast<float4*>(back + (size_t)r * ldb + c4) = make_float4(x[0], x[1], x[2], x[3]);
    } else {
        for (int c = c4; c < m; ++c) {
            put(dst + (size_t)r * ldd + c, get(src + (size_t)r * lds + c));
            if (back) back[(size_t)r * ldb + c] = get(dst + (size_t)r * ldd + c);
        }
    }
}

// hi = bf16(x), lo = bf16(x - hi) for a rows x cols block (fp32, stride lds) -> bf16 pair (stride ldo);
// with T the pair is written transposed (cols x rows, stride ldo) through a shared-memory tile.
__global__ void __launch_bounds__(256) split_kernel(const float* __restrict__ src, int lds, int rows, int cols,
                                                    __nv_bfloat16* __restrict__ hi, __nv_bfloat16* __restrict__ lo, int ldo,
                                                    int vec)
{
    // grid-stride over rows; a thread converts four consecutive columns (16-byte load, two 8-byte stores)
    const int c4 = (blockIdx.x * 256 + threadIdx.x) * 4;
    if (c4 >= cols) return;
    for (int r = blockIdx.y; r < rows; r += gridDim.y) {
        const float* p = src + (size_t)r * lds + c4;
        float x[4];
        if (vec && c4 + 3 < cols) {
            const float4 t = *reinterpret_cast<const float4*>(p);
            x[0] = t.x; x[1] = t.y; x[2] = t.z; x[3] = t.w;
        } else {
#pragma unroll
            for (int j = 0; j < 4; ++j) x[j] = (c4 + j < cols) ? p[j] : 0.0f;
        }
        __nv_bfloat16 h[4], l[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            h[j] = __float2bfloat16_rn(x[j]);
            l[j] = __float2bfloat16_rn(x[j] - __bfloat162float(h[j]));
        }
        __nv_bfloat16* ph = hi + (size_t)r * ldo + c4;
        __nv_bfloat16* pl = lo + (size_t)r * ldo + c4;
        if (vec && c4 + 3 < cols) {
            *reinterpret_cast<uint2*>(ph) = *reinterpret_cast<const uint2*>(h);
            *reinterpret_cast<uint2*>(pl) = *reinterpret_cast<const uint2*>(l);
        } else {
#pragma unroll
            for (int j = 0; j < 4; ++j)
                if (c4 + j < cols) { ph[j] = h[j]; pl[j] = l[j]; }
        }
    }
}

// hi/lo pair of the sum of `parts` fp32 planes (fixed order): the second half of a split-K product.
__global__ void __launch_bounds__(256) sum_split_kernel(const float* __restrict__ planes, size_t plane, int parts,
                                                        int ld, int rows, int cols, __nv_bfloat16* __restrict__ hi,
                                                        __nv_bfloat16* __restrict__ lo, int ldo)
{
    const int c4 = (blockIdx.x * 256 + threadIdx.x) * 4;
    const int r = blockIdx.y;
    if (c4 >= cols) return;                                   // cols is a multiple of 8, rows start 16-byte aligned
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int q = 0; q < parts; ++q) {
        const float4 t = *reinterpret_cast<const float4*>(planes + q * plane + (size_t)r * ld + c4);
        acc.x += t.x; acc.y += t.y; acc.z += t.z; acc.w += t.w;
    }
    const float x[4] = {acc.x, acc.y, acc.z, acc.w};
    __nv_bfloat16 h[4], l[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        h[j] = __float2bfloat16_rn(x[j]);
        l[j] = __float2bfloat16_rn(x[j] - __bfloat162float(h[j]));
    }
    *reinterpret_cast<uint2*>(hi + (size_t)r * ldo + c4) = *reinterpret_cast<const uint2*>(h);
    *reinterpret_cast<uint2*>(lo + (size_t)r * ldo + c4) = *reinterpret_cast<const uint2*>(l);
}

// Sum of `parts` fp32 planes (fixed order), rounded to tf32: the second half of a split-K tf32 product whose
// result feeds the next tf32 product.
__global__ void __launch_bounds__(256) sum_planes_kernel(const float* __restrict__ planes, size_t plane, int parts,
                                                         int ld, int rows, int cols, float scale, float* __restrict__ out,
                                                         int ldo)
{
    const int c4 = (blockIdx.x * 256 + threadIdx.x) * 4;
    const int r = blockIdx.y;
    if (c4 >= cols) return;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int q = 0; q < parts; ++q) {
        const float4 t = *reinterpret_cast<const float4*>(planes + q * plane + (size_t)r * ld + c4);
        acc.x += t.x; acc.y += t.y; acc.z += t.z; acc.w += t.w;
    }
    uint32_t o[4];
    asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(o[0]) : "f"(scale * acc.x));
    asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(o[1]) : "f"(scale * acc.y));
    asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(o[2]) : "f"(scale * acc.z));
    asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(o[3]) : "f"(scale * acc.w));
    *reinterpret_cast<uint4*>(out + (size_t)r * ldo + c4) = make_uint4(o[0], o[1], o[2], o[3]);
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

// Two split jobs in one launch (blockIdx.z selects the job): the A and B operands of one split-precision update.  A
// row takes min(256, cols / 4) threads (four columns each), the rest of the CTA's threads take further rows, so a thin
// block column keeps all 256 threads busy.
struct SplitJob { const float* src; int lds, rows, cols; __nv_bfloat16* hi; __nv_bfloat16* lo; int ldo, tpr; };

__global__ void __launch_bounds__(256) split_pair_kernel(const SplitJob ja, const SplitJob jb)
{
    const SplitJob& j = blockIdx.z ? jb : ja;
    const int tpr = j.tpr;                                   // threads per row (a power of two <= 256)
    const int c4 = (blockIdx.x * tpr + (threadIdx.x & (tpr - 1))) * 4;
    const int rpc = 256 / tpr;                               // rows per CTA and pass
    if (c4 >= j.cols) return;
    for (int r = blockIdx.y * rpc + threadIdx.x / tpr; r < j.rows; r += gridDim.y * rpc) {
        const float* p = j.src + (size_t)r * j.lds + c4;
        float x[4];
        if (c4 + 3 < j.cols) {
            const float4 t = *reinterpret_cast<const float4*>(p);
            x[0] = t.x; x[1] = t.y; x[2] = t.z; x[3] = t.w;
        } else {
#pragma unroll
            for (int q = 0; q < 4; ++q) x[q] = (c4 + q < j.cols) ? p[q] : 0.0f;
        }
        __nv_bfloat16 h[4], l[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            h[q] = __float2bfloat16_rn(x[q]);
            l[q] = __float2bfloat16_rn(x[q] - __bfloat162float(h[q]));
        }
        __nv_bfloat16* ph = j.hi + (size_t)r * j.ldo + c4;
        __nv_bfloat16* pl = j.lo + (size_t)r * j.ldo + c4;
        if (c4 + 3 < j.cols) {
            *reinterpret_cast<uint2*>(ph) = *reinterpret_cast<const uint2*>(h);
            *reinterpret_cast<uint2*>(pl) = *reinterpret_cast<const uint2*>(l);
        } else {
#pragma unroll
            for (int q = 0; q < 4; ++q)
                if (c4 + q < j.cols) { ph[q] = h[q]; pl[q] = l[q]; }
        }
    }
}

}  // namespace

int launch_split_pair(gelo_ctx* ctx, const float* A, int lda, int rows_a, int cols_a, void* Ahi, void* Alo, int ldoa,
                      const float* B, int ldb, int rows_b, int cols_b, void* Bhi, void* Blo, int ldob, cudaStream_t st)
{
    auto vec_ok = [](const float* s, int lds, const void* hi, const void* lo, int ldo) {
        return (lds & 3) == 0 && (ldo & 3) == 0 && (reinterpret_cast<uintptr_t>(s) & 15u) == 0 &&
               (reinterpret_cast<uintptr_t>(hi) & 7u) == 0 && (reinterpret_cast<uintptr_t>(lo) & 7u) == 0;
    };
    if (rows_a <= 0 || cols_a <= 0 || rows_b <= 0 || cols_b <= 0 || !vec_ok(A, lda, Ahi, Alo, ldoa) || !vec_ok(B, ldb, Bhi, Blo, ldob)) {
        GELO_TRY(launch_split(ctx, A, lda, rows_a, cols_a, Ahi, Alo, ldoa, false, st));
        return launch_split(ctx, B, ldb, rows_b, cols_b, Bhi, Blo, ldob, false, st);
    }
    auto job = [](const float* s, int lds, int rows, int cols, void* hi, void* lo, int ldo) {
        SplitJob j;
        j.src = s; j.lds = lds; j.rows = rows; j.cols = cols;
        j.hi = static_cast<__nv_bfloat16*>(hi); j.lo = static_cast<__nv_bfloat16*>(lo); j.ldo = ldo;
        int tpr = 1;
        while (tpr < 256 && tpr * 4 < cols) tpr *= 2;
        j.tpr = tpr;
        return j;
    };
    const SplitJob ja = job(A, lda, rows_a, cols_a, Ahi, Alo, ldoa), jb = job(B, ldb, rows_b, cols_b, Bhi, Blo, ldob);
    auto gx = [](const SplitJob& j) { return ceil_div(j.cols, 4 * j.tpr); };
    auto gy = [](const SplitJob& j) { return ceil_div(j.rows, 256 / j.tpr); };
    const int grid_x = gx(ja) > gx(jb) ? gx(ja) : gx(jb);
    int grid_y = gy(ja) > gy(jb) ? gy(ja) : gy(jb);
    const int cap = ceil_div(4 * ctx->sm_count, grid_x);      // a few CTAs per SM and job; rows beyond that are strided
    if (grid_y > cap) grid_y = cap;
    split_pair_kernel<<<dim3(grid_x, grid_y, 2), 256, 0, st>>>(ja, jb);
    return after_launch(ctx);
}

int launch_split(gelo_ctx* ctx, const float* src, int lds, int rows, int cols, void* hi, void* lo, int ldo,
                 bool transpose, cudaStream_t st)
{
    if (rows <= 0 || cols <= 0) return GELO_OK;
    if (transpose) {
        dim3 grid(ceil_div(cols, 32), ceil_div(rows, 32));
        split_transpose_kernel<<<grid, 256, 0, st>>>(src, lds, rows, cols, static_cast<__nv_bfloat16*>(hi),
                                                     static_cast<__nv_bfloat16*>(lo), ldo);
    } else {
        const int vec = ((lds & 3) == 0 && (ldo & 3) == 0 && (reinterpret_cast<uintptr_t>(src) & 15u) == 0 &&
                         (reinterpret_cast<uintptr_t>(hi) & 7u) == 0 && (reinterpret_cast<uintptr_t>(lo) & 7u) == 0) ? 1 : 0;
        const int gx = ceil_div(cols, 1024);
        int gy = ceil_div(8 * ctx->sm_count, gx);
        if (gy > rows) gy = rows;
        dim3 grid(gx, gy);
        split_kernel<<<grid, 256, 0, st>>>(src, lds, rows, cols, static_cast<__nv_bfloat16*>(hi),
                                           static_cast<__nv_bfloat16*>(lo), ldo, vec);
    }
    return after_launch(ctx);
}

int launch_sum_split(gelo_ctx* ctx, const float* planes, size_t plane, int parts, int ld, int rows, int cols, void* hi,
                     void* lo, int ldo, cudaStream_t st)
{
    if (rows <= 0 || cols <= 0) return GELO_OK;
    dim3 grid(ceil_div(cols, 1024), rows);
    sum_split_kernel<<<grid, 256, 0, st>>>(planes, plane, parts, ld, rows, cols, static_cast<__nv_bfloat16*>(hi),
                                           static_cast<__nv_bfloat16*>(lo), ldo);
    return after_launch(ctx);
}

// hi = x rounded to tf32, lo = (x - hi) rounded to tf32: both pass through the tensor core unchanged
__global__ void __launch_bounds__(256) split_tf32_kernel(const float* __restrict__ src, int lds, int rows, int cols,
                                                         float* __restrict__ hi, float* __restrict__ lo, int ldo)
{
    const int c4 = (blockIdx.x * 256 + threadIdx.x) * 4;
    if (c4 >= cols) return;
    for (int r = blockIdx.y; r < rows; r += gridDim.y) {
        const float4 t = *reinterpret_cast<const float4*>(src + (size_t)r * lds + c4);
        const float x[4] = {t.x, t.y, t.z, t.w};
        uint32_t h[4], l[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(h[j]) : "f"(x[j]));
            asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(l[j]) : "f"(x[j] - __uint_as_float(h[j])));
        }
        *reinterpret_cast<uint4*>(hi + (size_t)r * ldo + c4) = make_uint4(h[0], h[1], h[2], h[3]);
        *reinterpret_cast<uint4*>(lo + (size_t)r * ldo + c4) = make_uint4(l[0], l[1], l[2], l[3]);
    }
}

__global__ void __launch_bounds__(256) sum_planes_routed_kernel(const float* __restrict__ planes, size_t plane, int parts,
                                                                int cols, float* __restrict__ C0, float* __restrict__ C1,
                                                                float* __restrict__ C2, int ldc, int csplit)
{
    const int c4 = (blockIdx.x * 256 + threadIdx.x) * 4;
    const int r = blockIdx.y;
    if (c4 >= cols) return;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int q = 0; q < parts; ++q) {
        const float4 t = *reinterpret_cast<const float4*>(planes + q * plane + (size_t)r * cols + c4);
        acc.x += t.x; acc.y += t.y; acc.z += t.z; acc.w += t.w;
    }
    const int chunk = c4 / csplit;                            // csplit is a multiple of 8: a group of four never straddles
    float* base = chunk == 0 ? C0 : (chunk == 1 ? C1 : C2);
    *reinterpret_cast<float4*>(base + (size_t)r * ldc + (c4 - chunk * csplit)) = acc;
}

int launch_sum_planes_routed(gelo_ctx* ctx, const float* planes, size_t plane, int parts, int rows, int cols,
                             float* const C[3], int ldc, int csplit, cudaStream_t st)
{
    if (rows <= 0 || cols <= 0) return GELO_OK;
    dim3 grid(ceil_div(cols, 1024), rows);
    sum_planes_routed_kernel<<<grid, 256, 0, st>>>(planes, plane, parts, cols, C[0], C[1], C[2], ldc, csplit);
    return after_launch(ctx);
}

int launch_split_tf32(gelo_ctx* ctx, const float* src, int lds, int rows, int cols, float* hi, float* lo, int ldo,
                      cudaStream_t st)
{
    if (rows <= 0 || cols <= 0) return GELO_OK;
    if ((cols % 4) || (lds % 4) || (ldo % 4) || (reinterpret_cast<uintptr_t>(src) & 15u) ||
        (reinterpret_cast<uintptr_t>(hi) & 15u) || (reinterpret_cast<uintptr_t>(lo) & 15u))
        return GELO_ERR_INVALID;
    dim3 grid(ceil_div(cols, 1024), rows < 4096 ? rows : 4096);
    split_tf32_kernel<<<grid, 256, 0, st>>>(src, lds, rows, cols, hi, lo, ldo);
    return after_launch(ctx);
}

int launch_sum_planes(gelo_ctx* ctx, const float* planes, size_t plane, int parts, int ld, int rows, int cols, float scale,
                      float* out, int ldo, cudaStream_t st)
{
    if (rows <= 0 || cols <= 0) return GELO_OK;
    dim3 grid(ceil_div(cols, 1024), rows);
    sum_planes_kernel<<<grid, 256, 0, st>>>(planes, plane, parts, ld, rows, cols, scale, out, ldo);
    return after_launch(ctx);
}

int launch_finish_mixing(gelo_ctx* ctx, int m, const float* src, int lds, const float* sign_diag, int ldg,
                         int dtype, void* dst, void* dstT, int ldd, cudaStream_t st)
{
    dim3 grid(ceil_div(m, 32), ceil_div(m, 32));
    if (dtype == GELO_BF16)
        finish_mixing_kernel<__nv_bfloat16><<<grid, 256, 0, st>>>(m, src, lds, sign_diag, ldg,
            static_cast<__nv_bfloat16*>(dst), static_cast<__nv_bfloat16*>(dstT), ldd);
    else if (dtype == GELO_F16)
        finish_mixing_kernel<__half><<<grid, 256, 0, st>>>(m, src, lds, sign_diag, ldg,
            static_cast<__half*>(dst), static_cast<__half*>(dstT), ldd);
    else
        finish_mixing_kernel<float><<<grid, 256, 0, st>>>(m, src, lds, sign_diag, ldg,
            static_cast<float*>(dst), static_cast<float*>(dstT), ldd);
    return after_launch(ctx);
}

int launch_narrow(gelo_ctx* ctx, int m, const float* src, int lds, int dtype, void* dst, int ldd, cudaStream_t st, float* back,
                  int ldb)
{
    if ((lds % 4) || (ldd % 4) || (back && (ldb % 4)) || (reinterpret_cast<uintptr_t>(src) & 15u) ||
        (reinterpret_cast<uintptr_t>(dst) & 15u) || (reinterpret_cast<uintptr_t>(back) & 15u))
        return GELO_ERR_INVALID;
    dim3 grid(ceil_div(m, 1024), m);
    if (dtype == GELO_BF16)
        convert_kernel<float, __nv_bfloat16><<<grid, 256, 0, st>>>(m, src, lds, static_cast<__nv_bfloat16*>(dst), ldd, back, ldb);
    else if (dtype == GELO_F16)
        convert_kernel<float, __half><<<grid, 256, 0, st>>>(m, src, lds, static_cast<__half*>(dst), ldd, back, ldb);
    else
        convert_kernel<float, float><<<grid, 256, 0, st>>>(m, src, lds, static_cast<float*>(dst), ldd, back, ldb);
    return after_launch(ctx);
}

}  // namespace gelo
