// Shared-memory tiled FFMA GEMM: C = alpha * op(A) op(B) + beta * C with fp32
// accumulation.  It is the fp32-exact path of the three products of the offload
// (Eq. 1-3) and the workhorse of the trailing updates in the blocked QR and LU.
// The B operand may be the vertical stack of two matrices (Eq. 8: H_full = [H; S])
// and the output may be split into column thirds (Q | K | V).
#include "common.cuh"

namespace gelo {

namespace {

constexpr int BK = 16;
constexpr int kThreads = 256;

struct GemmParams {
    int M, N, K;
    const void* A; int lda;
    const void* B; int ldb;
    const void* B2; int b_split;
    void* C0; void* C1; void* C2; int ldc; int csplit;
    float alpha, beta;
};

__device__ __forceinline__ float ldf(const float* p) { return __ldg(p); }
__device__ __forceinline__ float ldf(const __nv_bfloat16* p) { return __bfloat162float(*p); }
__device__ __forceinline__ float ldf(const __half* p) { return __half2float(*p); }
__device__ __forceinline__ float ldc(const __half* p) { return __half2float(*p); }
__device__ __forceinline__ void stf(__half* p, float v) { *p = __float2half_rn(v); }
__device__ __forceinline__ float ldc(const float* p) { return *p; }
__device__ __forceinline__ float ldc(const __nv_bfloat16* p) { return __bfloat162float(*p); }
__device__ __forceinline__ void stf(float* p, float v) { *p = v; }
__device__ __forceinline__ void stf(__nv_bfloat16* p, float v) { *p = __float2bfloat16_rn(v); }

template <typename T, bool TA, bool TB, int BM, int BN>
__global__ void __launch_bounds__(kThreads) gemm_simt_kernel(const GemmParams prm)
{
    constexpr int RM = BM / 64, RN = BN / 64;
    constexpr int LA = BM * BK / kThreads, LB = BN * BK / kThreads;
    __shared__ __align__(16) float As[BK][BM + 4];
    __shared__ __align__(16) float Bs[BK][BN + 4];

    const T* __restrict__ A = static_cast<const T*>(prm.A);
    const T* __restrict__ B = static_cast<const T*>(prm.B);
    const T* __restrict__ B2 = static_cast<const T*>(prm.B2);
    const int tid = threadIdx.x;
    const int m0 = blockIdx.y * BM, n0 = blockIdx.x * BN;
    const int ty = tid >> 4, tx = tid & 15;

    float acc[RM * 4][RN * 4];
#pragma unroll
    for (int i = 0; i < RM * 4; ++i)
#pragma unroll
        for (int j = 0; j < RN * 4; ++j) acc[i][j] = 0.0f;

    float ra[LA], rb[LB];

    auto fetch = [&](int k0) {
#pragma unroll
        for (int i = 0; i < LA; ++i) {
            const int idx = tid + i * kThreads;
            int r, kk;
            if (TA) { r = idx % BM; kk = idx / BM; } else { kk = idx % BK; r = idx / BK; }
            const int gm = m0 + r, gk = k0 + kk;
            float v = 0.0f;
            if (gm < prm.M && gk < prm.K)
                v = TA ? ldf(A + (size_t)gk * prm.lda + gm) : ldf(A + (size_t)gm * prm.lda + gk);
            ra[i] = v;
        }
#pragma unroll
        for (int i = 0; i < LB; ++i) {
            const int idx = tid + i * kThreads;
            int c, kk;
            if (TB) { kk = idx % BK; c = idx / BK; } else { c = idx % BN; kk = idx / BN; }
            const int gn = n0 + c, gk = k0 + kk;
            float v = 0.0f;
            if (gn < prm.N && gk < prm.K) {
                if (TB) v = ldf(B + (size_t)gn * prm.ldb + gk);
                else if (gk < prm.b_split) v = ldf(B + (size_t)gk * prm.ldb + gn);
                else v = ldf(B2 + (size_t)(gk - prm.b_split) * prm.ldb + gn);
            }
            rb[i] = v;
        }
    };
    auto stash = [&]() {
#pragma unroll
        for (int i = 0; i < LA; ++i) {
            const int idx = tid + i * kThreads;
            int r, kk;
            if (TA) { r = idx % BM; kk = idx / BM; } else { kk = idx % BK; r = idx / BK; }
            As[kk][r] = ra[i];
        }
#pragma unroll
        for (int i = 0; i < LB; ++i) {
            const int idx = tid + i * kThreads;
            int c, kk;
            if (TB) { kk = idx % BK; c = idx / BK; } else { c = idx % BN; kk = idx / BN; }
            Bs[kk][c] = rb[i];
        }
    };

    fetch(0);
    for (int k0 = 0; k0 < prm.K; k0 += BK) {
        stash();
        __syncthreads();
        if (k0 + BK < prm.K) fetch(k0 + BK);
#pragma unroll
        for (int kk = 0; kk < BK; ++kk) {
            float a[RM * 4], b[RN * 4];
#pragma unroll
            for (int i = 0; i < RM; ++i) {
                const float4 v = *reinterpret_cast<const float4*>(&As[kk][ty * 4 + i * 64]);
                a[4 * i] = v.x; a[4 * i + 1] = v.y; a[4 * i + 2] = v.z; a[4 * i + 3] = v.w;
            }
#pragma unroll
            for (int j = 0; j < RN; ++j) {
                const float4 v = *reinterpret_cast<const float4*>(&Bs[kk][tx * 4 + j * 64]);
                b[4 * j] = v.x; b[4 * j + 1] = v.y; b[4 * j + 2] = v.z; b[4 * j + 3] = v.w;
            }
#pragma unroll
            for (int i = 0; i < RM * 4; ++i)
#pragma unroll
                for (int j = 0; j < RN * 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
        }
        __syncthreads();
    }

    T* const Cs[3] = { static_cast<T*>(prm.C0), static_cast<T*>(prm.C1), static_cast<T*>(prm.C2) };
#pragma unroll
    for (int i = 0; i < RM * 4; ++i) {
        const int gm = m0 + ty * 4 + (i >> 2) * 64 + (i & 3);
        if (gm >= prm.M) continue;
#pragma unroll
        for (int j = 0; j < RN * 4; ++j) {
            const int gn = n0 + tx * 4 + (j >> 2) * 64 + (j & 3);
            if (gn >= prm.N) continue;
            const int chunk = gn / prm.csplit;
            T* p = Cs[chunk] + (size_t)gm * prm.ldc + (gn - chunk * prm.csplit);
            float v = prm.alpha * acc[i][j];
            if (prm.beta != 0.0f) v += prm.beta * ldc(p);
            stf(p, v);
        }
    }
}

template <typename T, bool TA, bool TB>
void launch_tiles(const GemmParams& p, bool small, cudaStream_t st)
{
    if (small) {
        dim3 grid(ceil_div(p.N, 64), ceil_div(p.M, 64));
        gemm_simt_kernel<T, TA, TB, 64, 64><<<grid, kThreads, 0, st>>>(p);
    } else {
        dim3 grid(ceil_div(p.N, 128), ceil_div(p.M, 128));
        gemm_simt_kernel<T, TA, TB, 128, 128><<<grid, kThreads, 0, st>>>(p);
    }
}

}  // namespace

int launch_gemm_simt(gelo_ctx* ctx, const GemmArgs& g, cudaStream_t st)
{
    if (g.M <= 0 || g.N <= 0) return GELO_OK;
    if (g.K < 0 || !g.A || !g.B || !g.C[0] || g.nsplit < 1 || g.nsplit > 3 || g.N % g.nsplit != 0)
        return GELO_ERR_INVALID;
    if (g.B2 && g.transB) return GELO_ERR_INVALID;
    for (int i = 0; i < g.nsplit; ++i)
        if (!g.C[i]) return GELO_ERR_INVALID;
    GemmParams p;
    p.M = g.M; p.N = g.N; p.K = g.K;
    p.A = g.A; p.lda = g.lda; p.B = g.B; p.ldb = g.ldb;
    p.B2 = g.B2 ? g.B2 : g.B; p.b_split = g.B2 ? g.b_split : g.K;
    p.C0 = g.C[0]; p.C1 = g.C[g.nsplit > 1 ? 1 : 0]; p.C2 = g.C[g.nsplit > 2 ? 2 : 0];
    p.ldc = g.ldc; p.csplit = g.N / g.nsplit;
    p.alpha = g.alpha; p.beta = g.beta;
    const long tiles128 = (long)ceil_div(g.M, 128) * ceil_div(g.N, 128);
    const bool small = g.M <= 64 || g.N <= 64 || tiles128 < 2L * ctx->sm_count;
    if (g.dtype == GELO_BF16) {
        if (g.transA || g.transB) return GELO_ERR_UNSUPPORTED;
        launch_tiles<__nv_bfloat16, false, false>(p, small, st);
    } else if (g.dtype == GELO_F16) {
        if (g.transA || g.transB) return GELO_ERR_UNSUPPORTED;
        launch_tiles<__half, false, false>(p, small, st);
    } else {
        if (!g.transA && !g.transB) launch_tiles<float, false, false>(p, small, st);
        else if (g.transA && !g.transB) launch_tiles<float, true, false>(p, small, st);
        else if (!g.transA && g.transB) launch_tiles<float, false, true>(p, small, st);
        else launch_tiles<float, true, true>(p, small, st);
    }
    return after_launch(ctx);
}

}  // namespace gelo
