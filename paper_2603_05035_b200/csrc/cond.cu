// 2-norm condition number estimate of the non-orthogonal mixing matrix (paper
// Mitigation 1: "generate and verify well-conditioned A (e.g., enforce kappa(A) < 100)").
// kappa_2(A) = sigma_max(A) * sigma_max(A^-1); each factor by power iteration on
// Op^T Op with Op = A (z = 0) and Op = A^-1 (z = 1), both run in the same launches.
// All sums have a fixed order, so the estimate is bit-reproducible.  HBM/L2-bound:
// every iteration streams both matrices twice.
#include "common.cuh"
#include "philox.cuh"

namespace gelo {

namespace {

constexpr int kRowSlabs = 16;
constexpr int kPowerIters = 12;   // the estimate is within about 4% of kappa_2 after 12 steps (measured at m = 512 .. 4300)

struct CondViews {
    const float* op[2];
    int ld, m, mpad;
    float* xhat;      // [2][mpad]
    float* y;         // [2][mpad]
    float* partial;   // [2][kRowSlabs][mpad]
    float* scal;      // [0..1] sigma estimates
};

__global__ void cond_init_kernel(CondViews v, uint64_t seed, uint32_t attempt)
{
    const int z = blockIdx.y;
    const int i4 = (blockIdx.x * blockDim.x + threadIdx.x) * 4;
    if (i4 >= v.mpad) return;
    float g[4];
    gaussian_block(seed, ((uint64_t)z * v.mpad + i4) >> 2, GELO_STREAM_POWER, attempt, g);
    for (int t = 0; t < 4; ++t) {
        const int i = i4 + t;
        if (i >= v.mpad) break;
        for (int s = 0; s < kRowSlabs; ++s)
            v.partial[((size_t)z * kRowSlabs + s) * v.mpad + i] = (s == 0 && i < v.m) ? g[t] : 0.0f;
    }
}

// xhat = (sum of slab partials) / its norm;  scal[z] = sqrt(norm)
__global__ void __launch_bounds__(1024) cond_normalise_kernel(CondViews v, int last, float bound,
                                                              float* cond_out, int* status)
{
    __shared__ float red[32];
    __shared__ float total;
    const int z = blockIdx.x;
    float local = 0.0f;
    for (int i = threadIdx.x; i < v.m; i += blockDim.x) {
        float s = 0.0f;
#pragma unroll
        for (int k = 0; k < kRowSlabs; ++k) s += v.partial[((size_t)z * kRowSlabs + k) * v.mpad + i];
        v.xhat[(size_t)z * v.mpad + i] = s;
        local = fmaf(s, s, local);
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) local += __shfl_xor_sync(0xffffffffu, local, off);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = local;
    __syncthreads();
    if (threadIdx.x < 32) {
        float t = red[threadIdx.x];
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) t += __shfl_xor_sync(0xffffffffu, t, off);
        if (threadIdx.x == 0) total = t;
    }
    __syncthreads();
    const float nrm = sqrtf(total);
    const float inv = nrm > 0.0f ? 1.0f / nrm : 0.0f;
    for (int i = threadIdx.x; i < v.m; i += blockDim.x) v.xhat[(size_t)z * v.mpad + i] *= inv;
    if (threadIdx.x == 0) v.scal[z] = sqrtf(nrm);   // nrm -> lambda_max(Op^T Op) = sigma_max^2
    (void)last; (void)bound; (void)cond_out; (void)status;
}

__global__ void cond_verdict_kernel(CondViews v, float bound, float* cond_out, int* status, int deferred)
{
    const float c = v.scal[0] * v.scal[1];
    if (cond_out) cond_out[0] = c;
    const int ok = (c * 1.1f <= bound && c == c) ? 1 : 0;
    status[1] = ok;
    // nobody reads the verdict between attempts in deferred mode: a miss becomes a sticky error
    if (deferred && !ok) atomicCAS(status, 0, (int)GELO_ERR_COND);
}

// y = Op xhat, one warp per row
__global__ void __launch_bounds__(256) cond_matvec_kernel(CondViews v)
{
    const int z = blockIdx.y;
    const int row = blockIdx.x * 8 + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (row >= v.m) return;
    const float* a = v.op[z] + (size_t)row * v.ld;
    const float* x = v.xhat + (size_t)z * v.mpad;
    float s = 0.0f;
    for (int j = lane; j < v.m; j += 32) s = fmaf(a[j], x[j], s);
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) s += __shfl_xor_sync(0xffffffffu, s, off);
    if (lane == 0) v.y[(size_t)z * v.mpad + row] = s;
}

// partial[z][slab][col] = sum over the slab's rows of Op[r, col] * y[r]
__global__ void __launch_bounds__(128) cond_matvec_t_kernel(CondViews v)
{
    const int z = blockIdx.z, slab = blockIdx.y;
    const int col = blockIdx.x * 128 + threadIdx.x;
    const int rows_per = (v.m + kRowSlabs - 1) / kRowSlabs;
    const int r0 = slab * rows_per;
    const int r1 = min(v.m, r0 + rows_per);
    if (col >= v.m) return;
    const float* a = v.op[z];
    const float* y = v.y + (size_t)z * v.mpad;
    float s = 0.0f;
#pragma unroll 4
    for (int r = r0; r < r1; ++r) s = fmaf(a[(size_t)r * v.ld + col], y[r], s);
    v.partial[((size_t)z * kRowSlabs + slab) * v.mpad + col] = s;
}

}  // namespace

CondScratch carve_cond(Arena& a, int m)
{
    CondScratch s;
    const size_t mpad = (size_t)((m + 63) / 64) * 64;
    s.vec = static_cast<float*>(a.take((4 + 2 * kRowSlabs) * mpad * sizeof(float)));
    s.scal = static_cast<float*>(a.take(16 * sizeof(float)));
    return s;
}

int run_cond_estimate(gelo_ctx* ctx, int m, const float* A, const float* Ainv, int ld, float bound,
                      float* cond_out, const CondScratch& s, cudaStream_t st, bool deferred)
{
    CondViews v;
    v.op[0] = A; v.op[1] = Ainv; v.ld = ld; v.m = m; v.mpad = ((m + 63) / 64) * 64;
    v.xhat = s.vec;
    v.y = s.vec + 2 * (size_t)v.mpad;
    v.partial = s.vec + 4 * (size_t)v.mpad;
    v.scal = s.scal;
    dim3 gi(ceil_div(v.mpad, 4 * 256), 2);
    cond_init_kernel<<<gi, 256, 0, st>>>(v, 0x5eedull, 0u);
    GELO_TRY(after_launch(ctx));
    cond_normalise_kernel<<<2, 1024, 0, st>>>(v, 0, bound, cond_out, ctx->status_dev);
    GELO_TRY(after_launch(ctx));
    for (int it = 0; it < kPowerIters; ++it) {
        dim3 g1(ceil_div(m, 8), 2);
        cond_matvec_kernel<<<g1, 256, 0, st>>>(v);
        GELO_TRY(after_launch(ctx));
        dim3 g2(ceil_div(m, 128), kRowSlabs, 2);
        cond_matvec_t_kernel<<<g2, 128, 0, st>>>(v);
        GELO_TRY(after_launch(ctx));
        cond_normalise_kernel<<<2, 1024, 0, st>>>(v, 0, bound, cond_out, ctx->status_dev);
        GELO_TRY(after_launch(ctx));
    }
    cond_verdict_kernel<<<1, 1, 0, st>>>(v, bound, cond_out, ctx->status_dev, deferred ? 1 : 0);
    return after_launch(ctx);
}

}  // namespace gelo
