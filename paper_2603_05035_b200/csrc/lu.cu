// Blocked LU with partial pivoting and the explicit inverse of the non-orthogonal
// mixing matrix (paper Mitigation 1: "The TEE must compute A^-1 per batch").
//
//   P A = L U by right-looking panels of kPanel columns:
//       panel kernel (one CTA: lane = panel column, warps stripe rows, pivot = first
//       row of largest magnitude) -> row interchanges on the rest of the matrix ->
//       U12 = L11^-1 A12 -> A22 -= L21 U12 (GEMM)
//   A^-1 = U^-1 L^-1 P by two blocked triangular solves on the permuted identity,
//   each block step a small substitution kernel plus one GEMM update.
#include "common.cuh"

namespace gelo {

namespace {

constexpr int NB = kPanel;
constexpr int kPanelThreads = 1024;
constexpr int kPanelWarps = kPanelThreads / 32;

__global__ void __launch_bounds__(kPanelThreads)
lu_panel_kernel(float* __restrict__ M, int ld, int m, int j0, int jb, int* __restrict__ ipiv,
                int* __restrict__ status)
{
    __shared__ float best_v[kPanelWarps];
    __shared__ int best_r[kPanelWarps];
    __shared__ float rowj[NB];

    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    const bool col_ok = lane < jb;
    const unsigned full = 0xffffffffu;

    for (int c = 0; c < jb; ++c) {
        const int j = j0 + c;
        // ---- pivot search over rows j..m-1 of column j ---------------------------------
        float bv = -1.0f;
        int br = j;
        for (int r0 = j + warp * 32; r0 < m; r0 += kPanelWarps * 32) {
            const int r = r0 + lane;
            const float a = (r < m) ? fabsf(M[(size_t)r * ld + j]) : -1.0f;
            if (a > bv) { bv = a; br = r; }       // rows increase per lane: keeps the first maximum
        }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) {
            const float ov = __shfl_xor_sync(full, bv, off);
            const int orow = __shfl_xor_sync(full, br, off);
            if (ov > bv || (ov == bv && orow < br)) { bv = ov; br = orow; }
        }
        if (lane == 0) { best_v[warp] = bv; best_r[warp] = br; }
        __syncthreads();
        if (warp == 0) {
            float v = best_v[lane];
            int r = best_r[lane];
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) {
                const float ov = __shfl_xor_sync(full, v, off);
                const int orow = __shfl_xor_sync(full, r, off);
                if (ov > v || (ov == v && orow < r)) { v = ov; r = orow; }
            }
            // swap rows j and r inside the panel, publish the pivot row
            float top = col_ok ? M[(size_t)j * ld + j0 + lane] : 0.0f;
            if (r != j && col_ok) {
                const float low = M[(size_t)r * ld + j0 + lane];
                M[(size_t)r * ld + j0 + lane] = top;
                M[(size_t)j * ld + j0 + lane] = low;
                top = low;
            }
            rowj[lane] = top;
            if (lane == 0) {
                ipiv[j] = r;
                if (!(v > 0.0f)) atomicCAS(status, 0, (int)GELO_ERR_COND);   // exactly singular
            }
        }
        __syncthreads();
        // ---- eliminate below the pivot ----------------------------------------------------
        const float pivot = rowj[c];
        const float inv = (pivot != 0.0f) ? 1.0f / pivot : 0.0f;
        const float rj = rowj[lane];
        for (int r = j + 1 + warp; r < m; r += kPanelWarps) {
            float y = col_ok ? M[(size_t)r * ld + j0 + lane] : 0.0f;
            const float l = __shfl_sync(full, y, c) * inv;
            if (col_ok) {
                if (lane > c) M[(size_t)r * ld + j0 + lane] = fmaf(-l, rj, y);
                else if (lane == c) M[(size_t)r * ld + j0 + lane] = l;
            }
        }
        __syncthreads();
    }
}

// Applies the panel's interchanges (rows j0+c <-> ipiv[j0+c], c = 0..jb-1, in order) to
// columns [c_lo, c_hi) of X, skipping columns [skip_lo, skip_hi).
__global__ void swap_rows_kernel(float* __restrict__ X, int ld, int j0, int jb, const int* __restrict__ ipiv,
                                 int c_lo, int c_hi, int skip_lo, int skip_hi)
{
    const int col = c_lo + blockIdx.x * blockDim.x + threadIdx.x;
    if (col >= c_hi || (col >= skip_lo && col < skip_hi)) return;
    for (int c = 0; c < jb; ++c) {
        const int a = j0 + c, b = ipiv[a];
        if (a != b) {
            const float t = X[(size_t)a * ld + col];
            X[(size_t)a * ld + col] = X[(size_t)b * ld + col];
            X[(size_t)b * ld + col] = t;
        }
    }
}

// X[i0:i0+ib, c_lo:c_hi) <- L_ii^-1 X (unit lower, forward) or U_ii^-1 X (upper, backward);
// the ib x ib triangle sits at M[i0.., i0..].  One thread per column of X.
template <bool UPPER>
__global__ void __launch_bounds__(256)
tri_solve_block_kernel(const float* M, int ldm, float* X, int ldx,
                       int i0, int ib, int c_lo, int c_hi)
{
    __shared__ float tri[NB][NB + 1];
    for (int idx = threadIdx.x; idx < NB * NB; idx += blockDim.x) {
        const int r = idx / NB, c = idx % NB;
        tri[r][c] = (r < ib && c < ib) ? M[(size_t)(i0 + r) * ldm + i0 + c] : 0.0f;
    }
    __syncthreads();
    const int col = c_lo + blockIdx.x * blockDim.x + threadIdx.x;
    if (col >= c_hi) return;
    float x[NB];
#pragma unroll
    for (int i = 0; i < NB; ++i) x[i] = (i < ib) ? X[(size_t)(i0 + i) * ldx + col] : 0.0f;
    if (!UPPER) {
#pragma unroll
        for (int i = 1; i < NB; ++i) {
            float s = x[i];
#pragma unroll
            for (int t = 0; t < i; ++t) s = fmaf(-tri[i][t], x[t], s);
            x[i] = s;
        }
    } else {
#pragma unroll
        for (int i = NB - 1; i >= 0; --i) {
            if (i < ib) {
                float s = x[i];
#pragma unroll
                for (int t = i + 1; t < NB; ++t) s = fmaf(-tri[i][t], x[t], s);
                x[i] = s / tri[i][i];
            }
        }
    }
#pragma unroll
    for (int i = 0; i < NB; ++i)
        if (i < ib) X[(size_t)(i0 + i) * ldx + col] = x[i];
}

// perm = the row order produced by the interchanges; X = P (X[i, perm[i]] = 1).
__global__ void build_perm_kernel(const int* __restrict__ ipiv, int* __restrict__ perm, int m)
{
    extern __shared__ int sp[];
    for (int i = threadIdx.x; i < m; i += blockDim.x) sp[i] = i;
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int j = 0; j < m; ++j) {
            const int b = ipiv[j];
            if (b != j) { const int t = sp[j]; sp[j] = sp[b]; sp[b] = t; }
        }
    }
    __syncthreads();
    for (int i = threadIdx.x; i < m; i += blockDim.x) perm[i] = sp[i];
}

__global__ void permuted_identity_kernel(float* __restrict__ X, int ld, int m, const int* __restrict__ perm)
{
    const size_t total = (size_t)m * ld;
    for (size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x; idx < total;
         idx += (size_t)gridDim.x * blockDim.x) {
        const int r = (int)(idx / ld), c = (int)(idx % ld);
        X[idx] = (c == perm[r]) ? 1.0f : 0.0f;
    }
}

}  // namespace

LuScratch carve_lu(Arena& a, int m, int ld)
{
    LuScratch s;
    s.M = static_cast<float*>(a.take((size_t)m * ld * sizeof(float)));
    s.ipiv = static_cast<int*>(a.take((size_t)m * sizeof(int)));
    s.perm = static_cast<int*>(a.take((size_t)m * sizeof(int)));
    return s;
}

int run_lu_inverse(gelo_ctx* ctx, int m, const float* A, int ld, float* X, const LuScratch& s, cudaStream_t st)
{
    if ((size_t)m * sizeof(int) > 200 * 1024) return GELO_ERR_UNSUPPORTED;
    float* M = s.M;
    GELO_CUDA_OK(cudaMemcpyAsync(M, A, (size_t)m * ld * sizeof(float), cudaMemcpyDeviceToDevice, st));
    const int npanels = ceil_div(m, NB);
    for (int pnl = 0; pnl < npanels; ++pnl) {
        const int j0 = pnl * NB, jb = (m - j0 < NB) ? (m - j0) : NB;
        lu_panel_kernel<<<1, kPanelThreads, 0, st>>>(M, ld, m, j0, jb, s.ipiv, ctx->status_dev);
        GELO_TRY(after_launch(ctx));
        if (m > jb) {
            swap_rows_kernel<<<ceil_div(m, 256), 256, 0, st>>>(M, ld, j0, jb, s.ipiv, 0, m, j0, j0 + jb);
            GELO_TRY(after_launch(ctx));
        }
        const int nc = m - j0 - jb;
        if (nc <= 0) continue;
        tri_solve_block_kernel<false><<<ceil_div(nc, 256), 256, 0, st>>>(M, ld, M, ld, j0, jb, j0 + jb, m);
        GELO_TRY(after_launch(ctx));
        GemmArgs g;   // A22 -= L21 U12
        g.M = nc; g.N = nc; g.K = jb;
        g.A = M + (size_t)(j0 + jb) * ld + j0; g.lda = ld;
        g.B = M + (size_t)j0 * ld + j0 + jb; g.ldb = ld;
        g.C[0] = M + (size_t)(j0 + jb) * ld + j0 + jb; g.ldc = ld;
        g.alpha = -1.0f; g.beta = 1.0f;
        GELO_TRY(launch_gemm_simt(ctx, g, st));
    }
    // ---- X = P, then L Y = P, then U X = Y ----
    const size_t perm_smem = (size_t)m * sizeof(int);
    if (perm_smem > 48 * 1024)
        GELO_CUDA_OK(cudaFuncSetAttribute(build_perm_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)perm_smem));
    build_perm_kernel<<<1, 256, perm_smem, st>>>(s.ipiv, s.perm, m);
    GELO_TRY(after_launch(ctx));
    permuted_identity_kernel<<<4 * ctx->sm_count, 256, 0, st>>>(X, ld, m, s.perm);
    GELO_TRY(after_launch(ctx));
    for (int pnl = 0; pnl < npanels; ++pnl) {
        const int i0 = pnl * NB, ib = (m - i0 < NB) ? (m - i0) : NB;
        tri_solve_block_kernel<false><<<ceil_div(m, 256), 256, 0, st>>>(M, ld, X, ld, i0, ib, 0, m);
        GELO_TRY(after_launch(ctx));
        const int nr = m - i0 - ib;
        if (nr <= 0) continue;
        GemmArgs g;   // X[i0+ib:, :] -= L[i0+ib:, i0:i0+ib] X[i0:i0+ib, :]
        g.M = nr; g.N = m; g.K = ib;
        g.A = M + (size_t)(i0 + ib) * ld + i0; g.lda = ld;
        g.B = X + (size_t)i0 * ld; g.ldb = ld;
        g.C[0] = X + (size_t)(i0 + ib) * ld; g.ldc = ld;
        g.alpha = -1.0f; g.beta = 1.0f;
        GELO_TRY(launch_gemm_simt(ctx, g, st));
    }
    for (int pnl = npanels - 1; pnl >= 0; --pnl) {
        const int i0 = pnl * NB, ib = (m - i0 < NB) ? (m - i0) : NB;
        tri_solve_block_kernel<true><<<ceil_div(m, 256), 256, 0, st>>>(M, ld, X, ld, i0, ib, 0, m);
        GELO_TRY(after_launch(ctx));
        if (i0 <= 0) continue;
        GemmArgs g;   // X[0:i0, :] -= U[0:i0, i0:i0+ib] X[i0:i0+ib, :]
        g.M = i0; g.N = m; g.K = ib;
        g.A = M + i0; g.lda = ld;
        g.B = X + (size_t)i0 * ld; g.ldb = ld;
        g.C[0] = X; g.ldc = ld;
        g.alpha = -1.0f; g.beta = 1.0f;
        GELO_TRY(launch_gemm_simt(ctx, g, st));
    }
    return GELO_OK;
}

}  // namespace gelo
