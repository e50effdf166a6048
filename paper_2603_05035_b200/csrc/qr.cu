// Blocked Householder QR (compact WY) that turns an m x m Gaussian matrix into the
// orthogonal mixing matrix of the offload: A = Q diag(sign R_jj), A^-1 = A^T
// (paper Section 3.2 step 1.2; "If A is orthogonal, A^-1 = A^T").
//
//   for each panel of kPanel columns:
//       panel kernel   : Householder vectors V (unit diagonal), tau, and the
//                        triangular factor T with  H_1 ... H_b = I - V T V^T
//       trailing update: C <- (I - V T^T V^T) C   as three GEMMs
//   Q is then accumulated backwards, panel by panel, from the identity:
//       Q[j0:, j0:] <- (I - V T V^T) Q[j0:, j0:]
//
// The panel kernel is one CTA: lane = panel column, warps stripe over rows, so each
// row of the panel is one coalesced 128-byte access; column norms and the products
// v^T C of all remaining columns come from ONE block-wide reduction per column
// (warp partial sums in registers, cross-warp sums in shared memory).
#include <cooperative_groups.h>

#include "common.cuh"

namespace gelo {

namespace {

constexpr int NB = kPanel;          // 32: one lane per panel column
constexpr int kPanelThreads = 1024;
constexpr int kPanelWarps = kPanelThreads / 32;

// R: m x m (stride ld), panel = columns j0 .. j0+jb-1, rows j0 .. m-1 (in place).
// V: m x ld; this panel's reflectors go to columns j0 .. j0+jb-1 (rows < j0 untouched,
//    rows j0.. : zeros above the diagonal, 1 on it, v below).
// T: NB x NB, upper triangular, zero elsewhere.
__global__ void __launch_bounds__(kPanelThreads)
qr_panel_kernel(float* __restrict__ R, int ld, int m, int j0, int jb,
                float* __restrict__ V, float* __restrict__ T)
{
    __shared__ float red[kPanelWarps][NB + 1];
    __shared__ float dsum[NB];
    __shared__ float rowj[NB];
    __shared__ float tau_s[NB];
    __shared__ float gram[NB][NB + 1];
    __shared__ float t_s[NB][NB + 1];

    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    const bool col_ok = lane < jb;
    const unsigned full = 0xffffffffu;

    for (int c = 0; c < jb; ++c) {
        const int j = j0 + c;
        // ---- d[c'] = sum_{r > j} R[r, j] * R[r, j0 + c'] ------------------------------
        float acc = 0.0f;
        for (int r = j + 1 + warp; r < m; r += kPanelWarps) {
            const float y = col_ok ? R[(size_t)r * ld + j0 + lane] : 0.0f;
            const float x = __shfl_sync(full, y, c);
            acc = fmaf(x, y, acc);
        }
        red[warp][lane] = acc;
        __syncthreads();
        if (warp == 0) {
            float s = 0.0f;
#pragma unroll 8
            for (int w = 0; w < kPanelWarps; ++w) s += red[w][lane];
            dsum[lane] = s;
            rowj[lane] = col_ok ? R[(size_t)j * ld + j0 + lane] : 0.0f;
        }
        __syncthreads();
        // ---- reflector scalars (every thread, same values) --------------------------------
        const float alpha = rowj[c];
        const float sigma = dsum[c];
        float beta = alpha, tau = 0.0f, scale = 0.0f;
        if (sigma > 0.0f) {
            beta = -copysignf(sqrtf(fmaf(alpha, alpha, sigma)), alpha);
            tau = (beta - alpha) / beta;
            scale = 1.0f / (alpha - beta);
        }
        // w[c'] = v^T R[j:, c'] = R[j, c'] + scale * d[c']   (v = [1; scale * x])
        const float wv = (lane > c && col_ok) ? fmaf(scale, dsum[lane], rowj[lane]) : 0.0f;
        const float tw = tau * wv;
        // ---- apply H_c to the rest of the panel and store v ---------------------------------
        if (warp == 0) {
            // row j itself
            if (col_ok) {
                float y = rowj[lane];
                if (lane > c) y -= tw;
                else if (lane == c) y = beta;
                R[(size_t)j * ld + j0 + lane] = y;
                V[(size_t)j * ld + j0 + lane] = (lane == c) ? 1.0f : ((lane > c) ? 0.0f : V[(size_t)j * ld + j0 + lane]);
            }
            if (lane == 0) tau_s[c] = tau;
        }
        for (int r = j + 1 + warp; r < m; r += kPanelWarps) {
            float y = col_ok ? R[(size_t)r * ld + j0 + lane] : 0.0f;
            const float x = __shfl_sync(full, y, c);
            const float v = x * scale;
            if (col_ok) {
                if (lane > c) {
                    y = fmaf(-tw, v, y);
                    R[(size_t)r * ld + j0 + lane] = y;
                } else if (lane == c) {
                    R[(size_t)r * ld + j0 + lane] = 0.0f;     // below-diagonal part of R
                    V[(size_t)r * ld + j0 + lane] = v;
                }
            }
        }
        __syncthreads();
    }

    // ---- zero V above the diagonal of this panel (rows j0..j0+jb-1 were written column by
    //      column; entries with row < column inside the panel block must be zero) ----------
    for (int idx = threadIdx.x; idx < jb * NB; idx += kPanelThreads) {
        const int r = idx / NB, cc = idx % NB;
        if (cc < jb && r < cc) V[(size_t)(j0 + r) * ld + j0 + cc] = 0.0f;
    }
    __syncthreads();

    // ---- Gram matrix of the reflectors: gram[a][b] = sum_r V[r, a] V[r, b] ----------------
    for (int idx = threadIdx.x; idx < NB * (NB + 1); idx += kPanelThreads) (&gram[0][0])[idx] = 0.0f;
    __syncthreads();
    {
        float g[NB];
#pragma unroll
        for (int a = 0; a < NB; ++a) g[a] = 0.0f;
        for (int r = j0 + warp; r < m; r += kPanelWarps) {
            const float y = col_ok ? V[(size_t)r * ld + j0 + lane] : 0.0f;
#pragma unroll
            for (int a = 0; a < NB; ++a) g[a] = fmaf(__shfl_sync(full, y, a), y, g[a]);
        }
        // fixed summation order (warp 0, 1, ...) keeps the factor bit-reproducible
        for (int w = 0; w < kPanelWarps; ++w) {
            if (warp == w) {
#pragma unroll
                for (int a = 0; a < NB; ++a) gram[a][lane] += g[a];
            }
            __syncthreads();
        }
    }

    // ---- T (forward, columnwise): T[c][c] = tau_c, T[0:c, c] = -tau_c T[0:c, 0:c] gram[0:c, c]
    if (warp == 0) {
        for (int a = 0; a < NB; ++a) t_s[a][lane] = 0.0f;
        __syncwarp();
        for (int c = 0; c < jb; ++c) {
            const float tc = tau_s[c];
            float s = 0.0f;
            if (lane < c) {
                for (int b = lane; b < c; ++b) s = fmaf(t_s[lane][b], gram[b][c], s);
            }
            __syncwarp();
            if (lane < c) t_s[lane][c] = -tc * s;
            else if (lane == c) t_s[c][c] = tc;
            __syncwarp();
        }
        for (int a = 0; a < NB; ++a) T[a * NB + lane] = t_s[a][lane];
    }
}

// ---- register-resident panel on a thread-block cluster -----------------------------------
//
// The same Householder panel, but the whole panel lives in registers spread over a cluster of
// CS CTAs (CS * 32 warps; global warp g holds rows j0 + g, j0 + g + CS*32, ...; lane = panel
// column).  Per column there is ONE reduction: warp partial sums -> shared memory -> one vector
// per CTA, which every CTA stores into every other CTA's shared memory (distributed shared
// memory) followed by one cluster barrier.  The lanes that are idle in that reduction (columns
// already factorised) use it to accumulate V^T v for the triangular factor T, so no separate
// Gram pass is needed.  All sums run in a fixed order: results are bit-reproducible.
constexpr int kClusterMax = 8;
constexpr int kRowsPerThread = 17;                         // 8 CTAs * 32 warps * 17 rows >= 4352
constexpr int kClusterPanelMaxRows = kClusterMax * kPanelWarps * kRowsPerThread;

__global__ void __launch_bounds__(kPanelThreads, 1)
qr_panel_cluster_kernel(float* __restrict__ R, int ld, int m, int j0, int jb,
                        float* __restrict__ V, float* __restrict__ T)
{
    namespace cg = cooperative_groups;
    cg::cluster_group cluster = cg::this_cluster();
    const int CS = (int)cluster.num_blocks();
    const int rank = (int)cluster.block_rank();

    __shared__ float red[kPanelWarps][NB + 1];
    __shared__ float slot[2][kClusterMax][NB];
    __shared__ float rowbuf[2][NB];
    __shared__ float gram[NB][NB + 1];
    __shared__ float tau_s[NB];
    __shared__ float t_s[NB][NB + 1];

    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    const int gw = rank * kPanelWarps + warp;
    const int stride = CS * kPanelWarps;
    const bool col_ok = lane < jb;
    const unsigned full = 0xffffffffu;

    float x[kRowsPerThread];
#pragma unroll
    for (int i = 0; i < kRowsPerThread; ++i) {
        const int row = j0 + i * stride + gw;
        x[i] = (row < m && col_ok) ? R[(size_t)row * ld + j0 + lane] : 0.0f;
    }
    for (int idx = threadIdx.x; idx < NB * (NB + 1); idx += kPanelThreads) (&gram[0][0])[idx] = 0.0f;
    if (CS > 1) cluster.sync(); else __syncthreads();     // every CTA of the cluster is running before remote stores

    for (int c = 0; c <= jb; ++c) {
        const int j = j0 + c;
        const int par = c & 1;
        const int csrc = c & 31, psrc = (c - 1) & 31;
        // lanes >= c: x_c^T x_lane over rows > j;   lanes < c-1: v_{c-1}^T v_lane over rows >= j-1
        float acc = 0.0f;
#pragma unroll
        for (int i = 0; i < kRowsPerThread; ++i) {
            const int row = j0 + i * stride + gw;
            const float xc = __shfl_sync(full, x[i], csrc);
            const float xp = __shfl_sync(full, x[i], psrc);
            if (lane >= c) {
                if (row > j) acc = fmaf(xc, x[i], acc);
            } else if (lane < c - 1) {
                if (row == j - 1) acc += x[i];
                else if (row > j - 1) acc = fmaf(xp, x[i], acc);
            }
        }
        red[warp][lane] = acc;
        __syncthreads();
        if (warp == 0) {
            float s = 0.0f;
#pragma unroll 8
            for (int w = 0; w < kPanelWarps; ++w) s += red[w][lane];
            for (int r = 0; r < CS; ++r) cluster.map_shared_rank(&slot[par][rank][lane], r)[0] = s;
        }
        if (c < jb && rank == 0 && warp == c) {            // the warp that holds row j (its slot 0)
            for (int r = 0; r < CS; ++r) cluster.map_shared_rank(&rowbuf[par][lane], r)[0] = x[0];
        }
        if (CS > 1) cluster.sync(); else __syncthreads();

        float d_own = 0.0f, d_c = 0.0f;
        for (int r = 0; r < CS; ++r) { d_own += slot[par][r][lane]; d_c += slot[par][r][csrc]; }
        if (c > 0 && warp == 0 && lane < c - 1) gram[lane][c - 1] = d_own;
        if (c == jb) break;

        const float alpha = rowbuf[par][c];
        const float rj = rowbuf[par][lane];
        const float sigma = d_c;
        float beta = alpha, tau = 0.0f, scale = 0.0f;
        if (sigma > 0.0f) {
            beta = -copysignf(sqrtf(fmaf(alpha, alpha, sigma)), alpha);
            tau = (beta - alpha) / beta;
            scale = 1.0f / (alpha - beta);
        }
        const float wv = (lane > c && col_ok) ? fmaf(scale, d_own, rj) : 0.0f;
        const float tw = tau * wv;
        if (threadIdx.x == 0) tau_s[c] = tau;
#pragma unroll
        for (int i = 0; i < kRowsPerThread; ++i) {
            const int row = j0 + i * stride + gw;
            const float v = __shfl_sync(full, x[i], c) * scale;
            if (row == j) {
                if (lane > c) x[i] -= tw;
                else if (lane == c) x[i] = beta;
            } else if (row > j) {
                if (lane > c) x[i] = fmaf(-tw, v, x[i]);
                else if (lane == c) x[i] = v;
            }
        }
    }

    // ---- write back: R above / on the diagonal, reflectors below it ----
#pragma unroll
    for (int i = 0; i < kRowsPerThread; ++i) {
        const int row = j0 + i * stride + gw;
        if (row < m && col_ok) {
            const int diag = j0 + lane;
            R[(size_t)row * ld + j0 + lane] = (row <= diag) ? x[i] : 0.0f;
            V[(size_t)row * ld + j0 + lane] = (row > diag) ? x[i] : ((row == diag) ? 1.0f : 0.0f);
        }
    }
    // ---- T on CTA 0, warp 0 (it wrote gram and tau_s itself) ----
    if (rank == 0 && warp == 0) {
        for (int a = 0; a < NB; ++a) t_s[a][lane] = 0.0f;
        __syncwarp();
        for (int c = 0; c < jb; ++c) {
            const float tc = tau_s[c];
            float s = 0.0f;
            if (lane < c) {
                for (int b = lane; b < c; ++b) s = fmaf(t_s[lane][b], gram[b][c], s);
            }
            __syncwarp();
            if (lane < c) t_s[lane][c] = -tc * s;
            else if (lane == c) t_s[c][c] = tc;
            __syncwarp();
        }
        for (int a = 0; a < NB; ++a) T[a * NB + lane] = t_s[a][lane];
    }
}

// Launches the panel on the smallest cluster whose registers hold the rows.
int launch_qr_panel(gelo_ctx* ctx, float* R, int ld, int m, int j0, int jb, float* V, float* T, cudaStream_t st)
{
    const int rows = m - j0;
    if (rows > kClusterPanelMaxRows) {
        qr_panel_kernel<<<1, kPanelThreads, 0, st>>>(R, ld, m, j0, jb, V, T);
        return after_launch(ctx);
    }
    int cs = 1;
    while (cs < kClusterMax && cs * kPanelWarps * kRowsPerThread < rows) cs *= 2;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(cs, 1, 1);
    cfg.blockDim = dim3(kPanelThreads, 1, 1);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = cs; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&cfg, qr_panel_cluster_kernel, R, ld, m, j0, jb, V, T) != cudaSuccess) return GELO_ERR_CUDA;
    return after_launch(ctx);
}

__global__ void set_identity_kernel(float* __restrict__ Q, int ld, int m)
{
    const size_t total = (size_t)m * ld;
    for (size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x; idx < total;
         idx += (size_t)gridDim.x * blockDim.x) {
        const int r = (int)(idx / ld), c = (int)(idx % ld);
        Q[idx] = (r == c) ? 1.0f : 0.0f;
    }
}

}  // namespace

size_t qr_scratch_bytes(int m, int ld)
{
    Arena a; a.cap = ~size_t(0) >> 1;
    carve_qr(a, m, ld);
    return a.off + 256;
}

QrScratch carve_qr(Arena& a, int m, int ld)
{
    QrScratch s;
    s.V = static_cast<float*>(a.take((size_t)m * ld * sizeof(float)));
    s.T = static_cast<float*>(a.take((size_t)ceil_div(m, NB) * NB * NB * sizeof(float)));
    s.W1 = static_cast<float*>(a.take((size_t)NB * ld * sizeof(float)));
    s.W2 = static_cast<float*>(a.take((size_t)NB * ld * sizeof(float)));
    return s;
}

int run_householder_qr(gelo_ctx* ctx, int m, float* R, int ld, float* Q, const QrScratch& s, cudaStream_t st)
{
    const int npanels = ceil_div(m, NB);
    // ---- factorisation ----
    for (int pnl = 0; pnl < npanels; ++pnl) {
        const int j0 = pnl * NB, jb = (m - j0 < NB) ? (m - j0) : NB;
        float* Tp = s.T + (size_t)pnl * NB * NB;
        GELO_TRY(launch_qr_panel(ctx, R, ld, m, j0, jb, s.V, Tp, st));
        const int nc = m - j0 - jb, nr = m - j0;
        if (nc <= 0) continue;
        float* C = R + (size_t)j0 * ld + j0 + jb;
        const float* Vp = s.V + (size_t)j0 * ld + j0;
        GemmArgs g1;   // W1 (jb x nc) = V^T C
        g1.M = jb; g1.N = nc; g1.K = nr; g1.A = Vp; g1.lda = ld; g1.transA = true;
        g1.B = C; g1.ldb = ld; g1.C[0] = s.W1; g1.ldc = ld;
        GELO_TRY(launch_gemm_simt(ctx, g1, st));
        GemmArgs g2;   // W2 = T^T W1
        g2.M = jb; g2.N = nc; g2.K = jb; g2.A = Tp; g2.lda = NB; g2.transA = true;
        g2.B = s.W1; g2.ldb = ld; g2.C[0] = s.W2; g2.ldc = ld;
        GELO_TRY(launch_gemm_simt(ctx, g2, st));
        GemmArgs g3;   // C -= V W2
        g3.M = nr; g3.N = nc; g3.K = jb; g3.A = Vp; g3.lda = ld;
        g3.B = s.W2; g3.ldb = ld; g3.C[0] = C; g3.ldc = ld; g3.alpha = -1.0f; g3.beta = 1.0f;
        GELO_TRY(launch_gemm_simt(ctx, g3, st));
    }
    // ---- accumulate Q backwards from the identity ----
    set_identity_kernel<<<4 * ctx->sm_count, 256, 0, st>>>(Q, ld, m);
    GELO_TRY(after_launch(ctx));
    for (int pnl = npanels - 1; pnl >= 0; --pnl) {
        const int j0 = pnl * NB, jb = (m - j0 < NB) ? (m - j0) : NB;
        const int nr = m - j0;
        const float* Tp = s.T + (size_t)pnl * NB * NB;
        const float* Vp = s.V + (size_t)j0 * ld + j0;
        float* C = Q + (size_t)j0 * ld + j0;
        GemmArgs g1;   // W1 (jb x nr) = V^T Q[j0:, j0:]
        g1.M = jb; g1.N = nr; g1.K = nr; g1.A = Vp; g1.lda = ld; g1.transA = true;
        g1.B = C; g1.ldb = ld; g1.C[0] = s.W1; g1.ldc = ld;
        GELO_TRY(launch_gemm_simt(ctx, g1, st));
        GemmArgs g2;   // W2 = T W1
        g2.M = jb; g2.N = nr; g2.K = jb; g2.A = Tp; g2.lda = NB;
        g2.B = s.W1; g2.ldb = ld; g2.C[0] = s.W2; g2.ldc = ld;
        GELO_TRY(launch_gemm_simt(ctx, g2, st));
        GemmArgs g3;   // Q[j0:, j0:] -= V W2
        g3.M = nr; g3.N = nr; g3.K = jb; g3.A = Vp; g3.lda = ld;
        g3.B = s.W2; g3.ldb = ld; g3.C[0] = C; g3.ldc = ld; g3.alpha = -1.0f; g3.beta = 1.0f;
        GELO_TRY(launch_gemm_simt(ctx, g3, st));
    }
    return GELO_OK;
}

}  // namespace gelo
