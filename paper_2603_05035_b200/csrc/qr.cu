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
// CS CTAs (CS * 32 warps; global warp g holds rows j0 + g + i * CS * 32, i = 0 .. RPT-1; lane =
// panel column).  Per column there is ONE reduction: warp partial sums -> shared memory -> one
// vector per CTA, which every CTA stores into every other CTA's shared memory (distributed
// shared memory) followed by one cluster barrier.  Only the first row of a warp can lie on or
// above the pivot row, so all other rows run branch-free.  The lanes that are idle in the
// reduction (columns already factorised) carry V^T v for the triangular factor T, gathered
// during the previous column's update, so no separate Gram pass is needed.  All sums run in a
// fixed order: results are bit-reproducible.
constexpr int kClusterMax = 8;
constexpr int kMaxRowsPerThread = 28;                      // rows a thread can hold in registers (64 each at 1024 threads)
constexpr int kClusterPanelMaxRows = kClusterMax * kPanelWarps * kMaxRowsPerThread;   // 7168

template <int RPT>
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
    __shared__ float coef_s[NB];
    __shared__ float tw_s[NB];
    __shared__ float scal_s[2];

    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    const int gw = rank * kPanelWarps + warp;
    const int stride = CS * kPanelWarps;
    const bool col_ok = lane < jb;
    const unsigned full = 0xffffffffu;

    float x[RPT];
#pragma unroll
    for (int i = 0; i < RPT; ++i) {
        const int row = j0 + i * stride + gw;
        x[i] = (row < m && col_ok) ? R[(size_t)row * ld + j0 + lane] : 0.0f;
    }
    for (int idx = threadIdx.x; idx < NB * (NB + 1); idx += kPanelThreads) (&gram[0][0])[idx] = 0.0f;
    if (CS > 1) cluster.sync(); else __syncthreads();     // every CTA of the cluster is running before remote stores

    float g = 0.0f;                                        // v_{c-1}^T v_lane, gathered during the previous update
    for (int c = 0; c <= jb; ++c) {
        const int par = c & 1;
        const int csrc = c & 31;
        // ---- lanes >= c: x_c^T x_lane over the rows below the pivot row j = j0 + c ----
        // (column c of a row is fetched from lane c again in the update below rather than kept: registers decide how
        // many rows a thread can hold, and with them how few SMs a panel occupies)
        float acc = 0.0f;
#pragma unroll
        for (int i = 1; i < RPT; ++i) acc = fmaf(__shfl_sync(full, x[i], csrc), x[i], acc);
        if (gw > c) acc = fmaf(__shfl_sync(full, x[0], csrc), x[0], acc);   // a warp's first row is below row j only past warp c
        red[warp][lane] = (lane >= c) ? acc : ((lane < c - 1) ? g : 0.0f);
        __syncthreads();
        {
            // warp w sums entry w over the 32 warps (butterfly: fixed order) and lane r ships it to CTA r
            float s = red[lane][warp];
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) s += __shfl_xor_sync(full, s, off);
            if (lane < CS) cluster.map_shared_rank(&slot[par][rank][warp], lane)[0] = s;
        }
        if (c < jb && rank == 0 && warp == c) {            // the warp whose first row is row j
            for (int r = 0; r < CS; ++r) cluster.map_shared_rank(&rowbuf[par][lane], r)[0] = x[0];
        }
        if (CS > 1) cluster.sync(); else __syncthreads();

        // ---- warp 0 turns the sums into this column's reflector; everybody else only reads the result ----
        if (warp == 0) {
            float d_own = 0.0f;
            for (int r = 0; r < CS; ++r) d_own += slot[par][r][lane];
            if (c > 0 && lane < c - 1) gram[lane][c - 1] = d_own;
            if (c < jb) {
                const float sigma = __shfl_sync(full, d_own, c);
                const float alpha = rowbuf[par][c];
                const float rj = rowbuf[par][lane];
                float beta = alpha, tau = 0.0f, scale = 0.0f;
                if (sigma > 0.0f) {
                    beta = -copysignf(sqrtf(fmaf(alpha, alpha, sigma)), alpha);
                    tau = (beta - alpha) / beta;
                    scale = 1.0f / (alpha - beta);
                }
                const float wv = (lane > c && col_ok) ? fmaf(scale, d_own, rj) : 0.0f;
                const float tw = tau * wv;
                tw_s[lane] = tw;
                // x <- coef * x_c + (lane == c ? 0 : x):  -tw v for later columns, v itself in column c, nothing before
                coef_s[lane] = (lane > c) ? -tw * scale : ((lane == c) ? scale : 0.0f);
                if (lane == 0) { scal_s[0] = scale; scal_s[1] = beta; tau_s[c] = tau; }
            }
        }
        if (c == jb) break;
        __syncthreads();
        const float coef = coef_s[lane];
        const float scale = scal_s[0];
        // ---- apply H_c; every lane also gathers x_c^T x_lane (only lanes < c use it: v_c^T v_lane for T) ----
        float graw = 0.0f;
#pragma unroll
        for (int i = 1; i < RPT; ++i) {
            const float xci = __shfl_sync(full, x[i], csrc);
            graw = fmaf(xci, x[i], graw);
            x[i] = fmaf(coef, xci, (lane == c) ? 0.0f : x[i]);
        }
        g = 0.0f;
        const float xc0 = __shfl_sync(full, x[0], csrc);
        if (gw > c) {
            graw = fmaf(xc0, x[0], graw);
            x[0] = fmaf(coef, xc0, (lane == c) ? 0.0f : x[0]);
        } else if (gw == c) {                               // row j itself: v_c(j) = 1
            g = x[0];
            if (lane > c) x[0] -= tw_s[lane];
            else if (lane == c) x[0] = scal_s[1];
        }
        g = fmaf(scale, graw, g);
    }

    // ---- write back: R above / on the diagonal, reflectors below it ----
#pragma unroll
    for (int i = 0; i < RPT; ++i) {
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

template <int RPT>
cudaError_t launch_cluster_panel(int cs, cudaStream_t st, float* R, int ld, int m, int j0, int jb, float* V, float* T)
{
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
    return cudaLaunchKernelEx(&cfg, qr_panel_cluster_kernel<RPT>, R, ld, m, j0, jb, V, T);
}

// Launches the panel on the cluster / rows-per-thread combination that wastes the fewest row slots.
int launch_qr_panel(gelo_ctx* ctx, float* R, int ld, int m, int j0, int jb, float* V, float* T, cudaStream_t st)
{
    const int rows = m - j0;
    if (rows > kClusterPanelMaxRows) {
        qr_panel_kernel<<<1, kPanelThreads, 0, st>>>(R, ld, m, j0, jb, V, T);
        return after_launch(ctx);
    }
    // Alone on the GPU a panel spreads over as many SMs as give every thread at least two rows (shortest column
    // step); in a batch with many sampling lanes it packs up to 28 rows per thread and occupies as few SMs as
    // possible, since every SM it holds is one that the other lanes' kernels cannot use.
    const int rows_per_thread = ctx->tc_update_ctas > 0 ? kMaxRowsPerThread : 2;
    // (a cluster may have any size up to eight: five CTAs where four are too few, not eight)
    int cs = ceil_div(rows, kPanelWarps * rows_per_thread);
    if (cs > kClusterMax) cs = kClusterMax;
    const int rpt = ceil_div(rows, cs * kPanelWarps);
    ProfScope ps(ctx, PROF_QR_PANEL, 2.0 * rows * (double)jb * jb, st);   // flops of the column dots and updates
    cudaError_t e;
    if (rpt <= 2) e = launch_cluster_panel<2>(cs, st, R, ld, m, j0, jb, V, T);
    else if (rpt <= 3) e = launch_cluster_panel<3>(cs, st, R, ld, m, j0, jb, V, T);
    else if (rpt <= 5) e = launch_cluster_panel<5>(cs, st, R, ld, m, j0, jb, V, T);
    else if (rpt <= 7) e = launch_cluster_panel<7>(cs, st, R, ld, m, j0, jb, V, T);
    else if (rpt <= 9) e = launch_cluster_panel<9>(cs, st, R, ld, m, j0, jb, V, T);
    else if (rpt <= 11) e = launch_cluster_panel<11>(cs, st, R, ld, m, j0, jb, V, T);
    else if (rpt <= 13) e = launch_cluster_panel<13>(cs, st, R, ld, m, j0, jb, V, T);
    else if (rpt <= 15) e = launch_cluster_panel<15>(cs, st, R, ld, m, j0, jb, V, T);
    else if (rpt <= 17) e = launch_cluster_panel<17>(cs, st, R, ld, m, j0, jb, V, T);
    else if (rpt <= 20) e = launch_cluster_panel<20>(cs, st, R, ld, m, j0, jb, V, T);
    else if (rpt <= 24) e = launch_cluster_panel<24>(cs, st, R, ld, m, j0, jb, V, T);
    else e = launch_cluster_panel<28>(cs, st, R, ld, m, j0, jb, V, T);
    if (e != cudaSuccess) return GELO_ERR_CUDA;
    return after_launch(ctx);
}

__global__ void set_diagonal_kernel(float* __restrict__ Q, int ld, int m)
{
    const int r = blockIdx.x * blockDim.x + threadIdx.x;
    if (r < m) Q[(size_t)r * ld + r] = 1.0f;
}

// Q = I: a memset at copy speed, then the ones.
int set_identity(gelo_ctx* ctx, float* Q, int ld, int m, cudaStream_t st)
{
    GELO_CUDA_OK(cudaMemsetAsync(Q, 0, (size_t)m * ld * sizeof(float), st));
    set_diagonal_kernel<<<ceil_div(m, 256), 256, 0, st>>>(Q, ld, m);
    return after_launch(ctx);
}


// Gram matrix of an outer block's reflectors, S = V^T V (V: nr x ob, ob <= 128), as per-slab partial sums:
// CTA s accumulates rows [s * kGramRows, ...) in 32-row chunks staged in shared memory (256 threads, 8 x 8
// outputs each) and writes its 128 x 128 partial to part[s].
constexpr int kGramRows = 256;

__global__ void __launch_bounds__(256)
gram128_kernel(const float* __restrict__ V, int ld, int nr, int ob, float* __restrict__ part)
{
    __shared__ __align__(16) float vs[32][128 + 4];
    const int tid = threadIdx.x;
    const int ty = tid >> 4, tx = tid & 15;
    const int r0 = blockIdx.x * kGramRows;
    const int r1 = min(nr, r0 + kGramRows);
    float acc[8][8];
#pragma unroll
    for (int i = 0; i < 8; ++i)
#pragma unroll
        for (int j = 0; j < 8; ++j) acc[i][j] = 0.0f;
    for (int rb = r0; rb < r1; rb += 32) {
        // 32 rows x 128 columns: thread loads 4 float4 (row = tid / 32 + 8 i, column group = tid % 32)
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int rr = (tid >> 5) + 8 * i, c4 = (tid & 31) * 4;
            const int row = rb + rr;
            float4 t = make_float4(0.f, 0.f, 0.f, 0.f);
            if (row < r1) {
                const float* p = V + (size_t)row * ld + c4;
                if (c4 + 3 < ob) t = *reinterpret_cast<const float4*>(p);
                else {
                    if (c4 + 0 < ob) t.x = p[0];
                    if (c4 + 1 < ob) t.y = p[1];
                    if (c4 + 2 < ob) t.z = p[2];
                }
            }
            *reinterpret_cast<float4*>(&vs[rr][c4]) = t;
        }
        __syncthreads();
#pragma unroll 8
        for (int k = 0; k < 32; ++k) {
            const float4 a0 = *reinterpret_cast<const float4*>(&vs[k][ty * 4]);
            const float4 a1 = *reinterpret_cast<const float4*>(&vs[k][ty * 4 + 64]);
            const float4 b0 = *reinterpret_cast<const float4*>(&vs[k][tx * 4]);
            const float4 b1 = *reinterpret_cast<const float4*>(&vs[k][tx * 4 + 64]);
            const float a[8] = {a0.x, a0.y, a0.z, a0.w, a1.x, a1.y, a1.z, a1.w};
            const float b[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
#pragma unroll
            for (int i = 0; i < 8; ++i)
#pragma unroll
                for (int j = 0; j < 8; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
        }
        __syncthreads();
    }
    float* out = part + (size_t)blockIdx.x * 128 * 128;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const int r = ty * 4 + (i >> 2) * 64 + (i & 3);
#pragma unroll
        for (int h = 0; h < 2; ++h)
            *reinterpret_cast<float4*>(out + (size_t)r * 128 + tx * 4 + h * 64) =
                make_float4(acc[i][4 * h + 0], acc[i][4 * h + 1], acc[i][4 * h + 2], acc[i][4 * h + 3]);
    }
}

// Triangular factor of an outer block from the factors of its 32-column panels:
//   (I - V1 T1 V1^T)(I - V2 T2 V2^T) = I - [V1 V2] [[T1, -T1 (V1^T V2) T2], [0, T2]] [V1 V2]^T,
// applied panel after panel.  part: `slabs` partial Gram matrices of 128 rows with row stride ldp (summed here in
// slab order); T32: the panels' factors.  One CTA, everything in shared memory.
constexpr int kMergeSmemBytes = (2 * 128 * 129 + 96 * 33 + 32 * 33) * 4;

__global__ void __launch_bounds__(1024)
t_merge_kernel(const float* __restrict__ part, int slabs, int ldp, const float* __restrict__ T32, int ob, float* __restrict__ T128)
{
    extern __shared__ float msm[];
    float (*S)[129] = reinterpret_cast<float (*)[129]>(msm);
    float (*Tm)[129] = reinterpret_cast<float (*)[129]>(msm + 128 * 129);
    float (*x_s)[33] = reinterpret_cast<float (*)[33]>(msm + 2 * 128 * 129);
    float (*tk_s)[33] = reinterpret_cast<float (*)[33]>(msm + 2 * 128 * 129 + 96 * 33);
    const int tid = threadIdx.x;
    for (int idx = tid; idx < 128 * 128; idx += 1024) {
        float acc = 0.0f;
        for (int q = 0; q < slabs; ++q) acc += part[((size_t)q * 128 + (idx >> 7)) * ldp + (idx & 127)];
        S[idx >> 7][idx & 127] = acc;
        Tm[idx >> 7][idx & 127] = 0.0f;
    }
    __syncthreads();
    const int nsub = (ob + NB - 1) / NB;
    for (int k = 0; k < nsub; ++k) {
        {
            const int a = tid >> 5, b = tid & 31;                   // 1024 threads = one 32 x 32 factor
            const float t = T32[(size_t)k * NB * NB + tid];
            tk_s[a][b] = t;
            Tm[k * NB + a][k * NB + b] = t;
        }
        __syncthreads();
        const int rows = k * NB;                                    // rows of the already merged part
        // X = S[0:rows, k*32 : k*32+32] * T_k
        for (int idx = tid; idx < rows * NB; idx += 1024) {
            const int r = idx >> 5, cc = idx & 31;
            float acc = 0.0f;
            for (int b = 0; b <= cc; ++b) acc = fmaf(S[r][k * NB + b], tk_s[b][cc], acc);
            x_s[r][cc] = acc;
        }
        __syncthreads();
        // T[0:rows, k*32 : k*32+32] = -T[0:rows, 0:rows] * X   (upper triangular left factor)
        for (int idx = tid; idx < rows * NB; idx += 1024) {
            const int r = idx >> 5, cc = idx & 31;
            float acc = 0.0f;
            for (int q = r; q < rows; ++q) acc = fmaf(Tm[r][q], x_s[q][cc], acc);
            Tm[r][k * NB + cc] = -acc;
        }
        __syncthreads();
    }
    for (int idx = tid; idx < 128 * 128; idx += 1024) T128[idx] = Tm[idx >> 7][idx & 127];
}

// ---- the whole factorisation of a small matrix (m <= 128) in one launch ---------------------------------------
//
// A decode-shaped call mixes a few dozen rows, and for such a matrix the blocked path above is some thirty dependent
// launches of a few microseconds each.  Here one CTA does everything with the matrix in registers: eight consecutive
// lanes share COLUMN c (lane h of the group holds rows h, h + 8, ...), so applying a reflector to a column is a dozen
// private FMAs plus a three-step shuffle inside the group, and the only block-wide communication is the reflector
// itself, which the owners of column j write to shared memory once per column (one barrier per column).  The
// reflectors stay in shared memory; afterwards each group builds its column of Q = H_0 ... H_(m-1) by applying them
// backwards to e_c (only H_j with j <= c touch it), with no barrier at all.
// Same conventions as the blocked path: R (upper triangle, diagonal of either sign) overwrites G, Q is unsigned.
template <int RM>
__global__ void __launch_bounds__(8 * RM, 1)
qr_small_kernel(float* __restrict__ G, int ld, int m, float* __restrict__ Q)
{
    constexpr int RPT = RM / 8;
    extern __shared__ float qs_smem[];
    float* Vs = qs_smem;                      // RM x RM: row j = reflector j over the rows
    float* tau_s = qs_smem + RM * RM;
    const int c = threadIdx.x >> 3, h = threadIdx.x & 7;
    const unsigned gmask = 0xFFu << (threadIdx.x & 24);        // the eight lanes of this column
    auto group_sum = [&](float v) {
        v += __shfl_xor_sync(gmask, v, 1);
        v += __shfl_xor_sync(gmask, v, 2);
        v += __shfl_xor_sync(gmask, v, 4);
        return v;
    };
    float x[RPT];
#pragma unroll
    for (int i = 0; i < RPT; ++i) {
        const int r = h + 8 * i;
        x[i] = (r < m && c < m) ? G[(size_t)r * ld + c] : 0.0f;
    }
    for (int j = 0; j < m; ++j) {
        if (c == j) {
            float s = 0.0f, a = 0.0f;
#pragma unroll
            for (int i = 0; i < RPT; ++i) {
                const int r = h + 8 * i;
                s = fmaf((r > j) ? x[i] : 0.0f, x[i], s);
                a += (r == j) ? x[i] : 0.0f;
            }
            const float sigma = group_sum(s), alpha = group_sum(a);
            float beta = alpha, tau = 0.0f, scale = 0.0f;
            if (sigma > 0.0f) {
                beta = -copysignf(sqrtf(fmaf(alpha, alpha, sigma)), alpha);
                tau = (beta - alpha) / beta;
                scale = 1.0f / (alpha - beta);
            }
#pragma unroll
            for (int i = 0; i < RPT; ++i) {
                const int r = h + 8 * i;
                Vs[j * RM + r] = (r < j) ? 0.0f : ((r == j) ? 1.0f : x[i] * scale);
                x[i] = (r < j) ? x[i] : ((r == j) ? beta : 0.0f);
            }
            if (h == 0) tau_s[j] = tau;
        }
        __syncthreads();
        if (c > j && c < m) {
            const float* v = Vs + j * RM + h;
            float w = 0.0f;
#pragma unroll
            for (int i = 0; i < RPT; ++i) w = fmaf(v[8 * i], x[i], w);            // v is zero above row j
            const float tw = tau_s[j] * group_sum(w);
#pragma unroll
            for (int i = 0; i < RPT; ++i) x[i] = fmaf(-tw, v[8 * i], x[i]);
        }
    }
    if (c < m) {
#pragma unroll
        for (int i = 0; i < RPT; ++i) {
            const int r = h + 8 * i;
            if (r < m) G[(size_t)r * ld + c] = x[i];
        }
    }
    // ---- column c of Q ----
    if (c < m) {
#pragma unroll
        for (int i = 0; i < RPT; ++i) x[i] = (h + 8 * i == c) ? 1.0f : 0.0f;
        for (int j = c; j >= 0; --j) {
            const float* v = Vs + j * RM + h;
            float w = 0.0f;
#pragma unroll
            for (int i = 0; i < RPT; ++i) w = fmaf(v[8 * i], x[i], w);
            const float tw = tau_s[j] * group_sum(w);
#pragma unroll
            for (int i = 0; i < RPT; ++i) x[i] = fmaf(-tw, v[8 * i], x[i]);
        }
#pragma unroll
        for (int i = 0; i < RPT; ++i) {
            const int r = h + 8 * i;
            if (r < m) Q[(size_t)r * ld + c] = x[i];
        }
    }
}

template <int RM>
int launch_qr_small_rm(gelo_ctx* ctx, int m, float* G, int ld, float* Q, cudaStream_t st)
{
    const int smem = (RM * RM + RM) * (int)sizeof(float);
    static bool attr_done[64] = {};
    if (ctx->device >= 0 && ctx->device < 64 && !attr_done[ctx->device]) {
        GELO_CUDA_OK(cudaFuncSetAttribute(qr_small_kernel<RM>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
        attr_done[ctx->device] = true;
    }
    qr_small_kernel<RM><<<1, 8 * RM, smem, st>>>(G, ld, m, Q);
    return after_launch(ctx);
}

constexpr int kSmallQrRows = 128;

int launch_qr_small(gelo_ctx* ctx, int m, float* G, int ld, float* Q, cudaStream_t st)
{
    if (m <= 32) return launch_qr_small_rm<32>(ctx, m, G, ld, Q, st);
    if (m <= 64) return launch_qr_small_rm<64>(ctx, m, G, ld, Q, st);
    if (m <= 96) return launch_qr_small_rm<96>(ctx, m, G, ld, Q, st);
    return launch_qr_small_rm<128>(ctx, m, G, ld, Q, st);
}

}  // namespace


// Takes `bytes` from the idle region if it has that much left, else from the arena.
void* take_idle(Arena& a, char** idle, size_t* idle_bytes, size_t bytes)
{
    const size_t need = (bytes + 255) & ~size_t(255);
    if (idle && idle_bytes && *idle_bytes >= need) {
        void* p = *idle;
        *idle += need;
        *idle_bytes -= need;
        return p;
    }
    return a.take(bytes);
}

QrScratch carve_qr(Arena& a, int m, int ld, char** idle, size_t* idle_bytes)
{
    QrScratch s;
    s.V = static_cast<float*>(a.take((size_t)m * ld * sizeof(float)));
    s.T = static_cast<float*>(a.take((size_t)ceil_div(m, NB) * NB * NB * sizeof(float)));
    s.Wp = static_cast<float*>(take_idle(a, idle, idle_bytes, (size_t)kMaxSlabs * NB * ld * sizeof(float)));
    s.W2 = static_cast<float*>(a.take((size_t)NB * ld * sizeof(float)));
    s.T128 = static_cast<float*>(a.take((size_t)ceil_div(m, 128) * 128 * 128 * sizeof(float)));
    return s;
}

int run_householder_qr(gelo_ctx* ctx, int m, float* R, int ld, float* Q, const QrScratch& s, cudaStream_t st)
{
    if (m <= kSmallQrRows && ctx->fuse_small) return launch_qr_small(ctx, m, R, ld, Q, st);
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
        // C <- (I - V T^T V^T) C :  W2 = T^T (V^T C), then C -= V W2
        GELO_TRY(launch_vtc(ctx, Vp, ld, jb, C, ld, nr, nc, Tp, true, s.Wp, s.W2, ld, st));
        GELO_TRY(launch_rank_update(ctx, Vp, ld, s.W2, ld, C, ld, nr, nc, jb, st));
    }
    // ---- accumulate Q backwards from the identity ----
    GELO_TRY(set_identity(ctx, Q, ld, m, st));
    for (int pnl = npanels - 1; pnl >= 0; --pnl) {
        const int j0 = pnl * NB, jb = (m - j0 < NB) ? (m - j0) : NB;
        const int nr = m - j0;
        const float* Tp = s.T + (size_t)pnl * NB * NB;
        const float* Vp = s.V + (size_t)j0 * ld + j0;
        float* C = Q + (size_t)j0 * ld + j0;
        // Q[j0:, j0:] <- (I - V T V^T) Q[j0:, j0:]
        GELO_TRY(launch_vtc(ctx, Vp, ld, jb, C, ld, nr, nr, Tp, false, s.Wp, s.W2, ld, st));
        GELO_TRY(launch_rank_update(ctx, Vp, ld, s.W2, ld, C, ld, nr, nr, jb, st));
    }
    return GELO_OK;
}

int run_householder_qr_tc(gelo_ctx* ctx, int m, float* R, int ld, float* Q, const QrScratch& s, const TcScratch& tc,
                          cudaStream_t st)
{
    // reflector entries above a panel's first row are read (as zeros) by the block-level products
    GELO_CUDA_OK(cudaMemsetAsync(s.V, 0, (size_t)m * ld * sizeof(float), st));
    GELO_CUDA_OK(cudaFuncSetAttribute(t_merge_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kMergeSmemBytes));
    const int nblocks = ceil_div(m, kOuter);

    // One outer-block transformation C <- (I - V Top V^T) C on the tensor cores, Top = T^T or T.
    auto block_apply = [&](int b0, int ob, float* C, int nc, bool transpose_t) -> int {
        const int nr = m - b0;
        const int nc8 = (nc + 7) & ~7;
        const float* Vb = s.V + (size_t)b0 * ld + b0;
        const float* Tb = s.T128 + (size_t)(b0 / kOuter) * 128 * 128;
        GELO_TRY(launch_split(ctx, C, ld, nr, nc, tc.big[0], tc.big[1], ld, false, st));
        GELO_TRY(launch_split(ctx, Vb, ld, nr, ob, tc.panA[0], tc.panA[1], kOuter, false, st));
        GELO_TRY(launch_split(ctx, Vb, ld, nr, ob, tc.panAt[0], tc.panAt[1], ld, true, st));
        GELO_TRY(launch_split(ctx, Tb, 128, ob, ob, tc.tt[0], tc.tt[1], kOuter, transpose_t, st));
        // W = V^T C: a long, thin product, so the rows are cut into slices whose partial products are summed in a
        // fixed order by the kernel that also forms the (high, low) pair
        const int n_tiles = ceil_div(nc8, 256);
        int want = ceil_div(2 * (ctx->tc_update_ctas > 0 ? ctx->tc_update_ctas : ctx->sm_count), n_tiles);   // slices fill the CTAs this launch may use
        if (want > kMaxKSplit) want = kMaxKSplit;
        int used = 0;
        const size_t plane = (size_t)kOuter * ld;
        GELO_TRY(launch_gemm_tc_split_k(ctx, ob, nc8, nr, tc.panAt[0], tc.panAt[1], ld, tc.big[0], tc.big[1], ld, tc.wf32,
                                        plane, ld, want, &used, st));
        GELO_TRY(launch_sum_split(ctx, tc.wf32, plane, used, ld, ob, nc8, tc.rowB[0], tc.rowB[1], ld, st));
        // W2 = Top W
        GELO_TRY(launch_gemm_tc_split(ctx, ob, nc8, ob, tc.tt[0], tc.tt[1], kOuter, tc.rowB[0], tc.rowB[1], ld, nullptr, 0,
                                      tc.rowB2[0], tc.rowB2[1], ld, false, st));
        // C -= V W2
        return launch_gemm_tc_split(ctx, nr, nc, ob, tc.panA[0], tc.panA[1], kOuter, tc.rowB2[0], tc.rowB2[1], ld, C, ld,
                                    nullptr, nullptr, 0, false, st);
    };

    // ---- factorisation ----
    for (int blk = 0; blk < nblocks; ++blk) {
        const int b0 = blk * kOuter;
        const int ob = (m - b0 < kOuter) ? (m - b0) : kOuter;
        const int bend = b0 + ob;
        for (int j0 = b0; j0 < bend; j0 += NB) {
            const int jb = (bend - j0 < NB) ? (bend - j0) : NB;
            float* Tp = s.T + (size_t)(j0 / NB) * NB * NB;
            GELO_TRY(launch_qr_panel(ctx, R, ld, m, j0, jb, s.V, Tp, st));
            const int ncb = bend - (j0 + jb), nr = m - j0;
            if (ncb > 0) {
                float* C = R + (size_t)j0 * ld + j0 + jb;
                const float* Vp = s.V + (size_t)j0 * ld + j0;
                GELO_TRY(launch_vtc(ctx, Vp, ld, jb, C, ld, nr, ncb, Tp, true, s.Wp, s.W2, ld, st));
                GELO_TRY(launch_rank_update(ctx, Vp, ld, s.W2, ld, C, ld, nr, ncb, jb, st));
            }
        }
        // block factor: Gram of the block's reflectors (row slabs, summed in order), then the merge of the panel factors
        const float* Vb = s.V + (size_t)b0 * ld + b0;
        const int slabs = ceil_div(m - b0, kGramRows);
        gram128_kernel<<<slabs, 256, 0, st>>>(Vb, ld, m - b0, ob, tc.gram);
        GELO_TRY(after_launch(ctx));
        float* Tb = s.T128 + (size_t)blk * 128 * 128;
        t_merge_kernel<<<1, 1024, kMergeSmemBytes, st>>>(tc.gram, slabs, 128, s.T + (size_t)(b0 / NB) * NB * NB, ob, Tb);
        GELO_TRY(after_launch(ctx));
        const int nc = m - bend;
        if (nc > 0) GELO_TRY(block_apply(b0, ob, R + (size_t)b0 * ld + bend, nc, true));
    }
    // ---- accumulate Q backwards from the identity ----
    GELO_TRY(set_identity(ctx, Q, ld, m, st));
    for (int blk = nblocks - 1; blk >= 0; --blk) {
        const int b0 = blk * kOuter;
        const int ob = (m - b0 < kOuter) ? (m - b0) : kOuter;
        GELO_TRY(block_apply(b0, ob, Q + (size_t)b0 * ld + b0, m - b0, false));
    }
    return GELO_OK;
}

// Blocked QR whose level-3 work is tf32 products read straight from the fp32 matrices.  Panels of 32 columns and
// blocks of 128 run as in run_householder_qr_tc.  Blocks are grouped into superblocks of kSuper = 512 columns:
//   * inside a superblock a finished block is applied to the superblock's remaining columns only, and its factor
//     is merged into the superblock's factor:  with S = V_i^T V_(<i),
//         T(1..i) = [[T(1..i-1), -T(1..i-1) S^T T_i], [0, T_i]];
//   * the columns right of the superblock see ONE update C <- (I - V T^T V^T) C with all 512 reflectors, and Q is
//     accumulated backwards with one such update (with T) per superblock.
// A trailing update with 512 reflectors does four times the arithmetic of one with 128 per byte of C moved, which
// is what the 128-column updates were short of (they ran at the speed of the memory system, not of the tensor cores).
int run_householder_qr_tf32(gelo_ctx* ctx, int m, float* R, int ld, float* Q, const QrScratch& s, const TcScratch& tc,
                            cudaStream_t st)
{
    GELO_CUDA_OK(cudaMemsetAsync(s.V, 0, (size_t)m * ld * sizeof(float), st));
    GELO_CUDA_OK(cudaFuncSetAttribute(t_merge_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kMergeSmemBytes));
    const float back2 = (1.0f + kTf32TruncLoss) * (1.0f + kTf32TruncLoss);
    const int width = ctx->tc_update_ctas > 0 ? ctx->tc_update_ctas : ctx->sm_count;   // CTAs one launch may use
    // the Gram slots are read in full by the merge kernel; entries that no product writes must at least be finite
    GELO_CUDA_OK(cudaMemsetAsync(tc.sx, 0, (size_t)kOuter * (kSuper + kOuter) * sizeof(float), st));

    // C (nr x nc, rows from row r0 of the matrix) <- (I - V op(T) V^T) C with V = reflector columns c0 .. c0+kv-1
    // (rows from r0 = c0), T: kv x kv with row stride ldt; planes hold `maxsplit` slices of kv x ld.
    auto apply = [&](int c0, int kv, const float* T, int ldt, float* C, int nc, bool transpose_t, int maxsplit) -> int {
        const int nr = m - c0;
        const int nc8 = (nc + 7) & ~7;
        const float* Vb = s.V + (size_t)c0 * ld + c0;
        // W = V^T C contracts over all nr rows: with few output tiles the rows are cut into slices (summed in a fixed
        // order afterwards) so that the launch still fills its CTAs; with enough tiles it is one plain product
        const int tiles = ceil_div(kv, 128) * ceil_div(nc8, 256);
        int want = (2 * tiles >= width) ? 1 : ceil_div(2 * width, tiles);
        if (want > maxsplit) want = maxsplit;
        if (want <= 1) {
            GELO_TRY(launch_gemm_tf32(ctx, kv, nc8, nr, Vb, ld, true, C, ld, false, tc.w32[0], ld, true, 1.0f, 1, 0, nullptr, st));
        } else {
            int used = 0;
            const size_t plane = (size_t)kv * ld;
            GELO_TRY(launch_gemm_tf32(ctx, kv, nc8, nr, Vb, ld, true, C, ld, false, tc.wf32, ld, false, 1.0f, want, plane, &used, st));
            GELO_TRY(launch_sum_planes(ctx, tc.wf32, plane, used, ld, kv, nc8, 1.0f, tc.w32[0], ld, st));
        }
        GELO_TRY(launch_gemm_tf32(ctx, kv, nc8, kv, T, ldt, transpose_t, tc.w32[0], ld, false, tc.w32[1], ld, true, 1.0f, 1, 0,
                                  nullptr, st));
        return launch_gemm_tf32(ctx, nr, nc, kv, Vb, ld, false, tc.w32[1], ld, true, C, ld, false, 1.0f, 1, 0, nullptr, st);
    };

    const int nsuper = ceil_div(m, kSuper);
    // ---- factorisation ----
    for (int sb = 0; sb < nsuper; ++sb) {
        const int s0 = sb * kSuper;
        const int sw = (m - s0 < kSuper) ? (m - s0) : kSuper;
        const int send = s0 + sw;
        float* Ts = tc.tsuper + (size_t)sb * kSuper * kSuper;
        GELO_CUDA_OK(cudaMemsetAsync(Ts, 0, (size_t)kSuper * kSuper * sizeof(float), st));
        for (int b0 = s0; b0 < send; b0 += kOuter) {
            const int ob = (send - b0 < kOuter) ? (send - b0) : kOuter;
            const int bend = b0 + ob;
            for (int j0 = b0; j0 < bend; j0 += NB) {
                const int jb = (bend - j0 < NB) ? (bend - j0) : NB;
                float* Tp = s.T + (size_t)(j0 / NB) * NB * NB;
                GELO_TRY(launch_qr_panel(ctx, R, ld, m, j0, jb, s.V, Tp, st));
                const int ncb = bend - (j0 + jb), nr = m - j0;
                if (ncb > 0) {
                    float* C = R + (size_t)j0 * ld + j0 + jb;
                    const float* Vp = s.V + (size_t)j0 * ld + j0;
                    GELO_TRY(launch_vtc(ctx, Vp, ld, jb, C, ld, nr, ncb, Tp, true, s.Wp, s.W2, ld, st));
                    GELO_TRY(launch_rank_update(ctx, Vp, ld, s.W2, ld, C, ld, nr, ncb, jb, st));
                }
            }
            // S = V_i^T [V_(<i) | V_i]  (ob x (r + ob)): the block's own Gram matrix and its products with the reflectors
            // already merged, in one tf32 product over the rows from b0 down (both operands reach the tensor core
            // truncated, hence the scale)
            const float* Vb = s.V + (size_t)b0 * ld + b0;
            float* Tb = s.T128 + (size_t)(b0 / kOuter) * 128 * 128;
            const int r = b0 - s0;                           // reflector columns already merged
            const int ob8 = (ob + 7) & ~7;
            const int lds = kSuper + kOuter;
            {
                // all 128 columns of the block's slot where the row has them (columns past the block are still zero):
                // the merge kernel reads the whole 128 x 128 Gram slot
                const int nr = m - b0;
                const int ns = (r + kOuter <= ld - s0) ? r + kOuter : ld - s0;
                int want = ceil_div(2 * width, ceil_div(ns, 256));
                if (want > kMaxKSplit) want = kMaxKSplit;
                int used = 0;
                const size_t plane = (size_t)kOuter * ld;
                GELO_TRY(launch_gemm_tf32(ctx, ob, ns, nr, Vb, ld, true, s.V + (size_t)b0 * ld + s0, ld, false, tc.wf32, ld, false,
                                          1.0f, want, plane, &used, st));
                GELO_TRY(launch_sum_planes(ctx, tc.wf32, plane, used, ld, ob, ns, back2, tc.sx, lds, st));
            }
            // block factor T_i from its Gram matrix and the panel factors ...
            t_merge_kernel<<<1, 1024, kMergeSmemBytes, st>>>(tc.sx + r, 1, lds, s.T + (size_t)(b0 / NB) * NB * NB, ob, Tb);
            GELO_TRY(after_launch(ctx));
            // ... into the superblock's factor
            GELO_CUDA_OK(cudaMemcpy2DAsync(Ts + (size_t)r * kSuper + r, (size_t)kSuper * sizeof(float), Tb, 128 * sizeof(float),
                                           (size_t)ob * sizeof(float), ob, cudaMemcpyDeviceToDevice, st));
            if (r > 0) {
                // X = S^T T_i  (r x ob),  then  T[0:r, r:r+ob] = -T[0:r, 0:r] X  (that part of T is still zero)
                GELO_TRY(launch_gemm_tf32(ctx, r, ob8, ob, tc.sx, lds, true, Tb, 128, false, tc.xb, kOuter, true, 1.0f, 1, 0,
                                          nullptr, st));
                GELO_TRY(launch_gemm_tf32(ctx, r, ob, r, Ts, kSuper, false, tc.xb, kOuter, true, Ts + r, kSuper, false, 1.0f, 1, 0,
                                          nullptr, st));
            }
            // the block's own reflector on the remaining columns of the superblock
            if (send > bend) GELO_TRY(apply(b0, ob, Tb, 128, R + (size_t)b0 * ld + bend, send - bend, true, kMaxKSplit));
        }
        // the merged reflector on everything right of the superblock
        if (m > send) GELO_TRY(apply(s0, sw, Ts, kSuper, R + (size_t)s0 * ld + send, m - send, true, kSuperKSplit));
    }
    // ---- accumulate Q backwards from the identity, one superblock at a time ----
    GELO_TRY(set_identity(ctx, Q, ld, m, st));
    for (int sb = nsuper - 1; sb >= 0; --sb) {
        const int s0 = sb * kSuper;
        const int sw = (m - s0 < kSuper) ? (m - s0) : kSuper;
        GELO_TRY(apply(s0, sw, tc.tsuper + (size_t)sb * kSuper * kSuper, kSuper, Q + (size_t)s0 * ld + s0, m - s0, false,
                       kSuperKSplit));
    }
    return GELO_OK;
}

// The tf32 updates leave Q orthogonal to a few 1e-3 only (the tensor core truncates unrounded operands, which
// shrinks every block reflector a little).  One Newton-Schulz step, Q <- Q - Q D with D = (Q^T Q - I) / 2, squares
// that defect.
//   * D is symmetric: one tf32 product over the tiles on and above the diagonal (a little more than half of them),
//     mirrored by the epilogue.  Q is dense with log-uniformly spread mantissas, so the truncation loss of Q^T Q is the
//     known constant and is scaled back before the identity is subtracted; what is left in D is zero-mean noise of a
//     few 1e-4 (Frobenius norm over sqrt(m)), which bounds the polished defect.
//   * The correction Q D is small (D is a few 1e-3 per row), so 8 significant bits in each factor are plenty: D is
//     stored in bf16, Q is copied to bf16 once, and the product runs at the bf16 rate, subtracted from the fp32 Q in
//     place.  (Relative error of the correction 4e-3, i.e. about 1e-5 of Q.)
// D16 and Q16 are scratch for m x ld 16-bit values each.
int polish_orthogonal_tf32(gelo_ctx* ctx, int m, float* Q, int ld, float* D16, float* Q16, cudaStream_t st)
{
    const float back2 = (1.0f + kTf32TruncLoss) * (1.0f + kTf32TruncLoss);
    GELO_TRY(launch_gram_sym_bf16(ctx, m, Q, ld, D16, ld, back2, 1.0f, 0.5f, st));
    GELO_TRY(launch_narrow(ctx, m, Q, ld, GELO_BF16, Q16, ld, st));
    return launch_gemm_bf16_sub(ctx, m, m, m, Q16, ld, D16, ld, Q, ld, st);
}

}  // namespace gelo
