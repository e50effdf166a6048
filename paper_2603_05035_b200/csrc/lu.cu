// Blocked LU with partial pivoting and the explicit inverse of the non-orthogonal
// mixing matrix (paper Mitigation 1: "The TEE must compute A^-1 per batch").
//
//   P A = L U by right-looking panels of kPanel columns:
//       panel kernel (one CTA: lane = panel column, warps stripe rows, pivot = first
//       row of largest magnitude) -> row interchanges on the rest of the matrix ->
//       U12 = L11^-1 A12 -> A22 -= L21 U12 (GEMM)
//   A^-1 = U^-1 L^-1 P by two blocked triangular solves on the permuted identity,
//   each block step a small substitution kernel plus one GEMM update.
#include <cooperative_groups.h>

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

// ---- register-resident LU panel on a thread-block cluster ------------------------------------
//
// Same elimination, with the panel in registers spread over a cluster (global warp g holds rows
// j0 + g + i * CS * 32, i = 0 .. RPT-1; lane = panel column).  Per column every CTA publishes its
// best pivot candidate TOGETHER with that row's 32 panel values into every CTA's shared memory,
// and CTA 0 publishes the current row j; after one cluster barrier all CTAs know the winner
// (largest magnitude, smallest row on a tie), swap in registers and eliminate without further
// traffic.  Only a warp's first row can lie above row j, so the other rows run branch-free.
constexpr int kClusterMax = 8;
constexpr int kMaxRowsPerThread = 20;   // rows a thread can hold in registers (64 each at 1024 threads) without heavy spills
constexpr int kClusterPanelMaxRows = kClusterMax * kPanelWarps * kMaxRowsPerThread;

template <int RPT>
__global__ void __launch_bounds__(kPanelThreads, 1)
lu_panel_cluster_kernel(float* __restrict__ M, int ld, int m, int j0, int jb, int* __restrict__ ipiv,
                        int* __restrict__ status)
{
    namespace cg = cooperative_groups;
    cg::cluster_group cluster = cg::this_cluster();
    const int CS = (int)cluster.num_blocks();
    const int rank = (int)cluster.block_rank();

    __shared__ float cand_v[kPanelWarps];
    __shared__ int cand_r[kPanelWarps];
    __shared__ float win_v[2][kClusterMax];
    __shared__ int win_r[2][kClusterMax];
    __shared__ float win_row[2][kClusterMax][NB];
    __shared__ float rowj_buf[2][NB];
    __shared__ float coef_s[NB];
    __shared__ float prow_s[NB];
    __shared__ int pr_s;

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
        x[i] = (row < m && col_ok) ? M[(size_t)row * ld + j0 + lane] : 0.0f;
    }
    if (CS > 1) cluster.sync(); else __syncthreads();

    for (int c = 0; c < jb; ++c) {
        const int j = j0 + c;
        const int par = c & 1;
        // ---- this warp's candidate (same in every lane); rows ascend with i, strict > keeps the first ----
        // (column c of a row is fetched from lane c again for the elimination below rather than kept: registers
        // decide how many rows a thread can hold, and with them how few SMs a panel occupies)
        float bv = -1.0f;
        int bi = -1;
        {
            const float a0 = fabsf(__shfl_sync(full, x[0], c));
            if (gw >= c && j0 + gw < m) { bv = a0; bi = 0; }
        }
#pragma unroll
        for (int i = 1; i < RPT; ++i) {
            const float a = fabsf(__shfl_sync(full, x[i], c));
            if (a > bv && j0 + i * stride + gw < m) { bv = a; bi = i; }
        }
        const int br = (bi >= 0) ? j0 + bi * stride + gw : 0x7fffffff;
        if (lane == 0) { cand_v[warp] = bv; cand_r[warp] = br; }
        __syncthreads();
        // ---- this CTA's candidate: every warp reduces the 32 entries the same way ----
        float cv = cand_v[lane];
        int cr = cand_r[lane];
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) {
            const float ov = __shfl_xor_sync(full, cv, off);
            const int orow = __shfl_xor_sync(full, cr, off);
            if (ov > cv || (ov == cv && orow < cr)) { cv = ov; cr = orow; }
        }
        if (bi >= 0 && cr == br) {                          // this warp owns the CTA's candidate row
            float brow = x[0];
#pragma unroll
            for (int i = 1; i < RPT; ++i) if (i == bi) brow = x[i];
            if (lane < CS) {
                cluster.map_shared_rank(&win_v[par][rank], lane)[0] = cv;
                cluster.map_shared_rank(&win_r[par][rank], lane)[0] = cr;
            }
            for (int r = 0; r < CS; ++r) cluster.map_shared_rank(&win_row[par][rank][lane], r)[0] = brow;
        } else if (cv < 0.0f && warp == 0 && lane < CS) {   // a CTA without rows >= j publishes "nothing"
            cluster.map_shared_rank(&win_v[par][rank], lane)[0] = -1.0f;
            cluster.map_shared_rank(&win_r[par][rank], lane)[0] = 0x7fffffff;
        }
        if (rank == 0 && warp == c)                          // the warp whose first row is row j
            for (int r = 0; r < CS; ++r) cluster.map_shared_rank(&rowj_buf[par][lane], r)[0] = x[0];
        if (CS > 1) cluster.sync(); else __syncthreads();

        // ---- warp 0 picks the winner over the cluster and prepares the elimination coefficients ----
        if (warp == 0) {
            float pv = (lane < CS) ? win_v[par][lane] : -2.0f;
            int pr = (lane < CS) ? win_r[par][lane] : 0x7fffffff;
            int pw = lane;
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) {
                const float ov = __shfl_xor_sync(full, pv, off);
                const int orow = __shfl_xor_sync(full, pr, off);
                const int ow = __shfl_xor_sync(full, pw, off);
                if (ov > pv || (ov == pv && orow < pr)) { pv = ov; pr = orow; pw = ow; }
            }
            const float prow = win_row[par][pw][lane];       // pivot row, this lane's column
            const float pivot = __shfl_sync(full, prow, c);
            const float inv = (pivot != 0.0f) ? 1.0f / pivot : 0.0f;
            // x <- coef * x_c + (lane == c ? 0 : x):  the multiplier l = x_c / pivot in column c, -l * pivot row after it
            coef_s[lane] = (lane > c) ? -inv * prow : ((lane == c) ? inv : 0.0f);
            prow_s[lane] = prow;
            if (lane == 0) {
                pr_s = pr;
                if (rank == 0) {
                    ipiv[j] = pr;
                    if (!(pv > 0.0f)) atomicCAS(status, 0, (int)GELO_ERR_COND);
                }
            }
        }
        __syncthreads();
        const int pr = pr_s;
        const float coef = coef_s[lane];
        // ---- swap in registers ----
        if (pr != j) {
            const int poff = pr - j0;
            if (poff % stride == gw) {                       // this warp holds row pr: it receives old row j
                const int pi = poff / stride;
                const float oldj = rowj_buf[par][lane];
#pragma unroll
                for (int i = 0; i < RPT; ++i) if (i == pi) x[i] = oldj;
            }
            if (gw == c) x[0] = prow_s[lane];                // rank 0, warp c: row j receives the pivot row
        }
        // ---- eliminate below row j ----
#pragma unroll
        for (int i = 1; i < RPT; ++i) x[i] = fmaf(coef, __shfl_sync(full, x[i], c), (lane == c) ? 0.0f : x[i]);
        {
            const float xc0 = __shfl_sync(full, x[0], c);
            if (gw > c) x[0] = fmaf(coef, xc0, (lane == c) ? 0.0f : x[0]);
        }
    }
#pragma unroll
    for (int i = 0; i < RPT; ++i) {
        const int row = j0 + i * stride + gw;
        if (row < m && col_ok) M[(size_t)row * ld + j0 + lane] = x[i];
    }
}

template <int RPT>
cudaError_t launch_cluster_lu_panel(int cs, cudaStream_t st, float* M, int ld, int m, int j0, int jb, int* ipiv,
                                    int* status)
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
    return cudaLaunchKernelEx(&cfg, lu_panel_cluster_kernel<RPT>, M, ld, m, j0, jb, ipiv, status);
}

int launch_lu_panel(gelo_ctx* ctx, float* M, int ld, int m, int j0, int jb, int* ipiv, cudaStream_t st)
{
    const int rows = m - j0;
    if (rows > kClusterPanelMaxRows) {
        lu_panel_kernel<<<1, kPanelThreads, 0, st>>>(M, ld, m, j0, jb, ipiv, ctx->status_dev);
        return after_launch(ctx);
    }
    // alone on the GPU: as many SMs as give every thread at least two rows; in a batch with many sampling lanes: as
    // few SMs as hold the panel (every SM it occupies is one that the other lanes' kernels cannot use)
    const int rows_per_thread = ctx->tc_update_ctas > 0 ? kMaxRowsPerThread : 2;
    // (a cluster may have any size up to eight: five CTAs where four are too few, not eight)
    int cs = ceil_div(rows, kPanelWarps * rows_per_thread);
    if (cs > kClusterMax) cs = kClusterMax;
    const int rpt = ceil_div(rows, cs * kPanelWarps);
    int* sd = ctx->status_dev;
    ProfScope ps(ctx, PROF_LU_PANEL, 1.0 * rows * (double)jb * jb, st);   // flops of the eliminations
    cudaError_t e;
    if (rpt <= 2) e = launch_cluster_lu_panel<2>(cs, st, M, ld, m, j0, jb, ipiv, sd);
    else if (rpt <= 3) e = launch_cluster_lu_panel<3>(cs, st, M, ld, m, j0, jb, ipiv, sd);
    else if (rpt <= 5) e = launch_cluster_lu_panel<5>(cs, st, M, ld, m, j0, jb, ipiv, sd);
    else if (rpt <= 7) e = launch_cluster_lu_panel<7>(cs, st, M, ld, m, j0, jb, ipiv, sd);
    else if (rpt <= 9) e = launch_cluster_lu_panel<9>(cs, st, M, ld, m, j0, jb, ipiv, sd);
    else if (rpt <= 11) e = launch_cluster_lu_panel<11>(cs, st, M, ld, m, j0, jb, ipiv, sd);
    else if (rpt <= 13) e = launch_cluster_lu_panel<13>(cs, st, M, ld, m, j0, jb, ipiv, sd);
    else if (rpt <= 15) e = launch_cluster_lu_panel<15>(cs, st, M, ld, m, j0, jb, ipiv, sd);
    else if (rpt <= 17) e = launch_cluster_lu_panel<17>(cs, st, M, ld, m, j0, jb, ipiv, sd);
    else e = launch_cluster_lu_panel<20>(cs, st, M, ld, m, j0, jb, ipiv, sd);
    if (e != cudaSuccess) return GELO_ERR_CUDA;
    return after_launch(ctx);
}

// Row interchanges of a panel or an outer block, in two launches:
//   compose_swaps_kernel (one warp): turns rows j0+c <-> ipiv[j0+c], c = 0 .. jb-1 (in order, jb <= 128) into a
//       row permutation of the at most 2 jb rows they touch: table[0] = count, then (target row, source row) pairs;
//   swap_rows_kernel: every CTA moves 32 columns of those rows through a shared-memory tile (gather from the
//       source rows, scatter to the targets) for columns [c_lo, c_hi) minus [skip_lo, skip_hi).
constexpr int kSwapMaxRows = 256;

__global__ void __launch_bounds__(32)
compose_swaps_kernel(int j0, int jb, const int* __restrict__ ipiv, int* __restrict__ table)
{
    __shared__ int pos_s[kSwapMaxRows];       // row that receives ...
    __shared__ int src_s[kSwapMaxRows];       // ... the content this row had before the interchanges
    const int lane = threadIdx.x;
    int count = 0;
    for (int c = 0; c < jb; ++c) {
        const int a = j0 + c, b = ipiv[a];
        if (a == b) continue;
        int ia = -1, ib = -1;
        for (int base = 0; base < count; base += 32) {
            const int e = base + lane;
            const int p = (e < count) ? pos_s[e] : -1;
            const unsigned ma = __ballot_sync(0xffffffffu, p == a);
            const unsigned mb = __ballot_sync(0xffffffffu, p == b);
            if (ma) ia = base + __ffs(ma) - 1;
            if (mb) ib = base + __ffs(mb) - 1;
        }
        if (ia < 0) { ia = count; if (lane == 0) { pos_s[count] = a; src_s[count] = a; } ++count; }
        if (ib < 0) { ib = count; if (lane == 0) { pos_s[count] = b; src_s[count] = b; } ++count; }
        __syncwarp();
        if (lane == 0) { const int t = src_s[ia]; src_s[ia] = src_s[ib]; src_s[ib] = t; }
        __syncwarp();
    }
    if (lane == 0) table[0] = count;
    for (int e = lane; e < count; e += 32) { table[1 + 2 * e] = pos_s[e]; table[2 + 2 * e] = src_s[e]; }
}

__global__ void __launch_bounds__(256)
swap_rows_kernel(float* __restrict__ X, int ld, const int* __restrict__ table, int c_lo, int c_hi, int skip_lo,
                 int skip_hi)
{
    __shared__ float tile[kSwapMaxRows][33];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int count = table[0];
    int col = c_lo + blockIdx.x * 32 + lane;
    if (col >= skip_lo && col < skip_hi) col = c_hi;          // inactive lane
    const bool ok = col < c_hi;
    for (int e = warp; e < count; e += 8)
        if (ok) tile[e][lane] = X[(size_t)table[2 + 2 * e] * ld + col];
    __syncthreads();
    for (int e = warp; e < count; e += 8) {
        const int pos = table[1 + 2 * e], src = table[2 + 2 * e];
        if (ok && src != pos) X[(size_t)pos * ld + col] = tile[e][lane];
    }
}

int launch_swaps(gelo_ctx* ctx, float* X, int ld, int j0, int jb, const int* ipiv, int* table, bool compose,
                 int c_lo, int c_hi, int skip_lo, int skip_hi, cudaStream_t st)
{
    if (compose) {
        compose_swaps_kernel<<<1, 32, 0, st>>>(j0, jb, ipiv, table);
        GELO_TRY(after_launch(ctx));
    }
    if (c_hi <= c_lo) return GELO_OK;
    swap_rows_kernel<<<ceil_div(c_hi - c_lo, 32), 256, 0, st>>>(X, ld, table, c_lo, c_hi, skip_lo, skip_hi);
    return after_launch(ctx);
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

// The same solve for a whole outer block (ob <= 128 rows) in one launch: the block's triangle sits transposed in
// shared memory, every thread owns one column of X (its 128 entries in a shared-memory tile) and works through
// the four 32-row sub-blocks with the sub-block in registers: first the contributions of the rows already solved
// (32 independent FMAs per shared-memory value), then the 32 x 32 substitution.
// one 4-byte asynchronous copy global -> shared
__device__ __forceinline__ void cp_async_f32(float* smem_dst, const float* gsrc)
{
    const uint32_t d = (uint32_t)__cvta_generic_to_shared(smem_dst);
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(d), "l"(gsrc) : "memory");
}

constexpr int kTri128LtStride = 132;
constexpr int kTri128SmemBytes = (128 * kTri128LtStride + 128 * 129) * 4;

template <bool UPPER>
__global__ void __launch_bounds__(128)
tri_solve128_kernel(const float* M, int ldm, float* X, int ldx, int b0, int ob, int c_lo, int c_hi)
{
    extern __shared__ __align__(16) float tsm[];
    float (*Lt)[kTri128LtStride] = reinterpret_cast<float (*)[kTri128LtStride]>(tsm);   // Lt[t][i] = L[i][t]
    float (*tile)[129] = reinterpret_cast<float (*)[129]>(tsm + 128 * kTri128LtStride);
    const int tid = threadIdx.x;
    const int col = c_lo + blockIdx.x * 128 + tid;
    const bool ok = col < c_hi;
    // The two fills are pure latency (the arithmetic of the solve is about 6 us): every element goes straight from
    // global to shared memory as an asynchronous 4-byte copy, so that all 256 loads of a thread are in flight at once.
#pragma unroll 8
    for (int i = 0; i < 128; ++i) {
        if (i < ob && tid < ob) cp_async_f32(&Lt[tid][i], M + (size_t)(b0 + i) * ldm + b0 + tid);
        else Lt[tid][i] = 0.0f;
        if (ok && i < ob) cp_async_f32(&tile[i][tid], X + (size_t)(b0 + i) * ldx + col);
        else tile[i][tid] = 0.0f;
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    __syncthreads();
    const int nsub = (ob + NB - 1) / NB;
    for (int q = 0; q < nsub; ++q) {
        const int sidx = UPPER ? (nsub - 1 - q) : q;
        const int r0 = sidx * NB;
        float x[NB];
#pragma unroll
        for (int i = 0; i < NB; ++i) x[i] = tile[r0 + i][tid];
        const int t_lo = UPPER ? r0 + NB : 0;
        const int t_hi = UPPER ? nsub * NB : r0;
        for (int t = t_lo; t < t_hi; ++t) {
            const float xt = tile[t][tid];
            const float4* lp = reinterpret_cast<const float4*>(&Lt[t][r0]);
#pragma unroll
            for (int i4 = 0; i4 < NB / 4; ++i4) {
                const float4 l = lp[i4];
                x[4 * i4 + 0] = fmaf(-l.x, xt, x[4 * i4 + 0]);
                x[4 * i4 + 1] = fmaf(-l.y, xt, x[4 * i4 + 1]);
                x[4 * i4 + 2] = fmaf(-l.z, xt, x[4 * i4 + 2]);
                x[4 * i4 + 3] = fmaf(-l.w, xt, x[4 * i4 + 3]);
            }
        }
        if (!UPPER) {
#pragma unroll
            for (int i = 1; i < NB; ++i) {
                float sacc = x[i];
#pragma unroll
                for (int t = 0; t < i; ++t) sacc = fmaf(-Lt[r0 + t][r0 + i], x[t], sacc);
                x[i] = sacc;
            }
        } else {
#pragma unroll
            for (int i = NB - 1; i >= 0; --i) {
                if (r0 + i < ob) {
                    float sacc = x[i];
#pragma unroll
                    for (int t = i + 1; t < NB; ++t) sacc = fmaf(-Lt[r0 + t][r0 + i], x[t], sacc);
                    x[i] = sacc / Lt[r0 + i][r0 + i];
                }
            }
        }
#pragma unroll
        for (int i = 0; i < NB; ++i) tile[r0 + i][tid] = x[i];
    }
    if (ok) {
#pragma unroll 16
        for (int t = 0; t < 128; ++t)
            if (t < ob) X[(size_t)(b0 + t) * ldx + col] = tile[t][tid];
    }
}

template <bool UPPER>
int launch_tri_solve128(gelo_ctx* ctx, const float* M, int ldm, float* X, int ldx, int b0, int ob, int c_lo, int c_hi,
                        cudaStream_t st)
{
    if (c_hi <= c_lo) return GELO_OK;
    GELO_CUDA_OK(cudaFuncSetAttribute(tri_solve128_kernel<UPPER>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                      kTri128SmemBytes));
    tri_solve128_kernel<UPPER><<<ceil_div(c_hi - c_lo, 128), 128, kTri128SmemBytes, st>>>(M, ldm, X, ldx, b0, ob, c_lo, c_hi);
    return after_launch(ctx);
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

__global__ void permuted_ones_kernel(float* __restrict__ X, int ld, int m, const int* __restrict__ perm)
{
    const int r = blockIdx.x * blockDim.x + threadIdx.x;
    if (r < m) X[(size_t)r * ld + perm[r]] = 1.0f;
}

// X[:, perm[k]] = Z[:, k] for every column k (Z P for the permutation matrix P with P[k, perm[k]] = 1); the padding
// columns of X are cleared.  One CTA per row: the row is read in order and scattered inside its own 4 ld bytes.
__global__ void __launch_bounds__(256)
permute_columns_kernel(const float* __restrict__ Z, float* __restrict__ X, int ld, int m, const int* __restrict__ perm)
{
    const size_t row = (size_t)blockIdx.x * ld;
    for (int k = threadIdx.x; k < ld; k += 256) {
        if (k < m) X[row + perm[k]] = Z[row + k];
        else X[row + k] = 0.0f;
    }
}

__global__ void unit_diagonal_kernel(float* __restrict__ Z, int ld, int m)
{
    const int r = blockIdx.x * blockDim.x + threadIdx.x;
    if (r < m) Z[(size_t)r * ld + r] = 1.0f;
}

// X = P (X[i, perm[i]] = 1): a memset at copy speed, then the ones.
int set_permutation(gelo_ctx* ctx, float* X, int ld, int m, const int* perm, cudaStream_t st)
{
    GELO_CUDA_OK(cudaMemsetAsync(X, 0, (size_t)m * ld * sizeof(float), st));
    permuted_ones_kernel<<<ceil_div(m, 256), 256, 0, st>>>(X, ld, m, perm);
    return after_launch(ctx);
}

}  // namespace

LuScratch carve_lu(Arena& a, int m, int ld)
{
    (void)ld;
    LuScratch s;
    s.ipiv = static_cast<int*>(a.take((size_t)m * sizeof(int)));
    s.perm = static_cast<int*>(a.take((size_t)m * sizeof(int)));
    s.swap_table = static_cast<int*>(a.take((size_t)(2 * 256 + 4) * sizeof(int)));
    return s;
}

// Level-3 variant: outer blocks of kOuter columns.  Inside a block the 32-column panels and rank-32
// updates above run on the block only; everything outside the block is updated once per block by a
// split-precision tensor-core product (K = kOuter), which cuts the passes over the big matrices by four.
// Blocked LU with partial pivoting and the inverse, level-3 work on the tensor cores.  Panels of 32 columns and
// blocks of 128 are factorised as in run_lu_inverse; blocks are grouped into superblocks of kSuper = 512 columns.
// Inside a superblock a finished block updates the superblock's remaining columns only; everything right of (below)
// the superblock is updated ONCE with all 512 columns of L (rows of U), after the 512-row strip of U (of the
// right-hand sides) has been solved block by block.  The big matrices thus stream through the GPU once per 512
// columns instead of once per 128, which is what the 128-column updates were bound by.
int run_lu_inverse_tc(gelo_ctx* ctx, int m, const float* A, int ld, float* X, const LuScratch& s, const TcScratch& tc,
                      bool tf32, cudaStream_t st)
{
    float* M = s.M;
    GELO_CUDA_OK(cudaMemcpyAsync(M, A, (size_t)m * ld * sizeof(float), cudaMemcpyDeviceToDevice, st));
    auto at = [&](float* base, int r, int c) { return base + (size_t)r * ld + c; };
    for (int s0 = 0; s0 < m; s0 += kSuper) {
        const int sw = (m - s0 < kSuper) ? (m - s0) : kSuper;
        const int send = s0 + sw;
        for (int b0 = s0; b0 < send; b0 += kOuter) {
            const int ob = (send - b0 < kOuter) ? (send - b0) : kOuter;
            const int bend = b0 + ob;
            for (int j0 = b0; j0 < bend; j0 += NB) {
                const int jb = (bend - j0 < NB) ? (bend - j0) : NB;
                GELO_TRY(launch_lu_panel(ctx, M, ld, m, j0, jb, s.ipiv, st));
                if (ob > jb) {       // interchanges on the other columns of this block
                    GELO_TRY(launch_swaps(ctx, M, ld, j0, jb, s.ipiv, s.swap_table, true, b0, bend, j0, j0 + jb, st));
                }
                const int ncb = bend - (j0 + jb);
                if (ncb > 0) {
                    tri_solve_block_kernel<false><<<ceil_div(ncb, 256), 256, 0, st>>>(M, ld, M, ld, j0, jb, j0 + jb, bend);
                    GELO_TRY(after_launch(ctx));
                    GELO_TRY(launch_rank_update(ctx, M + (size_t)(j0 + jb) * ld + j0, ld, M + (size_t)j0 * ld + j0 + jb, ld,
                                                M + (size_t)(j0 + jb) * ld + j0 + jb, ld, m - j0 - jb, ncb, jb, st));
                }
            }
            if (m > ob) {            // the block's interchanges on everything left and right of it
                GELO_TRY(launch_swaps(ctx, M, ld, b0, ob, s.ipiv, s.swap_table, true, 0, m, b0, bend, st));
            }
            if (send > bend) {       // the rest of the superblock: U12 = L11^-1 A12, A22 -= L21 U12
                GELO_TRY(launch_tri_solve128<false>(ctx, M, ld, M, ld, b0, ob, bend, send, st));
                GELO_TRY(tc_update_f32(ctx, tc, tf32, m - bend, send - bend, ob, at(M, bend, b0), ld, at(M, b0, bend), ld,
                                       at(M, bend, bend), ld, st));
            }
        }
        const int nc = m - send;
        if (nc <= 0) continue;
        // the superblock's row strip of U, block row by block row
        for (int b0 = s0; b0 < send; b0 += kOuter) {
            const int ob = (send - b0 < kOuter) ? (send - b0) : kOuter;
            const int bend = b0 + ob;
            GELO_TRY(launch_tri_solve128<false>(ctx, M, ld, M, ld, b0, ob, send, m, st));
            if (send > bend)
                GELO_TRY(tc_update_f32(ctx, tc, tf32, send - bend, nc, ob, at(M, bend, b0), ld, at(M, b0, send), ld,
                                       at(M, bend, send), ld, st));
        }
        // A22 -= L21 U12 with all sw columns at once
        GELO_TRY(tc_update_f32(ctx, tc, tf32, nc, nc, sw, at(M, send, s0), ld, at(M, s0, send), ld, at(M, send, send), ld, st));
    }
    // ---- X = P, then L Y = P, then U X = Y ----
    const size_t perm_smem = (size_t)m * sizeof(int);
    if (perm_smem > 48 * 1024)
        GELO_CUDA_OK(cudaFuncSetAttribute(build_perm_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)perm_smem));
    build_perm_kernel<<<1, 256, perm_smem, st>>>(s.ipiv, s.perm, m);
    GELO_TRY(after_launch(ctx));
    if (s.Z) {
        // L Y = P: Y = L^-1 P, and L^-1 is unit lower triangular.  Z = L^-1 is built in place from the identity, every
        // block row touching only the columns left of its own end (the rest are zeros that stay zeros), which is a
        // third of the arithmetic of solving against the dense P; Y is Z with its columns permuted.
        float* Z = s.Z;
        GELO_CUDA_OK(cudaMemsetAsync(Z, 0, (size_t)m * ld * sizeof(float), st));
        unit_diagonal_kernel<<<ceil_div(m, 256), 256, 0, st>>>(Z, ld, m);
        GELO_TRY(after_launch(ctx));
        for (int s0 = 0; s0 < m; s0 += kSuper) {
            const int sw = (m - s0 < kSuper) ? (m - s0) : kSuper;
            const int send = s0 + sw;
            for (int b0 = s0; b0 < send; b0 += kOuter) {
                const int ob = (send - b0 < kOuter) ? (send - b0) : kOuter;
                const int bend = b0 + ob;
                GELO_TRY(launch_tri_solve128<false>(ctx, M, ld, Z, ld, b0, ob, 0, bend, st));
                if (send > bend)
                    GELO_TRY(tc_update_f32(ctx, tc, tf32, send - bend, bend, ob, at(M, bend, b0), ld, at(Z, b0, 0), ld,
                                           at(Z, bend, 0), ld, st));
            }
            if (m > send)
                GELO_TRY(tc_update_f32(ctx, tc, tf32, m - send, send, sw, at(M, send, s0), ld, at(Z, s0, 0), ld, at(Z, send, 0), ld,
                                       st));
        }
        permute_columns_kernel<<<m, 256, 0, st>>>(Z, X, ld, m, s.perm);
        GELO_TRY(after_launch(ctx));
    } else {
    GELO_TRY(set_permutation(ctx, X, ld, m, s.perm, st));
    for (int s0 = 0; s0 < m; s0 += kSuper) {
        const int sw = (m - s0 < kSuper) ? (m - s0) : kSuper;
        const int send = s0 + sw;
        for (int b0 = s0; b0 < send; b0 += kOuter) {
            const int ob = (send - b0 < kOuter) ? (send - b0) : kOuter;
            const int bend = b0 + ob;
            GELO_TRY(launch_tri_solve128<false>(ctx, M, ld, X, ld, b0, ob, 0, m, st));
            if (send > bend)
                GELO_TRY(tc_update_f32(ctx, tc, tf32, send - bend, m, ob, at(M, bend, b0), ld, at(X, b0, 0), ld, at(X, bend, 0),
                                       ld, st));
        }
        if (m > send)
            GELO_TRY(tc_update_f32(ctx, tc, tf32, m - send, m, sw, at(M, send, s0), ld, at(X, s0, 0), ld, at(X, send, 0), ld, st));
    }
    }
    const int nsuper = ceil_div(m, kSuper);
    for (int sb = nsuper - 1; sb >= 0; --sb) {
        const int s0 = sb * kSuper;
        const int sw = (m - s0 < kSuper) ? (m - s0) : kSuper;
        const int send = s0 + sw;
        const int nblk = ceil_div(sw, kOuter);
        for (int bi = nblk - 1; bi >= 0; --bi) {
            const int b0 = s0 + bi * kOuter;
            const int ob = (send - b0 < kOuter) ? (send - b0) : kOuter;
            GELO_TRY(launch_tri_solve128<true>(ctx, M, ld, X, ld, b0, ob, 0, m, st));
            if (b0 > s0)
                GELO_TRY(tc_update_f32(ctx, tc, tf32, b0 - s0, m, ob, at(M, s0, b0), ld, at(X, b0, 0), ld, at(X, s0, 0), ld, st));
        }
        if (s0 > 0) GELO_TRY(tc_update_f32(ctx, tc, tf32, s0, m, sw, at(M, 0, s0), ld, at(X, s0, 0), ld, X, ld, st));
    }
    return GELO_OK;
}

int run_lu_inverse(gelo_ctx* ctx, int m, const float* A, int ld, float* X, const LuScratch& s, cudaStream_t st)
{
    if ((size_t)m * sizeof(int) > 200 * 1024) return GELO_ERR_UNSUPPORTED;
    float* M = s.M;
    GELO_CUDA_OK(cudaMemcpyAsync(M, A, (size_t)m * ld * sizeof(float), cudaMemcpyDeviceToDevice, st));
    const int npanels = ceil_div(m, NB);
    for (int pnl = 0; pnl < npanels; ++pnl) {
        const int j0 = pnl * NB, jb = (m - j0 < NB) ? (m - j0) : NB;
        GELO_TRY(launch_lu_panel(ctx, M, ld, m, j0, jb, s.ipiv, st));
        if (m > jb) {
            GELO_TRY(launch_swaps(ctx, M, ld, j0, jb, s.ipiv, s.swap_table, true, 0, m, j0, j0 + jb, st));
        }
        const int nc = m - j0 - jb;
        if (nc <= 0) continue;
        tri_solve_block_kernel<false><<<ceil_div(nc, 256), 256, 0, st>>>(M, ld, M, ld, j0, jb, j0 + jb, m);
        GELO_TRY(after_launch(ctx));
        // A22 -= L21 U12
        GELO_TRY(launch_rank_update(ctx, M + (size_t)(j0 + jb) * ld + j0, ld, M + (size_t)j0 * ld + j0 + jb, ld,
                                    M + (size_t)(j0 + jb) * ld + j0 + jb, ld, nc, nc, jb, st));
    }
    // ---- X = P, then L Y = P, then U X = Y ----
    const size_t perm_smem = (size_t)m * sizeof(int);
    if (perm_smem > 48 * 1024)
        GELO_CUDA_OK(cudaFuncSetAttribute(build_perm_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)perm_smem));
    build_perm_kernel<<<1, 256, perm_smem, st>>>(s.ipiv, s.perm, m);
    GELO_TRY(after_launch(ctx));
    GELO_TRY(set_permutation(ctx, X, ld, m, s.perm, st));
    for (int pnl = 0; pnl < npanels; ++pnl) {
        const int i0 = pnl * NB, ib = (m - i0 < NB) ? (m - i0) : NB;
        tri_solve_block_kernel<false><<<ceil_div(m, 256), 256, 0, st>>>(M, ld, X, ld, i0, ib, 0, m);
        GELO_TRY(after_launch(ctx));
        const int nr = m - i0 - ib;
        if (nr <= 0) continue;
        // X[i0+ib:, :] -= L[i0+ib:, i0:i0+ib] X[i0:i0+ib, :]
        GELO_TRY(launch_rank_update(ctx, M + (size_t)(i0 + ib) * ld + i0, ld, X + (size_t)i0 * ld, ld,
                                    X + (size_t)(i0 + ib) * ld, ld, nr, m, ib, st));
    }
    for (int pnl = npanels - 1; pnl >= 0; --pnl) {
        const int i0 = pnl * NB, ib = (m - i0 < NB) ? (m - i0) : NB;
        tri_solve_block_kernel<true><<<ceil_div(m, 256), 256, 0, st>>>(M, ld, X, ld, i0, ib, 0, m);
        GELO_TRY(after_launch(ctx));
        if (i0 <= 0) continue;
        // X[0:i0, :] -= U[0:i0, i0:i0+ib] X[i0:i0+ib, :]
        GELO_TRY(launch_rank_update(ctx, M + i0, ld, X + (size_t)i0 * ld, ld, X, ld, i0, m, ib, st));
    }
    return GELO_OK;
}

}  // namespace gelo
