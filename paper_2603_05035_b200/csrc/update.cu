// Rank-32 building blocks of the blocked QR and LU (paper Section 3.2 step 1.2: the cost of
// generating A; Table 3 "A-gen (QR)").  With 32-column panels the trailing updates move
// 12 bytes per 64 flops, far below the machine's flop/byte ridge, so these kernels are built
// as HBM streamers: 16-byte coalesced accesses, every element of the trailing matrix read
// once per pass, fp32 arithmetic on the ordinary FMA pipes.
//
//   vtc_partial : Wp[s] = V[rows of slab s]^T * C[rows of slab s, :]        (split over rows)
//   w_reduce    : W = op(T) * sum_s Wp[s]                                    (fixed order)
//   rank_update : C -= A * B,  A: M x K (K <= 32),  B: K x N
#include "common.cuh"

namespace gelo {

namespace {

constexpr int NB = kPanel;

// ---- Wp[s][a][col] = sum_{r in slab s} V[r][a] * C[r][col] --------------------------------------
// One CTA owns 128 columns of C and one slab of rows.  Rows arrive in 32-row stages through a
// four-deep cp.async pipeline (C stage 16 KiB + V stage 4 KiB), so each CTA keeps ~60 KiB of
// loads in flight; out-of-range rows and columns are zero-filled by the copy itself.
// Thread (g, l) = (tid / 32, tid % 32) accumulates reflector columns 4g..4g+3 against C columns
// 4l..4l+3 from shared memory.
constexpr int kVtcStages = 4;
constexpr int kVtcRows = 32;
constexpr int kVtcStageFloats = kVtcRows * 128 + kVtcRows * NB;      // C tile then V tile
constexpr int kVtcSmemBytes = kVtcStages * kVtcStageFloats * 4;

__device__ __forceinline__ void cp_async16(float* smem_dst, const float* gmem_src, int src_bytes)
{
    const uint32_t d = (uint32_t)__cvta_generic_to_shared(smem_dst);
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(d), "l"(gmem_src), "r"(src_bytes) : "memory");
}

__global__ void __launch_bounds__(256)
vtc_partial_kernel(const float* __restrict__ V, int ldv, int kv, const float* __restrict__ C, int ldc,
                   int nr, int nc, int rows_per_slab, float* __restrict__ Wp, int ldw)
{
    extern __shared__ __align__(16) float vtc_smem[];
    const int tid = threadIdx.x;
    const int g = tid >> 5, l = tid & 31;
    const int n0 = blockIdx.x * 128;
    const int slab = blockIdx.y;
    const int r0 = slab * rows_per_slab;
    const int r1 = min(nr, r0 + rows_per_slab);
    const int ntiles = (r1 - r0 + kVtcRows - 1) / kVtcRows;

    auto issue = [&](int t) {
        if (t < ntiles) {
            float* cs = vtc_smem + (t % kVtcStages) * kVtcStageFloats;
            float* vs = cs + kVtcRows * 128;
            const int rbase = r0 + t * kVtcRows;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int rr = (tid >> 5) + 8 * i;
                const int row = rbase + rr;
                const int col = n0 + l * 4;
                int valid = (row < r1) ? min(4, nc - col) : 0;
                if (valid < 0) valid = 0;
                const float* src = C + (size_t)min(row, nr - 1) * ldc + (valid > 0 ? col : 0);
                cp_async16(cs + rr * 128 + l * 4, src, valid * 4);
            }
            {
                const int rr = tid >> 3, v4 = (tid & 7) * 4;
                const int row = rbase + rr;
                int valid = (row < r1) ? min(4, kv - v4) : 0;
                if (valid < 0) valid = 0;
                const float* src = V + (size_t)min(row, nr - 1) * ldv + (valid > 0 ? v4 : 0);
                cp_async16(vs + rr * NB + v4, src, valid * 4);
            }
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
    };

    float acc[4][4];
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[a][j] = 0.0f;

#pragma unroll
    for (int t = 0; t < kVtcStages - 1; ++t) issue(t);
    for (int t = 0; t < ntiles; ++t) {
        asm volatile("cp.async.wait_group %0;" ::"n"(kVtcStages - 2) : "memory");
        __syncthreads();
        issue(t + kVtcStages - 1);
        const float* cs = vtc_smem + (t % kVtcStages) * kVtcStageFloats;
        const float* vs = cs + kVtcRows * 128;
#pragma unroll 8
        for (int k = 0; k < kVtcRows; ++k) {
            const float4 c = *reinterpret_cast<const float4*>(cs + k * 128 + l * 4);
            const float4 v = *reinterpret_cast<const float4*>(vs + k * NB + g * 4);
            const float cc[4] = {c.x, c.y, c.z, c.w};
            const float vv[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
            for (int a = 0; a < 4; ++a)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[a][j] = fmaf(vv[a], cc[j], acc[a][j]);
        }
    }
    asm volatile("cp.async.wait_group 0;" ::: "memory");

    float* out = Wp + (size_t)slab * NB * ldw;
    const int col0 = n0 + l * 4;
#pragma unroll
    for (int a = 0; a < 4; ++a) {
        float* o = out + (size_t)(g * 4 + a) * ldw + col0;
        if (col0 + 3 < nc && (ldw & 3) == 0) {
            *reinterpret_cast<float4*>(o) = make_float4(acc[a][0], acc[a][1], acc[a][2], acc[a][3]);
        } else {
#pragma unroll
            for (int j = 0; j < 4; ++j)
                if (col0 + j < nc) o[j] = acc[a][j];
        }
    }
}

// ---- W[a][col] = sum_b Top[a][b] * (sum_s Wp[s][b][col]),  Top = T or T^T -------------------------
// One CTA per 32 columns: first the slab sums (thread = (row b, column)), then the 32 x 32 product.
__global__ void __launch_bounds__(256)
w_reduce_kernel(const float* __restrict__ Wp, int ldw, int slabs, int nc, const float* __restrict__ T,
                int transpose_t, float* __restrict__ W)
{
    __shared__ float t_s[NB][NB + 1];
    __shared__ float w_s[NB][NB + 1];
    const int tid = threadIdx.x;
    const int l = tid & 31, g = tid >> 5;
    for (int idx = tid; idx < NB * NB; idx += 256) {
        const int a = idx / NB, b = idx % NB;
        t_s[a][b] = !T ? (a == b ? 1.0f : 0.0f) : (transpose_t ? T[b * NB + a] : T[a * NB + b]);   // no T: identity
    }
    const int col = blockIdx.x * 32 + l;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int b = g + 8 * i;
        float s = 0.0f;
        if (col < nc)
            for (int sl = 0; sl < slabs; ++sl) s += Wp[((size_t)sl * NB + b) * ldw + col];
        w_s[b][l] = s;
    }
    __syncthreads();
    if (col >= nc) return;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int a = g + 8 * i;
        float s = 0.0f;
#pragma unroll
        for (int b = 0; b < NB; ++b) s = fmaf(t_s[a][b], w_s[b][l], s);
        W[(size_t)a * ldw + col] = s;
    }
}

// ---- C (M x N) -= A (M x K) * B (K x N), K <= 32 -------------------------------------------------------
// 128 x 128 tile, 256 threads, 8 x 8 outputs per thread; A and B tiles staged once in shared memory.
__global__ void __launch_bounds__(256)
rank_update_kernel(const float* __restrict__ A, int lda, const float* __restrict__ B, int ldb,
                   float* __restrict__ C, int ldc, int M, int N, int K)
{
    __shared__ __align__(16) float As[NB][128 + 4];
    __shared__ __align__(16) float Bs[NB][128 + 4];
    const int tid = threadIdx.x;
    const int m0 = blockIdx.y * 128, n0 = blockIdx.x * 128;
    const int ty = tid >> 4, tx = tid & 15;
    // the tile of C goes into the accumulators first, so its latency hides behind the staging
    const bool c_vec = ((ldc & 3) == 0) && ((reinterpret_cast<uintptr_t>(C) & 15u) == 0) && (n0 + 128 <= N);
    float acc[8][8];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const int gm = m0 + ty * 4 + (i >> 2) * 64 + (i & 3);
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int gn = n0 + tx * 4 + h * 64;
            const float* p = C + (size_t)gm * ldc + gn;
            if (gm < M && c_vec) {
                const float4 t = *reinterpret_cast<const float4*>(p);
                acc[i][4 * h + 0] = t.x; acc[i][4 * h + 1] = t.y; acc[i][4 * h + 2] = t.z; acc[i][4 * h + 3] = t.w;
            } else {
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][4 * h + j] = (gm < M && gn + j < N) ? p[j] : 0.0f;
            }
        }
    }
    const bool a_vec = ((lda & 3) == 0) && ((reinterpret_cast<uintptr_t>(A) & 15u) == 0) && K == NB;
    const bool b_vec = ((ldb & 3) == 0) && ((reinterpret_cast<uintptr_t>(B) & 15u) == 0) && (n0 + 128 <= N);
    // A tile: 128 rows x 32 k, four float4 per thread (8 threads per row)
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int idx = tid + i * 256;
        const int r = idx >> 3, k4 = (idx & 7) * 4;
        const int gm = m0 + r;
        float v[4] = {0.0f, 0.0f, 0.0f, 0.0f};
        if (gm < M) {
            if (a_vec) {
                const float4 t = *reinterpret_cast<const float4*>(A + (size_t)gm * lda + k4);
                v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w;
            } else {
#pragma unroll
                for (int j = 0; j < 4; ++j) if (k4 + j < K) v[j] = A[(size_t)gm * lda + k4 + j];
            }
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) As[k4 + j][r] = v[j];
    }
    // B tile: 32 k x 128 columns, four float4 per thread (32 threads per row)
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int idx = tid + i * 256;
        const int k = idx >> 5, c4 = (idx & 31) * 4;
        float4 t = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
        if (k < K) {
            if (b_vec) {
                t = *reinterpret_cast<const float4*>(B + (size_t)k * ldb + n0 + c4);
            } else {
                const float* p = B + (size_t)k * ldb + n0 + c4;
                if (n0 + c4 + 0 < N) t.x = p[0];
                if (n0 + c4 + 1 < N) t.y = p[1];
                if (n0 + c4 + 2 < N) t.z = p[2];
                if (n0 + c4 + 3 < N) t.w = p[3];
            }
        }
        *reinterpret_cast<float4*>(&Bs[k][c4]) = t;
    }
    __syncthreads();

#pragma unroll
    for (int k = 0; k < NB; ++k) {
        const float4 a0 = *reinterpret_cast<const float4*>(&As[k][ty * 4]);
        const float4 a1 = *reinterpret_cast<const float4*>(&As[k][ty * 4 + 64]);
        const float4 b0 = *reinterpret_cast<const float4*>(&Bs[k][tx * 4]);
        const float4 b1 = *reinterpret_cast<const float4*>(&Bs[k][tx * 4 + 64]);
        const float a[8] = {a0.x, a0.y, a0.z, a0.w, a1.x, a1.y, a1.z, a1.w};
        const float b[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
#pragma unroll
        for (int i = 0; i < 8; ++i)
#pragma unroll
            for (int j = 0; j < 8; ++j) acc[i][j] = fmaf(-a[i], b[j], acc[i][j]);
    }

#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const int gm = m0 + ty * 4 + (i >> 2) * 64 + (i & 3);
        if (gm >= M) continue;
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int gn = n0 + tx * 4 + h * 64;
            float* p = C + (size_t)gm * ldc + gn;
            if (c_vec) {
                *reinterpret_cast<float4*>(p) = make_float4(acc[i][4 * h + 0], acc[i][4 * h + 1], acc[i][4 * h + 2],
                                                            acc[i][4 * h + 3]);
            } else {
#pragma unroll
                for (int j = 0; j < 4; ++j)
                    if (gn + j < N) p[j] = acc[i][4 * h + j];
            }
        }
    }
}

}  // namespace

TcScratch carve_tc(Arena& a, int m, int ld, char** idle, size_t* idle_bytes)
{
    TcScratch t;
    for (int h = 0; h < 2; ++h) {
        t.panA[h] = a.take((size_t)m * kSuper * 2);
        t.panAt[h] = a.take((size_t)kOuter * ld * 2);
        t.rowB[h] = a.take((size_t)kSuper * ld * 2);
        t.rowB2[h] = a.take((size_t)kOuter * ld * 2);
        t.tt[h] = a.take((size_t)kOuter * kOuter * 2);
    }
    t.t128 = static_cast<float*>(a.take((size_t)kOuter * kOuter * 4));
    t.gram = static_cast<float*>(a.take((size_t)(m / 256 + 2) * kOuter * kOuter * 4));   // one partial Gram per 256-row slab
    t.wf32 = static_cast<float*>(take_idle(a, idle, idle_bytes, (size_t)kMaxKSplit * kOuter * ld * 4));
    for (int h = 0; h < 2; ++h) t.w32[h] = static_cast<float*>(take_idle(a, idle, idle_bytes, (size_t)kSuper * ld * 4));
    t.tsuper = static_cast<float*>(a.take((size_t)ceil_div(m, kSuper) * kSuper * kSuper * 4));
    t.sx = static_cast<float*>(a.take((size_t)kOuter * (kSuper + kOuter) * 4));
    t.xb = static_cast<float*>(a.take((size_t)kSuper * kOuter * 4));
    return t;
}

int tc_update_f32(gelo_ctx* ctx, const TcScratch& t, bool tf32, int M, int N, int K, const float* A, int lda,
                  const float* B, int ldb, float* C, int ldc, cudaStream_t st)
{
    if (M <= 0 || N <= 0 || K <= 0) return GELO_OK;
    if (K > kSuper) return GELO_ERR_INVALID;
    if (tf32) return launch_gemm_tf32(ctx, M, N, K, A, lda, false, B, ldb, true, C, ldc, false, 1.0f, 1, 0, nullptr, st);
    const int ldn = (N + 7) & ~7;
    const int ldk = (K + 63) & ~63;
    GELO_TRY(launch_split_pair(ctx, A, lda, M, K, t.panA[0], t.panA[1], ldk, B, ldb, K, N, t.rowB[0], t.rowB[1], ldn, st));
    return launch_gemm_tc_split(ctx, M, N, K, t.panA[0], t.panA[1], ldk, t.rowB[0], t.rowB[1], ldn, C, ldc,
                                nullptr, nullptr, 0, false, st);
}

int panel_slab_count(gelo_ctx* ctx, int nr, int nc)
{
    // enough CTAs to cover the GPU about twice (two CTAs fit per SM), slabs of at least 128 rows
    const int col_tiles = ceil_div(nc, 128);
    int slabs = ceil_div(2 * ctx->sm_count, col_tiles);
    const int max_by_rows = ceil_div(nr, 128);
    if (slabs > max_by_rows) slabs = max_by_rows;
    if (slabs > kMaxSlabs) slabs = kMaxSlabs;
    if (slabs < 1) slabs = 1;
    return slabs;
}

int launch_vtc(gelo_ctx* ctx, const float* V, int ldv, int kv, const float* C, int ldc, int nr, int nc,
               const float* T, bool transpose_t, float* Wp, float* W, int ldw, cudaStream_t st)
{
    if (nr <= 0 || nc <= 0) return GELO_OK;
    const int slabs = panel_slab_count(ctx, nr, nc);
    if ((reinterpret_cast<uintptr_t>(V) & 15u) || (reinterpret_cast<uintptr_t>(C) & 15u) || (ldv & 3) || (ldc & 3))
        return GELO_ERR_INVALID;                  // the 16-byte asynchronous copies need aligned rows
    static bool attr_done[64] = {};
    if (ctx->device >= 0 && ctx->device < 64 && !attr_done[ctx->device]) {
        GELO_CUDA_OK(cudaFuncSetAttribute(vtc_partial_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kVtcSmemBytes));
        attr_done[ctx->device] = true;
    }
    const int rows_per_slab = ceil_div(ceil_div(nr, slabs), kVtcRows) * kVtcRows;
    const int used_slabs = ceil_div(nr, rows_per_slab);
    dim3 g1(ceil_div(nc, 128), used_slabs);
    {
    ProfScope ps(ctx, PROF_VTC, 4.0 * nr * (double)(nc + kv) + 4.0 * NB * (double)nc * used_slabs, st);
    vtc_partial_kernel<<<g1, 256, kVtcSmemBytes, st>>>(V, ldv, kv, C, ldc, nr, nc, rows_per_slab, Wp, ldw);
    }
    GELO_TRY(after_launch(ctx));
    w_reduce_kernel<<<ceil_div(nc, 32), 256, 0, st>>>(Wp, ldw, used_slabs, nc, T, transpose_t ? 1 : 0, W);
    return after_launch(ctx);
}

int launch_rank_update(gelo_ctx* ctx, const float* A, int lda, const float* B, int ldb, float* C, int ldc,
                       int M, int N, int K, cudaStream_t st)
{
    if (M <= 0 || N <= 0 || K <= 0) return GELO_OK;
    if (K > NB) return GELO_ERR_INVALID;
    dim3 grid(ceil_div(N, 128), ceil_div(M, 128));
    {
        // algorithmic bytes: C read and written once, A and B read once
        ProfScope ps(ctx, PROF_RANK_UPDATE, 8.0 * M * (double)N + 4.0 * K * (double)(M + N), st);
        rank_update_kernel<<<grid, 256, 0, st>>>(A, lda, B, ldb, C, ldc, M, N, K);
    }
    return after_launch(ctx);
}

}  // namespace gelo
