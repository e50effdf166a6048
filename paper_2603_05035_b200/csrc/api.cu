// C-ABI entry points of the GELO offload library (see include/gelo.h): argument
// validation, workspace carving and the launch sequences.  No entry point except
// gelo_create / gelo_destroy allocates device memory.
#include <new>

#include "common.cuh"
#include <algorithm>
#include <utility>
#include <vector>

using namespace gelo;

namespace {

inline cudaStream_t as_stream(void* s) { return static_cast<cudaStream_t>(s); }
inline int round_up(int x, int to) { return (x + to - 1) / to * to; }
constexpr int kTcMinRows = 256;   // below this the factorisations are latency-bound anyway

// How a factorisation of an m x m sample stored as `dtype` runs its level-3 updates: 0 = fp32 FMA kernels,
// 2 = tensor cores with three bf16 products of split operands, 3 = tensor cores with one tf32 product.
// By default bf16 calls run the QR on tf32: its errors only perturb the orthogonality of a matrix that is rounded to
// bf16 (8 significant bits against tf32's 11) right afterwards, and its trailing matrix is itself an operand, which
// the split products would have to convert block after block.  The LU keeps the split products: the two triangular
// solves behind A^-1 amplify update errors by the conditioning of L and U, and its operands are thin panels only.
inline int level3_kind(const gelo_ctx* ctx, int m, int dtype, bool qr)
{
    if (ctx->level3 == 1) return 0;
    if (ctx->level3 == 2 || ctx->level3 == 3) return m > gelo::kPanel ? ctx->level3 : 0;
    if (dtype == GELO_F32 || m < kTcMinRows) return 0;
    return qr ? 3 : 2;
}

// Every scratch buffer of one call with sizes (n, k, d, p, dtype); carved in a fixed order so
// that gelo_workspace_bytes and the calls agree.
struct Layout {
    int m = 0, ldi = 0;
    float* G = nullptr;       // m x ldi  Gaussian, then R
    float* Qraw = nullptr;    // m x ldi
    float* A32 = nullptr;     // m x ldi
    float* X32 = nullptr;     // m x ldi
    QrScratch qr;
    LuScratch lu;
    CondScratch cond;
    TcScratch tc;
    ShieldScratch sh;
    float* cond_val = nullptr;
    void* A = nullptr;        // m x ldi, path dtype
    void* Ainv = nullptr;
    void* S = nullptr;        // k x d
    void* U = nullptr;        // m x d
    void* Yp = nullptr;       // m x p
    void* Hd = nullptr;       // n x d   staging of the host variants
    void* Yd = nullptr;       // n x p
    void* Hd2 = nullptr;      // second pair: the batched host variant alternates between the two
    void* Yd2 = nullptr;
    Tf32x3Scratch t3;         // fp32 path: tf32 (hi, lo) copies of the operands of the three products
};

Layout carve(Arena& a, int n, int k, int d, int p, int dtype, bool host_staging)
{
    Layout L;
    const size_t es = elem_size(dtype);
    L.m = n + k;
    L.ldi = gelo_mixing_ld(L.m);
    const size_t mat = (size_t)L.m * L.ldi;
    L.G = static_cast<float*>(a.take(mat * 4));
    L.Qraw = static_cast<float*>(a.take(mat * 4));
    L.A32 = static_cast<float*>(a.take(mat * 4));
    L.X32 = static_cast<float*>(a.take(mat * 4));
    // Buffers that are never alive together share memory:
    //   * while a QR runs, A32 and X32 are idle (they receive the signed Q0 / serve the polish and the LU afterwards):
    //     the QR's split-K planes, its W blocks and the rank-32 partial sums live in A32 (as far as they fit: they need
    //     4096 rows' worth, so this applies from m = 4096 up), the (high, low) pair of the trailing matrix in X32;
    //   * the reflectors V die with the QR and the LU's working copy M is born after it: one matrix.
    char* idle = reinterpret_cast<char*>(L.A32);          // (null in a size query: only the byte count matters then)
    size_t idle_bytes = mat * 4;
    L.qr = carve_qr(a, L.m, L.ldi, &idle, &idle_bytes);
    L.lu = carve_lu(a, L.m, L.ldi);
    L.lu.M = L.qr.V;
    L.lu.Z = L.G;                                          // the Gaussian / R is dead once A32 is formed
    L.cond = carve_cond(a, L.m);
    L.tc = carve_tc(a, L.m, L.ldi, &idle, &idle_bytes);
    for (int h = 0; h < 2; ++h)                            // 2 x (m x ld) 16-bit values: exactly the fp32 matrix X32
        L.tc.big[h] = L.X32 ? reinterpret_cast<char*>(L.X32) + (size_t)h * mat * 2 : nullptr;
    if (!a.base) { L.qr.Wp = nullptr; L.tc.wf32 = nullptr; L.tc.w32[0] = L.tc.w32[1] = nullptr; }
    L.sh = carve_shield(a, n);
    L.cond_val = static_cast<float*>(a.take(16));
    L.A = a.take(mat * es);
    L.Ainv = a.take(mat * es);
    L.S = a.take((size_t)(k > 0 ? k : 1) * d * es);
    L.U = a.take((size_t)L.m * d * es);
    L.Yp = a.take((size_t)L.m * p * es);
    if (dtype == GELO_F32 && d > 0 && p > 0) {
        const size_t wide = (size_t)(L.m > d ? L.m : d);
        L.t3.a_elems = (size_t)L.m * round_up((int)wide, 4);
        L.t3.b_elems = wide * round_up(p > d ? p : d, 32);
        for (int h = 0; h < 2; ++h) {
            L.t3.a[h] = static_cast<float*>(a.take(L.t3.a_elems * 4));
            L.t3.b[h] = static_cast<float*>(a.take(L.t3.b_elems * 4));
        }
        L.t3.c_elems = (size_t)L.m * (p > d ? p : d);
        L.t3.planes = static_cast<float*>(a.take(L.t3.c_elems * kTf32x3Slices * 4));
    }
    if (host_staging) {
        L.Hd = a.take((size_t)n * d * es);
        L.Yd = a.take((size_t)n * p * es);
        L.Hd2 = a.take((size_t)n * d * es);
        L.Yd2 = a.take((size_t)n * p * es);
    }
    return L;
}

// Lanes other than the first hold only what sampling needs, except for small batches (m <= 128), whose lanes also
// form their own shield rows and mixed matrix: those get an S and a U of their own (d columns wide).
inline int lane_width(int n, int k, int d) { return (n + k <= 128) ? d : 0; }

bool carve_ctx(gelo_ctx* ctx, int n, int k, int d, int p, int dtype, bool host_staging, Layout* out)
{
    if (!ctx->ws) return false;
    ctx->chain_valid = false;      // a single call reuses scratch that a later batch must not race with
    Arena a;
    a.base = static_cast<char*>(ctx->ws);
    a.cap = ctx->ws_bytes;
    *out = carve(a, n, k, d, p, dtype, host_staging);
    return a.ok;
}

bool bad_dtype(int t) { return t != GELO_F32 && t != GELO_BF16 && t != GELO_F16; }
bool bad_ld(int lda, int m) { return lda < m || (lda % 8) != 0; }
bool misaligned(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) != 0; }

struct DeviceGuard {
    int prev = -1;
    bool ok = true;
    explicit DeviceGuard(int dev) {
        if (cudaGetDevice(&prev) != cudaSuccess) { ok = false; return; }
        if (prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
    }
    ~DeviceGuard() { if (prev >= 0) cudaSetDevice(prev); }
};

__global__ void set_scalar_kernel(float* p, float v) { *p = v; }

int gemm_dispatch(gelo_ctx* ctx, const GemmArgs& g, cudaStream_t st)
{
    if (g.dtype != GELO_F32 && gemm_tc_supports(g)) return launch_gemm_tc(ctx, g, st);
    return launch_gemm_simt(ctx, g, st);
}

// A (and A^-1) for one attempt into L.A32 / L.X32 or straight into the outputs.
int sample_attempt(gelo_ctx* ctx, const Layout& L, int m, int kind, uint64_t seed, uint32_t attempt,
                   int dtype, void* A_out, void* Ainv_out, int lda, float* cond_dev, cudaStream_t st,
                   bool deferred = false, const uint64_t* seed_dev = nullptr)
{
    const int ldi = L.ldi;
    GELO_TRY(launch_gaussian(ctx, m, m, ldi, seed, GELO_STREAM_G0, attempt, 1.0f, nullptr, L.G, st, seed_dev));
    const int l3 = level3_kind(ctx, m, dtype, true);
    if (l3 == 3) GELO_TRY(run_householder_qr_tf32(ctx, m, L.G, ldi, L.Qraw, L.qr, L.tc, st));
    else if (l3) GELO_TRY(run_householder_qr_tc(ctx, m, L.G, ldi, L.Qraw, L.qr, L.tc, st));
    else GELO_TRY(run_householder_qr(ctx, m, L.G, ldi, L.Qraw, L.qr, st));
    if (kind == GELO_ORTHOGONAL) {
        // tf32 updates: polish Q (A32 and X32 are free for this kind).  The non-orthogonal kind skips it: there Q0 only
        // has to keep A = Q0 + gamma G1 well conditioned, and A^-1 comes from the LU of the stored A.
        if (l3 == 3) GELO_TRY(polish_orthogonal_tf32(ctx, m, L.Qraw, ldi, L.X32, L.A32, st));
        GELO_TRY(launch_finish_mixing(ctx, m, L.Qraw, ldi, L.G, ldi, dtype, A_out, Ainv_out, lda, st));
        if (cond_dev) {
            set_scalar_kernel<<<1, 1, 0, st>>>(cond_dev, 1.0f);
            GELO_TRY(after_launch(ctx));
        }
        return GELO_OK;
    }
    // Q0 (signed, fp32) -> A = Q0 + gamma / sqrt(m) * G1 -> stored type -> inverse of the stored A
    GELO_TRY(launch_finish_mixing(ctx, m, L.Qraw, ldi, L.G, ldi, GELO_F32, L.A32, nullptr, ldi, st));
    const float s = ctx->gamma / sqrtf((float)m);
    GELO_TRY(launch_gaussian(ctx, m, m, ldi, seed, GELO_STREAM_G1, attempt, s, L.A32, L.A32, st, seed_dev));
    // the inverse is that of the stored A: round, and carry on from the rounded values
    GELO_TRY(launch_narrow(ctx, m, L.A32, ldi, dtype, A_out, lda, st, dtype != GELO_F32 ? L.A32 : nullptr, ldi));
    // tensor-core updates serve the bf16 path; the fp32 path stays exact
    const int l3lu = level3_kind(ctx, m, dtype, false);
    if (l3lu) GELO_TRY(run_lu_inverse_tc(ctx, m, L.A32, ldi, L.X32, L.lu, L.tc, l3lu == 3, st));
    else GELO_TRY(run_lu_inverse(ctx, m, L.A32, ldi, L.X32, L.lu, st));
    GELO_TRY(launch_narrow(ctx, m, L.X32, ldi, dtype, Ainv_out, lda, st));
    // the verified matrices are the stored ones: what mix and unmix will read
    return run_cond_estimate(ctx, m, A_out, Ainv_out, lda, dtype, ctx->cond_bound, cond_dev ? cond_dev : L.cond_val, L.cond,
                             st, deferred);
}

int sample_mixing_impl(gelo_ctx* ctx, const Layout& L, int m, int kind, uint64_t seed, int dtype,
                       void* A_out, void* Ainv_out, int lda, float* cond_dev, cudaStream_t st)
{
    if (kind == GELO_ORTHOGONAL)
        return sample_attempt(ctx, L, m, kind, seed, 0u, dtype, A_out, Ainv_out, lda, cond_dev, st);
    for (int attempt = 0; attempt < ctx->max_attempts; ++attempt) {
        GELO_TRY(sample_attempt(ctx, L, m, kind, seed, (uint32_t)attempt, dtype, A_out, Ainv_out, lda, cond_dev, st));
        GELO_CUDA_OK(cudaMemcpyAsync(ctx->status_host, ctx->status_dev, kStatusWords * sizeof(int),
                                     cudaMemcpyDeviceToHost, st));
        GELO_CUDA_OK(cudaStreamSynchronize(st));
        if (ctx->status_host[1] == 1) return GELO_OK;
    }
    return GELO_ERR_COND;
}

// A product of the offload.  Large fp32 products run on the tensor cores as three tf32 products of (hi, lo) operand
// pairs when the call has scratch for the pairs (error about 1e-6, inside the fp32 path's 1e-4); everything else goes
// to the bf16 / half tensor-core kernel or the FFMA kernel.
int product(gelo_ctx* ctx, const GemmArgs& g, const Tf32x3Scratch* t3, cudaStream_t st)
{
    const int lda3 = round_up(g.K, 4), ldb3 = round_up(g.N, 32);
    if (g.dtype == GELO_F32 && t3 && t3->a[0] && !g.B2 && !g.transA && !g.transB && g.M >= 128 &&
        2.0 * g.M * (double)g.N * g.K >= 1e9 && (g.lda % 4) == 0 && (g.ldb % 4) == 0 && (g.ldc % 4) == 0 && (g.K % 4) == 0 &&
        (g.N % 4) == 0 && (g.N % g.nsplit) == 0 && ((g.N / g.nsplit) % 8) == 0 && !misaligned(g.A) && !misaligned(g.B) &&
        (size_t)g.M * lda3 <= t3->a_elems && (size_t)g.K * ldb3 <= t3->b_elems) {
        GELO_TRY(launch_split_tf32(ctx, static_cast<const float*>(g.A), g.lda, g.M, g.K, t3->a[0], t3->a[1], lda3, st));
        GELO_TRY(launch_split_tf32(ctx, static_cast<const float*>(g.B), g.ldb, g.K, g.N, t3->b[0], t3->b[1], ldb3, st));
        float* const C[3] = { static_cast<float*>(g.C[0]), static_cast<float*>(g.C[1]), static_cast<float*>(g.C[2]) };
        float* planes = (size_t)g.M * g.N <= t3->c_elems ? t3->planes : nullptr;
        return launch_gemm_tf32x3(ctx, g.M, g.N, g.K, t3->a[0], t3->a[1], lda3, t3->b[0], t3->b[1], ldb3, C, g.ldc, g.nsplit,
                                  planes, st);
    }
    return gemm_dispatch(ctx, g, st);
}

int mix_impl(gelo_ctx* ctx, const void* A, int lda, const void* H, const void* S, int n, int k, int d,
             int dtype, void* U, cudaStream_t st, const Tf32x3Scratch* t3 = nullptr)
{
    if (ctx->fuse_small && mix_small_supports(n, k, d, dtype) && !misaligned(H) && !misaligned(S) && !misaligned(U))
        return launch_mix_small(ctx, A, lda, H, S, n, k, d, dtype, U, st);
    GemmArgs g;
    g.M = n + k; g.N = d; g.K = n + k;
    g.A = A; g.lda = lda;
    g.B = H; g.ldb = d;
    if (k > 0) { g.B2 = S; g.b_split = n; }
    g.C[0] = U; g.ldc = d; g.dtype = dtype;
    return product(ctx, g, t3, st);
}

int project_impl(gelo_ctx* ctx, const void* U, const void* W, int m, int d, int p, int dtype, void* Yp,
                 cudaStream_t st, const Tf32x3Scratch* t3 = nullptr)
{
    // a product with few rows is a stream of W: the kernel of the small-batch path, without its unmixing half
    if (ctx->fuse_small && project_unmix_supports(ctx, m, 0, d, p, dtype, (m + 7) & ~7, 1) && !misaligned(U) && !misaligned(Yp))
        return launch_project_unmix(ctx, U, W, nullptr, 0, m, 0, d, p, dtype, Yp, nullptr, nullptr, st);
    GemmArgs g;
    g.M = m; g.N = p; g.K = d;
    g.A = U; g.lda = d; g.B = W; g.ldb = p;
    g.C[0] = Yp; g.ldc = p; g.dtype = dtype;
    return product(ctx, g, t3, st);
}

int unmix_impl(gelo_ctx* ctx, const void* Ainv, int lda, const void* Yp, int n, int k, int p, int dtype,
               void* Q, void* K, void* V, cudaStream_t st, const Tf32x3Scratch* t3 = nullptr)
{
    GemmArgs g;
    g.M = n; g.N = p; g.K = n + k;
    g.A = Ainv; g.lda = lda; g.B = Yp; g.ldb = p;
    g.dtype = dtype;
    if (K || V) { g.nsplit = 3; g.C[0] = Q; g.C[1] = K; g.C[2] = V; g.ldc = p / 3; }
    else { g.nsplit = 1; g.C[0] = Q; g.ldc = p; }
    return product(ctx, g, t3, st);
}

// The single-stage entry points have no scratch of their own; when the context holds a workspace with room for the
// operand pairs, their large fp32 products run on the tensor cores exactly as inside the whole call (so that a plain
// H W through gelo_project is timed on the same kernel as the obfuscated chain).  Without one they stay on the FMA kernel.
const Tf32x3Scratch* stage_pairs(gelo_ctx* ctx, int rows, int k, int d, int p, int dtype, Layout* L)
{
    if (dtype != GELO_F32 || !ctx->ws) return nullptr;
    return carve_ctx(ctx, rows, k, d, p, dtype, false, L) ? &L->t3 : nullptr;
}

// Eq. 2 and Eq. 3 of one call: one fused launch for a small batch (the weight is streamed once and Y' stays on chip),
// otherwise the two products with Y' in workspace memory.
int project_and_unmix(gelo_ctx* ctx, const void* U, const void* W, const void* Ainv, int lda, void* Yp, int n, int k, int d,
                      int p, int dtype, void* Q, void* K, void* V, cudaStream_t st, const Tf32x3Scratch* t3)
{
    if (ctx->fuse_small && project_unmix_supports(ctx, n, k, d, p, dtype, lda, (K || V) ? 3 : 1))
        return launch_project_unmix(ctx, U, W, Ainv, lda, n, k, d, p, dtype, Q, K, V, st);
    GELO_TRY(project_impl(ctx, U, W, n + k, d, p, dtype, Yp, st, t3));
    return unmix_impl(ctx, Ainv, lda, Yp, n, k, p, dtype, Q, K, V, st, t3);
}

int check_split(int p, const void* Q, const void* K, const void* V)
{
    if (!Q) return GELO_ERR_INVALID;
    if ((K == nullptr) != (V == nullptr)) return GELO_ERR_INVALID;
    if (K && (p % 3 != 0 || (p / 3) % 8 != 0)) return GELO_ERR_UNSUPPORTED;
    return GELO_OK;
}

int offload_impl(gelo_ctx* ctx, const Layout& L, const void* H, const void* W, int n, int k, int d, int p,
                 int kind, uint64_t seed, float shield_scale, int dtype, void* Q, void* K, void* V,
                 cudaStream_t st)
{
    const int m = n + k;
    GELO_TRY(sample_mixing_impl(ctx, L, m, kind, seed, dtype, L.A, L.Ainv, L.ldi, nullptr, st));
    GELO_TRY(run_shield_rows(ctx, H, n, d, k, shield_scale, seed, dtype, L.S, L.sh, st, ctx->shield_nu));
    GELO_TRY(mix_impl(ctx, L.A, L.ldi, H, k > 0 ? L.S : nullptr, n, k, d, dtype, L.U, st, &L.t3));
    return project_and_unmix(ctx, L.U, W, L.Ainv, L.ldi, L.Yp, n, k, d, p, dtype, Q, K, V, st, &L.t3);
}


__global__ void set_seed_kernel(uint64_t* slot, uint64_t seed) { *slot = seed; }

void drop_graphs(gelo_ctx* ctx)
{
    for (auto& g : ctx->graphs) cudaGraphExecDestroy(g.exec);
    ctx->graphs.clear();
}

// Samples (A, A^-1) of one batched call on a lane stream by replaying a launch graph of the whole sampling
// sequence (about a thousand dependent launches): one host call instead of a thousand, so a single host thread
// keeps all lanes busy.  The seed reaches the kernels through the lane's device slot.  The first use of a
// (lane scratch, kind, size, type) combination records the graph by stream capture.
int sample_on_lane(gelo_ctx* ctx, const Layout& L, int lane, int m, int kind, uint64_t seed, int dtype, cudaStream_t ls)
{
    uint64_t* slot = ctx->lane_seed_dev + lane * 8;
    set_seed_kernel<<<1, 1, 0, ls>>>(slot, seed);
    GELO_TRY(after_launch(ctx));
    if (ctx->prof_on)      // per-launch timing needs real launches
        return sample_attempt(ctx, L, m, kind, seed, 0u, dtype, L.A, L.Ainv, L.ldi, nullptr, ls, true, slot);
    for (auto& g : ctx->graphs) {
        if (g.key_ptr == L.G && g.m == m && g.kind == kind && g.dtype == dtype && g.level3 == ctx->level3 &&
            g.tc_ctas == ctx->tc_update_ctas) {
            GELO_CUDA_OK(cudaGraphLaunch(g.exec, ls));
            ctx->launches += g.launches;
            return GELO_OK;
        }
    }
    const long long before = ctx->launches;
    GELO_CUDA_OK(cudaStreamBeginCapture(ls, cudaStreamCaptureModeRelaxed));
    const int rc = sample_attempt(ctx, L, m, kind, seed, 0u, dtype, L.A, L.Ainv, L.ldi, nullptr, ls, true, slot);
    cudaGraph_t graph = nullptr;
    const cudaError_t ce = cudaStreamEndCapture(ls, &graph);
    if (rc != GELO_OK || ce != cudaSuccess || !graph) {
        if (graph) cudaGraphDestroy(graph);
        return rc != GELO_OK ? rc : GELO_ERR_CUDA;
    }
    gelo_ctx::SampleGraph g;
    g.key_ptr = L.G; g.m = m; g.kind = kind; g.dtype = dtype; g.level3 = ctx->level3; g.tc_ctas = ctx->tc_update_ctas;
    g.launches = ctx->launches - before;
    g.exec = nullptr;
    const cudaError_t ie = cudaGraphInstantiate(&g.exec, graph, 0);
    cudaGraphDestroy(graph);
    if (ie != cudaSuccess) return GELO_ERR_CUDA;
    ctx->graphs.push_back(g);
    GELO_CUDA_OK(cudaGraphLaunch(g.exec, ls));
    return GELO_OK;
}

// The whole path for a batch of independent calls.  Sampling A depends only on the seed, so up to
// `lanes` calls sample their mixing pairs concurrently on the context's lane streams (each with its
// own scratch) while the main stream runs shields and the three products of earlier calls.
//   lane stream:  [wait lane_free] sample A_i, A_i^-1 -> record lane_ready
//   main stream:  shield rows_i -> [wait lane_ready] mix, project, unmix -> record lane_free
// Non-orthogonal samples use the first attempt only; a missed condition bound is reported through
// the status word (GELO_ERR_COND) instead of a resample, because nothing here waits for the device.
int offload_batch_impl(gelo_ctx* ctx, int calls, const void* const* H, const void* const* W, int n, int k, int d,
                       int p, const int* kinds, const uint64_t* seeds, float shield_scale, int dtype,
                       void* const* Q, void* const* K, void* const* V, cudaStream_t st, bool host, bool wait = true)
{
    const int m = n + k;
    const int D = calls < ctx->lanes ? calls : ctx->lanes;
    if (!ctx->ws) return GELO_ERR_WORKSPACE;
    Arena a;
    a.base = static_cast<char*>(ctx->ws);
    a.cap = ctx->ws_bytes;
    Layout L[kMaxLanes];
    L[0] = carve(a, n, k, d, p, dtype, host);
    for (int i = 1; i < D; ++i) L[i] = carve(a, n, k, lane_width(n, k, d), 0, dtype, false);
    if (!a.ok) return GELO_ERR_WORKSPACE;
    const size_t es = elem_size(dtype);
    const bool split = K[0] != nullptr;
    const size_t third = (size_t)n * (p / 3) * es;
    // A small batch (the decode shape) is a stream of W per call and little else; its other launches are short and
    // latency-bound.  There the WHOLE call runs on its lane (sampling, shield rows, mixing, fused projection + unmixing,
    // on the lane's own S and U): the weight streams of different calls overlap at their seams and the caller's stream
    // only joins the lanes at the end of the batch.
    bool small = !host && D > 1 && ctx->fuse_small && lane_width(n, k, d) > 0 && mix_small_supports(n, k, d, dtype) &&
                 project_unmix_supports(ctx, n, k, d, p, dtype, L[0].ldi, split ? 3 : 1);
    for (int i = 0; i < calls && small; ++i) small = !misaligned(H[i]);
    if (small) {
        // calls that share an output buffer are promised call order: keep those on the caller's stream
        std::vector<std::pair<uintptr_t, uintptr_t>> out;
        out.reserve((size_t)calls * 3);
        const size_t bytes = split ? third : (size_t)n * p * es;
        for (int i = 0; i < calls; ++i) {
            out.emplace_back(reinterpret_cast<uintptr_t>(Q[i]), reinterpret_cast<uintptr_t>(Q[i]) + bytes);
            if (split) {
                out.emplace_back(reinterpret_cast<uintptr_t>(K[i]), reinterpret_cast<uintptr_t>(K[i]) + bytes);
                out.emplace_back(reinterpret_cast<uintptr_t>(V[i]), reinterpret_cast<uintptr_t>(V[i]) + bytes);
            }
        }
        std::sort(out.begin(), out.end());
        for (size_t i = 1; i < out.size() && small; ++i) small = out[i].first >= out[i - 1].second;
    }
    // with several lanes in flight each level-3 update takes a share of the SMs (ctx->lane_tc_share-th of them)
    ctx->tc_update_ctas = (D >= ctx->lane_tc_share && ctx->lane_tc_share > 1) ? ctx->sm_count / ctx->lane_tc_share : 0;

    // Back-to-back batches of the same shape on the same stream keep the lanes running across the seam: each
    // lane only waits until the products that read its previous pair are done.  Otherwise the lanes start after
    // everything already enqueued on the caller's stream.
    const int shape[6] = { n, k, d, p, dtype, (host ? 1 : 0) | (small ? 2 : 0) };
    bool same_shape = true;
    for (int i = 0; i < 6; ++i) same_shape = same_shape && ctx->chain_shape[i] == shape[i];
    const bool chained = ctx->chain_valid && ctx->chain_stream == st && ctx->chain_key == L[D - 1].G &&
                         ctx->chain_lanes == D && same_shape;
    if (!chained) {
        // a fresh start: the lanes AND the two copy streams begin after everything already on the caller's stream
        // (an earlier call of another shape may still be using the regions that this batch stages into)
        GELO_CUDA_OK(cudaEventRecord(ctx->batch_start, st));
        for (int l = 0; l < D; ++l) GELO_CUDA_OK(cudaStreamWaitEvent(ctx->lane_stream[l], ctx->batch_start, 0));
        if (host) {
            GELO_CUDA_OK(cudaStreamWaitEvent(ctx->copy_in, ctx->batch_start, 0));
            GELO_CUDA_OK(cudaStreamWaitEvent(ctx->copy_out, ctx->batch_start, 0));
        }
    }

    if (small) {
        // the lanes read H_i and write Q_i, K_i, V_i: not before this point of the caller's stream (a lane that runs on
        // from the previous batch may sample ahead of it)
        if (chained) GELO_CUDA_OK(cudaEventRecord(ctx->batch_start, st));
        for (int i = 0; i < calls; ++i) {
            const int l = i % D;
            cudaStream_t ls = ctx->lane_stream[l];
            GELO_TRY(sample_on_lane(ctx, L[l], l, m, kinds[i], seeds[i], dtype, ls));
            if (chained && i < D) GELO_CUDA_OK(cudaStreamWaitEvent(ls, ctx->batch_start, 0));
            GELO_TRY(run_shield_rows(ctx, H[i], n, d, k, shield_scale, seeds[i], dtype, L[l].S, L[l].sh, ls, ctx->shield_nu));
            GELO_TRY(mix_impl(ctx, L[l].A, L[l].ldi, H[i], k > 0 ? L[l].S : nullptr, n, k, d, dtype, L[l].U, ls, nullptr));
            GELO_TRY(project_and_unmix(ctx, L[l].U, W[i], L[l].Ainv, L[l].ldi, nullptr, n, k, d, p, dtype, Q[i],
                                       split ? K[i] : nullptr, split ? V[i] : nullptr, ls, nullptr));
        }
        for (int l = 0; l < D; ++l) {
            GELO_CUDA_OK(cudaEventRecord(ctx->lane_ready[l], ctx->lane_stream[l]));
            GELO_CUDA_OK(cudaStreamWaitEvent(st, ctx->lane_ready[l], 0));
        }
        for (int l = 0; l < D; ++l) GELO_CUDA_OK(cudaEventRecord(ctx->lane_free[l], st));
    }

    auto enqueue_sample = [&](int i) -> int {
        const int l = i % D;
        cudaStream_t ls = ctx->lane_stream[l];
        if (i >= D || chained) GELO_CUDA_OK(cudaStreamWaitEvent(ls, ctx->lane_free[l], 0));
        GELO_TRY(sample_on_lane(ctx, L[l], l, m, kinds[i], seeds[i], dtype, ls));
        GELO_CUDA_OK(cudaEventRecord(ctx->lane_ready[l], ls));
        return GELO_OK;
    };

    for (int i = 0; i < D && !small; ++i) GELO_TRY(enqueue_sample(i));
    // Host variant: activations come in on the context's copy-in stream and results leave on its copy-out stream,
    // through two staging pairs used alternately, so that the copies of call i overlap the products of calls i-1 and
    // i+1 (the two directions use different copy engines):
    //   copy-in :  [wait h_free_b]  H_i -> Hd_b                      -> record h_ready_b
    //   stream  :  [wait h_ready_b] shields  [wait lane_ready, y_free_b]  mix, project, unmix -> Yd_b
    //                                                                  -> record h_free_b, y_ready_b, lane_free
    //   copy-out:  [wait y_ready_b] Yd_b -> Q_i, K_i, V_i              -> record y_free_b
    // and at the end the caller's stream waits for the last copies out.
    for (int i = 0; i < calls && !small; ++i) {
        const int l = i % D;
        const int b = i & 1;
        const void* Hi = H[i];
        char* y = static_cast<char*>(b ? L[0].Yd2 : L[0].Yd);
        void *Qi = Q[i], *Ki = split ? K[i] : nullptr, *Vi = split ? V[i] : nullptr;
        if (host) {
            void* hd = b ? L[0].Hd2 : L[0].Hd;
            GELO_CUDA_OK(cudaStreamWaitEvent(ctx->copy_in, ctx->h_free[b], 0));
            GELO_CUDA_OK(cudaMemcpyAsync(hd, H[i], (size_t)n * d * es, cudaMemcpyHostToDevice, ctx->copy_in));
            GELO_CUDA_OK(cudaEventRecord(ctx->h_ready[b], ctx->copy_in));
            GELO_CUDA_OK(cudaStreamWaitEvent(st, ctx->h_ready[b], 0));
            Hi = hd;
            Qi = y; Ki = split ? y + third : nullptr; Vi = split ? y + 2 * third : nullptr;
        }
        GELO_TRY(run_shield_rows(ctx, Hi, n, d, k, shield_scale, seeds[i], dtype, L[0].S, L[0].sh, st, ctx->shield_nu));
        GELO_CUDA_OK(cudaStreamWaitEvent(st, ctx->lane_ready[l], 0));
        if (host) GELO_CUDA_OK(cudaStreamWaitEvent(st, ctx->y_free[b], 0));
        GELO_TRY(mix_impl(ctx, L[l].A, L[l].ldi, Hi, k > 0 ? L[0].S : nullptr, n, k, d, dtype, L[0].U, st, &L[0].t3));
        GELO_TRY(project_and_unmix(ctx, L[0].U, W[i], L[l].Ainv, L[l].ldi, L[0].Yp, n, k, d, p, dtype, Qi, Ki, Vi, st, &L[0].t3));
        GELO_CUDA_OK(cudaEventRecord(ctx->lane_free[l], st));
        if (host) {
            GELO_CUDA_OK(cudaEventRecord(ctx->h_free[b], st));
            GELO_CUDA_OK(cudaEventRecord(ctx->y_ready[b], st));
            GELO_CUDA_OK(cudaStreamWaitEvent(ctx->copy_out, ctx->y_ready[b], 0));
            if (split) {
                GELO_CUDA_OK(cudaMemcpyAsync(Q[i], y, third, cudaMemcpyDeviceToHost, ctx->copy_out));
                GELO_CUDA_OK(cudaMemcpyAsync(K[i], y + third, third, cudaMemcpyDeviceToHost, ctx->copy_out));
                GELO_CUDA_OK(cudaMemcpyAsync(V[i], y + 2 * third, third, cudaMemcpyDeviceToHost, ctx->copy_out));
            } else {
                GELO_CUDA_OK(cudaMemcpyAsync(Q[i], y, (size_t)n * p * es, cudaMemcpyDeviceToHost, ctx->copy_out));
            }
            GELO_CUDA_OK(cudaEventRecord(ctx->y_free[b], ctx->copy_out));
        }
        if (i + D < calls) GELO_TRY(enqueue_sample(i + D));
    }
    if (host) {
        GELO_CUDA_OK(cudaStreamWaitEvent(st, ctx->y_free[0], 0));
        GELO_CUDA_OK(cudaStreamWaitEvent(st, ctx->y_free[1], 0));
    }
    ctx->tc_update_ctas = 0;
    ctx->chain_valid = calls >= D && !ctx->prof_on;
    ctx->chain_stream = st;
    ctx->chain_key = L[D - 1].G;
    ctx->chain_lanes = D;
    for (int i = 0; i < 6; ++i) ctx->chain_shape[i] = shape[i];
    if (host && wait) GELO_CUDA_OK(cudaStreamSynchronize(st));
    return GELO_OK;
}

// ---- block-diagonal orthogonal mixing (a structured variant; the paper names structured orthogonal transforms as
//      future work) -------------------------------------------------------------------------------------------------
//
// The m = n + k mixed rows are dealt into nb = ceil(m / block) groups; group j takes the data rows
// [n j / nb, n (j+1) / nb) and the shield rows [k j / nb, k (j+1) / nb), so every group mixes its share of shield rows
// with its data rows.  Each group gets its own Haar-orthogonal A_j (Householder QR of a Gaussian, sampled on a lane of
// its own): U_j = A_j [H_j; S_j], one projection for all of U, Y_j = (A_j^T Y'_j)[data rows].  A-generation costs
// nb (8/3) b^3 instead of (8/3) m^3 and the two mixing products 2 m b (d + p) instead of 2 m^2 (d + p).
struct BlockPlan {
    int nb = 0, bmax = 0;
    int nd[kMaxLanes], ns[kMaxLanes], d0[kMaxLanes], s0[kMaxLanes];
};

bool plan_blocks(int n, int k, int block, BlockPlan* P)
{
    const int m = n + k;
    if (block <= 0 || (block % 64) != 0) return false;
    const int nb = (m + block - 1) / block;
    if (nb < 1 || nb > kMaxLanes || n < nb) return false;
    P->nb = nb; P->bmax = 0;
    for (int j = 0; j < nb; ++j) {
        P->d0[j] = (int)((long long)n * j / nb);
        P->s0[j] = (int)((long long)k * j / nb);
        P->nd[j] = (int)((long long)n * (j + 1) / nb) - P->d0[j];
        P->ns[j] = (int)((long long)k * (j + 1) / nb) - P->s0[j];
        if (P->nd[j] + P->ns[j] > P->bmax) P->bmax = P->nd[j] + P->ns[j];
    }
    return true;
}

size_t blockdiag_workspace(int n, int k, int d, int p, int dtype, int block, int lanes)
{
    BlockPlan P;
    if (!plan_blocks(n, k, block, &P)) return 0;
    Arena a;
    a.cap = ~size_t(0) >> 1;
    carve(a, P.bmax, 0, 0, 0, dtype, false);                  // lane 0 ...
    {   // ... which also carries the buffers of the whole call: S, U, Y'
        const size_t es = elem_size(dtype);
        a.take((size_t)(k > 0 ? k : 1) * d * es); a.take((size_t)(n + k) * d * es); a.take((size_t)(n + k) * p * es);
        carve_shield(a, n);
    }
    for (int i = 1; i < lanes; ++i) carve(a, P.bmax, 0, 0, 0, dtype, false);
    return a.off + 256;
}

int offload_blockdiag_impl(gelo_ctx* ctx, int calls, const void* const* H, const void* const* W, int n, int k, int d, int p,
                           int block, const uint64_t* seeds, float shield_scale, int dtype, void* const* Q, void* const* K,
                           void* const* V, cudaStream_t st)
{
    BlockPlan P;
    if (!plan_blocks(n, k, block, &P)) return GELO_ERR_UNSUPPORTED;
    const int D = ctx->lanes;
    if (P.nb > D) return GELO_ERR_UNSUPPORTED;                // all groups of a call are alive at once: one lane each
    if (!ctx->ws) return GELO_ERR_WORKSPACE;
    const int m = n + k;
    const size_t es = elem_size(dtype);
    Arena a;
    a.base = static_cast<char*>(ctx->ws);
    a.cap = ctx->ws_bytes;
    Layout L[kMaxLanes];
    L[0] = carve(a, P.bmax, 0, 0, 0, dtype, false);
    char* S = static_cast<char*>(a.take((size_t)(k > 0 ? k : 1) * d * es));
    char* U = static_cast<char*>(a.take((size_t)m * d * es));
    char* Yp = static_cast<char*>(a.take((size_t)m * p * es));
    ShieldScratch sh = carve_shield(a, n);
    for (int i = 1; i < D; ++i) L[i] = carve(a, P.bmax, 0, 0, 0, dtype, false);
    if (!a.ok) return GELO_ERR_WORKSPACE;
    const bool split = K[0] != nullptr;
    const int qcols = split ? p / 3 : p;
    ctx->chain_valid = false;                                 // this layout is not the one a later plain batch chains onto
    ctx->tc_update_ctas = (D >= ctx->lane_tc_share && ctx->lane_tc_share > 1) ? ctx->sm_count / ctx->lane_tc_share : 0;
    GELO_CUDA_OK(cudaEventRecord(ctx->batch_start, st));
    for (int l = 0; l < D; ++l) GELO_CUDA_OK(cudaStreamWaitEvent(ctx->lane_stream[l], ctx->batch_start, 0));

    const long long total = (long long)calls * P.nb;
    auto enqueue_sample = [&](long long v) -> int {
        const int l = (int)(v % D), c = (int)(v / P.nb), j = (int)(v % P.nb);
        cudaStream_t ls = ctx->lane_stream[l];
        if (v >= D) GELO_CUDA_OK(cudaStreamWaitEvent(ls, ctx->lane_free[l], 0));
        const uint64_t seed = seeds[c] ^ (0x9E3779B97F4A7C15ull * (uint64_t)(j + 1));     // a fresh A_j per group and call
        GELO_TRY(sample_on_lane(ctx, L[l], l, P.nd[j] + P.ns[j], GELO_ORTHOGONAL, seed, dtype, ls));
        GELO_CUDA_OK(cudaEventRecord(ctx->lane_ready[l], ls));
        return GELO_OK;
    };
    for (long long v = 0; v < total && v < D; ++v) GELO_TRY(enqueue_sample(v));
    for (int c = 0; c < calls; ++c) {
        const char* Hc = static_cast<const char*>(H[c]);
        GELO_TRY(run_shield_rows(ctx, Hc, n, d, k, shield_scale, seeds[c], dtype, S, sh, st, ctx->shield_nu));
        for (int j = 0; j < P.nb; ++j) {
            const int l = (int)(((long long)c * P.nb + j) % D);
            const int u0 = P.d0[j] + P.s0[j];
            GELO_CUDA_OK(cudaStreamWaitEvent(st, ctx->lane_ready[l], 0));
            GELO_TRY(mix_impl(ctx, L[l].A, L[l].ldi, Hc + (size_t)P.d0[j] * d * es, P.ns[j] ? S + (size_t)P.s0[j] * d * es : nullptr,
                              P.nd[j], P.ns[j], d, dtype, U + (size_t)u0 * d * es, st));
        }
        GELO_TRY(project_impl(ctx, U, W[c], m, d, p, dtype, Yp, st));
        for (int j = 0; j < P.nb; ++j) {
            const int l = (int)(((long long)c * P.nb + j) % D);
            const int u0 = P.d0[j] + P.s0[j];
            const size_t qoff = (size_t)P.d0[j] * qcols * es;
            GELO_TRY(unmix_impl(ctx, L[l].Ainv, L[l].ldi, Yp + (size_t)u0 * p * es, P.nd[j], P.ns[j], p, dtype,
                                static_cast<char*>(Q[c]) + qoff, split ? static_cast<char*>(K[c]) + qoff : nullptr,
                                split ? static_cast<char*>(V[c]) + qoff : nullptr, st));
            GELO_CUDA_OK(cudaEventRecord(ctx->lane_free[l], st));
        }
        for (int j = 0; j < P.nb; ++j) {
            const long long v = (long long)c * P.nb + j + D;
            if (v < total) GELO_TRY(enqueue_sample(v));
        }
    }
    ctx->tc_update_ctas = 0;
    return GELO_OK;
}

int check_batch_args(gelo_ctx* ctx, int calls, const void* const* H, const void* const* W, int n, int k, int d, int p,
                     const int* kinds, const uint64_t* seeds, int dtype, void* const* Q, void* const* K,
                     void* const* V, bool host)
{
    if (!ctx || calls < 0 || n <= 0 || k < 0 || d <= 0 || p <= 0 || (d % 8) != 0 || (p % 8) != 0 || bad_dtype(dtype))
        return GELO_ERR_INVALID;
    if (calls == 0) return GELO_OK;
    if (!H || !W || !kinds || !seeds || !Q || !K || !V) return GELO_ERR_INVALID;
    const bool split = K[0] != nullptr;
    for (int i = 0; i < calls; ++i) {
        if (!H[i] || !W[i] || misaligned(W[i]) || (kinds[i] != GELO_ORTHOGONAL && kinds[i] != GELO_NONORTHOGONAL))
            return GELO_ERR_INVALID;
        if ((K[i] != nullptr) != split) return GELO_ERR_INVALID;
        if (!host && (misaligned(H[i]) || misaligned(Q[i]) || misaligned(K[i]) || misaligned(V[i])))
            return GELO_ERR_INVALID;
        GELO_TRY(check_split(p, Q[i], K[i], V[i]));
    }
    return GELO_OK;
}

size_t batch_workspace(int n, int k, int d, int p, int dtype, int lanes)
{
    Arena a;
    a.cap = ~size_t(0) >> 1;
    carve(a, n, k, d, p, dtype, true);
    for (int i = 1; i < lanes; ++i) carve(a, n, k, lane_width(n, k, d), 0, dtype, false);
    return a.off + 256;
}

}  // namespace

extern "C" {

int gelo_create(gelo_ctx** out, int device)
{
    if (!out) return GELO_ERR_INVALID;
    *out = nullptr;
    int count = 0;
    if (cudaGetDeviceCount(&count) != cudaSuccess) return GELO_ERR_CUDA;
    if (device < 0 || device >= count) return GELO_ERR_INVALID;
    cudaDeviceProp prop;
    GELO_CUDA_OK(cudaGetDeviceProperties(&prop, device));
    if (prop.major != 10) return GELO_ERR_UNSUPPORTED;
    DeviceGuard guard(device);
    if (!guard.ok) return GELO_ERR_CUDA;
    gelo_ctx* ctx = new (std::nothrow) gelo_ctx();
    if (!ctx) return GELO_ERR_CUDA;
    ctx->device = device;
    ctx->sm_count = prop.multiProcessorCount;
    if (cudaMalloc(&ctx->status_dev, kStatusWords * sizeof(int)) != cudaSuccess ||
        cudaMemset(ctx->status_dev, 0, kStatusWords * sizeof(int)) != cudaSuccess ||
        cudaHostAlloc(&ctx->status_host, kStatusWords * sizeof(int), cudaHostAllocDefault) != cudaSuccess) {
        if (ctx->status_dev) cudaFree(ctx->status_dev);
        delete ctx;
        return GELO_ERR_CUDA;
    }
    bool lanes_ok = cudaEventCreateWithFlags(&ctx->batch_start, cudaEventDisableTiming) == cudaSuccess;
    for (int l = 0; l < kMaxLanes && lanes_ok; ++l)
        lanes_ok = cudaStreamCreateWithFlags(&ctx->lane_stream[l], cudaStreamNonBlocking) == cudaSuccess &&
                   cudaEventCreateWithFlags(&ctx->lane_ready[l], cudaEventDisableTiming) == cudaSuccess &&
                   cudaEventCreateWithFlags(&ctx->lane_free[l], cudaEventDisableTiming) == cudaSuccess;
    lanes_ok = lanes_ok && cudaMalloc(&ctx->lane_seed_dev, kMaxLanes * 8 * sizeof(uint64_t)) == cudaSuccess;
    lanes_ok = lanes_ok && cudaStreamCreateWithFlags(&ctx->copy_in, cudaStreamNonBlocking) == cudaSuccess &&
               cudaStreamCreateWithFlags(&ctx->copy_out, cudaStreamNonBlocking) == cudaSuccess;
    for (int b = 0; b < 2 && lanes_ok; ++b)
        lanes_ok = cudaEventCreateWithFlags(&ctx->h_ready[b], cudaEventDisableTiming) == cudaSuccess &&
                   cudaEventCreateWithFlags(&ctx->h_free[b], cudaEventDisableTiming) == cudaSuccess &&
                   cudaEventCreateWithFlags(&ctx->y_ready[b], cudaEventDisableTiming) == cudaSuccess &&
                   cudaEventCreateWithFlags(&ctx->y_free[b], cudaEventDisableTiming) == cudaSuccess;
    if (!lanes_ok) { gelo_destroy(ctx); return GELO_ERR_CUDA; }
    cudaDriverEntryPointQueryResult qres;
    void* fn = nullptr;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
        ctx->tmap_encode = fn;
    *out = ctx;
    return GELO_OK;
}

int gelo_destroy(gelo_ctx* ctx)
{
    if (!ctx) return GELO_ERR_INVALID;
    DeviceGuard guard(ctx->device);
    for (int l = 0; l < kMaxLanes; ++l) {
        if (ctx->lane_stream[l]) { cudaStreamSynchronize(ctx->lane_stream[l]); cudaStreamDestroy(ctx->lane_stream[l]); }
        if (ctx->lane_ready[l]) cudaEventDestroy(ctx->lane_ready[l]);
        if (ctx->lane_free[l]) cudaEventDestroy(ctx->lane_free[l]);
    }
    drop_graphs(ctx);
    if (ctx->copy_in) { cudaStreamSynchronize(ctx->copy_in); cudaStreamDestroy(ctx->copy_in); }
    if (ctx->copy_out) { cudaStreamSynchronize(ctx->copy_out); cudaStreamDestroy(ctx->copy_out); }
    for (int b = 0; b < 2; ++b) {
        if (ctx->h_ready[b]) cudaEventDestroy(ctx->h_ready[b]);
        if (ctx->h_free[b]) cudaEventDestroy(ctx->h_free[b]);
        if (ctx->y_ready[b]) cudaEventDestroy(ctx->y_ready[b]);
        if (ctx->y_free[b]) cudaEventDestroy(ctx->y_free[b]);
    }
    if (ctx->lane_seed_dev) cudaFree(ctx->lane_seed_dev);
    if (ctx->batch_start) cudaEventDestroy(ctx->batch_start);
    cudaFree(ctx->status_dev);
    cudaFreeHost(ctx->status_host);
    delete ctx;
    return GELO_OK;
}

size_t gelo_workspace_bytes(int n, int k, int d, int p, int dtype)
{
    if (n < 0 || k < 0 || d < 0 || p < 0 || bad_dtype(dtype) || n + k <= 0) return 0;
    Arena a;
    a.cap = ~size_t(0) >> 1;
    carve(a, n, k, d, p, dtype, true);
    return a.off + 256;
}

int gelo_set_workspace(gelo_ctx* ctx, void* dev_ws, size_t bytes)
{
    if (!ctx) return GELO_ERR_INVALID;
    if (dev_ws && (reinterpret_cast<uintptr_t>(dev_ws) & 255u)) return GELO_ERR_INVALID;
    drop_graphs(ctx);              // recorded launches point into the old workspace
    ctx->chain_valid = false;
    ctx->ws = dev_ws;
    ctx->ws_bytes = dev_ws ? bytes : 0;
    return GELO_OK;
}

int gelo_set_nonorthogonal(gelo_ctx* ctx, float gamma, float cond_bound, int max_attempts)
{
    if (!ctx || !(gamma >= 0.0f) || !(cond_bound >= 1.0f) || max_attempts < 1 || max_attempts > 64)
        return GELO_ERR_INVALID;
    drop_graphs(ctx);              // gamma and the bound are baked into recorded launches
    ctx->gamma = gamma;
    ctx->cond_bound = cond_bound;
    ctx->max_attempts = max_attempts;
    return GELO_OK;
}

int gelo_mixing_ld(int m) { return m <= 0 ? 0 : round_up(m, 64); }

int gelo_last_status(gelo_ctx* ctx, void* stream)
{
    if (!ctx) return GELO_ERR_INVALID;
    DeviceGuard guard(ctx->device);
    cudaStream_t st = as_stream(stream);
    GELO_CUDA_OK(cudaMemcpyAsync(ctx->status_host, ctx->status_dev, kStatusWords * sizeof(int),
                                 cudaMemcpyDeviceToHost, st));
    GELO_CUDA_OK(cudaMemsetAsync(ctx->status_dev, 0, sizeof(int), st));
    GELO_CUDA_OK(cudaStreamSynchronize(st));
    return ctx->status_host[0];
}

long long gelo_launch_count(gelo_ctx* ctx, int reset)
{
    if (!ctx) return -1;
    const long long v = ctx->launches;
    if (reset) ctx->launches = 0;
    return v;
}

const char* gelo_status_string(int s)
{
    switch (s) {
        case GELO_OK: return "ok";
        case GELO_ERR_INVALID: return "invalid argument";
        case GELO_ERR_WORKSPACE: return "workspace missing or too small";
        case GELO_ERR_COND: return "no mixing matrix within the condition-number bound";
        case GELO_ERR_TIMEOUT: return "a bounded device-side wait ran out";
        case GELO_ERR_CUDA: return "CUDA call failed";
        case GELO_ERR_UNSUPPORTED: return "unsupported request";
        default: return "unknown status";
    }
}

int gelo_philox_words(gelo_ctx* ctx, uint64_t seed, uint32_t stream_id, uint32_t attempt, uint64_t first,
                      uint64_t count, uint32_t* out_dev, void* stream)
{
    if (!ctx || (!out_dev && count)) return GELO_ERR_INVALID;
    DeviceGuard guard(ctx->device);
    return launch_philox_words(ctx, seed, stream_id, attempt, first, count, out_dev, as_stream(stream));
}

int gelo_sample_gaussian(gelo_ctx* ctx, int rows, int cols, int ld, uint64_t seed, uint32_t stream_id,
                         uint32_t attempt, float scale, float* out_dev, void* stream)
{
    if (!ctx || rows < 0 || cols < 0 || ld < cols) return GELO_ERR_INVALID;
    if (rows == 0 || cols == 0) return GELO_OK;
    if (!out_dev || misaligned(out_dev)) return GELO_ERR_INVALID;
    DeviceGuard guard(ctx->device);
    return launch_gaussian(ctx, rows, cols, ld, seed, stream_id, attempt, scale, nullptr, out_dev, as_stream(stream));
}

int gelo_qr_orthogonal(gelo_ctx* ctx, int m, float* G_dev, int ld, float* Q_dev, float* Qt_dev, void* stream)
{
    if (!ctx || m <= 0 || !G_dev || !Q_dev || ld < m) return GELO_ERR_INVALID;
    DeviceGuard guard(ctx->device);
    Layout L;
    if (!carve_ctx(ctx, m, 0, 0, 0, GELO_F32, false, &L)) return GELO_ERR_WORKSPACE;
    cudaStream_t st = as_stream(stream);
    const int tcp = level3_kind(ctx, m, GELO_F32, true);
    if (ld == L.ldi) {
        if (tcp == 3) GELO_TRY(run_householder_qr_tf32(ctx, m, G_dev, ld, L.Qraw, L.qr, L.tc, st));
        else if (tcp) GELO_TRY(run_householder_qr_tc(ctx, m, G_dev, ld, L.Qraw, L.qr, L.tc, st));
        else GELO_TRY(run_householder_qr(ctx, m, G_dev, ld, L.Qraw, L.qr, st));
        if (tcp == 3) GELO_TRY(polish_orthogonal_tf32(ctx, m, L.Qraw, ld, L.X32, L.A32, st));
        return launch_finish_mixing(ctx, m, L.Qraw, ld, G_dev, ld, GELO_F32, Q_dev, Qt_dev, ld, st);
    }
    GELO_CUDA_OK(cudaMemcpy2DAsync(L.G, (size_t)L.ldi * 4, G_dev, (size_t)ld * 4, (size_t)m * 4, m,
                                   cudaMemcpyDeviceToDevice, st));
    if (tcp == 3) GELO_TRY(run_householder_qr_tf32(ctx, m, L.G, L.ldi, L.Qraw, L.qr, L.tc, st));
    else if (tcp) GELO_TRY(run_householder_qr_tc(ctx, m, L.G, L.ldi, L.Qraw, L.qr, L.tc, st));
    else GELO_TRY(run_householder_qr(ctx, m, L.G, L.ldi, L.Qraw, L.qr, st));
    if (tcp == 3) GELO_TRY(polish_orthogonal_tf32(ctx, m, L.Qraw, L.ldi, L.X32, L.A32, st));
    GELO_TRY(launch_finish_mixing(ctx, m, L.Qraw, L.ldi, L.G, L.ldi, GELO_F32, Q_dev, Qt_dev, ld, st));
    return cudaMemcpy2DAsync(G_dev, (size_t)ld * 4, L.G, (size_t)L.ldi * 4, (size_t)m * 4, m,
                             cudaMemcpyDeviceToDevice, st) == cudaSuccess ? GELO_OK : GELO_ERR_CUDA;
}

int gelo_lu_inverse(gelo_ctx* ctx, int m, const float* A_dev, int ld, float* Ainv_dev, void* stream)
{
    if (!ctx || m <= 0 || !A_dev || !Ainv_dev || ld < m) return GELO_ERR_INVALID;
    DeviceGuard guard(ctx->device);
    Layout L;
    if (!carve_ctx(ctx, m, 0, 0, 0, GELO_F32, false, &L)) return GELO_ERR_WORKSPACE;
    cudaStream_t st = as_stream(stream);
    const int tcp = level3_kind(ctx, m, GELO_F32, false);
    if (ld == L.ldi) return tcp ? run_lu_inverse_tc(ctx, m, A_dev, ld, Ainv_dev, L.lu, L.tc, tcp == 3, st)
                                : run_lu_inverse(ctx, m, A_dev, ld, Ainv_dev, L.lu, st);
    GELO_CUDA_OK(cudaMemcpy2DAsync(L.A32, (size_t)L.ldi * 4, A_dev, (size_t)ld * 4, (size_t)m * 4, m,
                                   cudaMemcpyDeviceToDevice, st));
    if (tcp) GELO_TRY(run_lu_inverse_tc(ctx, m, L.A32, L.ldi, L.X32, L.lu, L.tc, tcp == 3, st));
    else GELO_TRY(run_lu_inverse(ctx, m, L.A32, L.ldi, L.X32, L.lu, st));
    return cudaMemcpy2DAsync(Ainv_dev, (size_t)ld * 4, L.X32, (size_t)L.ldi * 4, (size_t)m * 4, m,
                             cudaMemcpyDeviceToDevice, st) == cudaSuccess ? GELO_OK : GELO_ERR_CUDA;
}

int gelo_cond_estimate(gelo_ctx* ctx, int m, const float* A_dev, const float* Ainv_dev, int ld,
                       float* cond_dev, void* stream)
{
    if (!ctx || m <= 0 || !A_dev || !Ainv_dev || !cond_dev || ld < m) return GELO_ERR_INVALID;
    DeviceGuard guard(ctx->device);
    Layout L;
    if (!carve_ctx(ctx, m, 0, 0, 0, GELO_F32, false, &L)) return GELO_ERR_WORKSPACE;
    return run_cond_estimate(ctx, m, A_dev, Ainv_dev, ld, GELO_F32, ctx->cond_bound, cond_dev, L.cond, as_stream(stream));
}

int gelo_sample_mixing(gelo_ctx* ctx, int m, int kind, uint64_t seed, int dtype, void* A_dev, void* Ainv_dev,
                       int lda, float* cond_dev, void* stream)
{
    if (!ctx || m <= 0 || !A_dev || !Ainv_dev || bad_dtype(dtype) || bad_ld(lda, m) ||
        (kind != GELO_ORTHOGONAL && kind != GELO_NONORTHOGONAL) || misaligned(A_dev) || misaligned(Ainv_dev))
        return GELO_ERR_INVALID;
    DeviceGuard guard(ctx->device);
    Layout L;
    if (!carve_ctx(ctx, m, 0, 0, 0, dtype, false, &L)) return GELO_ERR_WORKSPACE;
    return sample_mixing_impl(ctx, L, m, kind, seed, dtype, A_dev, Ainv_dev, lda, cond_dev, as_stream(stream));
}

int gelo_shield_rows(gelo_ctx* ctx, const void* H_dev, int n, int d, int k, float scale, uint64_t seed,
                     int dtype, void* S_dev, void* stream)
{
    if (!ctx || n <= 0 || d <= 0 || k < 0 || bad_dtype(dtype) || (d % 8) != 0 || !H_dev || misaligned(H_dev))
        return GELO_ERR_INVALID;
    if (k == 0) return GELO_OK;
    if (!S_dev || misaligned(S_dev)) return GELO_ERR_INVALID;
    DeviceGuard guard(ctx->device);
    if (!ctx->ws) return GELO_ERR_WORKSPACE;
    Arena a;
    a.base = static_cast<char*>(ctx->ws);
    a.cap = ctx->ws_bytes;
    ShieldScratch sh = carve_shield(a, n);
    if (!a.ok) return GELO_ERR_WORKSPACE;
    ctx->chain_valid = false;
    return run_shield_rows(ctx, H_dev, n, d, k, scale, seed, dtype, S_dev, sh, as_stream(stream));
}

int gelo_shield_rows_t(gelo_ctx* ctx, const void* H_dev, int n, int d, int k, float scale, uint64_t seed, int nu,
                       int dtype, void* S_dev, void* stream)
{
    if (!ctx || n <= 0 || d <= 0 || k < 0 || bad_dtype(dtype) || (d % 8) != 0 || !H_dev || misaligned(H_dev) || nu < 3 || nu > 63)
        return GELO_ERR_INVALID;
    if (k == 0) return GELO_OK;
    if (!S_dev || misaligned(S_dev)) return GELO_ERR_INVALID;
    DeviceGuard guard(ctx->device);
    if (!ctx->ws) return GELO_ERR_WORKSPACE;
    Arena a;
    a.base = static_cast<char*>(ctx->ws);
    a.cap = ctx->ws_bytes;
    ShieldScratch sh = carve_shield(a, n);
    if (!a.ok) return GELO_ERR_WORKSPACE;
    ctx->chain_valid = false;
    return run_shield_rows(ctx, H_dev, n, d, k, scale, seed, dtype, S_dev, sh, as_stream(stream), nu);
}

int gelo_set_shield_student_t(gelo_ctx* ctx, int nu)
{
    if (!ctx || (nu != 0 && (nu < 3 || nu > 63))) return GELO_ERR_INVALID;
    ctx->shield_nu = nu;
    return GELO_OK;
}

int gelo_mix(gelo_ctx* ctx, const void* A_dev, int lda, const void* H_dev, const void* S_dev, int n, int k,
             int d, int dtype, void* U_dev, void* stream)
{
    if (!ctx || n <= 0 || k < 0 || d <= 0 || (d % 8) != 0 || bad_dtype(dtype) || !A_dev || !H_dev || !U_dev ||
        bad_ld(lda, n + k) || ((k > 0) != (S_dev != nullptr)) || misaligned(A_dev) || misaligned(H_dev) ||
        misaligned(S_dev) || misaligned(U_dev))
        return GELO_ERR_INVALID;
    DeviceGuard guard(ctx->device);
    return mix_impl(ctx, A_dev, lda, H_dev, S_dev, n, k, d, dtype, U_dev, as_stream(stream));
}

int gelo_project(gelo_ctx* ctx, const void* U_dev, const void* W_dev, int m, int d, int p, int dtype,
                 void* Yp_dev, void* stream)
{
    if (!ctx || m <= 0 || d <= 0 || p <= 0 || (d % 8) != 0 || (p % 8) != 0 || bad_dtype(dtype) || !U_dev ||
        !W_dev || !Yp_dev || misaligned(U_dev) || misaligned(W_dev) || misaligned(Yp_dev))
        return GELO_ERR_INVALID;
    DeviceGuard guard(ctx->device);
    Layout L;
    return project_impl(ctx, U_dev, W_dev, m, d, p, dtype, Yp_dev, as_stream(stream), stage_pairs(ctx, m, 0, d, p, dtype, &L));
}

int gelo_quantize_e4m3(gelo_ctx* ctx, const void* X_dev, int rows, int cols, int dtype, void* codes_dev, float* scale_dev,
                       void* stream)
{
    if (!ctx || rows <= 0 || cols <= 0 || (cols % 16) != 0 || bad_dtype(dtype) || !X_dev || !codes_dev || !scale_dev ||
        misaligned(X_dev) || misaligned(codes_dev) || (reinterpret_cast<uintptr_t>(scale_dev) & 7u))
        return GELO_ERR_INVALID;
    DeviceGuard guard(ctx->device);
    return launch_quantize_e4m3(ctx, X_dev, rows, cols, cols, dtype, codes_dev, cols, scale_dev, as_stream(stream));
}

int gelo_project_e4m3(gelo_ctx* ctx, const void* U8_dev, const float* u_scale_dev, const void* W8_dev, const float* w_scale_dev,
                      int m, int d, int p, void* Yp_dev, void* stream)
{
    if (!ctx || m <= 0 || d <= 0 || p <= 0 || (d % 16) != 0 || (p % 16) != 0 || !U8_dev || !W8_dev || !u_scale_dev ||
        !w_scale_dev || !Yp_dev || misaligned(U8_dev) || misaligned(W8_dev) || misaligned(Yp_dev))
        return GELO_ERR_INVALID;
    DeviceGuard guard(ctx->device);
    return launch_gemm_e4m3(ctx, m, p, d, U8_dev, d, W8_dev, p, u_scale_dev, w_scale_dev, Yp_dev, p, as_stream(stream));
}

int gelo_unmix(gelo_ctx* ctx, const void* Ainv_dev, int lda, const void* Yp_dev, int n, int k, int p, int dtype,
               void* Q_dev, void* K_dev, void* V_dev, void* stream)
{
    if (!ctx || n <= 0 || k < 0 || p <= 0 || (p % 8) != 0 || bad_dtype(dtype) || !Ainv_dev || !Yp_dev ||
        bad_ld(lda, n + k) || misaligned(Ainv_dev) || misaligned(Yp_dev) || misaligned(Q_dev) ||
        misaligned(K_dev) || misaligned(V_dev))
        return GELO_ERR_INVALID;
    GELO_TRY(check_split(p, Q_dev, K_dev, V_dev));
    DeviceGuard guard(ctx->device);
    Layout L;
    return unmix_impl(ctx, Ainv_dev, lda, Yp_dev, n, k, p, dtype, Q_dev, K_dev, V_dev, as_stream(stream),
                      stage_pairs(ctx, n, k, 8, p, dtype, &L));
}

int gelo_project_unmix(gelo_ctx* ctx, const void* U_dev, const void* W_dev, const void* Ainv_dev, int lda, int n, int k,
                       int d, int p, int dtype, void* Q_dev, void* K_dev, void* V_dev, void* stream)
{
    if (!ctx || n <= 0 || k < 0 || d <= 0 || p <= 0 || (d % 8) != 0 || (p % 8) != 0 || bad_dtype(dtype) || !U_dev || !W_dev ||
        !Ainv_dev || bad_ld(lda, n + k) || misaligned(U_dev) || misaligned(W_dev) || misaligned(Ainv_dev) || misaligned(Q_dev) ||
        misaligned(K_dev) || misaligned(V_dev))
        return GELO_ERR_INVALID;
    GELO_TRY(check_split(p, Q_dev, K_dev, V_dev));
    DeviceGuard guard(ctx->device);
    return launch_project_unmix(ctx, U_dev, W_dev, Ainv_dev, lda, n, k, d, p, dtype, Q_dev, K_dev, V_dev, as_stream(stream));
}

int gelo_set_small_batch_fusion(gelo_ctx* ctx, int on)
{
    if (!ctx) return GELO_ERR_INVALID;
    ctx->fuse_small = on != 0;
    return GELO_OK;
}

int gelo_qkv_offload(gelo_ctx* ctx, const void* H_dev, const void* W_dev, int n, int k, int d, int p, int kind,
                     uint64_t seed, float shield_scale, int dtype, void* Q_dev, void* K_dev, void* V_dev,
                     void* stream)
{
    if (!ctx || n <= 0 || k < 0 || d <= 0 || p <= 0 || (d % 8) != 0 || (p % 8) != 0 || bad_dtype(dtype) ||
        !H_dev || !W_dev || (kind != GELO_ORTHOGONAL && kind != GELO_NONORTHOGONAL) || misaligned(H_dev) ||
        misaligned(W_dev) || misaligned(Q_dev) || misaligned(K_dev) || misaligned(V_dev))
        return GELO_ERR_INVALID;
    GELO_TRY(check_split(p, Q_dev, K_dev, V_dev));
    DeviceGuard guard(ctx->device);
    if (kind == GELO_ORTHOGONAL && !ctx->prof_on) {
        // nothing to verify: run it as a batch of one, which replays the recorded sampling graph on a lane stream
        const void* H1[1] = { H_dev }; const void* W1[1] = { W_dev };
        void* Q1[1] = { Q_dev }; void* K1[1] = { K_dev }; void* V1[1] = { V_dev };
        const int kind1[1] = { kind }; const uint64_t seed1[1] = { seed };
        return offload_batch_impl(ctx, 1, H1, W1, n, k, d, p, kind1, seed1, shield_scale, dtype, Q1, K1, V1,
                                  as_stream(stream), false);
    }
    Layout L;
    if (!carve_ctx(ctx, n, k, d, p, dtype, false, &L)) return GELO_ERR_WORKSPACE;
    return offload_impl(ctx, L, H_dev, W_dev, n, k, d, p, kind, seed, shield_scale, dtype, Q_dev, K_dev, V_dev,
                        as_stream(stream));
}

int gelo_qkv_offload_host(gelo_ctx* ctx, const void* H_host, const void* W_dev, int n, int k, int d, int p,
                          int kind, uint64_t seed, float shield_scale, int dtype, void* Q_host, void* K_host,
                          void* V_host, void* stream)
{
    if (!ctx || n <= 0 || k < 0 || d <= 0 || p <= 0 || (d % 8) != 0 || (p % 8) != 0 || bad_dtype(dtype) ||
        !H_host || !W_dev || (kind != GELO_ORTHOGONAL && kind != GELO_NONORTHOGONAL) || misaligned(W_dev))
        return GELO_ERR_INVALID;
    GELO_TRY(check_split(p, Q_host, K_host, V_host));
    DeviceGuard guard(ctx->device);
    Layout L;
    if (!carve_ctx(ctx, n, k, d, p, dtype, true, &L)) return GELO_ERR_WORKSPACE;
    cudaStream_t st = as_stream(stream);
    const size_t es = elem_size(dtype);
    GELO_CUDA_OK(cudaMemcpyAsync(L.Hd, H_host, (size_t)n * d * es, cudaMemcpyHostToDevice, st));
    char* y = static_cast<char*>(L.Yd);
    const bool split = K_host != nullptr;
    const size_t third = (size_t)n * (p / 3) * es;
    GELO_TRY(offload_impl(ctx, L, L.Hd, W_dev, n, k, d, p, kind, seed, shield_scale, dtype, y,
                          split ? y + third : nullptr, split ? y + 2 * third : nullptr, st));
    if (split) {
        GELO_CUDA_OK(cudaMemcpyAsync(Q_host, y, third, cudaMemcpyDeviceToHost, st));
        GELO_CUDA_OK(cudaMemcpyAsync(K_host, y + third, third, cudaMemcpyDeviceToHost, st));
        GELO_CUDA_OK(cudaMemcpyAsync(V_host, y + 2 * third, third, cudaMemcpyDeviceToHost, st));
    } else {
        GELO_CUDA_OK(cudaMemcpyAsync(Q_host, y, (size_t)n * p * es, cudaMemcpyDeviceToHost, st));
    }
    GELO_CUDA_OK(cudaStreamSynchronize(st));
    return GELO_OK;
}

size_t gelo_batch_workspace_bytes(int n, int k, int d, int p, int dtype, int lanes)
{
    if (n < 0 || k < 0 || d < 0 || p < 0 || bad_dtype(dtype) || n + k <= 0 || lanes < 1 || lanes > kMaxLanes) return 0;
    return batch_workspace(n, k, d, p, dtype, lanes);
}

int gelo_set_lanes(gelo_ctx* ctx, int lanes)
{
    if (!ctx || lanes < 1 || lanes > kMaxLanes) return GELO_ERR_INVALID;
    ctx->lanes = lanes;
    return GELO_OK;
}

int gelo_qkv_offload_batch(gelo_ctx* ctx, int calls, const void* const* H_dev, const void* const* W_dev, int n, int k,
                           int d, int p, const int* kinds, const uint64_t* seeds, float shield_scale, int dtype,
                           void* const* Q_dev, void* const* K_dev, void* const* V_dev, void* stream)
{
    GELO_TRY(check_batch_args(ctx, calls, H_dev, W_dev, n, k, d, p, kinds, seeds, dtype, Q_dev, K_dev, V_dev, false));
    if (calls == 0) return GELO_OK;
    DeviceGuard guard(ctx->device);
    return offload_batch_impl(ctx, calls, H_dev, W_dev, n, k, d, p, kinds, seeds, shield_scale, dtype, Q_dev, K_dev,
                              V_dev, as_stream(stream), false);
}

int gelo_qkv_offload_batch_host(gelo_ctx* ctx, int calls, const void* const* H_host, const void* const* W_dev, int n,
                                int k, int d, int p, const int* kinds, const uint64_t* seeds, float shield_scale,
                                int dtype, void* const* Q_host, void* const* K_host, void* const* V_host, void* stream)
{
    GELO_TRY(check_batch_args(ctx, calls, H_host, W_dev, n, k, d, p, kinds, seeds, dtype, Q_host, K_host, V_host, true));
    if (calls == 0) return GELO_OK;
    DeviceGuard guard(ctx->device);
    return offload_batch_impl(ctx, calls, H_host, W_dev, n, k, d, p, kinds, seeds, shield_scale, dtype, Q_host, K_host,
                              V_host, as_stream(stream), true);
}

int gelo_qkv_offload_batch_host_async(gelo_ctx* ctx, int calls, const void* const* H_host, const void* const* W_dev,
                                      int n, int k, int d, int p, const int* kinds, const uint64_t* seeds,
                                      float shield_scale, int dtype, void* const* Q_host, void* const* K_host,
                                      void* const* V_host, void* stream)
{
    GELO_TRY(check_batch_args(ctx, calls, H_host, W_dev, n, k, d, p, kinds, seeds, dtype, Q_host, K_host, V_host, true));
    if (calls == 0) return GELO_OK;
    DeviceGuard guard(ctx->device);
    return offload_batch_impl(ctx, calls, H_host, W_dev, n, k, d, p, kinds, seeds, shield_scale, dtype, Q_host, K_host,
                              V_host, as_stream(stream), true, false);
}

size_t gelo_blockdiag_workspace_bytes(int n, int k, int d, int p, int dtype, int block, int lanes)
{
    if (n <= 0 || k < 0 || d <= 0 || p <= 0 || bad_dtype(dtype) || lanes < 1 || lanes > kMaxLanes) return 0;
    return blockdiag_workspace(n, k, d, p, dtype, block, lanes);
}

int gelo_qkv_offload_blockdiag_batch(gelo_ctx* ctx, int calls, const void* const* H_dev, const void* const* W_dev, int n,
                                     int k, int d, int p, int block, const uint64_t* seeds, float shield_scale, int dtype,
                                     void* const* Q_dev, void* const* K_dev, void* const* V_dev, void* stream)
{
    if (!ctx || calls < 0 || n <= 0 || k < 0 || d <= 0 || p <= 0 || (d % 8) != 0 || (p % 8) != 0 || bad_dtype(dtype))
        return GELO_ERR_INVALID;
    if (calls == 0) return GELO_OK;
    if (!H_dev || !W_dev || !seeds || !Q_dev || !K_dev || !V_dev) return GELO_ERR_INVALID;
    const bool split = K_dev[0] != nullptr;
    for (int i = 0; i < calls; ++i) {
        if (!H_dev[i] || !W_dev[i] || misaligned(H_dev[i]) || misaligned(W_dev[i]) || misaligned(Q_dev[i]) ||
            misaligned(K_dev[i]) || misaligned(V_dev[i]) || (K_dev[i] != nullptr) != split)
            return GELO_ERR_INVALID;
        GELO_TRY(check_split(p, Q_dev[i], K_dev[i], V_dev[i]));
    }
    DeviceGuard guard(ctx->device);
    return offload_blockdiag_impl(ctx, calls, H_dev, W_dev, n, k, d, p, block, seeds, shield_scale, dtype, Q_dev, K_dev,
                                  V_dev, as_stream(stream));
}

int gelo_profile_start(gelo_ctx* ctx)
{
    if (!ctx) return GELO_ERR_INVALID;
    for (auto& e : ctx->prof) { cudaEventDestroy(e.e0); cudaEventDestroy(e.e1); }
    ctx->prof.clear();
    ctx->prof_on = true;
    return GELO_OK;
}

int gelo_profile_stop(gelo_ctx* ctx, void* stream, double* out)
{
    if (!ctx || !out) return GELO_ERR_INVALID;
    DeviceGuard guard(ctx->device);
    ctx->prof_on = false;
    GELO_CUDA_OK(cudaStreamSynchronize(as_stream(stream)));
    for (int l = 0; l < kMaxLanes; ++l) GELO_CUDA_OK(cudaStreamSynchronize(ctx->lane_stream[l]));
    for (int i = 0; i < 3 * PROF_CLASSES; ++i) out[i] = 0.0;
    for (auto& e : ctx->prof) {
        float ms = 0.0f;
        if (cudaEventElapsedTime(&ms, e.e0, e.e1) == cudaSuccess && e.cls >= 0 && e.cls < PROF_CLASSES) {
            out[3 * e.cls + 0] += 1.0;
            out[3 * e.cls + 1] += ms;
            out[3 * e.cls + 2] += e.work;
        }
        cudaEventDestroy(e.e0);
        cudaEventDestroy(e.e1);
    }
    ctx->prof.clear();
    return GELO_OK;
}

int gelo_update_f32(gelo_ctx* ctx, int M, int N, int K, const float* A_dev, int lda, const float* B_dev, int ldb,
                    float* C_dev, int ldc, void* stream)
{
    if (!ctx || M <= 0 || N <= 0 || K <= 0 || K > kSuper || !A_dev || !B_dev || !C_dev || lda < K || ldb < N ||
        ldc < ((N + 7) & ~7) || (ldc % 4) != 0 || misaligned(C_dev))
        return GELO_ERR_INVALID;
    DeviceGuard guard(ctx->device);
    Layout L;
    if (!carve_ctx(ctx, M > N ? M : N, 0, 0, 0, GELO_F32, false, &L)) return GELO_ERR_WORKSPACE;
    return tc_update_f32(ctx, L.tc, ctx->level3 == 3, M, N, K, A_dev, lda, B_dev, ldb, C_dev, ldc, as_stream(stream));
}

int gelo_set_level3(gelo_ctx* ctx, int mode)
{
    if (!ctx || mode < 0 || mode > 3) return GELO_ERR_INVALID;
    ctx->level3 = mode;
    return GELO_OK;
}

int gelo_set_wait_limit_ns(gelo_ctx* ctx, unsigned long long ns)
{
    if (!ctx) return GELO_ERR_INVALID;
    drop_graphs(ctx);              // the limit is a launch parameter of the recorded kernels
    ctx->wait_limit_ns = ns;
    return GELO_OK;
}

int gelo_set_lane_share(gelo_ctx* ctx, int share)
{
    if (!ctx || share < 1 || share > 16) return GELO_ERR_INVALID;
    ctx->lane_tc_share = share;
    return GELO_OK;
}

}  // extern "C"
