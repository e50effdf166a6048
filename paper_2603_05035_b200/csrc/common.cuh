// Shared host-side declarations of the GELO library: context, status block,
// workspace carving and the internal launchers that the entry points chain.
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include <vector>

#include "../../include/gelo.h"

namespace gelo {

// Panel width of the blocked QR / LU factorisations.
constexpr int kPanel = 32;

// Device status block (ints).  [0]: first device-side error (gelo_status), sticky until read.
// [1]: verdict of the last condition-number check (1 = accepted).  [2]: detail word.
constexpr int kStatusWords = 8;
constexpr int kMaxLanes = 32;

// Kernel classes that the optional per-launch timing distinguishes.
enum ProfClass { PROF_RANK_UPDATE = 0, PROF_VTC = 1, PROF_GEMM_TC = 2, PROF_QR_PANEL = 3, PROF_LU_PANEL = 4,
                 PROF_CLASSES = 5 };
struct ProfEntry { int cls; double work; cudaEvent_t e0, e1; };

struct Arena {
    char* base = nullptr;
    size_t off = 0;
    size_t cap = 0;
    bool ok = true;
    void* take(size_t bytes) {
        size_t start = (off + 255) & ~size_t(255);
        if (start + bytes > cap) { ok = false; off = start + bytes; return nullptr; }
        off = start + bytes;
        return base ? base + start : nullptr;
    }
};

}  // namespace gelo

struct gelo_ctx {
    int device = 0;
    int sm_count = 0;
    void* ws = nullptr;
    size_t ws_bytes = 0;
    int* status_dev = nullptr;
    int* status_host = nullptr;   // pinned mirror
    float gamma = 0.5f;
    float cond_bound = 100.0f;
    int max_attempts = 8;
    int lane_tc_share = 4;        // batches with at least this many lanes give each level-3 update 1/share of the SMs
    int tc_update_ctas = 0;       // CTAs of a level-3 tensor-core launch (0: one per SM); batches with many lanes use fewer,
                                  // so that the updates of several lanes run side by side instead of queueing
    int level3 = 0;               // 0: tf32 tensor-core updates for bf16 calls with m >= 256; 1: always fp32 FMA;
                                  // 2: always tensor cores, three bf16 products of split operands; 3: always tensor cores, tf32
    long long launches = 0;
    unsigned long long wait_limit_ns = 2000000000ull;   // limit of every device-side barrier wait (gelo_set_wait_limit_ns)
    void* tmap_encode = nullptr;  // cuTensorMapEncodeTiled, resolved at creation
    int shield_nu = 0;            // shield rows of the whole-call entry points: 0 Gaussian, else Student-t with this many degrees of freedom
    bool fuse_small = true;       // calls with m <= 128 run projection and unmixing as one kernel (gelo_set_small_batch_fusion)
    int dec_group = 16;           // CTAs of the small-batch projection kernel that walk the k-blocks in step (0: all of them)
    bool tma_3d = true;           // N-major operand tiles as one three-dimensional TMA box where the layout allows
    // lanes of the batched entry points: each samples the mixing pair of one call on its own stream
    int lanes = 4;
    cudaStream_t lane_stream[gelo::kMaxLanes] = {};
    cudaEvent_t lane_ready[gelo::kMaxLanes] = {};   // A and A^-1 of the lane are complete
    cudaEvent_t lane_free[gelo::kMaxLanes] = {};    // the products that read them have been enqueued and finished
    cudaEvent_t batch_start = nullptr;
    // a batched call may chain onto the previous one (lanes wait for their own lane_free events only) when
    // nothing else has touched the workspace in between
    bool chain_valid = false;
    cudaStream_t chain_stream = nullptr;
    const void* chain_key = nullptr;
    int chain_lanes = 0;
    int chain_shape[6] = {0, 0, 0, 0, 0, 0};   // n, k, d, p, dtype, host staging of the batch a later one may chain onto
    // replayable launch graphs of the sampling sequence, one per (lane scratch, kind, size, type)
    struct SampleGraph { const void* key_ptr; int m, kind, dtype, level3, tc_ctas; cudaGraphExec_t exec; long long launches; };
    std::vector<SampleGraph> graphs;
    uint64_t* lane_seed_dev = nullptr;              // one seed slot per lane
    // the batched host variant moves activations in and results out on streams of their own, through two staging pairs
    cudaStream_t copy_in = nullptr, copy_out = nullptr;
    cudaEvent_t h_ready[2] = {}, h_free[2] = {}, y_ready[2] = {}, y_free[2] = {};
    // optional per-launch timing (gelo_profile_start / gelo_profile_stop)
    bool prof_on = false;
    std::vector<gelo::ProfEntry> prof;
};

namespace gelo {

#define GELO_CUDA_OK(expr)                                     \
    do {                                                       \
        cudaError_t gelo_e_ = (expr);                          \
        if (gelo_e_ != cudaSuccess) return GELO_ERR_CUDA;      \
    } while (0)

#define GELO_TRY(expr)                                         \
    do {                                                       \
        int gelo_s_ = (expr);                                  \
        if (gelo_s_ != GELO_OK) return gelo_s_;                \
    } while (0)

// Counts a launch and turns a launch error into a status.
static inline int after_launch(gelo_ctx* ctx) {
    ctx->launches += 1;
    return cudaPeekAtLastError() == cudaSuccess ? GELO_OK : GELO_ERR_CUDA;
}

// Brackets one launch with CUDA events on its stream while per-launch timing is on.
struct ProfScope {
    gelo_ctx* ctx; cudaStream_t st; cudaEvent_t e1 = nullptr;
    ProfScope(gelo_ctx* c, int cls, double work, cudaStream_t s) : ctx(c), st(s) {
        if (!c->prof_on) return;
        ProfEntry e; e.cls = cls; e.work = work; e.e0 = nullptr; e.e1 = nullptr;
        if (cudaEventCreate(&e.e0) != cudaSuccess || cudaEventCreate(&e.e1) != cudaSuccess) return;
        cudaEventRecord(e.e0, s);
        e1 = e.e1;
        c->prof.push_back(e);
    }
    ~ProfScope() { if (e1) cudaEventRecord(e1, st); }
};

static inline int ceil_div(int a, int b) { return (a + b - 1) / b; }
static inline size_t elem_size(int dtype) { return dtype == GELO_F32 ? 4 : 2; }

// ---- sampling ---------------------------------------------------------------------

int launch_philox_words(gelo_ctx*, uint64_t seed, uint32_t stream_id, uint32_t attempt,
                        uint64_t first, uint64_t count, uint32_t* out, cudaStream_t);

// out[i*ld + j] = (base ? base[i*ld + j] : 0) + scale * z(i*cols + j)
int launch_gaussian(gelo_ctx*, int rows, int cols, int ld, uint64_t seed, uint32_t stream_id,
                    uint32_t attempt, float scale, const float* base, float* out, cudaStream_t,
                    const uint64_t* seed_dev = nullptr);

// ---- fp32 SIMT GEMM ----------------------------------------------------------------

struct GemmArgs {
    int M = 0, N = 0, K = 0;
    const void* A = nullptr; int lda = 0; bool transA = false;   // op(A): M x K
    const void* B = nullptr; int ldb = 0; bool transB = false;   // op(B): K x N
    const void* B2 = nullptr; int b_split = 0;                   // rows >= b_split of op(B) come from B2 (not with transB)
    void* C[3] = {nullptr, nullptr, nullptr}; int ldc = 0;       // column block c / (N / nsplit) selects C[...]
    int nsplit = 1;
    float alpha = 1.0f, beta = 0.0f;
    int dtype = GELO_F32;                                        // storage type of A, B and C
};
int launch_gemm_simt(gelo_ctx*, const GemmArgs&, cudaStream_t);

// ---- bf16 tensor-core GEMM (tcgen05 / TMEM / TMA) ------------------------------------

// Same argument meaning as GemmArgs with dtype = GELO_BF16, transA = transB = false,
// alpha = 1, beta = 0.  Returns GELO_ERR_UNSUPPORTED for shapes it cannot take.
int launch_gemm_tc(gelo_ctx*, const GemmArgs&, cudaStream_t);
bool gemm_tc_supports(const GemmArgs&);
// Split-precision product on the tensor cores (operands as bf16 high / low pairs); see gemm_tc.cu.
int launch_gemm_tc_split(gelo_ctx*, int M, int N, int K, const void* Ahi, const void* Alo, int lda,
                         const void* Bhi, const void* Blo, int ldb, float* sub_from, int ldc, void* emit_hi,
                         void* emit_lo, int lde, bool narrow_tiles, cudaStream_t);
// Same product with the K range cut into `ksplit` slices whose fp32 partial products go to consecutive planes
// (plane stride in elements); returns the number of slices used in *used.
int launch_gemm_tc_split_k(gelo_ctx*, int M, int N, int K, const void* Ahi, const void* Alo, int lda, const void* Bhi,
                           const void* Blo, int ldb, float* planes, size_t plane, int ldp, int ksplit, int* used,
                           cudaStream_t);

// One-product tf32 GEMM straight from fp32 matrices (see gemm_tc.cu): C -= op(A) B in place, or C = op(A) B
// (optionally rounded to tf32, optionally as split-K planes).
int launch_gemm_tf32(gelo_ctx*, int M, int N, int K, const float* A, int lda, bool a_mn, const float* B, int ldb,
                     bool subtract, float* C, int ldc, bool round_out, float out_scale, int ksplit, size_t plane, int* used,
                     cudaStream_t, float diag_sub = 0.0f, float post_scale = 1.0f);
// D (m x m bf16) = post_scale * (out_scale * Q^T Q - diag_sub I): tf32 product over the tiles on and above the diagonal only
int launch_gram_sym_bf16(gelo_ctx*, int m, const float* Q, int ld, void* D, int ldd, float out_scale, float diag_sub,
                         float post_scale, cudaStream_t);
// C (fp32) -= A (bf16) B (bf16), in place
int launch_gemm_bf16_sub(gelo_ctx*, int M, int N, int K, const void* A, int lda, const void* B, int ldb, float* C, int ldc,
                         cudaStream_t);
// ---- E4M3 operands for the offloaded product (fp8.cu, gemm_tc.cu) ----
int launch_quantize_e4m3(gelo_ctx*, const void* x, int rows, int cols, int ld, int dtype, void* out, int ldo, float* scale,
                         cudaStream_t);
int launch_gemm_e4m3(gelo_ctx*, int M, int N, int K, const void* A8, int lda, const void* B8, int ldb, const float* sa,
                     const float* sb, void* C, int ldc, cudaStream_t);
// The tensor core drops the 13 low mantissa bits of an fp32 operand instead of rounding them.  For values whose
// mantissas are spread log-uniformly that loses 2^-11 / (2 ln 2) of the magnitude on average, coherently over all
// terms of a product; a result whose operand was truncated is scaled back by 1 + kTf32TruncLoss per such operand,
// which leaves a zero-mean error of about 3e-4 per term.  Operands that a kernel of this library rounded to tf32
// when it stored them pass through the tensor core unchanged and need no correction.
constexpr float kTf32TruncLoss = 3.5224e-4f;

// fp32 products on the tensor cores with fp32-grade accuracy: every operand is held as a pair of tf32 values
// (hi = x rounded to tf32, lo = the remainder rounded to tf32) and the product is accumulated as
// hi*hi + hi*lo + lo*hi in fp32 (the dropped lo*lo term is 2^-22 of the product).  C_q (q = 0 .. nsplit-1) receives
// the q-th column block of the M x N result; strides in elements, all multiples of 4, N / nsplit a multiple of 8.
// The tensor core adds into its fp32 accumulator with truncation, which costs about 2^-25 of the running sum per
// instruction, coherently: 5e-5 after the 1536 instructions of a K = 4096 product.  With `planes` (room for
// kTf32x3Slices * M * N floats) the K range is cut into that many slices with an accumulator each, summed afterwards in
// round-to-nearest fp32 in a fixed order, which brings the product back to a few 1e-6.
constexpr int kTf32x3Slices = 8;
int launch_gemm_tf32x3(gelo_ctx*, int M, int N, int K, const float* Ahi, const float* Alo, int lda, const float* Bhi,
                       const float* Blo, int ldb, float* const C[3], int ldc, int nsplit, float* planes, cudaStream_t);
// C_q[r, c] = sum over `parts` planes (M x N, dense) of the entry (r, q * csplit + c), planes added in order
int launch_sum_planes_routed(gelo_ctx*, const float* planes, size_t plane, int parts, int rows, int cols, float* const C[3],
                             int ldc, int csplit, cudaStream_t);
// hi / lo tf32 pair of a rows x cols fp32 block (cols a multiple of 4, 16-byte aligned rows)
int launch_split_tf32(gelo_ctx*, const float* src, int lds, int rows, int cols, float* hi, float* lo, int ldo, cudaStream_t);
// scratch of the tf32-pair products of the fp32 path: operand copies of at most a_elems / b_elems floats each
struct Tf32x3Scratch {
    float* a[2] = {nullptr, nullptr};
    float* b[2] = {nullptr, nullptr};
    float* planes = nullptr;              // kTf32x3Slices partial products of at most c_elems floats each
    size_t a_elems = 0, b_elems = 0, c_elems = 0;
};

// ---- projection and unmixing of a small batch in one kernel (decode.cu) ---------------------------------

// true when launch_project_unmix can serve the call: 16-bit storage, m = n + k <= 128, p a multiple of 64 whose
// 64-column boxes leave every CTA a slab of at most 128 columns
bool project_unmix_supports(const gelo_ctx*, int n, int k, int d, int p, int dtype, int lda, int nsplit);
// Q | K | V (or one n x p result in Q when K = V = nullptr) = (Ainv[0:n, 0:n+k] (U W)); U: (n+k) x d, W: d x p
int launch_project_unmix(gelo_ctx*, const void* U, const void* W, const void* Ainv, int lda, int n, int k, int d, int p,
                         int dtype, void* Q, void* K, void* V, cudaStream_t);

// U = A [H; S] for n + k <= 128 rows of a 16-bit type on the FMA pipes (one light launch instead of a tensor-core one)
bool mix_small_supports(int n, int k, int d, int dtype);
int launch_mix_small(gelo_ctx*, const void* A, int lda, const void* H, const void* S, int n, int k, int d, int dtype, void* U,
                     cudaStream_t);

// ---- factorizations -------------------------------------------------------------------

// ---- rank-32 updates of the factorisations (HBM streamers) ---------------------------------

constexpr int kMaxSlabs = 32;   // row slabs of the split V^T C product
// W (kPanel x nc, stride ldw) = op(T) * (V^T C);  V: nr x kv (stride ldv), C: nr x nc (stride ldc),
// T: kPanel x kPanel; Wp: kMaxSlabs * kPanel * ldw floats of scratch.
int launch_vtc(gelo_ctx*, const float* V, int ldv, int kv, const float* C, int ldc, int nr, int nc,
               const float* T, bool transpose_t, float* Wp, float* W, int ldw, cudaStream_t);
// C (M x N) -= A (M x K) * B (K x N), K <= kPanel
int launch_rank_update(gelo_ctx*, const float* A, int lda, const float* B, int ldb, float* C, int ldc,
                       int M, int N, int K, cudaStream_t);

struct QrScratch {       // all fp32
    float* V = nullptr;  // m x ld reflectors (unit diagonal, zeros above), all panels
    float* T = nullptr;  // ceil(m / kPanel) blocks of kPanel x kPanel
    float* Wp = nullptr; // kMaxSlabs x kPanel x ld partial products
    float* W2 = nullptr; // kPanel x ld
    float* T128 = nullptr; // ceil(m / 128) blocks of 128 x 128: triangular factors of the outer blocks
};
void* take_idle(Arena&, char** idle, size_t* idle_bytes, size_t bytes);
// `idle`, if given, is memory that nothing else uses while a factorisation runs (idle_bytes of it): scratch that lives
// only then is placed there instead of in the arena (see carve() in api.cu for who is idle when)
QrScratch carve_qr(Arena&, int m, int ld, char** idle = nullptr, size_t* idle_bytes = nullptr);
// Factorises R (m x m, stride ld, overwritten; its diagonal holds diag(R) afterwards) and
// writes the orthogonal factor Q with G = Q R.  The caller flips column j of Q where
// R_jj < 0 (launch_finish_mixing with sign_diag = R) to reach the unique factor.
int run_householder_qr(gelo_ctx*, int m, float* R, int ld, float* Q, const QrScratch&, cudaStream_t);
struct TcScratch;
// Same factorisation with 128-column outer blocks whose updates run on the tensor cores in split precision.
int run_householder_qr_tc(gelo_ctx*, int m, float* R, int ld, float* Q, const QrScratch&, const TcScratch&, cudaStream_t);
// The tf32 route: 128-column blocks grouped four by four; only the group's merged reflector (512 columns) is
// applied to the columns right of the group and, later, to Q, so the big matrices stream through the GPU once per
// 512 columns instead of once per 128.
int run_householder_qr_tf32(gelo_ctx*, int m, float* R, int ld, float* Q, const QrScratch&, const TcScratch&, cudaStream_t);
// One Newton-Schulz step Q <- Q - Q (Q^T Q - I) / 2 on the tensor cores in tf32: squares the orthogonality defect
// that tf32 updates leave in Q.  D and Qold are m x ld scratch matrices.
int polish_orthogonal_tf32(gelo_ctx*, int m, float* Q, int ld, float* D, float* Qold, cudaStream_t);

struct LuScratch {
    float* M = nullptr;   // m x ld working copy
    float* Z = nullptr;   // m x ld, optional: room for L^-1 (lets the forward solve skip the zero blocks); may not alias M, A or the result
    int* ipiv = nullptr;  // m
    int* perm = nullptr;  // m
    int* swap_table = nullptr;  // composed interchanges of one panel / block: count, then (target, source) pairs
};
LuScratch carve_lu(Arena&, int m, int ld);   // everything but the working copy M, which the caller points at memory of its choice
int run_lu_inverse(gelo_ctx*, int m, const float* A, int ld, float* Ainv, const LuScratch&, cudaStream_t);
struct TcScratch;
int run_lu_inverse_tc(gelo_ctx*, int m, const float* A, int ld, float* Ainv, const LuScratch&, const TcScratch&,
                      bool tf32, cudaStream_t);

struct CondScratch {
    float* vec = nullptr;     // iterate, image and row-slab partial sums for both operators
    float* scal = nullptr;    // 16 floats
};
CondScratch carve_cond(Arena&, int m);
// cond_out[0] = estimate; status_dev[1] = (estimate * 1.2 <= bound)
// A, Ainv: m x m matrices of type `dtype` with row stride ld (a multiple of 8)
int run_cond_estimate(gelo_ctx*, int m, const void* A, const void* Ainv, int ld, int dtype, float bound,
                      float* cond_out, const CondScratch&, cudaStream_t, bool deferred = false);

// ---- layout helpers ----------------------------------------------------------------------

// dst (rows x cols, stride ldd, dtype) = colscale-signed copy of src (fp32); dstT = its transpose.
// sign_diag (optional, fp32 matrix with stride lds): column j is multiplied by sign(sign_diag[j*lds + j]).
int launch_finish_mixing(gelo_ctx*, int m, const float* src, int lds_src, const float* sign_diag,
                         int lds_diag, int dtype, void* dst, void* dstT, int ldd, cudaStream_t);
// dst (dtype) = round(src fp32), m x m; back (optional, fp32, stride ldb, may alias src) = the stored values widened again
int launch_narrow(gelo_ctx*, int m, const float* src, int lds, int dtype, void* dst, int ldd, cudaStream_t,
                  float* back = nullptr, int ldb = 0);

// (hi, lo) bf16 pair of an fp32 block, optionally transposed (output is cols x rows then)
int launch_split(gelo_ctx*, const float* src, int lds, int rows, int cols, void* hi, void* lo, int ldo,
                 bool transpose, cudaStream_t);

// the same for two blocks in one launch (neither transposed)
int launch_split_pair(gelo_ctx*, const float* A, int lda, int rows_a, int cols_a, void* Ahi, void* Alo, int ldoa,
                      const float* B, int ldb, int rows_b, int cols_b, void* Bhi, void* Blo, int ldob, cudaStream_t);

int launch_sum_split(gelo_ctx*, const float* planes, size_t plane, int parts, int ld, int rows, int cols, void* hi,
                     void* lo, int ldo, cudaStream_t);
// out = scale * (sum of `parts` fp32 planes in plane order), rounded to tf32 (cols a multiple of 4)
int launch_sum_planes(gelo_ctx*, const float* planes, size_t plane, int parts, int ld, int rows, int cols, float scale,
                      float* out, int ldo, cudaStream_t);

// Scratch of the tensor-core level-3 updates (outer blocks of kOuter columns).
constexpr int kOuter = 128;
constexpr int kSuper = 4 * kOuter;        // columns whose reflectors reach the rest of the matrix in one tf32 update
constexpr int kMaxKSplit = 16;
constexpr int kSuperKSplit = kMaxKSplit * kOuter / kSuper;   // K slices of a kSuper-row product that fit the same planes
struct TcScratch {
    void* panA[2] = {nullptr, nullptr};    // m x kSuper          block column (V or L), hi / lo
    void* panAt[2] = {nullptr, nullptr};   // kOuter x ld         its transpose
    void* rowB[2] = {nullptr, nullptr};    // kSuper x ld         block row (W, U12 or X rows)
    void* rowB2[2] = {nullptr, nullptr};   // kOuter x ld
    void* tt[2] = {nullptr, nullptr};      // kOuter x kOuter     triangular factor (transposed or not)
    void* big[2] = {nullptr, nullptr};     // m x ld              trailing matrix as a pair
    float* t128 = nullptr;                 // kOuter x kOuter fp32
    float* gram = nullptr;                 // kOuter x kOuter fp32
    float* wf32 = nullptr;                 // kMaxKSplit planes of kOuter x ld fp32 (split-K partial products)
    float* w32[2] = {nullptr, nullptr};    // kSuper x ld fp32    block rows W and T W of the tf32 updates
    float* tsuper = nullptr;               // ceil(m / kSuper) merged triangular factors, kSuper x kSuper each
    float* sx = nullptr;                   // kOuter x (kSuper + kOuter)   V_i^T [V_(<i) | V_i] of the block being merged
    float* xb = nullptr;                   // kSuper x kOuter     its product with T_i
};
TcScratch carve_tc(Arena&, int m, int ld, char** idle = nullptr, size_t* idle_bytes = nullptr);   // all but big[], set by the caller
// C (M x N fp32) -= A (M x K fp32) * B (K x N fp32), K <= kSuper, on the tensor cores: three bf16 products of
// (high, low) operand pairs, or (tf32) one tf32 product straight from the fp32 operands
int tc_update_f32(gelo_ctx*, const TcScratch&, bool tf32, int M, int N, int K, const float* A, int lda, const float* B,
                  int ldb, float* C, int ldc, cudaStream_t);

// ---- shields ---------------------------------------------------------------------------------

struct ShieldScratch {
    float* norms = nullptr;   // n
    float* med = nullptr;     // 2
};
ShieldScratch carve_shield(Arena&, int n);
// nu = 0: Gaussian rows; 3 <= nu <= 63: standardised Student-t rows with nu degrees of freedom
int run_shield_rows(gelo_ctx*, const void* H, int n, int d, int k, float scale, uint64_t seed,
                    int dtype, void* S, const ShieldScratch&, cudaStream_t, int nu = 0);

}  // namespace gelo
