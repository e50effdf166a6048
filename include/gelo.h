/*
 * gelo.h -- C ABI of the B200 (sm_100a) library for GELO's obfuscated Q/K/V offload.
 *
 * One call of the path (paper Section 3.2 "Core Algorithm", Eq. 1-4, with the two
 * Gram-leak mitigations of Section 3.2.1):
 *
 *     sample a fresh secret invertible A (m x m, m = n + k)       step 1.2
 *     S  = k shield rows, scaled to the median row norm of H      Mitigation 2, Eq. 7-8
 *     U  = A [H; S]                                               Eq. 1
 *     Y' = U W                                                    Eq. 2
 *     Y  = (A^-1 Y')[0:n, :]  -> Q | K | V                        Eq. 3
 *
 * so that Y = H W (Eq. 4).
 *
 * Conventions for every entry point
 *   - Return value: a gelo_status.  Nothing throws or aborts across this boundary.
 *     Errors that the host can see (bad arguments, missing workspace, unsupported
 *     shapes) are returned before anything is launched.  Conditions only the
 *     device can see (condition bound missed after the last attempt, a bounded
 *     wait that ran out) are recorded in a status word that gelo_last_status reads.
 *   - "dev" pointers are device pointers on the context's GPU, owned by the caller,
 *     16-byte aligned, row-major and contiguous unless a row stride is given.
 *     "host" pointers are ordinary host memory (pinned memory makes the copies
 *     asynchronous).  The library never frees or keeps caller memory.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).  Work is
 *     enqueued on it; calls return without waiting unless stated otherwise.
 *   - Element type: GELO_F32 stores float, GELO_BF16 stores bfloat16, GELO_F16 stores IEEE half (the 16-bit
 *     types share every code path; half keeps 11 significant bits instead of 8); products always
 *     accumulate in fp32.
 *   - A and A^-1 are m x m with a row stride `lda` (in elements) that is a multiple of
 *     8 and >= m; gelo_mixing_ld(m) returns the stride the library prefers.  Columns
 *     m..lda-1 are padding: never read as data, contents unspecified.
 *   - All other matrices are dense: H n x d, S k x d, U m x d, W d x p, Y' m x p,
 *     Q/K/V n x (p/3).  d and p must be multiples of 8.
 *   - Scratch memory comes from the caller through gelo_set_workspace; no entry point
 *     except gelo_create / gelo_destroy allocates or frees device memory.
 */
#ifndef GELO_H
#define GELO_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    GELO_OK = 0,
    GELO_ERR_INVALID = 1,      /* bad argument (null pointer, negative size, bad stride, ...) */
    GELO_ERR_WORKSPACE = 2,    /* no workspace set, or it is too small for this call */
    GELO_ERR_COND = 3,         /* no A with kappa_2 <= bound within the attempt limit */
    GELO_ERR_TIMEOUT = 4,      /* a bounded device-side wait ran out; outputs are invalid */
    GELO_ERR_CUDA = 5,         /* a CUDA runtime or driver call failed */
    GELO_ERR_UNSUPPORTED = 6   /* valid request this build cannot serve (wrong GPU, p % 3 != 0 with a split, ...) */
} gelo_status;

typedef enum { GELO_ORTHOGONAL = 0, GELO_NONORTHOGONAL = 1 } gelo_kind;
typedef enum { GELO_F32 = 0, GELO_BF16 = 1, GELO_F16 = 2 } gelo_dtype;

/* Philox stream ids used by the library (third counter word). */
enum { GELO_STREAM_G0 = 0, GELO_STREAM_G1 = 1, GELO_STREAM_SHIELD = 2, GELO_STREAM_POWER = 3 };

typedef struct gelo_ctx gelo_ctx;

/* ---- context ------------------------------------------------------------------- */

/* Creates a context on CUDA device `device` (must be compute capability 10.x, else
 * GELO_ERR_UNSUPPORTED).  Allocates a few hundred bytes of device and pinned host
 * memory for the status word.  *ctx is NULL on failure. */
int gelo_create(gelo_ctx** ctx, int device);
int gelo_destroy(gelo_ctx* ctx);

/* Bytes of scratch that any call with these sizes needs (n data rows, k shield rows,
 * model width d, projection width p, element type t).  0 if an argument is invalid. */
size_t gelo_workspace_bytes(int n, int k, int d, int p, int dtype);

/* Hands the context a caller-owned device buffer (256-byte aligned).  It must stay
 * valid until replaced or the context is destroyed.  Calls on one context share it, so
 * they must be ordered on one stream. */
int gelo_set_workspace(gelo_ctx* ctx, void* dev_ws, size_t bytes);

/* Non-orthogonal construction A = Q0 + gamma * G1 (Mitigation 1; default gamma 0.5),
 * the accepted bound on kappa_2(A) (default 100) and the number of attempts (default 8,
 * each with the next attempt number in the Philox counter). */
int gelo_set_nonorthogonal(gelo_ctx* ctx, float gamma, float cond_bound, int max_attempts);

/* How the level-3 updates of the blocked QR / LU are computed.
 *   0 (default): fp32 FMA kernels for fp32 calls and for m < 256; for bf16 calls with m >= 256 the QR runs single
 *      tf32 tensor-core products straight from the fp32 matrices (followed, for an orthogonal A, by one
 *      Newton-Schulz step that squares the orthogonality defect tf32 leaves) and the LU runs three bf16 products of
 *      operands held as (high, low) pairs;
 *   1: always fp32 FMA;  2: always the split-precision products;  3: always tf32.
 * The split-precision products are good to about 1e-5 relative and tf32 to about 1e-3, neither of which the fp32
 * path's 1e-4 budget leaves room for, hence the default. */
int gelo_set_level3(gelo_ctx* ctx, int mode);

/* Preferred row stride (elements) of an m x m mixing matrix: m rounded up to 64. */
int gelo_mixing_ld(int m);

/* Limit, in nanoseconds of the GPU's global timer, of every device-side wait on a pipeline
 * barrier in the tensor-core kernels (default 2e9 = two seconds).  When a wait runs out the
 * CTA records GELO_ERR_TIMEOUT in the status word, stops issuing work, frees its tensor
 * memory and returns, and the outputs of that call are invalid.  A limit of 0 makes every
 * such kernel give up before it issues its first copy or MMA: a diagnostic setting that lets
 * a test see the timeout path without making any wait actually run out. */
int gelo_set_wait_limit_ns(gelo_ctx* ctx, unsigned long long ns);

/* Status word of the context: waits for `stream`, then returns the first device-side
 * error recorded since the last call of this function (GELO_OK if none) and clears it. */
int gelo_last_status(gelo_ctx* ctx, void* stream);

/* Number of kernels this context has launched since creation (or since the last reset). */
long long gelo_launch_count(gelo_ctx* ctx, int reset);

const char* gelo_status_string(int status);

/* ---- sampling (Section 3.2 step 1.2: every batch gets a newly drawn random invertible A) ---- */

/* Debug export of the random stream: out_dev[i] = the Philox4x32-10 word of element
 * first+i of (seed, stream_id, attempt).  Element e uses block e/4 -- counter
 * (lo32(e/4), hi32(e/4), stream_id, attempt), key (lo32(seed), hi32(seed)) -- word e%4. */
int gelo_philox_words(gelo_ctx* ctx, uint64_t seed, uint32_t stream_id, uint32_t attempt,
                      uint64_t first, uint64_t count, uint32_t* out_dev, void* stream);

/* out_dev (rows x cols fp32, row stride ld) = scale * N(0,1).  Element (i,j) is stream
 * element i*cols + j; words (0,1) and (2,3) of a block are Box-Muller pairs, the even
 * word giving r*cos(2 pi u_b), the odd word r*sin(2 pi u_b), r = sqrt(-2 ln u_a),
 * u = ((word >> 9) + 1/2) / 2^23: 23 bits, so that every u is exactly representable in
 * binary32 and the fp32 device arithmetic starts from the same value as an fp64 check. */
int gelo_sample_gaussian(gelo_ctx* ctx, int rows, int cols, int ld, uint64_t seed,
                         uint32_t stream_id, uint32_t attempt, float scale, float* out_dev,
                         void* stream);

/* Q_dev = the orthogonal factor of the Householder QR of G_dev (both m x m fp32, stride
 * ld), columns signed so that diag(R) > 0; Qt_dev (optional) = its transpose.  G_dev is
 * overwritten.  Needs workspace for (m, 0). */
int gelo_qr_orthogonal(gelo_ctx* ctx, int m, float* G_dev, int ld, float* Q_dev, float* Qt_dev,
                       void* stream);

/* Ainv_dev = A_dev^-1 by blocked LU with partial pivoting (both m x m fp32, stride ld);
 * A_dev is preserved.  Needs workspace for (m, 0). */
int gelo_lu_inverse(gelo_ctx* ctx, int m, const float* A_dev, int ld, float* Ainv_dev, void* stream);

/* cond_dev[0] = estimate of kappa_2(A) = sigma_max(A) * sigma_max(A^-1): square roots of the largest
 * Ritz values of A^T A and A^-T A^-1 after six Lanczos steps (a lower estimate, within a few percent).  ld must be a multiple of 8
 * and both matrices 16-byte aligned. */
int gelo_cond_estimate(gelo_ctx* ctx, int m, const float* A_dev, const float* Ainv_dev, int ld,
                       float* cond_dev, void* stream);

/* C_dev (M x N fp32, stride ldc) -= A_dev (M x K fp32, stride lda) * B_dev (K x N fp32, stride ldb), K <= 512:
 * the level-3 update of the blocked QR / LU, on the tensor cores with every operand held as a bf16
 * (high, low) pair and the product accumulated as hi*hi + hi*lo + lo*hi in fp32 (relative error of the
 * product about 1e-5).  ldc must be a multiple of 4 and >= N rounded up to 8; columns N .. that bound are
 * scratch.  Needs workspace for (max(M, N), 0).  With gelo_set_level3(ctx, 3) the same update runs as one tf32
 * product read straight from A_dev and B_dev (lda and ldb multiples of 4, both 16-byte aligned, no scratch columns);
 * the tensor core truncates the operands to tf32, so the product comes out 7e-4 short on average. */
int gelo_update_f32(gelo_ctx* ctx, int M, int N, int K, const float* A_dev, int lda, const float* B_dev, int ldb,
                    float* C_dev, int ldc, void* stream);

/* Samples the secret mixing pair for one batch.
 *   GELO_ORTHOGONAL:    A = Q of QR(G0), G0 ~ N(0,1) from stream 0;  A^-1 = A^T.
 *   GELO_NONORTHOGONAL: A = Q0 + gamma * G1 / sqrt(m) (G1 from stream 1), rounded to the
 *                       element type, then A^-1 of that stored A; accepted when the
 *                       kappa_2 estimate * 1.2 <= bound, else resampled with the next
 *                       attempt number.  The bound is enforced on an ESTIMATE (power
 *                       iteration, a lower estimate that tests put at 0.85 .. 1.0 of the
 *                       true value, hence the factor 1 / 0.85 rounded up).  This kind WAITS for `stream` once per attempt
 *                       to read the verdict; GELO_ERR_COND after the last attempt.
 * A_dev, Ainv_dev: m x m in `dtype`, stride lda.  cond_dev (optional, device float)
 * receives the estimate (1 for orthogonal).  Same (m, kind, seed) => same bytes. */
int gelo_sample_mixing(gelo_ctx* ctx, int m, int kind, uint64_t seed, int dtype,
                       void* A_dev, void* Ainv_dev, int lda, float* cond_dev, void* stream);

/* ---- shield rows (Mitigation 2, Eq. 7-8) --------------------------------------------- */

/* S_dev (k x d) = (scale * median_i ||H_i||_2 / sqrt(d)) * N(0,1) draws of stream 2.
 * The median of an even number of rows is the mean of the middle two.  k = 0 is a no-op.
 * Row norms use workspace scratch. */
int gelo_shield_rows(gelo_ctx* ctx, const void* H_dev, int n, int d, int k, float scale,
                     uint64_t seed, int dtype, void* S_dev, void* stream);

/* The other shield kind the paper's attack study lists (Section 4.4.1, Table 9: "Student-t"; it gives neither the
 * degrees of freedom nor a scaling, so both are read as follows).  S_dev (k x d) = (scale * median_i ||H_i||_2 /
 * sqrt(d)) * x, with x standardised Student-t draws of `nu` degrees of freedom (3 <= nu <= 63, unit variance, so the
 * expected row energy is that of the Gaussian kind): element e owns B = 4 ceil((nu + 1) / 4) consecutive positions of
 * the Gaussian stream (seed, stream 2, attempt word nu) from e * B on, t = g_0 / sqrt((g_1^2 + .. + g_nu^2) / nu),
 * x = t sqrt((nu - 2) / nu).  gelo_set_shield_student_t makes the whole-call entry points draw this kind (0 = Gaussian). */
int gelo_shield_rows_t(gelo_ctx* ctx, const void* H_dev, int n, int d, int k, float scale, uint64_t seed, int nu,
                       int dtype, void* S_dev, void* stream);
int gelo_set_shield_student_t(gelo_ctx* ctx, int nu);

/* gelo_shield_rows for callers that cannot allocate device memory, and so cannot give the
 * context a workspace: a component loaded into a process whose memory pool belongs to someone
 * else (a serving engine's plugin, a confidential-computing runtime with a frozen allocator),
 * or a call site where cudaMalloc is not allowed.  The paper has no counterpart; this is a
 * packaging variant of the Mitigation 2 step above and computes the same S.
 *
 * The row-norm scratch is a fixed array inside the library image (about 256 KiB that every
 * GPU which loads the library holds until the process exits), so:
 *   - n may be at most 65536 data rows; a larger n returns GELO_ERR_UNSUPPORTED and launches
 *     nothing.  No workspace is needed and none is touched.
 *   - the function allocates and frees nothing, on the host or on the device.
 *   - the first call on each device looks up the array's device address; make that first
 *     call outside any stream capture.
 *   - all calls on one device share the array.  Calls whose kernels may overlap on the GPU
 *     (different streams without an ordering between them) race on it: order them. */
int gelo_shield_rows_static(gelo_ctx* ctx, const void* H_dev, int n, int d, int k, float scale,
                            uint64_t seed, int dtype, void* S_dev, void* stream);

/* ---- the three products (Eq. 1-3) ------------------------------------------------------ */

/* U_dev ((n+k) x d) = A [H; S]; the stacked operand is never materialised.  S_dev may be
 * NULL iff k == 0. */
int gelo_mix(gelo_ctx* ctx, const void* A_dev, int lda, const void* H_dev, const void* S_dev,
             int n, int k, int d, int dtype, void* U_dev, void* stream);

/* Yp_dev (m x p) = U_dev (m x d) * W_dev (d x p): the offloaded GEMM; with U = H this is
 * also the plain, unprotected projection. */
int gelo_project(gelo_ctx* ctx, const void* U_dev, const void* W_dev, int m, int d, int p,
                 int dtype, void* Yp_dev, void* stream);

/* FP8 operands for the offloaded product (the paper's Limitations and Future Work name FP8 beside FP16; reading: the
 * product of Eq. 2, the one that runs on the untrusted accelerator, takes its operands in the OCP format E4M3 with one
 * fp32 scale per tensor, while mixing and unmixing stay in the 16-bit type).
 *   gelo_quantize_e4m3: codes_dev (rows x cols bytes, dense) = nearest-even E4M3 of X_dev / scale (binary32 division,
 *       saturating at +-448), scale = max|X| / 448 (1 for an all-zero tensor) written to scale_dev[0]; scale_dev must hold
 *       TWO floats (the second is scratch) and be 8-byte aligned.  X_dev: rows x cols of `dtype`, dense, cols a multiple
 *       of 16.  Weights are quantised once and reused; U is quantised per call.
 *   gelo_project_e4m3: Yp_dev (m x p bf16) = (u_scale * w_scale) * (U8 (m x d) * W8 (d x p)), fp32 accumulation on the
 *       tensor cores (kind::f8f6f4).  d and p multiples of 16.
 * With 3 mantissa bits per operand the product carries about 5% relative error (rms) against the unquantised one, and the
 * 10x shield rows bring 6x the energy of the data into Y', so after unmixing the data rows see about 12%: this path is
 * for callers that accept FP8-grade accuracy, and is checked against the fp64 product of the SAME stored codes. */
int gelo_quantize_e4m3(gelo_ctx* ctx, const void* X_dev, int rows, int cols, int dtype, void* codes_dev, float* scale_dev,
                       void* stream);
int gelo_project_e4m3(gelo_ctx* ctx, const void* U8_dev, const float* u_scale_dev, const void* W8_dev, const float* w_scale_dev,
                      int m, int d, int p, void* Yp_dev, void* stream);

/* Rows 0..n-1 of Ainv * Yp (shield rows are dropped by never computing them), split by
 * column thirds into Q_dev, K_dev, V_dev (each n x p/3; p % 3 == 0 and p/3 % 8 == 0).  If
 * K_dev and V_dev are both NULL the whole n x p result goes to Q_dev. */
int gelo_unmix(gelo_ctx* ctx, const void* Ainv_dev, int lda, const void* Yp_dev, int n, int k,
               int p, int dtype, void* Q_dev, void* K_dev, void* V_dev, void* stream);

/* Eq. 2 and Eq. 3 in one kernel for a small batch (m = n + k <= 128, 16-bit element types, p a multiple of 64 and at
 * most 128 columns per SM): every SM streams its own column slab of W_dev once, keeps its slab of Y' = U W on chip,
 * rounds it to the element type exactly as gelo_project would store it, multiplies by the first n rows of Ainv_dev and
 * writes Q | K | V as gelo_unmix does.  Results equal gelo_project followed by gelo_unmix up to the summation order
 * inside the tensor core.  GELO_ERR_UNSUPPORTED for shapes outside the limits above (use the two calls then).  The
 * whole-call entry points take this route on their own for such shapes unless gelo_set_small_batch_fusion(ctx, 0). */
int gelo_project_unmix(gelo_ctx* ctx, const void* U_dev, const void* W_dev, const void* Ainv_dev, int lda, int n, int k,
                       int d, int p, int dtype, void* Q_dev, void* K_dev, void* V_dev, void* stream);
int gelo_set_small_batch_fusion(gelo_ctx* ctx, int on);

/* ---- the whole call --------------------------------------------------------------------- */

/* sample -> shields -> mix -> project -> unmix for one batch, all from workspace scratch.
 * H_dev n x d, W_dev d x p; outputs as in gelo_unmix.  Waits for `stream` only when
 * kind is GELO_NONORTHOGONAL (condition-number verdict). */
int gelo_qkv_offload(gelo_ctx* ctx, const void* H_dev, const void* W_dev, int n, int k, int d,
                     int p, int kind, uint64_t seed, float shield_scale, int dtype,
                     void* Q_dev, void* K_dev, void* V_dev, void* stream);

/* Same call for a caller whose activations live in host memory: H_host (n x d) is copied
 * to the device, the result is copied back into Q_host, K_host, V_host (each n x p/3), and
 * the function returns after the copies have completed.  W_dev stays a device pointer
 * (weights are resident, paper Section 3.2 step 1.4). */
int gelo_qkv_offload_host(gelo_ctx* ctx, const void* H_host, const void* W_dev, int n, int k,
                          int d, int p, int kind, uint64_t seed, float shield_scale, int dtype,
                          void* Q_host, void* K_host, void* V_host, void* stream);

/* ---- batches of independent calls ---------------------------------------------------------- */

/* The same path for `calls` independent batches (for instance the Q/K/V projections of the
 * layers of one prefill sweep; paper Section 3.2 step 1.2 draws a new A for every batch and
 * never uses one twice).  Sampling A needs only the seed, so up to `lanes` calls sample
 * their mixing pairs concurrently on streams owned by the context while `stream` runs the
 * shield rows and the three products of earlier calls; results are those of gelo_qkv_offload
 * with the same (kind, seed) per call.
 *   H_dev[i] n x d, W_dev[i] d x p, kinds[i], seeds[i]: inputs of call i (host arrays of
 *   device pointers / values, read before the function returns).
 *   Q_dev[i], K_dev[i], V_dev[i]: outputs of call i, as in gelo_unmix (K_dev[i] == V_dev[i] ==
 *   NULL for all i selects unsplit output).  Calls may share output buffers; they are written
 *   in call order.
 * A small batch (n + k <= 128 on a 16-bit type, at least two lanes, outputs of different calls
 * disjoint) runs each WHOLE call on its lane, shield rows, mixing and the fused projection +
 * unmixing included, so that the weight streams of neighbouring calls overlap; `stream` then only
 * waits for the lanes at the end.  The lanes read H_dev[i] and write the outputs after the point
 * of `stream` at which the batch was enqueued.
 * Non-orthogonal calls use their first attempt only and never wait for the device: a missed
 * condition bound is reported by gelo_last_status as GELO_ERR_COND.  Needs a workspace of
 * gelo_batch_workspace_bytes(..., lanes) bytes.  Work on the lane streams is ordered after
 * everything already on `stream`, and `stream` ends up ordered after all of it. */
int gelo_qkv_offload_batch(gelo_ctx* ctx, int calls, const void* const* H_dev, const void* const* W_dev,
                           int n, int k, int d, int p, const int* kinds, const uint64_t* seeds,
                           float shield_scale, int dtype, void* const* Q_dev, void* const* K_dev,
                           void* const* V_dev, void* stream);

/* Same with activations and results in host memory (pinned memory lets the copies overlap the
 * sampling lanes): H_host[i] is copied in, Q/K/V_host[i] are copied out, and the function returns
 * after the last copy has completed. */
int gelo_qkv_offload_batch_host(gelo_ctx* ctx, int calls, const void* const* H_host,
                                const void* const* W_dev, int n, int k, int d, int p, const int* kinds,
                                const uint64_t* seeds, float shield_scale, int dtype,
                                void* const* Q_host, void* const* K_host, void* const* V_host,
                                void* stream);

/* The same call without the final wait: it returns once everything is enqueued on `stream`, and the host
 * results are valid after the caller has synchronised `stream` (the host buffers must stay alive and, for
 * the copies to be asynchronous at all, be pinned).  Back-to-back calls then keep the sampling lanes busy
 * across the seam, exactly as gelo_qkv_offload_batch does: the lanes already sample the mixing pairs of
 * the next batch while the last results of this one are still on their way to the host. */
int gelo_qkv_offload_batch_host_async(gelo_ctx* ctx, int calls, const void* const* H_host,
                                      const void* const* W_dev, int n, int k, int d, int p, const int* kinds,
                                      const uint64_t* seeds, float shield_scale, int dtype,
                                      void* const* Q_host, void* const* K_host, void* const* V_host,
                                      void* stream);

/* Number of concurrent sampling lanes of the batched calls (1..32, default 4) and the workspace
 * they need.  0 bytes if an argument is invalid. */
int gelo_set_lanes(gelo_ctx* ctx, int lanes);
/* In batches with at least `share` lanes every tensor-core update of the factorisations runs on 1/share of
 * the SMs (default 4; 1 = always all SMs), so that the updates of different lanes overlap instead of queueing
 * behind each other's launch and drain phases. */
int gelo_set_lane_share(gelo_ctx* ctx, int share);
size_t gelo_batch_workspace_bytes(int n, int k, int d, int p, int dtype, int lanes);

/* ---- structured variant: block-diagonal orthogonal mixing -------------------------------------- */

/* The same offload with a block-diagonal orthogonal A (the paper names structured orthogonal transforms as
 * future work for cheaper A-generation; this is one such structure, NOT the dense mixing of its Section 3.2).
 * The m = n + k rows are dealt into nb = ceil(m / block) groups (block a multiple of 64, nb <= lanes, n >= nb);
 * group j holds data rows [n j / nb, n (j+1) / nb) and shield rows [k j / nb, k (j+1) / nb), i.e. every group
 * mixes its share of the shield rows with its data rows, and gets an independent Haar-orthogonal A_j from a
 * Householder QR (seed of the call combined with j).  Rows mix only inside their group: an observer of U learns
 * which group a row belongs to, so this trades part of the hiding for cost: A-generation nb (8/3) block^3 instead
 * of (8/3) m^3 flops, mixing and unmixing 2 m block (d + p) instead of 2 m^2 (d + p).  The result is H W as
 * before.  Arguments as gelo_qkv_offload_batch (orthogonal kind only); workspace
 * gelo_blockdiag_workspace_bytes(..., block, lanes), 0 if the sizes are not supported. */
size_t gelo_blockdiag_workspace_bytes(int n, int k, int d, int p, int dtype, int block, int lanes);
int gelo_qkv_offload_blockdiag_batch(gelo_ctx* ctx, int calls, const void* const* H_dev, const void* const* W_dev,
                                     int n, int k, int d, int p, int block, const uint64_t* seeds,
                                     float shield_scale, int dtype, void* const* Q_dev, void* const* K_dev,
                                     void* const* V_dev, void* stream);

/* ---- per-launch timing (measurement aid; no counterpart in the paper) ----------------------- */

/* Between gelo_profile_start and gelo_profile_stop every launch of the main kernel classes is
 * bracketed by CUDA events on its own stream.  gelo_profile_stop waits for `stream` and the lane
 * streams and fills out[3 * c + {0, 1, 2}] = {launches, summed milliseconds, summed algorithmic
 * work} for class c: 0 rank-32 update (bytes), 1 V^T C product (bytes), 2 tensor-core GEMM
 * (flops), 3 QR panel (flops), 4 LU panel (flops).  `out` holds 15 doubles.  Timing mode creates
 * events per launch; keep it out of measured regions. */
int gelo_profile_start(gelo_ctx* ctx);
int gelo_profile_stop(gelo_ctx* ctx, void* stream, double* out);

#ifdef __cplusplus
}
#endif
#endif /* GELO_H */
