// bf16 tensor-core GEMM on sm_100a: tcgen05.mma with the accumulator in tensor memory, operands
// staged in shared memory by TMA, fp32 accumulation.  It serves
//   * the three products of the offload (Eq. 1-3): C = A B with bf16 operands and bf16 output,
//     the B operand optionally the stack [H; S] of Eq. 8, the output optionally split Q | K | V;
//   * the level-3 updates of the blocked QR / LU behind the sampling of A: fp32 matrices are held
//     as a bf16 (high, low) pair and the product is accumulated as hi*hi + hi*lo + lo*hi in fp32,
//     with an epilogue that either subtracts the result from an fp32 matrix in place or writes it
//     as a new (high, low) pair;
//   * the same level-3 updates in one product of kind::tf32 straight from the fp32 matrices (no operand
//     conversion passes at all): the A operand is either K-major (a row-major M x K matrix) or MN-major
//     (the transpose of a row-major K x M matrix, which is how V^T C reads the reflectors).
//
//   C (M x N)  (+)=  sum over segments s of  A_s (M x K_s, row-major)  *  B_s (K_s x N, row-major)
//
// * A tiles (128 rows x 64 k) land K-major, B tiles (64 k x BN columns, as 64-column boxes) land
//   N-major; both use the 128-byte swizzle that TMA writes and the MMA reads.
// * A segment names one A tensor map, one B tensor map and a starting k for each; the stacked
//   operand of the mixing product is two segments, a split-precision product is three.  TMA's
//   out-of-bounds zero fill handles every ragged edge (including a seam inside a k-block).
// * Persistent CTAs (one per SM), warp-specialised: warp 0 issues TMA, warp 1 issues MMA and owns
//   the tensor-memory allocation, warps 2-9 drain the accumulator (two warps per TMEM lane
//   quarter, half of the columns each).  Two accumulator stages let the epilogue of one tile
//   overlap the main loop of the next.
// * Every wait on an mbarrier is bounded in time (the context's wait limit, two seconds by default,
//   measured on the GPU's global timer); on expiry the CTA records GELO_ERR_TIMEOUT in the
//   context's status word, stops issuing work, releases tensor memory and returns.
#include <cuda.h>

#include "common.cuh"
#include "tc_ptx.cuh"

namespace gelo {

namespace {

using namespace tcx;

constexpr int BM = 128;
constexpr int BK = 64;
constexpr int kAccStages = 2;
constexpr int kEpiWarps = 8;
constexpr int kThreads = 64 + 32 * kEpiWarps;
constexpr uint32_t kABytes = BM * BK * 2;            // 16 KiB
constexpr uint32_t kTmemCols = 512;

enum TcMode { TC_STORE_BF16 = 0, TC_STORE_F32 = 1, TC_SUB_F32 = 2, TC_EMIT_SPLIT = 3, TC_STORE_SYM16 = 4 };

struct TcSegment { int a_sel, b_sel, a_k0, b_row0, kb; };

struct TcParams {
    int M, N;
    int nseg;
    TcSegment seg[3];
    int mode;
    void* C0; void* C1; void* C2;   // STORE_*: column-split outputs; SUB_F32: C0 fp32, C1/C2 optional hi/lo; EMIT_SPLIT: C0 hi, C1 lo
    int ldc, csplit, lde;           // lde: row stride of the hi/lo matrices written next to an fp32 C
    int ksplit, kb_per_split;       // K slices (TC_STORE_F32 only): slice q covers k-blocks [q*kb_per_split, ...) of every segment
    long long plane;                // and writes plane q of C0 (stride in elements)
    int round_tf32;                 // TC_STORE_F32: round the stored values to tf32 (they feed a later tf32 product)
    float out_scale;                // TC_STORE_F32 with round_tf32: factor applied before the rounding
    float diag_sub;                 // TC_STORE_F32 with round_tf32: subtracted from the scaled diagonal entries
    float post_scale;               //   ... and the factor applied after that: out = post_scale * (out_scale * acc - diag_sub [row == col])
    int a3d, b3d;                   // the MN-major A tile / the B tile arrives as ONE three-dimensional box (see make_map_nmajor)
    int out_f16;                    // TC_STORE_BF16: operands and output are IEEE half instead of bfloat16
    const float* scale_a;           // TC_STORE_BF16 with 8-bit operands: the per-tensor scales (device scalars); the
    const float* scale_b;           //   accumulator is multiplied by their product before it is rounded
    int tri, tri_tiles;             // TC_STORE_SYM16: the result is symmetric; only the tri_tiles tiles that reach the diagonal or lie
                                    // above it are computed, and what lies below them is filled in by mirroring
    uint32_t idesc;                 // instruction descriptor (filled in by the launcher)
    unsigned long long wait_ns;     // limit of every mbarrier wait, nanoseconds (filled in by the launcher from the context)
    int* status;
};

// Epilogue staging for the in-place subtraction: every epilogue warp owns two 32 x 32 fp32 boxes (4 KiB each)
// that TMA reduces into global memory.
constexpr uint32_t kStageBoxBytes = 32 * 32 * 4;
constexpr uint32_t kStagingBytes = kEpiWarps * 2 * kStageBoxBytes;

// A stage holds 128 bytes of k per A row (64 bf16 or 32 tf32 values) and the matching B rows, so both kinds share
// the shared-memory geometry: kTf32 only changes the element count per k-block, the box width of the N-major B tile
// (128 bytes = 64 bf16 or 32 fp32 columns) and the instruction.  kAMn (tf32 only): the A tile arrives as four
// boxes of 32 m-columns x 32 k-rows, i.e. laid out exactly like a 128-column B tile.
template <int BN, int kStages, bool kStaging, bool kTf32 = false, bool kAMn = false, bool kF8 = false>
struct TcCfg {
    static constexpr uint32_t kStagingUsed = kStaging ? kStagingBytes : 0u;
    static constexpr int kBKE = kF8 ? 128 : (kTf32 ? 32 : 64);             // elements of k per stage
    static constexpr int kBoxCols = kF8 ? 128 : (kTf32 ? 32 : 64);         // columns of one N-major box (128 bytes)
    static constexpr uint32_t kBoxBytes = (uint32_t)kBKE * 128u;           // one N-major box: kBKE rows of 128 bytes
    static constexpr uint32_t kBBytes = (BN / kBoxCols) * kBoxBytes;
    static constexpr uint32_t kStageBytes = kABytes + kBBytes;
    static constexpr uint32_t kSmemBytes = kStages * kStageBytes + kStagingUsed + 1024 /*alignment slack*/ + 256 /*barriers*/;
    // k advance per instruction inside an N-major (or MN-major A) tile: 16 bf16 rows or 8 tf32 rows of 128 bytes
    static constexpr uint32_t kMnStep = kF8 ? 4096u : (kTf32 ? 1024u : 2048u);   // 32 e4m3 rows, 16 bf16 rows or 8 tf32 rows
    // N-major tiles: bf16 in the 16-byte-chunk swizzle (atoms of 8 k-rows, 1024 bytes), fp32 in the 32-byte-chunk
    // swizzle (atoms of 4 k-rows, 512 bytes)
    static constexpr uint32_t kMnLayout = kTf32 ? 1u : 2u;
    static constexpr uint32_t kMnSbo = kTf32 ? 512u : 1024u;
    // Instruction descriptor: fp32 accumulate, operand formats (1 = bf16, 2 = tf32), A K-major or MN-major,
    // B N-major, M = 128, N = BN.
    static constexpr uint32_t kFmt = kF8 ? 0u : (kTf32 ? 2u : 1u);         // kind::f8f6f4: 0 = E4M3
    static constexpr uint32_t kInstrDesc = (1u << 4) | (kFmt << 7) | (kFmt << 10) | ((kAMn ? 1u : 0u) << 15) | (1u << 16) |
                                           ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
    static_assert(!kAMn || kTf32, "MN-major A is only wired up for the tf32 kind");
    static_assert(!(kF8 && kTf32), "one operand kind per instance");
};

// x = hi + lo with hi = bf16(x), lo = bf16(x - hi)
__device__ __forceinline__ void split2(float a, float b, uint32_t& hi, uint32_t& lo)
{
    const __nv_bfloat162 h = __floats2bfloat162_rn(a, b);
    const float2 hf = __bfloat1622float2(h);
    const __nv_bfloat162 l = __floats2bfloat162_rn(a - hf.x, b - hf.y);
    hi = *reinterpret_cast<const uint32_t*>(&h);
    lo = *reinterpret_cast<const uint32_t*>(&l);
}

// Row-tile and column-tile index of work item `tile`.  Ordinary products: row tiles fastest, then column tiles, then K
// slices.  Symmetric products (prm.tri, 128 x 256 tiles): column tile nt owns the row tiles mt <= 2 nt + 1, i.e. those
// whose first row is not below the tile's last column; they are enumerated column tile after column tile.
__device__ __forceinline__ void tile_coords(const TcParams& prm, int tile, int m_tiles, int mn_tiles, int& mt, int& nt, int& slice)
{
    if (prm.tri) {
        int t = tile;
        nt = 0;
        for (;;) {
            const int cnt = min(m_tiles, 2 * nt + 2);
            if (t < cnt) break;
            t -= cnt; ++nt;
        }
        mt = t; slice = 0;
        return;
    }
    const int mn = tile % mn_tiles;
    slice = tile / mn_tiles;
    mt = mn % m_tiles;
    nt = mn / m_tiles;
}

// One 8-column group of the epilogue: w[G*8 .. G*8+7] are the fp32 accumulator values of row gm, columns
// gn..gn+7 (G is a template parameter so that the register array is indexed by constants only).
template <int G>
__device__ __forceinline__ void epilogue_group(const TcParams& prm, int gm, int gn, const uint32_t (&w)[32], int slice)
{
    const uint32_t v[8] = {w[G * 8 + 0], w[G * 8 + 1], w[G * 8 + 2], w[G * 8 + 3],
                           w[G * 8 + 4], w[G * 8 + 5], w[G * 8 + 6], w[G * 8 + 7]};
    if (prm.mode == TC_STORE_BF16) {
        const uint32_t (&v0)[8] = v;
        const int chunk = gn / prm.csplit;
        void* base = chunk == 0 ? prm.C0 : (chunk == 1 ? prm.C1 : prm.C2);
        const size_t off = (size_t)gm * prm.ldc + (gn - chunk * prm.csplit);
        uint32_t v[8] = {v0[0], v0[1], v0[2], v0[3], v0[4], v0[5], v0[6], v0[7]};
        if (prm.scale_a) {
            const float sc = prm.scale_a[0] * prm.scale_b[0];
#pragma unroll
            for (int j = 0; j < 8; ++j) v[j] = __float_as_uint(sc * __uint_as_float(v[j]));
        }
        uint4 pk;
        if (prm.out_f16) {
            pk.x = pack_f16(v[0], v[1]); pk.y = pack_f16(v[2], v[3]);
            pk.z = pack_f16(v[4], v[5]); pk.w = pack_f16(v[6], v[7]);
        } else {
            pk.x = pack_bf16(v[0], v[1]); pk.y = pack_bf16(v[2], v[3]);
            pk.z = pack_bf16(v[4], v[5]); pk.w = pack_bf16(v[6], v[7]);
        }
        *reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(base) + off) = pk;
    } else if (prm.mode == TC_STORE_F32) {
        const int chunk = gn / prm.csplit;                    // column block -> C0 / C1 / C2 (0 unless the output is split)
        float* base = static_cast<float*>(chunk == 0 ? prm.C0 : (chunk == 1 ? prm.C1 : prm.C2));
        float4* dst = reinterpret_cast<float4*>(base + (size_t)slice * prm.plane + (size_t)gm * prm.ldc + (gn - chunk * prm.csplit));
        float f[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const float a = __uint_as_float(v[j]);
            f[j] = prm.round_tf32 ? round_tf32(prm.post_scale * (prm.out_scale * a - ((gm == gn + j) ? prm.diag_sub : 0.0f))) : a;
        }
        dst[0] = make_float4(f[0], f[1], f[2], f[3]);
        dst[1] = make_float4(f[4], f[5], f[6], f[7]);
    } else if (prm.mode == TC_EMIT_SPLIT) {
        uint4 hi, lo;
        split2(__uint_as_float(v[0]), __uint_as_float(v[1]), hi.x, lo.x);
        split2(__uint_as_float(v[2]), __uint_as_float(v[3]), hi.y, lo.y);
        split2(__uint_as_float(v[4]), __uint_as_float(v[5]), hi.z, lo.z);
        split2(__uint_as_float(v[6]), __uint_as_float(v[7]), hi.w, lo.w);
        const size_t off = (size_t)gm * prm.ldc + gn;
        *reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(prm.C0) + off) = hi;
        *reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(prm.C1) + off) = lo;
    }
}

// Symmetric result (TC_STORE_SYM16): 32 consecutive entries of row gm from column gn on, as
// post_scale * (out_scale * acc - diag_sub [on the diagonal]) in bf16.  Entries above the diagonal whose mirror image
// lies in a tile that is not computed (see tile_coords) are also written there; consecutive lanes hold consecutive
// rows, so those transposed stores are contiguous across the warp.
__device__ __forceinline__ void store_symmetric(const TcParams& prm, int gm, int gn, const uint32_t (&v)[32])
{
    __nv_bfloat16* D = static_cast<__nv_bfloat16*>(prm.C0);
    __align__(16) __nv_bfloat16 h[32];
#pragma unroll
    for (int j = 0; j < 32; ++j)
        h[j] = __float2bfloat16_rn(prm.post_scale * (prm.out_scale * __uint_as_float(v[j]) - ((gm == gn + j) ? prm.diag_sub : 0.0f)));
#pragma unroll
    for (int g = 0; g < 4; ++g)
        if (gn + 8 * g < prm.N)
            *reinterpret_cast<uint4*>(D + (size_t)gm * prm.ldc + gn + 8 * g) = *reinterpret_cast<const uint4*>(&h[8 * g]);
    const int my_pair = gm >> 8;                              // column tile of the mirrored entry
#pragma unroll
    for (int j = 0; j < 32; ++j) {
        const int c = gn + j;
        if (c > gm && c < prm.M && (c >> 7) > 2 * my_pair + 1) D[(size_t)c * prm.ldc + gm] = h[j];
    }
}

template <int BN, int kStages, bool kStaging, bool kTf32, bool kAMn, bool kF8>
__global__ void __launch_bounds__(kThreads, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap map_a0, const __grid_constant__ CUtensorMap map_a1,
               const __grid_constant__ CUtensorMap map_b0, const __grid_constant__ CUtensorMap map_b1,
               const __grid_constant__ CUtensorMap map_c, const TcParams prm)
{
    using Cfg = TcCfg<BN, kStages, kStaging, kTf32, kAMn, kF8>;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t tiles_base = (raw + 1023u) & ~1023u;                 // swizzle atoms need 1024-byte alignment
    uint8_t* gen_base = smem_raw + (tiles_base - raw);
    const uint32_t staging_base = tiles_base + kStages * Cfg::kStageBytes;      // 1024-byte aligned
    const uint32_t bar_base = staging_base + Cfg::kStagingUsed;
    uint8_t* bar_gen = gen_base + kStages * Cfg::kStageBytes + Cfg::kStagingUsed;
    // barrier layout (8 bytes each): full[kStages], empty[kStages], acc_full[2], acc_empty[2]; then tmem slot, abort
    auto full_bar = [&](int s) { return bar_base + 8u * s; };
    auto empty_bar = [&](int s) { return bar_base + 8u * (kStages + s); };
    auto acc_full_bar = [&](int a) { return bar_base + 8u * (2 * kStages + a); };
    auto acc_empty_bar = [&](int a) { return bar_base + 8u * (2 * kStages + kAccStages + a); };
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(bar_gen + 8 * (2 * kStages + 2 * kAccStages));
    volatile int* abort_flag = reinterpret_cast<volatile int*>(bar_gen + 8 * (2 * kStages + 2 * kAccStages) + 8);

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;

    const int m_tiles = (prm.M + BM - 1) / BM;
    const int n_tiles = (prm.N + BN - 1) / BN;
    const int mn_tiles = m_tiles * n_tiles;
    const int total_tiles = prm.tri ? prm.tri_tiles : mn_tiles * prm.ksplit;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        for (int a = 0; a < kAccStages; ++a) { mbar_init(acc_full_bar(a), 1); mbar_init(acc_empty_bar(a), kEpiWarps); }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32((const void*)tmem_slot)), "r"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        // ================= TMA producer =================
        if (lane == 0) {
            uint32_t it = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x) {
                int mt, nt, slice;
                tile_coords(prm, tile, m_tiles, mn_tiles, mt, nt, slice);
                const int m0 = mt * BM, n0 = nt * BN;
#pragma unroll
                for (int sg = 0; sg < 3; ++sg) {              // constant indices keep the parameters out of local memory
                    if (sg >= prm.nseg || !ok) break;
                    const TcSegment seg = prm.seg[sg];
                    const CUtensorMap* ma = seg.a_sel ? &map_a1 : &map_a0;
                    const CUtensorMap* mb = seg.b_sel ? &map_b1 : &map_b0;
                    const int kb_lo = slice * prm.kb_per_split;
                    const int kb_hi = min(seg.kb, kb_lo + prm.kb_per_split);
                    for (int kb = kb_lo; kb < kb_hi; ++kb, ++it) {
                        const int s = it % kStages;
                        const uint32_t ph = (it / kStages) & 1u;
                        if (!mbar_wait(empty_bar(s), ph ^ 1u, abort_flag, prm.wait_ns)) { ok = false; break; }
                        const uint32_t sa = tiles_base + s * Cfg::kStageBytes;
                        const uint32_t sb = sa + kABytes;
                        mbar_expect_tx(full_bar(s), Cfg::kStageBytes);
                        if (kAMn) {
                            if (prm.a3d) {
                                tma_load_3d(sa, ma, 0, seg.a_k0 + kb * Cfg::kBKE, m0 / Cfg::kBoxCols, full_bar(s));
                            } else {
#pragma unroll
                                for (int j = 0; j < BM / Cfg::kBoxCols; ++j)
                                    tma_load_2d(sa + j * Cfg::kBoxBytes, ma, m0 + j * Cfg::kBoxCols, seg.a_k0 + kb * Cfg::kBKE, full_bar(s));
                            }
                        } else {
                            tma_load_2d(sa, ma, seg.a_k0 + kb * Cfg::kBKE, m0, full_bar(s));
                        }
                        if (prm.b3d) {
                            tma_load_3d(sb, mb, 0, seg.b_row0 + kb * Cfg::kBKE, n0 / Cfg::kBoxCols, full_bar(s));
                        } else {
#pragma unroll
                            for (int j = 0; j < BN / Cfg::kBoxCols; ++j)
                                tma_load_2d(sb + j * Cfg::kBoxBytes, mb, n0 + j * Cfg::kBoxCols, seg.b_row0 + kb * Cfg::kBKE, full_bar(s));
                        }
                    }
                }
            }
            if (!ok) { *abort_flag = 1; atomicCAS(prm.status, 0, (int)GELO_ERR_TIMEOUT); }
        }
    } else if (warp == 1) {
        // ================= MMA issuer =================
        if (lane == 0) {
            uint32_t acc_it = 0;
            uint32_t s = 0, ph = 0;                   // operand stage and the parity of its "full" phase
            bool ready = false;                       // stage s is already known to be full (tested ahead, see tc_mma4_*_try)
            bool ok = true;
            // k advance per instruction in sixteen-byte units of the descriptors' start address
            constexpr uint64_t kAStep = kAMn ? (Cfg::kMnStep >> 4) : 2, kBStep = Cfg::kMnStep >> 4;
            for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x, ++acc_it) {
                const int slice = prm.tri ? 0 : tile / mn_tiles;
                int kb_total = 0;
#pragma unroll
                for (int sg = 0; sg < 3; ++sg)
                    if (sg < prm.nseg) {
                        const int kb_lo = slice * prm.kb_per_split;
                        const int kb_hi = min(prm.seg[sg].kb, kb_lo + prm.kb_per_split);
                        kb_total += max(0, kb_hi - kb_lo);
                    }
                const int a = acc_it % kAccStages;
                const uint32_t aph = (acc_it / kAccStages) & 1u;
                if (!mbar_wait(acc_empty_bar(a), aph ^ 1u, abort_flag, prm.wait_ns)) { ok = false; break; }
                tc_fence_after();
                const uint32_t tmem_d = tmem_base + (uint32_t)(a * BN);
                for (int kb = 0; kb < kb_total; ++kb) {
                    if (!ready && !mbar_wait(full_bar(s), ph, abort_flag, prm.wait_ns)) { ok = false; break; }
                    const uint32_t sa = tiles_base + s * Cfg::kStageBytes;
                    const uint32_t sb = sa + kABytes;
                    // A K-major: 8-row groups 1024 bytes apart, 32 bytes per k step.  A MN-major: like B.
                    const uint64_t da = kAMn ? smem_desc(sa, Cfg::kBoxBytes, Cfg::kMnSbo, Cfg::kMnLayout) : smem_desc(sa, 16, 1024);
                    // B: N-major, 128-byte-wide boxes kBoxBytes apart, k-row atoms kMnSbo bytes apart
                    const uint64_t db = smem_desc(sb, Cfg::kBoxBytes, Cfg::kMnSbo, Cfg::kMnLayout);
                    const uint32_t ns = (s + 1 == kStages) ? 0u : s + 1;
                    const uint32_t nph = (ns == 0u) ? (ph ^ 1u) : ph;
                    // four instructions of 32 bytes of k (16 bf16 / 8 tf32) per stage
                    ready = kF8 ? tc_mma4_f8_try(tmem_d, da, db, kAStep, kBStep, prm.idesc, kb != 0 ? 1u : 0u, full_bar(ns), nph)
                          : kTf32 ? tc_mma4_tf32_try(tmem_d, da, db, kAStep, kBStep, prm.idesc, kb != 0 ? 1u : 0u, full_bar(ns), nph)
                                  : tc_mma4_bf16_try(tmem_d, da, db, kAStep, kBStep, prm.idesc, kb != 0 ? 1u : 0u, full_bar(ns), nph);
                    tc_commit(empty_bar(s));          // frees the stage once these MMAs have read it
                    s = ns; ph = nph;
                }
                if (!ok) break;
                tc_commit(acc_full_bar(a));           // accumulator complete
            }
            if (!ok) { *abort_flag = 1; atomicCAS(prm.status, 0, (int)GELO_ERR_TIMEOUT); }
        }
    } else {
        // ================= epilogue (warps 2..9) =================
        const int quarter = warp & 3;                 // the TMEM lane quarter this warp may read
        const int half = (warp - 2) >> 2;             // which half of the tile's columns
        constexpr int kHalfCols = BN / 2;
        uint32_t acc_it = 0, box_it = 0;
        bool ok = true;
        for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x, ++acc_it) {
            const int a = acc_it % kAccStages;
            const uint32_t aph = (acc_it / kAccStages) & 1u;
            int mt, nt, slice;
            tile_coords(prm, tile, m_tiles, mn_tiles, mt, nt, slice);
            const int m0 = mt * BM, n0 = nt * BN;
            const int gm = m0 + quarter * 32 + lane;
            const bool row_ok = gm < prm.M;
            if (kStaging && prm.mode == TC_SUB_F32) {
                // C -= acc without reading C: the negated accumulator goes through a swizzled shared-memory box and
                // a TMA reduce-add into global memory (the addition happens at the L2); TMA clips at the matrix edge
                if (!mbar_wait(acc_full_bar(a), aph, abort_flag, prm.wait_ns)) { ok = false; break; }
                tc_fence_after();
                const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(a * BN);
                const uint32_t my_staging = staging_base + (uint32_t)(warp - 2) * 2u * kStageBoxBytes;
#pragma unroll 1
                for (int c = half * kHalfCols; c < (half + 1) * kHalfCols; c += 32, ++box_it) {
                    const uint32_t buf = my_staging + (box_it & 1u) * kStageBoxBytes;
                    if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");   // box of two chunks ago is free
                    __syncwarp();
                    uint32_t v[32];
                    tc_ld_32cols(taddr + c, v);
                    tc_ld_wait();
#pragma unroll
                    for (int j4 = 0; j4 < 8; ++j4) {
                        const uint32_t dst = buf + (uint32_t)lane * 128u + (uint32_t)((j4 ^ (lane & 7)) << 4);
                        asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};"
                                     ::"r"(dst), "f"(-__uint_as_float(v[4 * j4 + 0])), "f"(-__uint_as_float(v[4 * j4 + 1])),
                                       "f"(-__uint_as_float(v[4 * j4 + 2])), "f"(-__uint_as_float(v[4 * j4 + 3])) : "memory");
                    }
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                    __syncwarp();
                    if (lane == 0 && n0 + c < prm.N && m0 + quarter * 32 < prm.M) {
                        asm volatile(
                            "cp.reduce.async.bulk.tensor.2d.global.shared::cta.add.tile.bulk_group [%0, {%1, %2}], [%3];"
                            ::"l"(&map_c), "r"(n0 + c), "r"(m0 + quarter * 32), "r"(buf) : "memory");
                    }
                    if (lane == 0) asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                }
            } else {
                if (!mbar_wait(acc_full_bar(a), aph, abort_flag, prm.wait_ns)) { ok = false; break; }
                tc_fence_after();
                const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(a * BN);
#pragma unroll 1
                for (int c = half * kHalfCols; c < (half + 1) * kHalfCols; c += 32) {
                    uint32_t v[32];
                    tc_ld_32cols(taddr + c, v);
                    tc_ld_wait();
                    if (prm.mode == TC_STORE_SYM16) {
                        if (row_ok) store_symmetric(prm, gm, n0 + c, v);
                    } else if (row_ok) {
                        const int gn = n0 + c;
                        if (gn < prm.N) epilogue_group<0>(prm, gm, gn, v, slice);
                        if (gn + 8 < prm.N) epilogue_group<1>(prm, gm, gn + 8, v, slice);
                        if (gn + 16 < prm.N) epilogue_group<2>(prm, gm, gn + 16, v, slice);
                        if (gn + 24 < prm.N) epilogue_group<3>(prm, gm, gn + 24, v, slice);
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(acc_empty_bar(a));
        }
        if (lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");   // staged boxes fully written out
        if (!ok && lane == 0) { *abort_flag = 1; atomicCAS(prm.status, 0, (int)GELO_ERR_TIMEOUT); }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
    }
}

// ---- host side ----------------------------------------------------------------------------------

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// 2-D bf16 tensor map over a row-major matrix: `cols` contiguous elements per row, `rows` rows,
// row stride `ld` elements; box = box_cols x box_rows; 128-byte swizzle; zero fill out of bounds.
bool make_map(gelo_ctx* ctx, CUtensorMap* map, const void* ptr, uint64_t cols, uint64_t rows, uint64_t ld,
              uint32_t box_cols, uint32_t box_rows)
{
    EncodeTiledFn enc = reinterpret_cast<EncodeTiledFn>(ctx->tmap_encode);
    if (!enc) return false;
    const cuuint64_t dims[2] = { cols, rows };
    const cuuint64_t strides[1] = { ld * 2 };
    const cuuint32_t box[2] = { box_cols, box_rows };
    const cuuint32_t estr[2] = { 1, 1 };
    // (the copy engine only needs the element size and a zero fill: the same map serves IEEE half data)
    return enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Tensor map of an N-major operand tile: `box_rows` rows of k, `tile_cols` columns, held in shared memory as
// tile_cols / box_cols slabs of box_rows x 128 bytes (box_cols = 128 bytes of columns).  Where the rows are long
// enough, the matrix is described as a THREE-dimensional tensor {128 bytes of columns, rows, 128-byte column chunks}
// (strides: one row, 128 bytes), so that one copy instruction brings the whole tile in exactly that slab order; the
// producer thread then issues two copies per stage instead of up to nine (measured: 8% on the tf32 updates, nothing
// on the bf16 products).  In this view the last chunk of a row is read to its end even where it runs past
// `cols`, so it needs ld >= cols rounded up to a chunk (those columns only produce output columns that are never
// stored); otherwise *three_d = false and the map is the plain two-dimensional one (one copy per slab, zero fill
// past `cols`).  Rows past `rows` and chunks past the last one are zero-filled either way.
bool make_map_nmajor(gelo_ctx* ctx, CUtensorMap* map, const void* ptr, int elem_bytes, bool chunk32, uint64_t cols,
                     uint64_t rows, uint64_t ld, uint32_t box_rows, uint32_t tile_cols, bool* three_d)
{
    EncodeTiledFn enc = reinterpret_cast<EncodeTiledFn>(ctx->tmap_encode);
    if (!enc) return false;
    const uint32_t box_cols = 128u / (uint32_t)elem_bytes;
    const CUtensorMapDataType dt = elem_bytes == 4 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32
                                 : elem_bytes == 1 ? CU_TENSOR_MAP_DATA_TYPE_UINT8 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16;
    const CUtensorMapSwizzle sw = chunk32 ? CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B : CU_TENSOR_MAP_SWIZZLE_128B;
    const uint64_t chunks = (cols + box_cols - 1) / box_cols;
    if (ctx->tma_3d && ld >= chunks * box_cols && tile_cols / box_cols > 1) {
        const cuuint64_t dims[3] = { box_cols, rows, chunks };
        const cuuint64_t strides[2] = { ld * (uint64_t)elem_bytes, 128 };
        const cuuint32_t box[3] = { box_cols, box_rows, tile_cols / box_cols };
        const cuuint32_t estr[3] = { 1, 1, 1 };
        if (enc(map, dt, 3, const_cast<void*>(ptr), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, sw,
                CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS) {
            *three_d = true;
            return true;
        }
    }
    *three_d = false;
    const cuuint64_t dims[2] = { cols, rows };
    const cuuint64_t strides[1] = { ld * (uint64_t)elem_bytes };
    const cuuint32_t box[2] = { box_cols, box_rows };
    const cuuint32_t estr[2] = { 1, 1 };
    return enc(map, dt, 2, const_cast<void*>(ptr), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, sw,
               CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int BN, int kStages, bool kStaging, bool kTf32 = false, bool kAMn = false, bool kF8 = false>
int launch_tiles(gelo_ctx* ctx, const CUtensorMap& a0, const CUtensorMap& a1, const CUtensorMap& b0,
                 const CUtensorMap& b1, const CUtensorMap& c, const TcParams& p, double flops, cudaStream_t st)
{
    using Cfg = TcCfg<BN, kStages, kStaging, kTf32, kAMn, kF8>;
    static_assert(Cfg::kSmemBytes <= 227 * 1024, "shared memory budget");
    static bool attr_done[64] = {};
    if (ctx->device >= 0 && ctx->device < 64 && !attr_done[ctx->device]) {
        GELO_CUDA_OK(cudaFuncSetAttribute(gemm_tc_kernel<BN, kStages, kStaging, kTf32, kAMn, kF8>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                          (int)Cfg::kSmemBytes));
        attr_done[ctx->device] = true;
    }
    const int tiles = ceil_div(p.M, BM) * ceil_div(p.N, BN) * p.ksplit;
    int grid = tiles < ctx->sm_count ? tiles : ctx->sm_count;
    if (p.mode != TC_STORE_BF16 && ctx->tc_update_ctas > 0 && grid > ctx->tc_update_ctas) grid = ctx->tc_update_ctas;
    TcParams q = p;
    // both operands of a kind::f16 instruction have the same 16-bit format: 1 = bfloat16, 0 = IEEE half
    q.wait_ns = ctx->wait_limit_ns;
    q.idesc = (!kTf32 && !kF8 && p.out_f16) ? (Cfg::kInstrDesc & ~((7u << 7) | (7u << 10))) : Cfg::kInstrDesc;
    {
        ProfScope ps(ctx, PROF_GEMM_TC, flops, st);
        gemm_tc_kernel<BN, kStages, kStaging, kTf32, kAMn, kF8><<<grid, kThreads, Cfg::kSmemBytes, st>>>(a0, a1, b0, b1, c, q);
    }
    return after_launch(ctx);
}

// fp32 tensor map of the matrix that the subtracting epilogue reduces into: 32 x 32 boxes, 128-byte swizzle.
bool make_map_f32_box(gelo_ctx* ctx, CUtensorMap* map, const void* ptr, uint64_t cols, uint64_t rows, uint64_t ld,
                      uint32_t box_rows = 32, bool chunk32 = false)
{
    EncodeTiledFn enc = reinterpret_cast<EncodeTiledFn>(ctx->tmap_encode);
    if (!enc) return false;
    const cuuint64_t dims[2] = { cols, rows };
    const cuuint64_t strides[1] = { ld * 4 };
    const cuuint32_t box[2] = { 32, box_rows };
    const cuuint32_t estr[2] = { 1, 1 };
    // chunk32: the 128-byte swizzle that moves 32-byte chunks, which the MMA wants for fp32 tiles that are not K-major
    return enc(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<void*>(ptr), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, chunk32 ? CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B : CU_TENSOR_MAP_SWIZZLE_128B,
               CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

bool gemm_tc_supports(const GemmArgs& g)
{
    if (g.dtype == GELO_F32 || g.transA || g.transB || g.alpha != 1.0f || g.beta != 0.0f) return false;
    if (g.M <= 0 || g.N <= 0 || g.K <= 0) return false;
    if ((g.lda % 8) || (g.ldb % 8) || (g.ldc % 8) || (g.N % 8)) return false;
    if (g.nsplit < 1 || g.nsplit > 3 || g.N % g.nsplit || ((g.N / g.nsplit) % 8)) return false;
    if (!aligned16(g.A) || !aligned16(g.B) || (g.B2 && !aligned16(g.B2))) return false;
    for (int i = 0; i < g.nsplit; ++i)
        if (!g.C[i] || !aligned16(g.C[i])) return false;
    if (g.B2 && (g.b_split <= 0 || g.b_split >= g.K)) return false;
    return true;
}

int launch_gemm_tc(gelo_ctx* ctx, const GemmArgs& g, cudaStream_t st)
{
    if (!gemm_tc_supports(g)) return GELO_ERR_UNSUPPORTED;
    if (!ctx->tmap_encode) return GELO_ERR_CUDA;
    constexpr int BN = 256;
    const int rows_first = g.B2 ? g.b_split : g.K;
    CUtensorMap ma, mb, mb2;
    if (!make_map(ctx, &ma, g.A, (uint64_t)g.K, (uint64_t)g.M, (uint64_t)g.lda, BK, BM)) return GELO_ERR_CUDA;
    bool b3d = false, b3d2 = false;
    if (!make_map_nmajor(ctx, &mb, g.B, 2, false, (uint64_t)g.N, (uint64_t)rows_first, (uint64_t)g.ldb, BK, BN, &b3d)) return GELO_ERR_CUDA;
    if (g.B2) {
        if (!make_map_nmajor(ctx, &mb2, g.B2, 2, false, (uint64_t)g.N, (uint64_t)(g.K - g.b_split), (uint64_t)g.ldb, BK, BN, &b3d2))
            return GELO_ERR_CUDA;
        if (b3d2 != b3d) return GELO_ERR_CUDA;                // same width and stride: the same decision
    } else {
        mb2 = mb;
    }
    TcParams p = {};
    p.M = g.M; p.N = g.N;
    p.nseg = 1;
    p.seg[0] = TcSegment{0, 0, 0, 0, ceil_div(rows_first, BK)};
    if (g.B2) {
        const int a_k0 = g.b_split & ~7;                      // TMA needs a 16-byte aligned inner coordinate
        p.nseg = 2;
        p.seg[1] = TcSegment{0, 1, a_k0, a_k0 - g.b_split /* <= 0: rows above S read as zero */,
                             ceil_div(g.K - a_k0, BK)};
    }
    p.ksplit = 1; p.kb_per_split = 1 << 30; p.plane = 0;
    p.mode = TC_STORE_BF16;
    p.b3d = b3d ? 1 : 0;
    p.out_f16 = g.dtype == GELO_F16 ? 1 : 0;
    p.C0 = g.C[0]; p.C1 = g.C[g.nsplit > 1 ? 1 : 0]; p.C2 = g.C[g.nsplit > 2 ? 2 : 0];
    p.ldc = g.ldc; p.csplit = g.N / g.nsplit; p.lde = 0;
    p.status = ctx->status_dev;
    return launch_tiles<BN, 4, false>(ctx, ma, ma, mb, mb2, ma, p, 2.0 * g.M * (double)g.N * g.K, st);
}

// Split-precision product for the factorisations.  A = Ahi + Alo (M x K, stride lda), B = Bhi + Blo
// (K x N, stride ldb), all bf16; the tensor cores accumulate Ahi Bhi + Ahi Blo + Alo Bhi in fp32.
//   sub_from != nullptr : sub_from (fp32, stride ldc) -= product, and if emit_hi != nullptr the updated
//                         values are also written as a (hi, lo) pair with stride lde
//   sub_from == nullptr : the product itself is written as the pair (emit_hi, emit_lo), stride lde
int launch_gemm_tc_split(gelo_ctx* ctx, int M, int N, int K, const void* Ahi, const void* Alo, int lda,
                         const void* Bhi, const void* Blo, int ldb, float* sub_from, int ldc, void* emit_hi,
                         void* emit_lo, int lde, bool narrow_tiles, cudaStream_t st)
{
    if (M <= 0 || N <= 0 || K <= 0) return GELO_OK;
    if (!ctx->tmap_encode) return GELO_ERR_CUDA;
    if ((lda % 8) || (ldb % 8) || (!sub_from && (N % 8)) || !aligned16(Ahi) || !aligned16(Alo) || !aligned16(Bhi) || !aligned16(Blo))
        return GELO_ERR_INVALID;
    if (sub_from && ((ldc % 4) || !aligned16(sub_from))) return GELO_ERR_INVALID;
    if (emit_hi && ((lde % 8) || !aligned16(emit_hi) || !aligned16(emit_lo))) return GELO_ERR_INVALID;
    if (!sub_from && !emit_hi) return GELO_ERR_INVALID;
    CUtensorMap a0, a1, b0, b1;
    const uint32_t tile_cols = (!sub_from && narrow_tiles) ? 64 : 256;
    bool b3d = false, b3d1 = false;
    if (!make_map(ctx, &a0, Ahi, (uint64_t)K, (uint64_t)M, (uint64_t)lda, BK, BM) ||
        !make_map(ctx, &a1, Alo, (uint64_t)K, (uint64_t)M, (uint64_t)lda, BK, BM) ||
        !make_map_nmajor(ctx, &b0, Bhi, 2, false, (uint64_t)N, (uint64_t)K, (uint64_t)ldb, BK, tile_cols, &b3d) ||
        !make_map_nmajor(ctx, &b1, Blo, 2, false, (uint64_t)N, (uint64_t)K, (uint64_t)ldb, BK, tile_cols, &b3d1) || b3d != b3d1)
        return GELO_ERR_CUDA;
    TcParams p = {};
    p.M = M; p.N = N;
    const int kb = ceil_div(K, BK);
    p.nseg = 3;
    p.seg[0] = TcSegment{0, 0, 0, 0, kb};
    p.seg[1] = TcSegment{0, 1, 0, 0, kb};
    p.seg[2] = TcSegment{1, 0, 0, 0, kb};
    p.status = ctx->status_dev;
    p.csplit = N;
    p.b3d = b3d ? 1 : 0;
    p.ksplit = 1; p.kb_per_split = 1 << 30; p.plane = 0;
    CUtensorMap mc = a0;
    if (sub_from) {
        if (emit_hi) return GELO_ERR_UNSUPPORTED;
        if (!make_map_f32_box(ctx, &mc, sub_from, (uint64_t)N, (uint64_t)M, (uint64_t)ldc)) return GELO_ERR_CUDA;
        p.mode = TC_SUB_F32;
        p.C0 = sub_from; p.ldc = ldc;
    } else {
        p.mode = TC_EMIT_SPLIT;
        p.C0 = emit_hi; p.C1 = emit_lo; p.ldc = lde; p.lde = lde;
    }
    const double flops = 6.0 * M * (double)N * K;
    if (sub_from) return launch_tiles<256, 3, true>(ctx, a0, a1, b0, b1, mc, p, flops, st);
    if (narrow_tiles) return launch_tiles<64, 4, false>(ctx, a0, a1, b0, b1, mc, p, flops, st);
    return launch_tiles<256, 4, false>(ctx, a0, a1, b0, b1, mc, p, flops, st);
}


int launch_gemm_tc_split_k(gelo_ctx* ctx, int M, int N, int K, const void* Ahi, const void* Alo, int lda, const void* Bhi,
                           const void* Blo, int ldb, float* planes, size_t plane, int ldp, int ksplit, int* used,
                           cudaStream_t st)
{
    if (used) *used = 0;
    if (M <= 0 || N <= 0 || K <= 0) return GELO_OK;
    if (!ctx->tmap_encode) return GELO_ERR_CUDA;
    if ((lda % 8) || (ldb % 8) || (N % 8) || (ldp % 4) || !aligned16(Ahi) || !aligned16(Alo) || !aligned16(Bhi) ||
        !aligned16(Blo) || !aligned16(planes) || (plane % 4) || ksplit < 1)
        return GELO_ERR_INVALID;
    CUtensorMap a0, a1, b0, b1;
    bool b3d = false, b3d1 = false;
    if (!make_map(ctx, &a0, Ahi, (uint64_t)K, (uint64_t)M, (uint64_t)lda, BK, BM) ||
        !make_map(ctx, &a1, Alo, (uint64_t)K, (uint64_t)M, (uint64_t)lda, BK, BM) ||
        !make_map_nmajor(ctx, &b0, Bhi, 2, false, (uint64_t)N, (uint64_t)K, (uint64_t)ldb, BK, 256, &b3d) ||
        !make_map_nmajor(ctx, &b1, Blo, 2, false, (uint64_t)N, (uint64_t)K, (uint64_t)ldb, BK, 256, &b3d1) || b3d != b3d1)
        return GELO_ERR_CUDA;
    const int kb = ceil_div(K, BK);
    if (ksplit > kb) ksplit = kb;
    const int per = ceil_div(kb, ksplit);
    ksplit = ceil_div(kb, per);                    // no empty slice
    TcParams p = {};
    p.M = M; p.N = N;
    p.nseg = 3;
    p.seg[0] = TcSegment{0, 0, 0, 0, kb};
    p.seg[1] = TcSegment{0, 1, 0, 0, kb};
    p.seg[2] = TcSegment{1, 0, 0, 0, kb};
    p.status = ctx->status_dev;
    p.csplit = N;
    p.b3d = b3d ? 1 : 0;
    p.mode = TC_STORE_F32;
    p.C0 = planes; p.ldc = ldp; p.lde = 0;
    p.ksplit = ksplit; p.kb_per_split = per; p.plane = (long long)plane;
    if (used) *used = ksplit;
    return launch_tiles<256, 4, false>(ctx, a0, a1, b0, b1, a0, p, 6.0 * M * (double)N * K, st);
}

// One-product tf32 GEMM on fp32 matrices, fp32 accumulation:  P = op(A) (M x K) * B (K x N, row-major, stride ldb).
//   a_mn = false : A is row-major M x K (stride lda);  a_mn = true : A points at a row-major K x M matrix (stride lda)
//                  and the product uses its transpose.
//   mode TC_SUB_F32   : C (fp32, stride ldc) -= P, in place, by TMA reduce-add
//   mode TC_STORE_F32 : C = P, or with round_out C = post_scale * (out_scale * P - diag_sub * I) rounded to tf32, or
//                       with ksplit > 1 the partial products of the K slices
//                       go to consecutive planes of C (plane stride in elements); *used = slices written
int launch_gemm_tf32(gelo_ctx* ctx, int M, int N, int K, const float* A, int lda, bool a_mn, const float* B, int ldb,
                     bool subtract, float* C, int ldc, bool round_out, float out_scale, int ksplit, size_t plane, int* used,
                     cudaStream_t st, float diag_sub, float post_scale)
{
    if (used) *used = 0;
    if (M <= 0 || N <= 0 || K <= 0) return GELO_OK;
    if (!ctx->tmap_encode) return GELO_ERR_CUDA;
    if ((lda % 4) || (ldb % 4) || (ldc % 4) || !aligned16(A) || !aligned16(B) || !aligned16(C) || !C) return GELO_ERR_INVALID;
    if (!subtract && (N % 8)) return GELO_ERR_INVALID;
    if (subtract && ksplit > 1) return GELO_ERR_INVALID;
    CUtensorMap ma, mb, mc;
    bool a3d = false, b3d = false;
    const bool a_ok = a_mn ? make_map_nmajor(ctx, &ma, A, 4, true, (uint64_t)M, (uint64_t)K, (uint64_t)lda, 32, BM, &a3d)
                           : make_map_f32_box(ctx, &ma, A, (uint64_t)K, (uint64_t)M, (uint64_t)lda, BM);
    if (!a_ok || !make_map_nmajor(ctx, &mb, B, 4, true, (uint64_t)N, (uint64_t)K, (uint64_t)ldb, 32, 256, &b3d)) return GELO_ERR_CUDA;
    mc = ma;
    TcParams p = {};
    p.M = M; p.N = N;
    const int kb = ceil_div(K, 32);
    p.nseg = 1;
    p.seg[0] = TcSegment{0, 0, 0, 0, kb};
    p.status = ctx->status_dev;
    p.csplit = N;
    p.ksplit = 1; p.kb_per_split = 1 << 30; p.plane = 0;
    p.a3d = a3d ? 1 : 0; p.b3d = b3d ? 1 : 0;
    p.round_tf32 = round_out ? 1 : 0;
    p.out_scale = out_scale; p.diag_sub = diag_sub; p.post_scale = post_scale;
    p.C0 = C; p.ldc = ldc;
    const double flops = 2.0 * M * (double)N * K;
    if (subtract) {
        if (!make_map_f32_box(ctx, &mc, C, (uint64_t)N, (uint64_t)M, (uint64_t)ldc, 32)) return GELO_ERR_CUDA;
        p.mode = TC_SUB_F32;
        return a_mn ? launch_tiles<256, 3, true, true, true>(ctx, ma, ma, mb, mb, mc, p, flops, st)
                    : launch_tiles<256, 3, true, true, false>(ctx, ma, ma, mb, mb, mc, p, flops, st);
    }
    p.mode = TC_STORE_F32;
    if (ksplit > 1) {
        if (ksplit > kb) ksplit = kb;
        const int per = ceil_div(kb, ksplit);
        ksplit = ceil_div(kb, per);                // no empty slice
        p.ksplit = ksplit; p.kb_per_split = per; p.plane = (long long)plane;
    }
    if (used) *used = p.ksplit;
    return a_mn ? launch_tiles<256, 4, false, true, true>(ctx, ma, ma, mb, mb, mc, p, flops, st)
                : launch_tiles<256, 4, false, true, false>(ctx, ma, ma, mb, mb, mc, p, flops, st);
}

// D (m x m bf16, stride ldd) = post_scale * (out_scale * Q^T Q - diag_sub I) for a row-major fp32 Q (stride ld): one
// tf32 product in which only the tiles on and above the diagonal are computed (Q^T Q is symmetric) and the rest is
// mirrored by the epilogue.  ldd >= m rounded up to 8.
int launch_gram_sym_bf16(gelo_ctx* ctx, int m, const float* Q, int ld, void* D, int ldd, float out_scale, float diag_sub,
                         float post_scale, cudaStream_t st)
{
    if (m <= 0) return GELO_OK;
    if (!ctx->tmap_encode) return GELO_ERR_CUDA;
    const int m8 = (m + 7) & ~7;
    if ((ld % 4) || ld < m8 || (ldd % 8) || ldd < m8 || !aligned16(Q) || !aligned16(D)) return GELO_ERR_INVALID;
    CUtensorMap ma, mb;
    bool a3d = false, b3d = false;
    if (!make_map_nmajor(ctx, &ma, Q, 4, true, (uint64_t)m, (uint64_t)m, (uint64_t)ld, 32, BM, &a3d) ||
        !make_map_nmajor(ctx, &mb, Q, 4, true, (uint64_t)m8, (uint64_t)m, (uint64_t)ld, 32, 256, &b3d))
        return GELO_ERR_CUDA;
    TcParams p = {};
    p.M = m; p.N = m8;
    p.nseg = 1;
    p.seg[0] = TcSegment{0, 0, 0, 0, ceil_div(m, 32)};
    p.status = ctx->status_dev;
    p.csplit = m8;
    p.ksplit = 1; p.kb_per_split = 1 << 30; p.plane = 0;
    p.a3d = a3d ? 1 : 0; p.b3d = b3d ? 1 : 0;
    p.out_scale = out_scale; p.diag_sub = diag_sub; p.post_scale = post_scale;
    p.C0 = D; p.ldc = ldd;
    p.mode = TC_STORE_SYM16;
    p.tri = 1;
    const int m_tiles = ceil_div(m, BM), n_tiles = ceil_div(m8, 256);
    int tiles = 0;
    for (int nt = 0; nt < n_tiles; ++nt) tiles += (m_tiles < 2 * nt + 2) ? m_tiles : 2 * nt + 2;
    p.tri_tiles = tiles;
    return launch_tiles<256, 4, false, true, true>(ctx, ma, ma, mb, mb, ma, p, 2.0 * m * (double)m * m, st);
}

// C (M x N fp32, stride ldc) -= A (M x K bf16, stride lda) * B (K x N bf16, stride ldb), in place by TMA reduce-add.
int launch_gemm_bf16_sub(gelo_ctx* ctx, int M, int N, int K, const void* A, int lda, const void* B, int ldb, float* C, int ldc,
                         cudaStream_t st)
{
    if (M <= 0 || N <= 0 || K <= 0) return GELO_OK;
    if (!ctx->tmap_encode) return GELO_ERR_CUDA;
    if ((lda % 8) || (ldb % 8) || (ldc % 4) || !aligned16(A) || !aligned16(B) || !aligned16(C)) return GELO_ERR_INVALID;
    CUtensorMap ma, mb, mc;
    bool b3d = false;
    if (!make_map(ctx, &ma, A, (uint64_t)K, (uint64_t)M, (uint64_t)lda, BK, BM) ||
        !make_map_nmajor(ctx, &mb, B, 2, false, (uint64_t)N, (uint64_t)K, (uint64_t)ldb, BK, 256, &b3d) ||
        !make_map_f32_box(ctx, &mc, C, (uint64_t)N, (uint64_t)M, (uint64_t)ldc))
        return GELO_ERR_CUDA;
    TcParams p = {};
    p.M = M; p.N = N;
    p.nseg = 1;
    p.seg[0] = TcSegment{0, 0, 0, 0, ceil_div(K, BK)};
    p.status = ctx->status_dev;
    p.csplit = N;
    p.b3d = b3d ? 1 : 0;
    p.ksplit = 1; p.kb_per_split = 1 << 30; p.plane = 0;
    p.mode = TC_SUB_F32;
    p.C0 = C; p.ldc = ldc;
    return launch_tiles<256, 3, true>(ctx, ma, ma, mb, mb, mc, p, 2.0 * M * (double)N * K, st);
}

// Y (M x N, bf16) = (sa sb) A8 (M x K, E4M3, row stride lda bytes) * B8 (K x N, E4M3, row stride ldb bytes): the offloaded
// product on 8-bit operands (kind::f8f6f4, fp32 accumulation), sa and sb device scalars.  A stage holds 128 bytes of
// k per A row, i.e. 128 values, and the matching 128 rows of B in boxes of 128 columns.
int launch_gemm_e4m3(gelo_ctx* ctx, int M, int N, int K, const void* A8, int lda, const void* B8, int ldb, const float* sa,
                     const float* sb, void* C, int ldc, cudaStream_t st)
{
    if (M <= 0 || N <= 0 || K <= 0) return GELO_OK;
    if (!ctx->tmap_encode) return GELO_ERR_CUDA;
    if ((lda % 16) || (ldb % 16) || (ldc % 8) || (N % 8) || !aligned16(A8) || !aligned16(B8) || !aligned16(C) || !sa || !sb)
        return GELO_ERR_INVALID;
    EncodeTiledFn enc = reinterpret_cast<EncodeTiledFn>(ctx->tmap_encode);
    CUtensorMap ma, mb;
    {
        const cuuint64_t dims[2] = { (cuuint64_t)K, (cuuint64_t)M };
        const cuuint64_t strides[1] = { (cuuint64_t)lda };
        const cuuint32_t box[2] = { 128, BM };
        const cuuint32_t estr[2] = { 1, 1 };
        if (enc(&ma, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(A8), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return GELO_ERR_CUDA;
    }
    bool b3d = false;
    if (!make_map_nmajor(ctx, &mb, B8, 1, false, (uint64_t)N, (uint64_t)K, (uint64_t)ldb, 128, 256, &b3d)) return GELO_ERR_CUDA;
    TcParams p = {};
    p.M = M; p.N = N;
    p.nseg = 1;
    p.seg[0] = TcSegment{0, 0, 0, 0, ceil_div(K, 128)};
    p.ksplit = 1; p.kb_per_split = 1 << 30; p.plane = 0;
    p.mode = TC_STORE_BF16;
    p.b3d = b3d ? 1 : 0;
    p.C0 = C; p.C1 = C; p.C2 = C;
    p.ldc = ldc; p.csplit = N;
    p.scale_a = sa; p.scale_b = sb;
    p.status = ctx->status_dev;
    return launch_tiles<256, 4, false, false, false, true>(ctx, ma, ma, mb, mb, ma, p, 2.0 * M * (double)N * K, st);
}

int launch_gemm_tf32x3(gelo_ctx* ctx, int M, int N, int K, const float* Ahi, const float* Alo, int lda, const float* Bhi,
                       const float* Blo, int ldb, float* const C[3], int ldc, int nsplit, float* planes, cudaStream_t st)
{
    if (M <= 0 || N <= 0 || K <= 0) return GELO_OK;
    if (!ctx->tmap_encode) return GELO_ERR_CUDA;
    if (nsplit < 1 || nsplit > 3 || (N % nsplit) || ((N / nsplit) % 8) || (lda % 4) || (ldb % 4) || (ldc % 4) ||
        !aligned16(Ahi) || !aligned16(Alo) || !aligned16(Bhi) || !aligned16(Blo))
        return GELO_ERR_INVALID;
    for (int q = 0; q < nsplit; ++q)
        if (!C[q] || !aligned16(C[q])) return GELO_ERR_INVALID;
    CUtensorMap a0, a1, b0, b1;
    bool b3d = false, b3d1 = false;
    if (!make_map_f32_box(ctx, &a0, Ahi, (uint64_t)K, (uint64_t)M, (uint64_t)lda, BM) ||
        !make_map_f32_box(ctx, &a1, Alo, (uint64_t)K, (uint64_t)M, (uint64_t)lda, BM) ||
        !make_map_nmajor(ctx, &b0, Bhi, 4, true, (uint64_t)N, (uint64_t)K, (uint64_t)ldb, 32, 256, &b3d) ||
        !make_map_nmajor(ctx, &b1, Blo, 4, true, (uint64_t)N, (uint64_t)K, (uint64_t)ldb, 32, 256, &b3d1) || b3d != b3d1)
        return GELO_ERR_CUDA;
    TcParams p = {};
    p.M = M; p.N = N;
    const int kb = ceil_div(K, 32);
    p.nseg = 3;
    p.seg[0] = TcSegment{0, 0, 0, 0, kb};
    p.seg[1] = TcSegment{0, 1, 0, 0, kb};
    p.seg[2] = TcSegment{1, 0, 0, 0, kb};
    p.status = ctx->status_dev;
    p.b3d = b3d ? 1 : 0;
    p.ksplit = 1; p.kb_per_split = 1 << 30; p.plane = 0;
    p.mode = TC_STORE_F32;
    p.out_scale = 1.0f; p.post_scale = 1.0f;
    float* const Cq[3] = { C[0], C[nsplit > 1 ? 1 : 0], C[nsplit > 2 ? 2 : 0] };
    if (planes && kb >= 2 * kTf32x3Slices && aligned16(planes) && (N % 4) == 0) {
        const int per = ceil_div(kb, kTf32x3Slices);
        p.ksplit = ceil_div(kb, per); p.kb_per_split = per; p.plane = (long long)M * N;
        p.C0 = planes; p.C1 = planes; p.C2 = planes; p.ldc = N; p.csplit = N;
        GELO_TRY((launch_tiles<256, 4, false, true, false>(ctx, a0, a1, b0, b1, a0, p, 6.0 * M * (double)N * K, st)));
        return launch_sum_planes_routed(ctx, planes, (size_t)M * N, p.ksplit, M, N, Cq, ldc, N / nsplit, st);
    }
    p.C0 = Cq[0]; p.C1 = Cq[1]; p.C2 = Cq[2];
    p.ldc = ldc; p.csplit = N / nsplit;
    return launch_tiles<256, 4, false, true, false>(ctx, a0, a1, b0, b1, a0, p, 6.0 * M * (double)N * K, st);
}

}  // namespace gelo
