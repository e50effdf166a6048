// Projection and unmixing of a SMALL batch in one kernel (Eq. 2 and Eq. 3 for m = n + k <= 128 mixed rows, the
// decode-shaped call: a few dozen token rows against a weight of a hundred megabytes).
//
//     Y' = U W            (m x d) (d x p)      -- the offloaded contraction, bound by streaming W once from HBM
//     Y  = (A^-1 Y')[0:n] (n x m) (m x p)      -- tiny; applied to each column slab of Y' while it is still on chip
//
// A product with so few rows is a stream of W: what matters is that many SMs pull disjoint shares of it with long
// requests.  W is cut into boxes of 64 columns (128-byte rows; measured: 64-byte rows stream at 4.3 TB/s, 128-byte rows
// faster) and the boxes are dealt evenly over the CTAs (p = 12288: 192 boxes, 2 per CTA on 96 SMs), so that each CTA
// streams its own d x 128 slab through a TMA / mbarrier pipeline while re-reading the small U from L2.  The accumulator Y'_slab (m rows, padded to the 128 lanes of tensor memory) never goes to HBM:
// the epilogue warps round it to the storage type, exactly as the stand-alone projection would store it, lay it out
// in shared memory as the B operand of a second tcgen05 product with the first n rows of A^-1, and write the result
// straight into Q | K | V.  Two launches (gelo_project, gelo_unmix) and the round trip of Y' become one launch.
//
// Layouts.  U tiles and the A^-1 rows: K-major, 128-byte swizzle (as in gemm_tc.cu).  W boxes: 64 k-rows x 64
// columns, N-major with the 128-byte swizzle (atoms of 8 k-rows x 128 bytes; boxes 8192 bytes apart).  The Y' slab:
// N-major without swizzle, i.e. core matrices of 8 k-rows x 8 columns (128 contiguous bytes), 8-row groups 128 bytes
// apart, 8-column groups kpad * 16 bytes apart - which is what a thread holding one row of the accumulator can write
// as 16-byte pieces without bank conflicts.
// Warp roles: warp 0 issues TMA, warps 1-2 issue MMA for alternate k-blocks (warp 1 owns tensor memory), warps 3-6 are
// the epilogue (one per tensor-memory lane quarter).  Every barrier wait is bounded in time as in gemm_tc.cu.
#include <cuda.h>

#include "common.cuh"
#include "tc_ptx.cuh"

namespace gelo {

namespace {

using namespace tcx;

constexpr int kDecIssuers = 2;                           // MMA-issuing warps, each with its own accumulator of Y'
constexpr int kDecThreads = 32 * (1 + kDecIssuers + 4);
constexpr int kDecBK = 64;                              // k elements per stage: 128 bytes of a K-major row
// The MMA always multiplies 128 rows of A.  Only the first kpad rows of a U tile (m real ones, zero-filled up to a
// multiple of 16) are ever loaded; the rows behind them are whatever the following shared memory holds, and they only
// reach accumulator rows that nobody reads.  Every byte of shared memory not spent on those rows is a byte of W in flight.
constexpr uint32_t kDecRowBytes = kDecBK * 2;           // one K-major row of a tile: 128 bytes
constexpr uint32_t kDecAReach = 128 * kDecRowBytes;     // bytes the MMA reads from the start of an A tile
constexpr int kDecBoxCols = 64;                         // W arrives in boxes of 64 columns: 128-byte rows, the longest a swizzled box takes
constexpr uint32_t kDecBoxBytes = kDecBK * 128;         // one W box: 64 k-rows x 64 columns
constexpr int kDecMaxBoxes = 2;                         // boxes per CTA: slab of at most 128 columns
constexpr uint32_t kDecAccCols = 128;                   // columns of one accumulator (a slab is at most 128 columns wide)
constexpr uint32_t kDecTmemCols = 512;                  // two partial Y' slabs, then the Y slab (a power of two)

struct DecParams {
    int m, n, d;
    int kpad;                   // m rounded up to 16: the K extent of the second product, and the rows of a U tile
    int npad;                   // n rounded up to 16: the rows of A^-1 that are loaded
    int boxes, base, rem;       // p / 64 boxes; CTA i takes base + (i < rem) of them
    int stages;                 // operand stages that fit next to the fixed buffers
    int nbmax;                  // base + (rem > 0): boxes of the widest slab (stage stride)
    int group;                  // CTAs per group; group g walks the k-blocks starting from g * kstep (see the kernel)
    int kstep;
    void* C0; void* C1; void* C2;
    int ldc, csplit;
    int out_f16;
    int plain;                  // no second product: the rounded Y' slab itself is the result (m rows)
    unsigned long long wait_ns;
    int* status;
};

__device__ __forceinline__ void store8(void* base, size_t off, const uint32_t* v, int f16)
{
    uint4 pk;
    if (f16) { pk.x = pack_f16(v[0], v[1]); pk.y = pack_f16(v[2], v[3]); pk.z = pack_f16(v[4], v[5]); pk.w = pack_f16(v[6], v[7]); }
    else { pk.x = pack_bf16(v[0], v[1]); pk.y = pack_bf16(v[2], v[3]); pk.z = pack_bf16(v[4], v[5]); pk.w = pack_bf16(v[6], v[7]); }
    *reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(base) + off) = pk;
}

__global__ void __launch_bounds__(kDecThreads, 1)
project_unmix_kernel(const __grid_constant__ CUtensorMap map_u, const __grid_constant__ CUtensorMap map_w_wide,
                     const __grid_constant__ CUtensorMap map_w_narrow, const __grid_constant__ CUtensorMap map_ainv,
                     const DecParams prm)
{
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t tiles_base = (raw + 1023u) & ~1023u;
    uint8_t* gen_base = smem_raw + (tiles_base - raw);
    const uint32_t a_bytes = (uint32_t)prm.kpad * kDecRowBytes;                           // multiple of 2048
    const uint32_t stage_bytes = a_bytes + (uint32_t)prm.nbmax * kDecBoxBytes;
    const uint32_t ainv_tile = (uint32_t)prm.npad * kDecRowBytes;                         // one K-major tile of A^-1 rows
    const uint32_t ainv_base = tiles_base + (uint32_t)prm.stages * stage_bytes;           // 1024-byte aligned
    const uint32_t y_base = ainv_base + 2u * ainv_tile;
    const uint32_t y_bytes = (uint32_t)prm.kpad * 16u * (uint32_t)(prm.nbmax * 8);       // kpad x (nbmax * 64 columns) x 2 bytes
    const uint32_t bar_off = (uint32_t)prm.stages * stage_bytes + 2u * ainv_tile + ((y_bytes + 15u) & ~15u);
    const uint32_t bar_base = tiles_base + bar_off;
    uint8_t* bar_gen = gen_base + bar_off;
    // barriers (8 bytes each): full[stages], empty[stages], ainv_full, acc1_full, y_ready, acc2_full; then tmem slot, abort
    const int S = prm.stages;
    auto full_bar = [&](int s) { return bar_base + 8u * s; };
    auto empty_bar = [&](int s) { return bar_base + 8u * (S + s); };
    const uint32_t ainv_bar = bar_base + 8u * (2 * S), acc1_bar = ainv_bar + 8u, y_bar = ainv_bar + 16u, acc2_bar = ainv_bar + 24u;
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(bar_gen + 8 * (2 * S + 4));
    volatile int* abort_flag = reinterpret_cast<volatile int*>(bar_gen + 8 * (2 * S + 4) + 8);

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const int cta = blockIdx.x;
    const int nb = prm.base + (cta < prm.rem ? 1 : 0);                 // boxes of this CTA's slab
    const int box0 = cta * prm.base + min(cta, prm.rem);
    const int ncols = nb * kDecBoxCols;
    const int col0 = box0 * kDecBoxCols;
    const int nkb = (prm.d + kDecBK - 1) / kDecBK;
    // Every CTA needs every tile of U.  If all CTAs walked the k-blocks in the same order they would all ask the L2 for
    // the same few lines at the same moment; instead groups of neighbouring CTAs (neighbours read adjacent columns of
    // the same rows of W, which keeps the DRAM accesses long) start at different k-blocks and wrap around.
    const int kb_first = ((cta / prm.group) * prm.kstep) % nkb;

    if (threadIdx.x == 0) {
        for (int s = 0; s < S; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        mbar_init(ainv_bar, 1); mbar_init(acc1_bar, kDecIssuers); mbar_init(y_bar, 4); mbar_init(acc2_bar, 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32((const void*)tmem_slot)), "r"(kDecTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    // instruction descriptor: fp32 accumulate, both operands bf16 (1) or half (0), A K-major, B N-major, M = 128, N = ncols
    const uint32_t fmt = prm.out_f16 ? 0u : 1u;
    const uint32_t idesc = (1u << 4) | (fmt << 7) | (fmt << 10) | (1u << 16) | ((uint32_t)(ncols >> 3) << 17) | ((128u >> 4) << 24);

    if (warp == 0) {
        // ================= TMA producer =================
        if (lane == 0 && nb > 0) {
            bool ok = true;
            if (prm.wait_ns != 0 && !prm.plain) {
                // the first n rows of A^-1 (columns past m and rows past n arrive as zeros)
                mbar_expect_tx(ainv_bar, 2u * ainv_tile);
                tma_load_2d(ainv_base, &map_ainv, 0, 0, ainv_bar);
                tma_load_2d(ainv_base + ainv_tile, &map_ainv, kDecBK, 0, ainv_bar);
            }
            const CUtensorMap* mw = (nb == prm.nbmax) ? &map_w_wide : &map_w_narrow;
            int s = 0, kq = kb_first;
            uint32_t ph = 0;
            for (int kb = 0; kb < nkb; ++kb) {
                if (!mbar_wait(empty_bar(s), ph ^ 1u, abort_flag, prm.wait_ns)) { ok = false; break; }
                const uint32_t sa = tiles_base + (uint32_t)s * stage_bytes;
                mbar_expect_tx(full_bar(s), a_bytes + (uint32_t)nb * kDecBoxBytes);
                tma_load_3d(sa + a_bytes, mw, 0, kq * kDecBK, box0, full_bar(s));        // the W slab first: it comes from HBM
                tma_load_2d(sa, &map_u, kq * kDecBK, 0, full_bar(s));
                if (++s == S) { s = 0; ph ^= 1u; }
                if (++kq == nkb) kq = 0;
            }
            if (!ok) { *abort_flag = 1; atomicCAS(prm.status, 0, (int)GELO_ERR_TIMEOUT); }
        }
    } else if (warp <= kDecIssuers) {
        // ================= MMA issuers =================
        // A thread needs some 700 cycles to get through one k-block (barrier test, four instructions, commit), about
        // three times what the tensor core then spends on it, and the weight stream waits for the slower of the two.
        // Two threads therefore take alternate k-blocks, each into an accumulator of its own (the epilogue adds them).
        if (lane == 0 && nb > 0) {
            const int me = warp - 1;
            bool ok = true;
            const uint32_t acc = tmem_base + (uint32_t)me * kDecAccCols;
            int s = me % S;
            uint32_t ph = (uint32_t)(me / S) & 1u;
            for (int kb = me; kb < nkb; kb += kDecIssuers) {
                if (!mbar_wait(full_bar(s), ph, abort_flag, prm.wait_ns)) { ok = false; break; }
                const uint32_t sa = tiles_base + (uint32_t)s * stage_bytes;
                const uint32_t sb = sa + a_bytes;
                const uint64_t da0 = smem_desc(sa, 16, 1024, 2);                          // K-major, 128-byte swizzle
                const uint64_t db0 = smem_desc(sb, kDecBoxBytes, 1024, 2);                // N-major, 128-byte swizzle
#pragma unroll
                for (int ks = 0; ks < 4; ++ks)       // the start address field counts 16-byte units: 32 and 2048 bytes per step
                    tc_mma_bf16(acc, da0 + (uint64_t)(ks * 2), db0 + (uint64_t)(ks * 128), idesc, (kb != me || ks != 0) ? 1u : 0u);
                tc_commit(empty_bar(s));
                s += kDecIssuers;
                if (s >= S) { s -= S; ph ^= 1u; }
            }
            if (ok) {
                if (me < nkb) tc_commit(acc1_bar); else mbar_arrive(acc1_bar);            // (no k-block, nothing to wait for)
                // second product: Y_slab = A^-1[0:n, 0:kpad] * Y'_slab once the epilogue has laid Y'_slab out
                if (me == 0 && !prm.plain) {
                    if (mbar_wait(y_bar, 0, abort_flag, prm.wait_ns) && mbar_wait(ainv_bar, 0, abort_flag, prm.wait_ns)) {
                        tc_fence_after();
                        const int ksteps = prm.kpad >> 4;
                        for (int ks = 0; ks < ksteps; ++ks) {
                            const uint32_t at = ainv_base + (uint32_t)(ks >> 2) * ainv_tile + (uint32_t)(ks & 3) * 32u;
                            const uint64_t da = smem_desc(at, 16, 1024, 2);
                            // no swizzle: 8-row groups 128 bytes apart (leading offset), 8-column groups kpad * 16 apart (stride offset)
                            const uint64_t db = smem_desc(y_base + (uint32_t)ks * 256u, 128, (uint32_t)prm.kpad * 16u, 0);
                            tc_mma_bf16(tmem_base + (uint32_t)(kDecIssuers * kDecAccCols), da, db, idesc, ks != 0 ? 1u : 0u);
                        }
                        tc_commit(acc2_bar);
                    } else {
                        ok = false;
                    }
                }
            }
            if (!ok) { *abort_flag = 1; atomicCAS(prm.status, 0, (int)GELO_ERR_TIMEOUT); }
        }
    } else if (nb > 0) {
        // ================= epilogue (four warps, one per tensor-memory lane quarter) =================
        const int quarter = warp & 3;                    // the tensor-memory lane quarter this warp may read
        const int row = quarter * 32 + lane;
        bool ok = true;
        // ---- Y' slab: round to the storage type and lay it out as the B operand of the second product ----
        if (!mbar_wait(acc1_bar, 0, abort_flag, prm.wait_ns)) ok = false;
        if (ok) {
            tc_fence_after();
            if (quarter * 32 < prm.kpad) {
                const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16);
                const uint32_t row_off = (uint32_t)(row >> 3) * 128u + (uint32_t)(row & 7) * 16u;
                for (int c = 0; c < ncols; c += 32) {
                    uint32_t v[32];
                    tc_ld_32cols(taddr + c, v);
                    if (nkb > 1) {                            // the second issuer's share of the k-blocks
                        uint32_t w[32];
                        tc_ld_32cols(taddr + kDecAccCols + c, w);
                        tc_ld_wait();
#pragma unroll
                        for (int j = 0; j < 32; ++j) v[j] = __float_as_uint(__uint_as_float(v[j]) + __uint_as_float(w[j]));
                    } else {
                        tc_ld_wait();
                    }
                    if (prm.plain) {
                        if (row < prm.m) {
#pragma unroll
                            for (int g = 0; g < 4; ++g) {
                                const int gc = col0 + c + 8 * g;
                                const int chunk = gc / prm.csplit;
                                void* base = chunk == 0 ? prm.C0 : (chunk == 1 ? prm.C1 : prm.C2);
                                store8(base, (size_t)row * prm.ldc + (gc - chunk * prm.csplit), v + 8 * g, prm.out_f16);
                            }
                        }
                    } else if (row < prm.kpad) {
#pragma unroll
                        for (int g = 0; g < 4; ++g) {
                            uint32_t q0, q1, q2, q3;
                            if (prm.out_f16) {
                                q0 = pack_f16(v[8 * g + 0], v[8 * g + 1]); q1 = pack_f16(v[8 * g + 2], v[8 * g + 3]);
                                q2 = pack_f16(v[8 * g + 4], v[8 * g + 5]); q3 = pack_f16(v[8 * g + 6], v[8 * g + 7]);
                            } else {
                                q0 = pack_bf16(v[8 * g + 0], v[8 * g + 1]); q1 = pack_bf16(v[8 * g + 2], v[8 * g + 3]);
                                q2 = pack_bf16(v[8 * g + 4], v[8 * g + 5]); q3 = pack_bf16(v[8 * g + 6], v[8 * g + 7]);
                            }
                            const uint32_t dst = y_base + (uint32_t)((c >> 3) + g) * (uint32_t)prm.kpad * 16u + row_off;
                            asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "r"(q0), "r"(q1), "r"(q2), "r"(q3) : "memory");
                        }
                    }
                }
            }
            if (!prm.plain) {
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // the tensor core reads this through the async proxy
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(y_bar);
                // ---- Y slab: rows 0 .. n-1 to Q | K | V ----
                if (!mbar_wait(acc2_bar, 0, abort_flag, prm.wait_ns)) ok = false;
            }
        }
        if (ok && !prm.plain) {
            tc_fence_after();
            if (quarter * 32 < prm.n) {
                const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(kDecIssuers * kDecAccCols);
                for (int c = 0; c < ncols; c += 32) {
                    uint32_t v[32];
                    tc_ld_32cols(taddr + c, v);
                    tc_ld_wait();
                    if (row < prm.n) {
#pragma unroll
                        for (int g = 0; g < 4; ++g) {
                            const int gc = col0 + c + 8 * g;
                            const int chunk = gc / prm.csplit;
                            void* base = chunk == 0 ? prm.C0 : (chunk == 1 ? prm.C1 : prm.C2);
                            store8(base, (size_t)row * prm.ldc + (gc - chunk * prm.csplit), v + 8 * g, prm.out_f16);
                        }
                    }
                }
            }
        }
        if (!ok && lane == 0) { *abort_flag = 1; atomicCAS(prm.status, 0, (int)GELO_ERR_TIMEOUT); }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kDecTmemCols) : "memory");
    }
}

typedef CUresult (*EncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                             const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                             CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// K-major operand: rows x cols 16-bit elements, row stride ld; boxes of 64 columns x box_rows rows, 128-byte swizzle, zero fill
bool map_kmajor(gelo_ctx* ctx, CUtensorMap* map, const void* ptr, uint64_t cols, uint64_t rows, uint64_t ld, uint32_t box_rows)
{
    EncodeFn enc = reinterpret_cast<EncodeFn>(ctx->tmap_encode);
    const cuuint64_t dims[2] = { cols, rows };
    const cuuint64_t strides[1] = { ld * 2 };
    const cuuint32_t box[2] = { (cuuint32_t)kDecBK, box_rows };
    const cuuint32_t estr[2] = { 1, 1 };
    return enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// W (d x p, row stride p) as {64 columns, d rows, p / 64 boxes}: one copy brings `nb` boxes of 64 rows, each box landing
// as 64 rows of 128 bytes in the 128-byte swizzle
bool map_w_boxes(gelo_ctx* ctx, CUtensorMap* map, const void* W, uint64_t d, uint64_t p, uint32_t nb)
{
    EncodeFn enc = reinterpret_cast<EncodeFn>(ctx->tmap_encode);
    const cuuint64_t dims[3] = { (cuuint64_t)kDecBoxCols, d, p / kDecBoxCols };
    const cuuint64_t strides[2] = { p * 2, (cuuint64_t)kDecBoxCols * 2 };
    const cuuint32_t box[3] = { (cuuint32_t)kDecBoxCols, (cuuint32_t)kDecBK, nb };
    const cuuint32_t estr[3] = { 1, 1, 1 };
    return enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(W), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

constexpr uint32_t kDecSmemBudget = 227u * 1024u;

// ---- U = A [H; S] for a small batch (Eq. 1 / Eq. 8 with m = n + k <= 128) ----------------------------------------
// 2 m^2 d flops on a few hundred kilobytes: a tensor-core launch spends more on its set-up than this takes on the FMA
// pipes.  One CTA per 32 columns of U: A (widened to fp32) and the 32-column strip of the stacked [H; S] go to shared
// memory, every thread accumulates a 4 x 4 patch in fp32 (the products of two 16-bit values are exact in fp32).
__device__ __forceinline__ float widen(__nv_bfloat16 x) { return __bfloat162float(x); }
__device__ __forceinline__ float widen(__half x) { return __half2float(x); }
__device__ __forceinline__ void narrow4(__nv_bfloat16* p, const float (&v)[4])
{
    __nv_bfloat162 a = __floats2bfloat162_rn(v[0], v[1]), b = __floats2bfloat162_rn(v[2], v[3]);
    uint2 t; t.x = *reinterpret_cast<uint32_t*>(&a); t.y = *reinterpret_cast<uint32_t*>(&b);
    *reinterpret_cast<uint2*>(p) = t;
}
__device__ __forceinline__ void narrow4(__half* p, const float (&v)[4])
{
    __half2 a = __floats2half2_rn(v[0], v[1]), b = __floats2half2_rn(v[2], v[3]);
    uint2 t; t.x = *reinterpret_cast<uint32_t*>(&a); t.y = *reinterpret_cast<uint32_t*>(&b);
    *reinterpret_cast<uint2*>(p) = t;
}

template <typename T>
__global__ void __launch_bounds__(256)
mix_small_kernel(const T* __restrict__ A, int lda, const T* __restrict__ H, const T* __restrict__ S, int n, int k, int d,
                 T* __restrict__ U)
{
    extern __shared__ __align__(16) float mix_smem[];
    const int m = n + k;
    const int lds = m + 1;
    float* Hs = mix_smem;                     // m x 32 (16-byte aligned rows)
    float* As = mix_smem + m * 32;            // m x (m + 1)
    const int tid = threadIdx.x;
    const int c0 = blockIdx.x * 32;
    // All global loads of a thread are issued before any of them is used (16 bytes each; the row stride of A is a
    // multiple of 8 elements, so a group that starts inside a row may run into its padding, which is read and dropped).
    const int ga = (m + 7) >> 3;                             // 16-byte groups per row of A
    constexpr int kMaxA = (128 * 16 + 255) / 256, kMaxH = (128 * 4 + 255) / 256;
    uint4 ra[kMaxA], rh[kMaxH];
#pragma unroll
    for (int t = 0; t < kMaxA; ++t) {
        const int idx = tid + t * 256;
        if (idx < m * ga) {
            const int r = idx / ga, g = idx - r * ga;
            ra[t] = *reinterpret_cast<const uint4*>(A + (size_t)r * lda + g * 8);
        }
    }
#pragma unroll
    for (int t = 0; t < kMaxH; ++t) {                        // eight consecutive columns of the strip per step
        const int idx = tid + t * 256;
        const int r = idx >> 2, col = c0 + (idx & 3) * 8;
        rh[t] = make_uint4(0u, 0u, 0u, 0u);                  // (all-zero bits are 0.0 in both 16-bit types)
        if (idx < m * 4 && col < d)                          // d is a multiple of 8: a group is inside or outside
            rh[t] = *reinterpret_cast<const uint4*>((r < n ? H + (size_t)r * d : S + (size_t)(r - n) * d) + col);
    }
#pragma unroll
    for (int t = 0; t < kMaxA; ++t) {
        const int idx = tid + t * 256;
        if (idx < m * ga) {
            const int r = idx / ga, g = idx - r * ga;
            const T* e = reinterpret_cast<const T*>(&ra[t]);
#pragma unroll
            for (int j = 0; j < 8; ++j)
                if (g * 8 + j < m) As[r * lds + g * 8 + j] = widen(e[j]);
        }
    }
#pragma unroll
    for (int t = 0; t < kMaxH; ++t) {
        const int idx = tid + t * 256;
        if (idx < m * 4) {
            const T* e = reinterpret_cast<const T*>(&rh[t]);
            float4* dst = reinterpret_cast<float4*>(Hs + (idx >> 2) * 32 + (idx & 3) * 8);
            dst[0] = make_float4(widen(e[0]), widen(e[1]), widen(e[2]), widen(e[3]));
            dst[1] = make_float4(widen(e[4]), widen(e[5]), widen(e[6]), widen(e[7]));
        }
    }
    __syncthreads();
    const int ty = tid >> 3, tx = tid & 7;
    float acc[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = 0.0f;
    int rows[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) rows[i] = min(ty + 32 * i, m - 1);      // clamped rows are computed twice, stored once
    for (int kk = 0; kk < m; ++kk) {
        const float4 h = *reinterpret_cast<const float4*>(Hs + kk * 32 + tx * 4);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float a = As[rows[i] * lds + kk];
            acc[i][0] = fmaf(a, h.x, acc[i][0]); acc[i][1] = fmaf(a, h.y, acc[i][1]);
            acc[i][2] = fmaf(a, h.z, acc[i][2]); acc[i][3] = fmaf(a, h.w, acc[i][3]);
        }
    }
    const int col = c0 + tx * 4;
    if (col < d) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int r = ty + 32 * i;
            if (r < m) narrow4(U + (size_t)r * d + col, acc[i]);
        }
    }
}

}  // namespace

bool mix_small_supports(int n, int k, int d, int dtype)
{
    return dtype != GELO_F32 && n > 0 && k >= 0 && n + k <= 128 && d > 0 && (d % 8) == 0;
}

int launch_mix_small(gelo_ctx* ctx, const void* A, int lda, const void* H, const void* S, int n, int k, int d, int dtype,
                     void* U, cudaStream_t st)
{
    if (!mix_small_supports(n, k, d, dtype) || (k > 0 && !S)) return GELO_ERR_UNSUPPORTED;
    const int m = n + k;
    const int smem = (m * 32 + m * (m + 1)) * (int)sizeof(float);
    const int grid = ceil_div(d, 32);
    static bool attr_done[64] = {};
    if (ctx->device >= 0 && ctx->device < 64 && !attr_done[ctx->device]) {
        GELO_CUDA_OK(cudaFuncSetAttribute(mix_small_kernel<__half>, cudaFuncAttributeMaxDynamicSharedMemorySize, 96 * 1024));
        GELO_CUDA_OK(cudaFuncSetAttribute(mix_small_kernel<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, 96 * 1024));
        attr_done[ctx->device] = true;
    }
    if (dtype == GELO_F16) {
        mix_small_kernel<__half><<<grid, 256, smem, st>>>(static_cast<const __half*>(A), lda, static_cast<const __half*>(H),
                                                          static_cast<const __half*>(S), n, k, d, static_cast<__half*>(U));
    } else {
        mix_small_kernel<__nv_bfloat16><<<grid, 256, smem, st>>>(static_cast<const __nv_bfloat16*>(A), lda,
                                                                 static_cast<const __nv_bfloat16*>(H),
                                                                 static_cast<const __nv_bfloat16*>(S), n, k, d,
                                                                 static_cast<__nv_bfloat16*>(U));
    }
    return after_launch(ctx);
}

bool project_unmix_supports(const gelo_ctx* ctx, int n, int k, int d, int p, int dtype, int lda, int nsplit)
{
    const int m = n + k;
    if (dtype == GELO_F32 || m > 128 || n <= 0 || k < 0 || d <= 0 || p <= 0) return false;
    if ((d % 8) || (p % kDecBoxCols) || (lda % 8) || lda < m) return false;
    if (nsplit != 1 && nsplit != 3) return false;
    if (nsplit == 3 && ((p % 3) || ((p / 3) % 8))) return false;
    const int boxes = p / kDecBoxCols;
    const int ncta = boxes < ctx->sm_count ? boxes : ctx->sm_count;
    return (boxes + ncta - 1) / ncta <= kDecMaxBoxes;
}

// Q | K | V (or one n x p result when K = V = nullptr) = (Ainv[0:n, 0:m] (U W)) for m = n + k <= 128.  With
// Ainv == nullptr the kernel stops after the first product: the result is U W itself (n + k rows).
int launch_project_unmix(gelo_ctx* ctx, const void* U, const void* W, const void* Ainv, int lda, int n, int k, int d, int p,
                         int dtype, void* Q, void* K, void* V, cudaStream_t st)
{
    const int nsplit = (K || V) ? 3 : 1;
    if (!Ainv) lda = (n + k + 7) & ~7;
    if (!project_unmix_supports(ctx, n, k, d, p, dtype, lda, nsplit)) return GELO_ERR_UNSUPPORTED;
    if (!ctx->tmap_encode) return GELO_ERR_CUDA;
    const int m = n + k;
    DecParams prm = {};
    prm.m = m; prm.n = n; prm.d = d;
    prm.kpad = (m + 15) & ~15;
    prm.npad = (n + 15) & ~15;
    prm.boxes = p / kDecBoxCols;
    // as few CTAs as keep the widest slab no wider than it must be (p = 12288 on 148 SMs: 128 CTAs of 3 boxes each), which
    // evens the slabs out and leaves the other SMs to kernels of other streams
    const int widest = (prm.boxes + ctx->sm_count - 1) / ctx->sm_count;
    const int ncta = (prm.boxes + widest - 1) / widest;
    prm.base = prm.boxes / ncta; prm.rem = prm.boxes % ncta;
    prm.nbmax = prm.base + (prm.rem > 0 ? 1 : 0);
    const uint32_t a_bytes = (uint32_t)prm.kpad * kDecRowBytes;
    const uint32_t stage_bytes = a_bytes + (uint32_t)prm.nbmax * kDecBoxBytes;
    const uint32_t ainv_tile = (uint32_t)prm.npad * kDecRowBytes;
    const uint32_t y_bytes = (uint32_t)prm.kpad * 16u * (uint32_t)(prm.nbmax * 8);
    // behind the last A-type tile (the second tile of A^-1 rows) the MMA still reads up to 128 rows' worth of bytes:
    // the tail of the allocation (Y' slab, barriers, padding) is made long enough for that
    uint32_t tail = ((y_bytes + 15u) & ~15u) + 512u /*barriers*/;
    if (ainv_tile + tail < kDecAReach) tail = kDecAReach - ainv_tile;
    const uint32_t fixed = 2u * ainv_tile + tail + 1024u /*alignment*/;
    int stages = (int)((kDecSmemBudget - fixed) / stage_bytes);
    if (stages > 12) stages = 12;
    // A stage must always be consumed by the same issuer thread: a thread that saw only every other phase of a stage's
    // barrier could take the completed phase before last for the one it waits for (parities repeat after two phases).
    stages -= stages % kDecIssuers;
    if (stages < kDecIssuers) return GELO_ERR_UNSUPPORTED;
    prm.stages = stages;
    const uint32_t smem = (uint32_t)stages * stage_bytes + fixed;
    prm.group = ctx->dec_group > 0 ? ctx->dec_group : ncta;
    {
        const int nkb = ceil_div(d, kDecBK), groups = ceil_div(ncta, prm.group);
        prm.kstep = nkb / groups > 0 ? nkb / groups : 1;
    }
    prm.C0 = Q; prm.C1 = K ? K : Q; prm.C2 = V ? V : Q;
    prm.ldc = nsplit == 3 ? p / 3 : p;
    prm.csplit = nsplit == 3 ? p / 3 : p;
    prm.out_f16 = dtype == GELO_F16 ? 1 : 0;
    prm.plain = Ainv ? 0 : 1;
    prm.wait_ns = ctx->wait_limit_ns;
    prm.status = ctx->status_dev;
    CUtensorMap mu, mww, mwn, ma;
    if (!map_kmajor(ctx, &mu, U, (uint64_t)d, (uint64_t)m, (uint64_t)d, (uint32_t)prm.kpad) ||
        !map_kmajor(ctx, &ma, Ainv ? Ainv : U, (uint64_t)m, (uint64_t)n, (uint64_t)(Ainv ? lda : d), (uint32_t)prm.npad) ||
        !map_w_boxes(ctx, &mww, W, (uint64_t)d, (uint64_t)p, (uint32_t)prm.nbmax) ||
        !map_w_boxes(ctx, &mwn, W, (uint64_t)d, (uint64_t)p, (uint32_t)(prm.base > 0 ? prm.base : 1)))
        return GELO_ERR_CUDA;
    static bool attr_done[64] = {};
    if (ctx->device >= 0 && ctx->device < 64 && !attr_done[ctx->device]) {
        GELO_CUDA_OK(cudaFuncSetAttribute(project_unmix_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kDecSmemBudget));
        attr_done[ctx->device] = true;
    }
    {
        ProfScope ps(ctx, PROF_GEMM_TC, 2.0 * m * (double)d * p + 2.0 * n * (double)m * p, st);
        project_unmix_kernel<<<ncta, kDecThreads, smem, st>>>(mu, mww, mwn, ma, prm);
    }
    return after_launch(ctx);
}

}  // namespace gelo
