// bf16 tensor-core GEMM for the three products of the offload (Eq. 1-3) on sm_100a:
// tcgen05.mma with the accumulator in tensor memory, operands staged in shared memory by
// TMA, fp32 accumulation, bf16 (or fp32) output.
//
//   C (M x N) = A (M x K, row-major, K contiguous)  *  B (K x N, row-major, N contiguous)
//
// * A tiles (128 rows x 64 k) land K-major, B tiles (64 k x 256 columns, as four 64-column
//   boxes) land N-major; both use the 128-byte swizzle that TMA writes and the MMA reads.
// * The K loop may run over two stacked B matrices (H then the shield rows S, Eq. 8): the
//   producer simply switches tensor maps; a block that straddles the seam is issued once per
//   map and TMA's out-of-bounds zero fill removes the rows that belong to the other matrix.
// * Ragged M, N, K are handled by the same zero fill on loads and by guarded stores.
// * The epilogue routes column blocks to up to three outputs (Q | K | V) and casts.
// * Persistent CTAs (one per SM), warp-specialised: warp 0 issues TMA, warp 1 issues MMA and
//   owns the tensor-memory allocation, warps 2-5 drain the accumulator.  Two accumulator
//   stages (2 x 256 columns) let the epilogue of one tile overlap the main loop of the next.
// * Every wait on an mbarrier is bounded; on expiry the CTA records GELO_ERR_TIMEOUT in the
//   context's status word, stops issuing work, releases tensor memory and returns.
#include <cuda.h>

#include "common.cuh"

namespace gelo {

namespace {

constexpr int BM = 128;
constexpr int BN = 256;
constexpr int BK = 64;
constexpr int kStages = 4;
constexpr int kAccStages = 2;
constexpr int kThreads = 192;
constexpr uint32_t kABytes = BM * BK * 2;            // 16 KiB
constexpr uint32_t kBBoxBytes = 64 * BK * 2;         // 8 KiB per 64-column box
constexpr uint32_t kBBytes = (BN / 64) * kBBoxBytes; // 32 KiB
constexpr uint32_t kStageBytes = kABytes + kBBytes;
constexpr uint32_t kSmemBytes = kStages * kStageBytes + 1024 /*alignment slack*/ + 256 /*barriers*/;
constexpr uint32_t kTmemCols = 512;
constexpr unsigned long long kWaitLimit = 40ull * 1000 * 1000;   // try_wait rounds before giving up

struct TcParams {
    int M, N;
    int kb_first;        // k-blocks read through map B (rows 0 .. b_split-1 of the stacked operand)
    int kb_second;       // k-blocks read through map B2
    int a_k0_second;     // A column of the first k-block of the second part (multiple of 8)
    int b_row0_second;   // row of B2 that meets that column (may be negative: zero filled)
    void* C0; void* C1; void* C2;
    int ldc, csplit;
    int out_f32;         // 1: fp32 output, 0: bf16
    int* status;
};

// ---- PTX wrappers -----------------------------------------------------------------------

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait: false when the limit ran out or another thread already gave up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag)
{
    for (unsigned long long spin = 0; spin < kWaitLimit; ++spin) {
        if (mbar_try(bar, parity)) return true;
        if ((spin & 1023) == 1023 && *abort_flag) return false;
    }
    return false;
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar) : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tc_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

__device__ __forceinline__ void tc_mma_bf16(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b, uint32_t idesc,
                                            uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(accumulate) : "memory");
}

__device__ __forceinline__ void tc_ld_32cols(uint32_t taddr, uint32_t v[32])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
          "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
          "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
          "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
        : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tc_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor (sm_100 format): start address, leading and stride byte
// offsets in 16-byte units, descriptor version 1, 128-byte swizzle.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes)
{
    uint64_t d = 0;
    d |= (uint64_t)((addr >> 4) & 0x3FFF);
    d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFF) << 16;
    d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFF) << 32;
    d |= (uint64_t)1 << 46;       // version
    d |= (uint64_t)2 << 61;       // SWIZZLE_128B
    return d;
}

// Instruction descriptor: fp32 accumulate, bf16 x bf16, A K-major, B N-major, M = 128, N = BN.
constexpr uint32_t kInstrDesc = (1u << 4) | (1u << 7) | (1u << 10) | (0u << 15) | (1u << 16) |
                                ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);

__device__ __forceinline__ uint32_t pack_bf16(uint32_t a, uint32_t b)
{
    __nv_bfloat162 h = __floats2bfloat162_rn(__uint_as_float(a), __uint_as_float(b));
    return *reinterpret_cast<uint32_t*>(&h);
}

// ---- the kernel ------------------------------------------------------------------------------

__global__ void __launch_bounds__(kThreads, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
               const __grid_constant__ CUtensorMap map_b2, const TcParams prm)
{
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t tiles_base = (raw + 1023u) & ~1023u;                 // swizzle atoms need 1024-byte alignment
    uint8_t* gen_base = smem_raw + (tiles_base - raw);
    const uint32_t bar_base = tiles_base + kStages * kStageBytes;
    uint8_t* bar_gen = gen_base + kStages * kStageBytes;
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
    const int total_tiles = m_tiles * n_tiles;
    const int kb_total = prm.kb_first + prm.kb_second;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        for (int a = 0; a < kAccStages; ++a) { mbar_init(acc_full_bar(a), 1); mbar_init(acc_empty_bar(a), 4); }
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
                const int m0 = (tile % m_tiles) * BM;
                const int n0 = (tile / m_tiles) * BN;
                for (int kb = 0; kb < kb_total; ++kb, ++it) {
                    const int s = it % kStages;
                    const uint32_t ph = (it / kStages) & 1u;
                    if (!mbar_wait(empty_bar(s), ph ^ 1u, abort_flag)) { ok = false; break; }
                    const bool second = kb >= prm.kb_first;
                    const int a_k = second ? prm.a_k0_second + (kb - prm.kb_first) * BK : kb * BK;
                    const int b_row = second ? prm.b_row0_second + (kb - prm.kb_first) * BK : kb * BK;
                    const CUtensorMap* mb = second ? &map_b2 : &map_b;
                    const uint32_t sa = tiles_base + s * kStageBytes;
                    const uint32_t sb = sa + kABytes;
                    mbar_expect_tx(full_bar(s), kStageBytes);
                    tma_load_2d(sa, &map_a, a_k, m0, full_bar(s));
#pragma unroll
                    for (int j = 0; j < BN / 64; ++j)
                        tma_load_2d(sb + j * kBBoxBytes, mb, n0 + j * 64, b_row, full_bar(s));
                }
            }
            if (!ok) { *abort_flag = 1; atomicCAS(prm.status, 0, (int)GELO_ERR_TIMEOUT); }
        }
    } else if (warp == 1) {
        // ================= MMA issuer =================
        if (lane == 0) {
            uint32_t it = 0, acc_it = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x, ++acc_it) {
                const int a = acc_it % kAccStages;
                const uint32_t aph = (acc_it / kAccStages) & 1u;
                if (!mbar_wait(acc_empty_bar(a), aph ^ 1u, abort_flag)) { ok = false; break; }
                tc_fence_after();
                const uint32_t tmem_d = tmem_base + (uint32_t)(a * BN);
                for (int kb = 0; kb < kb_total; ++kb, ++it) {
                    const int s = it % kStages;
                    const uint32_t ph = (it / kStages) & 1u;
                    if (!mbar_wait(full_bar(s), ph, abort_flag)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t sa = tiles_base + s * kStageBytes;
                    const uint32_t sb = sa + kABytes;
#pragma unroll
                    for (int ks = 0; ks < BK / 16; ++ks) {
                        // A: K-major, 8-row groups 1024 bytes apart, 32 bytes per 16-wide k step
                        const uint64_t da = smem_desc(sa + ks * 32, 16, 1024);
                        // B: N-major, 64-column boxes 8192 bytes apart, 8-row k groups 1024 bytes apart
                        const uint64_t db = smem_desc(sb + ks * 2048, kBBoxBytes, 1024);
                        tc_mma_bf16(tmem_d, da, db, kInstrDesc, (kb | ks) != 0 ? 1u : 0u);
                    }
                    tc_commit(empty_bar(s));          // frees the stage once these MMAs have read it
                }
                if (!ok) break;
                tc_commit(acc_full_bar(a));           // accumulator complete
            }
            if (!ok) { *abort_flag = 1; atomicCAS(prm.status, 0, (int)GELO_ERR_TIMEOUT); }
        }
    } else {
        // ================= epilogue (warps 2..5) =================
        const int quarter = warp & 3;                 // the TMEM lane quarter this warp may read
        uint32_t acc_it = 0;
        bool ok = true;
        for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x, ++acc_it) {
            const int a = acc_it % kAccStages;
            const uint32_t aph = (acc_it / kAccStages) & 1u;
            const int m0 = (tile % m_tiles) * BM;
            const int n0 = (tile / m_tiles) * BN;
            if (!mbar_wait(acc_full_bar(a), aph, abort_flag)) { ok = false; break; }
            tc_fence_after();
            const int gm = m0 + quarter * 32 + lane;
            const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(a * BN);
#pragma unroll 1
            for (int c = 0; c < BN; c += 32) {
                uint32_t v[32];
                tc_ld_32cols(taddr + c, v);
                tc_ld_wait();
                if (gm < prm.M) {
#pragma unroll
                    for (int g = 0; g < 4; ++g) {
                        const int gn = n0 + c + g * 8;
                        if (gn < prm.N) {
                            const int chunk = gn / prm.csplit;
                            void* base = chunk == 0 ? prm.C0 : (chunk == 1 ? prm.C1 : prm.C2);
                            const size_t off = (size_t)gm * prm.ldc + (gn - chunk * prm.csplit);
                            if (prm.out_f32) {
                                float4* dst = reinterpret_cast<float4*>(static_cast<float*>(base) + off);
                                dst[0] = make_float4(__uint_as_float(v[g * 8 + 0]), __uint_as_float(v[g * 8 + 1]),
                                                     __uint_as_float(v[g * 8 + 2]), __uint_as_float(v[g * 8 + 3]));
                                dst[1] = make_float4(__uint_as_float(v[g * 8 + 4]), __uint_as_float(v[g * 8 + 5]),
                                                     __uint_as_float(v[g * 8 + 6]), __uint_as_float(v[g * 8 + 7]));
                            } else {
                                uint4 pk;
                                pk.x = pack_bf16(v[g * 8 + 0], v[g * 8 + 1]);
                                pk.y = pack_bf16(v[g * 8 + 2], v[g * 8 + 3]);
                                pk.z = pack_bf16(v[g * 8 + 4], v[g * 8 + 5]);
                                pk.w = pack_bf16(v[g * 8 + 6], v[g * 8 + 7]);
                                *reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(base) + off) = pk;
                            }
                        }
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(acc_empty_bar(a));
        }
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
    return enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

}  // namespace

bool gemm_tc_supports(const GemmArgs& g)
{
    if (g.dtype != GELO_BF16 || g.transA || g.transB || g.alpha != 1.0f || g.beta != 0.0f) return false;
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
    static bool attr_done[64] = {};
    if (ctx->device >= 0 && ctx->device < 64 && !attr_done[ctx->device]) {
        GELO_CUDA_OK(cudaFuncSetAttribute(gemm_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes));
        attr_done[ctx->device] = true;
    }
    const int rows_first = g.B2 ? g.b_split : g.K;
    CUtensorMap ma, mb, mb2;
    if (!make_map(ctx, &ma, g.A, (uint64_t)g.K, (uint64_t)g.M, (uint64_t)g.lda, BK, BM)) return GELO_ERR_CUDA;
    if (!make_map(ctx, &mb, g.B, (uint64_t)g.N, (uint64_t)rows_first, (uint64_t)g.ldb, 64, BK)) return GELO_ERR_CUDA;
    if (g.B2) {
        if (!make_map(ctx, &mb2, g.B2, (uint64_t)g.N, (uint64_t)(g.K - g.b_split), (uint64_t)g.ldb, 64, BK))
            return GELO_ERR_CUDA;
    } else {
        mb2 = mb;
    }
    TcParams p;
    p.M = g.M; p.N = g.N;
    p.kb_first = ceil_div(rows_first, BK);
    if (g.B2) {
        p.a_k0_second = g.b_split & ~7;                       // TMA needs a 16-byte aligned inner coordinate
        p.b_row0_second = p.a_k0_second - g.b_split;          // <= 0: rows above S read as zero
        p.kb_second = ceil_div(g.K - p.a_k0_second, BK);
    } else {
        p.a_k0_second = 0; p.b_row0_second = 0; p.kb_second = 0;
    }
    p.C0 = g.C[0]; p.C1 = g.C[g.nsplit > 1 ? 1 : 0]; p.C2 = g.C[g.nsplit > 2 ? 2 : 0];
    p.ldc = g.ldc; p.csplit = g.N / g.nsplit;
    p.out_f32 = 0;
    p.status = ctx->status_dev;
    const int tiles = ceil_div(g.M, BM) * ceil_div(g.N, BN);
    const int grid = tiles < ctx->sm_count ? tiles : ctx->sm_count;
    {
        ProfScope ps(ctx, PROF_GEMM_TC, 2.0 * g.M * (double)g.N * g.K, st);
        gemm_tc_kernel<<<grid, kThreads, kSmemBytes, st>>>(ma, mb, mb2, p);
    }
    return after_launch(ctx);
}

}  // namespace gelo
