// Inline-PTX wrappers shared by the tensor-core kernels of this library (sm_100a): mbarriers with time-bounded
// waits, TMA tile loads, tcgen05 MMA / commit / tensor-memory loads, shared-memory matrix descriptors.
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <stdint.h>

namespace gelo {
namespace tcx {

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
__device__ __forceinline__ unsigned long long global_ns()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}
// Bounded wait: false when `limit_ns` nanoseconds (by the GPU's global timer) have passed or another thread of the
// CTA already gave up.  A limit of zero gives up without looking at the barrier at all, so a CTA launched with it
// leaves before any copy or MMA has been issued.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, unsigned long long limit_ns)
{
    if (limit_ns == 0) return false;
    if (mbar_try(bar, parity)) return true;
    const unsigned long long t0 = global_ns();
    for (;;) {
#pragma unroll 1
        for (int spin = 0; spin < 256; ++spin)
            if (mbar_try(bar, parity)) return true;
        if (*abort_flag) return false;
        if (global_ns() - t0 > limit_ns) return false;
    }
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar) : "memory");
}

__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, int x, int y, int z, uint32_t bar)
{
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
        ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(z), "r"(bar) : "memory");
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

__device__ __forceinline__ void tc_mma_tf32(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b, uint32_t idesc,
                                            uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(accumulate) : "memory");
}

// The four MMA instructions of one operand stage (k advances by `astep` / `bstep` sixteen-byte units of the descriptors'
// start address), with a barrier test tucked in front of them: the test of the NEXT stage's "full" barrier takes about
// a hundred cycles to answer, and asked here its answer arrives while the four instructions issue instead of holding
// up the next stage.  Returns whether that barrier phase had completed.
#define GELO_TC_MMA4_TRY(KIND)                                                                                          \
    uint32_t ready;                                                                                                     \
    asm volatile(                                                                                                       \
        "{\n\t.reg .pred q, p;\n\t"                                                                                    \
        "mbarrier.try_wait.parity.shared::cta.b64 q, [%8], %9;\n\t"                                                     \
        "setp.ne.b32 p, %7, 0;\n\t"                                                                                     \
        "tcgen05.mma.cta_group::1.kind::" KIND " [%1], %2, %3, %6, p;\n\t"                                              \
        "tcgen05.mma.cta_group::1.kind::" KIND " [%1], %4, %5, %6, 1;\n\t"                                              \
        "tcgen05.mma.cta_group::1.kind::" KIND " [%1], %10, %11, %6, 1;\n\t"                                            \
        "tcgen05.mma.cta_group::1.kind::" KIND " [%1], %12, %13, %6, 1;\n\t"                                            \
        "selp.u32 %0, 1, 0, q;\n\t}"                                                                                    \
        : "=r"(ready)                                                                                                   \
        : "r"(tmem_d), "l"(da), "l"(db), "l"(da + astep), "l"(db + bstep), "r"(idesc), "r"(accumulate), "r"(next_bar),  \
          "r"(next_parity), "l"(da + 2 * astep), "l"(db + 2 * bstep), "l"(da + 3 * astep), "l"(db + 3 * bstep)          \
        : "memory");                                                                                                    \
    return ready != 0;

__device__ __forceinline__ bool tc_mma4_bf16_try(uint32_t tmem_d, uint64_t da, uint64_t db, uint64_t astep, uint64_t bstep,
                                                 uint32_t idesc, uint32_t accumulate, uint32_t next_bar, uint32_t next_parity)
{
    GELO_TC_MMA4_TRY("f16")
}
__device__ __forceinline__ bool tc_mma4_tf32_try(uint32_t tmem_d, uint64_t da, uint64_t db, uint64_t astep, uint64_t bstep,
                                                 uint32_t idesc, uint32_t accumulate, uint32_t next_bar, uint32_t next_parity)
{
    GELO_TC_MMA4_TRY("tf32")
}
__device__ __forceinline__ bool tc_mma4_f8_try(uint32_t tmem_d, uint64_t da, uint64_t db, uint64_t astep, uint64_t bstep,
                                               uint32_t idesc, uint32_t accumulate, uint32_t next_bar, uint32_t next_parity)
{
    GELO_TC_MMA4_TRY("f8f6f4")
}
#undef GELO_TC_MMA4_TRY

__device__ __forceinline__ float round_tf32(float x)
{
    uint32_t r;
    asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(r) : "f"(x));
    return __uint_as_float(r);
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
// Layout type 2: 128-byte swizzle of 16-byte chunks (8-row atoms).  Layout type 1: 128-byte swizzle of 32-byte
// chunks (4-row atoms), the only layout that 32-bit operands may use when they are not K-major.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes, uint32_t layout = 2)
{
    uint64_t d = 0;
    d |= (uint64_t)((addr >> 4) & 0x3FFF);
    d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFF) << 16;
    d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFF) << 32;
    d |= (uint64_t)1 << 46;       // version
    d |= (uint64_t)layout << 61;
    return d;
}



__device__ __forceinline__ uint32_t pack_bf16(uint32_t a, uint32_t b)
{
    __nv_bfloat162 h = __floats2bfloat162_rn(__uint_as_float(a), __uint_as_float(b));
    return *reinterpret_cast<uint32_t*>(&h);
}
__device__ __forceinline__ uint32_t pack_f16(uint32_t a, uint32_t b)
{
    __half2 h = __floats2half2_rn(__uint_as_float(a), __uint_as_float(b));
    return *reinterpret_cast<uint32_t*>(&h);
}

}  // namespace tcx
}  // namespace gelo
