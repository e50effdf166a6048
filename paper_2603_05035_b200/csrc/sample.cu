// On-device sampling for the secret mixing matrix and the shield rows
// (paper Section 3.2 step 1.2; Mitigation 2).  Philox4x32-10 as published by
// Salmon, Moraes, Dror and Shaw (SC'11); one 32-bit word per matrix element;
// Box-Muller on word pairs.  HBM-bound: each thread produces one 4-word block
// and writes four consecutive elements.
#include "common.cuh"
#include "philox.cuh"

namespace gelo {

__global__ void philox_words_kernel(uint64_t seed, uint32_t stream_id, uint32_t attempt,
                                    uint64_t first, uint64_t count, uint32_t* __restrict__ out)
{
    // thread t covers block (first / 4 + t); elements outside [first, first + count) are skipped
    const uint64_t q0 = first >> 2;
    const uint64_t t = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const uint64_t q = q0 + t;
    const uint64_t e0 = q << 2;
    if (e0 >= first + count) return;
    uint32_t w[4];
    philox_block(seed, q, stream_id, attempt, w);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const uint64_t e = e0 + i;
        if (e >= first && e < first + count) out[e - first] = w[i];
    }
}

__global__ void gaussian_kernel(int rows, int cols, int ld, uint64_t seed_value, const uint64_t* __restrict__ seed_ptr,
                                uint32_t stream_id, uint32_t attempt, float scale, const float* __restrict__ base,
                                float* __restrict__ out)
{
    // a replayed launch graph cannot change by-value arguments, so the seed may come from device memory
    const uint64_t seed = seed_ptr ? *seed_ptr : seed_value;
    const uint64_t total = (uint64_t)rows * (uint64_t)cols;
    const uint64_t q = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const uint64_t e0 = q << 2;
    if (e0 >= total) return;
    float z[4];
    gaussian_block(seed, q, stream_id, attempt, z);
    const uint64_t i0 = e0 / (uint64_t)cols;
    const uint32_t j0 = (uint32_t)(e0 - i0 * (uint64_t)cols);
    if (((cols | ld) & 3) == 0) {
        // the four elements share a row and start on a 16-byte boundary
        const size_t off = (size_t)i0 * ld + j0;
        float4 v = make_float4(scale * z[0], scale * z[1], scale * z[2], scale * z[3]);
        if (base) {
            const float4 b = *reinterpret_cast<const float4*>(base + off);
            v.x += b.x; v.y += b.y; v.z += b.z; v.w += b.w;
        }
        *reinterpret_cast<float4*>(out + off) = v;
    } else {
        uint64_t i = i0;
        uint32_t j = j0;
#pragma unroll
        for (int t = 0; t < 4; ++t) {
            if (e0 + t < total) {
                const size_t off = (size_t)i * ld + j;
                out[off] = (base ? base[off] : 0.0f) + scale * z[t];
            }
            if (++j == (uint32_t)cols) { j = 0; ++i; }
        }
    }
}

int launch_philox_words(gelo_ctx* ctx, uint64_t seed, uint32_t stream_id, uint32_t attempt,
                        uint64_t first, uint64_t count, uint32_t* out, cudaStream_t st)
{
    if (count == 0) return GELO_OK;
    const uint64_t blocks_needed = ((first + count + 3) >> 2) - (first >> 2);
    const unsigned threads = 256;
    const uint64_t grid = (blocks_needed + threads - 1) / threads;
    if (grid > 0x7fffffffull) return GELO_ERR_INVALID;
    philox_words_kernel<<<(unsigned)grid, threads, 0, st>>>(seed, stream_id, attempt, first, count, out);
    return after_launch(ctx);
}

int launch_gaussian(gelo_ctx* ctx, int rows, int cols, int ld, uint64_t seed, uint32_t stream_id,
                    uint32_t attempt, float scale, const float* base, float* out, cudaStream_t st,
                    const uint64_t* seed_dev)
{
    const uint64_t total = (uint64_t)rows * (uint64_t)cols;
    if (total == 0) return GELO_OK;
    const unsigned threads = 256;
    const uint64_t grid = ((total + 3) / 4 + threads - 1) / threads;
    if (grid > 0x7fffffffull) return GELO_ERR_INVALID;
    gaussian_kernel<<<(unsigned)grid, threads, 0, st>>>(rows, cols, ld, seed, seed_dev, stream_id, attempt, scale, base, out);
    return after_launch(ctx);
}

}  // namespace gelo
