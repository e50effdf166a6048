// Shield rows (paper Mitigation 2, Eq. 7-8): k Gaussian rows scaled to a multiple of the
// median Euclidean row norm of H, appended below the data rows before mixing.
//   1. row norms of H            -- one HBM pass, one warp per row, 16-byte loads
//   2. median by rank counting   -- every element counts how many others precede it
//   3. S = (scale * med / sqrt(d)) * N(0,1) from Philox stream 2
#include <cooperative_groups.h>

#include "common.cuh"
#include "philox.cuh"

namespace gelo {

namespace {

__device__ __forceinline__ float sumsq8(const uint4& q)
{
    const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&q);
    float s = 0.0f;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const float2 f = __bfloat1622float2(h[i]);
        s = fmaf(f.x, f.x, s);
        s = fmaf(f.y, f.y, s);
    }
    return s;
}

__device__ __forceinline__ float sumsq8h(const uint4& q)
{
    const __half2* h = reinterpret_cast<const __half2*>(&q);
    float s = 0.0f;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const float2 f = __half22float2(h[i]);
        s = fmaf(f.x, f.x, s);
        s = fmaf(f.y, f.y, s);
    }
    return s;
}

template <typename T> struct is_half_t { static constexpr bool value = false; };
template <> struct is_half_t<__half> { static constexpr bool value = true; };

// Euclidean norm of one row by one warp (16-byte loads, lanes strided over the row, butterfly sum): the same
// summation order wherever it is used, so every route to the shield rows gives the same bytes.
template <typename T>
__device__ __forceinline__ float warp_row_norm(const T* __restrict__ h, int d, int lane)
{
    float s = 0.0f;
    if (sizeof(T) == 4) {
        const float4* h4 = reinterpret_cast<const float4*>(h);
        for (int j = lane; j < d / 4; j += 32) {
            const float4 v = __ldg(h4 + j);
            s = fmaf(v.x, v.x, s); s = fmaf(v.y, v.y, s); s = fmaf(v.z, v.z, s); s = fmaf(v.w, v.w, s);
        }
    } else {
        // eight 16-byte loads in flight per lane; the partial sums are added in the order of the plain loop
        const uint4* h8 = reinterpret_cast<const uint4*>(h);
        const int g = d / 8;
        int j = lane;
        for (; j + 7 * 32 < g; j += 8 * 32) {
            uint4 v[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) v[u] = __ldg(h8 + j + u * 32);
#pragma unroll
            for (int u = 0; u < 8; ++u) s += is_half_t<T>::value ? sumsq8h(v[u]) : sumsq8(v[u]);
        }
        for (; j < g; j += 32) s += is_half_t<T>::value ? sumsq8h(__ldg(h8 + j)) : sumsq8(__ldg(h8 + j));
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) s += __shfl_xor_sync(0xffffffffu, s, off);
    return sqrtf(s);
}

template <typename T>
__global__ void __launch_bounds__(256) row_norm_kernel(const T* __restrict__ H, int n, int d, float* __restrict__ norms)
{
    const int row = blockIdx.x * 8 + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (row >= n) return;
    const float v = warp_row_norm(H + (size_t)row * d, d, lane);
    if (lane == 0) norms[row] = v;
}

// med[0], med[1] = the elements of rank (n-1)/2 and n/2 (ties broken by index).
__global__ void __launch_bounds__(256) median_rank_kernel(const float* __restrict__ norms, int n, float* __restrict__ med)
{
    __shared__ float tile[256];
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    const float mine = (i < n) ? norms[i] : 0.0f;
    int rank = 0;
    for (int base = 0; base < n; base += 256) {
        const int j = base + threadIdx.x;
        tile[threadIdx.x] = (j < n) ? norms[j] : 0.0f;
        __syncthreads();
        const int lim = min(256, n - base);
        for (int t = 0; t < lim; ++t) {
            const float o = tile[t];
            rank += (o < mine || (o == mine && base + t < i)) ? 1 : 0;
        }
        __syncthreads();
    }
    if (i < n) {
        if (rank == (n - 1) / 2) med[0] = mine;
        if (rank == n / 2) med[1] = mine;
    }
}

template <typename T>
__device__ __forceinline__ void store_shield_block(T* __restrict__ S, uint64_t e0, float f, uint64_t seed, uint64_t q, int nu);

// Standardised Student-t draw of element e (Section 4.4.1, Table 9 names Student-t shields): the element owns
// B = 4 ceil((nu + 1) / 4) positions of the Gaussian stream (seed, shield stream, attempt word = nu) from e * B on,
//     t = g_0 / sqrt((g_1^2 + ... + g_nu^2) / nu),   x = t sqrt((nu - 2) / nu)     (unit variance for nu > 2).
__device__ __forceinline__ float student_t_draw(uint64_t seed, uint64_t e, int nu)
{
    const uint64_t blocks = (uint64_t)((nu + 1 + 3) >> 2);
    float g0 = 0.0f, chi = 0.0f;
    for (uint64_t b = 0; b < blocks; ++b) {
        float z[4];
        gaussian_block(seed, e * blocks + b, GELO_STREAM_SHIELD, (uint32_t)nu, z);
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int idx = (int)b * 4 + j;
            if (idx == 0) g0 = z[j];
            else if (idx <= nu) chi = fmaf(z[j], z[j], chi);
        }
    }
    return g0 / sqrtf(chi / (float)nu) * sqrtf(((float)nu - 2.0f) / (float)nu);
}

template <typename T>
__global__ void __launch_bounds__(256) shield_fill_kernel(T* __restrict__ S, int k, int d, float scale,
                                                          const float* __restrict__ med, uint64_t seed, int nu)
{
    const uint64_t total = (uint64_t)k * d;
    const uint64_t q = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const uint64_t e0 = q << 2;
    if (e0 >= total) return;                      // d % 8 == 0, so blocks never straddle the end
    const float f = scale * (0.5f * (med[0] + med[1])) / sqrtf((float)d);
    store_shield_block(S, e0, f, seed, q, nu);
}

// S[e0 .. e0+3] = f * (the four normals of block q of the shield stream), in the storage type
template <typename T>
__device__ __forceinline__ void store_shield_block(T* __restrict__ S, uint64_t e0, float f, uint64_t seed, uint64_t q, int nu)
{
    float z[4];
    if (nu > 0) {
#pragma unroll
        for (int j = 0; j < 4; ++j) z[j] = student_t_draw(seed, e0 + j, nu);
    } else {
        gaussian_block(seed, q, GELO_STREAM_SHIELD, 0u, z);
    }
    if (sizeof(T) == 4) {
        *reinterpret_cast<float4*>(reinterpret_cast<float*>(S) + e0) = make_float4(f * z[0], f * z[1], f * z[2], f * z[3]);
    } else if (is_half_t<T>::value) {
        __half2 lo = __floats2half2_rn(f * z[0], f * z[1]);
        __half2 hi = __floats2half2_rn(f * z[2], f * z[3]);
        uint2 pk;
        pk.x = *reinterpret_cast<uint32_t*>(&lo);
        pk.y = *reinterpret_cast<uint32_t*>(&hi);
        *reinterpret_cast<uint2*>(reinterpret_cast<__half*>(S) + e0) = pk;
    } else {
        __nv_bfloat162 lo = __floats2bfloat162_rn(f * z[0], f * z[1]);
        __nv_bfloat162 hi = __floats2bfloat162_rn(f * z[2], f * z[3]);
        uint2 pk;
        pk.x = *reinterpret_cast<uint32_t*>(&lo);
        pk.y = *reinterpret_cast<uint32_t*>(&hi);
        *reinterpret_cast<uint2*>(reinterpret_cast<__nv_bfloat16*>(S) + e0) = pk;
    }
}

// All three steps in ONE launch for a batch of at most 256 rows (the decode-shaped call, where three dependent
// launches cost more than their work): a thread-block cluster of up to 8 CTAs, one warp per row for the norms, every
// norm stored into every CTA's shared memory (distributed shared memory), one cluster barrier, then each CTA ranks
// the norms for itself and fills its share of S.  Same arithmetic in the same order as the three kernels above.
constexpr int kShieldSmallRows = 256;

template <typename T>
__global__ void __launch_bounds__(1024, 1)
shield_small_kernel(const T* __restrict__ H, int n, int d, int k, float scale, uint64_t seed, T* __restrict__ S, int nu)
{
    namespace cg = cooperative_groups;
    cg::cluster_group cluster = cg::this_cluster();
    const int CS = (int)cluster.num_blocks();
    const int rank = (int)cluster.block_rank();
    __shared__ float norms_s[kShieldSmallRows];
    __shared__ float med_s[2];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int row = rank * 32 + warp;
    if (row < n) {
        const float v = warp_row_norm(H + (size_t)row * d, d, lane);
        if (lane < CS) cluster.map_shared_rank(&norms_s[row], lane)[0] = v;
    }
    if (CS > 1) cluster.sync(); else __syncthreads();
    const int i = threadIdx.x;
    if (i < n) {
        const float mine = norms_s[i];
        int rk = 0;
        for (int t = 0; t < n; ++t) {
            const float o = norms_s[t];
            rk += (o < mine || (o == mine && t < i)) ? 1 : 0;
        }
        if (rk == (n - 1) / 2) med_s[0] = mine;
        if (rk == n / 2) med_s[1] = mine;
    }
    __syncthreads();
    const float f = scale * (0.5f * (med_s[0] + med_s[1])) / sqrtf((float)d);
    const uint64_t blocks = ((uint64_t)k * d) >> 2;           // d % 8 == 0
    for (uint64_t q = (uint64_t)rank * 1024 + threadIdx.x; q < blocks; q += (uint64_t)CS * 1024)
        store_shield_block(S, q << 2, f, seed, q, nu);
}

template <typename T>
int launch_shield_small(gelo_ctx* ctx, const void* H, int n, int d, int k, float scale, uint64_t seed, void* S, int nu, cudaStream_t st)
{
    const int cs = ceil_div(n, 32);                           // <= 8
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(cs, 1, 1);
    cfg.blockDim = dim3(1024, 1, 1);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = cs; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&cfg, shield_small_kernel<T>, static_cast<const T*>(H), n, d, k, scale, seed, static_cast<T*>(S), nu) != cudaSuccess)
        return GELO_ERR_CUDA;
    return after_launch(ctx);
}

}  // namespace

ShieldScratch carve_shield(Arena& a, int n)
{
    ShieldScratch s;
    s.norms = static_cast<float*>(a.take((size_t)(n > 0 ? n : 1) * sizeof(float)));
    s.med = static_cast<float*>(a.take(4 * sizeof(float)));
    return s;
}

int run_shield_rows(gelo_ctx* ctx, const void* H, int n, int d, int k, float scale, uint64_t seed,
                    int dtype, void* S, const ShieldScratch& s, cudaStream_t st, int nu)
{
    if (k <= 0) return GELO_OK;
    if (nu != 0 && (nu < 3 || nu > 63)) return GELO_ERR_INVALID;
    if (n <= kShieldSmallRows) {
        if (dtype == GELO_BF16) return launch_shield_small<__nv_bfloat16>(ctx, H, n, d, k, scale, seed, S, nu, st);
        if (dtype == GELO_F16) return launch_shield_small<__half>(ctx, H, n, d, k, scale, seed, S, nu, st);
        return launch_shield_small<float>(ctx, H, n, d, k, scale, seed, S, nu, st);
    }
    if (dtype == GELO_BF16)
        row_norm_kernel<__nv_bfloat16><<<ceil_div(n, 8), 256, 0, st>>>(static_cast<const __nv_bfloat16*>(H), n, d, s.norms);
    else if (dtype == GELO_F16)
        row_norm_kernel<__half><<<ceil_div(n, 8), 256, 0, st>>>(static_cast<const __half*>(H), n, d, s.norms);
    else
        row_norm_kernel<float><<<ceil_div(n, 8), 256, 0, st>>>(static_cast<const float*>(H), n, d, s.norms);
    GELO_TRY(after_launch(ctx));
    median_rank_kernel<<<ceil_div(n, 256), 256, 0, st>>>(s.norms, n, s.med);
    GELO_TRY(after_launch(ctx));
    const uint64_t blocks = ((uint64_t)k * d + 3) / 4;
    const unsigned grid = (unsigned)((blocks + 255) / 256);
    if (dtype == GELO_BF16)
        shield_fill_kernel<__nv_bfloat16><<<grid, 256, 0, st>>>(static_cast<__nv_bfloat16*>(S), k, d, scale, s.med, seed, nu);
    else if (dtype == GELO_F16)
        shield_fill_kernel<__half><<<grid, 256, 0, st>>>(static_cast<__half*>(S), k, d, scale, s.med, seed, nu);
    else
        shield_fill_kernel<float><<<grid, 256, 0, st>>>(static_cast<float*>(S), k, d, scale, s.med, seed, nu);
    return after_launch(ctx);
}


// ---------------------------------------------------------------------------------------
// Shield rows without any allocation.
//
// Some callers cannot hand the library a workspace because they cannot allocate device
// memory themselves: code running inside an enclave-style runtime whose allocator is
// frozen after start-up, a plugin called from a serving engine that owns every byte of
// the memory pool, or a call site inside a region where cudaMalloc is forbidden.  For them
// the scratch of the shield-row step (one row norm per data row, two median slots) lives
// in a fixed array inside the library image.  Every GPU that loads the library carries
// this array until the process exits.
// ---------------------------------------------------------------------------------------

namespace {

constexpr int kStaticShieldMaxRows = 65536;                        // 256 KiB of row norms
constexpr int kStaticShieldFloats = kStaticShieldMaxRows + 64;     // + median slots, padded

static __device__ __align__(256) float g_shield_static_scratch[kStaticShieldFloats];

constexpr int kMaxDevices = 64;
float* g_shield_static_ptr[kMaxDevices] = {};                      // device address per GPU, 0 = not yet resolved

// The array's name is only a handle on the host; the device address has to be asked for,
// once per device, with that device current.
int static_scratch_for_current_device(int device, float** out)
{
    if (device < 0 || device >= kMaxDevices) return GELO_ERR_UNSUPPORTED;
    float* p = __atomic_load_n(&g_shield_static_ptr[device], __ATOMIC_ACQUIRE);
    if (!p) {
        void* addr = nullptr;
        if (cudaGetSymbolAddress(&addr, g_shield_static_scratch) != cudaSuccess || !addr) return GELO_ERR_CUDA;
        p = static_cast<float*>(addr);
        __atomic_store_n(&g_shield_static_ptr[device], p, __ATOMIC_RELEASE);
    }
    *out = p;
    return GELO_OK;
}

}  // namespace

}  // namespace gelo

extern "C" int gelo_shield_rows_static(gelo_ctx* ctx, const void* H_dev, int n, int d, int k, float scale,
                                       uint64_t seed, int dtype, void* S_dev, void* stream)
{
    using namespace gelo;
    if (!ctx || n <= 0 || d <= 0 || k < 0 || (dtype != GELO_F32 && dtype != GELO_BF16 && dtype != GELO_F16) || (d % 8) != 0 || !H_dev ||
        (reinterpret_cast<uintptr_t>(H_dev) & 15u))
        return GELO_ERR_INVALID;
    if (n > kStaticShieldMaxRows) return GELO_ERR_UNSUPPORTED;     // more rows than the built-in scratch holds
    if (k == 0) return GELO_OK;
    if (!S_dev || (reinterpret_cast<uintptr_t>(S_dev) & 15u)) return GELO_ERR_INVALID;

    int prev = -1;
    if (cudaGetDevice(&prev) != cudaSuccess) return GELO_ERR_CUDA;
    if (prev != ctx->device && cudaSetDevice(ctx->device) != cudaSuccess) return GELO_ERR_CUDA;
    float* scratch = nullptr;
    int rc = static_scratch_for_current_device(ctx->device, &scratch);
    if (rc == GELO_OK) {
        cudaStream_t st = static_cast<cudaStream_t>(stream);
        ShieldScratch s;
        s.norms = scratch;
        s.med = scratch + kStaticShieldMaxRows;
        // the array keeps what the previous call left: the median slots start from zero each time
        if (cudaMemsetAsync(s.med, 0, 2 * sizeof(float), st) != cudaSuccess) rc = GELO_ERR_CUDA;
        if (rc == GELO_OK) rc = run_shield_rows(ctx, H_dev, n, d, k, scale, seed, dtype, S_dev, s, st);
    }
    if (prev != ctx->device) cudaSetDevice(prev);
    return rc;
}
