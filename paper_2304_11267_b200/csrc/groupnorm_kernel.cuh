// Fused group normalisation (Sec. 3.1, Eq. 1): mean, variance, normalisation and the per-channel affine of one
// (sample, group) in one thread block, the group read from global memory ONCE.
//
// In the model's NCHW layout a group -- C/G consecutive channels of HW values -- is one contiguous run of memory: 80 KB
// at the 64 x 64 level of the UNet (fp16), less below.  The block copies it into shared memory while summing it, takes
// the variance from the centred values there (two passes over shared memory: no cancellation, no second trip to DRAM)
// and writes the result straight from shared memory.  Memory-bound: 4 bytes per fp16 element (2 read, 2 written).
// A group that does not fit shared memory, or whose channels are not multiples of 16 bytes, takes the streaming form:
// three passes over global memory (the second and third hit the L2).
#pragma once
#include <cuda_fp16.h>
#include <stdint.h>

namespace sd_attn {

constexpr int GN_THREADS = 512;
constexpr int GN_MAX_STAGED_BYTES = 200 * 1024;

__device__ __forceinline__ float gn_to_float(__half v) { return __half2float(v); }
__device__ __forceinline__ float gn_to_float(float v) { return v; }
__device__ __forceinline__ void gn_from_float(__half& d, float v) { d = __float2half_rn(v); }
__device__ __forceinline__ void gn_from_float(float& d, float v) { d = v; }

// Sum over the block; every thread gets the result.  `scratch` holds one float per warp (+1).
__device__ __forceinline__ float gn_block_sum(float v, float* scratch) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    __syncthreads();   // scratch may still be read from the previous reduction
    if (lane == 0) scratch[warp] = v;
    __syncthreads();
    float t = lane < (GN_THREADS >> 5) ? scratch[lane] : 0.f;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
    return t;
}

struct GroupNormArgs {
    const void* x;
    const void* gamma;   // may be null
    const void* beta;    // may be null
    void* y;
    int C, G;
    long long HW;
    float eps;
};

// Staged form.  VEC = elements per 16-byte piece; HW and the group size are multiples of VEC, so a piece never
// straddles two channels.  The group is fetched with asynchronous 16-byte copies straight into shared memory, all of a
// thread's copies in flight at once (with loads through registers, four at a time, the fetch of an 80 KB group was
// three DRAM round trips long).  Every thread only ever touches the pieces it fetched itself, so no barrier separates
// the passes; the two block-wide sums are the only meeting points.
// (Sharing a group out among the blocks of a thread-block cluster, partial sums through distributed shared memory, was
// measured and dropped: 8.3-8.6 us for the UNet's largest layer with 1, 2 or 4 blocks per group, 15 us with 8, and
// slower at large batch -- the call is bound by its launch and its five dependent phases, not by one SM's bandwidth.)
template <typename T, int VEC>
__global__ void __launch_bounds__(GN_THREADS)
groupnorm_staged_kernel(const GroupNormArgs a) {
    extern __shared__ uint4 gn_smem[];
    __shared__ float scratch[GN_THREADS / 32 + 1];
    const int cpg = a.C / a.G;
    const long long n_elems = (long long)cpg * a.HW;
    const int pieces = (int)(n_elems / VEC);
    const int n = blockIdx.x / a.G, g = blockIdx.x % a.G;
    const long long base = ((long long)n * a.C + (long long)g * cpg) * a.HW;
    const uint4* src = reinterpret_cast<const uint4*>(static_cast<const T*>(a.x) + base);
    uint4* dst = reinterpret_cast<uint4*>(static_cast<T*>(a.y) + base);

    const uint32_t smem0 = (uint32_t)__cvta_generic_to_shared(gn_smem);
    for (int p = threadIdx.x; p < pieces; p += GN_THREADS)
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem0 + (uint32_t)p * 16u), "l"(src + p) : "memory");
    asm volatile("cp.async.commit_group;" ::: "memory");
    asm volatile("cp.async.wait_group 0;" ::: "memory");

    float sum = 0.f;
    for (int p = threadIdx.x; p < pieces; p += GN_THREADS) {
        const uint4 v = gn_smem[p];
        const T* e = reinterpret_cast<const T*>(&v);
#pragma unroll
        for (int k = 0; k < VEC; ++k) sum += gn_to_float(e[k]);
    }
    const float mu = gn_block_sum(sum, scratch) / (float)n_elems;
    float sq = 0.f;
    for (int p = threadIdx.x; p < pieces; p += GN_THREADS) {
        const uint4 v = gn_smem[p];
        const T* e = reinterpret_cast<const T*>(&v);
#pragma unroll
        for (int k = 0; k < VEC; ++k) {
            const float d = gn_to_float(e[k]) - mu;
            sq = fmaf(d, d, sq);
        }
    }
    const float var = gn_block_sum(sq, scratch) / (float)n_elems;
    const float rstd = 1.0f / sqrtf(var + a.eps);
    const int pieces_per_channel = (int)(a.HW / VEC);
    const T* gamma = static_cast<const T*>(a.gamma);
    const T* beta = static_cast<const T*>(a.beta);
    for (int p = threadIdx.x; p < pieces; p += GN_THREADS) {
        const int c = g * cpg + p / pieces_per_channel;
        const float ga = gamma ? gn_to_float(gamma[c]) : 1.f, be = beta ? gn_to_float(beta[c]) : 0.f;
        const float scale = rstd * ga, shift = fmaf(-mu, scale, be);   // y = x * scale + shift
        uint4 v = gn_smem[p];
        T* e = reinterpret_cast<T*>(&v);
#pragma unroll
        for (int k = 0; k < VEC; ++k) gn_from_float(e[k], fmaf(gn_to_float(e[k]), scale, shift));
        dst[p] = v;
    }
}

// Streaming form: any sizes, three passes over global memory.
template <typename T>
__global__ void __launch_bounds__(GN_THREADS)
groupnorm_streaming_kernel(const GroupNormArgs a) {
    __shared__ float scratch[GN_THREADS / 32 + 1];
    const int cpg = a.C / a.G;
    const long long n_elems = (long long)cpg * a.HW;
    const int n = blockIdx.x / a.G, g = blockIdx.x % a.G;
    const long long base = ((long long)n * a.C + (long long)g * cpg) * a.HW;
    const T* x = static_cast<const T*>(a.x) + base;
    T* y = static_cast<T*>(a.y) + base;
    float sum = 0.f;
    for (long long i = threadIdx.x; i < n_elems; i += GN_THREADS) sum += gn_to_float(x[i]);
    const float mu = gn_block_sum(sum, scratch) / (float)n_elems;
    float sq = 0.f;
    for (long long i = threadIdx.x; i < n_elems; i += GN_THREADS) {
        const float d = gn_to_float(x[i]) - mu;
        sq = fmaf(d, d, sq);
    }
    const float var = gn_block_sum(sq, scratch) / (float)n_elems;
    const float rstd = 1.0f / sqrtf(var + a.eps);
    const T* gamma = static_cast<const T*>(a.gamma);
    const T* beta = static_cast<const T*>(a.beta);
    for (long long i = threadIdx.x; i < n_elems; i += GN_THREADS) {
        const int c = g * cpg + (int)(i / a.HW);
        const float ga = gamma ? gn_to_float(gamma[c]) : 1.f, be = beta ? gn_to_float(beta[c]) : 0.f;
        const float scale = rstd * ga, shift = fmaf(-mu, scale, be);
        gn_from_float(y[i], fmaf(gn_to_float(x[i]), scale, shift));
    }
}

}  // namespace sd_attn
