// Fused GEGLU (Sec. 3.1, Eq. 2): out[r][c] = x[r][c] * GELU(x[r][C + c]) -- split, error function and product in one
// pass over memory, nothing stored in between.
//
// Memory-bound: 6 bytes move per fp16 output element (4 read, 2 written) against about fifty arithmetic instructions, so
// the kernel is built for bytes in flight: every thread fetches UNROLL pairs of 16-byte pieces (one of each half of a
// row) before it computes anything, and the grid is a small multiple of the SM count walking the tensor with a stride.
// 1 + erf(z) is evaluated as erfc(-z) (the same function): erfcf keeps its relative accuracy for very negative gates,
// where erff is within an ulp of -1 and the sum would cancel.
#pragma once
#include <cuda_fp16.h>
#include <stdint.h>

namespace sd_attn {

__device__ __forceinline__ float geglu_one(float a, float g) {
    return a * (0.5f * g * erfcf(-0.70710678118654752f * g));
}

constexpr int GEGLU_THREADS = 256;
constexpr int GEGLU_UNROLL = 4;

// VEC elements per 16-byte piece: 8 (fp16) or 4 (fp32); C is a multiple of VEC and both tensors are 16-byte aligned.
template <typename T, int VEC>
__global__ void __launch_bounds__(GEGLU_THREADS)
geglu_vector_kernel(const T* __restrict__ x, T* __restrict__ out, long long pieces, int pieces_per_row) {
    const long long stride = (long long)gridDim.x * GEGLU_THREADS;
    const long long two_c = 2ll * pieces_per_row * VEC;
    for (long long p0 = (long long)blockIdx.x * GEGLU_THREADS + threadIdx.x; p0 < pieces; p0 += stride * GEGLU_UNROLL) {
        uint4 a[GEGLU_UNROLL], g[GEGLU_UNROLL];
#pragma unroll
        for (int u = 0; u < GEGLU_UNROLL; ++u) {
            const long long p = p0 + u * stride;
            if (p < pieces) {
                const long long r = p / pieces_per_row;
                const T* src = x + r * two_c + (p - r * pieces_per_row) * VEC;
                a[u] = __ldg(reinterpret_cast<const uint4*>(src));
                g[u] = __ldg(reinterpret_cast<const uint4*>(src + (long long)pieces_per_row * VEC));
            }
        }
#pragma unroll
        for (int u = 0; u < GEGLU_UNROLL; ++u) {
            const long long p = p0 + u * stride;
            if (p < pieces) {
                uint4 o;
                if (VEC == 8) {
                    const __half2* ah = reinterpret_cast<const __half2*>(&a[u]);
                    const __half2* gh = reinterpret_cast<const __half2*>(&g[u]);
                    __half2* oh = reinterpret_cast<__half2*>(&o);
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        const float2 af = __half22float2(ah[k]), gf = __half22float2(gh[k]);
                        oh[k] = __floats2half2_rn(geglu_one(af.x, gf.x), geglu_one(af.y, gf.y));
                    }
                } else {
                    const float* af = reinterpret_cast<const float*>(&a[u]);
                    const float* gf = reinterpret_cast<const float*>(&g[u]);
                    float* of = reinterpret_cast<float*>(&o);
#pragma unroll
                    for (int k = 0; k < 4; ++k) of[k] = geglu_one(af[k], gf[k]);
                }
                *reinterpret_cast<uint4*>(out + p * VEC) = o;
            }
        }
    }
}

// Any C: one element per thread and step.
template <typename T>
__global__ void __launch_bounds__(GEGLU_THREADS)
geglu_scalar_kernel(const T* __restrict__ x, T* __restrict__ out, long long elems, int C) {
    const long long stride = (long long)gridDim.x * GEGLU_THREADS;
    for (long long e = (long long)blockIdx.x * GEGLU_THREADS + threadIdx.x; e < elems; e += stride) {
        const long long r = e / C;
        const T* src = x + r * 2ll * C + (e - r * C);
        const float a = (float)src[0], g = (float)src[C];
        out[e] = (T)geglu_one(a, g);
    }
}

}  // namespace sd_attn
