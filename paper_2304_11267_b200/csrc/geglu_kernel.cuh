// Fused GEGLU (Sec. 3.1, Eq. 2): out[r][c] = x[r][c] * GELU(x[r][C + c]) -- split, error function and product in one
// pass over memory, nothing stored in between.
//
// Memory-bound -- if the arithmetic is kept short: 6 bytes move per fp16 output element (4 read, 2 written), which at the
// measured copy rate leaves an SM about 28 issue slots per element.  The library erfcf costs about 60 instructions per
// element (measured: 27 us for the 8192 x 1280 tensor, a third of the copy rate), so 1 + erf(g / sqrt 2) = erfc(-g / sqrt 2)
// is evaluated here as
//     erfc(z) = t * exp2(p(t) - z^2 log2 e),   t = 1 / (1 + z/2),   z = |g| / sqrt 2 >= 0,   erfc(-z) = 2 - erfc(z),
// with p the degree-10 polynomial fitted by gen_erfc_coeffs.py to log2(exp(z^2) erfc(z) / t) on z in [0, 10] (relative
// error of erfc in binary32: 6e-7 for z <= 2, growing with the rounding of z^2 like 2 z^2 * 2^-24 beyond): one
// reciprocal, one exp2, a dozen FMAs.  The form keeps its RELATIVE accuracy for very negative gates, where 1 + erf
// would cancel.  Every thread fetches UNROLL pairs of 16-byte pieces (one of each half of a row) before it computes
// anything, and the grid is a small multiple of the SM count walking the tensor with a stride.
#pragma once
#include <cuda_fp16.h>
#include <stdint.h>

namespace sd_attn {

// p(t), lowest order first: printed by gen_erfc_coeffs.py
template <int K>
__device__ __forceinline__ constexpr float geglu_p() {
    constexpr float P[11] = {-1.825843165e+00f, 1.445318174e+00f, 5.095620223e-01f, 3.360390315e-01f, -1.062030913e+00f,
                             2.482281915e+00f, -5.237285339e+00f, 6.225188260e+00f, -4.092804347e+00f, 1.428640074e+00f,
                             -2.090657097e-01f};
    return P[K];
}

__device__ __forceinline__ float geglu_one(float a, float g) {
    const float z = fabsf(g) * 0.70710678118654752f;
    float t, e;
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(t) : "f"(fmaf(0.5f, z, 1.0f)));
    float p = fmaf(geglu_p<10>(), t, geglu_p<9>());
    p = fmaf(p, t, geglu_p<8>());
    p = fmaf(p, t, geglu_p<7>());
    p = fmaf(p, t, geglu_p<6>());
    p = fmaf(p, t, geglu_p<5>());
    p = fmaf(p, t, geglu_p<4>());
    p = fmaf(p, t, geglu_p<3>());
    p = fmaf(p, t, geglu_p<2>());
    p = fmaf(p, t, geglu_p<1>());
    p = fmaf(p, t, geglu_p<0>());
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e) : "f"(fmaf(z * -1.4426950408889634f, z, p)));
    e *= t;                                        // erfc(z)
    const float two_phi = g < 0.f ? e : 2.0f - e;  // erfc(-g / sqrt 2) = 1 + erf(g / sqrt 2)
    return a * (0.5f * g * two_phi);
}

// The same for two elements at once on the packed binary32 pipe (one instruction, two results): the kernel is bound by
// instruction issue otherwise (34 instructions per element measured with the scalar form, 18 at the copy rate).
__device__ __forceinline__ uint64_t geglu_dup(float v) {
    const uint32_t b = __float_as_uint(v);
    return ((uint64_t)b << 32) | b;
}
__device__ __forceinline__ uint64_t geglu_mul2(uint64_t a, uint64_t b) {
    uint64_t d;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ uint64_t geglu_fma2(uint64_t a, uint64_t b, uint64_t c) {
    uint64_t d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ uint64_t geglu_add2(uint64_t a, uint64_t b) {
    uint64_t d;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ float2 geglu_two(float2 a, float2 g) {
    const uint32_t g0 = __float_as_uint(g.x), g1 = __float_as_uint(g.y);
    const uint64_t gg = ((uint64_t)g1 << 32) | g0;
    const uint64_t ag = ((uint64_t)(g1 & 0x7fffffffu) << 32) | (g0 & 0x7fffffffu);                 // |g|
    const uint64_t z = geglu_mul2(ag, geglu_dup(0.70710678118654752f));
    const uint64_t den = geglu_fma2(z, geglu_dup(0.5f), geglu_dup(1.0f));
    float t0, t1, e0, e1;
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(t0) : "f"(__uint_as_float((uint32_t)den)));
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(t1) : "f"(__uint_as_float((uint32_t)(den >> 32))));
    const uint64_t t = ((uint64_t)__float_as_uint(t1) << 32) | __float_as_uint(t0);
    uint64_t p = geglu_fma2(geglu_dup(geglu_p<10>()), t, geglu_dup(geglu_p<9>()));
    p = geglu_fma2(p, t, geglu_dup(geglu_p<8>()));
    p = geglu_fma2(p, t, geglu_dup(geglu_p<7>()));
    p = geglu_fma2(p, t, geglu_dup(geglu_p<6>()));
    p = geglu_fma2(p, t, geglu_dup(geglu_p<5>()));
    p = geglu_fma2(p, t, geglu_dup(geglu_p<4>()));
    p = geglu_fma2(p, t, geglu_dup(geglu_p<3>()));
    p = geglu_fma2(p, t, geglu_dup(geglu_p<2>()));
    p = geglu_fma2(p, t, geglu_dup(geglu_p<1>()));
    p = geglu_fma2(p, t, geglu_dup(geglu_p<0>()));
    const uint64_t arg = geglu_fma2(geglu_mul2(z, geglu_dup(-1.4426950408889634f)), z, p);
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e0) : "f"(__uint_as_float((uint32_t)arg)));
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e1) : "f"(__uint_as_float((uint32_t)(arg >> 32))));
    const uint64_t e = ((uint64_t)__float_as_uint(e1) << 32) | __float_as_uint(e0);
    // erfc(-g / sqrt 2): erfc(z) itself for a negative gate (no subtraction: it keeps its relative accuracy), 2 - erfc(z)
    // otherwise -- one select per element (slct picks its first operand where the third is >= 0)
    const uint64_t ez = geglu_mul2(e, t);
    const uint64_t two_minus = geglu_fma2(ez, geglu_dup(-1.0f), geglu_dup(2.0f));
    float w0, w1;
    asm("slct.f32.f32 %0, %1, %2, %3;" : "=f"(w0) : "f"(__uint_as_float((uint32_t)two_minus)), "f"(__uint_as_float((uint32_t)ez)), "f"(g.x));
    asm("slct.f32.f32 %0, %1, %2, %3;" : "=f"(w1) : "f"(__uint_as_float((uint32_t)(two_minus >> 32))), "f"(__uint_as_float((uint32_t)(ez >> 32))), "f"(g.y));
    const uint64_t two_phi = ((uint64_t)__float_as_uint(w1) << 32) | __float_as_uint(w0);
    const uint64_t half_a = geglu_mul2(((uint64_t)__float_as_uint(a.y) << 32) | __float_as_uint(a.x), geglu_dup(0.5f));
    const uint64_t o = geglu_mul2(half_a, geglu_mul2(gg, two_phi));
    return make_float2(__uint_as_float((uint32_t)o), __uint_as_float((uint32_t)(o >> 32)));
}

constexpr int GEGLU_THREADS = 256;
#ifndef SD_GEGLU_UNROLL
#define SD_GEGLU_UNROLL 1
#endif
#ifndef SD_GEGLU_BLOCKS_PER_SM
#define SD_GEGLU_BLOCKS_PER_SM 64
#endif
constexpr int GEGLU_UNROLL = SD_GEGLU_UNROLL;
constexpr int GEGLU_BLOCKS_PER_SM = SD_GEGLU_BLOCKS_PER_SM;

// VEC elements per 16-byte piece: 8 (fp16) or 4 (fp32); C is a multiple of VEC and both tensors are 16-byte aligned.
// A thread walks the tensor with the grid's stride, UNROLL pieces of each half per step, all of them requested before
// the first is used.  (Requesting the NEXT step's pieces before computing the current one -- software pipelining inside
// the thread -- measured slower: 18.5 against 16.5 us on the 8192 x 1280 tensor; enough blocks per SM overlap one
// another's loads and arithmetic already.  One piece per step and up to 64 blocks per SM measured best: 16.5 us there,
// 5.74 TB/s on a tensor sixteen times as large.)
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
                    for (int k = 0; k < 4; ++k)
                        oh[k] = __float22half2_rn(geglu_two(__half22float2(ah[k]), __half22float2(gh[k])));
                } else {
                    const float* af = reinterpret_cast<const float*>(&a[u]);
                    const float* gf = reinterpret_cast<const float*>(&g[u]);
                    float* of = reinterpret_cast<float*>(&o);
#pragma unroll
                    for (int k = 0; k < 4; k += 2) {
                        const float2 o2 = geglu_two(make_float2(af[k], af[k + 1]), make_float2(gf[k], gf[k + 1]));
                        of[k] = o2.x;
                        of[k + 1] = o2.y;
                    }
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
