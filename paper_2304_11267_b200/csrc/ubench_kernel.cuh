// Instruction-rate probes behind the joint roofline of the single-pass kernel (one exponential, a few FMA-pipe
// operations and 4 d tensor-core FLOPs per score element: which unit bounds a head dim depends on their rates).
// One block of 512 threads per SM runs a fixed number of independent chains of ONE kind of operation on registers
// and reports the clocks and the nanoseconds it took: results per clock per SM, and the SM clock that was in effect.
// Bounded (a fixed trip count, a few hundred microseconds), no memory traffic inside the timed part.
#pragma once
#include "softmax_math.cuh"

namespace sd_attn {

enum { UBENCH_EX2 = 0, UBENCH_FMA = 1, UBENCH_FMA_X2 = 2, UBENCH_SWEEP = 3, UBENCH_SWEEP_POLY = 4, UBENCH_OPS = 5 };
constexpr int UBENCH_THREADS = 512, UBENCH_CHAINS = 8;

template <int OP>
__global__ void __launch_bounds__(UBENCH_THREADS) ubench_kernel(int iters, float seed, long long* out, float* sink) {
    long long t0, t1;
    unsigned long long g0, g1;
    float keep = 0.f;
    if (OP == UBENCH_SWEEP || OP == UBENCH_SWEEP_POLY) {
        // the exp2 / row-sum / pack sweep of the kernels on 32 scores held in registers, as the softmax warps run it
        uint32_t s[32], packed[16];
#pragma unroll
        for (int i = 0; i < 32; ++i) s[i] = __float_as_uint(seed * (float)(i - 16) + 1e-3f * (float)threadIdx.x);
        const float c2 = 0.25f, nm = -3.f;
        const uint64_t c2c2 = pack_b64(__float_as_uint(c2), __float_as_uint(c2));
        const uint64_t nmnm = pack_b64(__float_as_uint(nm), __float_as_uint(nm));
        uint64_t acc[2] = {0ull, 0ull};
        asm volatile("mov.u64 %0, %globaltimer;" : "=l"(g0));
        t0 = clock64();
        for (int it = 0; it < iters; ++it) {
            exp2_pack_32<OP == UBENCH_SWEEP_POLY ? 2 : 0>(s, c2c2, nmnm, packed, acc);
#pragma unroll
            for (int i = 0; i < 16; ++i) s[2 * i] ^= packed[i] & 1u;   // the next round depends on this one's weights
        }
        t1 = clock64();
        asm volatile("mov.u64 %0, %globaltimer;" : "=l"(g1));
        keep = sum_f32x2(acc[0], acc[1]);
    } else {
        float a[UBENCH_CHAINS];
#pragma unroll
        for (int i = 0; i < UBENCH_CHAINS; ++i) a[i] = seed + 1e-3f * (float)threadIdx.x + (float)i;
        asm volatile("mov.u64 %0, %globaltimer;" : "=l"(g0));
        t0 = clock64();
        for (int it = 0; it < iters; ++it) {
#pragma unroll
            for (int i = 0; i < UBENCH_CHAINS; ++i) {
                if (OP == UBENCH_EX2) asm volatile("ex2.approx.ftz.f32 %0, %0;" : "+f"(a[i]));
                if (OP == UBENCH_FMA) asm volatile("fma.rn.f32 %0, %0, %1, %0;" : "+f"(a[i]) : "f"(seed));
                if (OP == UBENCH_FMA_X2 && (i & 1) == 0) {
                    uint64_t v = pack_b64(__float_as_uint(a[i]), __float_as_uint(a[i + 1]));
                    asm volatile("fma.rn.f32x2 %0, %0, %1, %0;" : "+l"(v) : "l"(0x3f0000003f000000ull));
                    uint32_t lo, hi;
                    unpack_b64(v, lo, hi);
                    a[i] = __uint_as_float(lo);
                    a[i + 1] = __uint_as_float(hi);
                }
            }
        }
        t1 = clock64();
        asm volatile("mov.u64 %0, %globaltimer;" : "=l"(g1));
#pragma unroll
        for (int i = 0; i < UBENCH_CHAINS; ++i) keep += a[i];
    }
    if (keep == 12345.678f) sink[0] = keep;   // keeps the chains alive without a store on the normal path
    if (threadIdx.x == 0) {
        out[2 * blockIdx.x] = t1 - t0;
        out[2 * blockIdx.x + 1] = (long long)(g1 - g0);
    }
}

// results one thread produces per trip of its loop
__host__ inline int ubench_results_per_trip(int op) { return (op == UBENCH_SWEEP || op == UBENCH_SWEEP_POLY) ? 32 : UBENCH_CHAINS; }

}  // namespace sd_attn
