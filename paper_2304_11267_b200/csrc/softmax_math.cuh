// Register-level pieces of the online softmax shared by the fused kernels: the row maximum and the
// exp2 / row-sum / fp16-pack sweep over one row of a score tile held in registers (raw fp32 bits).
//
// Both schedulers of an SM sub-partition issue one instruction per clock for ALL pipes, and the
// special-function unit retires one warp-wide exp2 per 8 clocks, so the sweep is written to spend
// as few issue slots per score element as it can:
//   maximum   the two high halves (bf16 truncations) of a pair of scores are merged by one byte
//             permute and folded with one packed bf16 max: 1 slot per pair.  The truncated maximum
//             is only a reference point (any value within a few units of the true one works, the
//             same value is used for the numerator, the row sum and the lazy rescale), so its 2^-8
//             relative slack is harmless.
//   exponent  s*c - m*c for a pair with one packed fp32x2 FMA, two exp2, one packed fp32x2 add
//             into the running sum, one conversion to packed fp16: 2.5 slots per element.
#pragma once
#include "tc_common.cuh"

namespace sd_attn {

__device__ __forceinline__ uint64_t pack_b64(uint32_t lo, uint32_t hi) {
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "r"(lo), "r"(hi));
    return r;
}
__device__ __forceinline__ void unpack_b64(uint64_t v, uint32_t& lo, uint32_t& hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=r"(lo), "=r"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t fma_f32x2(uint64_t a, uint64_t b, uint64_t c) {
    uint64_t d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ uint64_t add_f32x2(uint64_t a, uint64_t b) {
    uint64_t d;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ uint32_t high_halves(uint32_t a, uint32_t b) {   // {a[31:16], b[31:16]} as bf16x2
    uint32_t r;
    asm("prmt.b32 %0, %1, %2, 0x7632;" : "=r"(r) : "r"(a), "r"(b));
    return r;
}
__device__ __forceinline__ uint32_t max_bf16x2(uint32_t a, uint32_t b) {
    uint32_t r;
    asm("max.bf16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
    return r;
}

// Maximum of a full row of N scores (N a multiple of 8), to bf16 precision.
template <int N>
__device__ __forceinline__ float row_max_bf16(const uint32_t* s) {
    uint32_t m[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) m[k] = high_halves(s[2 * k], s[2 * k + 1]);
#pragma unroll
    for (int k = 4; k < N / 2; ++k) m[k & 3] = max_bf16x2(m[k & 3], high_halves(s[2 * k], s[2 * k + 1]));
    const uint32_t mm = max_bf16x2(max_bf16x2(m[0], m[1]), max_bf16x2(m[2], m[3]));
    return fmaxf(__uint_as_float(mm << 16), __uint_as_float(mm & 0xffff0000u));
}

// Maximum over the first `valid` of N scores (the key tile is ragged: the rest are zero-filled keys).
template <int N>
__device__ __forceinline__ float row_max_masked(const uint32_t* s, int valid) {
    float m[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
    for (int c = 0; c < N; ++c)
        if (c < valid) m[c & 3] = fmaxf(m[c & 3], __uint_as_float(s[c]));
    return fmaxf(fmaxf(m[0], m[1]), fmaxf(m[2], m[3]));
}

__device__ __forceinline__ uint64_t add_rm_f32x2(uint64_t a, uint64_t b) {   // round toward -inf
    uint64_t d;
    asm("add.rm.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ uint64_t sub_f32x2(uint64_t a, uint64_t b) {
    uint64_t d;
    asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__host__ __device__ constexpr uint64_t dup_f32(uint32_t bits) { return ((uint64_t)bits << 32) | bits; }

__device__ __forceinline__ uint64_t fma_rm_f32x2(uint64_t a, uint64_t b, uint64_t c) {   // round toward -inf
    uint64_t d;
    asm("fma.rm.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ float fma_sat(float a, float b, float c) {   // a * b + c clamped to [0, 1]
    float d;
    asm("fma.rn.sat.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}

// 2^(s*c2 + nm) for a PAIR of scores on the FMA pipe (see ex2_poly in tc_common.cuh for the method): the
// special-function unit is the bound of the d = 40 kernel, so a share of the pairs goes this way.
// The argument x = s*c2 + nm is clamped to [-126, 128] at both ends -- below, the exponent field would wrap; above,
// the result must come out huge or non-finite (a score far above a stale anchor: the caller's sum test then
// re-anchors the row), not wrap into garbage.  Both clamps and the scaling of the score are ONE saturating
// multiply-add per value: y = sat(s * (c2/254) + (nm + 126)/254) in [0, 1], and the rest works on
// x' = 254 y - 126 without ever forming it.  (x' differs from x by 1e-5 + 1e-7 |nm| at most: below the
// polynomial's error for every anchor a finite softmax of binary16 data can have.)
__device__ __forceinline__ void ex2_poly_pair(uint32_t s0, uint32_t s1, float c2_254, float nm_254, float& p0,
                                              float& p1) {
    constexpr uint64_t MAGIC_LO = dup_f32(0x4B3FFF82u);   // 1.5 * 2^23 - 126
    constexpr uint64_t WIDTH = dup_f32(0x437E0000u);      // 254
    constexpr uint64_t C3 = dup_f32(0x3D9FCB52u), C2 = dup_f32(0x3E677E26u);   // 0.07802452, 0.22606716
    constexpr uint64_t C1 = dup_f32(0x3F322226u), C0 = dup_f32(0x3F7FFB19u);   // 0.69583356, 0.9999252
    const uint64_t y = pack_b64(__float_as_uint(fma_sat(__uint_as_float(s0), c2_254, nm_254)),
                                __float_as_uint(fma_sat(__uint_as_float(s1), c2_254, nm_254)));
    const uint64_t t = fma_rm_f32x2(y, WIDTH, MAGIC_LO);              // low mantissa bits = floor(x')
    const uint64_t f = fma_f32x2(y, WIDTH, sub_f32x2(MAGIC_LO, t));   // x' - floor(x'), in [0, 1]
    uint64_t p = fma_f32x2(f, C3, C2);
    p = fma_f32x2(p, f, C1);
    p = fma_f32x2(p, f, C0);
    uint32_t t0, t1, q0, q1;
    unpack_b64(t, t0, t1);
    unpack_b64(p, q0, q1);
    p0 = __uint_as_float(q0 + (t0 << 23));
    p1 = __uint_as_float(q1 + (t1 << 23));
}

// Which of the 16 pairs of a 32-score chunk take the polynomial: POLY of every 8.
template <int POLY>
__device__ __forceinline__ constexpr bool pair_uses_poly(int k) {
    return POLY == 0 ? false
         : POLY == 1 ? (k & 7) == 0
         : POLY == 2 ? (k & 3) == 0
         : POLY == 3 ? ((k & 7) == 0 || (k & 7) == 3 || (k & 7) == 6)
                     : (k & 1) == 0;
}

// p = exp2(s*c2 + neg_mc) for 32 scores -> 16 packed pairs of 16-bit weights (binary16, or bfloat16 when BF);
// adds the 32 weights into acc[0..1].
template <int POLY, int PAIRS = 16, bool BF = false>
__device__ __forceinline__ void exp2_pack_32(const uint32_t* s, uint64_t c2c2, uint64_t nmnm, uint32_t* packed,
                                             uint64_t* acc) {
    // the polynomial's pairs take the score itself, with the constants of the clamped form (see ex2_poly_pair)
    const float c2_254 = __uint_as_float((uint32_t)c2c2) * (1.f / 254.f);
    const float nm_254 = fmaf(__uint_as_float((uint32_t)nmnm), 1.f / 254.f, 126.f / 254.f);
#pragma unroll
    for (int k = 0; k < PAIRS; ++k) {
        float p0, p1;
        if (pair_uses_poly<POLY>(k)) {
            ex2_poly_pair(s[2 * k], s[2 * k + 1], c2_254, nm_254, p0, p1);
        } else {
            const uint64_t x = fma_f32x2(pack_b64(s[2 * k], s[2 * k + 1]), c2c2, nmnm);
            uint32_t x0, x1;
            unpack_b64(x, x0, x1);
            p0 = ex2_approx(__uint_as_float(x0));
            p1 = ex2_approx(__uint_as_float(x1));
        }
        acc[k & 1] = add_f32x2(acc[k & 1], pack_b64(__float_as_uint(p0), __float_as_uint(p1)));
        packed[k] = pack_16x2<BF>(p0, p1);
    }
}

// 16 scores -> 8 packed pairs.
template <int POLY, bool BF = false>
__device__ __forceinline__ void exp2_pack_16(const uint32_t* s, uint64_t c2c2, uint64_t nmnm, uint32_t* packed,
                                             uint64_t* acc) {
    exp2_pack_32<POLY, 8, BF>(s, c2c2, nmnm, packed, acc);
}

// The same for a ragged tile: scores at column >= valid get weight zero (also when the scale is zero).
template <int PAIRS = 16, bool BF = false>
__device__ __forceinline__ void exp2_pack_32_masked(const uint32_t* s, float c2, float neg_mc, int first_col, int valid,
                                                    uint32_t* packed, float& sum) {
#pragma unroll
    for (int k = 0; k < PAIRS; ++k) {
        float p0 = ex2_approx(fmaf(__uint_as_float(s[2 * k]), c2, neg_mc));
        float p1 = ex2_approx(fmaf(__uint_as_float(s[2 * k + 1]), c2, neg_mc));
        if (first_col + 2 * k >= valid) p0 = 0.f;
        if (first_col + 2 * k + 1 >= valid) p1 = 0.f;
        sum += p0 + p1;
        packed[k] = pack_16x2<BF>(p0, p1);
    }
}

__device__ __forceinline__ float sum_f32x2(uint64_t a, uint64_t b) {
    uint32_t a0, a1, b0, b1;
    unpack_b64(a, a0, a1);
    unpack_b64(b, b0, b1);
    return (__uint_as_float(a0) + __uint_as_float(a1)) + (__uint_as_float(b0) + __uint_as_float(b1));
}

}  // namespace sd_attn
