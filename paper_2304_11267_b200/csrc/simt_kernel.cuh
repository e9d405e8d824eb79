// CUDA-core attention kernel: binary16 or binary32 storage, binary32 arithmetic throughout.
//
// It evaluates Eq. 3 with the single-pass running (max, sum) form of the softmax reductions of
// Eq. 4 (the FlashAttention recurrence of Sec. 3.2.2) using plain FMAs -- no tensor cores, hence
// no TF32 rounding -- and is the library's binary32 path and the on-device cross-check of the
// tensor-core kernels.
//
// Work split: a block owns 32 query rows (8 warps x 4 rows); keys stream through shared memory
// in chunks of 32.  In the score phase lane j owns key j of the chunk; in the P.V phase lane c
// owns output channels c, c+32, ... and the weights travel by warp shuffle.
#pragma once
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include "tc_common.cuh"

namespace sd_attn {

constexpr int SIMT_ROWS_PER_WARP = 4;
constexpr int SIMT_WARPS = 8;
constexpr int SIMT_BLOCK_ROWS = SIMT_ROWS_PER_WARP * SIMT_WARPS;  // 32 query rows per block
constexpr int SIMT_CHUNK = 32;                                    // keys per shared-memory chunk

__host__ __device__ inline int simt_k_stride(int d) { return ((d + 3) / 4) * 4 + 4; }

__host__ inline size_t simt_smem_bytes(int d) {
    const int cc = (d + 31) / 32;
    return sizeof(float) * (size_t)(SIMT_BLOCK_ROWS * simt_k_stride(d) + SIMT_CHUNK * simt_k_stride(d) +
                                    SIMT_CHUNK * 32 * cc);
}

__device__ inline float to_f32(float x) { return x; }
__device__ inline float to_f32(__half x) { return __half2float(x); }
__device__ inline float to_f32(__nv_bfloat16 x) { return __bfloat162float(x); }
__device__ inline void from_f32(float* p, float x) { *p = x; }
__device__ inline void from_f32(__half* p, float x) { *p = __float2half_rn(x); }
__device__ inline void from_f32(__nv_bfloat16* p, float x) { *p = __float2bfloat16_rn(x); }

template <typename T, int CC>  // CC = ceil(d / 32) output channels per lane
__global__ void __launch_bounds__(SIMT_WARPS * 32)
simt_attention_kernel(const T* __restrict__ q, const T* __restrict__ k, const T* __restrict__ v,
                      T* __restrict__ out, int Nq, int Nk, int d, float scale, HeadLayout lq, HeadLayout lk) {
    extern __shared__ __align__(16) float simt_smem[];
    const int ks = simt_k_stride(d);
    const int vs = 32 * CC;
    float* Qs = simt_smem;                        // [32][ks], zero padded
    float* Ks = Qs + SIMT_BLOCK_ROWS * ks;        // [32][ks]
    float* Vs = Ks + SIMT_CHUNK * ks;             // [32][vs]

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int bh = blockIdx.y;   // lq places the heads of q and out (Nq rows each), lk those of k and v (Nk rows)
    const int row0 = blockIdx.x * SIMT_BLOCK_ROWS;
    const T* qb = head_row(q, lq, bh, row0);
    const T* kb = head_row(k, lk, bh, 0);
    const T* vb = head_row(v, lk, bh, 0);
    const long long ldq = lq.ld, ldk = lk.ld;

    for (int idx = tid; idx < SIMT_BLOCK_ROWS * ks; idx += blockDim.x) {
        const int r = idx / ks, c = idx - r * ks;
        Qs[idx] = (c < d && row0 + r < Nq) ? to_f32(qb[r * ldq + c]) : 0.f;
    }

    float m[SIMT_ROWS_PER_WARP], l[SIMT_ROWS_PER_WARP], o[SIMT_ROWS_PER_WARP][CC];
#pragma unroll
    for (int r = 0; r < SIMT_ROWS_PER_WARP; ++r) {
        m[r] = -INFINITY;
        l[r] = 0.f;
#pragma unroll
        for (int cc = 0; cc < CC; ++cc) o[r][cc] = 0.f;
    }

    for (int j0 = 0; j0 < Nk; j0 += SIMT_CHUNK) {
        __syncthreads();  // previous chunk fully consumed (and Qs written, first time round)
        for (int idx = tid; idx < SIMT_CHUNK * ks; idx += blockDim.x) {
            const int r = idx / ks, c = idx - r * ks;
            Ks[idx] = (c < d && j0 + r < Nk) ? to_f32(kb[(j0 + r) * ldk + c]) : 0.f;
        }
        for (int idx = tid; idx < SIMT_CHUNK * vs; idx += blockDim.x) {
            const int r = idx / vs, c = idx - r * vs;
            Vs[idx] = (c < d && j0 + r < Nk) ? to_f32(vb[(j0 + r) * ldk + c]) : 0.f;
        }
        __syncthreads();

        // scores of this lane's key against the warp's four query rows, four partial sums each
        float4 acc[SIMT_ROWS_PER_WARP];
#pragma unroll
        for (int r = 0; r < SIMT_ROWS_PER_WARP; ++r) acc[r] = make_float4(0.f, 0.f, 0.f, 0.f);
        const float* krow = Ks + lane * ks;
        const float* qrow = Qs + warp * SIMT_ROWS_PER_WARP * ks;
        for (int c = 0; c < ks - 4; c += 4) {
            const float4 kk = *reinterpret_cast<const float4*>(krow + c);
#pragma unroll
            for (int r = 0; r < SIMT_ROWS_PER_WARP; ++r) {
                const float4 qq = *reinterpret_cast<const float4*>(qrow + r * ks + c);
                acc[r].x = fmaf(qq.x, kk.x, acc[r].x);
                acc[r].y = fmaf(qq.y, kk.y, acc[r].y);
                acc[r].z = fmaf(qq.z, kk.z, acc[r].z);
                acc[r].w = fmaf(qq.w, kk.w, acc[r].w);
            }
        }
        const bool valid = (j0 + lane) < Nk;
        float p[SIMT_ROWS_PER_WARP];
#pragma unroll
        for (int r = 0; r < SIMT_ROWS_PER_WARP; ++r) {
            const float a = valid ? scale * ((acc[r].x + acc[r].y) + (acc[r].z + acc[r].w)) : -INFINITY;
            float mx = a;
#pragma unroll
            for (int s = 16; s > 0; s >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, s));
            const float m_new = fmaxf(m[r], mx);     // finite: every chunk holds a valid key
            const float alpha = expf(m[r] - m_new);  // exp(-inf) = 0 on the first chunk
            p[r] = expf(a - m_new);                  // masked keys: exp(-inf) = 0
            l[r] = l[r] * alpha + p[r];              // per-lane partial of S; summed at the end
#pragma unroll
            for (int cc = 0; cc < CC; ++cc) o[r][cc] *= alpha;
            m[r] = m_new;
        }
        // o_c += sum_j p_j v_jc, lane = channel
#pragma unroll 4
        for (int j = 0; j < SIMT_CHUNK; ++j) {
            float pj[SIMT_ROWS_PER_WARP];
#pragma unroll
            for (int r = 0; r < SIMT_ROWS_PER_WARP; ++r) pj[r] = __shfl_sync(0xffffffffu, p[r], j);
#pragma unroll
            for (int cc = 0; cc < CC; ++cc) {
                const float vv = Vs[j * vs + cc * 32 + lane];
#pragma unroll
                for (int r = 0; r < SIMT_ROWS_PER_WARP; ++r) o[r][cc] = fmaf(pj[r], vv, o[r][cc]);
            }
        }
    }

#pragma unroll
    for (int r = 0; r < SIMT_ROWS_PER_WARP; ++r) {
        float s = l[r];
#pragma unroll
        for (int sft = 16; sft > 0; sft >>= 1) s += __shfl_xor_sync(0xffffffffu, s, sft);
        const int row = row0 + warp * SIMT_ROWS_PER_WARP + r;
        if (row < Nq) {
            T* orow = head_row(out, lq, bh, row);
#pragma unroll
            for (int cc = 0; cc < CC; ++cc) {
                const int c = cc * 32 + lane;
                if (c < d) from_f32(orow + c, o[r][cc] / s);
            }
        }
    }
}

}  // namespace sd_attn
