// Winograd convolution F(4x4, 3x3) (Sec. 3.3; the tile size Table 2 selects) for stride-1, pad-1 3x3 convolutions
// of channels-last fp16 tensors, as four kernels:
//
//   filter transform   U[xi][k][c] = 128 * (G g G^T)[xi]          once per layer ("Weight" x4 of Table 2)
//   input transform    V[xi][t][c] = (B^T d B)[xi]                 per call; t = 4x4 output tile, d its 6x6 input patch
//   36 GEMMs           M[xi][t][k] = sum_c V[xi][t][c] U[xi][k][c] tcgen05, fp32 accumulators in tensor memory
//   output transform   y tile      = A^T M A / 128 + bias          per call
//
// with xi = 0..35 the position in the 6x6 transformed tile.  The transforms are the standard ones for the
// interpolation points 0, +-1, +-2, infinity; they are evaluated in fp32 and rounded once to fp16 where the tensor
// core wants fp16 (U and V).  U carries a factor 128 (exact, removed in the output transform) because the entries
// of G reach 1/24 * 1/24: weights of size 1e-3 would otherwise land in fp16's subnormals.
//
// On this machine the point of the transformed domain is the 2.25x fewer tensor-core FLOPs of the GEMM stage against
// the 2.25x more bytes of V -- which, like M, is written and read back through the 126 MB L2 (V: 12 MB, M: 24 MB at
// the UNet's largest 3x3 layer), not through HBM.
#pragma once
#include <cuda.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "tc_common.cuh"

namespace sd_attn {

constexpr int WG_TILE = 4;                 // output tile edge m
constexpr int WG_PATCH = 6;                // input patch edge m + 2
constexpr int WG_XI = 36;                  // positions of the transformed tile
constexpr float WG_FILTER_SCALE = 128.f;   // carried by U, removed by the output transform

// ------------------------------------------------------------------------------------------------ transforms
// B^T d (one column of d, six values) for the points 0, +-1, +-2, inf.
__device__ __forceinline__ void wg_bt(const float (&d)[6], float (&o)[6]) {
    o[0] = 4.f * d[0] - 5.f * d[2] + d[4];
    o[1] = -4.f * (d[1] + d[2]) + d[3] + d[4];
    o[2] = 4.f * (d[1] - d[2]) - d[3] + d[4];
    o[3] = -2.f * d[1] - d[2] + 2.f * d[3] + d[4];
    o[4] = 2.f * d[1] - d[2] - 2.f * d[3] + d[4];
    o[5] = 4.f * d[1] - 5.f * d[3] + d[5];
}
// G g (three values -> six)
__device__ __forceinline__ void wg_g(const float (&g)[3], float (&o)[6]) {
    o[0] = 0.25f * g[0];
    o[1] = -(g[0] + g[1] + g[2]) * (1.f / 6.f);
    o[2] = -(g[0] - g[1] + g[2]) * (1.f / 6.f);
    o[3] = g[0] * (1.f / 24.f) + g[1] * (1.f / 12.f) + g[2] * (1.f / 6.f);
    o[4] = g[0] * (1.f / 24.f) - g[1] * (1.f / 12.f) + g[2] * (1.f / 6.f);
    o[5] = g[2];
}
// A^T m (six values -> four)
__device__ __forceinline__ void wg_at(const float (&m)[6], float (&o)[4]) {
    o[0] = m[0] + m[1] + m[2] + m[3] + m[4];
    o[1] = m[1] - m[2] + 2.f * (m[3] - m[4]);
    o[2] = m[1] + m[2] + 4.f * (m[3] + m[4]);
    o[3] = m[1] - m[2] + 8.f * (m[3] - m[4]) + m[5];
}

// w [K][3][3][C] fp16 -> U [36][K][C] fp16; one thread per (k, c).
__global__ void __launch_bounds__(256) winograd_filter_kernel(const __half* __restrict__ w, __half* __restrict__ U,
                                                              int K, int C) {
    const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= (long long)K * C) return;
    const int k = (int)(idx / C), c = (int)(idx - (long long)k * C);
    float g[3][3], t[6][3];
#pragma unroll
    for (int r = 0; r < 3; ++r)
#pragma unroll
        for (int s = 0; s < 3; ++s) g[r][s] = __half2float(w[(((long long)k * 3 + r) * 3 + s) * C + c]);
#pragma unroll
    for (int s = 0; s < 3; ++s) {   // G g: down the columns
        const float col[3] = {g[0][s], g[1][s], g[2][s]};
        float o[6];
        wg_g(col, o);
#pragma unroll
        for (int a = 0; a < 6; ++a) t[a][s] = o[a];
    }
#pragma unroll
    for (int a = 0; a < 6; ++a) {   // (G g) G^T: along the rows
        float o[6];
        wg_g(t[a], o);
#pragma unroll
        for (int b = 0; b < 6; ++b)
            U[((long long)(a * 6 + b) * K + k) * C + c] = __float2half_rn(o[b] * WG_FILTER_SCALE);
    }
}

struct WinogradArgs {
    int N, H, W, C, K;
    int tiles_y, tiles_x;   // ceil(H / 4), ceil(W / 4)
    int T;                  // N * tiles_y * tiles_x
    int n_chunk;            // output channels per GEMM CTA (multiple of 16, <= WG_MAX_N_CHUNK)
    int tmem_cols;          // power of two >= n_chunk
    int stages;             // ring depth of the GEMM's operand tiles
    int* status;
};

// x [N][H][W][C] fp16 -> V [36][T][C] fp16; one thread per (tile, four channels): 8-byte loads and stores.
__global__ void __launch_bounds__(128) winograd_input_kernel(const __half* __restrict__ x, __half* __restrict__ V,
                                                             const WinogradArgs a) {
    pdl_launch_dependents();   // the next kernel of the stream may start its set-up
    pdl_wait();                // x may come from the previous kernel of the stream; V may still be read by it
    const int cq = a.C >> 2;
    const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= (long long)a.T * cq) return;
    const int t = (int)(idx / cq), c = (int)(idx - (long long)t * cq) * 4;
    const int n = t / (a.tiles_y * a.tiles_x), ty = (t / a.tiles_x) % a.tiles_y, tx = t % a.tiles_x;
    const int i0 = ty * WG_TILE - 1, j0 = tx * WG_TILE - 1;
    float d[6][6][4];
#pragma unroll
    for (int r = 0; r < 6; ++r)
#pragma unroll
        for (int s = 0; s < 6; ++s) {
            const int i = i0 + r, j = j0 + s;
            uint2 raw = make_uint2(0u, 0u);
            if (i >= 0 && i < a.H && j >= 0 && j < a.W)
                raw = __ldg(reinterpret_cast<const uint2*>(x + (((long long)n * a.H + i) * a.W + j) * a.C + c));
            const float2 lo = __half22float2(*reinterpret_cast<const __half2*>(&raw.x));
            const float2 hi = __half22float2(*reinterpret_cast<const __half2*>(&raw.y));
            d[r][s][0] = lo.x; d[r][s][1] = lo.y; d[r][s][2] = hi.x; d[r][s][3] = hi.y;
        }
#pragma unroll
    for (int e = 0; e < 4; ++e) {
#pragma unroll
        for (int s = 0; s < 6; ++s) {   // B^T d: down the columns
            const float col[6] = {d[0][s][e], d[1][s][e], d[2][s][e], d[3][s][e], d[4][s][e], d[5][s][e]};
            float o[6];
            wg_bt(col, o);
#pragma unroll
            for (int r = 0; r < 6; ++r) d[r][s][e] = o[r];
        }
#pragma unroll
        for (int r = 0; r < 6; ++r) {   // (B^T d) B: along the rows
            const float row[6] = {d[r][0][e], d[r][1][e], d[r][2][e], d[r][3][e], d[r][4][e], d[r][5][e]};
            float o[6];
            wg_bt(row, o);
#pragma unroll
            for (int s = 0; s < 6; ++s) d[r][s][e] = o[s];
        }
    }
#pragma unroll
    for (int r = 0; r < 6; ++r)
#pragma unroll
        for (int s = 0; s < 6; ++s) {
            const __half2 lo = __floats2half2_rn(d[r][s][0], d[r][s][1]), hi = __floats2half2_rn(d[r][s][2], d[r][s][3]);
            uint2 raw;
            raw.x = *reinterpret_cast<const uint32_t*>(&lo);
            raw.y = *reinterpret_cast<const uint32_t*>(&hi);
            *reinterpret_cast<uint2*>(V + ((long long)(r * 6 + s) * a.T + t) * a.C + c) = raw;
        }
}

// M [36][T][K] fp32 -> y [N][H][W][K] fp16 (+ bias); one thread per (tile, output channel pair).
__global__ void __launch_bounds__(128) winograd_output_kernel(const float* __restrict__ M, const __half* __restrict__ bias,
                                                              __half* __restrict__ y, const WinogradArgs a) {
    pdl_launch_dependents();
    pdl_wait();                // M is complete once the GEMM kernel has finished
    const int kp = a.K >> 1;
    const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= (long long)a.T * kp) return;
    const int t = (int)(idx / kp), k = (int)(idx - (long long)t * kp) * 2;
    const int n = t / (a.tiles_y * a.tiles_x), ty = (t / a.tiles_x) % a.tiles_y, tx = t % a.tiles_x;
    float2 m[6][6];
#pragma unroll
    for (int r = 0; r < 6; ++r)
#pragma unroll
        for (int s = 0; s < 6; ++s)
            m[r][s] = *reinterpret_cast<const float2*>(M + ((long long)(r * 6 + s) * a.T + t) * a.K + k);
    float2 h[4][6];
#pragma unroll
    for (int s = 0; s < 6; ++s) {   // A^T m: down the columns
        const float cx[6] = {m[0][s].x, m[1][s].x, m[2][s].x, m[3][s].x, m[4][s].x, m[5][s].x};
        const float cy[6] = {m[0][s].y, m[1][s].y, m[2][s].y, m[3][s].y, m[4][s].y, m[5][s].y};
        float ox[4], oy[4];
        wg_at(cx, ox);
        wg_at(cy, oy);
#pragma unroll
        for (int r = 0; r < 4; ++r) h[r][s] = make_float2(ox[r], oy[r]);
    }
    float2 b = make_float2(0.f, 0.f);
    if (bias) b = __half22float2(*reinterpret_cast<const __half2*>(bias + k));
#pragma unroll
    for (int r = 0; r < 4; ++r) {   // (A^T m) A: along the rows
        const float rx[6] = {h[r][0].x, h[r][1].x, h[r][2].x, h[r][3].x, h[r][4].x, h[r][5].x};
        const float ry[6] = {h[r][0].y, h[r][1].y, h[r][2].y, h[r][3].y, h[r][4].y, h[r][5].y};
        float ox[4], oy[4];
        wg_at(rx, ox);
        wg_at(ry, oy);
        const int i = ty * WG_TILE + r;
#pragma unroll
        for (int s = 0; s < 4; ++s) {
            const int j = tx * WG_TILE + s;
            if (i < a.H && j < a.W)
                *reinterpret_cast<__half2*>(y + (((long long)n * a.H + i) * a.W + j) * a.K + k) =
                    __floats2half2_rn(fmaf(ox[s], 1.f / WG_FILTER_SCALE, b.x), fmaf(oy[s], 1.f / WG_FILTER_SCALE, b.y));
        }
    }
}

// ------------------------------------------------------------------------------------------------ the 36 GEMMs
// One CTA: a 128-row tile of T, n_chunk output channels, one xi.  Warp 0 feeds a ring of (V tile, U tile) stages
// by TMA, 64 input channels at a time; warp 1 issues the MMAs (fp32 accumulator of n_chunk columns in tensor
// memory) and frees a stage with the commit that follows its four steps; warps 2..5 read the accumulator (thread =
// row) and store M.  Every wait is bounded and reports to the status block.
constexpr int WG_THREADS = 192;
constexpr int WG_MAX_STAGES = 4;
enum { SITE_W_EMPTY = 50, SITE_W_FULL = 51, SITE_W_DONE = 52 };

__host__ __device__ inline int wg_stage_bytes(int n_chunk) { return (TILE_M + n_chunk) * CHUNK_ROW_BYTES; }
constexpr int WG_MAX_N_CHUNK = 176;   // ring of three stages and the epilogue's staging tile both fit twice per SM
__host__ inline size_t winograd_gemm_smem_bytes(int n_chunk, int stages) {
    const size_t ring = (size_t)stages * (size_t)((wg_stage_bytes(n_chunk) + 1023) & ~1023);
    const size_t staging = (size_t)TILE_M * (n_chunk + 4) * sizeof(float);   // the epilogue reuses the ring
    return (ring > staging ? ring : staging) + 1024;
}

__global__ void __launch_bounds__(WG_THREADS, 1)
winograd_gemm_kernel(const __grid_constant__ CUtensorMap tmap_v, const __grid_constant__ CUtensorMap tmap_u,
                     float* __restrict__ M, const WinogradArgs args) {
    extern __shared__ uint8_t wg_smem_raw[];
    __shared__ __align__(8) uint64_t bar_full[WG_MAX_STAGES], bar_empty[WG_MAX_STAGES], bar_done;
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;

    const int tid = threadIdx.x, warp = tid >> 5;
    if (tid == 0) pdl_launch_dependents();
    const int t0 = blockIdx.x * TILE_M, k0 = blockIdx.y * args.n_chunk, xi = blockIdx.z;
    const int n_chunk = args.n_chunk, stages = args.stages;
    const int c_steps = (args.C + CHUNK_COLS - 1) / CHUNK_COLS;
    const uint32_t smem_base = (smem_u32(wg_smem_raw) + 1023u) & ~1023u;
    const uint32_t stage_pitch = (uint32_t)((wg_stage_bytes(n_chunk) + 1023) & ~1023);

    if (tid == 0) {
        abort_flag = 0;
        for (int s = 0; s < stages; ++s) {
            mbar_init(smem_u32(&bar_full[s]), 1);
            mbar_init(smem_u32(&bar_empty[s]), 1);
        }
        mbar_init(smem_u32(&bar_done), 1);
        mbar_init_fence();
        tma_prefetch_desc(&tmap_v);
        tma_prefetch_desc(&tmap_u);
    }
    if (warp == 0) {
        tmem_alloc(smem_u32(&tmem_base_slot), (uint32_t)args.tmem_cols);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    // Set-up (barriers, tensor memory) overlapped the tail of the input transform; V is complete, and M free to be
    // overwritten, once that kernel -- which itself waited for the previous call's output transform -- has finished.
    pdl_wait();
    const uint32_t tmem_d = tmem_base_slot;
    volatile int* abort_p = &abort_flag;

    if (warp == 0) {
        if (elect_one()) {
            // ---------------------------------------------------------------- TMA producer
            int s = 0, pe = 1;   // parity of the bar_empty phase that frees stage s (from step `stages` on)
            for (int j = 0; j < c_steps; ++j, ++s) {
                if (s == stages) { s = 0; pe ^= 1; }
                if (j >= stages && !mbar_wait(smem_u32(&bar_empty[s]), pe, abort_p, args.status, SITE_W_EMPTY, j)) break;
                const uint32_t a_dst = smem_base + s * stage_pitch, b_dst = a_dst + TILE_M * CHUNK_ROW_BYTES;
                const uint32_t bar = smem_u32(&bar_full[s]);
                mbar_arrive_expect_tx(bar, (uint32_t)wg_stage_bytes(n_chunk));
                tma_load_3d(a_dst, &tmap_v, bar, j * CHUNK_COLS, t0, xi);
                tma_load_3d(b_dst, &tmap_u, bar, j * CHUNK_COLS, k0, xi);
            }
        }
    } else if (warp == 1) {
        if (elect_one()) {
            // ---------------------------------------------------------------- MMA issuer
            const uint32_t idesc = idesc_f16(TILE_M, n_chunk, false, false, false);
            int s = 0, pf = 0;
            bool ok = true;
            for (int j = 0; j < c_steps && ok; ++j, ++s) {
                if (s == stages) { s = 0; pf ^= 1; }
                ok = mbar_wait(smem_u32(&bar_full[s]), pf, abort_p, args.status, SITE_W_FULL, j);
                if (!ok) break;
                tc_fence_after_sync();
                const uint32_t a_src = smem_base + s * stage_pitch, b_src = a_src + TILE_M * CHUNK_ROW_BYTES;
#pragma unroll
                for (int kk = 0; kk < 4; ++kk) {
                    const uint64_t a_desc = smem_desc_sw128(a_src + kk * 32, 16, 1024);
                    const uint64_t b_desc = smem_desc_sw128(b_src + kk * 32, 16, 1024);
                    mma_f16_ss(tmem_d, a_desc, b_desc, idesc, j > 0 || kk > 0);
                }
                tc_commit(smem_u32(&bar_empty[s]));   // the stage may be refilled once these MMAs have read it
            }
            if (ok) tc_commit(smem_u32(&bar_done));
        }
    } else {
        // -------------------------------------------------------------------- epilogue
        // Thread = row of the tile when it reads the accumulator; a row of M is n_chunk consecutive floats, so the
        // tile goes through shared memory (the operand ring is idle by now: every MMA has completed) and leaves as
        // whole rows, a warp writing 512 contiguous bytes at a time.  Each warp stages and writes its own 32 rows.
        bool ok = mbar_wait(smem_u32(&bar_done), 0, abort_p, args.status, SITE_W_DONE, blockIdx.x);
        ok = __all_sync(0xffffffffu, ok);
        if (ok) {
            tc_fence_after_sync();
            const int q = warp & 3, lane = tid & 31;       // a warp reads the 32 lanes of its quarter (warp id mod 4)
            const uint32_t lane_off = (uint32_t)(q * 32) << 16;
            const int pitch = n_chunk + 4;                 // floats; + 4 keeps the 16-byte row writes off each other's banks
            float* stage = reinterpret_cast<float*>(wg_smem_raw + (smem_base - smem_u32(wg_smem_raw))) + q * 32 * pitch;
            for (int g = 0; g < (n_chunk >> 4); ++g) {
                uint32_t r[16];
                tmem_ld16(tmem_d + lane_off + g * 16, r);
                tmem_wait_ld();
#pragma unroll
                for (int c = 0; c < 16; c += 4)
                    *reinterpret_cast<uint4*>(stage + lane * pitch + g * 16 + c) = make_uint4(r[c], r[c + 1], r[c + 2], r[c + 3]);
            }
            __syncwarp();
            const int cols = min(n_chunk, args.K - k0);    // a multiple of 8: K and k0 are
            for (int rr = 0; rr < 32; ++rr) {
                const int row = t0 + q * 32 + rr;
                if (row >= args.T) break;
                float* mrow = M + ((long long)xi * args.T + row) * args.K + k0;
                for (int c = lane * 4; c < cols; c += 128)
                    *reinterpret_cast<uint4*>(mrow + c) = *reinterpret_cast<const uint4*>(stage + rr * pitch + c);
            }
        }
    }
    if (abort_flag && tid == 0) {
        // gave up: let the copies that may still be in flight land before shared memory is released
        for (int s = 0; s < stages; ++s) mbar_drain(smem_u32(&bar_full[s]), 0);
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem_d, (uint32_t)args.tmem_cols);
}

}  // namespace sd_attn
