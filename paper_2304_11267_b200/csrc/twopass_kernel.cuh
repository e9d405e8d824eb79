// Two-pass "partially fused softmax" comparator (Sec. 3.2.1, Eq. 4, Fig. 2), for sm_100a.
//
// This is the paper's first optimisation kept as a second path so that what fusion saves can be
// measured: the score matrix A = Q K^T * scale IS written to HBM (binary32), but the softmax is
// never run as an op of its own.
//   pass 1  twopass_scores_kernel: A tile by tile (tcgen05.mma into tensor memory), stored to HBM;
//           the row reductions are done in stages -- a partial (max, sum of exp) per block of 128
//           columns, merged into the running [L_i, S_i] -- and the N x 2 tensor [L, S] is written
//           at the end of the same launch.
//   pass 2  twopass_pv_kernel: loads A, applies exp(a - L_i) / S_i element-wise while building the
//           left operand of the product with V (fp16 tiles in swizzled shared memory), and
//           accumulates O = P V in tensor memory.  No P tensor exists in HBM.
#pragma once
#include <cuda.h>

#include "cross_kernel.cuh"  // TILE_M, CHUNK_COLS, CHUNK_ROW_BYTES
#include "tc_common.cuh"

namespace sd_attn {

constexpr int TWOPASS_BN = 128;        // key columns per block of the staged reduction
constexpr int TWOPASS_THREADS = 256;
constexpr int TP_STAGE_COLS = 64;      // columns staged through shared memory at a time (pass 1)
constexpr int TP_STAGE_LD = TP_STAGE_COLS + 1;

struct TwoPassArgs {
    float* scores;   // [BH][Nq][Nk] binary32, the matrix A
    float* stats;    // [BH][Nq][2]  binary32, (L_i, S_i) of Eq. 4
    __half* out;     // [BH][Nq][d]
    int Nq, Nk, d;
    int dpad, nch;
    float scale;     // as given (natural units); |scale| goes to the epilogue, the sign to the MMA
    int negate;
    int* status;
};

__host__ inline void twopass_fill_args(TwoPassArgs* a, float* scores, float* stats, __half* out, int Nq, int Nk, int d,
                                       float scale, int* status) {
    a->scores = scores; a->stats = stats; a->out = out;
    a->Nq = Nq; a->Nk = Nk; a->d = d;
    a->dpad = (d + 15) / 16 * 16;
    a->nch = (d + CHUNK_COLS - 1) / CHUNK_COLS;
    a->scale = scale < 0.f ? -scale : scale;
    a->negate = scale < 0.f;
    a->status = status;
}

__host__ inline size_t twopass_scores_smem_bytes(int nch) {
    // Q tile + two K stages + the store staging buffer
    return (size_t)nch * TILE_M * CHUNK_ROW_BYTES + (size_t)2 * nch * TWOPASS_BN * CHUNK_ROW_BYTES +
           (size_t)TILE_M * TP_STAGE_LD * sizeof(float) + 1024;
}
__host__ inline size_t twopass_pv_smem_bytes(int nch) {
    // two P tiles (128 x 128 fp16) + two V stages
    return (size_t)2 * 2 * TILE_M * CHUNK_ROW_BYTES + (size_t)2 * nch * TWOPASS_BN * CHUNK_ROW_BYTES + 1024;
}

enum { SITE_T_Q = 20, SITE_T_K = 21, SITE_T_S = 22, SITE_T_V = 23, SITE_T_MMA = 24, SITE_T_O = 25 };

static constexpr float TP_LOG2E = 1.4426950408889634f;

// ---------------------------------------------------------------------------------------- pass 1
__global__ void __launch_bounds__(TWOPASS_THREADS)
twopass_scores_kernel(const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_k,
                      const TwoPassArgs args) {
    extern __shared__ uint8_t tp1_smem_raw[];
    __shared__ __align__(8) uint64_t bar_q, bar_k[2], bar_s[2];
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int tile = blockIdx.x, bh = blockIdx.y;
    const int row0 = tile * TILE_M;
    const int nch = args.nch;
    const int n_kv = (args.Nk + TWOPASS_BN - 1) / TWOPASS_BN;

    const uint32_t smem_base = (smem_u32(tp1_smem_raw) + 1023u) & ~1023u;
    const uint32_t q_smem = smem_base;
    const uint32_t k_tile_bytes = nch * TWOPASS_BN * CHUNK_ROW_BYTES;
    const uint32_t k_smem = q_smem + nch * TILE_M * CHUNK_ROW_BYTES;
    float* stage = reinterpret_cast<float*>(tp1_smem_raw + (smem_base - smem_u32(tp1_smem_raw)) +
                                            nch * TILE_M * CHUNK_ROW_BYTES + 2 * k_tile_bytes);
    volatile int* abort_p = &abort_flag;

    if (tid == 0) {
        abort_flag = 0;
        mbar_init(smem_u32(&bar_q), 1);
        for (int s = 0; s < 2; ++s) {
            mbar_init(smem_u32(&bar_k[s]), 1);
            mbar_init(smem_u32(&bar_s[s]), 1);
        }
        mbar_init_fence();
    }
    if (warp == 0) {
        tmem_alloc(smem_u32(&tmem_base_slot), 256);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = tmem_base_slot;
    const uint32_t idesc = idesc_f16(TILE_M, TWOPASS_BN, false, false, args.negate != 0);
    const int ksteps = (args.d + 15) / 16;

    auto load_k = [&](int j) {
        const int s = j & 1;
        const uint32_t bar = smem_u32(&bar_k[s]);
        mbar_arrive_expect_tx(bar, k_tile_bytes);
        for (int ch = 0; ch < nch; ++ch)
            tma_load_4d(k_smem + s * k_tile_bytes + ch * TWOPASS_BN * CHUNK_ROW_BYTES, &tmap_k, bar, ch * CHUNK_COLS,
                        j * TWOPASS_BN, bh, 0);
    };
    auto issue_s = [&](int j) {   // S_(j&1) = Q K_j^T
        const int s = j & 1;
        for (int kk = 0; kk < ksteps; ++kk) {
            const int ch = kk >> 2, within = (kk & 3) * 32;
            mma_f16_ss(tmem_base + s * TWOPASS_BN,
                       smem_desc_sw128(q_smem + ch * TILE_M * CHUNK_ROW_BYTES + within, 16, 1024),
                       smem_desc_sw128(k_smem + s * k_tile_bytes + ch * TWOPASS_BN * CHUNK_ROW_BYTES + within, 16, 1024),
                       idesc, kk > 0);
        }
        tc_commit(smem_u32(&bar_s[s]));
    };

    bool ok = true;
    if (tid == 0) {
        const uint32_t bq = smem_u32(&bar_q);
        mbar_arrive_expect_tx(bq, nch * TILE_M * CHUNK_ROW_BYTES);
        for (int ch = 0; ch < nch; ++ch)
            tma_load_4d(q_smem + ch * TILE_M * CHUNK_ROW_BYTES, &tmap_q, bq, ch * CHUNK_COLS, row0, bh, 0);
        load_k(0);
        if (n_kv > 1) load_k(1);
        ok = mbar_wait(bq, 0, abort_p, args.status, SITE_T_Q, tile) &&
             mbar_wait(smem_u32(&bar_k[0]), 0, abort_p, args.status, SITE_T_K, 0);
        if (ok) {
            tc_fence_after_sync();
            issue_s(0);
        }
    }

    // rows are owned by warps 0-3 (thread = row = TMEM lane); warps 4-7 only help with the stores
    const bool owner = warp < 4;
    const uint32_t lane_off = (uint32_t)((warp & 3) * 32) << 16;
    float L_run = -INFINITY, S_run = 0.f;   // natural-log units, as Eq. 4 defines them

    for (int j = 0; j < n_kv; ++j) {
        const int s = j & 1;
        // launch the next tile's MMA before consuming this one (its S buffer was released by the
        // __syncthreads at the end of iteration j-1)
        if (tid == 0 && ok && j + 1 < n_kv) {
            ok = mbar_wait(smem_u32(&bar_k[s ^ 1]), ((j + 1) >> 1) & 1, abort_p, args.status, SITE_T_K, j + 1);
            if (ok) {
                tc_fence_after_sync();
                issue_s(j + 1);
            }
        }
        // block-uniform decision: the loop body holds __syncthreads, so all warps leave together
        const bool got = mbar_wait(smem_u32(&bar_s[s]), (j >> 1) & 1, abort_p, args.status, SITE_T_S, j);
        if (!__syncthreads_and(got)) break;
        tc_fence_after_sync();
        // K stage s is free again (its MMA has completed): prefetch tile j+2 into it
        if (tid == 0 && j + 2 < n_kv) load_k(j + 2);

        const int col0 = j * TWOPASS_BN;
        // stage 1 of the reduction: this block's partial maximum
        float bmax = -INFINITY;
        if (owner) {
#pragma unroll
            for (int g = 0; g < TWOPASS_BN / 16; ++g) {
                uint32_t x[16];
                tmem_ld16(tmem_base + s * TWOPASS_BN + lane_off + g * 16, x);
                tmem_wait_ld();
#pragma unroll
                for (int c = 0; c < 16; ++c)
                    if (col0 + g * 16 + c < args.Nk) bmax = fmaxf(bmax, __uint_as_float(x[c]) * args.scale);
            }
        }
        float bsum = 0.f;
        for (int half = 0; half < TWOPASS_BN / TP_STAGE_COLS; ++half) {
            if (owner) {
#pragma unroll
                for (int g = 0; g < TP_STAGE_COLS / 16; ++g) {
                    uint32_t x[16];
                    tmem_ld16(tmem_base + s * TWOPASS_BN + lane_off + half * TP_STAGE_COLS + g * 16, x);
                    tmem_wait_ld();
#pragma unroll
                    for (int c = 0; c < 16; ++c) {
                        const float a = __uint_as_float(x[c]) * args.scale;
                        if (col0 + half * TP_STAGE_COLS + g * 16 + c < args.Nk)
                            bsum += ex2_approx((a - bmax) * TP_LOG2E);
                        stage[tid * TP_STAGE_LD + g * 16 + c] = a;
                    }
                }
            }
            __syncthreads();
            // coalesced store of the staged 128 x 64 block of A: lane = column
            for (int r = warp; r < TILE_M; r += TWOPASS_THREADS / 32) {
                const int row = row0 + r;
                if (row >= args.Nq) break;
                float* dst = args.scores + ((size_t)bh * args.Nq + row) * args.Nk;
#pragma unroll
                for (int cc = 0; cc < TP_STAGE_COLS; cc += 32) {
                    const int col = col0 + half * TP_STAGE_COLS + cc + lane;
                    if (col < args.Nk) dst[col] = stage[r * TP_STAGE_LD + cc + lane];
                }
            }
            __syncthreads();
        }
        // stage 2: merge the block partial into the running (L, S)
        if (owner) {
            const float L_new = fmaxf(L_run, bmax);
            S_run = S_run * ex2_approx((L_run - L_new) * TP_LOG2E) + bsum * ex2_approx((bmax - L_new) * TP_LOG2E);
            L_run = L_new;
        }
        tc_fence_before_sync();
        __syncthreads();   // every reader of S_(j&1) is done: the MMA of tile j+2 may overwrite it
    }

    if (owner && row0 + tid < args.Nq && !abort_flag) {
        float2* st = reinterpret_cast<float2*>(args.stats) + ((size_t)bh * args.Nq + row0 + tid);
        *st = make_float2(L_run, S_run);
    }
    tc_fence_before_sync();
    __syncthreads();
    if (tid == 0 && abort_flag) {
        mbar_drain(smem_u32(&bar_q), 0);
        mbar_drain(smem_u32(&bar_k[0]), 0);
        mbar_drain(smem_u32(&bar_k[1]), 0);
    }
    __syncthreads();
    if (warp == 0) {
        __syncwarp();
        tmem_dealloc(tmem_base, 256);
    }
}

// ---------------------------------------------------------------------------------------- pass 2
__global__ void __launch_bounds__(TWOPASS_THREADS)
twopass_pv_kernel(const __grid_constant__ CUtensorMap tmap_v, const TwoPassArgs args) {
    extern __shared__ uint8_t tp2_smem_raw[];
    __shared__ __align__(8) uint64_t bar_v[2], bar_mma[2], bar_o;
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;
    __shared__ float row_L[TILE_M], row_invS[TILE_M];

    const int tid = threadIdx.x, warp = tid >> 5;
    const int tile = blockIdx.x, bh = blockIdx.y;
    const int row0 = tile * TILE_M;
    const int nch = args.nch, dpad = args.dpad;
    const int n_kv = (args.Nk + TWOPASS_BN - 1) / TWOPASS_BN;
    const int tmem_cols = dpad <= 64 ? 64 : (dpad <= 128 ? 128 : 256);

    const uint32_t smem_base_u32 = (smem_u32(tp2_smem_raw) + 1023u) & ~1023u;
    uint8_t* smem_base_ptr = tp2_smem_raw + (smem_base_u32 - smem_u32(tp2_smem_raw));
    const uint32_t p_tile_bytes = 2 * TILE_M * CHUNK_ROW_BYTES;       // two 64-key chunks
    const uint32_t v_tile_bytes = nch * TWOPASS_BN * CHUNK_ROW_BYTES;
    const uint32_t p_smem = smem_base_u32;
    const uint32_t v_smem = p_smem + 2 * p_tile_bytes;
    volatile int* abort_p = &abort_flag;

    if (tid == 0) {
        abort_flag = 0;
        for (int s = 0; s < 2; ++s) {
            mbar_init(smem_u32(&bar_v[s]), 1);
            mbar_init(smem_u32(&bar_mma[s]), 1);
        }
        mbar_init(smem_u32(&bar_o), 1);
        mbar_init_fence();
    }
    if (warp == 0) {
        tmem_alloc(smem_u32(&tmem_base_slot), tmem_cols);
        tmem_relinquish();
    }
    if (tid < TILE_M) {
        const int row = row0 + tid;
        float2 ls = make_float2(0.f, 1.f);
        if (row < args.Nq) ls = reinterpret_cast<const float2*>(args.stats)[(size_t)bh * args.Nq + row];
        row_L[tid] = ls.x;
        row_invS[tid] = 1.f / ls.y;
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_o = tmem_base_slot;
    const uint32_t idesc = idesc_f16(TILE_M, dpad, false, true, false);

    auto load_v = [&](int j) {
        const int s = j & 1;
        const uint32_t bar = smem_u32(&bar_v[s]);
        mbar_arrive_expect_tx(bar, v_tile_bytes);
        for (int ch = 0; ch < nch; ++ch)
            tma_load_4d(v_smem + s * v_tile_bytes + ch * TWOPASS_BN * CHUNK_ROW_BYTES, &tmap_v, bar, ch * CHUNK_COLS,
                        j * TWOPASS_BN, bh, 0);
    };
    if (tid == 0) {
        tma_prefetch_desc(&tmap_v);
        load_v(0);
    }

    const bool vec_ok = (args.Nk & 3) == 0;   // rows of A are then 16-byte aligned
    bool ok = true;
    for (int j = 0; j < n_kv; ++j) {
        const int s = j & 1;
        // buffers of parity s were last read by the MMA of tile j-2
        if (j >= 2) ok = mbar_wait(smem_u32(&bar_mma[s]), ((j >> 1) - 1) & 1, abort_p, args.status, SITE_T_MMA, j);
        ok = __syncthreads_and(ok);   // block-uniform: the loop body holds __syncthreads
        if (!ok) break;
        if (tid == 0 && j + 1 < n_kv) {
            // V stage s^1 was last read by the MMA of tile j-1
            bool free1 = true;
            if (j >= 1) free1 = mbar_wait(smem_u32(&bar_mma[s ^ 1]), ((j - 1) >> 1) & 1, abort_p, args.status, SITE_T_MMA, j);
            if (free1) load_v(j + 1);
        }
        // element-wise softmax fused into the operand load: p = exp(a - L_i) / S_i  ->  fp16, swizzled
        uint8_t* p_tile = smem_base_ptr + s * p_tile_bytes;
        const int col0 = j * TWOPASS_BN;
        for (int item = tid; item < TILE_M * (TWOPASS_BN / 8); item += TWOPASS_THREADS) {
            const int r = item >> 4, cg = item & 15;       // 8 consecutive columns of one row
            const int row = row0 + r, col = col0 + cg * 8;
            float a[8];
            if (row < args.Nq && vec_ok && col + 8 <= args.Nk) {
                const float4* src = reinterpret_cast<const float4*>(args.scores + ((size_t)bh * args.Nq + row) * args.Nk + col);
                const float4 lo = __ldcs(src), hi = __ldcs(src + 1);
                a[0] = lo.x; a[1] = lo.y; a[2] = lo.z; a[3] = lo.w;
                a[4] = hi.x; a[5] = hi.y; a[6] = hi.z; a[7] = hi.w;
            } else {
#pragma unroll
                for (int c = 0; c < 8; ++c)
                    a[c] = (row < args.Nq && col + c < args.Nk)
                               ? args.scores[((size_t)bh * args.Nq + row) * args.Nk + col + c]
                               : -INFINITY;   // exp(-inf) = 0: no weight
            }
            const float L = row_L[r], invS = row_invS[r];
            uint4 packed;
            uint32_t* pk = reinterpret_cast<uint32_t*>(&packed);
#pragma unroll
            for (int c = 0; c < 4; ++c)
                pk[c] = pack_half2(ex2_approx((a[2 * c] - L) * TP_LOG2E) * invS,
                                   ex2_approx((a[2 * c + 1] - L) * TP_LOG2E) * invS);
            const int chunk = cg >> 3, unit = cg & 7;
            *reinterpret_cast<uint4*>(p_tile + chunk * TILE_M * CHUNK_ROW_BYTES + r * CHUNK_ROW_BYTES +
                                      ((unit ^ (r & 7)) << 4)) = packed;
        }
        fence_proxy_async_smem();   // generic-proxy writes of P -> visible to the tensor core
        __syncthreads();
        if (tid == 0) {
            if (mbar_wait(smem_u32(&bar_v[s]), (j >> 1) & 1, abort_p, args.status, SITE_T_V, j)) {
                tc_fence_after_sync();
                const uint32_t pa = p_smem + s * p_tile_bytes, vb = v_smem + s * v_tile_bytes;
#pragma unroll
                for (int kk = 0; kk < TWOPASS_BN / 16; ++kk) {
                    const int ch = kk >> 2, within = (kk & 3) * 32;
                    mma_f16_ss(tmem_o, smem_desc_sw128(pa + ch * TILE_M * CHUNK_ROW_BYTES + within, 16, 1024),
                               smem_desc_sw128(vb + kk * 16 * CHUNK_ROW_BYTES, TWOPASS_BN * CHUNK_ROW_BYTES, 1024),
                               idesc, j > 0 || kk > 0);
                }
                tc_commit(smem_u32(&bar_mma[s]));
                if (j == n_kv - 1) tc_commit(smem_u32(&bar_o));
            }
        }
    }

    if (ok) ok = mbar_wait(smem_u32(&bar_o), 0, abort_p, args.status, SITE_T_O, tile);
    ok = __syncthreads_and(ok);
    if (ok && warp < 4) {
        tc_fence_after_sync();
        const uint32_t lane_off = (uint32_t)(warp * 32) << 16;
        const int row = row0 + tid;
        __half* orow = args.out + ((size_t)bh * args.Nq + row) * args.d;
        for (int g = 0; g < (dpad >> 4); ++g) {
            uint32_t x[16];
            tmem_ld16(tmem_o + lane_off + g * 16, x);
            tmem_wait_ld();
            uint4 lo, hi;
            lo.x = pack_half2(__uint_as_float(x[0]), __uint_as_float(x[1]));
            lo.y = pack_half2(__uint_as_float(x[2]), __uint_as_float(x[3]));
            lo.z = pack_half2(__uint_as_float(x[4]), __uint_as_float(x[5]));
            lo.w = pack_half2(__uint_as_float(x[6]), __uint_as_float(x[7]));
            hi.x = pack_half2(__uint_as_float(x[8]), __uint_as_float(x[9]));
            hi.y = pack_half2(__uint_as_float(x[10]), __uint_as_float(x[11]));
            hi.z = pack_half2(__uint_as_float(x[12]), __uint_as_float(x[13]));
            hi.w = pack_half2(__uint_as_float(x[14]), __uint_as_float(x[15]));
            if (row < args.Nq) {
                if (g * 16 + 8 <= args.d) *reinterpret_cast<uint4*>(orow + g * 16) = lo;
                if (g * 16 + 16 <= args.d) *reinterpret_cast<uint4*>(orow + g * 16 + 8) = hi;
            }
        }
    }
    tc_fence_before_sync();
    __syncthreads();
    if (tid == 0 && abort_flag) {
        mbar_drain(smem_u32(&bar_v[0]), 0);
        mbar_drain(smem_u32(&bar_v[1]), 0);
    }
    __syncthreads();
    if (warp == 0) {
        __syncwarp();
        tmem_dealloc(tmem_o, tmem_cols);
    }
}

}  // namespace sd_attn
