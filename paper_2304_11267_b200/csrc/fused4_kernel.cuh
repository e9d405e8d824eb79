// Fused single-pass attention for small head dims (d <= 64, i.e. the d = 40 layers of the UNet).
//
// At d = 40 a score element costs only 160 tensor-core FLOPs but one exponential, and the special
// function unit retires 16 exponentials per clock per SM: the softmax, not the tensor pipe, bounds the
// kernel.  Two softmax warps per scheduler keep that unit about 95% busy only while both are inside
// their exponential loop; loads from tensor memory, barrier waits and the tensor-core round trip leave
// it idle.  This kernel therefore runs FOUR query tiles of 128 rows per CTA -- four softmax warpgroups,
// four warps per scheduler -- over key tiles of 64, so that some group is always in its exponentials:
//   warps 0-15   softmax of tiles 0..3 (thread = query row = TMEM lane), 112 registers each
//   warp 16      TMA producer          warps 17-20  MMA issuers, one per tile (32 registers each;
//                warps 21-23 only fill the second control warpgroup so that setmaxnreg applies)
// Tensor memory (512 columns): per tile S_t (64 columns, fp32) and O_t (dpad <= 64 columns); the packed
// fp16 weights P_t overwrite the first 32 columns of S_t, so the next S_t is issued after the P V
// product of the current key tile (in issue order on the same thread).
// The running-max rescale of O_t is lazy (only when the max grew by more than 2^8) and safe without
// an extra barrier: S_t(j) being ready implies that the P V product of tile j-1 has completed.
#pragma once
#include <cuda.h>

#include "cross_kernel.cuh"  // TILE_M, CHUNK_COLS, CHUNK_ROW_BYTES
#include "fused_kernel.cuh"  // FUSED_RESCALE_LOG2, FUSED_TRACE
#include "tc_common.cuh"

namespace sd_attn {

constexpr int F4_TILES = 4;
constexpr int F4_BN = 64;
constexpr int F4_THREADS = 24 * 32;   // 16 softmax warps + 8 control warps (producer, 4 issuers, 3 idle)
constexpr int F4_SOFTMAX_REGS = 104;  // after setmaxnreg: 512 * 104 + 256 * 32 = 61440 of the 65536 registers
constexpr int F4_CONTROL_REGS = 32;
constexpr int F4_STAGES = 8;
constexpr int F4_MAX_D = 64;

struct Fused4Args {
    __half* out;  // [BH][Nq][d]
    int Nq, Nk, d;
    int dpad;     // d rounded up to 16 (<= 64)
    float scale_log2e;
    int negate;
    int* status;
#ifdef SD_ATTN_TRACE
    long long* trace;
#endif
};

__host__ inline size_t fused4_smem_bytes() {
    return (size_t)F4_TILES * TILE_M * CHUNK_ROW_BYTES + (size_t)F4_STAGES * 2 * F4_BN * CHUNK_ROW_BYTES + 1024;
}

enum { SITE_G_Q = 30, SITE_G_KV = 31, SITE_G_EMPTY = 32, SITE_G_S = 33, SITE_G_P = 34, SITE_G_O = 35 };

__global__ void __launch_bounds__(F4_THREADS, 1)
fused4_attention_kernel(const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_k,
                        const __grid_constant__ CUtensorMap tmap_v, const Fused4Args args) {
    extern __shared__ uint8_t f4_smem_raw[];
    __shared__ __align__(8) uint64_t bar_q_full[F4_TILES], bar_s_full[F4_TILES], bar_p_full[F4_TILES],
        bar_o_done[F4_TILES];
    __shared__ __align__(8) uint64_t bar_kv_full[F4_STAGES], bar_kv_empty[F4_STAGES];
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int bh = blockIdx.y;
    const int row_base = blockIdx.x * F4_TILES * TILE_M;
    int n_qtiles = (args.Nq - row_base + TILE_M - 1) / TILE_M;
    if (n_qtiles > F4_TILES) n_qtiles = F4_TILES;
    const int n_kv = (args.Nk + F4_BN - 1) / F4_BN;
    const int dpad = args.dpad;

    const uint32_t smem_base = (smem_u32(f4_smem_raw) + 1023u) & ~1023u;
    constexpr uint32_t q_tile_bytes = TILE_M * CHUNK_ROW_BYTES;     // one 64-column chunk (d <= 64)
    constexpr uint32_t kv_tile_bytes = F4_BN * CHUNK_ROW_BYTES;
    const uint32_t q_smem = smem_base;                              // [4][128 rows][128 B]
    const uint32_t kv_smem = q_smem + F4_TILES * q_tile_bytes;      // [stages][K | V][64 rows][128 B]
    volatile int* abort_p = &abort_flag;

    if (tid == 0) {
        abort_flag = 0;
        for (int t = 0; t < F4_TILES; ++t) {
            mbar_init(smem_u32(&bar_q_full[t]), 1);
            mbar_init(smem_u32(&bar_s_full[t]), 1);
            mbar_init(smem_u32(&bar_p_full[t]), 4);    // one arrival per softmax warp
            mbar_init(smem_u32(&bar_o_done[t]), 1);
        }
        for (int s = 0; s < F4_STAGES; ++s) {
            mbar_init(smem_u32(&bar_kv_full[s]), 1);
            mbar_init(smem_u32(&bar_kv_empty[s]), n_qtiles);   // one commit per issuer
        }
        mbar_init_fence();
    }
    if (warp == 16) {
        tmem_alloc(smem_u32(&tmem_base_slot), 512);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = tmem_base_slot;
    // columns: S_0 S_1 S_2 S_3 (64 each) | O_0 O_1 O_2 O_3 (dpad each)
    const uint32_t tmem_o0 = tmem_base + F4_TILES * F4_BN;

    // All four warps of a warpgroup must execute the SAME setmaxnreg instruction: one site per kind.
    if (warp >= 16) setmaxnreg_dec<F4_CONTROL_REGS>();
    if (warp == 16) {
        // ------------------------------------------------------------ TMA producer
        if (elect_one()) {
            tma_prefetch_desc(&tmap_q);
            tma_prefetch_desc(&tmap_k);
            tma_prefetch_desc(&tmap_v);
            for (int t = 0; t < n_qtiles; ++t) {
                const uint32_t bar = smem_u32(&bar_q_full[t]);
                mbar_arrive_expect_tx(bar, q_tile_bytes);
                tma_load_3d(q_smem + t * q_tile_bytes, &tmap_q, bar, 0, row_base + t * TILE_M, bh);
            }
            for (int j = 0; j < n_kv; ++j) {
                const int s = j % F4_STAGES;
                if (j >= F4_STAGES && !mbar_wait(smem_u32(&bar_kv_empty[s]), ((j / F4_STAGES) - 1) & 1, abort_p,
                                                 args.status, SITE_G_EMPTY, j))
                    break;
                const uint32_t k_dst = kv_smem + s * 2 * kv_tile_bytes, v_dst = k_dst + kv_tile_bytes;
                const uint32_t bar = smem_u32(&bar_kv_full[s]);
                mbar_arrive_expect_tx(bar, 2 * kv_tile_bytes);
                tma_load_3d(k_dst, &tmap_k, bar, 0, j * F4_BN, bh);
                tma_load_3d(v_dst, &tmap_v, bar, 0, j * F4_BN, bh);
            }
        }
    } else if (warp > 16) {
        // ------------------------------------------------------------ MMA issuer of query tile t
        const int t = warp - 17;
        if (t < F4_TILES && t < n_qtiles && elect_one()) {
            const uint32_t idesc_s = idesc_f16(TILE_M, F4_BN, false, false, args.negate != 0);
            const uint32_t idesc_o = idesc_f16(TILE_M, dpad, false, true, false);
            const int ksteps_s = (args.d + 15) / 16;   // <= 4: all inside one swizzled 64-column chunk
            const uint64_t q_desc = smem_desc_sw128(q_smem + t * q_tile_bytes, 16, 1024);
            const uint64_t k_desc = smem_desc_sw128(kv_smem, 16, 1024);
            const uint64_t v_desc = smem_desc_sw128(kv_smem + kv_tile_bytes, F4_BN * CHUNK_ROW_BYTES, 1024);
            constexpr uint32_t stage_off = (2 * kv_tile_bytes) >> 4;
            const uint32_t tmem_s = tmem_base + t * F4_BN;
            const uint32_t tmem_o = tmem_o0 + t * dpad;
            const uint32_t b_sfull = smem_u32(&bar_s_full[t]), b_pfull = smem_u32(&bar_p_full[t]);

            auto issue_s = [&](int s) {   // S_t = Q_t K_s^T
                const uint64_t kd = k_desc + (uint64_t)(s * stage_off);
#pragma unroll
                for (int kk = 0; kk < 4; ++kk)
                    if (kk < ksteps_s) mma_f16_ss(tmem_s, q_desc + (uint64_t)(kk * 2), kd + (uint64_t)(kk * 2), idesc_s, kk > 0);
                tc_commit(b_sfull);
            };
            auto issue_o = [&](int s, bool accumulate) {   // O_t (+)= P_t V_s
                const uint64_t vd = v_desc + (uint64_t)(s * stage_off);
#pragma unroll
                for (int kk = 0; kk < F4_BN / 16; ++kk)
                    mma_f16_ts(tmem_o, tmem_s + kk * 8, vd + (uint64_t)(kk * ((16 * CHUNK_ROW_BYTES) >> 4)), idesc_o,
                               accumulate || kk > 0);
            };

            bool ok = mbar_wait(smem_u32(&bar_q_full[t]), 0, abort_p, args.status, SITE_G_Q, t) &&
                      mbar_wait(smem_u32(&bar_kv_full[0]), 0, abort_p, args.status, SITE_G_KV, 0);
            if (ok) {
                tc_fence_after_sync();
                issue_s(0);
            }
            for (int j = 0; j < n_kv && ok; ++j) {
                const int s = j % F4_STAGES, s1 = (j + 1) % F4_STAGES;
                if (j + 1 < n_kv)   // landed long ago: keep this wait off the critical path
                    ok = mbar_wait(smem_u32(&bar_kv_full[s1]), ((j + 1) / F4_STAGES) & 1, abort_p, args.status,
                                   SITE_G_KV, j + 1);
                if (t == 0) FUSED_TRACE(4, j, 0);
                if (ok) ok = mbar_wait(b_pfull, j & 1, abort_p, args.status, SITE_G_P, j);
                if (!ok) break;
                tc_fence_after_sync();
                if (t == 0) FUSED_TRACE(4, j, 1);
                issue_o(s, j > 0);
                tc_commit(smem_u32(&bar_kv_empty[s]));   // this issuer is done with K_j and V_j
                if (j + 1 < n_kv) issue_s(s1);           // also tells the softmax that O_t holds tiles 0..j
                else tc_commit(smem_u32(&bar_o_done[t]));
                if (t == 0) FUSED_TRACE(4, j, 2);
            }
        }
    } else {
        // ------------------------------------------------------------ softmax warps
        setmaxnreg_inc<F4_SOFTMAX_REGS>();
        const int t = warp >> 2;                 // query tile of this warpgroup
        if (t < n_qtiles) {
            const int r = tid & (TILE_M - 1);    // row inside the tile = TMEM lane
            const uint32_t lane_off = (uint32_t)((warp & 3) * 32) << 16;
            const uint32_t tmem_s = tmem_base + t * F4_BN + lane_off;
            const uint32_t tmem_o = tmem_o0 + t * dpad + lane_off;
            const uint32_t b_sfull = smem_u32(&bar_s_full[t]), b_pfull = smem_u32(&bar_p_full[t]);
            const float c2 = args.scale_log2e;
            float m_run = -INFINITY;  // running max, in raw score units
            float l_run = 0.f;        // running sum of p (relative to m_run)
            bool ok = true;
            const bool tracer = (warp & 3) == 0 && lane == 0;
            for (int j = 0; j < n_kv; ++j) {
                if (tracer) FUSED_TRACE(t, j, 0);
                ok = mbar_wait(b_sfull, j & 1, abort_p, args.status, SITE_G_S, j);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                tc_fence_after_sync();
                if (tracer) FUSED_TRACE(t, j, 1);
                const int valid = args.Nk - j * F4_BN;   // columns >= valid are zero-filled keys
                uint32_t s[F4_BN];
                tmem_ld32(tmem_s, &s[0]);
                tmem_ld32(tmem_s + 32, &s[32]);
                tmem_wait_ld();
                if (tracer) FUSED_TRACE(t, j, 2);
                float mx[8];
#pragma unroll
                for (int c = 0; c < 8; ++c) mx[c] = -INFINITY;
                if (valid >= F4_BN) {
#pragma unroll
                    for (int c = 0; c < F4_BN; ++c) mx[c & 7] = fmaxf(mx[c & 7], __uint_as_float(s[c]));
                } else {   // zero-filled key rows take no part in the maximum
#pragma unroll
                    for (int c = 0; c < F4_BN; ++c)
                        if (c < valid) mx[c & 7] = fmaxf(mx[c & 7], __uint_as_float(s[c]));
                }
                const float row_max = fmaxf(fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3])),
                                            fmaxf(fmaxf(mx[4], mx[5]), fmaxf(mx[6], mx[7])));
                if (j == 0) {
                    m_run = row_max;
                } else {
                    const bool grow = (row_max - m_run) * c2 > FUSED_RESCALE_LOG2;
                    if (__any_sync(0xffffffffu, grow)) {
                        // rare: rescale O_t in 8-column pieces, then fetch the row of S_t again (its
                        // registers are reused here to keep the common path within the register budget)
                        const float alpha = grow ? ex2_approx((m_run - row_max) * c2) : 1.f;
                        if (grow) m_run = row_max;
                        l_run *= alpha;
                        for (int g = 0; g < (dpad >> 4); ++g) {
                            tmem_ld16(tmem_o + g * 16, *reinterpret_cast<uint32_t(*)[16]>(&s[0]));
                            tmem_wait_ld();
#pragma unroll
                            for (int c = 0; c < 16; ++c) s[c] = __float_as_uint(__uint_as_float(s[c]) * alpha);
                            tmem_st16(tmem_o + g * 16, *reinterpret_cast<uint32_t(*)[16]>(&s[0]));
                        }
                        tmem_wait_st();
                        tmem_ld32(tmem_s, &s[0]);
                        tmem_ld32(tmem_s + 32, &s[32]);
                        tmem_wait_ld();
                    }
                }
                const float neg_mc = -m_run * c2;
                if (tracer) FUSED_TRACE(t, j, 3);
                float sum[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                for (int g = 0; g < F4_BN / 32; ++g) {
                    uint32_t packed[16];
#pragma unroll
                    for (int c = 0; c < 32; c += 2) {
                        float p0 = ex2_approx(fmaf(__uint_as_float(s[g * 32 + c]), c2, neg_mc));
                        float p1 = ex2_approx(fmaf(__uint_as_float(s[g * 32 + c + 1]), c2, neg_mc));
                        if (valid < F4_BN) {   // zero-filled key rows carry no weight (also when scale == 0)
                            if (g * 32 + c >= valid) p0 = 0.f;
                            if (g * 32 + c + 1 >= valid) p1 = 0.f;
                        }
                        sum[(c >> 1) & 3] += p0 + p1;
                        packed[c >> 1] = pack_half2(p0, p1);
                    }
                    tmem_st16(tmem_s + g * 16, packed);   // P_t over columns of S_t that already sit in registers
                }
                l_run += (sum[0] + sum[1]) + (sum[2] + sum[3]);
                if (tracer) FUSED_TRACE(t, j, 4);
                tmem_wait_st();
                tc_fence_before_sync();
                if (lane == 0) mbar_arrive(b_pfull);
                if (tracer) FUSED_TRACE(t, j, 5);
            }
            if (ok) ok = mbar_wait(smem_u32(&bar_o_done[t]), 0, abort_p, args.status, SITE_G_O, t);
            ok = __all_sync(0xffffffffu, ok);
            if (ok) {
                tc_fence_after_sync();
                const float inv = 1.f / l_run;
                const int row = row_base + t * TILE_M + r;
                __half* orow = args.out + ((size_t)bh * args.Nq + row) * args.d;
                for (int g = 0; g < (dpad >> 4); ++g) {
                    uint32_t x[16];
                    tmem_ld16(tmem_o + g * 16, x);
                    tmem_wait_ld();
                    uint4 lo, hi;
                    lo.x = pack_half2(__uint_as_float(x[0]) * inv, __uint_as_float(x[1]) * inv);
                    lo.y = pack_half2(__uint_as_float(x[2]) * inv, __uint_as_float(x[3]) * inv);
                    lo.z = pack_half2(__uint_as_float(x[4]) * inv, __uint_as_float(x[5]) * inv);
                    lo.w = pack_half2(__uint_as_float(x[6]) * inv, __uint_as_float(x[7]) * inv);
                    hi.x = pack_half2(__uint_as_float(x[8]) * inv, __uint_as_float(x[9]) * inv);
                    hi.y = pack_half2(__uint_as_float(x[10]) * inv, __uint_as_float(x[11]) * inv);
                    hi.z = pack_half2(__uint_as_float(x[12]) * inv, __uint_as_float(x[13]) * inv);
                    hi.w = pack_half2(__uint_as_float(x[14]) * inv, __uint_as_float(x[15]) * inv);
                    if (row < args.Nq) {
                        if (g * 16 + 8 <= args.d) *reinterpret_cast<uint4*>(orow + g * 16) = lo;
                        if (g * 16 + 16 <= args.d) *reinterpret_cast<uint4*>(orow + g * 16 + 8) = hi;
                    }
                }
            }
        }
    }

    // ------------------------------------------------------------ teardown (every thread arrives)
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 16 && lane == 0 && abort_flag) {
        for (int s = 0; s < F4_STAGES; ++s) mbar_drain(smem_u32(&bar_kv_full[s]), 0);
    }
    __syncthreads();
    if (warp == 16) {
        __syncwarp();
        tmem_dealloc(tmem_base, 512);
    }
}

}  // namespace sd_attn
