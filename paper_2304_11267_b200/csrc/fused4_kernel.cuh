// Fused single-pass attention for small head dims (d <= 64, i.e. the d = 40 layers of the UNet).
//
// At d = 40 a score element costs only 160 tensor-core FLOPs but one exponential, and the special
// function unit retires 16 exponentials per clock per SM: the softmax, not the tensor pipe, bounds the
// kernel.  Two softmax warps per scheduler keep that unit busy only while both are inside their
// exponential sweep; loads from tensor memory, barrier waits and the tensor-core round trip leave it
// idle.  This kernel therefore runs FOUR query tiles of 128 rows per CTA -- four softmax warpgroups,
// four warps per scheduler -- over key tiles of 64:
//   warps 0-15   softmax of tiles 0..3 (thread = query row = TMEM lane), 104 registers each
//   warp 16      TMA producer          warps 17-20  MMA issuers, one per tile (32 registers each;
//                warps 21-23 only fill the second control warpgroup so that setmaxnreg applies)
// Tensor memory (512 columns): per tile S_t (64 fp32 columns) and O_t (dpad <= 64 columns); the packed
// fp16 weights P_t overwrite the first 32 columns of S_t, so the next S_t follows the P V product of the
// current key tile in issue order on the same thread.  (A 48-wide key tile with P_t in columns of its
// own, which takes the tensor-core round trip off the softmax's path, measured slower: the fixed cost
// per key tile outweighs it.)
// No per-tile maximum is taken.  The exponent is anchored FUSED_HEADROOM_LOG2 above the maximum of the row's
// first key tile; a later tile is evaluated against that anchor as it stands, and only when its weights sum to
// more than FUSED_TILE_SUM_LIMIT (a score far above the anchor: rare) is the tile's maximum taken, O_t and the
// row sum rescaled and the tile redone.  Any anchor gives the same result in exact arithmetic; this one keeps
// every weight inside binary16's normal range where it matters.
#pragma once
#include <cuda.h>

#include "cross_kernel.cuh"  // TILE_M, CHUNK_COLS, CHUNK_ROW_BYTES
#include "fused_kernel.cuh"  // FUSED_HEADROOM_LOG2, FUSED_TILE_SUM_LIMIT, FUSED_TRACE, FUSED_POLY_PER8
#include "softmax_math.cuh"
#include "tc_common.cuh"

namespace sd_attn {

constexpr int F4_TILES = 4;
constexpr int F4_BN = 64;
constexpr int F4_THREADS = 24 * 32;   // 16 softmax warps + 8 control warps (producer, 4 issuers, 3 idle)
constexpr int F4_SOFTMAX_REGS = 104;  // after setmaxnreg: 512 * 104 + 256 * 32 = 768 * 80, the launch allocation
constexpr int F4_CONTROL_REGS = 32;
constexpr int F4_STAGES = 8;
constexpr int F4_MAX_D = 64;

struct Fused4Args {
    __half* out;  // [BH][Nq][d], or as `lay` says (spare-buffer kernel only)
    HeadLayout lay;
    int Nq, Nk, d;
    int dpad;     // d rounded up to 16 (<= 64)
    int tiles_per_cta;   // spare-buffer kernel only: 1..4 query tiles per CTA (small problems spread over more SMs)
    int nch;             // spare-buffer kernel only: 64-column chunks per row (1..3)
    int stages;          // spare-buffer kernel only: K/V ring depth (2..8)
    int split_buffers;   // spare-buffer kernel, split variant only: score buffers of the lone tile (2..5)
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

enum { SITE_G_Q = 30, SITE_G_KV = 31, SITE_G_EMPTY = 32, SITE_G_S = 33, SITE_G_P = 34, SITE_G_O = 35, SITE_G_PV = 37 };

__global__ void __launch_bounds__(F4_THREADS, 1)
fused4_attention_kernel(const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_k,
                        const __grid_constant__ CUtensorMap tmap_v, const Fused4Args args) {
    constexpr int BN = F4_BN;
    extern __shared__ uint8_t f4_smem_raw[];
    // per query tile: Q landed | S ready (MMA) | P ready (softmax) | P V done (MMA)
    __shared__ __align__(8) uint64_t bar_q_full[F4_TILES], bar_s_full[F4_TILES], bar_p_full[F4_TILES],
        bar_pv_done[F4_TILES];
    __shared__ __align__(8) uint64_t bar_kv_full[F4_STAGES], bar_kv_empty[F4_STAGES];
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;

    const int tid = threadIdx.x, lane = tid & 31;
    // through a shuffle so that the compiler knows the warp index is warp-uniform (descriptor arithmetic of the
    // issuer then lives in uniform registers)
    const int warp = __shfl_sync(0xffffffffu, tid >> 5, 0);
    const int bh = blockIdx.y;
    const int row_base = blockIdx.x * F4_TILES * TILE_M;
    int n_qtiles = (args.Nq - row_base + TILE_M - 1) / TILE_M;
    if (n_qtiles > F4_TILES) n_qtiles = F4_TILES;
    const int n_kv = (args.Nk + BN - 1) / BN;
    const int dpad = args.dpad;

    const uint32_t smem_base = (smem_u32(f4_smem_raw) + 1023u) & ~1023u;
    constexpr uint32_t q_tile_bytes = TILE_M * CHUNK_ROW_BYTES;     // one 64-column chunk (d <= 64)
    constexpr uint32_t kv_tile_bytes = BN * CHUNK_ROW_BYTES;
    const uint32_t q_smem = smem_base;                              // [4][128 rows][128 B]
    const uint32_t kv_smem = q_smem + F4_TILES * q_tile_bytes;      // [stages][K | V][64 rows][128 B]
    volatile int* abort_p = &abort_flag;

    if (tid == 0) {
        abort_flag = 0;
        for (int t = 0; t < F4_TILES; ++t) {
            mbar_init(smem_u32(&bar_q_full[t]), 1);
            mbar_init(smem_u32(&bar_s_full[t]), 1);
            mbar_init(smem_u32(&bar_p_full[t]), 4);    // one arrival per softmax warp
            mbar_init(smem_u32(&bar_pv_done[t]), 1);
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
    const uint32_t tmem_o0 = tmem_base + F4_TILES * BN;   // columns: S_0..S_3 | O_0..O_3

    // All four warps of a warpgroup must execute the SAME setmaxnreg instruction: one site per kind.
    // setmaxnreg only moves registers INSIDE the CTA's launch allocation (768 threads x registers per thread as
    // compiled): an increase the decreases do not cover blocks for ever, so the host checks the compiled count.
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
                tma_load_4d(q_smem + t * q_tile_bytes, &tmap_q, bar, 0, row_base + t * TILE_M, bh, 0);
            }
            for (int j = 0; j < n_kv; ++j) {
                const int s = j % F4_STAGES;
                if (j >= F4_STAGES && !mbar_wait(smem_u32(&bar_kv_empty[s]), ((j / F4_STAGES) - 1) & 1, abort_p,
                                                 args.status, SITE_G_EMPTY, j))
                    break;
                const uint32_t k_dst = kv_smem + s * 2 * kv_tile_bytes, v_dst = k_dst + kv_tile_bytes;
                const uint32_t bar = smem_u32(&bar_kv_full[s]);
                mbar_arrive_expect_tx(bar, 2 * kv_tile_bytes);
                tma_load_4d(k_dst, &tmap_k, bar, 0, j * BN, bh, 0);
                tma_load_4d(v_dst, &tmap_v, bar, 0, j * BN, bh, 0);
            }
        }
    } else if (warp > 16) {
        // ------------------------------------------------------------ MMA issuer of query tile t
        const int t = warp - 17;
        if (t < F4_TILES && t < n_qtiles && elect_one()) {
            const uint32_t idesc_s = idesc_f16(TILE_M, BN, false, false, args.negate != 0);
            const uint32_t idesc_o = idesc_f16(TILE_M, dpad, false, true, false);
            const int ksteps_s = (args.d + 15) / 16;   // <= 4: all inside one swizzled 64-column chunk
            const uint64_t q_desc = smem_desc_sw128(q_smem + t * q_tile_bytes, 16, 1024);
            const uint64_t k_desc = smem_desc_sw128(kv_smem, 16, 1024);
            const uint64_t v_desc = smem_desc_sw128(kv_smem + kv_tile_bytes, BN * CHUNK_ROW_BYTES, 1024);
            constexpr uint32_t stage_off = (2 * kv_tile_bytes) >> 4;
            const uint32_t tmem_s = tmem_base + t * BN;
            const uint32_t tmem_o = tmem_o0 + t * dpad;
            const uint32_t b_sfull = smem_u32(&bar_s_full[t]), b_pfull = smem_u32(&bar_p_full[t]);
            const uint32_t b_pvdone = smem_u32(&bar_pv_done[t]);

            auto issue_s = [&](int s) {   // S_t = Q_t K_s^T
                const uint64_t kd = k_desc + (uint64_t)(s * stage_off);
#pragma unroll
                for (int kk = 0; kk < 4; ++kk)
                    if (kk < ksteps_s) mma_f16_ss(tmem_s, q_desc + (uint64_t)(kk * 2), kd + (uint64_t)(kk * 2), idesc_s, kk > 0);
                tc_commit(b_sfull);
            };
            auto issue_o = [&](int s, bool accumulate) {   // O_t (+)= P_t V_s, P_t in the first columns of S_t
                const uint64_t vd = v_desc + (uint64_t)(s * stage_off);
#pragma unroll
                for (int kk = 0; kk < BN / 16; ++kk)
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
                if (j + 1 < n_kv) issue_s(s1);                // the softmax waits for this one: commit it first
                tc_commit(b_pvdone);                          // O_t holds tiles 0..j
                tc_commit(smem_u32(&bar_kv_empty[s]));        // this issuer is done with K_j and V_j
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
            const uint32_t tmem_s = tmem_base + t * BN + lane_off;
            const uint32_t tmem_o = tmem_o0 + t * dpad + lane_off;
            const uint32_t b_sfull = smem_u32(&bar_s_full[t]), b_pfull = smem_u32(&bar_p_full[t]);
            const uint32_t b_pvdone = smem_u32(&bar_pv_done[t]);
            const float c2 = args.scale_log2e;
            float m_run = 0.f;        // anchor of the exponent: a bound on the running max, times scale*log2(e)
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
                const int valid = args.Nk - j * BN;   // columns >= valid are zero-filled keys
                uint32_t s[BN];
                tmem_ld32(tmem_s, &s[0]);
                tmem_ld32(tmem_s + 32, &s[32]);
                tmem_wait_ld();
                if (tracer) FUSED_TRACE(t, j, 2);
                const bool ragged = valid < BN;   // only the last key tile can be
                if (j == 0) {
                    const float row_max = ragged ? row_max_masked<BN>(s, valid) : row_max_bf16<BN>(s);
                    m_run = row_max * c2 + FUSED_HEADROOM_LOG2;
                }
                if (tracer) FUSED_TRACE(t, j, 3);
                // The weights of this tile are taken against the anchor as it stands; the tile's own maximum is
                // NOT computed.  A row whose weights sum to more than FUSED_TILE_SUM_LIMIT has met a score far above
                // its anchor: only then (rare) is the maximum taken, O_t and the row sum rescaled and the tile redone.
                uint32_t packed[BN / 2];
                float tile_sum;
#pragma unroll 1
                for (int attempt = 0; attempt < 2; ++attempt) {
                    const float neg_mc = -m_run;
                    if (!ragged) {
                        const uint64_t c2c2 = pack_b64(__float_as_uint(c2), __float_as_uint(c2));
                        const uint64_t nmnm = pack_b64(__float_as_uint(neg_mc), __float_as_uint(neg_mc));
                        uint64_t acc[2] = {0ull, 0ull};
                        exp2_pack_32<FUSED_POLY_PER8>(&s[0], c2c2, nmnm, &packed[0], acc);
                        exp2_pack_32<FUSED_POLY_PER8>(&s[32], c2c2, nmnm, &packed[16], acc);
                        tile_sum = sum_f32x2(acc[0], acc[1]);
                    } else {
                        tile_sum = 0.f;
                        exp2_pack_32_masked(&s[0], c2, neg_mc, 0, valid, &packed[0], tile_sum);
                        exp2_pack_32_masked(&s[32], c2, neg_mc, 32, valid, &packed[16], tile_sum);
                    }
                    const bool over = !(tile_sum <= FUSED_TILE_SUM_LIMIT);
                    if (attempt == 1 || !__any_sync(0xffffffffu, over)) break;
                    // S_t(j) being ready means the P V product of tile j-1 was issued before it and has completed,
                    // so O_t may be touched; nothing of P_t(j) has been stored yet, so the scores are still in
                    // tensor memory.  The first registers of the score row are borrowed for O_t (register budget).
                    tmem_ld32(tmem_s, &s[0]);
                    tmem_ld32(tmem_s + 32, &s[32]);
                    tmem_wait_ld();
                    // (the exact maximum: the truncated one may lie below it by more than the headroom)
                    const float row_max = row_max_masked<BN>(s, ragged ? valid : BN);
                    const float m_new = row_max * c2 + FUSED_HEADROOM_LOG2;
                    const float alpha = over ? ex2_approx(m_run - m_new) : 1.f;
                    if (over) m_run = m_new;
                    l_run *= alpha;
                    if (j > 0) {
                        for (int g = 0; g < (dpad >> 4); ++g) {
                            tmem_ld16(tmem_o + g * 16, *reinterpret_cast<uint32_t(*)[16]>(&s[0]));
                            tmem_wait_ld();
#pragma unroll
                            for (int c = 0; c < 16; ++c) s[c] = __float_as_uint(__uint_as_float(s[c]) * alpha);
                            tmem_st16(tmem_o + g * 16, *reinterpret_cast<uint32_t(*)[16]>(&s[0]));
                        }
                        tmem_wait_st();
                    }
                    tmem_ld32(tmem_s, &s[0]);
                    tmem_ld32(tmem_s + 32, &s[32]);
                    tmem_wait_ld();
                }
                l_run += tile_sum;
                tmem_st32(tmem_s, packed);   // P_t over the first columns of S_t, whose scores sit in registers
                if (tracer) FUSED_TRACE(t, j, 4);
                tmem_wait_st();
                tc_fence_before_sync();
                if (lane == 0) mbar_arrive(b_pfull);
                if (tracer) FUSED_TRACE(t, j, 5);
            }
            if (ok) ok = mbar_wait(b_pvdone, (n_kv - 1) & 1, abort_p, args.status, SITE_G_O, t);
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
