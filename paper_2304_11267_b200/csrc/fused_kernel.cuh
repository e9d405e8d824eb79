// Fused single-pass attention (the FlashAttention evaluation of Eq. 3, Sec. 3.2.2) for sm_100a.
//
// The score matrix never leaves the chip: keys and values stream through shared memory in tiles of
// BN keys, S = Q K^T lands in tensor memory, the softmax reductions of Eq. 4 are kept as running
// per-row (max, sum), and O accumulates in tensor memory.  The paper keeps this kernel to d = 40
// because its accumulators live in registers on mobile GPUs; here they live in the 512-column
// tensor memory, so every head dim up to 160 takes the same path.
//
// One CTA owns TWO tiles of 128 query rows, each with its own softmax warpgroup and its own MMA
// issuer, so that the tensor pipe works for one tile while the other is in its softmax:
//   warps 0-3  softmax of tile 0 (thread = query row = TMEM lane)      warp 8       TMA producer
//   warps 4-7  softmax of tile 1                                        warps 9, 10  MMA issuers
// Per key tile j and query tile t:
//   S_t = Q_t K_j^T          tcgen05.mma, both operands from swizzled shared memory
//   softmax warps            read the row of S_t into registers (S_t is then free for tile j+1); row max;
//                            O_t is rescaled only when the running max grew by more than 2^8 (so
//                            p <= 256 fits fp16); p = exp2(s*c - m*c), a fixed share of them evaluated on
//                            the FMA pipe; P_t written back to tensor memory as packed fp16
//   O_t += P_t V_j           tcgen05.mma, P from tensor memory, V as an N-major shared-memory operand
// Tensor memory (512 columns) holds S_0 S_1 | P_0 P_1 | O_0 O_1, i.e. 3*BN + 2*dpad columns: key
// tiles are 128 wide for d <= 64 and 64 wide above.  P_t has columns of its own, so the next S_t is
// issued as soon as the row of S_t sits in the softmax registers and the tensor-core round trip stays
// off the softmax's path.
// All waits are bounded; an expired wait raises a block-wide abort flag and the kernel returns.
#pragma once
#include <cuda.h>

#include "cross_kernel.cuh"  // TILE_M, CHUNK_COLS, CHUNK_ROW_BYTES
#include "softmax_math.cuh"
#include "tc_common.cuh"

namespace sd_attn {

constexpr int FUSED_THREADS = 352;
constexpr int FUSED_MAX_STAGES = 4;
constexpr int FUSED_MAX_KSTEPS = 10;   // MMA steps of the Q K^T contraction at the largest head dim (160)
constexpr int FUSED_SMEM_BUDGET = 220 * 1024;
// The anchor of the exponent starts FUSED_HEADROOM_LOG2 above the first tile's row max (weights <= 2^-6: the
// eight binades below that are still normal binary16, and what lies further down rounds without bias) and O is
// rescaled only when a later row max exceeds the anchor by more than FUSED_RESCALE_LOG2 (weights <= 2^12, far
// inside binary16's range).  Measured on the "peaked" inputs: headroom 3 re-anchors about one warp-tile in 130
// and costs 3.5% of the 4096-token call; headroom 6 re-anchors almost never, with the same error.
#ifndef SD_ATTN_RESCALE_LOG2
#define SD_ATTN_RESCALE_LOG2 12.0f
#endif
#ifndef SD_ATTN_HEADROOM_LOG2
#define SD_ATTN_HEADROOM_LOG2 6.0f
#endif
constexpr float FUSED_RESCALE_LOG2 = SD_ATTN_RESCALE_LOG2;
constexpr float FUSED_HEADROOM_LOG2 = SD_ATTN_HEADROOM_LOG2;
// The four-tile kernel does not take a key tile's maximum at all: it re-anchors a row only when the weights of
// one tile sum to more than this (so no weight exceeds it: 2^12 is far inside binary16's range).
constexpr float FUSED_TILE_SUM_LIMIT = 4096.0f;
#ifndef SD_ATTN_POLY_PER8
#define SD_ATTN_POLY_PER8 0
#endif
constexpr int FUSED_POLY_PER8 = SD_ATTN_POLY_PER8;  // of every 8 exponentials, this many use the FMA pipe

struct FusedArgs {
    __half* out;  // [BH][Nq][d]
    int Nq, Nk, d;
    int dpad;     // d rounded up to 16
    int nch;      // 64-column chunks per row
    int stages;   // K/V ring depth
    int tiles_per_cta;   // 1 or 2 query tiles per CTA (one when the problem has too few tiles to fill the SMs)
    float scale_log2e;
    int negate;
    int* status;
#ifdef SD_ATTN_TRACE
    long long* trace;   // timeline probe of block (0,0): [role][tile j < 40][8 slots] clock64 stamps
#endif
};

#ifdef SD_ATTN_TRACE
#define FUSED_TRACE(role, j, slot)                                                              \
    do {                                                                                        \
        if (args.trace && blockIdx.x == 0 && blockIdx.y == 0 && (j) < 40)                       \
            args.trace[((role) * 40 + (j)) * 8 + (slot)] = clock64();                           \
    } while (0)
#else
#define FUSED_TRACE(role, j, slot) do { } while (0)
#endif

// key tiles of 128 while S_0 S_1 | P_0 P_1 | O_0 O_1 fit the 512 tensor-memory columns, else of 64
__host__ inline int fused_block_n(int d) { return ((d + 15) / 16 * 16) <= 64 ? 128 : 64; }

__host__ inline void fused_fill_args(FusedArgs* a, __half* out, int Nq, int Nk, int d, float scale_log2e, bool negate,
                                     int* status) {
    a->out = out;
    a->Nq = Nq; a->Nk = Nk; a->d = d;
    a->dpad = (d + 15) / 16 * 16;
    a->nch = (d + CHUNK_COLS - 1) / CHUNK_COLS;
    const int bn = fused_block_n(d);
    const int q_bytes = 2 * a->nch * TILE_M * CHUNK_ROW_BYTES;
    const int stage_bytes = 2 * a->nch * bn * CHUNK_ROW_BYTES;
    int stages = (FUSED_SMEM_BUDGET - q_bytes) / stage_bytes;
    if (stages > FUSED_MAX_STAGES) stages = FUSED_MAX_STAGES;
    a->stages = stages;
    a->scale_log2e = scale_log2e;
    a->negate = negate ? 1 : 0;
    a->status = status;
    a->tiles_per_cta = 2;
}

__host__ inline size_t fused_smem_bytes(const FusedArgs& a) {
    const int bn = fused_block_n(a.d);
    return (size_t)2 * a.nch * TILE_M * CHUNK_ROW_BYTES + (size_t)a.stages * 2 * a.nch * bn * CHUNK_ROW_BYTES + 1024;
}
__host__ inline size_t fused_smem_bytes_max() { return FUSED_SMEM_BUDGET + 1024; }

enum {
    SITE_F_Q = 10, SITE_F_KV = 11, SITE_F_EMPTY = 13, SITE_F_S = 14, SITE_F_P = 15, SITE_F_O = 16,
    SITE_F_SFREE = 17, SITE_F_PFREE = 18
};

template <int BN>
__global__ void __launch_bounds__(FUSED_THREADS, 1)
fused_attention_kernel(const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_k,
                       const __grid_constant__ CUtensorMap tmap_v, const FusedArgs args) {
    extern __shared__ uint8_t fused_smem_raw[];
    // per query tile: Q landed | S ready (MMA) | S consumed (softmax) | P ready (softmax) | P V done (MMA)
    __shared__ __align__(8) uint64_t bar_q_full[2], bar_s_full[2], bar_s_free[2], bar_p_full[2], bar_pv_done[2];
    __shared__ __align__(8) uint64_t bar_kv_full[FUSED_MAX_STAGES], bar_kv_empty[FUSED_MAX_STAGES];
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int bh = blockIdx.y;
    const int row_base = blockIdx.x * args.tiles_per_cta * TILE_M;
    const int n_qtiles = (args.tiles_per_cta == 2 && row_base + TILE_M < args.Nq) ? 2 : 1;
    const int n_kv = (args.Nk + BN - 1) / BN;
    const int nch = args.nch, dpad = args.dpad, stages = args.stages;

    const uint32_t smem_base = (smem_u32(fused_smem_raw) + 1023u) & ~1023u;
    const uint32_t q_tile_bytes = nch * TILE_M * CHUNK_ROW_BYTES;
    const uint32_t kv_tile_bytes = nch * BN * CHUNK_ROW_BYTES;
    const uint32_t q_smem = smem_base;                       // [2][nch][128 rows][128 B]
    const uint32_t kv_smem = q_smem + 2 * q_tile_bytes;      // [stages][K | V][nch][BN rows][128 B]
    volatile int* abort_p = &abort_flag;

    if (tid == 0) {
        abort_flag = 0;
        for (int t = 0; t < 2; ++t) {
            mbar_init(smem_u32(&bar_q_full[t]), 1);
            mbar_init(smem_u32(&bar_s_full[t]), 1);
            mbar_init(smem_u32(&bar_s_free[t]), 4);    // one arrival per softmax warp
            mbar_init(smem_u32(&bar_p_full[t]), 4);
            mbar_init(smem_u32(&bar_pv_done[t]), 1);
        }
        for (int s = 0; s < FUSED_MAX_STAGES; ++s) {
            mbar_init(smem_u32(&bar_kv_full[s]), 1);
            mbar_init(smem_u32(&bar_kv_empty[s]), n_qtiles);   // one commit per issuer
        }
        mbar_init_fence();
    }
    if (warp == 9) {
        tmem_alloc(smem_u32(&tmem_base_slot), 512);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = tmem_base_slot;
    // columns: S_0 | S_1 | P_0 | P_1 | O_0 | O_1
    const uint32_t tmem_p0 = tmem_base + 2 * BN;
    constexpr uint32_t tmem_p_stride = BN / 2;
    const uint32_t tmem_o0 = tmem_base + 3 * BN;

    if (warp == 8) {
        // ------------------------------------------------------------ TMA producer
        if (elect_one()) {
            tma_prefetch_desc(&tmap_q);
            tma_prefetch_desc(&tmap_k);
            tma_prefetch_desc(&tmap_v);
            for (int t = 0; t < n_qtiles; ++t) {
                const uint32_t bar = smem_u32(&bar_q_full[t]);
                mbar_arrive_expect_tx(bar, q_tile_bytes);
                for (int ch = 0; ch < nch; ++ch)
                    tma_load_4d(q_smem + t * q_tile_bytes + ch * TILE_M * CHUNK_ROW_BYTES, &tmap_q, bar,
                                ch * CHUNK_COLS, row_base + t * TILE_M, bh, 0);
            }
            for (int j = 0; j < n_kv; ++j) {
                const int s = j % stages;
                if (j >= stages &&
                    !mbar_wait(smem_u32(&bar_kv_empty[s]), ((j / stages) - 1) & 1, abort_p, args.status, SITE_F_EMPTY, j))
                    break;
                const uint32_t k_dst = kv_smem + s * 2 * kv_tile_bytes, v_dst = k_dst + kv_tile_bytes;
                const uint32_t bar = smem_u32(&bar_kv_full[s]);
                mbar_arrive_expect_tx(bar, 2 * kv_tile_bytes);
                for (int ch = 0; ch < nch; ++ch)
                    tma_load_4d(k_dst + ch * BN * CHUNK_ROW_BYTES, &tmap_k, bar, ch * CHUNK_COLS, j * BN, bh, 0);
                for (int ch = 0; ch < nch; ++ch)
                    tma_load_4d(v_dst + ch * BN * CHUNK_ROW_BYTES, &tmap_v, bar, ch * CHUNK_COLS, j * BN, bh, 0);
            }
        }
    } else if (warp >= 9) {
        // ------------------------------------------------------------ MMA issuer of query tile t
        const int t = warp - 9;
        if (t < n_qtiles && elect_one()) {
            const uint32_t idesc_s = idesc_f16(TILE_M, BN, false, false, args.negate != 0);
            const uint32_t idesc_o = idesc_f16(TILE_M, dpad, false, true, false);
            const int ksteps_s = (args.d + 15) / 16;
            // descriptors differ only in their low word (the start address >> 4): precompute the offsets
            const uint64_t q_desc = smem_desc_sw128(q_smem + t * q_tile_bytes, 16, 1024);
            const uint64_t k_desc = smem_desc_sw128(kv_smem, 16, 1024);
            const uint64_t v_desc = smem_desc_sw128(kv_smem + kv_tile_bytes, BN * CHUNK_ROW_BYTES, 1024);
            uint32_t q_off[FUSED_MAX_KSTEPS], k_off[FUSED_MAX_KSTEPS];
#pragma unroll
            for (int kk = 0; kk < FUSED_MAX_KSTEPS; ++kk) {
                q_off[kk] = ((kk >> 2) * TILE_M * CHUNK_ROW_BYTES + (kk & 3) * 32) >> 4;
                k_off[kk] = ((kk >> 2) * BN * CHUNK_ROW_BYTES + (kk & 3) * 32) >> 4;
            }
            const uint32_t stage_off = (2 * kv_tile_bytes) >> 4;
            const uint32_t tmem_s = tmem_base + t * BN;
            const uint32_t tmem_p = tmem_p0 + t * tmem_p_stride;
            const uint32_t tmem_o = tmem_o0 + t * dpad;
            const uint32_t b_sfull = smem_u32(&bar_s_full[t]), b_sfree = smem_u32(&bar_s_free[t]);
            const uint32_t b_pfull = smem_u32(&bar_p_full[t]), b_pvdone = smem_u32(&bar_pv_done[t]);

            auto issue_s = [&](int s) {   // S_t = Q_t K_s^T
                const uint64_t kd = k_desc + (uint64_t)(s * stage_off);
#pragma unroll
                for (int kk = 0; kk < FUSED_MAX_KSTEPS; ++kk)
                    if (kk < ksteps_s) mma_f16_ss(tmem_s, q_desc + q_off[kk], kd + k_off[kk], idesc_s, kk > 0);
                tc_commit(b_sfull);
            };
            auto issue_o = [&](int s, bool accumulate) {   // O_t (+)= P_t V_s
                const uint64_t vd = v_desc + (uint64_t)(s * stage_off);
#pragma unroll
                for (int kk = 0; kk < BN / 16; ++kk)
                    mma_f16_ts(tmem_o, tmem_p + kk * 8, vd + (uint64_t)(kk * ((16 * CHUNK_ROW_BYTES) >> 4)), idesc_o,
                               accumulate || kk > 0);
            };

            bool ok = mbar_wait(smem_u32(&bar_q_full[t]), 0, abort_p, args.status, SITE_F_Q, t) &&
                      mbar_wait(smem_u32(&bar_kv_full[0]), 0, abort_p, args.status, SITE_F_KV, 0);
            if (ok) {
                tc_fence_after_sync();
                issue_s(0);
            }
            for (int j = 0; j < n_kv && ok; ++j) {
                const int s = j % stages;
                const int s1 = (j + 1) % stages;
                FUSED_TRACE(2 + t, j, 0);
                if (j + 1 < n_kv)   // the next K/V tile landed long ago: take this wait off the critical path
                    ok = mbar_wait(smem_u32(&bar_kv_full[s1]), ((j + 1) / stages) & 1, abort_p, args.status, SITE_F_KV, j + 1);
                if (ok && j + 1 < n_kv) {
                    // S_t is free once its row sits in the softmax registers: start tile j+1 right away
                    ok = mbar_wait(b_sfree, j & 1, abort_p, args.status, SITE_F_SFREE, j);
                    if (!ok) break;
                    tc_fence_after_sync();
                    FUSED_TRACE(2 + t, j, 1);
                    issue_s(s1);
                    FUSED_TRACE(2 + t, j, 2);
                }
                if (ok) ok = mbar_wait(b_pfull, j & 1, abort_p, args.status, SITE_F_P, j);
                if (!ok) break;
                tc_fence_after_sync();
                FUSED_TRACE(2 + t, j, 3);
                issue_o(s, j > 0);
                tc_commit(b_pvdone);                          // O_t holds tiles 0..j; P_t may be rewritten
                tc_commit(smem_u32(&bar_kv_empty[s]));        // this issuer is done with K_j and V_j
                FUSED_TRACE(2 + t, j, 4);
            }
        }
    } else {
        // ------------------------------------------------------------ softmax warps
        const int t = warp >> 2;                 // query tile of this warpgroup
        if (t < n_qtiles) {
            const int r = tid & (TILE_M - 1);    // row inside the tile = TMEM lane
            const uint32_t lane_off = (uint32_t)((warp & 3) * 32) << 16;
            const uint32_t tmem_s = tmem_base + t * BN + lane_off;
            const uint32_t tmem_p = tmem_p0 + t * tmem_p_stride + lane_off;
            const uint32_t tmem_o = tmem_o0 + t * dpad + lane_off;
            const uint32_t b_sfull = smem_u32(&bar_s_full[t]), b_sfree = smem_u32(&bar_s_free[t]);
            const uint32_t b_pfull = smem_u32(&bar_p_full[t]), b_pvdone = smem_u32(&bar_pv_done[t]);
            const bool tracer = (warp & 3) == 0 && lane == 0;
            const float c2 = args.scale_log2e;
            float m_run = -INFINITY;  // anchor of the exponent: a bound on the running max, times scale*log2(e)
            float l_run = 0.f;        // running sum of p (relative to m_run)
            bool ok = true;
            for (int j = 0; j < n_kv; ++j) {
                if (tracer) FUSED_TRACE(t, j, 0);
                ok = mbar_wait(b_sfull, j & 1, abort_p, args.status, SITE_F_S, j);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                tc_fence_after_sync();
                if (tracer) FUSED_TRACE(t, j, 1);
                const int valid = args.Nk - j * BN;   // columns >= valid are zero-filled keys
                // the whole row of S_t into registers with one wait, then hand S_t back
                uint32_t s[BN];
#pragma unroll
                for (int g = 0; g < BN / 32; ++g) tmem_ld32(tmem_s + g * 32, &s[g * 32]);
                tmem_wait_ld();
                tc_fence_before_sync();
                if (lane == 0) mbar_arrive(b_sfree);
                if (tracer) FUSED_TRACE(t, j, 2);
                const bool ragged = valid < BN;   // only the last key tile can be
                const float row_max = row_max_masked<BN>(s, ragged ? valid : BN);   // exact: it decides the anchor alone
                const float row_max2 = row_max * c2;   // in log2 units, as the exponent sees it
                if (j == 0) {
                    m_run = row_max2 + FUSED_HEADROOM_LOG2;
                } else {
                    // P_t and O_t belong to the tensor pipe until the P V product of tile j-1 has completed
                    ok = mbar_wait(b_pvdone, (j - 1) & 1, abort_p, args.status, SITE_F_PFREE, j);
                    ok = __all_sync(0xffffffffu, ok);
                    if (!ok) break;
                    tc_fence_after_sync();
                    const bool grow = row_max2 - m_run > FUSED_RESCALE_LOG2;
                    if (__any_sync(0xffffffffu, grow)) {
                        const float m_new = row_max2 + FUSED_HEADROOM_LOG2;
                        const float alpha = grow ? ex2_approx(m_run - m_new) : 1.f;
                        if (grow) m_run = m_new;
                        l_run *= alpha;
                        for (int g = 0; g < (dpad >> 4); ++g) {
                            uint32_t x[16];
                            tmem_ld16(tmem_o + g * 16, x);
                            tmem_wait_ld();
#pragma unroll
                            for (int c = 0; c < 16; ++c) x[c] = __float_as_uint(__uint_as_float(x[c]) * alpha);
                            tmem_st16(tmem_o + g * 16, x);
                        }
                    }
                }
                const float neg_mc = -m_run;
                if (tracer) FUSED_TRACE(t, j, 3);
                if (!ragged) {
                    const uint64_t c2c2 = pack_b64(__float_as_uint(c2), __float_as_uint(c2));
                    const uint64_t nmnm = pack_b64(__float_as_uint(neg_mc), __float_as_uint(neg_mc));
                    uint64_t acc[2] = {0ull, 0ull};
#pragma unroll
                    for (int g = 0; g < BN / 32; ++g) {
                        uint32_t packed[16];
                        exp2_pack_32<FUSED_POLY_PER8>(&s[g * 32], c2c2, nmnm, packed, acc);
                        tmem_st16(tmem_p + g * 16, packed);
                    }
                    l_run += sum_f32x2(acc[0], acc[1]);
                } else {
                    float sum = 0.f;
#pragma unroll
                    for (int g = 0; g < BN / 32; ++g) {
                        uint32_t packed[16];
                        exp2_pack_32_masked(&s[g * 32], c2, neg_mc, g * 32, valid, packed, sum);
                        tmem_st16(tmem_p + g * 16, packed);
                    }
                    l_run += sum;
                }
                if (tracer) FUSED_TRACE(t, j, 4);
                tmem_wait_st();
                tc_fence_before_sync();
                if (lane == 0) mbar_arrive(b_pfull);
                if (tracer) FUSED_TRACE(t, j, 5);
            }
            if (ok) ok = mbar_wait(b_pvdone, (n_kv - 1) & 1, abort_p, args.status, SITE_F_O, t);
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
    if (warp == 8 && lane == 0 && abort_flag) {
        // gave up somewhere: give copies still in flight a bounded chance to land
        for (int s = 0; s < stages; ++s) mbar_drain(smem_u32(&bar_kv_full[s]), 0);
    }
    __syncthreads();
    if (warp == 9) {
        __syncwarp();
        tmem_dealloc(tmem_base, 512);
    }
}

}  // namespace sd_attn
