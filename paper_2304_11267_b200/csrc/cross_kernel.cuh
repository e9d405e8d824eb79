// Cross-attention kernel: every key of a (batch, head) fits ONE shared-memory tile (Nk <= 128,
// the 77 text tokens of Stable Diffusion), so the softmax of Eq. 3 needs no running rescale: the
// row maximum L and the sum S of Eq. 4 come from a single pass over the 128 x Nk score tile.
//
// One CTA (4 warps) per tile of 128 query rows:
//   TMA: Q tile, K, V  ->  128-byte-swizzled shared memory (columns beyond d and rows beyond Nk
//        are zero-filled by the copy engine, so padding costs no HBM bytes)
//   tcgen05.mma  S = Q K^T          (fp16 x fp16 -> fp32 in tensor memory, N = Nk rounded to 16)
//   softmax      one thread per query row: read its row of S, max, exp2, sum; the unnormalised
//                weights go back to tensor memory as packed fp16 over the columns S occupied
//   tcgen05.mma  O = P V            (P from tensor memory, V as an N-major shared-memory operand)
//   epilogue     O / S_i -> fp16 -> global
// Several CTAs are resident per SM, so one tile's loads overlap another's arithmetic.
#pragma once
#include <cuda.h>

#include "tc_common.cuh"

namespace sd_attn {

constexpr int CROSS_THREADS = 128;
constexpr int TILE_M = 128;          // query rows per tile = TMEM lanes
constexpr int CHUNK_COLS = 64;       // fp16 elements per 128-byte swizzled row
constexpr int CHUNK_ROW_BYTES = 128;

struct CrossArgs {
    __half* out;        // [BH][Nq][d], or as `lay` says
    HeadLayout lay;
    int Nq, Nk, d;
    int kn;             // Nk rounded up to a multiple of 16 (the MMA N of S, the K of P.V)
    int dpad;           // d rounded up to a multiple of 16 (the MMA N of O)
    int nch;            // 64-column chunks per row: ceil(d / 64)
    int tmem_cols;      // power of two >= kn + dpad
    float scale_log2e;  // |scale| * log2(e)
    int negate;         // scale < 0: the MMA negates Q instead
    int* status;        // device status block
};

__host__ inline size_t cross_smem_bytes(int nch, int kn) {
    return (size_t)nch * (TILE_M + 2 * kn) * CHUNK_ROW_BYTES + 1024;  // + slack for 1024-byte alignment
}

enum { SITE_X_LOAD_QK = 1, SITE_X_LOAD_V = 2, SITE_X_S = 3, SITE_X_O = 4 };

template <bool BF = false>   // BF: bfloat16 tensors
__global__ void __launch_bounds__(CROSS_THREADS)
cross_attention_kernel(const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_k,
                       const __grid_constant__ CUtensorMap tmap_v, const CrossArgs args) {
    extern __shared__ uint8_t cross_smem_raw[];
    __shared__ __align__(8) uint64_t bars[4];  // 0: Q+K landed, 1: V landed, 2: S ready, 3: O ready
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;

    const int tid = threadIdx.x, warp = tid >> 5;
    if (threadIdx.x == 0) pdl_launch_dependents();   // the next kernel of the stream may start its set-up
    const int tile = blockIdx.x, bh = blockIdx.y;
    const int row0 = tile * TILE_M;
    const int kn = args.kn, nch = args.nch, dpad = args.dpad;

    const uint32_t smem_base = (smem_u32(cross_smem_raw) + 1023u) & ~1023u;
    const uint32_t q_smem = smem_base;
    const uint32_t k_smem = q_smem + nch * TILE_M * CHUNK_ROW_BYTES;
    const uint32_t v_smem = k_smem + nch * kn * CHUNK_ROW_BYTES;
    const uint32_t bar_qk = smem_u32(&bars[0]), bar_v = smem_u32(&bars[1]);
    const uint32_t bar_s = smem_u32(&bars[2]), bar_o = smem_u32(&bars[3]);

    if (tid == 0) {
        abort_flag = 0;
        mbar_init(bar_qk, 1);
        mbar_init(bar_v, 1);
        mbar_init(bar_s, 1);
        mbar_init(bar_o, 1);
        mbar_init_fence();
        tma_prefetch_desc(&tmap_q);
        tma_prefetch_desc(&tmap_k);
        tma_prefetch_desc(&tmap_v);
    }
    if (warp == 0) {
        tmem_alloc(smem_u32(&tmem_base_slot), (uint32_t)args.tmem_cols);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    // Set-up (barriers, tensor memory) overlapped the tail of the previous kernel of the stream; global memory and
    // every bounded wait come after it has completed.
    pdl_wait();
    const uint32_t tmem_base = tmem_base_slot;
    const uint32_t tmem_s = tmem_base;          // S: kn fp32 columns; P (packed fp16) reuses them
    const uint32_t tmem_o = tmem_base + kn;     // O: dpad fp32 columns
    volatile int* abort_p = &abort_flag;
    bool ok = true;

    if (tid == 0) {
        const int bz = bh / args.lay.heads, hz = bh - bz * args.lay.heads;
        mbar_arrive_expect_tx(bar_qk, (uint32_t)(nch * (TILE_M + kn) * CHUNK_ROW_BYTES));
        for (int ch = 0; ch < nch; ++ch)
            tma_load_4d(q_smem + ch * TILE_M * CHUNK_ROW_BYTES, &tmap_q, bar_qk, ch * CHUNK_COLS, row0, hz, bz);
        for (int ch = 0; ch < nch; ++ch)
            tma_load_4d(k_smem + ch * kn * CHUNK_ROW_BYTES, &tmap_k, bar_qk, ch * CHUNK_COLS, 0, hz, bz);
        mbar_arrive_expect_tx(bar_v, (uint32_t)(nch * kn * CHUNK_ROW_BYTES));
        for (int ch = 0; ch < nch; ++ch)
            tma_load_4d(v_smem + ch * kn * CHUNK_ROW_BYTES, &tmap_v, bar_v, ch * CHUNK_COLS, 0, hz, bz);

        // S = Q K^T: contraction over d in steps of 16 columns (32 bytes inside a swizzled row)
        if (mbar_wait(bar_qk, 0, abort_p, args.status, SITE_X_LOAD_QK, tile)) {
            tc_fence_after_sync();
            const uint32_t idesc = idesc_f16(TILE_M, kn, false, false, args.negate != 0, BF);
            const int ksteps = (args.d + 15) / 16;
            for (int kk = 0; kk < ksteps; ++kk) {
                const int ch = kk >> 2, within = (kk & 3) * 32;
                const uint64_t a_desc = smem_desc_sw128(q_smem + ch * TILE_M * CHUNK_ROW_BYTES + within, 16, 1024);
                const uint64_t b_desc = smem_desc_sw128(k_smem + ch * kn * CHUNK_ROW_BYTES + within, 16, 1024);
                mma_f16_ss(tmem_s, a_desc, b_desc, idesc, kk > 0);
            }
            tc_commit(bar_s);
        }
    }

    // ---- softmax: thread = query row = TMEM lane
    ok = mbar_wait(bar_s, 0, abort_p, args.status, SITE_X_S, tile);
    ok = __all_sync(0xffffffffu, ok);
    const uint32_t lane_off = (uint32_t)(warp * 32) << 16;
    float row_sum = 0.f;
    if (ok) {
        tc_fence_after_sync();
        const int groups = kn >> 4;
        float row_max = -INFINITY;
        for (int g = 0; g < groups; ++g) {
            uint32_t r[16];
            tmem_ld16(tmem_s + lane_off + g * 16, r);
            tmem_wait_ld();
#pragma unroll
            for (int c = 0; c < 16; ++c)
                if (g * 16 + c < args.Nk) row_max = fmaxf(row_max, __uint_as_float(r[c]));
        }
        const float c2 = args.scale_log2e;
        const float neg_mc = -row_max * c2;
        for (int g = 0; g < groups; ++g) {
            uint32_t r[16], packed[8];
            tmem_ld16(tmem_s + lane_off + g * 16, r);
            tmem_wait_ld();
            float p[16];
#pragma unroll
            for (int c = 0; c < 16; ++c) {
                const float e = ex2_approx(fmaf(__uint_as_float(r[c]), c2, neg_mc));
                p[c] = (g * 16 + c < args.Nk) ? e : 0.f;   // zero-filled key rows carry no weight
                row_sum += p[c];
            }
#pragma unroll
            for (int c = 0; c < 8; ++c) packed[c] = pack_16x2<BF>(p[2 * c], p[2 * c + 1]);
            tmem_st8(tmem_s + lane_off + g * 8, packed);    // overwrites columns already consumed
        }
        tmem_wait_st();
    }
    tc_fence_before_sync();
    __syncthreads();

    // ---- O = P V: contraction over keys in steps of 16 rows (two 8-row swizzle groups)
    if (tid == 0 && ok) {
        if (mbar_wait(bar_v, 0, abort_p, args.status, SITE_X_LOAD_V, tile)) {
            tc_fence_after_sync();
            const uint32_t idesc = idesc_f16(TILE_M, dpad, false, true, false, BF);
            for (int kk = 0; kk < (kn >> 4); ++kk) {
                const uint64_t b_desc = smem_desc_sw128(v_smem + kk * 16 * CHUNK_ROW_BYTES,
                                                        (uint32_t)(kn * CHUNK_ROW_BYTES), 1024);
                mma_f16_ts(tmem_o, tmem_s + kk * 8, b_desc, idesc, kk > 0);
            }
            tc_commit(bar_o);
        }
    }

    // ---- epilogue
    if (ok) ok = mbar_wait(bar_o, 0, abort_p, args.status, SITE_X_O, tile);
    ok = __all_sync(0xffffffffu, ok);
    if (ok) {
        tc_fence_after_sync();
        const float inv = 1.f / row_sum;
        const int row = row0 + tid;
        __half* orow = head_row(args.out, args.lay, bh, row);
        for (int g = 0; g < (dpad >> 4); ++g) {
            uint32_t r[16];
            tmem_ld16(tmem_o + lane_off + g * 16, r);
            tmem_wait_ld();
            uint4 lo, hi;
            lo.x = pack_16x2<BF>(__uint_as_float(r[0]) * inv, __uint_as_float(r[1]) * inv);
            lo.y = pack_16x2<BF>(__uint_as_float(r[2]) * inv, __uint_as_float(r[3]) * inv);
            lo.z = pack_16x2<BF>(__uint_as_float(r[4]) * inv, __uint_as_float(r[5]) * inv);
            lo.w = pack_16x2<BF>(__uint_as_float(r[6]) * inv, __uint_as_float(r[7]) * inv);
            hi.x = pack_16x2<BF>(__uint_as_float(r[8]) * inv, __uint_as_float(r[9]) * inv);
            hi.y = pack_16x2<BF>(__uint_as_float(r[10]) * inv, __uint_as_float(r[11]) * inv);
            hi.z = pack_16x2<BF>(__uint_as_float(r[12]) * inv, __uint_as_float(r[13]) * inv);
            hi.w = pack_16x2<BF>(__uint_as_float(r[14]) * inv, __uint_as_float(r[15]) * inv);
            if (row < args.Nq) {
                if (g * 16 + 8 <= args.d) *reinterpret_cast<uint4*>(orow + g * 16) = lo;
                if (g * 16 + 16 <= args.d) *reinterpret_cast<uint4*>(orow + g * 16 + 8) = hi;
            }
        }
    } else if (tid == 0) {
        // gave up: let the copies that may still be in flight land before shared memory is released
        mbar_drain(bar_qk, 0);
        mbar_drain(bar_v, 0);
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem_base, (uint32_t)args.tmem_cols);
}

}  // namespace sd_attn
