// Persistent cross-attention kernel for the text-conditioning shape of the UNet: 65..80 keys (the 77
// text tokens), any head dim up to 160.  Memory-bound: per tile of 128 query rows it reads Q and writes O
// once; K and V (12-50 KB per head) stay in L2.
//
// cross_kernel.cuh runs one tile per CTA, start to finish, and leans on CTA-level overlap; its launch,
// tensor-memory allocation, descriptor fetch and drain are paid per tile and HBM sits idle meanwhile.
// Here ONE CTA per SM walks a contiguous range of (head, tile) items with every stage overlapped:
//   warps 0 .. 4*NWG-1   NWG softmax groups; group w owns items w, w+NWG, ... (thread = query row): exp2, row sum,
//                        weights back to tensor memory, 1 / row sum to shared memory -- and on to its next item
//   next 4 warps         the epilogue warpgroup: for every item in turn, O_w / row sum -> fp16 -> global.  (With the
//                        softmax warps doing their own epilogue a group spent a third of an item waiting for the
//                        P V product and writing out, and four groups did not hide it.)
//   next warp            producer: the Q tile of item i into ring stage i % NS (several in flight); K and V
//                        of a head once per head, double-buffered.  (The copy engine spends about 7 clocks per
//                        80-byte row of a d = 40 tensor, measured, so fetching K and V per item -- 160 more rows --
//                        would make it the bound.  A single warp of 128-bit cp.async copies for Q measured slower.)
//   two more warps       MMA issuers: one thread issues S_w = Q K^T as soon as a stage lands, another O_w = P_w V
//                        when the weights are ready
// Q at head dims up to 48 (four groups): a tiled TMA load of 128 rows of 80 bytes keeps the copy engine busy for
// 900-1300 clocks, which became the bound of the kernel once the softmax no longer was.  The tile is 10 KB of
// CONTIGUOUS global memory, so it is fetched with one untiled bulk copy into a raw ring stage instead, and the softmax
// group that will use it rewrites it (thread = row: five 16-byte loads, six swizzled 16-byte stores, columns 40..47
// zeroed) into its own MMA-layout buffer while it waits for tensor-core work anyway.
// Tensor memory: per group S_w (80 columns; the packed fp16 weights overwrite the first 40) and O_w
// (dpad columns), so NWG = 512 / (80 + dpad) capped at 4: four groups at d = 40, three at 80, two at 160.
// No running rescale is needed: all keys of a row are in the tile.  The exponent is anchored X2_HEADROOM_LOG2 above
// the score of the row's FIRST key instead of the row maximum (any anchor gives the same weights in exact
// arithmetic); only if the weights of a row then sum to more than X2_SUM_LIMIT -- its maximum lies far above its
// first score: rare -- does the warp take the true maximum and redo the row.  That keeps the maximum off the path
// and lets a row be processed in two pieces (48 + 32 columns) with half the registers.
#pragma once
#include <cuda.h>

#include "cross_kernel.cuh"  // TILE_M, CHUNK_COLS, CHUNK_ROW_BYTES
#include "softmax_math.cuh"
#include "tc_common.cuh"

namespace sd_attn {

constexpr int X2_KN = 80;            // keys rounded up to the MMA N granule; the kernel serves 65..80 keys
constexpr int X2_MAX_STAGES = 8;
constexpr int X2_MAX_KSTEPS = 10;
constexpr int X2_SMEM_BUDGET = 216 * 1024;
// four-group variant, after setmaxnreg: 512 * 96 + 128 * 64 + 128 * 32 = 61440 = 768 * 80, the launch allocation
constexpr int X2_SOFTMAX_REGS = 96;
constexpr int X2_EPILOGUE_REGS = 64;
constexpr int X2_CONTROL_REGS = 32;
constexpr float X2_HEADROOM_LOG2 = 8.0f;   // weights of the first key: 2^-8
constexpr float X2_SUM_LIMIT = 4096.0f;    // no weight above 2^12 reaches the binary16 pack

constexpr int X2_GROUP_MAX = 5;      // problems of one shape per launch (the parameter block stays under 4 KB)

struct Cross2Problem {   // one problem of a launch
    CUtensorMap tq, tk, tv;          // swizzled tiles of 64 columns
    CUtensorMap tq_rows, tout_rows;  // four-group variant with strided rows: unswizzled tiles of d columns
    const __half* q;    // [BH][Nq][d]: the four-group variant fetches Q tiles with untiled bulk copies
    __half* out;        // [BH][Nq][d], or as Cross2Args::lay says
    float scale_log2e;  // |scale| * log2(e)
    int negate;         // scale < 0: the tensor core negates Q
};

template <int NP>   // NP = 1: a launch of one problem (the problem index folds away at compile time); else X2_GROUP_MAX
struct Cross2ArgsT {
    Cross2Problem prob[NP];
    int n_prob, BH;     // problems in this launch; (batch, head) pairs of each.  Heads are counted through all
                        // problems ("global head" = problem * BH + head), items through all global heads
    HeadLayout lay;
    int Nq, Nk, d;
    int dpad, nch;
    int strided_rows;   // four-group variant: a tile's rows are not one contiguous run (token-major tensors): Q and the
                        // output move as unswizzled tiles of d columns through tmap_q_rows / tmap_out_rows
    int stages;         // depth of the Q ring
    int tiles_per_bh;   // ceil(Nq / 128)
    int n_items;        // n_prob * BH * tiles_per_bh
    int* status;
};
using Cross2Args = Cross2ArgsT<X2_GROUP_MAX>;


__host__ inline int cross2_groups(int d) {
    const int g = 512 / (X2_KN + (d + 15) / 16 * 16);
    return g > 4 ? 4 : g;
}
__host__ inline int cross2_threads(int groups) { return groups * 128 + 256; }   // + epilogue and control warpgroups
__host__ inline int cross2_q_bytes(int nch) { return nch * TILE_M * CHUNK_ROW_BYTES; }
__host__ inline int cross2_kv_bytes(int nch) { return nch * X2_KN * CHUNK_ROW_BYTES; }
// shared memory: [2 head buffers][K | V] then the Q ring
__host__ inline int cross2_stages(int nch) {
    int s = (X2_SMEM_BUDGET - 4 * cross2_kv_bytes(nch)) / cross2_q_bytes(nch);
    return s > X2_MAX_STAGES ? X2_MAX_STAGES : s;
}
__host__ inline size_t cross2_smem_bytes(int nch) {
    return (size_t)4 * cross2_kv_bytes(nch) + (size_t)cross2_stages(nch) * cross2_q_bytes(nch) + 1024;
}
// four-group variant (d <= 48): [2 head buffers][K | V], four MMA-layout Q buffers, then the ring of raw Q tiles
__host__ inline int cross2_raw_bytes(int d) { return (TILE_M * d * 2 + 127) & ~127; }
__host__ inline int cross2_dense_stages(int d) {   // a multiple of 4: a stage then always serves the same group
    int s = (X2_SMEM_BUDGET - 4 * cross2_kv_bytes(1) - 4 * cross2_q_bytes(1)) / cross2_raw_bytes(d) - 2;
    s = s > X2_MAX_STAGES ? X2_MAX_STAGES : s;
    return s / 4 * 4;
}
__host__ inline size_t cross2_dense_smem_bytes(int d) {   // ... and two output staging tiles of the raw size
    return (size_t)4 * cross2_kv_bytes(1) + (size_t)4 * cross2_q_bytes(1) +
           (size_t)(cross2_dense_stages(d) + 2) * cross2_raw_bytes(d) + 1024;
}
__host__ inline bool cross2_supports(int Nk, int d) { return Nk > 64 && Nk <= X2_KN && d % 8 == 0 && d <= 160; }

enum {
    SITE_Y_STAGE = 40, SITE_Y_EMPTY = 41, SITE_Y_S = 42, SITE_Y_P = 43, SITE_Y_O = 44, SITE_Y_OFREE = 45,
    SITE_Y_KV = 46, SITE_Y_KVEMPTY = 47, SITE_Y_PV = 48
};

// S = Q K^T over KS contraction steps of 16 columns, offsets folded at compile time.
template <int KS>
__device__ __forceinline__ void issue_qk(uint32_t tmem_s, uint64_t q_desc, uint64_t k_desc, uint32_t idesc) {
#pragma unroll
    for (int kk = 0; kk < KS; ++kk)
        mma_f16_ss(tmem_s, q_desc + (uint64_t)(((kk >> 2) * TILE_M * CHUNK_ROW_BYTES + (kk & 3) * 32) >> 4),
                   k_desc + (uint64_t)(((kk >> 2) * X2_KN * CHUNK_ROW_BYTES + (kk & 3) * 32) >> 4), idesc, kk > 0);
}

template <int NWG, bool BF = false, int NP = X2_GROUP_MAX>   // BF: bfloat16 tensors; NP: see Cross2ArgsT
__global__ void __launch_bounds__(NWG * 128 + 256, 1)
cross2_attention_kernel(const __grid_constant__ Cross2ArgsT<NP> args) {
    constexpr bool GROUPED = NP > 1;
    extern __shared__ uint8_t x2_smem_raw[];
    __shared__ __align__(8) uint64_t bar_full[X2_MAX_STAGES], bar_empty[X2_MAX_STAGES];
    __shared__ __align__(8) uint64_t bar_kv_full[2], bar_kv_empty[2];
    __shared__ __align__(8) uint64_t bar_s_full[NWG], bar_p_full[NWG], bar_o_full[NWG], bar_o_free[NWG], bar_pv_done[NWG];
    __shared__ __align__(8) uint64_t bar_q_ready[NWG];   // four-group variant: the group's MMA-layout Q buffer is written
    __shared__ float inv_sum[NWG][2][TILE_M];   // 1 / row sum of the group's current and previous item
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;

    constexpr int EPILOGUE_WARP0 = NWG * 4;
    constexpr int LOADER_WARP = NWG * 4 + 4, S_ISSUER_WARP = NWG * 4 + 5, O_ISSUER_WARP = NWG * 4 + 6;
    constexpr int S2_ISSUER_WARP = NWG * 4 + 7;   // second S issuer: the odd items
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (threadIdx.x == 0) pdl_launch_dependents();   // the next kernel of the stream may start its set-up
    if (!GROUPED && threadIdx.x == 32) {   // the tensor maps are kernel parameters: their fetch need not wait for anything
        tma_prefetch_desc(&args.prob[0].tq);
        tma_prefetch_desc(&args.prob[0].tk);
        tma_prefetch_desc(&args.prob[0].tv);
        if (NWG == 4 && args.strided_rows) {
            tma_prefetch_desc(&args.prob[0].tq_rows);
            tma_prefetch_desc(&args.prob[0].tout_rows);
        }
    }
    const int nch = args.nch, dpad = args.dpad, stages = args.stages;
    // contiguous range of items for this CTA: consecutive items share a head, so K and V are fetched rarely
    const int per = args.n_items / gridDim.x, extra = args.n_items % gridDim.x;
    const int item0 = blockIdx.x * per + min((int)blockIdx.x, extra);
    const int n_local = per + ((int)blockIdx.x < extra ? 1 : 0);
    const int bh0 = item0 / args.tiles_per_bh;   // global head of the first item; head "group" g = global head - bh0
    const int prob0 = GROUPED ? bh0 / args.BH : 0, hb0 = bh0 - prob0 * args.BH;   // its problem and its head inside that problem
    if (GROUPED && threadIdx.x == 32 && n_local > 0) {   // (several problems: the maps of the CTA's first one)
        const Cross2Problem& p0 = args.prob[prob0];
        tma_prefetch_desc(&p0.tq);
        tma_prefetch_desc(&p0.tk);
        tma_prefetch_desc(&p0.tv);
        if (NWG == 4 && args.strided_rows) {
            tma_prefetch_desc(&p0.tq_rows);
            tma_prefetch_desc(&p0.tout_rows);
        }
    }

    const uint32_t smem_base = (smem_u32(x2_smem_raw) + 1023u) & ~1023u;
    const uint32_t q_bytes = nch * TILE_M * CHUNK_ROW_BYTES, kv_bytes = nch * X2_KN * CHUNK_ROW_BYTES;
    constexpr bool DENSE_Q = NWG == 4;                     // d <= 48: one chunk, Q by untiled bulk copy + rewrite
    const uint32_t kv_smem = smem_base;                    // [2][K | V]
    const uint32_t q_smem = smem_base + 4 * kv_bytes;      // [stages][nch][128 rows][128 B]; DENSE_Q: [NWG] of them
    const uint32_t raw_bytes = (TILE_M * args.d * 2 + 127) & ~127;
    const uint32_t raw_smem = q_smem + NWG * q_bytes;      // DENSE_Q: [stages] raw tiles of 128 rows x 2d bytes
    const uint32_t out_smem = raw_smem + stages * raw_bytes;   // DENSE_Q: [2] output tiles in the same dense layout
    volatile int* abort_p = &abort_flag;

    if (tid == 0) {
        abort_flag = 0;
        for (int s = 0; s < X2_MAX_STAGES; ++s) {
            mbar_init(smem_u32(&bar_full[s]), 1);
            mbar_init(smem_u32(&bar_empty[s]), DENSE_Q ? 4 : 1);   // DENSE_Q: the four warps that read the raw tile
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(smem_u32(&bar_kv_full[b]), 1);
            mbar_init(smem_u32(&bar_kv_empty[b]), 1);
        }
        for (int w = 0; w < NWG; ++w) {
            mbar_init(smem_u32(&bar_s_full[w]), 1);
            mbar_init(smem_u32(&bar_p_full[w]), 4);   // one arrival per softmax warp
            mbar_init(smem_u32(&bar_o_full[w]), 1);
            mbar_init(smem_u32(&bar_o_free[w]), 4);
            mbar_init(smem_u32(&bar_pv_done[w]), 1);
            mbar_init(smem_u32(&bar_q_ready[w]), 4);
        }
        mbar_init_fence();
    }
    if (warp == S_ISSUER_WARP) {
        tmem_alloc(smem_u32(&tmem_base_slot), 512);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    // Set-up (barriers, tensor memory) overlapped the tail of the previous kernel of the stream; global memory and
    // every bounded wait come after it has completed.
    pdl_wait();
    tc_fence_after_sync();
    const uint32_t tmem_base = tmem_base_slot;
    const uint32_t tmem_o0 = tmem_base + NWG * X2_KN;   // columns: S_0 .. S_{NWG-1} | O_0 .. O_{NWG-1}

    // With four softmax groups the register file is the limit (a row of 80 scores per thread): the control
    // warpgroup (producer, two issuers, one idle warp) hands registers over.  All four warps of a warpgroup
    // must execute the SAME setmaxnreg instruction, hence one site per kind.
    // setmaxnreg only moves registers INSIDE the CTA's launch allocation (threads x registers per thread as
    // compiled): an increase that the decreases do not cover blocks for ever.  The host checks, from the
    // compiled register count, that 512 * X2_SOFTMAX_REGS + 128 * X2_CONTROL_REGS fits before using this variant.
    constexpr bool REBALANCE = NWG == 4;
    if (REBALANCE && warp >= LOADER_WARP) setmaxnreg_dec<X2_CONTROL_REGS>();
    if (warp == LOADER_WARP) {
        // ------------------------------------------------------------ TMA producer
        if (elect_one()) {
            int g_prev = 0;   // K and V of the first head: fetched by the first S issuer, at the same time as Q here
            for (int i = 0; i < n_local; ++i) {
                const int item = item0 + i, gh = item / args.tiles_per_bh, tile = item - gh * args.tiles_per_bh;
                const int s = i % stages, g = gh - bh0;
                const int pi = GROUPED ? gh / args.BH : 0, bh = gh - pi * args.BH;   // problem, head inside it
                const Cross2Problem& pr = args.prob[pi];
                const int bz = bh / args.lay.heads, hz = bh - bz * args.lay.heads;
                if (g != g_prev) {
                    // a new head: its K and V go into buffer g & 1 once the head two back has been consumed
                    if (g >= 2 && !mbar_wait(smem_u32(&bar_kv_empty[g & 1]), ((g >> 1) - 1) & 1, abort_p, args.status,
                                             SITE_Y_KVEMPTY, i))
                        break;
                    const uint32_t bar = smem_u32(&bar_kv_full[g & 1]), dst = kv_smem + (g & 1) * 2 * kv_bytes;
                    mbar_arrive_expect_tx(bar, 2 * kv_bytes);
                    for (int ch = 0; ch < nch; ++ch)
                        tma_load_4d(dst + ch * X2_KN * CHUNK_ROW_BYTES, &pr.tk, bar, ch * CHUNK_COLS, 0, hz, bz);
                    for (int ch = 0; ch < nch; ++ch)
                        tma_load_4d(dst + kv_bytes + ch * X2_KN * CHUNK_ROW_BYTES, &pr.tv, bar, ch * CHUNK_COLS, 0, hz, bz);
                    g_prev = g;
                }
                if (i >= stages &&
                    !mbar_wait(smem_u32(&bar_empty[s]), ((i / stages) - 1) & 1, abort_p, args.status, SITE_Y_EMPTY, i))
                    break;
                const uint32_t bar = smem_u32(&bar_full[s]), dst = q_smem + s * q_bytes;
                if (DENSE_Q) {
                    int rows = args.Nq - tile * TILE_M;
                    if (rows > TILE_M) rows = TILE_M;
                    const uint32_t bytes = (uint32_t)rows * args.d * 2;   // d % 8 == 0: a multiple of 16
                    if (args.strided_rows) {   // the same dense tile, row by row (rows past Nq arrive as zeros)
                        mbar_arrive_expect_tx(bar, raw_bytes);
                        tma_load_4d(raw_smem + s * raw_bytes, &pr.tq_rows, bar, 0, tile * TILE_M, hz, bz);
                        continue;
                    }
                    mbar_arrive_expect_tx(bar, bytes);
                    bulk_load(raw_smem + s * raw_bytes, pr.q + ((size_t)bh * args.Nq + (size_t)tile * TILE_M) * args.d, bytes, bar);
                    continue;
                }
                mbar_arrive_expect_tx(bar, q_bytes);
                for (int ch = 0; ch < nch; ++ch)
                    tma_load_4d(dst + ch * TILE_M * CHUNK_ROW_BYTES, &pr.tq, bar, ch * CHUNK_COLS, tile * TILE_M, hz, bz);
            }
        }
    } else if (warp == S_ISSUER_WARP || warp == S2_ISSUER_WARP || warp == O_ISSUER_WARP) {
        // ------------------------------------------------------------ MMA issuers
        // An issuer is one thread sharing a scheduler with busy softmax warps: each barrier test and each
        // tcgen05.mma costs it tens to hundreds of clocks, and a single thread doing both products of every
        // item became the bound of the kernel.  So the work is split: two threads issue S = Q K^T (even and odd
        // items: nothing orders the scores of different items; each satisfied wait and each MMA costs such a thread
        // about 250 clocks, 1300 per item, which alone set the pace of the kernel with one thread) and free Q stages,
        // a third issues O = P V (and frees K/V buffers).  S of item i+NWG reuses the columns of S/P of item i, so
        // an S issuer waits for that item's P V product to COMPLETE (bar_pv_done).
        if (elect_one()) {
            struct Cursor { int i, s, sph, w, n, g, t, hb, p; };
            const int t_first = item0 - bh0 * args.tiles_per_bh;
            auto advance = [&](Cursor& c) {   // item bookkeeping without divisions
                ++c.i;
                if (++c.s == stages) { c.s = 0; c.sph ^= 1; }
                if (++c.w == NWG) { c.w = 0; ++c.n; }
                if (++c.t == args.tiles_per_bh) {   // the next head, and past a problem's last head the next problem
                    c.t = 0; ++c.g;
                    if (GROUPED && ++c.hb == args.BH) { c.hb = 0; ++c.p; }
                }
            };
            Cursor c = {0, 0, 0, 0, 0, 0, t_first, hb0, prob0};
            bool ok = true;
            if (warp == S_ISSUER_WARP && n_local > 0) {
                // K and V of the CTA's first head, while the producer thread fetches the first Q tiles: a copy
                // instruction holds its thread for several hundred clocks, and the first scores wait for all three.
                const uint32_t bar = smem_u32(&bar_kv_full[0]);
                const int bz0 = hb0 / args.lay.heads, hz0 = hb0 - bz0 * args.lay.heads;
                mbar_arrive_expect_tx(bar, 2 * kv_bytes);
                for (int ch = 0; ch < nch; ++ch)
                    tma_load_4d(kv_smem + ch * X2_KN * CHUNK_ROW_BYTES, &args.prob[prob0].tk, bar, ch * CHUNK_COLS, 0, hz0, bz0);
                for (int ch = 0; ch < nch; ++ch)
                    tma_load_4d(kv_smem + kv_bytes + ch * X2_KN * CHUNK_ROW_BYTES, &args.prob[prob0].tv, bar, ch * CHUNK_COLS, 0, hz0, bz0);
            }
            if (warp != O_ISSUER_WARP) {
                const int parity = warp == S_ISSUER_WARP ? 0 : 1;
                uint32_t idesc_s = idesc_f16(TILE_M, X2_KN, false, false, args.prob[prob0].negate != 0, BF);
                int p_desc = prob0;   // the problem idesc_s was made for (only the sign of the scale differs)
                const int ksteps_s = (args.d + 15) / 16;
                const uint64_t q_desc0 = smem_desc_sw128(q_smem, 16, 1024);
                const uint64_t k_desc0 = smem_desc_sw128(kv_smem, 16, 1024);
                const uint32_t q_stage_off = q_bytes >> 4, kv_buf_off = (2 * kv_bytes) >> 4;
                int g_waited = -1;   // K and V of this head have been seen to land
                for (; c.i < n_local && ok; advance(c)) {
                    if ((c.i & 1) != parity) continue;
                    ok = (DENSE_Q ? mbar_wait(smem_u32(&bar_q_ready[c.w]), c.n & 1, abort_p, args.status, SITE_Y_STAGE, c.i)
                                  : mbar_wait(smem_u32(&bar_full[c.s]), c.sph, abort_p, args.status, SITE_Y_STAGE, c.i));
                    if (ok && c.g != g_waited) {
                        ok = mbar_wait(smem_u32(&bar_kv_full[c.g & 1]), (c.g >> 1) & 1, abort_p, args.status, SITE_Y_KV, c.i);
                        g_waited = c.g;
                    }
                    if (ok && c.n >= 1)   // the group's previous item no longer needs these columns
                        ok = mbar_wait(smem_u32(&bar_pv_done[c.w]), (c.n - 1) & 1, abort_p, args.status, SITE_Y_PV, c.i);
                    if (!ok) break;
                    tc_fence_after_sync();
                    if (GROUPED && c.p != p_desc) {
                        p_desc = c.p;
                        idesc_s = idesc_f16(TILE_M, X2_KN, false, false, args.prob[p_desc].negate != 0, BF);
                    }
                    const uint64_t qd = q_desc0 + (uint64_t)((DENSE_Q ? c.w : c.s) * q_stage_off);
                    const uint64_t kd = k_desc0 + (uint64_t)((c.g & 1) * kv_buf_off);
                    const uint32_t ts = tmem_base + c.w * X2_KN;
                    if (ksteps_s == 3) issue_qk<3>(ts, qd, kd, idesc_s);
                    else if (ksteps_s == 5) issue_qk<5>(ts, qd, kd, idesc_s);
                    else if (ksteps_s == 10) issue_qk<10>(ts, qd, kd, idesc_s);
                    else
                        for (int kk = 0; kk < ksteps_s; ++kk)
                            mma_f16_ss(ts, qd + (uint64_t)(((kk >> 2) * TILE_M * CHUNK_ROW_BYTES + (kk & 3) * 32) >> 4),
                                       kd + (uint64_t)(((kk >> 2) * X2_KN * CHUNK_ROW_BYTES + (kk & 3) * 32) >> 4), idesc_s,
                                       kk > 0);
                    tc_commit(smem_u32(&bar_s_full[c.w]));
                    if (!DENSE_Q) tc_commit(smem_u32(&bar_empty[c.s]));   // the Q stage is free once this product has read it
                }
            } else {
                const uint32_t idesc_o = idesc_f16(TILE_M, dpad, false, true, false, BF);
                const uint64_t v_desc0 = smem_desc_sw128(kv_smem + kv_bytes, X2_KN * CHUNK_ROW_BYTES, 1024);
                const uint32_t kv_buf_off = (2 * kv_bytes) >> 4;
                for (; c.i < n_local && ok; advance(c)) {
                    if (c.n >= 1)   // O_w of the group's previous item must have been read out
                        ok = mbar_wait(smem_u32(&bar_o_free[c.w]), (c.n - 1) & 1, abort_p, args.status, SITE_Y_OFREE, c.i);
                    if (ok) ok = mbar_wait(smem_u32(&bar_p_full[c.w]), c.n & 1, abort_p, args.status, SITE_Y_P, c.i);
                    if (!ok) break;
                    tc_fence_after_sync();
                    const uint64_t vd = v_desc0 + (uint64_t)((c.g & 1) * kv_buf_off);
#pragma unroll
                    for (int kk = 0; kk < X2_KN / 16; ++kk)   // O_w = P_w V, P_w in the first columns of S_w
                        mma_f16_ts(tmem_o0 + c.w * dpad, tmem_base + c.w * X2_KN + kk * 8,
                                   vd + (uint64_t)(kk * ((16 * CHUNK_ROW_BYTES) >> 4)), idesc_o, kk > 0);
                    tc_commit(smem_u32(&bar_o_full[c.w]));
                    tc_commit(smem_u32(&bar_pv_done[c.w]));
                    // last item of its head: every S product of this head completed before its softmax ran
                    if (c.i + 1 == n_local || c.t + 1 == args.tiles_per_bh) tc_commit(smem_u32(&bar_kv_empty[c.g & 1]));
                }
            }
        }
    } else if (warp < NWG * 4) {
        // ------------------------------------------------------------ softmax warps
        if (REBALANCE) setmaxnreg_inc<X2_SOFTMAX_REGS>();
        const int w = warp >> 2;
        const int r = tid & (TILE_M - 1);
        const uint32_t lane_off = (uint32_t)((warp & 3) * 32) << 16;
        const uint32_t tmem_s = tmem_base + w * X2_KN + lane_off;
        const int valid = args.Nk;
        bool ok = true;
        const float c2_one = args.prob[0].scale_log2e;
        // the problem of this group's current item, advanced NWG items at a time without divisions
        int it_t = item0 - bh0 * args.tiles_per_bh + w, it_hb = hb0, it_p = prob0;
        auto settle = [&]() {
            while (GROUPED && it_t >= args.tiles_per_bh) {
                it_t -= args.tiles_per_bh;
                if (++it_hb == args.BH) { it_hb = 0; ++it_p; }
            }
        };
        // DENSE_Q: rewrite the raw Q tile of item j (ring stage j % stages; j = w mod NWG and stages is a multiple of
        // NWG, so this group is the only consumer of that stage's barrier) into the group's MMA-layout buffer: row r
        // is 128 bytes at r * 128, its 16-byte chunk c at position c ^ (r & 7) (the 128-byte swizzle).
        // (rows past the end of a head -- the bulk copy of a ragged last tile brings only the rows there are, and what
        // the stage held before stays behind them -- are rewritten as zeros: a row's result never depends on another
        // row's data, but the decision to redo a row with its true maximum is taken per WARP, and stale rows must not
        // take part in it, or the bits of the valid rows beside them would depend on what ran before)
        int rw_tile = item0 - bh0 * args.tiles_per_bh + w;   // tile, inside its head, of the item rewritten next
        const bool ragged_heads = (args.Nq % TILE_M) != 0;
        auto rewrite_q = [&](int j) -> bool {
            const int s = j % stages;
            bool good = mbar_wait(smem_u32(&bar_full[s]), (j / stages) & 1, abort_p, args.status, SITE_Y_STAGE, j);
            good = __all_sync(0xffffffffu, good);
            if (!good) return false;
            bool live = true;
            if (ragged_heads) {   // (only a head's last tile can be ragged, and only when Nq is no multiple of 128)
                while (rw_tile >= args.tiles_per_bh) rw_tile -= args.tiles_per_bh;
                live = rw_tile * TILE_M + r < args.Nq;
                rw_tile += NWG;
            }
            const uint32_t src = raw_smem + s * raw_bytes + r * (args.d * 2);
            const uint32_t dst = q_smem + w * q_bytes + r * CHUNK_ROW_BYTES;
            const int chunks = args.d >> 3;   // 16-byte chunks of real data per row (<= 6)
            uint4 v[6];
#pragma unroll
            for (int c = 0; c < 6; ++c) v[c] = (live && c < chunks) ? ld_shared_v4(src + c * 16) : make_uint4(0u, 0u, 0u, 0u);
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&bar_empty[s]));   // the raw stage may be refilled
#pragma unroll
            for (int c = 0; c < 6; ++c) st_shared_v4(dst + ((c ^ (r & 7)) << 4), v[c]);
            fence_proxy_async_smem();   // generic-proxy stores before the tensor core reads them
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&bar_q_ready[w]));
            return true;
        };
        if (DENSE_Q && w < n_local) ok = rewrite_q(w);
        for (int i = w; i < n_local && ok; i += NWG, it_t += NWG) {
            const int n = i / NWG;
            settle();
            const float c2 = GROUPED ? args.prob[it_p].scale_log2e : c2_one;
            ok = mbar_wait(smem_u32(&bar_s_full[w]), n & 1, abort_p, args.status, SITE_Y_S, i);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after_sync();
            if (DENSE_Q && i + NWG < n_local) {   // S of this item is done: the Q buffer may take the next one
                ok = rewrite_q(i + NWG);
                if (!ok) break;
            }
            uint32_t packed[X2_KN / 2];
            float row_sum, anchor = 0.f;
#pragma unroll 1
            for (int attempt = 0; attempt < 2; ++attempt) {
                uint64_t acc[2] = {0ull, 0ull};
                float tail = 0.f;
                {   // columns 0..47
                    uint32_t s[48];
                    tmem_ld32(tmem_s, &s[0]);
                    tmem_ld16(tmem_s + 32, *reinterpret_cast<uint32_t(*)[16]>(&s[32]));
                    tmem_wait_ld();
                    if (attempt == 0) anchor = __uint_as_float(s[0]) * c2 + X2_HEADROOM_LOG2;
                    const float neg_mc = -anchor;
                    const uint64_t c2c2 = pack_b64(__float_as_uint(c2), __float_as_uint(c2));
                    const uint64_t nmnm = pack_b64(__float_as_uint(neg_mc), __float_as_uint(neg_mc));
                    exp2_pack_32<0, 16, BF>(&s[0], c2c2, nmnm, &packed[0], acc);
                    exp2_pack_16<0, BF>(&s[32], c2c2, nmnm, &packed[16], acc);
                }
                {   // columns 48..79: the last 16 hold the keys past Nk (zero-filled) and are masked
                    uint32_t s[32];
                    tmem_ld32(tmem_s + 48, &s[0]);
                    tmem_wait_ld();
                    const float neg_mc = -anchor;
                    const uint64_t c2c2 = pack_b64(__float_as_uint(c2), __float_as_uint(c2));
                    const uint64_t nmnm = pack_b64(__float_as_uint(neg_mc), __float_as_uint(neg_mc));
                    exp2_pack_16<0, BF>(&s[0], c2c2, nmnm, &packed[24], acc);
                    exp2_pack_32_masked<8, BF>(&s[16], c2, neg_mc, 64, valid, &packed[32], tail);
                }
                row_sum = sum_f32x2(acc[0], acc[1]) + tail;   // S_i of Eq. 4, relative to the anchor
                const bool over = !(row_sum <= X2_SUM_LIMIT);
                if (attempt == 1 || !__any_sync(0xffffffffu, over)) break;
                // rare: the row maximum lies far above the first score.  Nothing has been stored yet: take L_i of
                // Eq. 4 from the scores and redo the row.
                float row_max;
                {
                    uint32_t s[32];
                    tmem_ld32(tmem_s, &s[0]);
                    tmem_wait_ld();
                    row_max = row_max_masked<32>(s, 32);
                    tmem_ld32(tmem_s + 32, &s[0]);
                    tmem_wait_ld();
                    row_max = fmaxf(row_max, row_max_masked<32>(s, 32));
                    tmem_ld16(tmem_s + 64, *reinterpret_cast<uint32_t(*)[16]>(&s[0]));
                    tmem_wait_ld();
                    row_max = fmaxf(row_max, row_max_masked<16>(s, valid - 64));
                }
                anchor = row_max * c2;
            }
            tmem_st32(tmem_s, &packed[0]);    // P_w over the first 40 columns of S_w
            tmem_st8(tmem_s + 32, *reinterpret_cast<uint32_t(*)[8]>(&packed[32]));
            inv_sum[w][n & 1][r] = 1.f / row_sum;   // for the epilogue warpgroup
            tmem_wait_st();
            tc_fence_before_sync();
            __syncwarp();                           // every lane's store before lane 0's arrival
            if (lane == 0) mbar_arrive(smem_u32(&bar_p_full[w]));
        }
    } else if (warp < LOADER_WARP) {
        // ------------------------------------------------------------ epilogue warpgroup: every item in turn
        if (REBALANCE) setmaxnreg_dec<X2_EPILOGUE_REGS>();
        const int r = tid & (TILE_M - 1);
        const uint32_t lane_off = (uint32_t)((warp & 3) * 32) << 16;
        bool ok = true;
        int w = 0, n = 0;
        int bh = hb0, pi = prob0, tile = item0 - bh0 * args.tiles_per_bh;   // head inside its problem, problem, tile
        auto next_item = [&]() {
            if (++w == NWG) { w = 0; ++n; }
            if (++tile == args.tiles_per_bh) {
                tile = 0;
                if (++bh == args.BH && GROUPED) { bh = 0; ++pi; }
            }
        };
        for (int i = 0; i < n_local; ++i) {
            const uint32_t tmem_o = tmem_o0 + w * dpad + lane_off;
            // bar_o_full[w] completes after the O issuer saw bar_p_full[w], which the softmax warps arrived on after
            // writing inv_sum: the values are in shared memory by then.  (bar_p_full itself must not be waited on
            // here: a second consumer may fall two phases behind, and a parity wait cannot tell.)
            if (DENSE_Q && tid == EPILOGUE_WARP0 * 32) bulk_wait_read<1>();   // staging tile i & 1 has been read out
            ok = mbar_wait(smem_u32(&bar_o_full[w]), n & 1, abort_p, args.status, SITE_Y_O, i);
            // one decision for the whole warpgroup (its warps meet at a named barrier below: none may leave alone);
            // the barrier also publishes the bulk_wait_read above
            ok = DENSE_Q ? named_barrier_and(1, 128, ok) : __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after_sync();
            const float inv = inv_sum[w][n & 1][r];
            const int row = tile * TILE_M + r;
            const Cross2Problem& pr = args.prob[pi];
            __half* orow = head_row(pr.out, args.lay, bh, row);
            if (DENSE_Q) {
                // The tile is one contiguous piece of global memory: rows go to a dense staging tile in shared memory
                // (thread = row) and ONE bulk copy writes it out -- full lines instead of five strided 16-byte stores
                // per thread.  Two staging tiles: the copy of the item before last must have read its tile.
                const uint32_t stage = out_smem + (i & 1) * raw_bytes;
                uint32_t x[48];
                tmem_ld32(tmem_o, &x[0]);
                if (dpad > 32) tmem_ld16(tmem_o + 32, *reinterpret_cast<uint32_t(*)[16]>(&x[32]));
                tmem_wait_ld();
                tc_fence_before_sync();
                if (lane == 0) mbar_arrive(smem_u32(&bar_o_free[w]));   // O_w is in registers
                const uint32_t dst = stage + r * (args.d * 2);
#pragma unroll
                for (int g = 0; g < 6; ++g) {
                    uint4 v8;
                    v8.x = pack_16x2<BF>(__uint_as_float(x[g * 8 + 0]) * inv, __uint_as_float(x[g * 8 + 1]) * inv);
                    v8.y = pack_16x2<BF>(__uint_as_float(x[g * 8 + 2]) * inv, __uint_as_float(x[g * 8 + 3]) * inv);
                    v8.z = pack_16x2<BF>(__uint_as_float(x[g * 8 + 4]) * inv, __uint_as_float(x[g * 8 + 5]) * inv);
                    v8.w = pack_16x2<BF>(__uint_as_float(x[g * 8 + 6]) * inv, __uint_as_float(x[g * 8 + 7]) * inv);
                    if (g * 8 + 8 <= args.d) st_shared_v4(dst + g * 16, v8);
                }
                fence_proxy_async_smem();   // generic-proxy stores before the bulk copy reads them
                named_barrier(1, 128);
                if (tid == EPILOGUE_WARP0 * 32) {
                    int rows = args.Nq - tile * TILE_M;
                    if (rows > TILE_M) rows = TILE_M;
                    if (args.strided_rows) {   // rows past Nq are clipped by the hardware
                        const int bz = bh / args.lay.heads, hz = bh - bz * args.lay.heads;
                        tma_store_4d(&pr.tout_rows, stage, 0, tile * TILE_M, hz, bz);
                    } else {
                        bulk_store(pr.out + ((size_t)bh * args.Nq + (size_t)tile * TILE_M) * args.d, stage,
                                   (uint32_t)rows * args.d * 2);
                    }
                    bulk_commit();
                }
                next_item();
                continue;
            }
            // O / S_i -> fp16 -> global, 32 columns per tensor-memory round trip (dpad is a multiple of 16)
            for (int c0 = 0; c0 < dpad; c0 += 32) {
                uint32_t x[32];
                tmem_ld16(tmem_o + c0, *reinterpret_cast<uint32_t(*)[16]>(&x[0]));
                if (c0 + 16 < dpad) tmem_ld16(tmem_o + c0 + 16, *reinterpret_cast<uint32_t(*)[16]>(&x[16]));
                tmem_wait_ld();
                if (c0 + 32 >= dpad) {   // all of O_w is in registers: the next product of this group may overwrite it
                    tc_fence_before_sync();
                    if (lane == 0) mbar_arrive(smem_u32(&bar_o_free[w]));
                }
                if (row < args.Nq) {
#pragma unroll
                    for (int g = 0; g < 4; ++g) {
                        uint4 v8;
                        v8.x = pack_16x2<BF>(__uint_as_float(x[g * 8 + 0]) * inv, __uint_as_float(x[g * 8 + 1]) * inv);
                        v8.y = pack_16x2<BF>(__uint_as_float(x[g * 8 + 2]) * inv, __uint_as_float(x[g * 8 + 3]) * inv);
                        v8.z = pack_16x2<BF>(__uint_as_float(x[g * 8 + 4]) * inv, __uint_as_float(x[g * 8 + 5]) * inv);
                        v8.w = pack_16x2<BF>(__uint_as_float(x[g * 8 + 6]) * inv, __uint_as_float(x[g * 8 + 7]) * inv);
                        if (c0 + g * 8 + 8 <= args.d) *reinterpret_cast<uint4*>(orow + c0 + g * 8) = v8;
                    }
                }
            }
            next_item();
        }
        if (DENSE_Q && tid == EPILOGUE_WARP0 * 32) bulk_wait_all();   // shared memory must outlive the copies
    }

    // ------------------------------------------------------------ teardown (every thread arrives)
    tc_fence_before_sync();
    __syncthreads();
    if (warp == LOADER_WARP && lane == 0 && abort_flag) {
        mbar_drain(smem_u32(&bar_kv_full[0]), 0);   // gave up: let a K/V fetch still in flight land
        mbar_drain(smem_u32(&bar_kv_full[1]), 0);
    }
    __syncthreads();
    if (warp == S_ISSUER_WARP) {
        __syncwarp();
        tmem_dealloc(tmem_base, 512);
    }
}

}  // namespace sd_attn
