// Fused single-pass attention with one SPARE score buffer that takes the tensor-core round trip off the
// softmax's path: T query tiles per CTA share T + 1 score buffers.  T is at most 4 at d <= 48 (the d = 40 layers of
// the UNet), 3 at d <= 80, 2 at d <= 160: (T + 1) * 64 score columns and T * dpad output columns fill the 512
// columns of tensor memory.
//
// In the four-tile kernel the weights P_t(j) overwrite the scores S_t(j), so S_t(j+1) can only follow the
// product P_t(j) V(j): after every key tile a softmax warpgroup idles for the round trip softmax -> MMA issue ->
// tensor pipe -> softmax (450-550 clocks of 2500), and four warps per scheduler do not hide it.  With d <= 48 the
// four output accumulators need 192 of the 512 tensor-memory columns, which leaves room for FIVE 64-column score
// buffers for the four tiles.  The (tile, key tile) steps are put in one global order k = T*j + t (T tiles);
// step k uses buffer k mod (T+1); S(k + T + 1) is issued right behind P(k) V(k) -- into the buffer that product
// frees -- and belongs to the tile that comes NEXT in the rotation, not to the tile that just finished.  So when a
// tile finishes key tile j its scores for j+1 were requested a quarter of a period earlier, by its neighbour's
// hand-off, and are normally there.
//
//   warps 0-15   softmax of tiles 0..3 (thread = query row = TMEM lane)
//   warp 16      TMA producer          warps 17-20  MMA issuers: issuer t multiplies P_t V and then requests the
//                scores of tile t+1 (32 registers each; warps 21-23 only fill the control warpgroup)
//
// A CTA takes 1 to 4 query tiles (Fused4Args::tiles_per_cta): the host gives a small problem fewer tiles per CTA so
// that it spreads over more SMs; with one tile the rotation degenerates to two alternating score buffers.
// One tile per CTA normally runs the SPLIT variant instead (template parameter, see below): the other softmax
// warpgroups, idle otherwise, take a share of the tile's score columns each.
// The anchor scheme of the exponent (no per-tile maximum) is described in fused_common.cuh.
//
// One launch serves up to F4_GROUP_MAX problems of one shape (a tensor-map triple, an output pointer and a scale
// each).  A UNIT is the group of up to T query tiles of a head that share a CTA's K/V stream.  Two ways to deal the
// units out:
//   whole units   one CTA per (problem, unit), all key tiles.
//   shares        the work of a problem is the line of its W = units x key tiles steps (unit, key tile), and CTA c of
//                 G takes the steps [c W / G, (c + 1) W / G) of EVERY problem of the launch in turn -- one or two
//                 SEGMENTS (unit, first key tile, count) per problem.  The host launches one CTA per SM, so that no
//                 SM idles in a last, partly filled wave (the 512 query tiles of the 4096-token call: 128 units on
//                 148 SMs).  A unit whose key tiles are cut between CTAs is finished through global scratch: each
//                 piece stores its unnormalised accumulator, anchor and row sum, and whichever piece's warpgroup
//                 arrives last (a counter per query tile) combines all pieces in key order -- nobody waits, and
//                 neither the cut points (a function of the problem's shape and G only) nor the order of additions
//                 depend on who arrives last or on what else is in the launch, so the bits repeat.
// Between two segments of a CTA the barriers are re-initialised behind a CTA-wide barrier (all asynchronous
// arrivals of the finished segment have been waited for by then); tensor memory and shared memory carry on.
#pragma once
#include <cuda.h>

#include "fused_common.cuh"  // Fused4Args, F4_* constants, SITE_G_*

namespace sd_attn {


constexpr int F4S_MAX_DPAD = 160;
constexpr int F4S_MAX_KSTEPS = 10;          // MMA steps of Q K^T at the largest head dim
constexpr int F4S_SMEM_BUDGET = 220 * 1024;
__host__ inline int f4s_max_tiles(int dpad) {   // (T + 1) * 64 + T * dpad <= 512
    const int t = (512 - F4_BN) / (F4_BN + dpad);
    return t > F4_TILES ? F4_TILES : t;
}
// Of every 8 exponentials this many are evaluated by the degree-3 polynomial on the FMA pipe instead of the
// special function unit, which is the busiest unit of this kernel (measured: 0 -> 100 us, 2 -> 95 us, 3 -> 96 us on
// the 4096-token d = 40 call).
#ifndef SD_ATTN_F4S_POLY_PER8
#define SD_ATTN_F4S_POLY_PER8 2
#endif
constexpr int F4S_POLY_PER8 = SD_ATTN_F4S_POLY_PER8;
constexpr int F4S_BUFFERS = F4_TILES + 1;
#ifndef SD_ATTN_F4S_SOFTMAX_REGS
#define SD_ATTN_F4S_SOFTMAX_REGS 104   // 512 * 104 + 256 * 32 = 768 * 80, the launch allocation
#define SD_ATTN_F4S_CONTROL_REGS 32
#endif
constexpr int F4S_SOFTMAX_REGS = SD_ATTN_F4S_SOFTMAX_REGS;
constexpr int F4S_CONTROL_REGS = SD_ATTN_F4S_CONTROL_REGS;
static_assert(512 * F4S_SOFTMAX_REGS + 256 * F4S_CONTROL_REGS == 768 * 80, "setmaxnreg budget");

// Shares: a query tile's piece was stored and its arrival counted (see the softmax warps' epilogue).  If it was the
// last of its unit's pieces, this warpgroup (thread = row r) combines them all, in key order,
// o = sum_c 2^(m_c - m) O_c / sum_c 2^(m_c - m) l_c with m = max_c m_c.  The pieces of a unit lie with the CTAs
// c_first .. c_last (CTA c begins at step c W / G of the problem).  Kept out of line: it runs once or twice per
// CTA and must not cost the key-tile loop registers.
template <bool BF>
__device__ __noinline__ void f4s_combine_pieces(const Fused4Args& args, int t, int r, int prob_i, int unit, int c_first, int c_last) {
    const int dpad = args.dpad, n_kv_all = args.n_kv;
    const long long u0 = (long long)unit * n_kv_all, Wl = (long long)args.n_units * n_kv_all, Gl = gridDim.x;
    auto piece_of = [&](int c) -> const float* {
        const long long begin = (long long)c * Wl / Gl;
        return args.part + ((2 * (size_t)prob_i * gridDim.x + 2 * (size_t)c + (u0 < begin ? 0 : 1)) * args.part_slot_floats) +
               (size_t)t * (dpad + 2) * TILE_M + r;
    };
    float m_all = -INFINITY, l_all = 0.f;
    for (int c = c_first; c <= c_last; ++c) m_all = fmaxf(m_all, __ldcg(piece_of(c) + dpad * TILE_M));
    for (int c = c_first; c <= c_last; ++c)
        l_all += ex2_approx(__ldcg(piece_of(c) + dpad * TILE_M) - m_all) * __ldcg(piece_of(c) + (dpad + 1) * TILE_M);
    const float inv = 1.f / l_all;
    const int quad = unit % args.units_per_head, bh = unit / args.units_per_head;
    const int row = quad * args.tiles_per_cta * TILE_M + t * TILE_M + r;
    __half* orow = head_row(args.prob[prob_i].out, args.lay, bh, row);
    // 24 columns at a time (d is a multiple of 8), the loads of two pieces in flight together
    for (int c0 = 0; c0 < args.d; c0 += 24) {
        float acc[24];
#pragma unroll
        for (int k = 0; k < 24; ++k) acc[k] = 0.f;
        for (int c = c_first; c <= c_last; c += 2) {
            const float* pa = piece_of(c);
            const bool two = c + 1 <= c_last;
            const float* pb = two ? piece_of(c + 1) : pa;
            float xa[24], xb[24];
#pragma unroll
            for (int k = 0; k < 24; ++k) xa[k] = c0 + k < args.d ? __ldcg(pa + (c0 + k) * TILE_M) : 0.f;
#pragma unroll
            for (int k = 0; k < 24; ++k) xb[k] = (two && c0 + k < args.d) ? __ldcg(pb + (c0 + k) * TILE_M) : 0.f;
            const float fa = ex2_approx(__ldcg(pa + dpad * TILE_M) - m_all) * inv;
            const float fb = two ? ex2_approx(__ldcg(pb + dpad * TILE_M) - m_all) * inv : 0.f;
#pragma unroll
            for (int k = 0; k < 24; ++k) acc[k] = fmaf(xb[k], fb, fmaf(xa[k], fa, acc[k]));
        }
#pragma unroll
        for (int k = 0; k < 24; k += 8) {
            uint4 o;
            o.x = pack_16x2<BF>(acc[k + 0], acc[k + 1]); o.y = pack_16x2<BF>(acc[k + 2], acc[k + 3]);
            o.z = pack_16x2<BF>(acc[k + 4], acc[k + 5]); o.w = pack_16x2<BF>(acc[k + 6], acc[k + 7]);
            if (row < args.Nq && c0 + k + 8 <= args.d) *reinterpret_cast<uint4*>(orow + c0 + k) = o;
        }
    }
}

// Shares: the thread's row of a piece -- O from tensor memory, anchor, row sum -- to the scratch, as
// [tile][dpad + 2 columns: O, anchor, row sum][128 rows], so that a warp writes whole 128-byte lines.
__device__ __noinline__ void f4s_store_piece(float* piece, uint32_t tmem_o, int dpad, float m_run, float l_run) {
    for (int g = 0; g < (dpad >> 4); ++g) {
        uint32_t x[16];
        tmem_ld16(tmem_o + g * 16, x);
        tmem_wait_ld();
#pragma unroll
        for (int c = 0; c < 16; ++c) piece[(g * 16 + c) * TILE_M] = __uint_as_float(x[c]);
    }
    piece[dpad * TILE_M] = m_run;
    piece[(dpad + 1) * TILE_M] = l_run;
    __threadfence();
}

// SPLIT > 1 (only with ONE query tile per CTA): the key tiles are dealt out among SPLIT warpgroups ("parts": part g
// takes key tiles g, g + SPLIT, ...), each with an exponent anchor, a row sum and an accumulator O_g of its own over
// ITS keys, combined once at the end.  A lone tile is bound by the chain of latencies of one warp per scheduler
// (tcgen05.ld -> exp2 -> tcgen05.st -> hand-over: 1400-1500 clocks per key tile, measured, against 600 per tile
// with four tiles resident); the parts work on different key tiles at the same time, so their chains overlap as
// those of four query tiles do, and they need no agreement on an anchor because their products never share an
// accumulator.  The score buffers run ahead of the products (NB of them, a multiple of SPLIT), and the MMAs come from
// two threads: the products of key tile j from one, the scores of key tile j + NB from the other.
template <int POLY, int NCH, int SPLIT = 1, bool BF = false>   // NCH: 64-column chunks per row (head dim <= 64 * NCH); BF: bfloat16 tensors
__global__ void __launch_bounds__(F4_THREADS, 1)
fused4s_attention_kernel(const __grid_constant__ Fused4Args args) {
    constexpr int BN = F4_BN;
    extern __shared__ uint8_t f4s_smem_raw[];
    // per (tile, buffer): S ready (MMA) | P ready (softmax).  per tile: Q landed | P V of key tile j done | all of
    // O_t done.  The score barriers are per tile AND buffer so that every barrier has ONE consumer that takes its
    // phases in order (a parity wait is only sound for a waiter exactly one phase behind): tile t meets buffer b
    // every NB key tiles, and the buffer cannot come back to it before its previous contents were consumed.
    // (one block of memory, so that a warp can (re-)initialise them side by side: see init_barriers)
    struct Barriers {
        uint64_t s_full[F4_TILES][F4S_BUFFERS], p_full[F4_TILES][F4S_BUFFERS];   // p_full: 4 arrivals, one per softmax warp
        uint64_t q_full[F4_TILES], pv_done[F4_TILES], o_final[F4_TILES];
        uint64_t kv_full[F4_STAGES];
        uint64_t buf_free[F4S_BUFFERS];   // SPLIT > 1: the products reading a buffer's weights are done
        uint64_t kv_empty[F4_STAGES];     // one commit per issuer: as many arrivals as the unit has query tiles
    };
    constexpr int N_BARRIERS = sizeof(Barriers) / sizeof(uint64_t);
    constexpr int P_FULL_FIRST = F4_TILES * F4S_BUFFERS, P_FULL_END = 2 * F4_TILES * F4S_BUFFERS;
    constexpr int KV_EMPTY_FIRST = N_BARRIERS - F4_STAGES;
    __shared__ __align__(8) Barriers bars;
    auto& bar_s_full = bars.s_full;
    auto& bar_p_full = bars.p_full;
    auto& bar_q_full = bars.q_full;
    auto& bar_pv_done = bars.pv_done;
    auto& bar_o_final = bars.o_final;
    auto& bar_kv_full = bars.kv_full;
    auto& bar_kv_empty = bars.kv_empty;
    auto& bar_buf_free = bars.buf_free;
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;
    // A piece whose arrival number among the pieces of its unit is being fetched: {ticket, problem, unit, pending?} per
    // query tile.  The ticket is looked at after the CTA-wide barrier that ends the segment, so that nobody waits
    // for the counter's round trip to the L2.
    __shared__ int piece_ticket[F4_TILES][4];
    // the segment the CTA works on, written by the scheduling thread: live? | problem | unit | first key tile | key
    // tiles | query tiles | nothing follows  (in shared memory so that no role carries the walk in registers)
    __shared__ int seg_desc[8];
    __shared__ float2 part_ml[SPLIT > 1 ? SPLIT : 1][SPLIT > 1 ? TILE_M : 1];   // SPLIT > 1: (anchor, row sum) of every part

    const int tid = threadIdx.x, lane = tid & 31;
    const int warp = __shfl_sync(0xffffffffu, tid >> 5, 0);   // warp-uniform for the compiler
    if (threadIdx.x == 0) pdl_launch_dependents();   // the next kernel of the stream may start its set-up
    const int n_kv_all = args.n_kv;
    if (threadIdx.x == 32) {   // the tensor maps are kernel parameters: their fetch need not wait for anything
        const int p0 = args.shares ? 0 : (int)(blockIdx.x / args.n_units);
        tma_prefetch_desc(&args.prob[p0].tq);
        tma_prefetch_desc(&args.prob[p0].tk);
        tma_prefetch_desc(&args.prob[p0].tv);
    }
    const int dpad = args.dpad;
    constexpr int nch = NCH;
    const int stages = args.stages;   // K/V ring depth

    const uint32_t smem_base = (smem_u32(f4s_smem_raw) + 1023u) & ~1023u;
    constexpr uint32_t q_tile_bytes = nch * TILE_M * CHUNK_ROW_BYTES;   // [chunk][128 rows][128 B]
    constexpr uint32_t kv_tile_bytes = nch * BN * CHUNK_ROW_BYTES;      // [chunk][64 rows][128 B]
    const uint32_t q_smem = smem_base;                              // [tiles per CTA] query tiles
    const uint32_t kv_smem = q_smem + args.tiles_per_cta * q_tile_bytes;   // [stages][K | V]
    volatile int* abort_p = &abort_flag;

    // (Re-)initialise every barrier for a segment of `tiles` query tiles, one warp at it (lane i takes barriers i,
    // i + 32, ...); `again`: they hold a finished segment's state.
    auto init_barriers = [&](int tiles, bool again) {
        uint64_t* flat = reinterpret_cast<uint64_t*>(&bars);
        // Retire them all first, fence, then initialise them all.  (mbarrier.inval and mbarrier.init of ONE barrier
        // issued back to back came out wrong on the GPU: ring barriers of the next segment completed an arrival
        // early and the last query tiles multiplied by the wrong V tile.)
        if (again) {
            for (int i = lane; i < N_BARRIERS; i += 32) mbar_inval(smem_u32(flat + i));
            __threadfence_block();
            fence_proxy_async_smem();
            __syncwarp();
        }
        for (int i = lane; i < N_BARRIERS; i += 32)
            mbar_init(smem_u32(flat + i), i >= KV_EMPTY_FIRST ? (uint32_t)tiles : (i >= P_FULL_FIRST && i < P_FULL_END) ? 4u : 1u);
        mbar_init_fence();
        __syncwarp();
    };
    // The scheduling warp (an otherwise idle control warp, all lanes in step) walks this CTA's steps: [w_begin, w_end)
    // of the W = units x key tiles of a problem -- of every problem in turn when the launch deals shares out.
    constexpr int SCHED_WARP = 21;
    const int W = args.n_units * n_kv_all;                             // (the host keeps it below 2^31)
    const int G = args.shares ? (int)gridDim.x : args.n_units;         // CTAs among which a problem's steps are dealt out
    const int cta = args.shares ? (int)blockIdx.x : (int)(blockIdx.x % args.n_units);   // this CTA among them
    const int w_begin = (int)((long long)cta * W / G), w_end = (int)((long long)(cta + 1) * W / G);
    int sched_w = w_begin, sched_prob = args.shares ? 0 : (int)(blockIdx.x / args.n_units);
    const int sched_prob_end = args.shares ? args.n_prob : sched_prob + 1;
    // publishes the next segment (or "none") and (re-)initialises the barriers for it
    auto next_segment = [&](bool again) {
        if (!(sched_w < w_end)) {   // on to this CTA's share of the next problem
            sched_w = w_begin;
            ++sched_prob;
        }
        if (sched_prob >= sched_prob_end || !(w_begin < w_end)) {
            if (lane == 0) seg_desc[0] = 0;
            return;
        }
        const int unit = sched_w / n_kv_all, j0 = sched_w - unit * n_kv_all;
        const int n = (w_end - sched_w) < (n_kv_all - j0) ? (w_end - sched_w) : (n_kv_all - j0);
        const int quad = unit % args.units_per_head;
        int tiles = (args.Nq - quad * args.tiles_per_cta * TILE_M + TILE_M - 1) / TILE_M;
        if (tiles > args.tiles_per_cta) tiles = args.tiles_per_cta;
        sched_w += n;
        if (lane == 0) {
            seg_desc[0] = 1; seg_desc[1] = sched_prob; seg_desc[2] = unit; seg_desc[3] = j0; seg_desc[4] = n;
            seg_desc[5] = tiles;
            seg_desc[6] = !(sched_w < w_end) && sched_prob + 1 == sched_prob_end;
        }
        init_barriers(tiles, again);
    };
    if (warp == SCHED_WARP) {
        if (lane == 0) abort_flag = 0;
        if (lane < F4_TILES) piece_ticket[lane][3] = 0;
        next_segment(false);
    }
    if (warp == 16) {
        tmem_alloc(smem_u32(&tmem_base_slot), 512);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    // Set-up (barriers, tensor memory) overlapped the tail of the previous kernel of the stream; global memory and
    // every bounded wait come after it has completed.
    pdl_wait();
    const uint32_t tmem_base = tmem_base_slot;
    // columns: the score buffers | O_0 .. O_{T-1} (SPLIT > 1: the parts' O_0 .. O_{SPLIT-1})
    const uint32_t tmem_o0 = tmem_base + (SPLIT > 1 ? args.split_buffers : args.tiles_per_cta + 1) * BN;

    // Behind the CTA-wide barrier that ends a segment: was this query tile's piece the last of its unit's to arrive?
    auto combine_if_last = [&](int t) {
        if (!piece_ticket[t][3]) return;
        const int ticket = piece_ticket[t][0], prob_i = piece_ticket[t][1], unit = piece_ticket[t][2];
        named_barrier(2 + t, TILE_M);                // everybody has read the box
        const int r = tid & (TILE_M - 1);
        if (r == 0) piece_ticket[t][3] = 0;
        const long long u0 = (long long)unit * n_kv_all;
        const int c_first = (int)(((u0 + 1) * G - 1) / W), c_last = (int)(((u0 + n_kv_all) * G - 1) / W);
        if (ticket != c_last - c_first) return;
        __threadfence();
        if (r == 0) args.part_count[((size_t)prob_i * args.n_units + unit) * F4_TILES + t] = 0;   // as the next launch expects it
        f4s_combine_pieces<BF>(args, t, r, prob_i, unit, c_first, c_last);
    };

    // One setmaxnreg site per kind, executed by whole warpgroups; the budget is the CTA's launch allocation.  The
    // control warps and the softmax warps each walk the CTA's segments in a loop of their own (the code behind a
    // setmaxnreg must be reachable from that one only) and meet at the CTA-wide barriers between segments.
    if (warp >= 16) {
    setmaxnreg_dec<F4S_CONTROL_REGS>();
    for (;;) {
    // ------------------------------------------------------------ the segment: key tiles j0 .. j0 + n_kv - 1 of a unit
    if (!seg_desc[0]) break;
    const int prob_i = seg_desc[1], unit = seg_desc[2], j0 = seg_desc[3], n_kv = seg_desc[4], T = seg_desc[5];
    const bool last_segment = seg_desc[6] != 0;
    const int quad = unit % args.units_per_head, bh = unit / args.units_per_head;
    const Fused4Problem& pr = args.prob[prob_i];
    const int row_base = quad * args.tiles_per_cta * TILE_M;
    const int NB = SPLIT > 1 ? args.split_buffers : T + 1;   // score buffers in the rotation
    if (warp == 16) {
        // ------------------------------------------------------------ TMA producer
        if (elect_one()) {
            // In the order the issuers need them: Q_0 and the first key tile first (a tile of 80-byte rows costs the
            // TMA unit about 7 clocks per row, so the order decides when the first scores can start).
            const int bz = bh / args.lay.heads, hz = bh - bz * args.lay.heads;
            auto load_q = [&](int t) {
                const uint32_t bar = smem_u32(&bar_q_full[t]);
                mbar_arrive_expect_tx(bar, q_tile_bytes);
                for (int ch = 0; ch < nch; ++ch)
                    tma_load_4d(q_smem + t * q_tile_bytes + ch * TILE_M * CHUNK_ROW_BYTES, &pr.tq, bar, ch * CHUNK_COLS,
                                row_base + t * TILE_M, hz, bz);
            };
            load_q(0);
            int s = 0, pe = 1;   // stage of key tile j; parity of the kv_empty phase that frees it (from j = stages on)
            for (int j = 0; j < n_kv; ++j, ++s) {
                if (s == stages) { s = 0; pe ^= 1; }
                // (eight stages ahead of the issuers: it sleeps between polls, which is worth 1% of the call)
                if (j >= stages && !mbar_wait_lazy(smem_u32(&bar_kv_empty[s]), pe, abort_p, args.status, SITE_G_EMPTY, j))
                    break;
                const uint32_t k_dst = kv_smem + s * 2 * kv_tile_bytes, v_dst = k_dst + kv_tile_bytes;
                const uint32_t bar = smem_u32(&bar_kv_full[s]);
                mbar_arrive_expect_tx(bar, 2 * kv_tile_bytes);
                for (int ch = 0; ch < nch; ++ch)
                    tma_load_4d(k_dst + ch * BN * CHUNK_ROW_BYTES, &pr.tk, bar, ch * CHUNK_COLS, (j0 + j) * BN, hz, bz);
                for (int ch = 0; ch < nch; ++ch)
                    tma_load_4d(v_dst + ch * BN * CHUNK_ROW_BYTES, &pr.tv, bar, ch * CHUNK_COLS, (j0 + j) * BN, hz, bz);
                if (j == 0)
                    for (int t = 1; t < T; ++t) load_q(t);
            }
            // Another segment follows: the issuers' last commits on the ring (never waited for above) must have
            // landed before the barriers are initialised again.
            if (!last_segment) {
                for (int j = n_kv > stages ? n_kv - stages : 0; j < n_kv; ++j)
                    if (!mbar_wait(smem_u32(&bar_kv_empty[j % stages]), (j / stages) & 1, abort_p, args.status, SITE_G_EMPTY, j))
                        break;
            }
        }
        __syncwarp();
    } else if (warp > 16 && warp <= 16 + F4_TILES) {
        // ------------------------------------------------------------ MMA issuer of the steps of query tile t
        // Issuer t waits for P of its own tile's step k = T*j + t, issues O_t += P V(j), and then -- behind that
        // product, on the same thread, into the buffer it frees -- the scores of step k + NB, which belong to the
        // NEXT tile of the rotation.
        const int t = warp - 17;
        if ((t < T || (SPLIT > 1 && t == 1)) && elect_one()) {
            const uint32_t idesc_s = idesc_f16(TILE_M, BN, false, false, pr.negate != 0, BF);
            const uint32_t idesc_o = idesc_f16(TILE_M, dpad, false, true, false, BF);
            const int ksteps_s = (args.d + 15) / 16;   // 16 columns each; four to a swizzled 64-column chunk
            const int tn = (t + 1 == T) ? 0 : t + 1;   // the tile whose scores this thread requests
            const uint64_t q_desc = smem_desc_sw128(q_smem + tn * q_tile_bytes, 16, 1024);
            const uint64_t q_desc_own = smem_desc_sw128(q_smem + t * q_tile_bytes, 16, 1024);
            const uint64_t q_desc_own_split = smem_desc_sw128(q_smem, 16, 1024);   // SPLIT > 1: the one tile
            const uint64_t k_desc0 = smem_desc_sw128(kv_smem, 16, 1024);
            const uint64_t v_desc0 = smem_desc_sw128(kv_smem + kv_tile_bytes, BN * CHUNK_ROW_BYTES, 1024);
            constexpr uint32_t stage_off = (2 * kv_tile_bytes) >> 4;
            const uint32_t tmem_o = tmem_o0 + t * dpad;
            const uint32_t b_pvdone = smem_u32(&bar_pv_done[t]);

            auto issue_s = [&](uint64_t qd, int tile, int st, int b) {   // scores of (tile, K in stage st) into buffer b
                const uint64_t kd = k_desc0 + (uint64_t)(st * stage_off);
                const uint32_t ts = tmem_base + b * BN;
                // The issuer's instruction stream is on the hand-off path (one predicated-off MMA per step cost 4% on
                // the 9216-token call; hoisting the address arithmetic above the wait cost registers and 1%): the variant
                // for head dims up to 48 issues at most three steps, and exactly three without predicates for d = 40.
                constexpr int KS_MAX = (NCH == 1 && POLY != 0 && SPLIT == 1) ? 3 : 4 * NCH;   // (POLY != 0, SPLIT == 1: the d <= 48 variant)
                if (KS_MAX == 3 && ksteps_s == 3) {
#pragma unroll
                    for (int kk = 0; kk < 3; ++kk)
                        mma_f16_ss(ts, qd + (uint64_t)(kk * 2), kd + (uint64_t)(kk * 2), idesc_s, kk > 0);
                } else {
#pragma unroll
                    for (int kk = 0; kk < KS_MAX; ++kk)
                        if (kk < ksteps_s)
                            mma_f16_ss(ts, qd + (uint64_t)(((kk >> 2) * TILE_M * CHUNK_ROW_BYTES + (kk & 3) * 32) >> 4),
                                       kd + (uint64_t)(((kk >> 2) * BN * CHUNK_ROW_BYTES + (kk & 3) * 32) >> 4), idesc_s, kk > 0);
                }
                tc_commit(smem_u32(&bar_s_full[tile][b]));
            };
            auto issue_o = [&](int j, int st, int b) {   // O_t (+)= P V(j), V in stage st, P in the first 32 columns of buffer b
                const uint64_t vd = v_desc0 + (uint64_t)(st * stage_off);
                const uint32_t tp = tmem_base + b * BN;
                if (SPLIT > 1) {
                    // key tile j belongs to part j % SPLIT: O_g (+)= P(j) V(j), the first of the part's tiles overwrites
                    const uint32_t to = tmem_o + (j % SPLIT) * dpad;
#pragma unroll
                    for (int kk = 0; kk < BN / 16; ++kk)
                        mma_f16_ts(to, tp + kk * 8, vd + (uint64_t)(kk * ((16 * CHUNK_ROW_BYTES) >> 4)), idesc_o, j >= SPLIT || kk > 0);
                } else {
#pragma unroll
                    for (int kk = 0; kk < BN / 16; ++kk)
                        mma_f16_ts(tmem_o, tp + kk * 8, vd + (uint64_t)(kk * ((16 * CHUNK_ROW_BYTES) >> 4)), idesc_o, j > 0 || kk > 0);
                }
            };

            if (SPLIT > 1) {
                // One tile, NB score buffers: step j uses buffer j % NB.  A lone issuing thread needs about 1000 clocks
                // per key tile (two waits, seven to nine MMAs, three commits) and would pace the kernel, so the work
                // is split: thread 0 issues the products O_g (+)= P_g V(j), thread 1 the scores of key tile j + NB
                // into the buffer those products free.  MMAs of different threads are not ordered by the tensor pipe,
                // so thread 1 waits for the products' COMPLETION (bar_buf_free of that buffer); with NB >= 3 that
                // round trip is off everybody's path: the parts may run NB - 1 key tiles ahead of the products.
                bool ok = true;
                if (t == 1) {
                    ok = mbar_wait(smem_u32(&bar_q_full[0]), 0, abort_p, args.status, SITE_G_Q, 0);
                    int b = 0, ph = 0;                 // buffer and its bar_buf_free phase
                    int sn = 0, pn = 0;                // stage and phase of the key tile whose scores are requested
                    for (int jn = 0; jn < n_kv && ok; ++jn) {
                        ok = mbar_wait(smem_u32(&bar_kv_full[sn]), pn, abort_p, args.status, SITE_G_KV, jn);
                        if (ok && jn >= NB) {          // the products of key tile jn - NB have read their weights
                            ok = mbar_wait(smem_u32(&bar_buf_free[b]), ph, abort_p, args.status, SITE_G_PV, jn);
                        }
                        if (!ok) break;
                        tc_fence_after_sync();
                        issue_s(q_desc_own_split, 0, sn, b);
                        if (++b == NB) { b = 0; if (jn >= NB) ph ^= 1; }
                        if (++sn == stages) { sn = 0; pn ^= 1; }
                    }
                } else {
                    int b = 0, ph = 0;
                    int sj = 0;                        // stage of key tile j
                    for (int j = 0; j < n_kv && ok; ++j) {
                        ok = mbar_wait(smem_u32(&bar_p_full[0][b]), ph, abort_p, args.status, SITE_G_P, j);
                        if (!ok) break;
                        tc_fence_after_sync();
                        issue_o(j, sj, b);
                        tc_commit(smem_u32(&bar_pv_done[j % SPLIT]));       // the part's O_g holds its key tiles up to j
                        tc_commit(smem_u32(&bar_buf_free[b]));              // buffer b may take new scores
                        tc_commit(smem_u32(&bar_kv_empty[sj]));             // done with K(j), V(j): S(j) completed long ago
                        if (j == n_kv - 1) tc_commit(smem_u32(&bar_o_final[0]));
                        if (++b == NB) { b = 0; ph ^= 1; }
                        if (++sj == stages) sj = 0;
                    }
                }
            }
            bool ok = SPLIT == 1 && mbar_wait(smem_u32(&bar_kv_full[0]), 0, abort_p, args.status, SITE_G_KV, 0) &&
                      mbar_wait(smem_u32(&bar_q_full[t]), 0, abort_p, args.status, SITE_G_Q, t);
            if (ok) {
                // the first T+1 steps fill the buffers: step t (own tile, key tile 0) into buffer t; the last issuer
                // also requests step T (tile 0, key tile 1) into the spare buffer T
                tc_fence_after_sync();
                issue_s(q_desc_own, t, 0, t);   // stage 0
                ok = mbar_wait(smem_u32(&bar_q_full[tn]), 0, abort_p, args.status, SITE_G_Q, tn);
                if (ok && t == T - 1 && n_kv > 1) {
                    ok = mbar_wait(smem_u32(&bar_kv_full[1]), 0, abort_p, args.status, SITE_G_KV, 1);   // stages >= 2
                    if (ok) {
                        tc_fence_after_sync();
                        issue_s(q_desc, tn, 1, T);   // stage 1
                    }
                }
            }
            // own step k = T*j + t: buffer b = k % NB, which tile t meets for the (j / NB)-th time (as in the softmax
            // warps); it requests step k + NB = (tn, jn) into the same buffer
            int b = t, ph = 0, jm = 0;
            const int jn_off = (t + 1 == T) ? 2 : 1;
            int sj = 0;                                 // stage of key tile j
            int sn = jn_off % stages, pn = (jn_off / stages) & 1;   // stage and phase of key tile jn = j + jn_off
            for (int j = 0; j < n_kv && ok; ++j) {
                const int jn = j + jn_off;
                const bool more = jn < n_kv;
                if (more)   // landed long ago: keep this wait off the critical path
                    ok = mbar_wait(smem_u32(&bar_kv_full[sn]), pn, abort_p, args.status, SITE_G_KV, jn);
                // (plain tests first: the hardware's suspension inside try_wait costs this hand-over about 1% of the call)
                if (ok) ok = mbar_wait_eager(smem_u32(&bar_p_full[t][b]), ph, abort_p, args.status, SITE_G_P, j);
                if (!ok) break;
                tc_fence_after_sync();
                issue_o(j, sj, b);
                if (more) issue_s(q_desc, tn, sn, b);               // into the buffer P is read from: behind it, in order
                tc_commit(b_pvdone);                                // O_t holds key tiles 0..j
                tc_commit(smem_u32(&bar_kv_empty[sj]));             // this issuer is done with K(j), V(j)
                if (j == n_kv - 1) tc_commit(smem_u32(&bar_o_final[t]));
                b = (b == 0) ? NB - 1 : b - 1;              // k += NB - 1
                if (++jm == NB) { jm = 0; ph ^= 1; }
                if (++sj == stages) sj = 0;
                if (++sn == stages) { sn = 0; pn ^= 1; }
            }
        }
        __syncwarp();
    }
    // Every asynchronous arrival of this segment has been waited for (see the end of each role), so the barriers can
    // start over for the next one; tensor memory and shared memory simply carry on.
    tc_fence_before_sync();
    __syncthreads();
    if (last_segment || abort_flag) break;
    if (warp == SCHED_WARP) next_segment(true);
    __syncthreads();
    tc_fence_after_sync();
    }   // the next segment of this CTA
    } else {
    setmaxnreg_inc<F4S_SOFTMAX_REGS>();
    for (;;) {
    // ------------------------------------------------------------ the segment: key tiles j0 .. j0 + n_kv - 1 of a unit
    if (!seg_desc[0]) break;
    const int prob_i = seg_desc[1], unit = seg_desc[2], j0 = seg_desc[3], n_kv = seg_desc[4], T = seg_desc[5];
    const bool last_segment = seg_desc[6] != 0;
    const int quad = unit % args.units_per_head, bh = unit / args.units_per_head;
    const Fused4Problem& pr = args.prob[prob_i];
    const int row_base = quad * args.tiles_per_cta * TILE_M;
    const int NB = SPLIT > 1 ? args.split_buffers : T + 1;   // score buffers in the rotation
    {
        // ------------------------------------------------------------ softmax warps
        const int t = warp >> 2;                 // query tile of this warpgroup
        if (SPLIT > 1) {
            // ---- one query tile, SPLIT parts: warpgroup g takes the key tiles j = g, g + SPLIT, ... whole
            const int g = t;
            if (g < SPLIT) {
                const int r = tid & (TILE_M - 1);    // row inside the tile = TMEM lane
                const uint32_t lane_off = (uint32_t)((warp & 3) * 32) << 16;
                const uint32_t tmem_og = tmem_o0 + g * dpad + lane_off;
                const uint32_t b_pvdone = smem_u32(&bar_pv_done[g]);   // products of THIS part's key tiles
                const float c2 = pr.scale_log2e;
                float m_run = 0.f, l_run = 0.f;   // anchor and row sum over this part's keys
                bool ok = true;
                // NB is a multiple of SPLIT, so buffer b = j % NB always meets the same part: one consumer per barrier.
                // The part's i-th key tile uses buffer (g + SPLIT i) % NB, phase ((g + SPLIT i) / NB) & 1.
                int b = g, ph = 0;
                for (int j = g, i = 0; j < n_kv; j += SPLIT, ++i) {
                    const uint32_t tmem_s = tmem_base + b * BN + lane_off;
                    ok = mbar_wait(smem_u32(&bar_s_full[0][b]), ph, abort_p, args.status, SITE_G_S, j);
                    ok = __all_sync(0xffffffffu, ok);
                    if (!ok) break;
                    tc_fence_after_sync();
                    const int valid = args.Nk - (j0 + j) * BN;   // columns >= valid are zero-filled keys
                    uint32_t s[BN];
                    tmem_ld32(tmem_s, &s[0]);
                    tmem_ld32(tmem_s + 32, &s[32]);
                    tmem_wait_ld();
                    const bool ragged = valid < BN;   // only the last key tile can be
                    if (i == 0) {
                        const float row_max = ragged ? row_max_masked<BN>(s, valid) : row_max_bf16<BN>(s);
                        m_run = row_max * c2 + FUSED_HEADROOM_LOG2;
                    }
                    uint32_t packed[BN / 2];
                    float tile_sum;
#pragma unroll 1
                    for (int attempt = 0; attempt < 2; ++attempt) {
                        const float neg_mc = -m_run;
                        if (!ragged) {
                            const uint64_t c2c2 = pack_b64(__float_as_uint(c2), __float_as_uint(c2));
                            const uint64_t nmnm = pack_b64(__float_as_uint(neg_mc), __float_as_uint(neg_mc));
                            uint64_t acc[2] = {0ull, 0ull};
                            exp2_pack_32<POLY, 16, BF>(&s[0], c2c2, nmnm, &packed[0], acc);
                            exp2_pack_32<POLY, 16, BF>(&s[32], c2c2, nmnm, &packed[16], acc);
                            tile_sum = sum_f32x2(acc[0], acc[1]);
                        } else {
                            tile_sum = 0.f;
                            exp2_pack_32_masked<16, BF>(&s[0], c2, neg_mc, 0, valid, &packed[0], tile_sum);
                            exp2_pack_32_masked<16, BF>(&s[32], c2, neg_mc, 32, valid, &packed[16], tile_sum);
                        }
                        const bool over = !(tile_sum <= FUSED_TILE_SUM_LIMIT);
                        if (attempt == 1 || !__any_sync(0xffffffffu, over)) break;
                        // Rare: a score far above the anchor (see the unsplit path below).  O_g may be touched once the
                        // product of this part's previous key tile has completed; nothing of this tile's weights is
                        // stored yet.  The first registers of the row are borrowed for O_g.
                        if (i > 0) {
                            ok = mbar_wait(b_pvdone, (i - 1) & 1, abort_p, args.status, SITE_G_PV, j);
                            ok = __all_sync(0xffffffffu, ok);
                            if (!ok) break;
                            tc_fence_after_sync();
                        }
                        // (the exact maximum: the truncated one may lie below it by more than the headroom)
                        const float row_max = row_max_masked<BN>(s, ragged ? valid : BN);
                        const float m_new = row_max * c2 + FUSED_HEADROOM_LOG2;
                        const float alpha = over ? ex2_approx(m_run - m_new) : 1.f;
                        if (over) m_run = m_new;
                        l_run *= alpha;
                        if (i > 0) {
                            for (int cg = 0; cg < (dpad >> 4); ++cg) {
                                tmem_ld16(tmem_og + cg * 16, *reinterpret_cast<uint32_t(*)[16]>(&s[0]));
                                tmem_wait_ld();
#pragma unroll
                                for (int c = 0; c < 16; ++c) s[c] = __float_as_uint(__uint_as_float(s[c]) * alpha);
                                tmem_st16(tmem_og + cg * 16, *reinterpret_cast<uint32_t(*)[16]>(&s[0]));
                            }
                            tmem_wait_st();
                        }
                        tmem_ld32(tmem_s, &s[0]);
                        tmem_ld32(tmem_s + 32, &s[32]);
                        tmem_wait_ld();
                    }
                    if (!ok) break;
                    l_run += tile_sum;
                    tmem_st32(tmem_s, packed);   // P(j) over the first columns of the buffer, whose scores sit in registers
                    tmem_wait_st();
                    // every phase of the part's completion barrier is consumed in order, one own key tile late: the
                    // product of key tile j - SPLIT has had SPLIT tiles' time to finish
                    if (i > 0) {
                        ok = mbar_wait(b_pvdone, (i - 1) & 1, abort_p, args.status, SITE_G_PV, j);
                        ok = __all_sync(0xffffffffu, ok);
                        if (!ok) break;
                    }
                    tc_fence_before_sync();
                    if (lane == 0) mbar_arrive(smem_u32(&bar_p_full[0][b]));
                    b += SPLIT;
                    if (b >= NB) { b -= NB; ph ^= 1; }
                }
                // ---- combine the parts: o = sum_g 2^(m_g - m) O_g / sum_g 2^(m_g - m) l_g, m = max_g m_g
                part_ml[g][r] = make_float2(m_run, l_run);
                if (ok) ok = mbar_wait(smem_u32(&bar_o_final[0]), 0, abort_p, args.status, SITE_G_O, g);
                ok = named_barrier_and(1, SPLIT * 128, ok);   // every part's (m, l) is in shared memory, every product done
                if (ok) {
                    tc_fence_after_sync();
                    float f[SPLIT];
                    float m_all = -INFINITY, l_all = 0.f;
#pragma unroll
                    for (int p2 = 0; p2 < SPLIT; ++p2)
                        if (part_ml[p2][r].y > 0.f) m_all = fmaxf(m_all, part_ml[p2][r].x);
#pragma unroll
                    for (int p2 = 0; p2 < SPLIT; ++p2) {
                        const float2 ml = part_ml[p2][r];
                        f[p2] = ml.y > 0.f ? ex2_approx(ml.x - m_all) : 0.f;   // a part without keys counts nothing
                        l_all += f[p2] * ml.y;
                    }
                    const float inv = 1.f / l_all;
#pragma unroll
                    for (int p2 = 0; p2 < SPLIT; ++p2) f[p2] *= inv;
                    const int row = row_base + r;
                    __half* orow = head_row(pr.out, args.lay, bh, row);
                    // the column groups of 16 are shared out among the parts; a thread reads its row of every O_p
                    for (int cg = g; cg < (dpad >> 4); cg += SPLIT) {
                        float acc[16];
#pragma unroll
                        for (int c = 0; c < 16; ++c) acc[c] = 0.f;
#pragma unroll
                        for (int p2 = 0; p2 < SPLIT; ++p2) {
                            if (p2 >= n_kv) continue;   // a part without a key tile never wrote its accumulator
                            uint32_t x[16];
                            tmem_ld16(tmem_o0 + p2 * dpad + lane_off + cg * 16, x);
                            tmem_wait_ld();
#pragma unroll
                            for (int c = 0; c < 16; ++c) acc[c] = fmaf(__uint_as_float(x[c]), f[p2], acc[c]);
                        }
                        uint4 lo, hi;
                        lo.x = pack_16x2<BF>(acc[0], acc[1]);   lo.y = pack_16x2<BF>(acc[2], acc[3]);
                        lo.z = pack_16x2<BF>(acc[4], acc[5]);   lo.w = pack_16x2<BF>(acc[6], acc[7]);
                        hi.x = pack_16x2<BF>(acc[8], acc[9]);   hi.y = pack_16x2<BF>(acc[10], acc[11]);
                        hi.z = pack_16x2<BF>(acc[12], acc[13]); hi.w = pack_16x2<BF>(acc[14], acc[15]);
                        if (row < args.Nq) {
                            if (cg * 16 + 8 <= args.d) *reinterpret_cast<uint4*>(orow + cg * 16) = lo;
                            if (cg * 16 + 16 <= args.d) *reinterpret_cast<uint4*>(orow + cg * 16 + 8) = hi;
                        }
                    }
                }
            }
        } else if (t < T) {
            const int r = tid & (TILE_M - 1);    // row inside the tile = TMEM lane
            const uint32_t lane_off = (uint32_t)((warp & 3) * 32) << 16;
            const uint32_t tmem_o = tmem_o0 + t * dpad + lane_off;
            const uint32_t b_pvdone = smem_u32(&bar_pv_done[t]);
            const float c2 = pr.scale_log2e;
            float m_run = 0.f;   // anchor of the exponent: a bound on the running max, times scale*log2(e)
            float l_run = 0.f;   // running sum of p (relative to m_run)
            bool ok = true;
            // step k = T*j + t uses buffer k % NB; k grows by T = NB - 1 per key tile, so the buffer index walks down and
            // tile t meets each buffer every NB key tiles: phase (j / NB) & 1 of that (tile, buffer) barrier pair
            int b = t % NB, ph = 0, jm = 0;
            for (int j = 0; j < n_kv; ++j) {
                const uint32_t tmem_s = tmem_base + b * BN + lane_off;
                ok = mbar_wait(smem_u32(&bar_s_full[t][b]), ph, abort_p, args.status, SITE_G_S, j);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                tc_fence_after_sync();
                const int valid = args.Nk - (j0 + j) * BN;   // columns >= valid are zero-filled keys
                uint32_t s[BN];
                tmem_ld32(tmem_s, &s[0]);
                tmem_ld32(tmem_s + 32, &s[32]);
                tmem_wait_ld();
                const bool ragged = valid < BN;   // only the last key tile can be
                if (j == 0) {
                    const float row_max = ragged ? row_max_masked<BN>(s, valid) : row_max_bf16<BN>(s);
                    m_run = row_max * c2 + FUSED_HEADROOM_LOG2;
                }
                uint32_t packed[BN / 2];
                float tile_sum;
#pragma unroll 1
                for (int attempt = 0; attempt < 2; ++attempt) {
                    const float neg_mc = -m_run;
                    if (!ragged) {
                        const uint64_t c2c2 = pack_b64(__float_as_uint(c2), __float_as_uint(c2));
                        const uint64_t nmnm = pack_b64(__float_as_uint(neg_mc), __float_as_uint(neg_mc));
                        uint64_t acc[2] = {0ull, 0ull};
                        exp2_pack_32<POLY, 16, BF>(&s[0], c2c2, nmnm, &packed[0], acc);
                        exp2_pack_32<POLY, 16, BF>(&s[32], c2c2, nmnm, &packed[16], acc);
                        tile_sum = sum_f32x2(acc[0], acc[1]);
                    } else {
                        tile_sum = 0.f;
                        exp2_pack_32_masked<16, BF>(&s[0], c2, neg_mc, 0, valid, &packed[0], tile_sum);
                        exp2_pack_32_masked<16, BF>(&s[32], c2, neg_mc, 32, valid, &packed[16], tile_sum);
                    }
                    const bool over = !(tile_sum <= FUSED_TILE_SUM_LIMIT);
                    if (attempt == 1 || !__any_sync(0xffffffffu, over)) break;
                    // Rare: a row of this warp met a score far above its anchor.  O_t may be touched once the P V
                    // product of key tile j-1 has completed (that of j-2 has: see the wait before the hand-off below);
                    // nothing of P_t(j) has been stored yet, so the scores are still in tensor memory.  The first
                    // registers of the row are borrowed for O_t.
                    if (j > 0) {
                        ok = mbar_wait(b_pvdone, (j - 1) & 1, abort_p, args.status, SITE_G_PV, j);
                        ok = __all_sync(0xffffffffu, ok);
                        if (!ok) break;
                        tc_fence_after_sync();
                    }
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
                if (!ok) break;
                l_run += tile_sum;
                tmem_st32(tmem_s, packed);   // P_t(j) over the first columns of the buffer, whose scores sit in registers
                tmem_wait_st();
                // A parity wait is only sound while the waiter is at most one phase behind.  The scores of this tile
                // are requested by ANOTHER issuer than the one that multiplies P_t V, so nothing else orders this
                // warp against its own tile's products: it consumes every phase of pv_done here, before it hands
                // P_t(j) over (P V(j) cannot complete earlier), when P V(j-1) has had a whole step to finish.
                if (j > 0) {
                    ok = mbar_wait(b_pvdone, (j - 1) & 1, abort_p, args.status, SITE_G_PV, j);
                    ok = __all_sync(0xffffffffu, ok);
                    if (!ok) break;
                }
                tc_fence_before_sync();
                if (lane == 0) mbar_arrive(smem_u32(&bar_p_full[t][b]));
                b = (b == 0) ? NB - 1 : b - 1;              // k += NB - 1
                if (++jm == NB) { jm = 0; ph ^= 1; }
            }
            if (ok) ok = mbar_wait(smem_u32(&bar_o_final[t]), 0, abort_p, args.status, SITE_G_O, t);
            // (the last phase of the product barrier, never consumed above: nothing of this segment is in flight after it)
            if (ok) ok = mbar_wait(b_pvdone, (n_kv - 1) & 1, abort_p, args.status, SITE_G_PV, n_kv);
            ok = __all_sync(0xffffffffu, ok);
            const int row = row_base + t * TILE_M + r;
            __half* orow = head_row(pr.out, args.lay, bh, row);
            if (ok && j0 == 0 && n_kv == n_kv_all) {   // all key tiles of the unit: no pieces to combine
                tc_fence_after_sync();
                const float inv = 1.f / l_run;
                for (int g = 0; g < (dpad >> 4); ++g) {
                    uint32_t x[16];
                    tmem_ld16(tmem_o + g * 16, x);
                    tmem_wait_ld();
                    uint4 lo, hi;
                    lo.x = pack_16x2<BF>(__uint_as_float(x[0]) * inv, __uint_as_float(x[1]) * inv);
                    lo.y = pack_16x2<BF>(__uint_as_float(x[2]) * inv, __uint_as_float(x[3]) * inv);
                    lo.z = pack_16x2<BF>(__uint_as_float(x[4]) * inv, __uint_as_float(x[5]) * inv);
                    lo.w = pack_16x2<BF>(__uint_as_float(x[6]) * inv, __uint_as_float(x[7]) * inv);
                    hi.x = pack_16x2<BF>(__uint_as_float(x[8]) * inv, __uint_as_float(x[9]) * inv);
                    hi.y = pack_16x2<BF>(__uint_as_float(x[10]) * inv, __uint_as_float(x[11]) * inv);
                    hi.z = pack_16x2<BF>(__uint_as_float(x[12]) * inv, __uint_as_float(x[13]) * inv);
                    hi.w = pack_16x2<BF>(__uint_as_float(x[14]) * inv, __uint_as_float(x[15]) * inv);
                    if (row < args.Nq) {
                        if (g * 16 + 8 <= args.d) *reinterpret_cast<uint4*>(orow + g * 16) = lo;
                        if (g * 16 + 16 <= args.d) *reinterpret_cast<uint4*>(orow + g * 16 + 8) = hi;
                    }
                }
            } else if (ok) {
                // ---- a piece of the unit's key range: (O, anchor, row sum) of the thread's row to the scratch.  A CTA
                // has at most two pieces per problem (its first segment may begin and its last may end inside a
                // unit): slot 0 for one that begins inside a unit, slot 1 for one that begins a unit.
                tc_fence_after_sync();
                float* piece = args.part + ((2 * (size_t)prob_i * gridDim.x + 2 * (size_t)blockIdx.x + (j0 > 0 ? 0 : 1)) * args.part_slot_floats) +
                               (size_t)t * (dpad + 2) * TILE_M + r;
                f4s_store_piece(piece, tmem_o, dpad, m_run, l_run);
                named_barrier(2 + t, TILE_M);
                if (r == 0) {   // the counter's answer is looked at behind the barrier that ends the segment
                    piece_ticket[t][0] = atomicAdd(args.part_count + ((size_t)prob_i * args.n_units + unit) * F4_TILES + t, 1);
                    piece_ticket[t][1] = prob_i;
                    piece_ticket[t][2] = unit;
                    piece_ticket[t][3] = 1;
                }
            }
        }
    }
    // Every asynchronous arrival of this segment has been waited for (see the end of each role), so the barriers can
    // start over for the next one; tensor memory and shared memory simply carry on.
    tc_fence_before_sync();
    __syncthreads();
    if (SPLIT == 1 && !abort_flag) combine_if_last(warp >> 2);
    if (last_segment || abort_flag) break;
    if (warp == SCHED_WARP) next_segment(true);
    __syncthreads();
    tc_fence_after_sync();
    }   // the next segment of this CTA
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
