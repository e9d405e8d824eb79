// Constants and launch arguments of the fused single-pass attention kernel (fused4s_kernel.cuh).
#pragma once
#include <cuda.h>

#include "cross_kernel.cuh"  // TILE_M, CHUNK_COLS, CHUNK_ROW_BYTES
#include "softmax_math.cuh"
#include "tc_common.cuh"

namespace sd_attn {

// The exponent of a row is anchored FUSED_HEADROOM_LOG2 above the maximum of the row's first key tile (weights
// <= 2^-6: the eight binades below that are still normal binary16, and what lies further down rounds without
// bias).  No per-tile maximum is taken afterwards: a later tile is evaluated against the anchor as it stands, and
// only when its weights sum to more than FUSED_TILE_SUM_LIMIT (so no weight exceeds it: 2^12 is far inside
// binary16's range) is that tile's maximum taken, the accumulator and the row sum rescaled and the tile redone.
// Any anchor gives the same result in exact arithmetic.  Measured on the "peaked" inputs: headroom 3 re-anchors
// about one warp-tile in 130 and costs 3.5% of the 4096-token call; headroom 6 re-anchors almost never, with the
// same error.
constexpr float FUSED_HEADROOM_LOG2 = 6.0f;
constexpr float FUSED_TILE_SUM_LIMIT = 4096.0f;

constexpr int F4_TILES = 4;           // query tiles of 128 rows per CTA, at most
constexpr int F4_BN = 64;             // keys per key tile
constexpr int F4_THREADS = 24 * 32;   // 16 softmax warps + 8 control warps (producer, 4 issuers, 3 idle)
constexpr int F4_STAGES = 8;          // K/V ring depth, at most

constexpr int F4_GROUP_MAX = 8;       // problems of one shape per launch (the parameter block stays under 4 KB)

struct Fused4Problem {   // one problem of a launch
    CUtensorMap tq, tk, tv;
    __half* out;         // [BH][Nq][d], or as Fused4Args::lay says
    float scale_log2e;   // |scale| * log2(e)
    int negate;          // scale < 0: the tensor core negates Q
};

struct Fused4Args {
    Fused4Problem prob[F4_GROUP_MAX];
    HeadLayout lay;
    int n_prob, BH;      // problems in this launch; (batch, head) pairs of each
    int Nq, Nk, d;
    int dpad;            // d rounded up to 16
    int tiles_per_cta;   // 1..4 query tiles per unit (small problems spread over more SMs)
    int units_per_head;  // ceil(query tiles of a head / tiles_per_cta)
    int n_units;         // units of ONE problem: BH * units_per_head
    int shares;          // 0: one CTA per (problem, unit); 1: every CTA takes a share of every problem's steps
    int n_kv;            // key tiles: ceil(Nk / 64)
    int nch;             // 64-column chunks per row (1..3)
    int stages;          // K/V ring depth (2..8)
    int split_buffers;   // split variant only: score buffers of the lone tile (2..5)
    int* status;
    // pieces of units whose key tiles are cut between CTAs (shares only): per problem two slots of part_slot_floats
    // per CTA, each [tile][dpad + 2 columns: O, anchor, row sum][128 rows]; arrival counters per (problem, unit,
    // tile), zero between launches
    float* part;
    int* part_count;
    int part_slot_floats;
};

// wait sites reported in the device status block
enum { SITE_G_Q = 30, SITE_G_KV = 31, SITE_G_EMPTY = 32, SITE_G_S = 33, SITE_G_P = 34, SITE_G_O = 35, SITE_G_PV = 37 };

}  // namespace sd_attn
