// Internal declarations shared by the translation units of libmint_lora.so.
// Nothing here is part of the C ABI.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "mint_lora.h"

namespace mint {
constexpr int kRankCapHost = 128;  // largest slot rank any kernel here handles
}

// ---- plan blob ------------------------------------------------------------
// Header words (int32) at the start of the plan blob.
enum {
  PH_MAGIC = 0,
  PH_T,
  PH_K,
  PH_NUM_ITEMS,
  PH_NUM_SLOTS,
  PH_NUM_EXPERTS,
  PH_NUM_ACTIVE,
  PH_NUM_SEGMENTS,
  PH_MAX_SEGMENT,
  PH_SUM_RANK,
  PH_NOT_RESIDENT,
  PH_BAD_EXPERT,
  PH_GEN_LO,
  PH_GEN_HI,
  PH_NCHUNK0,   // number of tiles in list g (MINT_NUM_TILE_LISTS entries)
  PH_NCHUNK1,
  PH_LANES,     // number of cost lanes G the lane tables were cut for
  PH_ROWS_SHRINK,  // sum over list-1 tiles of mint_tile_rows_shrink
  PH_ROWS_EXPAND,  // sum over list-1 tiles of mint_tile_rows_expand
  PH_MAX_TILE_ROWS,  // largest mint_tile_rows_shrink of a list-1 tile that the streamed shrink handles
  PH_NUM_DENSE,      // number of 128-row tiles of dense segments (tensor-core kernels)
  PH_NUM_SCATTERED,  // how many of them hold tokens that are not consecutive rows (listed as ~tile in dense_tile)
  PH_WORDS = 32
};
#define MINT_PLAN_MAGIC 0x4D4C5032  // "MLP2"
#define MINT_NUM_TILE_LISTS 2
#define MINT_MAX_LANES 1024
// Tile list g cuts every segment into runs of at most mint_tile_tokens(g) items.
// In list 1, the list of the streamed kernels, the segments of rank-1 adapters
// (other than dense segments) are cut into runs of 8 instead: a rank-1 tile of
// up to 8 tokens takes the FMA path, which costs a fraction of what a tensor-core
// tile of rank 1 costs (one useful column in eight), for one more read of the
// single row of A and of B per 8 tokens.
__host__ __device__ constexpr int mint_tile_tokens(int g) { return g == 0 ? 8 : 32; }
__host__ __device__ constexpr int mint_tile_tokens_rank1(int g) { return 8; }

// Cost of a tile per column block, in rows of streamed bytes: the rows it moves
// (rank + len for the shrink, rank + 2 len for the expand: y is read and
// written) plus a constant for what a block costs whatever its height (an
// iteration of a warp waits for memory once, and narrow tiles do not fill the
// tensor-core shapes).  The lanes' shares are equal in this cost.
#define MINT_TILE_COST_SHRINK 8
#define MINT_TILE_COST_EXPAND 8
// Tiles of rank 1 with at most 8 tokens take the FMA path: a row costs less there, but a
// piece of such a tile costs its latencies whatever its size (measured per piece and per block).
__host__ __device__ constexpr int mint_tile_rows_shrink(int rank, int len) {
  return (rank == 1 && len <= 8) ? 5 + len : rank + len + MINT_TILE_COST_SHRINK;
}
__host__ __device__ constexpr int mint_tile_rows_expand(int rank, int len) {
  return (rank == 1 && len <= 8) ? 4 + len : rank + 2 * len + MINT_TILE_COST_EXPAND;
}

// One tile of list 1 with everything a streaming kernel needs to start on it:
// no dependent lookups through segment or slot arrays.  rank and scale are the
// slot's values when the plan was made (the plan's generation guards them).
// rows_shrink / rows_expand are the exclusive prefix sums, over tiles, of
// (rank + len) and (rank + 2 len): the row counts whose product with a
// projection's width gives the bytes the shrink and the expand stream.
// lane_lo..lane_hi bound the shrink lanes (of the plan's G) whose share can
// meet this tile: the lanes j with  rows_shrink - W/G < j W/G < rows_shrink + rank + len.
struct __align__(16) TileDesc {
  int32_t off;     // first position of the tile in perm
  int32_t len;     // 1..32 items
  int32_t slot;
  int32_t expert;  // 0 for dense plans
  int32_t rank;
  float scale;
  int32_t rows_shrink;
  int32_t rows_expand;
  int32_t lane_lo;
  int32_t lane_hi;
  int32_t dense;   // 1: the tile belongs to a dense segment; it runs on the 128-row tensor-core kernels
  int32_t pad1;
};

// A batch of at least MINT_DENSE_MIN_BATCH items may hold dense segments: runs of
// at least MINT_DENSE_MIN_SEGMENT items of one adapter (segmented prefill).  Their
// shrink (the d -> r contraction over 128-row tiles) runs on the tcgen05 kernel;
// the plan excludes their tiles from the streamed shrink's area and lists the
// 128-row tiles (every fourth 32-item tile of such a segment) in dense_tile.
#define MINT_DENSE_MIN_BATCH 4096
#define MINT_DENSE_MIN_SEGMENT 128
// The tensor-core shrink splits a wide d over up to MINT_DENSE_SPLIT_MAX CTAs per
// tile (one per MINT_DENSE_SPLIT_COLUMNS columns); part s of the v of dense tile t is
// workspace slot  dense_slot0 + s * tiles_ub + t,  and the tensor-core expand adds the parts.
#define MINT_DENSE_SPLIT_MAX 4
#define MINT_DENSE_SPLIT_COLUMNS 5120
__host__ __device__ constexpr int mint_dense_splits(int d) {
  return d / MINT_DENSE_SPLIT_COLUMNS < 1 ? 1
         : (d / MINT_DENSE_SPLIT_COLUMNS > MINT_DENSE_SPLIT_MAX ? MINT_DENSE_SPLIT_MAX : d / MINT_DENSE_SPLIT_COLUMNS);
}

// Start of cost lane j in the rows x column-blocks area: the tile that holds it
// and j * rows_total = q * G + r, so that the position for CB column blocks is
// q * CB + r * CB / G without any 64-bit division.
// rows / w: the row prefix sum and the row count of that tile, so that a lane
// finds its first column block without reading the tile's descriptor.
struct __align__(16) LaneStart {
  int32_t tile;
  int32_t q;
  int32_t r;
  int32_t rows;
  int32_t w;
  int32_t pad[3];
};

// Byte offsets of every array inside the plan blob (host-computed, passed by value).
struct PlanOffsets {
  int64_t header;      // int32[PH_WORDS]
  int64_t perm;        // int32[P]        item indices grouped by key (inactive items after the active ones)
  int64_t seg_start;   // int32[P+1]
  int64_t seg_key;     // int32[P]
  int64_t seg_slot;    // int32[P]
  int64_t seg_expert;  // int32[P]
  int64_t tile_seg[MINT_NUM_TILE_LISTS];  // int32[P]  segment of tile c
  int64_t tile_off[MINT_NUM_TILE_LISTS];  // int32[P]  first position (in perm) of tile c
  int64_t tile_desc;   // TileDesc[tile upper bound of list 1]
  int64_t dense_tile;  // int32[tile upper bound of list 1]  first list-1 tile c of every 128-row dense tile (~c: its tokens are scattered)
  int64_t lane_shrink; // LaneStart[MINT_MAX_LANES + 1]  start of cost lane j in the shrink rows
  int64_t lane_expand; // LaneStart[MINT_MAX_LANES + 1]  same for the expand rows
  int64_t key_a, key_b, idx_a, idx_b;     // int32[P]  radix-sort ping-pong scratch
  int64_t cta_hist;    // int32[16 + (ctas + 4) * (key_space + 1)]  counters, per-CTA key counts and per-key starts, segment and first tiles of the grid-wide sort
                       // (only when mint_plan_presort_ctas(P, key_space) > 0)
  int64_t total;
};
// Batches of many items over a small key space are sorted by a counting sort that runs on one CTA per
// 1024 items (three short kernels) before the single-CTA plan kernel derives the rest; returns the
// number of those CTAs, or 0 when the plan kernel sorts by itself.
int32_t mint_plan_presort_ctas(int64_t P, int64_t key_space);
PlanOffsets mint_plan_offsets(int64_t P, int64_t key_space);
// Upper bound on the number of tiles of list g, computable without reading the plan.
int64_t mint_tile_upper_bound(int g, int64_t P, int64_t key_space);

// Device view of a plan: typed pointers into the blob.
struct PlanView {
  const int32_t *header;
  const int32_t *perm;
  const int32_t *seg_start;
  const int32_t *seg_key;
  const int32_t *seg_slot;
  const int32_t *seg_expert;
  const int32_t *tile_seg[MINT_NUM_TILE_LISTS];
  const int32_t *tile_off[MINT_NUM_TILE_LISTS];
  const TileDesc *tile_desc;
  const int32_t *dense_tile;
  const LaneStart *lane_shrink;
  const LaneStart *lane_expand;
};
PlanView mint_plan_view(const void *plan_dev, int64_t P, int64_t key_space);
// Number of cost lanes plans are cut for on the current device (three per SM).
int32_t mint_device_lanes(int32_t *lanes_out);
// A plan, bind or evict kernel was enqueued: the next apply must not start before it has
// completed (an apply kernel reads the plan and the slot table before its dependency wait), so
// its first kernel is launched without programmatic stream serialization.  take returns the
// mark and clears it.
void mint_mark_tables_changed();
bool mint_take_tables_changed();

// ---- host handles ----------------------------------------------------------
struct mint_pool {
  mint_pool_desc desc;
};

struct SlotBinding {
  int64_t catalog_id;  // -1 = empty
  int32_t rank;
  float scale;
};

struct mint_slot_table {
  int64_t catalog_size;
  int32_t num_slots;
  int32_t *id_to_slot_dev;
  int32_t *slot_rank_dev;
  float *slot_scale_dev;
  int64_t generation;
  int32_t max_rank;          // largest rank currently bound
  int32_t *id_to_slot_host;  // mirror [catalog_size]
  SlotBinding *slots_host;   // mirror [num_slots]
};

// ---- error reporting --------------------------------------------------------
int32_t mint_fail(int32_t code, const char *fmt, ...);
int32_t mint_check_cuda(cudaError_t e, const char *what);

// ---- kernel launchers (each returns MINT_OK or MINT_ERR_CUDA) ---------------
struct TableDev {
  const int32_t *id_to_slot;
  const int32_t *slot_rank;
  const float *slot_scale;
  int64_t catalog_size;
  int32_t num_slots;
  int32_t gen_lo, gen_hi;
};

int32_t mint_launch_plan(const TableDev &tab, const int64_t *ids, int32_t T, const int32_t *expert_ids,
                         int32_t K, int32_t num_experts, int32_t lanes, void *plan_dev, int32_t *status,
                         cudaStream_t stream);

struct DenseArgs {
  const uint16_t *A;   // [slot][r_max][d]
  const uint16_t *B;   // [slot][r_max][n]
  int32_t d, n, r_max, num_slots;
  int32_t T;
  const uint16_t *x;
  int64_t ldx;
  uint16_t *y;
  int64_t ldy;
  float *v;            // [T][r_max] (unfused calls)
  int32_t *status;
};
int32_t mint_launch_shrink(const DenseArgs &a, const TableDev &tab, const void *plan_dev, cudaStream_t s);
int32_t mint_launch_expand(const DenseArgs &a, const TableDev &tab, const void *plan_dev, cudaStream_t s);
int32_t mint_launch_fused(const DenseArgs &a, const TableDev &tab, const void *plan_dev, cudaStream_t s);

// Streamed fused path (per-warp cp.async rings + warp MMA) for ranks up to 64: one
// shrink and one expand launch cover up to 8 projections that share a plan.
bool mint_stream_supported(int32_t max_bound_rank);
size_t mint_stream_workspace_bytes(int32_t T, int32_t num_slots, int32_t r_max);
// Tensor-core shrink of the dense segments' 128-row tiles (between the two streamed kernels).
// withhold_for_selftest: the kernel issues no tensor-core work and signals none of its barriers, and its
// waits give up after 2 ms: every CTA with a tile reports MINT_ERR_TIMEOUT and writes nothing.
int32_t mint_launch_dense_shrink(const DenseArgs *args, int nprob, const TableDev &tab, const void *plan_dev,
                                 void *const *workspaces, int32_t lanes, int32_t dense_slot0, int32_t dense_stride,
                                 cudaStream_t s, bool withhold_for_selftest = false);
// Tensor-core expand of the same tiles (after the streamed expand, which skips them).
int32_t mint_launch_dense_expand(const DenseArgs *args, int nprob, const TableDev &tab, const void *plan_dev,
                                 void *const *workspaces, int32_t lanes, int32_t dense_slot0, int32_t dense_stride,
                                 cudaStream_t s);
int32_t mint_launch_stream(const DenseArgs *args, int nprob, const TableDev &tab, const void *plan_dev,
                           void *const *workspaces, cudaStream_t s);

// Weight gradients of up to 16 pool tensors in one launch:
//   out[slot][k][:] += scale_slot * sum over the slot's tokens of coef[t][k] * act[t][:]
// for the rank rows k of the slot (the padding rows are not touched).
struct GradJobHost {
  const float *coef;      // [T][r_max] fp32, token order
  const uint16_t *act;    // [T][ld] bf16
  int64_t ld;
  float *out;             // [slots][r_max][width] fp32 (MoE: [slots][experts][r_max][width], or packed
                          // [slots][experts][width][r_max])
  int32_t width, r_max;
  const int32_t *row_map = nullptr;   // MoE: row of act that pair p reads (nullptr: p)
  int64_t act_rows = 0;               // rows of act (0: not checked)
  int32_t packed = 0;
};
// dx[p, :] += scale * u[p, :] . A[slot][expert]^T over the pairs of a MoE plan (A packed [slot][E][d][r_max])
int32_t mint_launch_moe_dx(const uint16_t *A, const float *u, uint16_t *dx, int64_t lddx, int32_t d, int32_t r_max,
                           int32_t T, int32_t K, int32_t E, const TableDev &tab, const void *plan_dev,
                           int32_t *status, cudaStream_t s);
// K, E: items per token and experts of the plan (1, 0 for dense plans)
int32_t mint_launch_grad_weights(const GradJobHost *jobs, int njobs, int32_t T, const TableDev &tab,
                                 const void *plan_dev, int32_t *status, cudaStream_t s, int32_t K = 1, int32_t E = 0);

// x . A^T of up to 8 problems as tensors v_out[i] ([T][r_max] fp32, token order) through the streamed shrink
// (bound ranks up to 64).  Entries of tokens without an adapter and of ranks at or above a slot's rank are
// not written.
int32_t mint_launch_stream_shrink_v(const DenseArgs *args, int nprob, const TableDev &tab, const void *plan_dev,
                                    void *const *workspaces, float *const *v_out, cudaStream_t s);
// The same launcher by phases: bit 0 of `phases` = the shrink (v_out, when given, receives x . A^T in token
// order), bit 1 = the expand.  The expand alone relies on the parts that an earlier shrink-only call with
// the same problems, plan and workspaces left in the workspaces.
int32_t mint_launch_stream_phases(const DenseArgs *args, int nprob, const TableDev &tab, const void *plan_dev,
                                  void *const *workspaces, cudaStream_t s, int phases, float *const *v_out);

// MoE apply on the streamed kernels (pool r_max of 8, 16, 32 or 64; bound ranks up to 64).
bool mint_stream_moe_supported(int32_t r_max, int32_t max_bound_rank);
size_t mint_stream_moe_workspace_bytes(int64_t pairs, int64_t key_space, int32_t r_max);

struct MoEArgs {
  const uint16_t *A;   // [slot][E][d][r_max]
  const uint16_t *B;   // [slot][E][r_max][n]
  int32_t d, n, r_max, num_slots, num_experts;
  int32_t T, K;
  const uint16_t *x;
  int64_t ldx, x_rows;
  const int32_t *x_row;
  const float *pair_weight;
  uint16_t *y;
  int64_t ldy;
  int32_t *status;
};
int32_t mint_launch_moe(const MoEArgs &a, const TableDev &tab, const void *plan_dev, cudaStream_t s);
// nprob problems that share the plan, the row map and the pair weights (args[0]'s are used)
int32_t mint_launch_stream_moe(const MoEArgs *args, int nprob, const TableDev &tab, const void *plan_dev,
                               void *const *workspaces, cudaStream_t s);
// v_out[i] ([T*K][r_max] fp32, pair order) = routing weight times the pair's x row times A[slot][expert];
// rank_major: the tensors behind args[i].A are stored [slot][expert][r_max][d] and row p of x belongs to pair p.
int32_t mint_launch_stream_moe_shrink_v(const MoEArgs *args, int nprob, bool rank_major, const TableDev &tab,
                                        const void *plan_dev, void *const *workspaces, float *const *v_out,
                                        cudaStream_t s);

int32_t mint_launch_table_init(int32_t *id_to_slot, int64_t catalog_size, int32_t *slot_rank,
                               float *slot_scale, int32_t num_slots, cudaStream_t s);
struct BindBatch {
  static constexpr int kMax = 128;
  int32_t count;
  int64_t id[kMax];
  int32_t slot[kMax];   // -1 = evict (id unbound; slot in old_slot emptied)
  int32_t old_slot[kMax];
  int32_t rank[kMax];
  float scale[kMax];
};
int32_t mint_launch_bind(int32_t *id_to_slot, int32_t *slot_rank, float *slot_scale,
                         const BindBatch &batch, cudaStream_t s);
