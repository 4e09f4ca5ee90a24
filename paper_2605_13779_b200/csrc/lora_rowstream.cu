// Streamed LoRA apply: the fused path of mint_lora_apply_fused, of its grouped
// form and (with the packed per-expert layout) of mint_moe_lora_apply.
//
//   shrink_rows_kernel : v[tile] = X[tile rows, :] . A_slot           (d -> r)
//   expand_rows_kernel : Y[tile rows, :] += s_slot * v[tile] . B_slot  (r -> n)
//
// Work split.  The work of a call is the area  rows x column blocks  where
// rows runs over the plan's tiles (a tile = at most 32 tokens of one segment)
// and columns over the column blocks (32 elements of d for the shrink, 64
// elements of n for the expand) of all projections of the call, laid side by
// side.  A tile counts as many rows as a column block of it costs
// (mint_tile_rows_shrink / _expand), and every projection's columns are
// preceded by a few empty blocks that stand for the fixed cost of starting on a
// (tile, projection) piece.  The grid is two CTAs per SM ("lanes"); lane c
// takes the c-th equal share of the area, walked tile by tile: a share starts
// in the middle of one tile, covers whole tiles, and ends in the middle of
// another.  The plan tabulates the tile in which every lane starts.
//
// Data path.  Everything a piece streams is a set of rows that are contiguous
// in memory: token rows of x (or y) and the slot's rows of A (or B).  A CTA is
// one producer warp and four consumer warps around a ring of shared-memory
// stages.  The producer walks the lane's share piece by piece and fills stage
// after stage: a stage holds the same run of columns of every row of the piece
// (the fewer rows, the longer the run), and every row segment is ONE bulk
// asynchronous copy (cp.async.bulk, 128 bytes to 2 KB) that signals the stage's
// mbarrier with its byte count.  The producer never waits for the consumers
// except for a free stage, so the memory pipeline runs on across piece
// boundaries, through the hand-over of v and through every barrier of the
// consumers.  The consumers take the stages in order: operand fragments of the
// warp-level tensor-core MMA (m16n8k16, bf16 in, fp32 accumulate) come out of
// the stage with ldmatrix (rows beyond the tile's length or the slot's rank
// are never copied: their fragment rows repeat the last real row, and the
// outputs they feed are never stored), the four warps split the stage's
// columns.  Rows are padded by 16 bytes in the stage so that the eight rows of
// an ldmatrix fall into different banks.
//  - shrink: accumulators stay in registers over all stages of a piece; at its
//    end the four warps' sums are added in warp order through shared memory and
//    the [len][rank] result goes to the lane's slot of the workspace.
//  - expand: at the start of a piece the consumers add the shrink lanes' parts
//    of v (times the pair weight in a MoE call) and turn them into MMA operand
//    fragments, bf16 head plus bf16 remainder (two MMAs carry about 16
//    significant bits of the fp32 shrink result) while the producer is already
//    filling stages.  y of a stage is updated in shared memory (one fp32 fma of
//    scale and accumulator onto y, one round-to-nearest-even) and written back
//    with 128-bit stores that cover whole sectors.
//  - tiles of rank 1 with at most 8 tokens (most of a large-catalog decode
//    batch) skip the MMA: plain fp32 FMAs.
//  - packed MoE pools store A as [d][r_max]: the rows of a run of columns of d
//    are one contiguous block, copied with a single bulk copy and read with
//    transposing ldmatrix.
//
// v travels from the shrink to the expand through a small L2-resident
// workspace: every shrink lane writes the sum over its own columns of a tile
// (slot tile + lane, so no two writers meet), and the expand, which knows the
// shrink's split from the same arithmetic, adds the lanes of a tile in lane
// order.  No atomics, no fences, and the result does not depend on scheduling.
//
// Every wait on an mbarrier is bounded (about a second); a wait that runs out
// records MINT_ERR_TIMEOUT, tells the other warps of the CTA to stop, and the
// producer waits (bounded again) for its copies in flight before it returns.
//
// Launch overlap: both kernels let their successor become resident at once
// (griddepcontrol.launch_dependents first thing) and are launched with
// programmatic stream serialization.  Everything a kernel reads before its
// dependency wait is the plan, the slot table and, as L2 prefetches only, pool
// weights; activations, y and v are touched only after the wait, and every CTA
// executes the wait before it exits so that completion stays transitive along
// the stream.
#include <algorithm>
#include <atomic>

#include "mint_device.cuh"

using namespace mint;

namespace {

constexpr int kConsumerWarps = 4;
constexpr int kConsumers = kConsumerWarps * 32;
constexpr int kThreads = kConsumers + 32;   // + the producer warp
constexpr int kCtasPerSm = 2;
constexpr int kStages = 6;
constexpr int kStageBytes = 14336;
constexpr int kMaxRun = 1024;             // longest run of columns of a stage
constexpr int kTileRowsMax = 32;          // plan tile list 1
constexpr int kStreamRankCap = 64;        // larger ranks take the CUDA-core cluster kernel
constexpr int kBatchTiles = 16;           // tile descriptors the producer stages at a time
constexpr int kBatchItems = kBatchTiles * kTileRowsMax;
constexpr int kShrinkBlock = 32;          // elements of d per column block
constexpr int kExpandBlock = 64;          // elements of n per column block
constexpr int kShrinkGrain = 128;         // smallest lane share in (row x block) units: 128 x 64 B
constexpr int kExpandGrain = 64;          //                                           64 x 128 B
// What starting on a (tile, projection) costs a lane, in column blocks of that tile.  Every projection's
// columns are preceded by this many empty blocks in the area.
constexpr int kShrinkPieceBlocks = 32;
constexpr int kExpandPieceBlocks = 16;
constexpr int kMaxParts = 8;              // shrink lanes that may share one tile of one projection
constexpr int kMaxProblems = MINT_MAX_GROUP;

struct StreamProblem {
  const uint16_t *A;   // [slot][r_max][d]; packed MoE pools: [slot][expert][d][r_max]
  const uint16_t *B;   // [slot][r_max][n];                   [slot][expert][r_max][n]
  const uint16_t *x;
  uint16_t *y;
  int64_t ldx, ldy;
  int32_t d, n, r_max;
  int32_t cb0_shrink, cb0_expand;  // first virtual column block of this problem
  float *ws_part;      // slots of 32 * r_max floats: slot (tile + lane): that lane's sum, [len][rank] packed;
                       // slot (dense_slot0 + s * tiles_ub + tile): part s of the v of a dense segment's tile
};

struct StreamParams {
  StreamProblem prob[kMaxProblems];
  int32_t nprob;
  int32_t T;
  int32_t K;                          // items per token: 1, or the routed experts per token of a MoE plan
  int32_t num_experts;                // 0 for dense projections
  int32_t weights_per_slot;           // weight blocks per slot: 1, or the number of experts
  const int32_t *x_row;               // MoE: row of x that pair p reads (nullptr: p)
  const float *pair_weight;           // MoE: weight of pair p (nullptr: 1)
  int64_t x_rows;                     // MoE: rows of x (range check of x_row)
  int32_t lanes;                      // cost lanes G the plan's lane tables were cut for
  int32_t cb_shrink, cb_expand;       // virtual column blocks of the whole call
  int32_t cb_shrink_widest;           // column blocks of the widest d of the call
  int32_t dense_slot0;                // first workspace slot of the dense segments' tiles (slot dense_slot0 + tile)
  int32_t *status;
  TableDev tab;
  PlanView pv;
};

// What the producer tells the consumers about a stage.
enum { kStageData = 0, kStageEnd = 1 };
enum { kFlagFirst = 1, kFlagLast = 2 };
struct __align__(16) StageHdr {
  int32_t kind;
  int32_t tile;        // plan tile: the part of v goes to / comes from workspace slot tile + lane
  int32_t prob;
  int32_t col0;        // first column of d (shrink) or n (expand) in the stage
  int32_t ncols;       // columns in the stage (a multiple of 8)
  int32_t pitch;       // bytes between consecutive rows of the stage
  int32_t rank, len;
  int32_t flags;       // first / last stage of the piece
  float scale;
  int32_t lane_lo, lane_hi, rows_shrink;   // the tile's place in the shrink's area (the expand looks up the lanes)
  int32_t w_off;       // byte offset of the first weight row (token rows start at 0)
  int32_t pad[2];
  int32_t rows[kTileRowsMax];   // expand: the rows of y
};

struct Smem {
  uint64_t full[kStages];
  uint64_t empty[kStages];
  uint64_t cbar;                          // barrier of the consumer warps (bounded, unlike bar.sync)
  int32_t abort_flag;
  int32_t range[4];
  int32_t pad0[1];
  StageHdr hdr[kStages];
  TileDesc pdesc[kBatchTiles];            // the producer's batch of tile descriptors
  int32_t prows[kBatchItems];             // and of row indices
  union {
    float scratch[kConsumerWarps * 2 * 4 * 128];   // shrink: [warp][m-tile][n-tile][lane][4] MMA fragments
    struct {
      uint4 vfrag[2 * 4 * 2 * 32];        // expand: v as MMA A fragments [m-tile][k-step][head/remainder][lane]
      float vsum[kTileRowsMax * kStreamRankCap];   // v of the current tile, [len][rank], weighted
    } e;
  } u;
  __align__(128) uint8_t ring[kStages * kStageBytes];
};

// ---- small device helpers ------------------------------------------------------
__device__ __forceinline__ void pdl_launch_dependents() {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ uint32_t smem_addr(const void *p) {
  return (uint32_t)__cvta_generic_to_shared(p);
}
// Asks L2 for a whole run of bytes with one instruction (16-byte aligned, a multiple of 16 bytes).
__device__ __forceinline__ void prefetch_l2_bulk(const void *p, uint32_t bytes) {
  asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(p), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_init(uint64_t *bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void fence_mbar_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void mbar_arrive(uint64_t *bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_addr(bar)) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t *bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ uint64_t global_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}
__device__ __forceinline__ bool mbar_try(uint32_t a, uint32_t parity) {
  uint32_t done;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(done)
      : "r"(a), "r"(parity)
      : "memory");
  return done != 0;
}
// Bounded wait for the phase with the given parity: false after about a second, or as soon as
// another warp of the CTA has given up.
__device__ __forceinline__ bool mbar_wait(uint64_t *bar, uint32_t parity, const volatile int32_t *abort_flag) {
  const uint32_t a = smem_addr(bar);
  if (mbar_try(a, parity)) return true;
  uint64_t t0 = 0;
  for (uint32_t it = 0;; ++it) {
    if (mbar_try(a, parity)) return true;
    if ((it & 63u) == 63u) {
      if (*abort_flag) return false;
      const uint64_t now = global_ns();
      if (t0 == 0) t0 = now;
      else if (now - t0 > 1000000000ull) return false;
    }
  }
}
// One row segment: global -> shared, completion counted in bytes on the stage's mbarrier.
__device__ __forceinline__ void bulk_copy(uint32_t dst, const void *src, uint32_t bytes, uint64_t *bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(dst), "l"(src), "r"(bytes), "r"(smem_addr(bar))
               : "memory");
}
// Four 8x8 bf16 matrices (eight 16-byte rows each; lane i gives the address of row i % 8 of
// matrix i / 8): lane (g, t) gets elements [g][2t], [g][2t+1] of each ...
__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(addr)
               : "memory");
}
// ... or, transposed, elements [2t][g], [2t+1][g].
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(addr)
               : "memory");
}
__device__ __forceinline__ uint4 lds128(uint32_t addr) {
  uint4 r;
  asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w) : "r"(addr) : "memory");
  return r;
}
__device__ __forceinline__ uint32_t lds32(uint32_t addr) {
  uint32_t r;
  asm volatile("ld.shared.u32 %0, [%1];" : "=r"(r) : "r"(addr) : "memory");
  return r;
}
__device__ __forceinline__ void sts32(uint32_t addr, uint32_t v) {
  asm volatile("st.shared.u32 [%0], %1;" ::"r"(addr), "r"(v) : "memory");
}
__device__ __forceinline__ void sts128(uint32_t addr, const uint4 &v) {
  asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(addr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}
// D(16x8, f32) += A(16x16, bf16, row) * B(16x8, bf16, col)
__device__ __forceinline__ void mma_bf16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                         uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
      "{%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// ---- the share of one lane -------------------------------------------------------
// Position P in the rows x column-blocks area of a kernel, counted tile by tile:
// tile t covers [rows(t) * CB, rows(t + 1) * CB), and inside it column block
// cb = (P - rows(t) * CB) / w_t  where w_t is the tile's row count.
template <bool kExpand>
__device__ __forceinline__ int tile_rows(int rank, int len) {
  return kExpand ? mint_tile_rows_expand(rank, len) : mint_tile_rows_shrink(rank, len);
}

struct Area {
  int64_t W;     // rows of the whole area
  int CB;        // column blocks of the whole call
  int G;         // lanes the plan's table was cut for
  int active;    // lanes that take work (at most the grid size)
  const LaneStart *table;
};

template <bool kExpand>
__device__ __forceinline__ Area make_area(const StreamParams &P) {
  Area a;
  a.W = P.pv.header[kExpand ? PH_ROWS_EXPAND : PH_ROWS_SHRINK];
  a.CB = kExpand ? P.cb_expand : P.cb_shrink;
  a.G = P.lanes;
  a.table = kExpand ? P.pv.lane_expand : P.pv.lane_shrink;
  int64_t g = a.W * a.CB / (kExpand ? kExpandGrain : kShrinkGrain);
  if (!kExpand) {
    // The expand adds the parts of every shrink lane that met a tile: keep the
    // largest tile of the widest projection within kMaxParts lane shares.
    const int64_t big = (int64_t)P.pv.header[PH_MAX_TILE_ROWS] * P.cb_shrink_widest;
    if (big > 0) g = min(g, (int64_t)(kMaxParts - 1) * a.W * a.CB / big);
  }
  if (g < 1) g = 1;
  if (g > (int64_t)gridDim.x) g = gridDim.x;
  if (g > a.G) g = a.G;
  a.active = (int)g;
  return a;
}
// Table index of active lane c (c == active: the end of the area).
__device__ __forceinline__ int lane_index(const Area &a, int c) {
  return (int)((unsigned)c * (unsigned)a.G / (unsigned)a.active);
}
// Where table lane j starts relative to row `rows` of the area, in (row x column block)
// units: (q - rows) * CB + r * CB / G.  The caller knows the result is small.
__device__ __forceinline__ int64_t lane_offset(const Area &a, const LaneStart &ls, int rows) {
  return (int64_t)(ls.q - rows) * a.CB + (int)((unsigned)ls.r * (unsigned)a.CB / (unsigned)a.G);
}

struct CtaRange {
  int t0, cb0, t1, cb1;  // share = [(t0, cb0), (t1, cb1))
  int t_end;             // one past the last tile the share touches
};

// Plan checks and this lane's share (all threads).  Nothing of the plan beyond its header is read
// before the header has been checked.
template <bool kExpand>
__device__ __forceinline__ bool prologue(const StreamParams &P, Smem &S, Area &area, CtaRange &R, bool report_errors) {
  if (!plan_ok(P.pv.header, P.T, P.K, P.tab.num_slots, P.num_experts, P.tab.gen_lo, P.tab.gen_hi,
               report_errors ? P.status : nullptr))
    return false;
  if (P.pv.header[PH_LANES] != P.lanes) {
    if (threadIdx.x == 0 && report_errors) report(P.status, MINT_ERR_SHAPE_MISMATCH, P.pv.header[PH_LANES]);
    return false;
  }
  if (P.pv.header[PH_NCHUNK1] == 0) return false;
  // nothing streamed: every tile belongs to a dense segment (the tensor-core kernels take those)
  if (P.pv.header[kExpand ? PH_ROWS_EXPAND : PH_ROWS_SHRINK] == 0) return false;
  area = make_area<kExpand>(P);
  const int c = blockIdx.x;
  if (c >= area.active) return false;
  if (threadIdx.x < 2) {   // thread 0: the cut where this lane starts; thread 1: where it ends
    const int j = lane_index(area, c + threadIdx.x);
    const LaneStart ls = area.table[j];
    const int cb = j < area.G ? (int)(lane_offset(area, ls, ls.rows) / ls.w) : 0;
    S.range[2 * threadIdx.x] = ls.tile;
    S.range[2 * threadIdx.x + 1] = cb;
  }
  __syncthreads();
  R.t0 = S.range[0];
  R.cb0 = S.range[1];
  R.t1 = S.range[2];
  R.cb1 = S.range[3];
  R.t_end = (R.cb1 > 0) ? R.t1 + 1 : R.t1;
  return R.t_end > R.t0;
}

// ================================================================================
// producer
// ================================================================================
// Longest run of columns (a power of two from 64 to kMaxRun) such that `rows` padded rows, plus
// `block_bytes_per_col` bytes per column of an unpadded block, fit a stage.
__device__ __forceinline__ int stage_run(int rows, int block_bytes_per_col) {
  int cw = kMaxRun;
  while (cw > 64 && rows * (2 * cw + 16) + cw * block_bytes_per_col > kStageBytes) cw >>= 1;
  return cw;
}

template <bool kExpand, bool kPacked>
__device__ void produce(const StreamParams &P, Smem &S, const Area &area, const CtaRange &R) {
  constexpr int kBlock = kExpand ? kExpandBlock : kShrinkBlock;
  const int lane = threadIdx.x & 31;
  const uint32_t ring0 = smem_addr(S.ring);
  uint32_t it = 0;
  bool ok = true;
  for (int tb = R.t0; tb < R.t_end && ok; tb += kBatchTiles) {
    const int ntile = min(kBatchTiles, R.t_end - tb);
    __syncwarp();
    {
      const int4 *src = reinterpret_cast<const int4 *>(P.pv.tile_desc + tb);
      int4 *dst = reinterpret_cast<int4 *>(S.pdesc);
      for (int i = lane; i < ntile * (int)(sizeof(TileDesc) / 16); i += 32) dst[i] = src[i];
    }
    __syncwarp();
    const int off0 = S.pdesc[0].off;
    const int nitems = S.pdesc[ntile - 1].off + S.pdesc[ntile - 1].len - off0;
    for (int i = lane; i < nitems; i += 32) {
      const int p = P.pv.perm[off0 + i];
      int row = p;
      if (!kExpand && kPacked) {   // the rows of x that the pairs read
        if (P.x_row) row = P.x_row[p];
        if (row < 0 || row >= P.x_rows) {
          report(P.status, MINT_ERR_BAD_INDEX, p);
          row = -1;
        }
      }
      S.prows[i] = row;
    }
    __syncwarp();
    for (int ti = 0; ti < ntile && ok; ++ti) {
      const int t = tb + ti;
      const int va = (t == R.t0) ? R.cb0 : 0;
      const int vb = (t == R.t1) ? R.cb1 : area.CB;
      if (va >= vb) continue;
      const TileDesc &td = S.pdesc[ti];
      if (td.dense) continue;   // it runs on the 128-row tensor-core kernels
      const int32_t *rows = S.prows + (td.off - off0);
      const int r = td.rank, len = td.len;
      const int wslot = td.slot * P.weights_per_slot + td.expert;
      for (int p = 0; p < P.nprob && ok; ++p) {
        const StreamProblem &pb = P.prob[p];
        const int width = kExpand ? pb.n : pb.d;
        const int first = kExpand ? pb.cb0_expand : pb.cb0_shrink;
        const int count = (width + kBlock - 1) / kBlock;
        const int lo = max(va, first) - first, hi = min(vb, first + count) - first;
        if (lo >= hi) continue;
        // ---- one piece: columns [c_begin, c_end) of every row of the tile and of the slot
        const int c_begin = lo * kBlock, c_end = min(hi * kBlock, width);
        const bool packed_a = !kExpand && kPacked;
        const int cw = packed_a ? stage_run(len, pb.r_max * 2) : stage_run(len + r, 0);
        const int pitch = 2 * cw + 16;
        const int w_off = len * pitch;
        // this lane's rows: token rows first, then weight rows (three at most: 96 rows)
        const int nrows = packed_a ? len : len + r;
        const uint16_t *src[3];
        uint32_t dst[3];
        bool zero[3];
#pragma unroll
        for (int q = 0; q < 3; ++q) {
          const int i = lane + 32 * q;
          src[q] = nullptr;
          zero[q] = false;
          dst[q] = (uint32_t)(i * pitch);
          if (i < len) {
            const int row = rows[i];
            if (row >= 0) src[q] = (kExpand ? pb.y + (int64_t)row * pb.ldy : pb.x + (int64_t)row * pb.ldx);
            else zero[q] = true;   // a pair whose row of x is out of range: its x counts as zero
          } else if (i < nrows) {
            const uint16_t *w = (kExpand ? pb.B : pb.A) + (int64_t)wslot * pb.r_max * width;
            src[q] = w + (int64_t)(i - len) * width;
          }
        }
        const uint16_t *a_block = packed_a ? pb.A + (int64_t)wslot * pb.d * pb.r_max : nullptr;
        int n_valid = 0;   // rows that are really copied
        for (int i = 0; i < len; ++i) n_valid += rows[i] >= 0;
        n_valid += packed_a ? 0 : r;
        for (int c0 = c_begin; c0 < c_end; c0 += cw) {
          const int ncols = min(cw, c_end - c0);
          const int s = (int)(it % kStages);
          if (!mbar_wait(&S.empty[s], ((it / kStages) & 1u) ^ 1u, &S.abort_flag)) {
            ok = false;
            break;
          }
          StageHdr &h = S.hdr[s];
          if (lane == 0) {
            h.kind = kStageData;
            h.tile = t;
            h.prob = p;
            h.col0 = c0;
            h.ncols = ncols;
            h.pitch = pitch;
            h.rank = r;
            h.len = len;
            h.flags = (c0 == c_begin ? kFlagFirst : 0) | (c0 + cw >= c_end ? kFlagLast : 0);
            h.scale = td.scale;
            h.lane_lo = td.lane_lo;
            h.lane_hi = td.lane_hi;
            h.rows_shrink = td.rows_shrink;
            h.w_off = w_off;
          }
          if (lane < len) h.rows[lane] = rows[lane];
          const uint32_t base = ring0 + (uint32_t)(s * kStageBytes);
          const uint32_t bytes = (uint32_t)ncols * 2u;
#pragma unroll
          for (int q = 0; q < 3; ++q)
            if (zero[q])
              for (uint32_t o = 0; o < bytes; o += 16) sts128(base + dst[q] + o, make_uint4(0u, 0u, 0u, 0u));
          __syncwarp();
          if (lane == 0)
            mbar_arrive_expect_tx(&S.full[s], (uint32_t)n_valid * bytes + (packed_a ? bytes * (uint32_t)pb.r_max : 0u));
#pragma unroll
          for (int q = 0; q < 3; ++q)
            if (src[q]) bulk_copy(base + dst[q], src[q] + c0, bytes, &S.full[s]);
          if (packed_a && lane == 0)   // A[d][r_max]: the rows c0 .. c0 + ncols are one contiguous block
            bulk_copy(base + (uint32_t)w_off, a_block + (int64_t)c0 * pb.r_max, bytes * (uint32_t)pb.r_max, &S.full[s]);
          ++it;
        }
      }
    }
  }
  // the end marker, or, after a wait that ran out, the copies still in flight
  if (ok) {
    const int s = (int)(it % kStages);
    if (mbar_wait(&S.empty[s], ((it / kStages) & 1u) ^ 1u, &S.abort_flag)) {
      if (lane == 0) {
        S.hdr[s].kind = kStageEnd;
        mbar_arrive(&S.full[s]);
      }
      return;
    }
    ok = false;
  }
  if (lane == 0) {
    S.abort_flag = 1;
    report(P.status, MINT_ERR_TIMEOUT, (int32_t)blockIdx.x);
  }
  // every stage this warp armed completes on its own: wait for the bytes before the CTA's memory goes away
  for (uint32_t j = it > (uint32_t)kStages ? it - kStages : 0; j < it; ++j) {
    const uint32_t a = smem_addr(&S.full[j % kStages]);
    const uint64_t t0 = global_ns();
    while (!mbar_try(a, (j / kStages) & 1u) && global_ns() - t0 < 100000000ull) {
    }
  }
}

// ================================================================================
// consumers
// ================================================================================
struct Cursor {
  uint32_t it;       // stages consumed so far
  uint32_t cphase;   // phase of the consumers' barrier
  __device__ __forceinline__ int stage() const { return (int)(it % kStages); }
};

// Barrier of the four consumer warps on an mbarrier, so that the wait is bounded like every other
// wait here: false when it ran out or another warp of the CTA has given up.
__device__ __forceinline__ bool consumer_sync(Smem &S, Cursor &cur) {
  __syncwarp();
  if ((threadIdx.x & 31) == 0) mbar_arrive(&S.cbar);
  const bool ok = mbar_wait(&S.cbar, cur.cphase & 1u, &S.abort_flag);
  cur.cphase ^= 1u;
  return ok;
}

// Waits until stage `cur` is full; false when the wait ran out (or another warp gave up).
__device__ __forceinline__ bool stage_wait(Smem &S, const StreamParams &P, const Cursor &cur) {
  if (mbar_wait(&S.full[cur.stage()], (cur.it / kStages) & 1u, &S.abort_flag)) return true;
  if ((threadIdx.x & 31) == 0 && !S.abort_flag) {
    S.abort_flag = 1;
    report(P.status, MINT_ERR_TIMEOUT, (int32_t)blockIdx.x);
  }
  return false;
}
// This warp is done with the stage.
__device__ __forceinline__ void stage_release(Smem &S, Cursor &cur) {
  __syncwarp();
  if ((threadIdx.x & 31) == 0) mbar_arrive(&S.empty[cur.stage()]);
  ++cur.it;
}

// ---- shrink ----------------------------------------------------------------------
// Tensor-core body: MT groups of 16 token rows, NT2 groups of 16 rank rows.  The warp takes
// every fourth 16-column step of a stage; the accumulators live over the whole piece.
template <int MT, int NT2, bool kPacked>
__device__ __forceinline__ bool shrink_mma(const StreamParams &P, Smem &S, Cursor &cur) {
  constexpr int NT = 2 * NT2;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, tid = threadIdx.x;
  const StageHdr *h = &S.hdr[cur.stage()];
  const int r = h->rank, len = h->len, tile = h->tile, pitch = h->pitch, w_off = h->w_off;
  const StreamProblem &pb = P.prob[h->prob];
  const uint32_t ring0 = smem_addr(S.ring);
  // ldmatrix row addresses of this lane.  Token rows: matrix m = lane / 8 is rows 8 (m & 1) .. + 7,
  // columns 8 (m / 2) .. + 7 of the 16 x 16 step; rows beyond the tile repeat its last row.
  uint32_t a_off[MT];
#pragma unroll
  for (int mt = 0; mt < MT; ++mt) {
    const int row = min(mt * 16 + (lane & 7) + 8 * ((lane >> 3) & 1), len - 1);
    a_off[mt] = (uint32_t)(row * pitch + (lane >> 4) * 16);
  }
  // Rank rows: matrix m is ranks 8 (m / 2) .. + 7, columns 8 (m & 1) .. + 7 (rank-major A), or, for
  // the packed layout [column][rank], columns 8 (m & 1) .. + 7 as rows and ranks 8 (m / 2) .. + 7.
  uint32_t b_off[NT2];
#pragma unroll
  for (int np = 0; np < NT2; ++np) {
    if (kPacked) {
      const int krow = (lane & 7) + 8 * ((lane >> 3) & 1);
      const int n0 = min(np * 16 + 8 * (lane >> 4), pb.r_max - 8);
      b_off[np] = (uint32_t)(w_off + (krow * pb.r_max + n0) * 2);
    } else {
      const int rank = min(np * 16 + (lane & 7) + 8 * (lane >> 4), r - 1);
      b_off[np] = (uint32_t)(w_off + rank * pitch + ((lane >> 3) & 1) * 16);
    }
  }
  const uint32_t b_step = kPacked ? (uint32_t)(16 * pb.r_max * 2) : 32u;
  float acc[MT][NT][4];
#pragma unroll
  for (int a = 0; a < MT; ++a)
#pragma unroll
    for (int b = 0; b < NT; ++b)
#pragma unroll
      for (int e = 0; e < 4; ++e) acc[a][b][e] = 0.f;

  for (;;) {
    const uint32_t base = ring0 + (uint32_t)(cur.stage() * kStageBytes);
    const int ncols = h->ncols;
    const int nsteps = (ncols + 15) >> 4;
#pragma unroll 1
    for (int ks = warp; ks < nsteps; ks += kConsumerWarps) {
      uint32_t a[MT][4], b[NT2][4];
#pragma unroll
      for (int mt = 0; mt < MT; ++mt) ldmatrix_x4(a[mt], base + a_off[mt] + (uint32_t)ks * 32u);
#pragma unroll
      for (int np = 0; np < NT2; ++np) {
        if (kPacked) ldmatrix_x4_trans(b[np], base + b_off[np] + (uint32_t)ks * b_step);
        else ldmatrix_x4(b[np], base + b_off[np] + (uint32_t)ks * 32u);
      }
      if (ks * 16 + 8 >= ncols) {   // the last step holds 8 columns only: the other 8 are not part of d
#pragma unroll
        for (int mt = 0; mt < MT; ++mt) a[mt][2] = a[mt][3] = 0u;
#pragma unroll
        for (int np = 0; np < NT2; ++np) b[np][1] = b[np][3] = 0u;
      }
#pragma unroll
      for (int mt = 0; mt < MT; ++mt)
#pragma unroll
        for (int np = 0; np < NT2; ++np) {
          mma_bf16(acc[mt][2 * np], a[mt][0], a[mt][1], a[mt][2], a[mt][3], b[np][0], b[np][1]);
          mma_bf16(acc[mt][2 * np + 1], a[mt][0], a[mt][1], a[mt][2], a[mt][3], b[np][2], b[np][3]);
        }
    }
    const bool last = (h->flags & kFlagLast) != 0;
    stage_release(S, cur);
    if (last) break;
    if (!stage_wait(S, P, cur)) return false;
    h = &S.hdr[cur.stage()];
  }
  // add the four warps' sums in warp order, four groups of 8 ranks at a time; element (l, j) of the
  // [len][rank] result goes to this lane's slot of the workspace
  float *dst = pb.ws_part + (size_t)(tile + blockIdx.x) * ((size_t)kTileRowsMax * pb.r_max);
#pragma unroll
  for (int nt0 = 0; nt0 < NT; nt0 += 4) {
    if (!consumer_sync(S, cur)) return false;   // the gather of the previous pass (or piece) has read the scratch
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
      for (int q = 0; q < 4; ++q)
        if (nt0 + q < NT)
          *reinterpret_cast<float4 *>(S.u.scratch + (((warp * 2 + mt) * 4 + q) * 32 + lane) * 4) =
              make_float4(acc[mt][nt0 + q][0], acc[mt][nt0 + q][1], acc[mt][nt0 + q][2], acc[mt][nt0 + q][3]);
    if (!consumer_sync(S, cur)) return false;
    const int j0 = nt0 * 8, jr = min(32, r - j0);
    for (int i = tid; i < len * jr; i += kConsumers) {
      const int l = i / jr, j = i - l * jr;
      const int mt = l >> 4, g = l & 15, q = j >> 3, cc = j & 7;
      const int frag = ((g & 7) * 4 + (cc >> 1)) * 4 + (g >> 3) * 2 + (cc & 1);
      float s = 0.f;
#pragma unroll
      for (int w = 0; w < kConsumerWarps; ++w) s += S.u.scratch[((w * 2 + mt) * 4 + q) * 128 + frag];
      dst[l * r + j0 + j] = s;
    }
  }
  return true;
}

// rank-1 tiles of at most 8 tokens: fp32 FMAs, every thread takes 16-byte chunks of the stage's run.
__device__ __forceinline__ bool shrink_fma(const StreamParams &P, Smem &S, Cursor &cur) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, tid = threadIdx.x;
  const StageHdr *h = &S.hdr[cur.stage()];
  const int len = h->len, tile = h->tile, pitch = h->pitch, w_off = h->w_off;
  const StreamProblem &pb = P.prob[h->prob];
  const uint32_t ring0 = smem_addr(S.ring);
  float acc[8];
#pragma unroll
  for (int l = 0; l < 8; ++l) acc[l] = 0.f;
  for (;;) {
    const uint32_t base = ring0 + (uint32_t)(cur.stage() * kStageBytes);
    const int nchunk = h->ncols >> 3;
#pragma unroll 1
    for (int c = tid; c < nchunk; c += kConsumers) {
      float wf[8];
      unpack8(lds128(base + (uint32_t)(w_off + c * 16)), wf);
#pragma unroll
      for (int l = 0; l < 8; ++l)
        if (l < len) {
          float xf[8];
          unpack8(lds128(base + (uint32_t)(l * pitch + c * 16)), xf);
#pragma unroll
          for (int e = 0; e < 8; ++e) acc[l] = fmaf(xf[e], wf[e], acc[l]);
        }
    }
    const bool last = (h->flags & kFlagLast) != 0;
    stage_release(S, cur);
    if (last) break;
    if (!stage_wait(S, P, cur)) return false;
    h = &S.hdr[cur.stage()];
  }
  if (!consumer_sync(S, cur)) return false;   // the gather of the previous piece has read the scratch
#pragma unroll
  for (int l = 0; l < 8; ++l) {
    const float s = warp_sum(acc[l]);
    if (lane == 0) S.u.scratch[warp * 8 + l] = s;
  }
  if (!consumer_sync(S, cur)) return false;
  if (tid < len) {
    float s = 0.f;
#pragma unroll
    for (int w = 0; w < kConsumerWarps; ++w) s += S.u.scratch[w * 8 + tid];
    pb.ws_part[(size_t)(tile + blockIdx.x) * ((size_t)kTileRowsMax * pb.r_max) + tid] = s;
  }
  return true;
}

template <bool kPacked>
__device__ __forceinline__ bool shrink_piece(const StreamParams &P, Smem &S, Cursor &cur) {
  const StageHdr &h = S.hdr[cur.stage()];
  const int r = h.rank, len = h.len;
  if (!kPacked && r == 1 && len <= 8) return shrink_fma(P, S, cur);
  // (ranks in groups of 16, tokens in groups of 16: the shapes the 16 x 16 fragment loads come in)
  const int ng = kPacked ? (P.prob[0].r_max <= 16 ? 1 : (P.prob[0].r_max <= 32 ? 2 : 4))
                         : (r <= 16 ? 1 : (r <= 32 ? 2 : 4));
#define MINT_SHRINK_CASE(MT)                                              \
  if (ng == 1) return shrink_mma<MT, 1, kPacked>(P, S, cur);              \
  else if (ng == 2) return shrink_mma<MT, 2, kPacked>(P, S, cur);         \
  else return shrink_mma<MT, 4, kPacked>(P, S, cur)
  if (len <= 16) { MINT_SHRINK_CASE(1); }
  else { MINT_SHRINK_CASE(2); }
#undef MINT_SHRINK_CASE
}

// ---- expand ------------------------------------------------------------------------
// Splits v into a bf16 head and a bf16 remainder so that two MMAs carry about
// 16 significant bits of the fp32 shrink result into the expand.
__device__ __forceinline__ void split_pair(float a, float b, uint32_t &hi, uint32_t &lo) {
  hi = pack_bf16x2(a, b);
  lo = pack_bf16x2(a - bf16lo(hi), b - bf16hi(hi));
}

// The shrink lanes whose share met the columns of problem p in the tile: they
// are consecutive lanes, found from the area arithmetic of the shrink kernel
// alone.  Eight threads share the work: thread k looks at the candidate lanes
// c_a + k, c_a + k + 8, ... (all its table reads go out together), and the
// eight combine their findings with shuffles.  All consumer threads call this
// together for the same tile and problem.
__device__ __forceinline__ void shrink_parts(const StreamParams &P, const Area &sa, const StageHdr &h, int &first,
                                             int &count) {
  const int k = threadIdx.x & 7;
  const StreamProblem &pb = P.prob[h.prob];
  const int w_t = tile_rows<false>(h.rank, h.len);
  const int blocks = (pb.d + kShrinkBlock - 1) / kShrinkBlock;
  const int span = w_t * sa.CB;   // the tile's extent in area units
  // Table lanes that can meet the columns of THIS problem inside the tile: the problem covers the
  // area positions [pos_lo, pos_hi) and table lane j starts at about j W CB / G (one lane of margin
  // on either side; the exact test below decides).
  const int64_t wcb = sa.W * sa.CB;
  const int64_t pos_lo = (int64_t)h.rows_shrink * sa.CB + (int64_t)pb.cb0_shrink * w_t;
  const int64_t pos_hi = pos_lo + (int64_t)blocks * w_t;
  const int j_lo = max(h.lane_lo, (int)(pos_lo * sa.G / wcb) - 1);
  const int j_hi = min(h.lane_hi, (int)((pos_hi * sa.G + wcb - 1) / wcb) + 1);
  // active lanes c with table index in [j_lo, j_hi]: index(c) = c G / active
  const int c_a = (int)(((unsigned)(j_lo + 1) * (unsigned)sa.active - 1u) / (unsigned)sa.G);
  const int c_b = (int)(((unsigned)(j_hi + 1) * (unsigned)sa.active - 1u) / (unsigned)sa.G);
  unsigned long long mask = 0;   // bit i: lane c_a + i holds a part
  for (int i = k; c_a + i <= c_b && i < 64; i += 8) {
    const int c2 = c_a + i;
    const int64_t p0 = lane_offset(sa, sa.table[lane_index(sa, c2)], h.rows_shrink);
    const int64_t p1 = lane_offset(sa, sa.table[lane_index(sa, c2 + 1)], h.rows_shrink);
    if (p0 < span && p1 > 0) {
      const int va = p0 <= 0 ? 0 : (int)p0 / w_t;
      const int vb = p1 >= span ? sa.CB : (int)p1 / w_t;
      if (max(va, pb.cb0_shrink) < min(vb, pb.cb0_shrink + blocks)) mask |= 1ull << i;
    }
  }
#pragma unroll
  for (int o = 1; o < 8; o <<= 1) mask |= __shfl_xor_sync(0xffffffffu, mask, o);
  first = mask ? c_a + __ffsll((long long)mask) - 1 : 0;
  count = __popcll(mask);
}

// vsum[i] = weight(row of i) * sum, in lane order, of the shrink lanes' parts of element i of the
// [len][rank] result (all consumer threads).  Consecutive threads take consecutive elements, and
// the loads of four elements times four parts go out together.
__device__ __forceinline__ void sum_parts(const StreamParams &P, const StreamProblem &pb, const StageHdr &h, int first,
                                          int count, float *vsum) {
  const size_t slot_floats = (size_t)kTileRowsMax * pb.r_max;
  const float *part0 = pb.ws_part + (size_t)(h.tile + first) * slot_floats;
  const int nel = h.len * h.rank;
  for (int i0 = threadIdx.x; i0 < nel; i0 += 4 * kConsumers) {
    float s[4] = {0.f, 0.f, 0.f, 0.f};
    for (int k0 = 0; k0 < count; k0 += 4) {
      float v[4][4];
#pragma unroll
      for (int k = 0; k < 4; ++k)
#pragma unroll
        for (int e = 0; e < 4; ++e)
          v[k][e] = (k0 + k < count && i0 + e * kConsumers < nel)
                        ? __ldcg(part0 + (size_t)(k0 + k) * slot_floats + i0 + e * kConsumers)
                        : 0.f;
#pragma unroll
      for (int k = 0; k < 4; ++k)
#pragma unroll
        for (int e = 0; e < 4; ++e) s[e] += v[k][e];
    }
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const int i = i0 + e * kConsumers;
      if (i < nel) {
        // MoE: the pair's routing weight multiplies its row of v
        const float w = P.pair_weight ? __ldg(P.pair_weight + h.rows[i / h.rank]) : 1.f;
        vsum[i] = w * s[e];
      }
    }
  }
}

// Tensor-core body: MT groups of 16 token rows, KS steps of 16 ranks.  A warp takes a contiguous
// quarter of the 16-column groups of every stage.
template <int MT, int KS>
__device__ __forceinline__ bool expand_mma(const StreamParams &P, Smem &S, Cursor &cur) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, t = lane & 3;
  const StageHdr *h = &S.hdr[cur.stage()];
  const int r = h->rank, len = h->len, pitch = h->pitch, w_off = h->w_off;
  const float scale = h->scale;
  const StreamProblem &pb = P.prob[h->prob];
  const uint32_t ring0 = smem_addr(S.ring);
  // B rows of a 16-rank step as four transposed 8x8 matrices: matrix m is ranks 8 (m & 1) .. + 7,
  // columns 8 (m / 2) .. + 7 of the 16-column group; ranks beyond the slot's repeat its last row
  // (v is zero there).
  uint32_t b_off[KS];
#pragma unroll
  for (int ks = 0; ks < KS; ++ks) {
    const int krow = min(ks * 16 + (lane & 7) + 8 * ((lane >> 3) & 1), r - 1);
    b_off[ks] = (uint32_t)(w_off + krow * pitch + (lane >> 4) * 16);
  }
  for (;;) {
    const uint32_t base = ring0 + (uint32_t)(cur.stage() * kStageBytes);
    const int ncols = h->ncols;
    const int ngroups = (ncols + 15) >> 4;
    const int g0 = warp * ngroups / kConsumerWarps, g1 = (warp + 1) * ngroups / kConsumerWarps;
#pragma unroll 1
    for (int cg = g0; cg < g1; ++cg) {
      float acc[MT][2][4];
#pragma unroll
      for (int a = 0; a < MT; ++a)
#pragma unroll
        for (int b = 0; b < 2; ++b)
#pragma unroll
          for (int e = 0; e < 4; ++e) acc[a][b][e] = 0.f;
#pragma unroll
      for (int ks = 0; ks < KS; ++ks) {
        uint32_t b[4];
        ldmatrix_x4_trans(b, base + b_off[ks] + (uint32_t)cg * 32u);
#pragma unroll
        for (int mt = 0; mt < MT; ++mt) {
          const uint4 vh = S.u.e.vfrag[((mt * 4 + ks) * 2 + 0) * 32 + lane];
          const uint4 vl = S.u.e.vfrag[((mt * 4 + ks) * 2 + 1) * 32 + lane];
          mma_bf16(acc[mt][0], vh.x, vh.y, vh.z, vh.w, b[0], b[1]);
          mma_bf16(acc[mt][1], vh.x, vh.y, vh.z, vh.w, b[2], b[3]);
          mma_bf16(acc[mt][0], vl.x, vl.y, vl.z, vl.w, b[0], b[1]);
          mma_bf16(acc[mt][1], vl.x, vl.y, vl.z, vl.w, b[2], b[3]);
        }
      }
      // acc[mt][nt][0], [1]: row 16 mt + g, columns 16 cg + 8 nt + 2t, + 1; [2], [3]: row + 8
#pragma unroll
      for (int mt = 0; mt < MT; ++mt)
#pragma unroll
        for (int nt = 0; nt < 2; ++nt)
#pragma unroll
          for (int hh = 0; hh < 2; ++hh) {
            const int row = mt * 16 + g + 8 * hh, col = cg * 16 + nt * 8 + 2 * t;
            if (row < len && col < ncols) {
              const uint32_t addr = base + (uint32_t)(row * pitch + col * 2);
              const uint32_t w = lds32(addr);
              sts32(addr, pack_bf16x2(fmaf(scale, acc[mt][nt][2 * hh], bf16lo(w)),
                                      fmaf(scale, acc[mt][nt][2 * hh + 1], bf16hi(w))));
            }
          }
    }
    __syncwarp();
    // this warp's columns of every row of the tile go back to memory, 16 bytes per lane
    {
      const int cbeg = g0 * 16, cend = min(g1 * 16, ncols);
      const int cpr = (cend - cbeg) >> 3;
      if (cpr > 0) {
        uint16_t *ybase = pb.y + h->col0 + cbeg;
        for (int q = lane; q < len * cpr; q += 32) {
          const int row = q / cpr, ch = q - row * cpr;
          *reinterpret_cast<uint4 *>(ybase + (int64_t)h->rows[row] * pb.ldy + ch * 8) =
              lds128(base + (uint32_t)(row * pitch + cbeg * 2 + ch * 16));
        }
      }
    }
    fence_async_smem();   // this warp's writes to the stage are ordered before the copies that refill it
    const bool last = (h->flags & kFlagLast) != 0;
    stage_release(S, cur);
    if (last) break;
    if (!stage_wait(S, P, cur)) return false;
    h = &S.hdr[cur.stage()];
  }
  return true;
}

// rank-1 tiles of at most 8 tokens: fp32 FMAs; every thread adds the shrink lanes' parts of the
// few v it needs by itself.
__device__ __forceinline__ bool expand_fma(const StreamParams &P, Smem &S, Cursor &cur, int first, int count) {
  const int tid = threadIdx.x;
  const StageHdr *h = &S.hdr[cur.stage()];
  const int len = h->len, pitch = h->pitch, w_off = h->w_off;
  const StreamProblem &pb = P.prob[h->prob];
  const uint32_t ring0 = smem_addr(S.ring);
  float sv[8];
  uint16_t *yr[8];
  {
    const size_t slot_floats = (size_t)kTileRowsMax * pb.r_max;
    const float *part0 = pb.ws_part + (size_t)(h->tile + first) * slot_floats;
#pragma unroll
    for (int l = 0; l < 8; ++l) sv[l] = 0.f;
    for (int k0 = 0; k0 < count; k0 += 4) {   // in lane order; the loads of four parts go out together
      float v[4][8];
#pragma unroll
      for (int k = 0; k < 4; ++k)
#pragma unroll
        for (int l = 0; l < 8; ++l)
          v[k][l] = (k0 + k < count && l < len) ? __ldcg(part0 + (size_t)(k0 + k) * slot_floats + l) : 0.f;
#pragma unroll
      for (int k = 0; k < 4; ++k)
#pragma unroll
        for (int l = 0; l < 8; ++l) sv[l] += v[k][l];
    }
#pragma unroll
    for (int l = 0; l < 8; ++l) {
      const int row = h->rows[l < len ? l : 0];
      // MoE: the pair's routing weight multiplies its v
      const float w = (P.pair_weight && l < len) ? __ldg(P.pair_weight + row) : 1.f;
      sv[l] = h->scale * (w * sv[l]);
      yr[l] = pb.y + (int64_t)row * pb.ldy;
    }
  }
  for (;;) {
    const uint32_t base = ring0 + (uint32_t)(cur.stage() * kStageBytes);
    const int nchunk = h->ncols >> 3, col0 = h->col0;
#pragma unroll 1
    for (int c = tid; c < nchunk; c += kConsumers) {
      float wf[8];
      unpack8(lds128(base + (uint32_t)(w_off + c * 16)), wf);
#pragma unroll
      for (int l = 0; l < 8; ++l)
        if (l < len) {
          float yf[8];
          unpack8(lds128(base + (uint32_t)(l * pitch + c * 16)), yf);
#pragma unroll
          for (int e = 0; e < 8; ++e) yf[e] = fmaf(sv[l], wf[e], yf[e]);
          *reinterpret_cast<uint4 *>(yr[l] + col0 + c * 8) = pack8(yf);
        }
    }
    const bool last = (h->flags & kFlagLast) != 0;
    stage_release(S, cur);
    if (last) break;
    if (!stage_wait(S, P, cur)) return false;
    h = &S.hdr[cur.stage()];
  }
  return true;
}

__device__ __forceinline__ bool expand_piece(const StreamParams &P, Smem &S, const Area &shrink_area, Cursor &cur) {
  const StageHdr &h = S.hdr[cur.stage()];
  const StreamProblem &pb = P.prob[h.prob];
  const int tid = threadIdx.x;
  const int r = h.rank, len = h.len;
  int first, count;
  shrink_parts(P, shrink_area, h, first, count);
  if (r == 1 && len <= 8) return expand_fma(P, S, cur, first, count);
  const int MT = len <= 16 ? 1 : 2, KS = (r + 15) >> 4;
  if (!consumer_sync(S, cur)) return false;   // the previous piece no longer reads v
  sum_parts(P, pb, h, first, count, S.u.e.vsum);
  if (!consumer_sync(S, cur)) return false;
  // one thread per (m-tile, k-step, lane): four (head, remainder) register pairs
  for (int i = tid; i < MT * KS * 32; i += kConsumers) {
    const int ln = i & 31, ks = (i >> 5) % KS, mt = (i >> 5) / KS;
    const int g = ln >> 2, t = ln & 3;
    uint32_t hi[4], lo[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const int row = mt * 16 + g + (q & 1) * 8, k = ks * 16 + 2 * t + (q >> 1) * 8;
      const float a = (row < len && k < r) ? S.u.e.vsum[row * r + k] : 0.f;
      const float b = (row < len && k + 1 < r) ? S.u.e.vsum[row * r + k + 1] : 0.f;
      split_pair(a, b, hi[q], lo[q]);
    }
    S.u.e.vfrag[((mt * 4 + ks) * 2 + 0) * 32 + ln] = make_uint4(hi[0], hi[1], hi[2], hi[3]);
    S.u.e.vfrag[((mt * 4 + ks) * 2 + 1) * 32 + ln] = make_uint4(lo[0], lo[1], lo[2], lo[3]);
  }
  if (!consumer_sync(S, cur)) return false;
#define MINT_EXPAND_CASE(MT_)                                   \
  if (KS == 1) return expand_mma<MT_, 1>(P, S, cur);            \
  else if (KS == 2) return expand_mma<MT_, 2>(P, S, cur);       \
  else if (KS == 3) return expand_mma<MT_, 3>(P, S, cur);       \
  else return expand_mma<MT_, 4>(P, S, cur)
  if (MT == 1) { MINT_EXPAND_CASE(1); }
  else { MINT_EXPAND_CASE(2); }
#undef MINT_EXPAND_CASE
}

// ================================================================================
// kernels
// ================================================================================
template <bool kExpand, bool kPacked>
__device__ __forceinline__ void rows_kernel_body(const StreamParams &P, Smem &S) {
  pdl_launch_dependents();
  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(&S.full[s], 1);
      mbar_init(&S.empty[s], kConsumerWarps);
    }
    mbar_init(&S.cbar, kConsumerWarps);
    S.abort_flag = 0;
    fence_mbar_init();
  }
  Area area;
  CtaRange R;
  // The plan and the slot table were complete before this call's kernels started when the kernel
  // before this one in the stream is one of them; a plan or a bind kernel right before it is waited
  // for first (the launch then carries no programmatic serialization).
  if (!prologue<kExpand>(P, S, area, R, !kExpand)) {   // errors of the plan are reported once, by the shrink
    pdl_wait();
    return;
  }
  pdl_wait();   // activations, y and the workspace belong to earlier kernels until here
  if (threadIdx.x >= kConsumers) {
    produce<kExpand, kPacked>(P, S, area, R);
    return;
  }
  const Area shrink_area = kExpand ? make_area<false>(P) : area;
  Cursor cur{0u, 0u};
  for (;;) {
    if (!stage_wait(S, P, cur)) return;
    if (S.hdr[cur.stage()].kind == kStageEnd) return;
    const bool ok = kExpand ? expand_piece(P, S, shrink_area, cur) : shrink_piece<kPacked>(P, S, cur);
    if (!ok) return;
  }
}

template <bool kPacked>
__global__ void __launch_bounds__(kThreads, kCtasPerSm) shrink_rows_kernel(const __grid_constant__ StreamParams P) {
  extern __shared__ __align__(128) uint8_t dyn_smem[];
  rows_kernel_body<false, kPacked>(P, *reinterpret_cast<Smem *>(dyn_smem));
}

__global__ void __launch_bounds__(kThreads, kCtasPerSm) expand_rows_kernel(const __grid_constant__ StreamParams P) {
  extern __shared__ __align__(128) uint8_t dyn_smem[];
  rows_kernel_body<true, false>(P, *reinterpret_cast<Smem *>(dyn_smem));
}

// ---- host side -----------------------------------------------------------------
// Slots of 32 x r_max floats: tile + lane for the streamed parts; with dense segments (batches of at
// least MINT_DENSE_MIN_BATCH tokens) MINT_DENSE_SPLIT_MAX more per tile for the parts of the tensor-core shrink.
size_t workspace_bytes(int64_t tiles, int32_t r_max, bool dense) {
  const int64_t slots = tiles + MINT_MAX_LANES + (dense ? (int64_t)MINT_DENSE_SPLIT_MAX * tiles : 0);
  return (size_t)slots * kTileRowsMax * r_max * sizeof(float) + 256;
}

int32_t kernel_attributes() {
  static bool attrs_set = false;
  if (attrs_set) return MINT_OK;
  int32_t st;
  st = mint_check_cuda(cudaFuncSetAttribute(shrink_rows_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                            (int)sizeof(Smem)), "shrink_rows shared memory");
  if (st) return st;
  st = mint_check_cuda(cudaFuncSetAttribute(shrink_rows_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                            (int)sizeof(Smem)), "shrink_rows (packed) shared memory");
  if (st) return st;
  st = mint_check_cuda(cudaFuncSetAttribute(expand_rows_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                            (int)sizeof(Smem)), "expand_rows shared memory");
  if (st) return st;
  attrs_set = true;
  return MINT_OK;
}

// The grid: kCtasPerSm lanes per SM, at most the lanes the plan's tables were cut for.
int32_t grid_lanes(int32_t plan_lanes, int32_t *out) {
  int dev = 0, sms = 0;
  int32_t st = mint_check_cuda(cudaGetDevice(&dev), "cudaGetDevice");
  if (st) return st;
  if ((st = mint_check_cuda(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev), "SM count"))) return st;
  *out = std::min(plan_lanes, sms * kCtasPerSm);
  return MINT_OK;
}

}  // namespace

bool mint_stream_supported(int32_t r_max_bound) { return r_max_bound <= kStreamRankCap; }

// The packed-layout shrink reads A[d][r_max] in 16-byte segments of 8 ranks.
bool mint_stream_moe_supported(int32_t r_max, int32_t r_max_bound) {
  return r_max_bound <= kStreamRankCap && (r_max == 8 || r_max == 16 || r_max == 32 || r_max == 64);
}

size_t mint_stream_moe_workspace_bytes(int64_t pairs, int64_t key_space, int32_t r_max) {
  return workspace_bytes(mint_tile_upper_bound(1, pairs, key_space), r_max, false);
}

size_t mint_stream_workspace_bytes(int32_t T, int32_t num_slots, int32_t r_max) {
  return workspace_bytes(mint_tile_upper_bound(1, T, num_slots), r_max, T >= MINT_DENSE_MIN_BATCH);
}

// MoE expert LoRA apply on the streamed kernels: the plan's items are the
// (token, k) pairs grouped by (expert, slot); the weight block of a tile is
// (slot, expert); the shrink reads row x_row[p] of x, the expand updates row p of y.
int32_t mint_launch_stream_moe(const MoEArgs &a, const TableDev &tab, const void *plan_dev, void *workspace,
                               cudaStream_t s) {
  int32_t lanes = 0, grid = 0;
  int32_t st = mint_device_lanes(&lanes);
  if (st) return st;
  if ((st = grid_lanes(lanes, &grid))) return st;
  if ((st = kernel_attributes())) return st;
  const int64_t pairs = (int64_t)a.T * a.K;
  const int64_t key_space = (int64_t)tab.num_slots * a.num_experts;
  const int64_t tiles = mint_tile_upper_bound(1, pairs, key_space);
  if (tiles == 0) return MINT_OK;
  StreamParams P = {};
  StreamProblem &pb = P.prob[0];
  pb.A = a.A; pb.B = a.B; pb.x = a.x; pb.y = a.y;
  pb.ldx = a.ldx; pb.ldy = a.ldy;
  pb.d = a.d; pb.n = a.n; pb.r_max = a.r_max;
  pb.cb0_shrink = kShrinkPieceBlocks;
  pb.cb0_expand = kExpandPieceBlocks;
  pb.ws_part = static_cast<float *>(workspace);
  P.nprob = 1;
  P.T = a.T;
  P.K = a.K;
  P.num_experts = a.num_experts;
  P.weights_per_slot = a.num_experts;
  P.x_row = a.x_row;
  P.pair_weight = a.pair_weight;
  P.x_rows = a.x_rows;
  P.lanes = lanes;
  P.cb_shrink = kShrinkPieceBlocks + (a.d + kShrinkBlock - 1) / kShrinkBlock;
  P.cb_expand = kExpandPieceBlocks + (a.n + kExpandBlock - 1) / kExpandBlock;
  P.cb_shrink_widest = P.cb_shrink;
  P.dense_slot0 = (int32_t)(tiles + MINT_MAX_LANES);
  P.status = a.status;
  P.tab = tab;
  P.pv = mint_plan_view(plan_dev, pairs, key_space);

  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)grid);
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = sizeof(Smem);
  cfg.stream = s;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  // the first apply after a plan or a bind waits for that kernel in full: it reads the plan at once
  cfg.numAttrs = mint_take_tables_changed() ? 0 : 1;
  st = mint_check_cuda(cudaLaunchKernelEx(&cfg, shrink_rows_kernel<true>, P), "shrink_rows (packed) launch");
  if (st) return st;
  cfg.numAttrs = 1;
  return mint_check_cuda(cudaLaunchKernelEx(&cfg, expand_rows_kernel, P), "expand_rows launch");
}

int32_t mint_launch_stream(const DenseArgs *args, int nprob, const TableDev &tab, const void *plan_dev,
                           void *const *workspaces, cudaStream_t s) {
  if (nprob < 1 || nprob > kMaxProblems)
    return mint_fail(MINT_ERR_INVALID_ARG, "grouped apply: 1..%d problems", kMaxProblems);
  int32_t lanes = 0, grid = 0;
  int32_t st = mint_device_lanes(&lanes);
  if (st) return st;
  if ((st = grid_lanes(lanes, &grid))) return st;
  if ((st = kernel_attributes())) return st;
  const int32_t T = args[0].T;
  const int64_t tiles = mint_tile_upper_bound(1, T, tab.num_slots);
  if (tiles == 0) return MINT_OK;
  StreamParams P = {};
  int cb_s = 0, cb_e = 0, cb_widest = 0;
  for (int i = 0; i < nprob; ++i) {
    const DenseArgs &a = args[i];
    StreamProblem &pb = P.prob[i];
    pb.A = a.A; pb.B = a.B; pb.x = a.x; pb.y = a.y;
    pb.ldx = a.ldx; pb.ldy = a.ldy;
    pb.d = a.d; pb.n = a.n; pb.r_max = a.r_max;
    cb_s += kShrinkPieceBlocks;
    cb_e += kExpandPieceBlocks;
    pb.cb0_shrink = cb_s;
    pb.cb0_expand = cb_e;
    cb_s += (a.d + kShrinkBlock - 1) / kShrinkBlock;
    cb_widest = std::max(cb_widest, (a.d + kShrinkBlock - 1) / kShrinkBlock);
    cb_e += (a.n + kExpandBlock - 1) / kExpandBlock;
    pb.ws_part = static_cast<float *>(workspaces[i]);
  }
  P.nprob = nprob;
  P.T = T;
  P.K = 1;
  P.num_experts = 0;
  P.weights_per_slot = 1;
  P.lanes = lanes;
  P.cb_shrink = cb_s;
  P.cb_expand = cb_e;
  P.cb_shrink_widest = cb_widest;
  P.dense_slot0 = (int32_t)(tiles + MINT_MAX_LANES);
  P.status = args[0].status;
  P.tab = tab;
  P.pv = mint_plan_view(plan_dev, T, tab.num_slots);

  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)grid);
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = sizeof(Smem);
  cfg.stream = s;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  // the first apply after a plan or a bind waits for that kernel in full: it reads the plan at once
  cfg.numAttrs = mint_take_tables_changed() ? 0 : 1;
  st = mint_check_cuda(cudaLaunchKernelEx(&cfg, shrink_rows_kernel<false>, P), "shrink_rows launch");
  if (st) return st;
  cfg.numAttrs = 1;
  const bool dense = T >= MINT_DENSE_MIN_BATCH;   // the plan may have given dense segments to the tensor-core kernels
  if (dense) {
    st = mint_launch_dense_shrink(args, nprob, tab, plan_dev, workspaces, lanes, P.dense_slot0, (int32_t)tiles, s);
    if (st) return st;
  }
  st = mint_check_cuda(cudaLaunchKernelEx(&cfg, expand_rows_kernel, P), "expand_rows launch");
  if (st || !dense) return st;
  return mint_launch_dense_expand(args, nprob, tab, plan_dev, workspaces, lanes, P.dense_slot0, (int32_t)tiles, s);
}

// ---- fused apply without a caller-provided workspace -------------------------------
// The workspace of the fused apply, held by the library itself so that a caller
// that cannot allocate device memory needs none: MINT_STATIC_WORKSPACE_BYTES of
// every GPU that loads this library, until the process exits.
static __device__ __align__(256) unsigned char g_static_workspace[MINT_STATIC_WORKSPACE_BYTES];

extern "C" int32_t mint_lora_apply_fused_static(const mint_pool *pool, const mint_slot_table *table,
                                                const void *plan_dev, int32_t T, const void *x_dev, int64_t ldx,
                                                void *y_dev, int64_t ldy, int32_t *status_dev,
                                                mint_stream_t stream) {
  if (!pool || !table) return mint_fail(MINT_ERR_INVALID_ARG, "apply_fused_static: null argument");
  // (tables that hold ranks above the streamed kernels' limit take the cluster kernel, which needs no workspace)
  const size_t need = mint_stream_supported(table->max_rank) ? mint_lora_apply_workspace_bytes(pool, T) : 0;
  if (need > (size_t)MINT_STATIC_WORKSPACE_BYTES)
    return mint_fail(MINT_ERR_WORKSPACE_TOO_SMALL,
                     "apply_fused_static: this batch needs %zu workspace bytes, the built-in workspace has %zu; "
                     "use mint_lora_apply_fused with a workspace of your own",
                     need, (size_t)MINT_STATIC_WORKSPACE_BYTES);
  // The array's name is only a handle on the host: its device address is looked
  // up once per device, with that device current.
  static std::atomic<void *> address[64];
  int dev = 0;
  int32_t st = mint_check_cuda(cudaGetDevice(&dev), "cudaGetDevice");
  if (st) return st;
  if (dev < 0 || dev >= 64) return mint_fail(MINT_ERR_UNSUPPORTED, "apply_fused_static: device ordinal %d", dev);
  void *ptr = address[dev].load(std::memory_order_acquire);
  if (ptr == nullptr) {
    st = mint_check_cuda(cudaGetSymbolAddress(&ptr, g_static_workspace), "address of the built-in workspace");
    if (st) return st;
    address[dev].store(ptr, std::memory_order_release);   // two first callers store the same value
  }
  return mint_lora_apply_fused(pool, table, plan_dev, T, x_dev, ldx, y_dev, ldy, ptr,
                               (size_t)MINT_STATIC_WORKSPACE_BYTES, status_dev, stream);
}
