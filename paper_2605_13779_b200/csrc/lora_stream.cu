// Streamed LoRA apply: the fused path of mint_lora_apply_fused, of its grouped
// form and (with the packed per-expert layout) of mint_moe_lora_apply.
//
//   shrink_stream_kernel : v[tile] = X[tile rows, :] . A_slot           (d -> r)
//   expand_stream_kernel : Y[tile rows, :] += s_slot * v[tile] . B_slot  (r -> n)
//
// Work split.  The work of a call is the area  rows x column blocks  where
// rows runs over the plan's tiles (a tile = at most 32 tokens of one segment)
// and columns over the column blocks (32 elements of d for the shrink, 64
// elements of n for the expand) of all projections of the call, laid side by
// side.  A tile counts as many rows as a column block of it costs: the rows it
// streams (rank + len for the shrink, rank + 2 len for the expand) plus a
// constant (mint_tile_rows_shrink / _expand), and every projection's columns
// are preceded by a few empty blocks that stand for the fixed cost of starting
// on a (tile, projection) piece.  The grid is three 128-thread CTAs per SM
// ("lanes"); lane c takes the c-th equal share of the area, walked tile by
// tile: a share starts in the middle of one tile, covers whole tiles, and ends
// in the middle of another.  The plan tabulates the tile in which every lane
// starts (that does not depend on the widths), so a lane finds its work with
// two table reads, and the lanes finish at about the same time.
//
// Data path.  No block-level staging: every warp owns a ring of 512-byte slots in
// shared memory (kRingSlots, Ring<N>); each lane copies the 16-byte segments it
// will use itself into its own column of the ring with cp.async and reads them
// back after cp.async.wait_group, so the pipeline needs no barrier and no
// registers for the bytes in flight.  The segments are exactly the operand
// fragments of the warp-level tensor-core MMA (m16n8k16, bf16 in, fp32 accumulate).
//  - shrink: both operands have the reduction index contiguous in memory (a row
//    of x, a row of A).  Lane (g, t) of a warp loads 16 bytes = 8 consecutive
//    elements of row g at offset 8 t of a 32-element block; elements (0,1) and
//    (2,3) serve as the two k-halves of one MMA step, (4,5) and (6,7) of the
//    next.  Both operands use the same permutation of k, so the sum is unchanged
//    and every 32-byte sector fetched is used in full.  Rows beyond the tile's
//    length or the slot's rank are not loaded at all (zero registers).
//  - expand: B is [rank][n] with n contiguous.  Lane (g, t) loads 16 bytes of
//    rows 2t, 2t+1, 2t+8, 2t+9 at the 8-column chunk c(g) = 4 (g & 1) + g / 2
//    of a 64-column block and pairs them with one byte-permute per MMA tile;
//    tile j holds the columns 8 c(g) + j, so the lane ends up owning the chunks
//    t and 4 + t of y for rows g and g+8, and every y access of the warp covers
//    64 contiguous bytes (two whole sectors) of each of eight rows: y is read,
//    updated (one fp32 fma, one round-to-nearest-even) and written with 128-bit
//    accesses.  (Chunks 2t and 2t + 1 would give each lane 32 contiguous bytes
//    but make every access touch half sectors, which halves the bandwidth.)  v enters as a bf16 head plus a bf16 remainder (two
//    MMAs), about 16 significant bits of the fp32 shrink result.
//  - tiles of rank 1 with at most 8 tokens (most of a large-catalog decode
//    batch) skip the MMA: plain fp32 FMAs over fully coalesced 512-byte warp loads.
// The four warps of a CTA split the column blocks of a piece; HBM latency is
// hidden by the cp.async rings of 12 warps per SM (an iteration of N segments
// runs kRingSlots / N iterations ahead) and, before the dependency wait of a
// launch, by prefetching the weights of the lane's first piece into L2.
//
// v travels from the shrink to the expand through a small L2-resident
// workspace: every shrink lane writes the sum over its own columns of a tile
// (slot tile + lane, so no two writers meet), and the expand, which knows the
// shrink's split from the same arithmetic, adds the lanes of a tile in lane
// order while it builds its operand fragments.  No atomics, no fences, and the
// result does not depend on scheduling.
//
// Launch overlap: both kernels let their successor become resident at once
// (griddepcontrol.launch_dependents first thing) and are launched with
// programmatic stream serialization.  Before its dependency wait a kernel reads
// only the plan, the slot table and pool weights, which no apply kernel writes
// (the first apply kernel after a plan, bind or evict kernel is launched without
// programmatic serialization, so those have completed before it starts);
// activations, y and v are touched only after the wait, and every CTA executes
// the wait before it exits so that completion stays transitive along the stream.
#include <algorithm>
#include <atomic>

#include "mint_device.cuh"

using namespace mint;

namespace {

constexpr int kWarps = 4;
constexpr int kThreads = kWarps * 32;
constexpr int kCtasPerSm = 3;
constexpr int kRingSlots = 26;            // 512-byte slots (16 B per lane) of a warp's staging ring
constexpr int kRingBytes = kRingSlots * 512;
constexpr int kTileRowsMax = 32;          // plan tile list 1
constexpr int kStreamRankCap = 64;        // larger ranks take the CUDA-core cluster kernel
constexpr int kBatchTiles = 16;           // tile descriptors staged in shared memory at a time
constexpr int kBatchItems = kBatchTiles * kTileRowsMax;
constexpr int kShrinkBlock = 32;          // elements of d per column block
constexpr int kExpandBlock = 64;          // elements of n per column block
constexpr int kShrinkGrain = 128;         // smallest lane share in (row x block) units: 128 x 64 B
constexpr int kExpandGrain = 64;          //                                           64 x 128 B
// What starting on a (tile, projection) costs a lane, in column blocks of that tile: the pipeline fill, the
// barriers and the hand-over of v.  Every projection's columns are preceded by this many empty blocks in
// the area, so a share that meets several projections gets fewer real blocks.
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
  int32_t dual;        // packed MoE pools: 1: the shrink pieces of this problem also shrink the next one, which
                       // reads the same x (gate and up); 2: this problem's v comes from the previous one's pieces
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
  int32_t lanes;                      // grid size = the plan's lane count
  int32_t cb_shrink, cb_expand;       // virtual column blocks of the whole call
  int32_t cb_shrink_widest;           // column blocks of the widest d of the call
  int32_t dense_slot0;                // first workspace slot of the dense segments' tiles (slot dense_slot0 + tile)
  int32_t *status;
  TableDev tab;
  PlanView pv;
};

// ---- small device helpers ------------------------------------------------------
__device__ __forceinline__ void pdl_launch_dependents() {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void prefetch_l2(const void *p) {
  asm volatile("prefetch.global.L2 [%0];" ::"l"(p));
}
__device__ __forceinline__ uint32_t smem_addr(const void *p) {
  return (uint32_t)__cvta_generic_to_shared(p);
}
// 16-byte asynchronous copy global -> shared, L2 only; zero-fills when !valid (nothing is read then).
__device__ __forceinline__ void cp_async16(uint32_t dst, const void *src, bool valid) {
  const int bytes = valid ? 16 : 0;
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
  asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ uint4 zero4() { return make_uint4(0u, 0u, 0u, 0u); }
// Four 8x8 bf16 matrices (eight 16-byte rows each; lane i gives the address of row i % 8 of
// matrix i / 8), transposed: lane (g, t) gets elements [2t][g], [2t+1][g] of each.
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(addr)
               : "memory");
}
__device__ __forceinline__ uint4 lds128(uint32_t addr) {
  uint4 r;
  asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w) : "r"(addr));
  return r;
}

// A warp's private staging ring.  Every lane copies the 16-byte segments it will
// use itself into its own column of the ring (slot s, lane l at byte (s * 32 +
// l) * 16) and reads them back after cp.async.wait_group: no thread ever reads
// another thread's copy, so the pipeline needs no barrier, costs no registers
// for the bytes in flight, and an iteration of N segments runs kRingSlots / N
// iterations ahead.
template <int N>
struct Ring {
  static constexpr int kDepth = kRingSlots / N;
  static_assert(kDepth >= 1, "an iteration does not fit the ring");
  uint32_t base;   // shared-memory address of this lane's column
  __device__ __forceinline__ uint32_t slot(int it, int i) const {
    return base + (uint32_t)(((it % kDepth) * N + i) * 512);
  }
};

// D(16x8, f32) += A(16x16, bf16, row) * B(16x8, bf16, col)
__device__ __forceinline__ void mma_bf16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                         uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
      "{%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pair_lo(uint32_t a, uint32_t b) { return __byte_perm(a, b, 0x5410); }
__device__ __forceinline__ uint32_t pair_hi(uint32_t a, uint32_t b) { return __byte_perm(a, b, 0x7632); }
__device__ __forceinline__ uint32_t word(const uint4 &q, int i) {
  return i == 0 ? q.x : (i == 1 ? q.y : (i == 2 ? q.z : q.w));
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
  int G;         // lanes the plan's table was cut for (= grid size)
  int active;    // lanes that take work
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

struct CtaShared {
  TileDesc desc[kBatchTiles];
  int32_t rows[kBatchItems];
  int32_t part_first[kBatchTiles * kMaxProblems];   // expand: first shrink lane holding a part of (tile, problem)
  int16_t part_count[kBatchTiles * kMaxProblems];   //         and how many consecutive lanes do
  int32_t range[4];
};

template <bool kExpand>
__device__ __forceinline__ bool prologue(const StreamParams &P, CtaShared &sh, Area &area, CtaRange &R,
                                         bool report_errors) {
  // (Nothing of the plan beyond its header is read before the header has been checked: a blob
  // made for another batch size has its arrays elsewhere.)
  const int c = blockIdx.x;
  if (!plan_ok(P.pv.header, P.T, P.K, P.tab.num_slots, P.num_experts, P.tab.gen_lo, P.tab.gen_hi,
               report_errors ? P.status : nullptr))
    return false;
  if (P.pv.header[PH_LANES] != P.lanes) {
    if (threadIdx.x == 0 && report_errors) report(P.status, MINT_ERR_SHAPE_MISMATCH, P.pv.header[PH_LANES]);
    return false;
  }
  const int ntiles = P.pv.header[PH_NCHUNK1];
  if (ntiles == 0) return false;
  // nothing streamed: every tile belongs to a dense segment (the tensor-core kernels take those)
  if (P.pv.header[kExpand ? PH_ROWS_EXPAND : PH_ROWS_SHRINK] == 0) return false;
  area = make_area<kExpand>(P);
  if (c >= area.active) return false;
  if (threadIdx.x < 2) {   // thread 0: the cut where this lane starts; thread 1: where it ends
    const int j = lane_index(area, c + threadIdx.x);
    const LaneStart ls = area.table[j];
    const int cb = j < area.G ? (int)(lane_offset(area, ls, ls.rows) / ls.w) : 0;
    sh.range[2 * threadIdx.x] = ls.tile;
    sh.range[2 * threadIdx.x + 1] = cb;
  }
  __syncthreads();
  R.t0 = sh.range[0];
  R.cb0 = sh.range[1];
  R.t1 = sh.range[2];
  R.cb1 = sh.range[3];
  R.t_end = (R.cb1 > 0) ? R.t1 + 1 : R.t1;
  return R.t_end > R.t0;
}

// Stages the descriptors and the row indices of tiles [tb, tb + ntile) (all threads).
// kRowsOfX (the shrink of a MoE call): the rows are those of x that the pairs
// read; a pair whose row is out of range is reported and gets row -1 (its x
// counts as zero, so its y stays as it is).
template <bool kRowsOfX>
__device__ __forceinline__ void load_batch(const StreamParams &P, CtaShared &sh, int tb, int ntile) {
  __syncthreads();  // every warp is done with the previous batch
  const int4 *src = reinterpret_cast<const int4 *>(P.pv.tile_desc + tb);
  int4 *dst = reinterpret_cast<int4 *>(sh.desc);
  for (int i = threadIdx.x; i < ntile * (int)(sizeof(TileDesc) / 16); i += kThreads) dst[i] = src[i];
  __syncthreads();
  const int off0 = sh.desc[0].off;
  const int nitems = sh.desc[ntile - 1].off + sh.desc[ntile - 1].len - off0;
  for (int i = threadIdx.x; i < nitems; i += kThreads) {
    const int p = P.pv.perm[off0 + i];
    int row = p;
    if (kRowsOfX) {
      if (P.x_row) row = P.x_row[p];
      if (row < 0 || row >= P.x_rows) {
        report(P.status, MINT_ERR_BAD_INDEX, p);
        row = -1;
      }
    }
    sh.rows[i] = row;
  }
  __syncthreads();
}

struct Piece {
  int t;        // tile
  int p;        // problem
  int lo, hi;   // column blocks of the problem [lo, hi)
  int blocks;   // column blocks of the problem's whole width
  const int32_t *rows;   // the tile's row indices (shared memory)
  int r, len;
  int slot;     // weight block: the slot, or slot * experts + expert
  float scale;
  int lane_lo, lane_hi;   // bounds of the shrink lanes that can meet this tile
  int ti;                 // index of the tile in the staged batch
};

// Walks the pieces of one batch of tiles in order; f(piece) is called by all threads.
template <bool kExpand, class F>
__device__ __forceinline__ void walk_batch(const StreamParams &P, const Area &area, const CtaRange &R,
                                           const CtaShared &sh, int tb, int ntile, F &&f) {
  constexpr int kBlock = kExpand ? kExpandBlock : kShrinkBlock;
  for (int ti = 0; ti < ntile; ++ti) {
    const int t = tb + ti;
    const int va = (t == R.t0) ? R.cb0 : 0;
    const int vb = (t == R.t1) ? R.cb1 : area.CB;
    if (va >= vb) continue;
    if (sh.desc[ti].dense) continue;   // it runs on the 128-row tensor-core kernels
    Piece pc;
    pc.t = t;
    pc.ti = ti;
    pc.r = sh.desc[ti].rank;
    pc.len = sh.desc[ti].len;
    pc.scale = sh.desc[ti].scale;
    pc.slot = sh.desc[ti].slot * P.weights_per_slot + sh.desc[ti].expert;
    pc.lane_lo = sh.desc[ti].lane_lo;
    pc.lane_hi = sh.desc[ti].lane_hi;
    pc.rows = sh.rows + (sh.desc[ti].off - sh.desc[0].off);
    for (int p = 0; p < P.nprob; ++p) {
      const StreamProblem &pb = P.prob[p];
      if (!kExpand && pb.dual == 2) continue;   // shrunk together with the problem before it
      const int width = kExpand ? pb.n : pb.d;
      const int first = kExpand ? pb.cb0_expand : pb.cb0_shrink;
      const int count = (width + kBlock - 1) / kBlock;
      const int lo = max(va, first) - first, hi = min(vb, first + count) - first;
      if (lo >= hi) continue;
      pc.p = p;
      pc.lo = lo;
      pc.hi = hi;
      pc.blocks = count;
      f(pc);
    }
  }
}

// Pulls the rows of a piece into L2 (all threads): the weight rows, which no apply
// kernel writes, may go before the dependency wait; activations only after it.
template <bool kExpand, bool kPackedA = false>
__device__ __forceinline__ void prefetch_piece(const StreamProblem &pb, const Piece &pc, bool weights, bool acts) {
  constexpr int kBlock = kExpand ? kExpandBlock : kShrinkBlock;
  const int width = kExpand ? pb.n : pb.d;
  const int c0 = pc.lo * kBlock, c1 = min(pc.hi * kBlock, width);
  const int lines = ((c1 - c0) * 2 + 127) / 128 + 1;   // one address per 128 bytes, plus the last 16 bytes
  if (weights && kPackedA) {
    // A[d][r_max]: the piece's rows c0..c1 are one contiguous run
    const uint16_t *w = pb.A + ((int64_t)pc.slot * pb.d + c0) * pb.r_max;
    const int total = (c1 - c0) * pb.r_max;
    for (int i = threadIdx.x * 64; i < total; i += kThreads * 64) prefetch_l2(w + i);
  } else if (weights) {
    const uint16_t *w = (kExpand ? pb.B : pb.A) + (int64_t)pc.slot * pb.r_max * width;
    for (int i = threadIdx.x; i < pc.r * lines; i += kThreads) {
      const int row = i / lines, ln = i - row * lines;
      prefetch_l2(w + (int64_t)row * width + min(c0 + ln * 64, c1 - 8));
    }
  }
  if (acts) {
    const uint16_t *a = kExpand ? pb.y : pb.x;
    const int64_t ld = kExpand ? pb.ldy : pb.ldx;
    for (int i = threadIdx.x; i < pc.len * lines; i += kThreads) {
      const int row = i / lines, ln = i - row * lines;
      prefetch_l2(a + (int64_t)pc.rows[row] * ld + min(c0 + ln * 64, c1 - 8));
    }
  }
}

// ================================================================================
// shrink
// ================================================================================
// Tensor-core body for ranks [rh, rh + 8 NT) of the piece: this warp's blocks.
// XG = groups of 8 token rows, NT = groups of 8 rank rows: only row groups that
// exist take a slot of the staging ring, so a skinny tile runs deep.
template <int XG, int NT>
__device__ __forceinline__ void shrink_mma(const StreamProblem &pb, const Piece &pc, int rh, uint32_t ring_base,
                                           float *scratch) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, t = lane & 3;
  constexpr int N = XG + NT;
  constexpr int MT = (XG + 1) / 2;
  Ring<N> ring{ring_base};
  const uint16_t *A_slot = pb.A + (int64_t)pc.slot * pb.r_max * pb.d;
  const uint16_t *src[N];   // this lane's row of every operand fragment (nullptr: the row does not exist)
#pragma unroll
  for (int i = 0; i < XG; ++i) {
    const int row = i * 8 + g;
    src[i] = row < pc.len ? pb.x + (int64_t)pc.rows[row] * pb.ldx + t * 8 : nullptr;
  }
#pragma unroll
  for (int i = 0; i < NT; ++i) {
    const int row = rh + i * 8 + g;
    src[XG + i] = row < pc.r ? A_slot + (int64_t)row * pb.d + t * 8 : nullptr;
  }
  float acc[MT][NT][4];
#pragma unroll
  for (int a = 0; a < MT; ++a)
#pragma unroll
    for (int b = 0; b < NT; ++b)
#pragma unroll
      for (int e = 0; e < 4; ++e) acc[a][b][e] = 0.f;

  const int first = pc.lo + warp;
  const int iters = first < pc.hi ? (pc.hi - first + kWarps - 1) / kWarps : 0;
  auto issue = [&](int it) {
    if (it < iters) {
      const int col = (first + it * kWarps) * kShrinkBlock;
      const bool ok = col + t * 8 < pb.d;
#pragma unroll
      for (int i = 0; i < N; ++i) cp_async16(ring.slot(it, i), src[i] ? src[i] + col : pb.A, ok && src[i]);
    }
    cp_async_commit();
  };
#pragma unroll 1
  for (int it = 0; it < Ring<N>::kDepth - 1; ++it) issue(it);
#pragma unroll 1
  for (int it = 0; it < iters; ++it) {
    issue(it + Ring<N>::kDepth - 1);
    cp_async_wait<Ring<N>::kDepth - 1>();
    uint4 xa[2 * MT], wb[NT];
#pragma unroll
    for (int i = 0; i < 2 * MT; ++i) xa[i] = i < XG ? lds128(ring.slot(it, i)) : zero4();
#pragma unroll
    for (int i = 0; i < NT; ++i) wb[i] = lds128(ring.slot(it, XG + i));
#pragma unroll
    for (int ks = 0; ks < 2; ++ks)
#pragma unroll
      for (int mt = 0; mt < MT; ++mt)
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
          mma_bf16(acc[mt][nt], word(xa[2 * mt], 2 * ks), word(xa[2 * mt + 1], 2 * ks),
                   word(xa[2 * mt], 2 * ks + 1), word(xa[2 * mt + 1], 2 * ks + 1), word(wb[nt], 2 * ks),
                   word(wb[nt], 2 * ks + 1));
  }
  cp_async_wait<0>();
  __syncthreads();   // the gather of the previous pass has read the scratch
  // scratch[warp][mt][nt][lane][4]
#pragma unroll
  for (int mt = 0; mt < MT; ++mt)
#pragma unroll
    for (int nt = 0; nt < NT; ++nt)
      *reinterpret_cast<float4 *>(scratch + (((warp * 2 + mt) * 4 + nt) * 32 + lane) * 4) =
          make_float4(acc[mt][nt][0], acc[mt][nt][1], acc[mt][nt][2], acc[mt][nt][3]);
}

// The same for the packed MoE layout A[d][r_max] (RG = r_max / 8 groups of 8
// ranks per row of A): the 32 rows of a column block are one contiguous run of
// memory, which the warp copies with coalesced 16-byte segments into its ring,
// each segment going where an 8x8 matrix of the transposing ldmatrix expects it:
// matrix (k-step, k-half, rank group), row j <-> row k = 8 (j / 2) + 4 step + 2 half + j % 2
// of the block, the same permutation of k that the x fragments use.  A pass covers
// min(RG, 4) rank groups from rank rh on; segments of rank groups at or beyond
// the slot's rank are not read.
// kDual (RG <= 2): the rank groups of a second pool with the same shape follow those of the
// first (pb2: same x, same d and r_max), so that one pass over x shrinks both.
template <int XG, int RG, bool kDual = false>
__device__ __forceinline__ void shrink_mma_packed(const StreamProblem &pb, const Piece &pc, int rh,
                                                  uint32_t ring_base, float *scratch,
                                                  const StreamProblem *pb2 = nullptr) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, t = lane & 3;
  constexpr int NT = kDual ? 2 * RG : (RG < 4 ? RG : 4);
  static_assert(!kDual || RG <= 2, "two pools share a pass only up to 16 ranks each");
  constexpr int N = XG + NT;
  constexpr int MT = (XG + 1) / 2;
  Ring<N> ring{ring_base};
  const uint32_t warp_base = ring_base - (uint32_t)lane * 16;
  const uint16_t *A_w = pb.A + (int64_t)pc.slot * pb.d * pb.r_max;
  const uint16_t *A_w2 = kDual ? pb2->A + (int64_t)pc.slot * pb.d * pb.r_max : nullptr;
  const uint16_t *xsrc[XG];
#pragma unroll
  for (int i = 0; i < XG; ++i) {
    const int row = i * 8 + g;
    const int xr = row < pc.len ? pc.rows[row] : -1;
    xsrc[i] = xr >= 0 ? pb.x + (int64_t)xr * pb.ldx + t * 8 : nullptr;
  }
  // this lane's segment of every 512-byte slot of a block of A: where it comes from, where it goes
  int a_off[NT], a_k[NT];
  uint32_t a_dst[NT];
  bool a_second[NT];
#pragma unroll
  for (int j = 0; j < NT; ++j) {
    const int c = j * 32 + lane, k = c / NT, rgl = c % NT;
    const int rg = kDual ? rgl % RG : (rh >> 3) + rgl;   // rank group inside its pool
    a_second[j] = kDual && rgl >= RG;
    a_off[j] = k * pb.r_max + rg * 8;
    a_k[j] = rg * 8 < pc.r ? k : (1 << 30);
    const int m = (((k >> 2) & 1) * 2 + ((k >> 1) & 1)) * NT + rgl, jj = 2 * (k >> 3) + (k & 1);
    a_dst[j] = (uint32_t)((m * 8 + jj) * 16);
  }
  // ldmatrix addresses: NT == 1: one x4 gives (step 0: half 0, half 1; step 1: half 0, half 1);
  // otherwise one x4 per (step, pair of rank groups): (group: half 0, half 1; group + 1: half 0, half 1)
  uint32_t lm_off[NT == 1 ? 1 : NT];
  if (NT == 1) {
    lm_off[0] = (uint32_t)lane * 16;
  } else {
#pragma unroll
    for (int ks = 0; ks < 2; ++ks)
#pragma unroll
      for (int np = 0; np < NT / 2; ++np) {
        const int mi = lane >> 3, h = mi & 1, nt = 2 * np + (mi >> 1);
        lm_off[ks * (NT / 2) + np] = (uint32_t)((((ks * 2 + h) * NT + nt) * 8 + (lane & 7)) * 16);
      }
  }
  float acc[MT][NT][4];
#pragma unroll
  for (int a = 0; a < MT; ++a)
#pragma unroll
    for (int b = 0; b < NT; ++b)
#pragma unroll
      for (int e = 0; e < 4; ++e) acc[a][b][e] = 0.f;

  const int first = pc.lo + warp;
  const int iters = first < pc.hi ? (pc.hi - first + kWarps - 1) / kWarps : 0;
  auto a_region = [&](int it) { return warp_base + (uint32_t)(((it % Ring<N>::kDepth) * N + XG) * 512); };
  auto issue = [&](int it) {
    if (it < iters) {
      const int col = (first + it * kWarps) * kShrinkBlock;
      const bool ok = col + t * 8 < pb.d;
#pragma unroll
      for (int i = 0; i < XG; ++i) cp_async16(ring.slot(it, i), xsrc[i] ? xsrc[i] + col : pb.A, ok && xsrc[i]);
      const uint16_t *blk = A_w + (int64_t)col * pb.r_max;
      const uint16_t *blk2 = kDual ? A_w2 + (int64_t)col * pb.r_max : nullptr;
      const uint32_t dst = a_region(it);
#pragma unroll
      for (int j = 0; j < NT; ++j) {
        const bool ok_a = col + a_k[j] < pb.d;
        cp_async16(dst + a_dst[j], ok_a ? ((kDual && a_second[j]) ? blk2 : blk) + a_off[j] : pb.A, ok_a);
      }
    }
    cp_async_commit();
  };
#pragma unroll 1
  for (int it = 0; it < Ring<N>::kDepth - 1; ++it) issue(it);
#pragma unroll 1
  for (int it = 0; it < iters; ++it) {
    issue(it + Ring<N>::kDepth - 1);
    cp_async_wait<Ring<N>::kDepth - 1>();
    __syncwarp();   // every lane's segments of this block have landed
    uint4 xa[2 * MT];
#pragma unroll
    for (int i = 0; i < 2 * MT; ++i) xa[i] = i < XG ? lds128(ring.slot(it, i)) : zero4();
    const uint32_t region = a_region(it);
    uint32_t wb[2][NT][2];   // [k-step][rank group][k-half]
    if (NT == 1) {
      uint32_t r4[4];
      ldmatrix_x4_trans(r4, region + lm_off[0]);
      wb[0][0][0] = r4[0]; wb[0][0][1] = r4[1]; wb[1][0][0] = r4[2]; wb[1][0][1] = r4[3];
    } else {
#pragma unroll
      for (int ks = 0; ks < 2; ++ks)
#pragma unroll
        for (int np = 0; np < NT / 2; ++np) {
          uint32_t r4[4];
          ldmatrix_x4_trans(r4, region + lm_off[ks * (NT / 2) + np]);
          wb[ks][2 * np][0] = r4[0]; wb[ks][2 * np][1] = r4[1];
          wb[ks][2 * np + 1][0] = r4[2]; wb[ks][2 * np + 1][1] = r4[3];
        }
    }
    __syncwarp();   // all lanes have read the block before its slots are refilled
#pragma unroll
    for (int ks = 0; ks < 2; ++ks)
#pragma unroll
      for (int mt = 0; mt < MT; ++mt)
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
          mma_bf16(acc[mt][nt], word(xa[2 * mt], 2 * ks), word(xa[2 * mt + 1], 2 * ks),
                   word(xa[2 * mt], 2 * ks + 1), word(xa[2 * mt + 1], 2 * ks + 1), wb[ks][nt][0], wb[ks][nt][1]);
  }
  cp_async_wait<0>();
  __syncthreads();   // the gather of the previous pass has read the scratch
#pragma unroll
  for (int mt = 0; mt < MT; ++mt)
#pragma unroll
    for (int nt = 0; nt < NT; ++nt)
      *reinterpret_cast<float4 *>(scratch + (((warp * 2 + mt) * 4 + nt) * 32 + lane) * 4) =
          make_float4(acc[mt][nt][0], acc[mt][nt][1], acc[mt][nt][2], acc[mt][nt][3]);
}

// rank-1 tiles of at most L tokens: fp32 FMAs over coalesced 512-byte warp loads.
template <int L>
__device__ __forceinline__ void shrink_vec(const StreamProblem &pb, const Piece &pc, uint32_t ring_base,
                                           float *scratch) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  constexpr int N = 1 + L;
  Ring<N> ring{ring_base};
  const uint16_t *w = pb.A + (int64_t)pc.slot * pb.r_max * pb.d;
  const uint16_t *xr[L];
#pragma unroll
  for (int l = 0; l < L; ++l) xr[l] = pb.x + (int64_t)pc.rows[l < pc.len ? l : 0] * pb.ldx;
  float acc[L];
#pragma unroll
  for (int l = 0; l < L; ++l) acc[l] = 0.f;
  const int c0 = pc.lo * kShrinkBlock + warp * 256 + lane * 8, c1 = min(pc.hi * kShrinkBlock, pb.d);
  constexpr int kStep = kWarps * 256;
  const int iters = (c1 - (pc.lo * kShrinkBlock + warp * 256) + kStep - 1) / kStep;   // <= 0: nothing for this warp
  auto issue = [&](int it) {
    if (it < iters) {
      const int col = c0 + it * kStep;
      const bool ok = col < c1;
      cp_async16(ring.slot(it, 0), ok ? w + col : w, ok);
#pragma unroll
      for (int l = 0; l < L; ++l) cp_async16(ring.slot(it, 1 + l), ok ? xr[l] + col : w, ok && l < pc.len);
    }
    cp_async_commit();
  };
#pragma unroll 1
  for (int it = 0; it < Ring<N>::kDepth - 1; ++it) issue(it);
#pragma unroll 1
  for (int it = 0; it < iters; ++it) {
    issue(it + Ring<N>::kDepth - 1);
    cp_async_wait<Ring<N>::kDepth - 1>();
    float wf[8];
    unpack8(lds128(ring.slot(it, 0)), wf);
#pragma unroll
    for (int l = 0; l < L; ++l) {
      float xf[8];
      unpack8(lds128(ring.slot(it, 1 + l)), xf);
#pragma unroll
      for (int e = 0; e < 8; ++e) acc[l] = fmaf(xf[e], wf[e], acc[l]);
    }
  }
  cp_async_wait<0>();
  __syncthreads();   // the gather of the previous pass has read the scratch
#pragma unroll
  for (int l = 0; l < L; ++l) {
    const float s = warp_sum(acc[l]);
    if (lane == 0) scratch[warp * 8 + l] = s;
  }
}

struct SmemShrink {
  CtaShared sh;
  float scratch[kWarps * 2 * 4 * 128];   // [warp][m-tile][n-tile][lane][4] MMA fragments, or [warp][8] sums
};

template <bool kPacked>
__device__ __forceinline__ void shrink_piece(const StreamParams &P, SmemShrink &S, uint32_t ring_base,
                                             const Piece &pc) {
  const StreamProblem &pb = P.prob[pc.p];
  const int tid = threadIdx.x;
  const size_t slot_floats = (size_t)kTileRowsMax * pb.r_max;
  // the sum over this lane's columns; the expand adds the lanes of a tile in lane order
  float *dst = pb.ws_part + (size_t)(pc.t + blockIdx.x) * slot_floats;
  const bool vec = !kPacked && pc.r == 1 && pc.len <= 8;
  if (kPacked && pb.dual == 1) {
    // this problem and the next one (same x, same shape, at most 16 ranks) in one pass over x
    const StreamProblem &pb2 = P.prob[pc.p + 1];
    const int rg = pb.r_max >> 3;
#define MINT_SHRINK_CASE(XG)                                                                    \
  if (rg == 1) shrink_mma_packed<XG, 1, true>(pb, pc, 0, ring_base, S.scratch, &pb2);          \
  else shrink_mma_packed<XG, 2, true>(pb, pc, 0, ring_base, S.scratch, &pb2)
    if (pc.len <= 16) { MINT_SHRINK_CASE(2); }
    else { MINT_SHRINK_CASE(4); }
#undef MINT_SHRINK_CASE
    __syncthreads();
    float *dst2 = pb2.ws_part + (size_t)(pc.t + blockIdx.x) * slot_floats;
    for (int i = tid; i < 2 * pc.len * pc.r; i += kThreads) {
      const int second = i >= pc.len * pc.r, e = second ? i - pc.len * pc.r : i;
      const int l = e / pc.r, j = e - l * pc.r;
      const int mt = l >> 4, g = l & 15, nt = second * rg + (j >> 3), cc = j & 7;
      const int frag = ((g & 7) * 4 + (cc >> 1)) * 4 + (g >> 3) * 2 + (cc & 1);
      float s = 0.f;
#pragma unroll
      for (int w = 0; w < kWarps; ++w) s += S.scratch[((w * 2 + mt) * 4 + nt) * 128 + frag];
      (second ? dst2 : dst)[l * pc.r + j] = s;
    }
    return;
  }
  for (int rh = 0; rh < pc.r; rh += 32) {
    const int rr = min(32, pc.r - rh);
    // (the bodies wait, right before they write the scratch, until the previous gather has read it)
    if (kPacked) {
      const int rg = pb.r_max >> 3;
#define MINT_SHRINK_CASE(XG)                                                          \
  if (rg == 1) shrink_mma_packed<XG, 1>(pb, pc, rh, ring_base, S.scratch);            \
  else if (rg == 2) shrink_mma_packed<XG, 2>(pb, pc, rh, ring_base, S.scratch);       \
  else if (rg == 4) shrink_mma_packed<XG, 4>(pb, pc, rh, ring_base, S.scratch);       \
  else shrink_mma_packed<XG, 8>(pb, pc, rh, ring_base, S.scratch)
      // (one group of 8 token rows would run the same MMAs as two; fewer bodies keep the kernel's code small)
      if (pc.len <= 16) { MINT_SHRINK_CASE(2); }
      else { MINT_SHRINK_CASE(4); }
#undef MINT_SHRINK_CASE
    } else if (vec) {
      if (pc.len == 1) shrink_vec<1>(pb, pc, ring_base, S.scratch);
      else if (pc.len == 2) shrink_vec<2>(pb, pc, ring_base, S.scratch);
      else if (pc.len <= 4) shrink_vec<4>(pb, pc, ring_base, S.scratch);
      else shrink_vec<8>(pb, pc, ring_base, S.scratch);
    } else {
      const int ng = rr <= 8 ? 1 : (rr <= 16 ? 2 : 4);
#define MINT_SHRINK_CASE(XG)                                                        \
  if (ng == 1) shrink_mma<XG, 1>(pb, pc, rh, ring_base, S.scratch);                 \
  else if (ng == 2) shrink_mma<XG, 2>(pb, pc, rh, ring_base, S.scratch);            \
  else shrink_mma<XG, 4>(pb, pc, rh, ring_base, S.scratch)
      // (one group of 8 token rows would run the same MMAs as two; fewer bodies keep the kernel's code small)
      if (pc.len <= 16) { MINT_SHRINK_CASE(2); }
      else { MINT_SHRINK_CASE(4); }
#undef MINT_SHRINK_CASE
    }
    __syncthreads();
    // add the four warps' sums in warp order; element (l, rh + j) of the [len][rank] result
    for (int i = tid; i < pc.len * rr; i += kThreads) {
      const int l = i / rr, j = i - l * rr;
      float s = 0.f;
      if (vec) {
#pragma unroll
        for (int w = 0; w < kWarps; ++w) s += S.scratch[w * 8 + l];
      } else {
        const int mt = l >> 4, g = l & 15, nt = j >> 3, cc = j & 7;
        const int frag = ((g & 7) * 4 + (cc >> 1)) * 4 + (g >> 3) * 2 + (cc & 1);
#pragma unroll
        for (int w = 0; w < kWarps; ++w) s += S.scratch[((w * 2 + mt) * 4 + nt) * 128 + frag];
      }
      dst[l * pc.r + rh + j] = s;
    }
  }
}

constexpr size_t kRingsBytes = (size_t)kWarps * kRingBytes;

template <bool kPacked>
__global__ void __launch_bounds__(kThreads, kCtasPerSm) shrink_stream_kernel(const __grid_constant__ StreamParams P) {
  extern __shared__ __align__(128) uint8_t dyn_smem[];   // the four warps' rings
  __shared__ SmemShrink S;
  pdl_launch_dependents();
  Area area;
  CtaRange R;
  if (!prologue<false>(P, S.sh, area, R, true)) {
    pdl_wait();
    return;
  }
  const uint32_t ring_base =
      smem_addr(dyn_smem) + (uint32_t)((threadIdx.x >> 5) * kRingBytes + (threadIdx.x & 31) * 16);
  bool waited = false;
  for (int tb = R.t0; tb < R.t_end; tb += kBatchTiles) {
    const int ntile = min(kBatchTiles, R.t_end - tb);
    load_batch<kPacked>(P, S.sh, tb, ntile);
    if (!waited) {
      // while the previous kernel still runs: pull this lane's A rows into L2
      bool first_piece = true;   // only the piece the lane starts with: the rest follow behind its stream
      walk_batch<false>(P, area, R, S.sh, tb, ntile, [&](const Piece &pc) {
        if (first_piece) prefetch_piece<false, kPacked>(P.prob[pc.p], pc, true, false);
        first_piece = false;
      });
      pdl_wait();   // activations and the workspace belong to earlier kernels until here
      waited = true;
    }
    walk_batch<false>(P, area, R, S.sh, tb, ntile, [&](const Piece &pc) { shrink_piece<kPacked>(P, S, ring_base, pc); });
  }
}

// ================================================================================
// expand
// ================================================================================
// A piece of the expand runs in three steps.  (1) Every warp requests the first
// blocks of its share of the piece.  (2) While they are on their way, the CTA
// adds the shrink lanes' parts of v, element by element with coalesced loads
// (times the pair's routing weight in a MoE call), and turns the sums into MMA
// operand fragments.  (3) The warps stream their blocks.

// Splits v into a bf16 head and a bf16 remainder so that two MMAs carry about
// 16 significant bits of the fp32 shrink result into the expand.
__device__ __forceinline__ void split_pair(float a, float b, uint32_t &hi, uint32_t &lo) {
  hi = pack_bf16x2(a, b);
  lo = pack_bf16x2(a - bf16lo(hi), b - bf16hi(hi));
}

struct SmemExpand {
  CtaShared sh;
  // v of the current tile as MMA A-operand fragments: [m-tile][k-step][head/remainder][lane] x 4 registers
  uint4 vfrag[2 * 4 * 2 * 32];
  float vsum[kTileRowsMax * kStreamRankCap];   // v of the current tile, [len][rank], weighted
};

// 8 output columns of one row: y += scale * acc[j][e] for column j, stored with one 128-bit write
__device__ __forceinline__ void update8(uint16_t *yp, const uint4 &old, float scale, const float (&acc)[8][4], int e) {
  float f[8];
  unpack8(old, f);
#pragma unroll
  for (int j = 0; j < 8; ++j) f[j] = fmaf(scale, acc[j][e], f[j]);
  *reinterpret_cast<uint4 *>(yp) = pack8(f);
}

// The addresses a lane streams in a piece of the tensor-core path.  YG = groups
// of 8 token rows (two 16-byte segments of y each), KG = groups of 8 rank rows
// of B (rows 8 kg + 2t and 8 kg + 2t + 1): only groups that exist take slots of
// the staging ring.
template <int YG, int KG>
struct ExpandLane {
  static constexpr int N = 2 * KG + 2 * YG;
  static constexpr int MT = (YG + 1) / 2, KS = (KG + 1) / 2;
  Ring<N> ring;
  const uint16_t *bsrc[2 * KG];
  uint16_t *ysrc[YG];
  int first, iters, t, bchunk;

  __device__ __forceinline__ void init(const StreamProblem &pb, const Piece &pc, uint32_t ring_base) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = lane >> 2;
    t = lane & 3;
    ring.base = ring_base;
    const uint16_t *B_slot = pb.B + (int64_t)pc.slot * pb.r_max * pb.n;
    // n index g of every MMA tile stands for the 8-column chunk (g & 1) * 4 + (g >> 1) of the block, so that
    // the accumulators of lane (g, t) (n = 2t and 2t + 1) are the chunks t and 4 + t: one y access of the
    // warp then covers 64 contiguous bytes of each of 8 rows
    bchunk = (g & 1) * 4 + (g >> 1);
#pragma unroll
    for (int i = 0; i < 2 * KG; ++i) {
      const int k = (i >> 1) * 8 + 2 * t + (i & 1);
      bsrc[i] = k < pc.r ? B_slot + (int64_t)k * pb.n + bchunk * 8 : nullptr;
    }
#pragma unroll
    for (int i = 0; i < YG; ++i) {
      const int row = i * 8 + g;
      ysrc[i] = row < pc.len ? pb.y + (int64_t)pc.rows[row] * pb.ldy + t * 8 : nullptr;
    }
    first = pc.lo + warp;
    iters = first < pc.hi ? (pc.hi - first + kWarps - 1) / kWarps : 0;
  }
  __device__ __forceinline__ void issue(const StreamProblem &pb, int it) const {
    if (it < iters) {
      const int n0 = (first + it * kWarps) * kExpandBlock;
      const bool ok_b = n0 + bchunk * 8 < pb.n;
      const bool ok_y0 = n0 + t * 8 < pb.n, ok_y1 = n0 + 32 + t * 8 < pb.n;
#pragma unroll
      for (int i = 0; i < 2 * KG; ++i)
        cp_async16(ring.slot(it, i), bsrc[i] ? bsrc[i] + n0 : pb.B, ok_b && bsrc[i]);
#pragma unroll
      for (int i = 0; i < YG; ++i) {
        cp_async16(ring.slot(it, 2 * KG + 2 * i), ysrc[i] ? ysrc[i] + n0 : pb.B, ok_y0 && ysrc[i]);
        cp_async16(ring.slot(it, 2 * KG + 2 * i + 1), ysrc[i] ? ysrc[i] + n0 + 32 : pb.B, ok_y1 && ysrc[i]);
      }
    }
    cp_async_commit();
  }
};

// Step 1: the first blocks of this warp.
template <int YG, int KG>
__device__ __forceinline__ void expand_mma_fill(const StreamProblem &pb, const Piece &pc, uint32_t ring_base) {
  ExpandLane<YG, KG> L;
  L.init(pb, pc, ring_base);
#pragma unroll 1
  for (int it = 0; it < Ring<ExpandLane<YG, KG>::N>::kDepth - 1; ++it) L.issue(pb, it);
}

// Step 3: the blocks of this warp; the requests of expand_mma_fill are under way.
template <int YG, int KG>
__device__ __forceinline__ void expand_mma(const StreamProblem &pb, const Piece &pc, uint32_t ring_base,
                                           const SmemExpand &S) {
  using Lane = ExpandLane<YG, KG>;
  constexpr int N = Lane::N, MT = Lane::MT, KS = Lane::KS;
  constexpr int kDepth = Ring<N>::kDepth;
  const int lane = threadIdx.x & 31;
  Lane L;
  L.init(pb, pc, ring_base);
  const int t = L.t;
#pragma unroll 1
  for (int it = 0; it < L.iters; ++it) {
    L.issue(pb, it + kDepth - 1);
    cp_async_wait<kDepth - 1>();
    const int n0 = (L.first + it * kWarps) * kExpandBlock;
    const bool ok_y0 = n0 + t * 8 < pb.n, ok_y1 = n0 + 32 + t * 8 < pb.n;
#pragma unroll
    for (int mt = 0; mt < MT; ++mt) {
      float acc[8][4];
#pragma unroll
      for (int j = 0; j < 8; ++j)
#pragma unroll
        for (int e = 0; e < 4; ++e) acc[j][e] = 0.f;
#pragma unroll
      for (int ks = 0; ks < KS; ++ks) {
        // B rows 2t, 2t+1 (group 2 ks) and 2t+8, 2t+9 (group 2 ks + 1) of this k-step
        uint4 bq[4];
#pragma unroll
        for (int i = 0; i < 4; ++i)
          bq[i] = (2 * ks + (i >> 1) < KG) ? lds128(L.ring.slot(it, 2 * (2 * ks + (i >> 1)) + (i & 1))) : zero4();
        const uint4 vh = S.vfrag[((mt * 4 + ks) * 2 + 0) * 32 + lane];
        const uint4 vl = S.vfrag[((mt * 4 + ks) * 2 + 1) * 32 + lane];
        // four tiles at a time: the four head MMAs, then the four remainder MMAs, so that the two
        // MMAs into one accumulator are not back to back
#pragma unroll
        for (int j0 = 0; j0 < 8; j0 += 4) {
          uint32_t b0[4], b1[4];
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const int j = j0 + i;
            b0[i] = (j & 1) ? pair_hi(word(bq[0], j >> 1), word(bq[1], j >> 1))
                            : pair_lo(word(bq[0], j >> 1), word(bq[1], j >> 1));
            b1[i] = (j & 1) ? pair_hi(word(bq[2], j >> 1), word(bq[3], j >> 1))
                            : pair_lo(word(bq[2], j >> 1), word(bq[3], j >> 1));
          }
#pragma unroll
          for (int i = 0; i < 4; ++i) mma_bf16(acc[j0 + i], vh.x, vh.y, vh.z, vh.w, b0[i], b1[i]);
#pragma unroll
          for (int i = 0; i < 4; ++i) mma_bf16(acc[j0 + i], vl.x, vl.y, vl.z, vl.w, b0[i], b1[i]);
        }
      }
      // acc[j][0], [1]: row g, columns 8 t + j and 32 + 8 t + j; acc[j][2], [3]: row g + 8
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        if (2 * mt + h < YG) {
          uint16_t *yr = L.ysrc[2 * mt + h];
          if (yr) {
            if (ok_y0) update8(yr + n0, lds128(L.ring.slot(it, 2 * KG + 2 * (2 * mt + h))), pc.scale, acc, 2 * h);
            if (ok_y1)
              update8(yr + n0 + 32, lds128(L.ring.slot(it, 2 * KG + 2 * (2 * mt + h) + 1)), pc.scale, acc,
                      2 * h + 1);
          }
        }
      }
    }
  }
  cp_async_wait<0>();
}

// rank-1 tiles of at most L tokens: fp32 FMAs over coalesced 512-byte warp loads.
template <int L>
struct ExpandVecLane {
  static constexpr int N = 1 + L;
  static constexpr int kStep = kWarps * 256;
  Ring<N> ring;
  const uint16_t *w;
  uint16_t *yr[L];
  int c0, c1, iters, len;
  __device__ __forceinline__ void init(const StreamProblem &pb, const Piece &pc, uint32_t ring_base) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    ring.base = ring_base;
    w = pb.B + (int64_t)pc.slot * pb.r_max * pb.n;
    len = pc.len;
#pragma unroll
    for (int l = 0; l < L; ++l) yr[l] = pb.y + (int64_t)pc.rows[l < pc.len ? l : 0] * pb.ldy;
    c0 = pc.lo * kExpandBlock + warp * 256 + lane * 8;
    c1 = min(pc.hi * kExpandBlock, pb.n);
    iters = (c1 - (pc.lo * kExpandBlock + warp * 256) + kStep - 1) / kStep;   // <= 0: nothing for this warp
  }
  __device__ __forceinline__ void issue(int it) const {
    if (it < iters) {
      const int col = c0 + it * kStep;
      const bool ok = col < c1;
      cp_async16(ring.slot(it, 0), ok ? w + col : w, ok);
#pragma unroll
      for (int l = 0; l < L; ++l) cp_async16(ring.slot(it, 1 + l), ok ? yr[l] + col : w, ok && l < len);
    }
    cp_async_commit();
  }
};

// An FMA-path piece needs no barrier of the CTA: every thread adds the shrink lanes' parts of the few v it
// needs by itself (the same few addresses for all threads) while the first blocks are on their way, so the
// warps of a CTA run through such pieces independently of one another.
template <int L>
__device__ __forceinline__ void expand_vec(const StreamParams &P, const StreamProblem &pb, const Piece &pc,
                                           uint32_t ring_base, int first, int count) {
  constexpr int kDepth = Ring<1 + L>::kDepth;
  ExpandVecLane<L> V;
  V.init(pb, pc, ring_base);
#pragma unroll 1
  for (int it = 0; it < kDepth - 1; ++it) V.issue(it);
  float sv[L];
  {
    const size_t slot_floats = (size_t)kTileRowsMax * pb.r_max;
    const float *part0 = pb.ws_part + (size_t)(pc.t + first) * slot_floats;
#pragma unroll
    for (int l = 0; l < L; ++l) sv[l] = 0.f;
    for (int k0 = 0; k0 < count; k0 += 4) {   // in lane order; the loads of four parts go out together
      float v[4][L];
#pragma unroll
      for (int k = 0; k < 4; ++k)
#pragma unroll
        for (int l = 0; l < L; ++l)
          v[k][l] = (k0 + k < count && l < pc.len) ? __ldcg(part0 + (size_t)(k0 + k) * slot_floats + l) : 0.f;
#pragma unroll
      for (int k = 0; k < 4; ++k)
#pragma unroll
        for (int l = 0; l < L; ++l) sv[l] += v[k][l];
    }
#pragma unroll
    for (int l = 0; l < L; ++l) {
      // MoE: the pair's routing weight multiplies its v
      const float w = (P.pair_weight && l < pc.len) ? __ldg(P.pair_weight + pc.rows[l]) : 1.f;
      sv[l] = pc.scale * (w * sv[l]);
    }
  }
#pragma unroll 1
  for (int it = 0; it < V.iters; ++it) {
    V.issue(it + kDepth - 1);
    cp_async_wait<kDepth - 1>();
    const int col = V.c0 + it * ExpandVecLane<L>::kStep;
    if (col < V.c1) {
      float wf[8];
      unpack8(lds128(V.ring.slot(it, 0)), wf);
#pragma unroll
      for (int l = 0; l < L; ++l)
        if (l < pc.len) {
          float yf[8];
          unpack8(lds128(V.ring.slot(it, 1 + l)), yf);
#pragma unroll
          for (int e = 0; e < 8; ++e) yf[e] = fmaf(sv[l], wf[e], yf[e]);
          *reinterpret_cast<uint4 *>(V.yr[l] + col) = pack8(yf);
        }
    }
  }
  cp_async_wait<0>();
}

// The shrink lanes whose share met the columns of problem p in the tile: they
// are consecutive lanes, found from the area arithmetic of the shrink kernel
// alone.  Eight threads share one (tile, problem): thread k looks at the
// candidate lanes c_a + k, c_a + k + 8, ... (all its table reads go out
// together), and the eight combine their findings with shuffles.  All threads
// of the CTA call this together; item = the (tile, problem) of this group of
// eight threads, valid = whether there is one.
__device__ __forceinline__ void shrink_parts(const StreamParams &P, const Area &sa, const TileDesc &d, int p,
                                             bool valid, int &first, int &count) {
  const int k = threadIdx.x & 7;
  const StreamProblem &pb = P.prob[valid ? p : 0];
  const int w_t = tile_rows<false>(d.rank, d.len);
  const int blocks = (pb.d + kShrinkBlock - 1) / kShrinkBlock;
  const int span = w_t * sa.CB;   // the tile's extent in area units
  // Table lanes that can meet the columns of THIS problem inside the tile: the problem covers the
  // area positions [pos_lo, pos_hi) and table lane j starts at about j W CB / G (one lane of margin
  // on either side; the exact test below decides).  A tile of a call with many projections can
  // meet far more lanes than one problem of it does, so the tile's own bounds are not enough.
  const int64_t wcb = sa.W * sa.CB;
  const int64_t pos_lo = (int64_t)d.rows_shrink * sa.CB + (int64_t)pb.cb0_shrink * w_t;
  const int64_t pos_hi = pos_lo + (int64_t)blocks * w_t;
  const int j_lo = max(d.lane_lo, (int)(pos_lo * sa.G / wcb) - 1);
  const int j_hi = min(d.lane_hi, (int)((pos_hi * sa.G + wcb - 1) / wcb) + 1);
  // active lanes c with table index in [j_lo, j_hi]: index(c) = c G / active
  const int c_a = (int)(((unsigned)(j_lo + 1) * (unsigned)sa.active - 1u) / (unsigned)sa.G);
  const int c_b = (int)(((unsigned)(j_hi + 1) * (unsigned)sa.active - 1u) / (unsigned)sa.G);
  unsigned long long mask = 0;   // bit i: lane c_a + i holds a part (at most kMaxParts + margin candidates)
  if (valid && !d.dense) {
    for (int i = k; c_a + i <= c_b && i < 64; i += 8) {
      const int c2 = c_a + i;
      const int64_t p0 = lane_offset(sa, sa.table[lane_index(sa, c2)], d.rows_shrink);
      const int64_t p1 = lane_offset(sa, sa.table[lane_index(sa, c2 + 1)], d.rows_shrink);
      if (p0 < span && p1 > 0) {
        const int va = p0 <= 0 ? 0 : (int)p0 / w_t;
        const int vb = p1 >= span ? sa.CB : (int)p1 / w_t;
        if (max(va, pb.cb0_shrink) < min(vb, pb.cb0_shrink + blocks)) mask |= 1ull << i;
      }
    }
  }
#pragma unroll
  for (int o = 1; o < 8; o <<= 1) mask |= __shfl_xor_sync(0xffffffffu, mask, o);
  first = mask ? c_a + __ffsll((long long)mask) - 1 : 0;
  count = __popcll(mask);
  if (valid && d.dense) {   // the tensor-core shrink leaves the complete v of the tile in the slot dense_slot0 + tile
    first = P.dense_slot0;
    count = 1;
  }
}

// Step 2a (all threads): vsum[i] = weight(row of i) * sum, in lane order, of the shrink
// lanes' parts of element i of the [len][rank] result.  Consecutive threads take
// consecutive elements, and the loads of four elements times four parts go out together.
__device__ __forceinline__ void sum_parts(const StreamParams &P, const StreamProblem &pb, const Piece &pc,
                                          int first, int count, float *vsum) {
  const size_t slot_floats = (size_t)kTileRowsMax * pb.r_max;
  const float *part0 = pb.ws_part + (size_t)(pc.t + first) * slot_floats;
  const int nel = pc.len * pc.r;
  for (int i0 = threadIdx.x; i0 < nel; i0 += 4 * kThreads) {
    float s[4] = {0.f, 0.f, 0.f, 0.f};
    for (int k0 = 0; k0 < count; k0 += 4) {
      float v[4][4];
#pragma unroll
      for (int k = 0; k < 4; ++k)
#pragma unroll
        for (int e = 0; e < 4; ++e)
          v[k][e] = (k0 + k < count && i0 + e * kThreads < nel)
                        ? __ldcg(part0 + (size_t)(k0 + k) * slot_floats + i0 + e * kThreads)
                        : 0.f;
#pragma unroll
      for (int k = 0; k < 4; ++k)
#pragma unroll
        for (int e = 0; e < 4; ++e) s[e] += v[k][e];
    }
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const int i = i0 + e * kThreads;
      if (i < nel) {
        // MoE: the pair's routing weight multiplies its row of v
        const float w = P.pair_weight ? __ldg(P.pair_weight + pc.rows[i / pc.r]) : 1.f;
        vsum[i] = w * s[e];
      }
    }
  }
}

__device__ __forceinline__ void expand_piece(const StreamParams &P, SmemExpand &S, uint32_t ring_base,
                                             const Piece &pc) {
  const StreamProblem &pb = P.prob[pc.p];
  const int tid = threadIdx.x;
  const bool vec = pc.r == 1 && pc.len <= 8;
  const int first = S.sh.part_first[pc.ti * kMaxProblems + pc.p];
  const int count = S.sh.part_count[pc.ti * kMaxProblems + pc.p];
  // row groups as the tensor-core body is instantiated: 1, 2 or 4 groups of 8 tokens; 2, 4 or 8 of 8 ranks
  // (a single group of ranks would run the same MMAs as two; fewer bodies keep the kernel's code small)
  const int yg = pc.len <= 8 ? 1 : (pc.len <= 16 ? 2 : 4);
  const int kg = pc.r <= 16 ? 2 : (pc.r <= 32 ? 4 : 8);
  const int MT = (yg + 1) >> 1, KS = (kg + 1) >> 1;
  if (vec) {
    if (pc.len == 1) expand_vec<1>(P, pb, pc, ring_base, first, count);
    else if (pc.len == 2) expand_vec<2>(P, pb, pc, ring_base, first, count);
    else if (pc.len <= 4) expand_vec<4>(P, pb, pc, ring_base, first, count);
    else expand_vec<8>(P, pb, pc, ring_base, first, count);
    return;
  }
  // step 1
  {
#define MINT_EXPAND_CASE(YG)                                     \
  if (kg == 2) expand_mma_fill<YG, 2>(pb, pc, ring_base);        \
  else if (kg == 4) expand_mma_fill<YG, 4>(pb, pc, ring_base);   \
  else expand_mma_fill<YG, 8>(pb, pc, ring_base)
    if (yg == 1) { MINT_EXPAND_CASE(1); }
    else if (yg == 2) { MINT_EXPAND_CASE(2); }
    else { MINT_EXPAND_CASE(4); }
#undef MINT_EXPAND_CASE
  }
  // step 2
  __syncthreads();   // the previous piece no longer reads v
  sum_parts(P, pb, pc, first, count, S.vsum);
  __syncthreads();
  {
    // one thread per (m-tile, k-step, lane): four (head, remainder) register pairs
    for (int i = tid; i < MT * KS * 32; i += kThreads) {
      const int ln = i & 31, ks = (i >> 5) % KS, mt = (i >> 5) / KS;
      const int g = ln >> 2, t = ln & 3;
      uint32_t hi[4], lo[4];
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const int row = mt * 16 + g + (q & 1) * 8, k = ks * 16 + 2 * t + (q >> 1) * 8;
        const float a = (row < pc.len && k < pc.r) ? S.vsum[row * pc.r + k] : 0.f;
        const float b = (row < pc.len && k + 1 < pc.r) ? S.vsum[row * pc.r + k + 1] : 0.f;
        split_pair(a, b, hi[q], lo[q]);
      }
      S.vfrag[((mt * 4 + ks) * 2 + 0) * 32 + ln] = make_uint4(hi[0], hi[1], hi[2], hi[3]);
      S.vfrag[((mt * 4 + ks) * 2 + 1) * 32 + ln] = make_uint4(lo[0], lo[1], lo[2], lo[3]);
    }
    __syncthreads();
  }
  // step 3
  {
#define MINT_EXPAND_CASE(YG)                                        \
  if (kg == 2) expand_mma<YG, 2>(pb, pc, ring_base, S);             \
  else if (kg == 4) expand_mma<YG, 4>(pb, pc, ring_base, S);        \
  else expand_mma<YG, 8>(pb, pc, ring_base, S)
    if (yg == 1) { MINT_EXPAND_CASE(1); }
    else if (yg == 2) { MINT_EXPAND_CASE(2); }
    else { MINT_EXPAND_CASE(4); }
#undef MINT_EXPAND_CASE
  }
}

__global__ void __launch_bounds__(kThreads, kCtasPerSm) expand_stream_kernel(const __grid_constant__ StreamParams P) {
  extern __shared__ __align__(128) uint8_t dyn_smem[];   // the four warps' rings
  __shared__ SmemExpand S;
  pdl_launch_dependents();
  Area area;
  CtaRange R;
  // The plan, the slot table and B were complete before the shrink kernel of
  // this call started, so they may be read before the dependency wait; y and v
  // may not.  Errors of the plan were already reported by the shrink kernel.
  if (!prologue<true>(P, S.sh, area, R, false)) {
    pdl_wait();
    return;
  }
  const Area shrink_area = make_area<false>(P);
  const uint32_t ring_base =
      smem_addr(dyn_smem) + (uint32_t)((threadIdx.x >> 5) * kRingBytes + (threadIdx.x & 31) * 16);
  bool waited = false;
  for (int tb = R.t0; tb < R.t_end; tb += kBatchTiles) {
    const int ntile = min(kBatchTiles, R.t_end - tb);
    // descriptors first; then the row indices and the lane-table entries are requested together
    __syncthreads();   // every warp is done with the previous batch
    {
      const int4 *src = reinterpret_cast<const int4 *>(P.pv.tile_desc + tb);
      int4 *dst = reinterpret_cast<int4 *>(S.sh.desc);
      for (int i = threadIdx.x; i < ntile * (int)(sizeof(TileDesc) / 16); i += kThreads) dst[i] = src[i];
    }
    __syncthreads();
    const int off0 = S.sh.desc[0].off;
    const int nitems = S.sh.desc[ntile - 1].off + S.sh.desc[ntile - 1].len - off0;
    int row_of[kBatchItems / kThreads];
#pragma unroll
    for (int u = 0; u < kBatchItems / kThreads; ++u) {
      const int i = threadIdx.x + u * kThreads;
      row_of[u] = i < nitems ? P.pv.perm[off0 + i] : 0;
    }
    // which shrink lanes hold the parts of v of every (tile, projection) of the batch
    for (int i0 = 0; i0 < ntile * P.nprob; i0 += kThreads / 8) {
      const int i = i0 + (int)(threadIdx.x >> 3);
      const bool valid = i < ntile * P.nprob;
      const int ti = valid ? i / P.nprob : 0, p = valid ? i - ti * P.nprob : 0;
      int first, count;
      shrink_parts(P, shrink_area, S.sh.desc[ti], p, valid, first, count);
      if (valid && (threadIdx.x & 7) == 0) {
        S.sh.part_first[ti * kMaxProblems + p] = first;
        S.sh.part_count[ti * kMaxProblems + p] = (int16_t)count;
      }
    }
#pragma unroll
    for (int u = 0; u < kBatchItems / kThreads; ++u) {
      const int i = threadIdx.x + u * kThreads;
      if (i < nitems) S.sh.rows[i] = row_of[u];
    }
    if (!waited) {
      // while the shrink kernel still runs: pull this lane's B rows into L2
      bool first_piece = true;   // only the piece the lane starts with
      walk_batch<true>(P, area, R, S.sh, tb, ntile, [&](const Piece &pc) {
        if (first_piece) prefetch_piece<true>(P.prob[pc.p], pc, true, false);
        first_piece = false;
      });
      pdl_wait();   // the shrink kernel has completed: v is final, y belongs to this kernel
      waited = true;
    }
    __syncthreads();
    walk_batch<true>(P, area, R, S.sh, tb, ntile, [&](const Piece &pc) { expand_piece(P, S, ring_base, pc); });
  }
}

// ---- host side -----------------------------------------------------------------
// Slots of 32 x r_max floats: tile + lane for the streamed parts; with dense segments (batches of at
// least MINT_DENSE_MIN_BATCH tokens) MINT_DENSE_SPLIT_MAX more per tile for the parts of the tensor-core shrink.
size_t workspace_bytes(int64_t tiles, int32_t r_max, bool dense) {
  const int64_t slots = tiles + MINT_MAX_LANES + (dense ? (int64_t)MINT_DENSE_SPLIT_MAX * tiles : 0);
  return (size_t)slots * kTileRowsMax * r_max * sizeof(float) + 256;
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

static int32_t stream_kernel_attributes() {
  static bool attrs_set = false;
  if (attrs_set) return MINT_OK;
  int32_t st;
  st = mint_check_cuda(cudaFuncSetAttribute(shrink_stream_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                            (int)kRingsBytes), "shrink_stream shared memory");
  if (st) return st;
  st = mint_check_cuda(cudaFuncSetAttribute(shrink_stream_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                            (int)kRingsBytes), "shrink_stream (packed) shared memory");
  if (st) return st;
  st = mint_check_cuda(cudaFuncSetAttribute(expand_stream_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                            (int)kRingsBytes), "expand_stream shared memory");
  if (st) return st;
  attrs_set = true;
  return MINT_OK;
}

// MoE expert LoRA apply on the streamed kernels: the plan's items are the
// (token, k) pairs grouped by (expert, slot); the weight block of a tile is
// (slot, expert); the shrink reads row x_row[p] of x, the expand updates row p of y.
// Kernel parameters of nprob MoE problems that share the plan, the row map and the pair weights
// (share_x: consecutive problems that read one x through pools of one shape are shrunk together).
static StreamParams moe_stream_params(const MoEArgs *args, int nprob, const TableDev &tab, const void *plan_dev,
                                      void *const *workspaces, int32_t lanes, bool share_x) {
  const MoEArgs &a0 = args[0];
  const int64_t pairs = (int64_t)a0.T * a0.K;
  const int64_t key_space = (int64_t)tab.num_slots * a0.num_experts;
  const int64_t tiles = mint_tile_upper_bound(1, pairs, key_space);
  StreamParams P = {};
  int cb_s = 0, cb_e = 0, cb_widest = 0;
  for (int i = 0; i < nprob; ++i) {
    const MoEArgs &a = args[i];
    StreamProblem &pb = P.prob[i];
    pb.A = a.A; pb.B = a.B; pb.x = a.x; pb.y = a.y;
    pb.ldx = a.ldx; pb.ldy = a.ldy;
    pb.d = a.d; pb.n = a.n; pb.r_max = a.r_max;
    pb.ws_part = static_cast<float *>(workspaces[i]);
    cb_e += kExpandPieceBlocks;
    pb.cb0_expand = cb_e;
    cb_e += (a.n + kExpandBlock - 1) / kExpandBlock;
    // Two consecutive projections that read the same x through pools of the same shape and at most 16
    // ranks (gate and up) are shrunk in one pass over x: the second takes no columns of the shrink's
    // area and finds its parts where the first one's are.
    const bool follows = i > 0 && P.prob[i - 1].dual == 1;
    if (follows) {
      pb.dual = 2;
      pb.cb0_shrink = P.prob[i - 1].cb0_shrink;
      continue;
    }
    cb_s += kShrinkPieceBlocks;
    pb.cb0_shrink = cb_s;
    cb_s += (a.d + kShrinkBlock - 1) / kShrinkBlock;
    cb_widest = std::max(cb_widest, kShrinkPieceBlocks + (a.d + kShrinkBlock - 1) / kShrinkBlock);
    if (i + 1 < nprob) {
      const MoEArgs &b = args[i + 1];
      if (share_x && b.x == a.x && b.ldx == a.ldx && b.d == a.d && b.r_max == a.r_max && a.r_max <= 16) pb.dual = 1;
    }
  }
  P.nprob = nprob;
  P.T = a0.T;
  P.K = a0.K;
  P.num_experts = a0.num_experts;
  P.weights_per_slot = a0.num_experts;
  P.x_row = a0.x_row;
  P.pair_weight = a0.pair_weight;
  P.x_rows = a0.x_rows;
  P.lanes = lanes;
  P.cb_shrink = cb_s;
  P.cb_expand = cb_e;
  P.cb_shrink_widest = cb_widest;
  P.dense_slot0 = (int32_t)(tiles + MINT_MAX_LANES);
  P.status = a0.status;
  P.tab = tab;
  P.pv = mint_plan_view(plan_dev, pairs, key_space);
  return P;
}

int32_t mint_launch_stream_moe(const MoEArgs *args, int nprob, const TableDev &tab, const void *plan_dev,
                               void *const *workspaces, cudaStream_t s) {
  if (nprob < 1 || nprob > kMaxProblems)
    return mint_fail(MINT_ERR_INVALID_ARG, "grouped MoE apply: 1..%d problems", kMaxProblems);
  int32_t lanes = 0;
  int32_t st = mint_device_lanes(&lanes);
  if (st) return st;
  if ((st = stream_kernel_attributes())) return st;
  if (mint_tile_upper_bound(1, (int64_t)args[0].T * args[0].K, (int64_t)tab.num_slots * args[0].num_experts) == 0)
    return MINT_OK;
  const StreamParams P = moe_stream_params(args, nprob, tab, plan_dev, workspaces, lanes, true);

  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)lanes);
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = kRingsBytes;
  cfg.stream = s;
  cfg.attrs = attr;
  // the first apply after a plan or a bind waits for that kernel in full: it reads the plan at once
  cfg.numAttrs = mint_take_tables_changed() ? 0 : 1;
  st = mint_check_cuda(cudaLaunchKernelEx(&cfg, shrink_stream_kernel<true>, P), "shrink_stream (packed) launch");
  if (st) return st;
  cfg.numAttrs = 1;
  return mint_check_cuda(cudaLaunchKernelEx(&cfg, expand_stream_kernel, P), "expand_stream launch");
}

size_t mint_stream_workspace_bytes(int32_t T, int32_t num_slots, int32_t r_max) {
  return workspace_bytes(mint_tile_upper_bound(1, T, num_slots), r_max, T >= MINT_DENSE_MIN_BATCH);
}

// ---- v in token order from the streamed shrink ----------------------------------------
// The backward needs x . A^T (and dy . B^T) of every token as a tensor of its own.  The streamed
// shrink leaves a tile's v as parts, one per lane that met the tile; this kernel adds them, in lane
// order as the expand would, and writes row l of a tile to row perm[off + l] of v[T][r_max]
// (ranks below the slot's rank only).  One CTA per (tile, problem).
struct GatherV {
  float *v[kMaxProblems];
};

__global__ void __launch_bounds__(kThreads) gather_v_kernel(const __grid_constant__ StreamParams P, const GatherV out) {
  __shared__ int32_t part_first, part_count;
  pdl_launch_dependents();
  // (before the wait: only the plan, complete before the shrink kernel of this call started)
  const int t = blockIdx.x, p = blockIdx.y;
  if (!plan_ok(P.pv.header, P.T, P.K, P.tab.num_slots, P.num_experts, P.tab.gen_lo, P.tab.gen_hi, nullptr) ||
      P.pv.header[PH_LANES] != P.lanes || t >= P.pv.header[PH_NCHUNK1]) {
    pdl_wait();
    return;
  }
  const TileDesc d = P.pv.tile_desc[t];
  if (!d.dense) {
    const Area shrink_area = make_area<false>(P);
    int first, count;
    shrink_parts(P, shrink_area, d, p, threadIdx.x < 8, first, count);   // (eight threads look per item)
    if (threadIdx.x == 0) {
      part_first = first;
      part_count = count;
    }
  }
  pdl_wait();   // the shrink kernels have completed: the parts are final
  __syncthreads();
  const int nel = d.len * d.rank;
  const StreamProblem &pb = P.prob[p];
  const size_t slot_floats = (size_t)kTileRowsMax * pb.r_max;
  // dense segments: the tensor-core shrink left one part per share of d in slots of their own
  const int count = d.dense ? mint_dense_splits(pb.d) : part_count;
  const size_t stride = d.dense ? (size_t)(P.dense_slot0 - MINT_MAX_LANES) * slot_floats : slot_floats;
  const float *part0 = pb.ws_part + (size_t)(t + (d.dense ? P.dense_slot0 : part_first)) * slot_floats;
  for (int i = threadIdx.x; i < nel; i += kThreads) {
    float s = 0.f;
    for (int k0 = 0; k0 < count; k0 += 4) {
      float part[4];
#pragma unroll
      for (int k = 0; k < 4; ++k) part[k] = k0 + k < count ? __ldcg(part0 + (size_t)(k0 + k) * stride + i) : 0.f;
#pragma unroll
      for (int k = 0; k < 4; ++k) s += part[k];
    }
    const int l = i / d.rank, j = i - l * d.rank;
    const int item = P.pv.perm[d.off + l];
    // (MoE: the pair's routing weight multiplies its row, as it does in the forward expand)
    out.v[p][(size_t)item * pb.r_max + j] = P.pair_weight ? __ldg(P.pair_weight + item) * s : s;
  }
}

// The streamed fused apply of up to eight problems.  phases: bit 0 = the shrink (and the tensor-core
// shrink of dense segments), bit 1 = the expand (and theirs).  v_out, when given, receives x . A^T of
// every problem in token order ([T][r_max] fp32) right after the shrink.  A call with the expand alone
// relies on the parts an earlier call with the same problems, plan and workspaces left behind.
int32_t mint_launch_stream_phases(const DenseArgs *args, int nprob, const TableDev &tab, const void *plan_dev,
                                  void *const *workspaces, cudaStream_t s, int phases, float *const *v_out) {
  if (nprob < 1 || nprob > kMaxProblems)
    return mint_fail(MINT_ERR_INVALID_ARG, "grouped apply: 1..%d problems", kMaxProblems);
  int32_t lanes = 0;
  int32_t st = mint_device_lanes(&lanes);
  if (st) return st;
  if ((st = stream_kernel_attributes())) return st;
  const int32_t T = args[0].T;
  const int64_t tiles = mint_tile_upper_bound(1, T, tab.num_slots);
  if (tiles == 0) return MINT_OK;
  StreamParams P = {};
  GatherV out = {};
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
    if (v_out) out.v[i] = v_out[i];
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
  cfg.gridDim = dim3((unsigned)lanes);
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = kRingsBytes;
  cfg.stream = s;
  cfg.attrs = attr;
  const bool dense = T >= MINT_DENSE_MIN_BATCH;   // the plan may have given dense segments to the tensor-core kernels
  if (phases & 1) {
    // the first apply after a plan or a bind waits for that kernel in full: it reads the plan at once
    cfg.numAttrs = mint_take_tables_changed() ? 0 : 1;
    st = mint_check_cuda(cudaLaunchKernelEx(&cfg, shrink_stream_kernel<false>, P), "shrink_stream launch");
    if (st) return st;
    if (dense) {
      st = mint_launch_dense_shrink(args, nprob, tab, plan_dev, workspaces, lanes, P.dense_slot0, (int32_t)tiles, s);
      if (st) return st;
    }
    if (v_out) {
      cudaLaunchConfig_t gcfg = cfg;   // (it follows a shrink kernel of this call: programmatic launch)
      gcfg.gridDim = dim3((unsigned)tiles, (unsigned)nprob);
      gcfg.dynamicSmemBytes = 0;
      gcfg.numAttrs = 1;
      if ((st = mint_check_cuda(cudaLaunchKernelEx(&gcfg, gather_v_kernel, P, out), "gather_v launch"))) return st;
    }
  }
  if (!(phases & 2)) return MINT_OK;
  cfg.numAttrs = mint_take_tables_changed() ? 0 : 1;
  st = mint_check_cuda(cudaLaunchKernelEx(&cfg, expand_stream_kernel, P), "expand_stream launch");
  if (st || !dense) return st;
  return mint_launch_dense_expand(args, nprob, tab, plan_dev, workspaces, lanes, P.dense_slot0, (int32_t)tiles, s);
}

int32_t mint_launch_stream(const DenseArgs *args, int nprob, const TableDev &tab, const void *plan_dev,
                           void *const *workspaces, cudaStream_t s) {
  return mint_launch_stream_phases(args, nprob, tab, plan_dev, workspaces, s, 3, nullptr);
}

// x . A^T of every problem into v_out[i] ([T][r_max] fp32, token order; rows of tokens without an adapter
// and ranks at or above the slot's rank are not written).  Workspaces as for mint_launch_stream.
int32_t mint_launch_stream_shrink_v(const DenseArgs *args, int nprob, const TableDev &tab, const void *plan_dev,
                                    void *const *workspaces, float *const *v_out, cudaStream_t s) {
  return mint_launch_stream_phases(args, nprob, tab, plan_dev, workspaces, s, 1, v_out);
}

// The same for the (token, k) pairs of a MoE plan: v_out[i] ([T*K][r_max] fp32, pair order) = the pair's
// routing weight times x[x_row[p]] . A[slot][expert] (packed pools, A as [d][r_max]) or, with rank_major,
// times x[p] . A[slot][expert]^T for tensors stored as [slot][expert][r_max][d] -- which is how the backward
// gets dy . B^T out of a pool's B.  Workspaces as for mint_launch_stream_moe.
int32_t mint_launch_stream_moe_shrink_v(const MoEArgs *args, int nprob, bool rank_major, const TableDev &tab,
                                        const void *plan_dev, void *const *workspaces, float *const *v_out,
                                        cudaStream_t s) {
  if (nprob < 1 || nprob > kMaxProblems)
    return mint_fail(MINT_ERR_INVALID_ARG, "MoE shrink: 1..%d problems", kMaxProblems);
  int32_t lanes = 0;
  int32_t st = mint_device_lanes(&lanes);
  if (st) return st;
  if ((st = stream_kernel_attributes())) return st;
  const int64_t tiles =
      mint_tile_upper_bound(1, (int64_t)args[0].T * args[0].K, (int64_t)tab.num_slots * args[0].num_experts);
  if (tiles == 0) return MINT_OK;
  const StreamParams P = moe_stream_params(args, nprob, tab, plan_dev, workspaces, lanes, false);
  GatherV out = {};
  for (int i = 0; i < nprob; ++i) out.v[i] = v_out[i];
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)lanes);
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = kRingsBytes;
  cfg.stream = s;
  cfg.attrs = attr;
  cfg.numAttrs = mint_take_tables_changed() ? 0 : 1;
  if (rank_major)
    st = mint_check_cuda(cudaLaunchKernelEx(&cfg, shrink_stream_kernel<false>, P), "shrink_stream launch");
  else
    st = mint_check_cuda(cudaLaunchKernelEx(&cfg, shrink_stream_kernel<true>, P), "shrink_stream (packed) launch");
  if (st) return st;
  cfg.gridDim = dim3((unsigned)tiles, (unsigned)nprob);
  cfg.dynamicSmemBytes = 0;
  cfg.numAttrs = 1;
  return mint_check_cuda(cudaLaunchKernelEx(&cfg, gather_v_kernel, P, out), "gather_v launch");
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
