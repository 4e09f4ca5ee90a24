// Streamed LoRA apply for dense projections: the fused path of
// mint_lora_apply_fused and of its grouped form.
//
//   shrink_stream_kernel : v[tile] = X[tile rows, :] . A_slot           (d -> r)
//   expand_stream_kernel : Y[tile rows, :] += s_slot * v[tile] . B_slot  (r -> n)
//
// Both kernels are persistent: one CTA per SM ("lane"), and every lane moves the
// same number of bytes.  The work of a call is the area  rows x columns  where
// rows runs over the plan's tiles (a tile = at most 32 tokens of one segment,
// contributing rank + len rows to the shrink and rank + 2 len rows to the
// expand) and columns over the 16-element column blocks of all projections of
// the call, laid side by side.  Lane c takes the c-th equal share of that area,
// walked tile by tile: a share starts in the middle of one tile, covers whole
// tiles, and ends in the middle of another.  The plan tabulates the tile in
// which every lane starts (it does not depend on the widths), so a lane finds
// its work with two table reads.
//
// Inside a CTA a load warp streams the rows of its share through a ring of
// 16 KB shared-memory stages with bulk asynchronous copies (cp.async.bulk,
// one per row, completion counted in bytes on an mbarrier); four consumer
// warps do the arithmetic out of shared memory; in the expand a store warp
// writes the updated y rows back with bulk stores.  HBM latency is hidden by
// the bytes in flight in the ring, not by registers.  The arithmetic is the
// warp-level tensor-core MMA (m16n8k16, bf16 in, fp32 accumulate) with ldmatrix
// operand fetches; tiles that are both short and of very low rank (rank <= 4,
// at most 8 tokens) use plain fp32 FMAs, because padding them to an MMA tile
// would multiply the shared-memory reads.
//
// v travels from the shrink to the expand through a small L2-resident
// workspace.  A tile whose columns are shared by several lanes gets one partial
// sum per lane; the lane that completes the tile (a ticket counted in column
// blocks) adds the partials in lane order, so the result does not depend on
// scheduling.  The expand carries v as a bf16 head plus a bf16 remainder (two
// MMAs), about 16 significant bits of the fp32 shrink result.
//
// Launch overlap: both kernels allow their successor to become resident at once
// (griddepcontrol.launch_dependents first thing) and are launched with
// programmatic stream serialization.  Before its dependency wait a kernel reads
// only the plan, the slot table and pool weights, which no apply kernel writes;
// activations, y and v are touched only after the wait, and every CTA executes
// the wait before it exits so that completion stays transitive along the stream.
// The shrink CTA is small (4 stages) and the expand CTA large (7 stages) so that
// one of each fits on an SM: the expand of a call streams B while its shrink
// still runs, and the shrink of the next call is resident before this expand ends.
#include <algorithm>

#include "mint_device.cuh"

using namespace mint;

namespace {

constexpr int kConsumerWarps = 4;
constexpr int kConsumerThreads = kConsumerWarps * 32;
constexpr int kStageBytes = 16384;
constexpr int kShrinkStages = 4;
constexpr int kExpandStages = 7;
constexpr int kShrinkThreads = kConsumerThreads + 32;   // + load warp
constexpr int kExpandThreads = kConsumerThreads + 64;   // + load warp + store warp
constexpr int kTileRowsMax = 32;                        // plan tile list 1
constexpr int kStreamRankCap = 64;                      // larger ranks take the CUDA-core cluster kernel
constexpr int kBatchTiles = 32;                         // tile descriptors staged in shared memory at a time
constexpr int kBatchItems = kBatchTiles * kTileRowsMax;
constexpr int kGrainUnits = 512;                        // smallest lane share: 512 row-blocks of 32 B
constexpr int kMaxProblems = MINT_MAX_GROUP;
constexpr int kSlotFloats = kTileRowsMax * kStreamRankCap;  // upper bound of one v tile

struct StreamProblem {
  const uint16_t *A;   // [slot][r_max][d]
  const uint16_t *B;   // [slot][r_max][n]
  const uint16_t *x;
  uint16_t *y;
  int64_t ldx, ldy;
  int32_t d, n, r_max;
  int32_t cb0_shrink, cb0_expand;  // first virtual column block of this problem
  float *ws_v;         // [tiles_ub][32 * r_max]         complete shrink result of a tile, [len][rank] packed
  float *ws_part;      // [tiles_ub + lanes][32 * r_max] partial sums of tiles shared by several lanes
  int32_t *ws_ticket;  // [tiles_ub], zero between launches
};

struct StreamParams {
  StreamProblem prob[kMaxProblems];
  int32_t nprob;
  int32_t T;
  int32_t lanes;                      // grid size = the plan's lane count
  int32_t cb_shrink, cb_expand;       // virtual column blocks of the whole call
  int32_t *status;
  TableDev tab;
  PlanView pv;
};

// ---- PTX wrappers ------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_addr(const void *p) {
  return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mbar_init(uint64_t *bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t *bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr(bar)), "r"(bytes)
               : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t *bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_addr(bar)) : "memory");
}
__device__ __forceinline__ uint64_t global_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}
// Bounded wait for the phase with the given parity.  Gives up (false) after two
// seconds, or as soon as another role of the CTA has raised the abort flag.
__device__ __forceinline__ bool mbar_wait(uint64_t *bar, uint32_t parity, volatile int *abort_flag) {
  const uint32_t a = smem_addr(bar);
  uint64_t t0 = 0;
  for (uint32_t it = 0;; ++it) {
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done)
        : "r"(a), "r"(parity)
        : "memory");
    if (done) return true;
    if ((it & 63u) == 63u) {
      if (*abort_flag) return false;
      const uint64_t now = global_ns();
      if (t0 == 0) t0 = now;
      else if (now - t0 > 2000000000ull) return false;
    }
  }
}
// global -> shared bulk copy; completion is counted in bytes on the mbarrier
__device__ __forceinline__ void bulk_load(void *dst_smem, const void *src, uint32_t bytes, uint64_t *bar) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
          smem_addr(dst_smem)),
      "l"(src), "r"(bytes), "r"(smem_addr(bar))
      : "memory");
}
// shared -> global bulk copy, tracked by the issuing thread's bulk group
__device__ __forceinline__ void bulk_store(void *dst, const void *src_smem, uint32_t bytes) {
  asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(dst),
               "r"(smem_addr(src_smem)), "r"(bytes)
               : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_read_all() {
  asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
}
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void fence_mbar_init() {
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void pdl_launch_dependents() {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
// barrier among the consumer warps only
__device__ __forceinline__ void consumer_sync() { asm volatile("bar.sync 1, %0;" ::"n"(kConsumerThreads) : "memory"); }

__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(addr));
}
// D(16x8, f32) += A(16x16, bf16, row) * B(16x8, bf16, col)
__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
      "{%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

__host__ __device__ inline int round_up(int v, int m) { return (v + m - 1) / m * m; }

// ---- the share of one lane -------------------------------------------------------
// Position P in the rows x column-blocks area of a kernel, counted tile by tile:
// tile t covers [rows(t) * CB, rows(t + 1) * CB), and inside it column block
// kb = (P - rows(t) * CB) / w_t  where w_t is the tile's row count.
struct LaneCut {
  int tile;   // tile holding the cut (number of tiles for the end of the area)
  int cb;     // virtual column block inside that tile where the cut falls
};

template <bool kExpand>
__device__ __forceinline__ int tile_rows(const TileDesc &d) {
  return kExpand ? d.rank + 2 * d.len : d.rank + d.len;
}

template <bool kExpand>
__device__ __forceinline__ LaneCut lane_cut(const StreamParams &P, int c, int active) {
  const int G = P.lanes;
  const int64_t j = (int64_t)c * G / active;
  const int32_t *table = kExpand ? P.pv.lane_expand : P.pv.lane_shrink;
  LaneCut cut;
  cut.tile = table[j];
  cut.cb = 0;
  if (j >= G) return cut;
  const int CB = kExpand ? P.cb_expand : P.cb_shrink;
  const int64_t W = P.pv.header[kExpand ? PH_ROWS_EXPAND : PH_ROWS_SHRINK];
  const TileDesc d = P.pv.tile_desc[cut.tile];
  const int64_t pos = j * W * CB / G;
  const int64_t base = (int64_t)(kExpand ? d.rows_expand : d.rows_shrink) * CB;
  cut.cb = (int)((pos - base) / tile_rows<kExpand>(d));
  return cut;
}

template <bool kExpand>
__device__ __forceinline__ int active_lanes(const StreamParams &P) {
  const int64_t W = P.pv.header[kExpand ? PH_ROWS_EXPAND : PH_ROWS_SHRINK];
  const int64_t units = W * (kExpand ? P.cb_expand : P.cb_shrink);
  int64_t g = units / kGrainUnits;
  if (g < 1) g = 1;
  if (g > P.lanes) g = P.lanes;
  return (int)g;
}

// ---- stage geometry ----------------------------------------------------------------
struct Geo {
  bool mma;     // tensor-core path (else fp32 FMA path)
  int w_rows;   // rows reserved for weight rows in a stage
  int pitch;    // bytes between rows of a stage
  int cw;       // chunk width in elements (multiple of 16)
};

template <bool kExpand>
__device__ __forceinline__ Geo geometry(int r, int len) {
  Geo g;
  g.mma = !(r <= 4 && len <= 8);
  int rows;
  if (!g.mma) {
    g.w_rows = r;
    rows = r + len;
  } else if (kExpand) {
    g.w_rows = round_up(r, 16);          // k of the MMA; rows beyond the rank are masked in registers
    rows = g.w_rows + len;
  } else {
    g.w_rows = round_up(r, 16);          // n of the MMA, fetched as pairs of 8-row tiles
    rows = g.w_rows + round_up(len, 16);
  }
  int cw = ((kStageBytes / rows) - 16) / 2;
  g.cw = cw / 16 * 16;                    // >= 64 for rows <= 96
  g.pitch = g.cw * 2 + 16;                // odd multiple of 16 B: conflict-free ldmatrix
  return g;
}

// ---- what every role of a CTA shares -----------------------------------------------
struct CtaShared {
  TileDesc desc[kBatchTiles];
  int32_t rows[kBatchItems];
  int32_t lane_tile[MINT_MAX_LANES + 1];
  int32_t lane_cb[MINT_MAX_LANES + 1];
  int32_t contrib[MINT_MAX_LANES];   // lanes holding a partial of the tile being completed
  int32_t ncontrib;
  int32_t flag;        // consumer broadcast (ticket result)
  int32_t abort_flag;
};

struct CtaRange {
  int t0, cb0, t1, cb1;  // share = [(t0, cb0), (t1, cb1))
  int t_end;             // one past the last tile the share touches
  int CB;
  int nprob;
  int c, lanes;
};

struct Piece {
  int t;        // tile
  int p;        // problem
  int lo, hi;   // column blocks of the problem [lo, hi)
  int col0, col1;
  int row0;     // index of the tile's first row in CtaShared::rows
  int r, len;
  float scale;
  int slot;
  Geo g;
};

// Walks the pieces and chunks of one batch of tiles in the one order every role
// follows.  V provides piece_begin / chunk / piece_end; returning false stops.
template <bool kExpand, class V>
__device__ __forceinline__ bool walk_batch(const StreamParams &P, const CtaRange &R, const CtaShared &sh, int tb,
                                           int ntile, V &v) {
  for (int ti = 0; ti < ntile; ++ti) {
    const int t = tb + ti;
    const int va = (t == R.t0) ? R.cb0 : 0;
    const int vb = (t == R.t1) ? R.cb1 : R.CB;
    if (va >= vb) continue;
    Piece pc;
    pc.t = t;
    pc.r = sh.desc[ti].rank;
    pc.len = sh.desc[ti].len;
    pc.scale = sh.desc[ti].scale;
    pc.slot = sh.desc[ti].slot;
    pc.row0 = sh.desc[ti].off - sh.desc[0].off;
    pc.g = geometry<kExpand>(pc.r, pc.len);
    for (int p = 0; p < R.nprob; ++p) {
      const StreamProblem &pb = P.prob[p];
      const int width = kExpand ? pb.n : pb.d;
      const int first = kExpand ? pb.cb0_expand : pb.cb0_shrink;
      const int count = (width + 15) >> 4;
      const int lo = max(va, first) - first, hi = min(vb, first + count) - first;
      if (lo >= hi) continue;
      pc.p = p;
      pc.lo = lo;
      pc.hi = hi;
      pc.col0 = lo * 16;
      pc.col1 = min(hi * 16, width);
      if (!v.piece_begin(pc)) return false;
      for (int col = pc.col0; col < pc.col1; col += pc.g.cw)
        if (!v.chunk(pc, col, min(pc.g.cw, pc.col1 - col))) return false;
      if (!v.piece_end(pc)) return false;
    }
  }
  return true;
}

// Column blocks [lo, hi) of problem p that lane c2 covers in tile t (empty: lo >= hi).
template <bool kExpand>
__device__ __forceinline__ void lane_piece(const StreamParams &P, const CtaShared &sh, int CB, int c2, int t, int p,
                                           int &lo, int &hi) {
  const int ta = sh.lane_tile[c2], tb = sh.lane_tile[c2 + 1];
  int va = CB, vb = 0;
  if (t >= ta && t <= tb) {
    va = (t == ta) ? sh.lane_cb[c2] : 0;
    vb = (t == tb) ? sh.lane_cb[c2 + 1] : CB;
  }
  const StreamProblem &pb = P.prob[p];
  const int width = kExpand ? pb.n : pb.d;
  const int first = kExpand ? pb.cb0_expand : pb.cb0_shrink;
  const int count = (width + 15) >> 4;
  lo = max(va, first) - first;
  hi = min(vb, first + count) - first;
}

// ---- common prologue ------------------------------------------------------------------
// Validates the plan, tabulates the cuts of all lanes in shared memory and
// returns this CTA's share.  false: nothing to do (or the plan was refused).
template <bool kExpand>
__device__ __forceinline__ bool prologue(const StreamParams &P, CtaShared &sh, CtaRange &R, bool report_errors) {
  if (!plan_ok(P.pv.header, P.T, 1, P.tab.num_slots, 0, P.tab.gen_lo, P.tab.gen_hi,
               report_errors ? P.status : nullptr))
    return false;
  if (P.pv.header[PH_LANES] != P.lanes) {
    if (threadIdx.x == 0 && report_errors) report(P.status, MINT_ERR_SHAPE_MISMATCH, P.pv.header[PH_LANES]);
    return false;
  }
  const int ntiles = P.pv.header[PH_NCHUNK1];
  if (ntiles == 0) return false;
  const int lanes = active_lanes<kExpand>(P);
  for (int c = threadIdx.x; c <= lanes; c += blockDim.x) {
    const LaneCut cut = lane_cut<kExpand>(P, c, lanes);
    sh.lane_tile[c] = cut.tile;
    sh.lane_cb[c] = cut.cb;
  }
  if (threadIdx.x == 0) {
    sh.flag = 0;
    sh.abort_flag = 0;
  }
  __syncthreads();
  R.c = blockIdx.x;
  R.lanes = lanes;
  R.CB = kExpand ? P.cb_expand : P.cb_shrink;
  R.nprob = P.nprob;
  if (R.c >= lanes) return false;
  R.t0 = sh.lane_tile[R.c];
  R.cb0 = sh.lane_cb[R.c];
  R.t1 = sh.lane_tile[R.c + 1];
  R.cb1 = sh.lane_cb[R.c + 1];
  R.t_end = (R.cb1 > 0) ? R.t1 + 1 : R.t1;
  return R.t_end > R.t0;
}

// Stages the descriptors and the row indices of tiles [tb, tb + ntile) (all threads).
__device__ __forceinline__ void load_batch(const StreamParams &P, CtaShared &sh, int tb, int ntile) {
  __syncthreads();  // every role is done with the previous batch
  const int4 *src = reinterpret_cast<const int4 *>(P.pv.tile_desc + tb);
  int4 *dst = reinterpret_cast<int4 *>(sh.desc);
  for (int i = threadIdx.x; i < ntile * 2; i += blockDim.x) dst[i] = src[i];
  __syncthreads();
  const int off0 = sh.desc[0].off;
  const int nitems = sh.desc[ntile - 1].off + sh.desc[ntile - 1].len - off0;
  for (int i = threadIdx.x; i < nitems; i += blockDim.x) sh.rows[i] = P.pv.perm[off0 + i];
  __syncthreads();
}

// ================================================================================
// shrink
// ================================================================================
struct ShrinkLoader {
  const StreamParams &P;
  const CtaShared &sh;
  uint8_t *stages;
  uint64_t *full, *empty;
  volatile int *abort_flag;
  uint32_t q;

  __device__ __forceinline__ bool piece_begin(const Piece &) { return true; }
  __device__ __forceinline__ bool piece_end(const Piece &) { return true; }
  __device__ __forceinline__ bool chunk(const Piece &pc, int col, int width) {
    const int lane = threadIdx.x & 31;
    const uint32_t s = q % kShrinkStages;
    if (!mbar_wait(&empty[s], ((q / kShrinkStages) & 1u) ^ 1u, abort_flag)) return false;
    const StreamProblem &pb = P.prob[pc.p];
    uint8_t *stage = stages + (size_t)s * kStageBytes;
    const uint32_t row_bytes = (uint32_t)width * 2u;
    if (lane == 0) mbar_arrive_expect_tx(&full[s], row_bytes * (uint32_t)(pc.r + pc.len));
    __syncwarp();
    const uint16_t *A_slot = pb.A + (int64_t)pc.slot * pb.r_max * pb.d;
    for (int i = lane; i < pc.r + pc.len; i += 32) {
      const uint16_t *src;
      uint8_t *dst;
      if (i < pc.r) {
        src = A_slot + (int64_t)i * pb.d + col;
        dst = stage + (size_t)i * pc.g.pitch;
      } else {
        src = pb.x + (int64_t)sh.rows[pc.row0 + i - pc.r] * pb.ldx + col;
        dst = stage + (size_t)(pc.g.w_rows + i - pc.r) * pc.g.pitch;
      }
      bulk_load(dst, src, row_bytes, &full[s]);
    }
    ++q;
    return true;
  }
};

struct ShrinkConsumer {
  const StreamParams &P;
  CtaShared &sh;
  const CtaRange &R;
  uint8_t *stages;
  uint64_t *full, *empty;
  float *scratch;   // [4 warps][2 m-tiles][2 n-tiles][128] partial MMA tiles, or [4][32] FMA sums
  volatile int *abort_flag;
  uint32_t q;
  float acc[2][2][4];   // MMA path: [m-tile][n-tile of this warp's pair][fragment]
  float facc[8][4];     // FMA path: [token][rank]

  __device__ __forceinline__ bool piece_begin(const Piece &pc) {
    if (pc.g.mma) {
#pragma unroll
      for (int a = 0; a < 2; ++a)
#pragma unroll
        for (int b = 0; b < 2; ++b)
#pragma unroll
          for (int e = 0; e < 4; ++e) acc[a][b][e] = 0.f;
    } else {
#pragma unroll
      for (int l = 0; l < 8; ++l)
#pragma unroll
        for (int j = 0; j < 4; ++j) facc[l][j] = 0.f;
    }
    return true;
  }

  // How the four warps share the output tiles of the MMA path: n-tiles go in
  // pairs (16 ranks); with fewer than four pairs the warps also split k.
  __device__ __forceinline__ static void warp_role(int r, int warp, int &pair, int &kpart, int &ksplit) {
    const int pairs = (r + 15) >> 4;
    ksplit = pairs >= 3 ? 1 : (pairs == 2 ? 2 : 4);
    const int owners = kConsumerWarps / ksplit;
    pair = warp % owners;
    kpart = warp / owners;
  }

  template <int MT>
  __device__ __forceinline__ void mma_chunk(const Piece &pc, const uint8_t *stage, int width) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    int pair, kpart, ksplit;
    warp_role(pc.r, warp, pair, kpart, ksplit);
    if (pair * 16 >= pc.r) return;
    const bool second = pair * 16 + 8 < pc.r;
    const int ksteps = (width + 15) >> 4;
    const bool half_tail = (width & 15) != 0;
    const uint32_t w_base = smem_addr(stage);
    const uint32_t x_base = w_base + (uint32_t)(pc.g.w_rows * pc.g.pitch);
    const int m = lane >> 3;
    const uint32_t w_lane = w_base + (uint32_t)((pair * 16 + (m >> 1) * 8 + (lane & 7)) * pc.g.pitch + (m & 1) * 16);
    const uint32_t x_lane = x_base + (uint32_t)((lane & 15) * pc.g.pitch + (lane >> 4) * 16);
    for (int ks = kpart; ks < ksteps; ks += ksplit) {
      uint32_t b[4];
      ldmatrix_x4(b, w_lane + ks * 32);
      const bool tail = half_tail && ks == ksteps - 1;
      if (tail) b[1] = b[3] = 0u;   // columns beyond the width were never loaded
#pragma unroll
      for (int mt = 0; mt < MT; ++mt) {
        uint32_t xa[4];
        ldmatrix_x4(xa, x_lane + (uint32_t)(mt * 16 * pc.g.pitch) + ks * 32);
        if (tail) xa[2] = xa[3] = 0u;
        mma_bf16(acc[mt][0], xa, b[0], b[1]);
        if (second) mma_bf16(acc[mt][1], xa, b[2], b[3]);
      }
    }
  }

  __device__ __forceinline__ void fma_chunk(const Piece &pc, const uint8_t *stage, int width) {
    for (int v = threadIdx.x; v < (width >> 3); v += kConsumerThreads) {
      float af[4][8];
#pragma unroll
      for (int j = 0; j < 4; ++j)
        if (j < pc.r) unpack8(*reinterpret_cast<const uint4 *>(stage + (size_t)j * pc.g.pitch + v * 16), af[j]);
#pragma unroll
      for (int l = 0; l < 8; ++l) {
        if (l < pc.len) {
          float xf[8];
          unpack8(*reinterpret_cast<const uint4 *>(stage + (size_t)(pc.g.w_rows + l) * pc.g.pitch + v * 16), xf);
#pragma unroll
          for (int j = 0; j < 4; ++j)
            if (j < pc.r) {
#pragma unroll
              for (int e = 0; e < 8; ++e) facc[l][j] = fmaf(xf[e], af[j][e], facc[l][j]);
            }
        }
      }
    }
  }

  __device__ __forceinline__ bool chunk(const Piece &pc, int, int width) {
    const uint32_t s = q % kShrinkStages;
    if (!mbar_wait(&full[s], (q / kShrinkStages) & 1u, abort_flag)) return false;
    const uint8_t *stage = stages + (size_t)s * kStageBytes;
    if (!pc.g.mma) fma_chunk(pc, stage, width);
    else if (pc.len <= 16) mma_chunk<1>(pc, stage, width);
    else mma_chunk<2>(pc, stage, width);
    __syncwarp();
    if ((threadIdx.x & 31) == 0) mbar_arrive(&empty[s]);
    ++q;
    return true;
  }

  // The reduced [len][rank] result of this piece, element i = l * rank + j.
  __device__ __forceinline__ float gather(const Piece &pc, int i) const {
    const int l = i / pc.r, j = i - l * pc.r;
    if (!pc.g.mma) {
      float s = 0.f;
#pragma unroll
      for (int w = 0; w < kConsumerWarps; ++w) s += scratch[w * 32 + l * 4 + j];
      return s;
    }
    int pair, kpart, ksplit;
    warp_role(pc.r, 0, pair, kpart, ksplit);
    const int owners = kConsumerWarps / ksplit;
    const int mt = l >> 4, g = l & 15, nt = j >> 3, cc = j & 7;
    const int frag = ((g & 7) * 4 + (cc >> 1)) * 4 + (g >> 3) * 2 + (cc & 1);
    float s = 0.f;
    for (int k = 0; k < ksplit; ++k) {
      const int w = (nt >> 1) + k * owners;
      s += scratch[((w * 2 + mt) * 2 + (nt & 1)) * 128 + frag];
    }
    return s;
  }

  __device__ __forceinline__ bool piece_end(const Piece &pc) {
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    consumer_sync();   // the previous piece's readers are done with the scratch
    if (pc.g.mma) {
#pragma unroll
      for (int mt = 0; mt < 2; ++mt)
#pragma unroll
        for (int h = 0; h < 2; ++h)
          *reinterpret_cast<float4 *>(scratch + ((warp * 2 + mt) * 2 + h) * 128 + lane * 4) =
              make_float4(acc[mt][h][0], acc[mt][h][1], acc[mt][h][2], acc[mt][h][3]);
    } else {
#pragma unroll
      for (int l = 0; l < 8; ++l)
#pragma unroll
        for (int j = 0; j < 4; ++j)
          if (l < pc.len && j < pc.r) {
            const float s = warp_sum(facc[l][j]);
            if (lane == 0) scratch[warp * 32 + l * 4 + j] = s;
          }
    }
    consumer_sync();
    const StreamProblem &pb = P.prob[pc.p];
    const int cnt = pc.len * pc.r;
    const size_t slot_floats = (size_t)kTileRowsMax * pb.r_max;
    const int blocks = (pb.d + 15) >> 4;
    float *v_tile = pb.ws_v + (size_t)pc.t * slot_floats;
    if (pc.hi - pc.lo == blocks) {   // this lane covers the whole width: the result is final
      for (int i = tid; i < cnt; i += kConsumerThreads) v_tile[i] = gather(pc, i);
      return true;
    }
    float *part = pb.ws_part + (size_t)(pc.t + R.c) * slot_floats;
    for (int i = tid; i < cnt; i += kConsumerThreads) part[i] = gather(pc, i);
    __threadfence();
    consumer_sync();
    if (tid == 0) {
      const int done = atomicAdd(&pb.ws_ticket[pc.t], pc.hi - pc.lo) + (pc.hi - pc.lo);
      sh.flag = (done == blocks);
    }
    consumer_sync();
    if (!sh.flag) return true;
    // last lane of the tile: add the partials of all lanes in lane order
    __threadfence();
    if (warp == 0) {
      int count = 0;
      for (int base = 0; base < R.lanes; base += 32) {
        const int c2 = base + lane;
        int lo = 1, hi = 0;
        if (c2 < R.lanes) lane_piece<false>(P, sh, R.CB, c2, pc.t, pc.p, lo, hi);
        const unsigned m = __ballot_sync(0xffffffffu, lo < hi);
        if (lo < hi) sh.contrib[count + __popc(m & ((1u << lane) - 1u))] = c2;
        count += __popc(m);
      }
      if (lane == 0) sh.ncontrib = count;
    }
    consumer_sync();
    const int ncontrib = sh.ncontrib;
    for (int i = tid; i < cnt; i += kConsumerThreads) {
      float s = 0.f;
      for (int k = 0; k < ncontrib; ++k)
        s += __ldcg(pb.ws_part + (size_t)(pc.t + sh.contrib[k]) * slot_floats + i);
      v_tile[i] = s;
    }
    if (tid == 0) pb.ws_ticket[pc.t] = 0;   // leave the tickets zero for the next launch
    return true;
  }
};

struct SmemShrink {
  CtaShared sh;
  float scratch[kConsumerWarps * 2 * 2 * 128];
  uint64_t full[kShrinkStages], empty[kShrinkStages];
};
constexpr size_t kShrinkSmem = 128 + (size_t)kShrinkStages * kStageBytes + sizeof(SmemShrink);

__global__ void __launch_bounds__(kShrinkThreads, 3) shrink_stream_kernel(const StreamParams P) {
  extern __shared__ uint8_t dyn_smem_raw[];
  uint8_t *dyn = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(dyn_smem_raw) + 127) & ~(uintptr_t)127);
  uint8_t *stages = dyn;
  SmemShrink &S = *reinterpret_cast<SmemShrink *>(dyn + (size_t)kShrinkStages * kStageBytes);
  const int warp = threadIdx.x >> 5;

  pdl_launch_dependents();
  if (threadIdx.x == 0) {
    for (int s = 0; s < kShrinkStages; ++s) {
      mbar_init(&S.full[s], 1);
      mbar_init(&S.empty[s], kConsumerWarps);
    }
    fence_mbar_init();
  }
  CtaRange R;
  const bool work = prologue<false>(P, S.sh, R, true);   // ends with a __syncthreads when the plan is valid
  if (!work) {
    pdl_wait();
    return;
  }
  volatile int *abort_flag = &S.sh.abort_flag;
  ShrinkLoader loader{P, S.sh, stages, S.full, S.empty, abort_flag, 0};
  ShrinkConsumer consumer{P, S.sh, R, stages, S.full, S.empty, S.scratch, abort_flag, 0};
  bool waited = false, ok = true;
  for (int tb = R.t0; tb < R.t_end; tb += kBatchTiles) {
    const int ntile = min(kBatchTiles, R.t_end - tb);
    load_batch(P, S.sh, tb, ntile);
    if (!waited) {
      pdl_wait();   // activations, v and the tickets belong to earlier kernels until here
      waited = true;
    }
    if (*abort_flag) break;
    if (warp < kConsumerWarps) ok = walk_batch<false>(P, R, S.sh, tb, ntile, consumer);
    else ok = walk_batch<false>(P, R, S.sh, tb, ntile, loader);
    if (!ok) {
      *abort_flag = 1;
      if ((threadIdx.x & 31) == 0) report(P.status, MINT_ERR_TIMEOUT, blockIdx.x);
    }
  }
  if (*abort_flag && warp == kConsumerWarps) {
    // give the copies this warp issued a bounded chance to land before the CTA leaves
    const uint32_t q = loader.q;
    int never = 0;
    for (uint32_t i = q > kShrinkStages ? q - kShrinkStages : 0; i < q; ++i)
      mbar_wait(&S.full[i % kShrinkStages], (i / kShrinkStages) & 1u, &never);
  }
}

// ================================================================================
// expand
// ================================================================================
struct ExpandLoader {
  const StreamParams &P;
  const CtaShared &sh;
  uint8_t *stages;
  uint64_t *full, *empty;
  volatile int *abort_flag;
  uint32_t q;
  // Chunks [0, limit) were given their weight rows before the dependency wait
  // (pass 0, weights only) and get their y rows in pass 1; later chunks get both.
  int pass;          // 0: weights only, stop at `limit` chunks; 1: the rest
  uint32_t limit;    // pass 0: chunks to prefetch; pass 1: chunks whose weights are already in flight

  __device__ __forceinline__ bool piece_begin(const Piece &) { return true; }
  __device__ __forceinline__ bool piece_end(const Piece &) { return true; }
  __device__ __forceinline__ bool chunk(const Piece &pc, int col, int width) {
    const int lane = threadIdx.x & 31;
    if (pass == 0 && q >= limit) return false;
    const uint32_t s = q % kExpandStages;
    const bool weights = pass == 0 || q >= limit;
    const bool outputs = pass == 1;
    if (weights && !mbar_wait(&empty[s], ((q / kExpandStages) & 1u) ^ 1u, abort_flag)) return false;
    const StreamProblem &pb = P.prob[pc.p];
    uint8_t *stage = stages + (size_t)s * kStageBytes;
    const uint32_t row_bytes = (uint32_t)width * 2u;
    if (lane == 0) {
      if (weights) mbar_arrive_expect_tx(&full[s], row_bytes * (uint32_t)pc.r);
      if (outputs) mbar_arrive_expect_tx(&full[s], row_bytes * (uint32_t)pc.len);
    }
    __syncwarp();
    if (weights) {
      const uint16_t *B_slot = pb.B + (int64_t)pc.slot * pb.r_max * pb.n;
      for (int i = lane; i < pc.r; i += 32)
        bulk_load(stage + (size_t)i * pc.g.pitch, B_slot + (int64_t)i * pb.n + col, row_bytes, &full[s]);
    }
    if (outputs) {
      for (int i = lane; i < pc.len; i += 32)
        bulk_load(stage + (size_t)(pc.g.w_rows + i) * pc.g.pitch,
                  pb.y + (int64_t)sh.rows[pc.row0 + i] * pb.ldy + col, row_bytes, &full[s]);
    }
    ++q;
    return true;
  }
};

// Splits v into a bf16 head and a bf16 remainder so that two MMAs carry about
// 16 significant bits of the fp32 shrink result into the expand.
__device__ __forceinline__ void split_pair(float a, float b, uint32_t &hi, uint32_t &lo) {
  hi = pack_bf16x2(a, b);
  lo = pack_bf16x2(a - bf16lo(hi), b - bf16hi(hi));
}

struct ExpandConsumer {
  const StreamParams &P;
  CtaShared &sh;
  uint8_t *stages;
  uint64_t *full, *done;
  float *vs;        // [32][64] fp32 v of the current tile, zero beyond len / rank; then [8][4] for the FMA path
  volatile int *abort_flag;
  uint32_t q;
  uint32_t vh[2][4][4], vl[2][4][4];   // v as MMA A-operand fragments [m-tile][k-step]
  uint32_t kmask[4][2];                // keeps only B rows below the rank, per k-step and fragment register

  __device__ __forceinline__ bool piece_begin(const Piece &pc) {
    const int tid = threadIdx.x, lane = tid & 31;
    const StreamProblem &pb = P.prob[pc.p];
    const float *v_tile = pb.ws_v + (size_t)pc.t * kTileRowsMax * pb.r_max;
    consumer_sync();   // the previous piece no longer reads vs
    if (pc.g.mma) {
      const int m_pad = round_up(pc.len, 16);
      for (int i = tid; i < m_pad * pc.g.w_rows; i += kConsumerThreads) {
        const int l = i / pc.g.w_rows, j = i - l * pc.g.w_rows;
        vs[l * kStreamRankCap + j] = (l < pc.len && j < pc.r) ? __ldcg(&v_tile[l * pc.r + j]) : 0.f;
      }
    } else {
      for (int i = tid; i < pc.len * pc.r; i += kConsumerThreads) vs[kSlotFloats + i] = __ldcg(&v_tile[i]);
    }
    consumer_sync();
    if (pc.g.mma) {
      const int g = lane >> 2, t = lane & 3;
#pragma unroll
      for (int mt = 0; mt < 2; ++mt)
#pragma unroll
        for (int ks = 0; ks < 4; ++ks) {
          if (mt * 16 < pc.len && ks * 16 < pc.r) {
            const float *r0 = vs + (mt * 16 + g) * kStreamRankCap + ks * 16 + 2 * t;
            const float *r1 = r0 + 8 * kStreamRankCap;
            split_pair(r0[0], r0[1], vh[mt][ks][0], vl[mt][ks][0]);
            split_pair(r1[0], r1[1], vh[mt][ks][1], vl[mt][ks][1]);
            split_pair(r0[8], r0[9], vh[mt][ks][2], vl[mt][ks][2]);
            split_pair(r1[8], r1[9], vh[mt][ks][3], vl[mt][ks][3]);
          }
        }
#pragma unroll
      for (int ks = 0; ks < 4; ++ks)
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          const int k = ks * 16 + h * 8 + 2 * t;   // B rows k and k + 1 sit in this register
          kmask[ks][h] = (k < pc.r ? 0x0000FFFFu : 0u) | (k + 1 < pc.r ? 0xFFFF0000u : 0u);
        }
    }
    return true;
  }
  __device__ __forceinline__ bool piece_end(const Piece &) { return true; }

  template <int MT, int KS>
  __device__ __forceinline__ void mma_chunk(const Piece &pc, uint8_t *stage, int width) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = lane >> 2, t = lane & 3;
    const uint32_t b_base = smem_addr(stage);
    uint8_t *y_base = stage + (size_t)pc.g.w_rows * pc.g.pitch;
    const int pairs = (width + 15) >> 4;
    const int m = lane >> 3;
    const uint32_t b_lane = b_base + (uint32_t)(((m & 1) * 8 + (lane & 7)) * pc.g.pitch + (m >> 1) * 16);
    for (int p = warp; p < pairs; p += kConsumerWarps) {
      float acc[MT][2][4];
#pragma unroll
      for (int mt = 0; mt < MT; ++mt)
#pragma unroll
        for (int nt = 0; nt < 2; ++nt)
#pragma unroll
          for (int e = 0; e < 4; ++e) acc[mt][nt][e] = 0.f;
#pragma unroll
      for (int ks = 0; ks < KS; ++ks) {
        uint32_t b[4];
        ldmatrix_x4_trans(b, b_lane + (uint32_t)(ks * 16 * pc.g.pitch) + p * 32);
        b[0] &= kmask[ks][0];
        b[1] &= kmask[ks][1];
        b[2] &= kmask[ks][0];
        b[3] &= kmask[ks][1];
#pragma unroll
        for (int mt = 0; mt < MT; ++mt) {
          mma_bf16(acc[mt][0], vh[mt][ks], b[0], b[1]);
          mma_bf16(acc[mt][0], vl[mt][ks], b[0], b[1]);
          mma_bf16(acc[mt][1], vh[mt][ks], b[2], b[3]);
          mma_bf16(acc[mt][1], vl[mt][ks], b[2], b[3]);
        }
      }
#pragma unroll
      for (int mt = 0; mt < MT; ++mt)
#pragma unroll
        for (int nt = 0; nt < 2; ++nt) {
          const int col = p * 16 + nt * 8 + 2 * t;
          if (col < width) {
#pragma unroll
            for (int h = 0; h < 2; ++h) {
              const int row = mt * 16 + g + h * 8;
              if (row < pc.len) {
                uint32_t *yp = reinterpret_cast<uint32_t *>(y_base + (size_t)row * pc.g.pitch + col * 2);
                const uint32_t w = *yp;
                *yp = pack_bf16x2(fmaf(pc.scale, acc[mt][nt][2 * h], bf16lo(w)),
                                  fmaf(pc.scale, acc[mt][nt][2 * h + 1], bf16hi(w)));
              }
            }
          }
        }
    }
  }

  __device__ __forceinline__ void fma_chunk(const Piece &pc, uint8_t *stage, int width) {
    const float *vc = vs + kSlotFloats;   // [len][rank]
    uint8_t *y_base = stage + (size_t)pc.g.w_rows * pc.g.pitch;
    for (int v = threadIdx.x; v < (width >> 3); v += kConsumerThreads) {
      float bf[4][8];
#pragma unroll
      for (int j = 0; j < 4; ++j)
        if (j < pc.r) unpack8(*reinterpret_cast<const uint4 *>(stage + (size_t)j * pc.g.pitch + v * 16), bf[j]);
#pragma unroll
      for (int l = 0; l < 8; ++l) {
        if (l < pc.len) {
          uint4 *yp = reinterpret_cast<uint4 *>(y_base + (size_t)l * pc.g.pitch + v * 16);
          float yf[8], dl[8];
          unpack8(*yp, yf);
#pragma unroll
          for (int e = 0; e < 8; ++e) dl[e] = 0.f;
#pragma unroll
          for (int j = 0; j < 4; ++j)
            if (j < pc.r) {
              const float vv = vc[l * pc.r + j];
#pragma unroll
              for (int e = 0; e < 8; ++e) dl[e] = fmaf(vv, bf[j][e], dl[e]);
            }
#pragma unroll
          for (int e = 0; e < 8; ++e) yf[e] = fmaf(pc.scale, dl[e], yf[e]);
          *yp = pack8(yf);
        }
      }
    }
  }

  __device__ __forceinline__ bool chunk(const Piece &pc, int, int width) {
    const uint32_t s = q % kExpandStages;
    if (!mbar_wait(&full[s], (q / kExpandStages) & 1u, abort_flag)) return false;
    uint8_t *stage = stages + (size_t)s * kStageBytes;
    const int ks = pc.g.w_rows >> 4;
    if (!pc.g.mma) fma_chunk(pc, stage, width);
    else if (pc.len <= 16) {
      if (ks == 1) mma_chunk<1, 1>(pc, stage, width);
      else if (ks == 2) mma_chunk<1, 2>(pc, stage, width);
      else if (ks == 3) mma_chunk<1, 3>(pc, stage, width);
      else mma_chunk<1, 4>(pc, stage, width);
    } else {
      if (ks == 1) mma_chunk<2, 1>(pc, stage, width);
      else if (ks == 2) mma_chunk<2, 2>(pc, stage, width);
      else if (ks == 3) mma_chunk<2, 3>(pc, stage, width);
      else mma_chunk<2, 4>(pc, stage, width);
    }
    fence_async_smem();   // this thread's y updates become visible to the bulk-copy engine
    __syncwarp();
    if ((threadIdx.x & 31) == 0) mbar_arrive(&done[s]);
    ++q;
    return true;
  }
};

struct ExpandStorer {
  const StreamParams &P;
  const CtaShared &sh;
  uint8_t *stages;
  uint64_t *done, *empty;
  volatile int *abort_flag;
  uint32_t q;

  __device__ __forceinline__ bool piece_begin(const Piece &) { return true; }
  __device__ __forceinline__ bool piece_end(const Piece &) { return true; }
  __device__ __forceinline__ bool chunk(const Piece &pc, int col, int width) {
    const int lane = threadIdx.x & 31;
    const uint32_t s = q % kExpandStages;
    if (!mbar_wait(&done[s], (q / kExpandStages) & 1u, abort_flag)) return false;
    const StreamProblem &pb = P.prob[pc.p];
    uint8_t *y_base = stages + (size_t)s * kStageBytes + (size_t)pc.g.w_rows * pc.g.pitch;
    for (int l = lane; l < pc.len; l += 32)
      bulk_store(pb.y + (int64_t)sh.rows[pc.row0 + l] * pb.ldy + col, y_base + (size_t)l * pc.g.pitch,
                 (uint32_t)width * 2u);
    bulk_commit();
    bulk_wait_read_all();   // the stores have read their shared-memory source: the stage may be refilled
    __syncwarp();
    if (lane == 0) mbar_arrive(&empty[s]);
    ++q;
    return true;
  }
};

struct SmemExpand {
  CtaShared sh;
  float vs[kSlotFloats + 32];
  uint64_t full[kExpandStages], empty[kExpandStages], done[kExpandStages];
};
constexpr size_t kExpandSmem = 128 + (size_t)kExpandStages * kStageBytes + sizeof(SmemExpand);

__global__ void __launch_bounds__(kExpandThreads, 2) expand_stream_kernel(const StreamParams P) {
  extern __shared__ uint8_t dyn_smem_raw[];
  uint8_t *dyn = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(dyn_smem_raw) + 127) & ~(uintptr_t)127);
  uint8_t *stages = dyn;
  SmemExpand &S = *reinterpret_cast<SmemExpand *>(dyn + (size_t)kExpandStages * kStageBytes);
  const int warp = threadIdx.x >> 5;

  pdl_launch_dependents();
  if (threadIdx.x == 0) {
    for (int s = 0; s < kExpandStages; ++s) {
      mbar_init(&S.full[s], 2);   // one arrival with the weight bytes, one with the y bytes
      mbar_init(&S.empty[s], 1);
      mbar_init(&S.done[s], kConsumerWarps);
    }
    fence_mbar_init();
  }
  CtaRange R;
  // The plan, the slot table and B were complete before the shrink kernel of
  // this call started, so they may be read before the dependency wait; y and v
  // may not.  Errors of the plan were already reported by the shrink kernel.
  const bool work = prologue<true>(P, S.sh, R, false);
  if (!work) {
    pdl_wait();
    return;
  }
  volatile int *abort_flag = &S.sh.abort_flag;
  ExpandLoader loader{P, S.sh, stages, S.full, S.empty, abort_flag, 0, 1, 0};
  ExpandConsumer consumer{P, S.sh, stages, S.full, S.done, S.vs, abort_flag, 0};
  ExpandStorer storer{P, S.sh, stages, S.done, S.empty, abort_flag, 0};
  bool waited = false, ok = true;
  for (int tb = R.t0; tb < R.t_end; tb += kBatchTiles) {
    const int ntile = min(kBatchTiles, R.t_end - tb);
    load_batch(P, S.sh, tb, ntile);
    if (!waited) {
      if (warp == kConsumerWarps) {   // weights of the first ring-full of chunks go out before the wait
        loader.pass = 0;
        loader.limit = kExpandStages;
        walk_batch<true>(P, R, S.sh, tb, ntile, loader);
        loader.limit = loader.q;
        loader.q = 0;
        loader.pass = 1;
      }
      pdl_wait();   // the shrink kernel has completed: v is final, y belongs to this kernel
      waited = true;
    }
    if (*abort_flag) break;
    if (warp < kConsumerWarps) ok = walk_batch<true>(P, R, S.sh, tb, ntile, consumer);
    else if (warp == kConsumerWarps) ok = walk_batch<true>(P, R, S.sh, tb, ntile, loader);
    else ok = walk_batch<true>(P, R, S.sh, tb, ntile, storer);
    if (!ok) {
      *abort_flag = 1;
      if ((threadIdx.x & 31) == 0) report(P.status, MINT_ERR_TIMEOUT, blockIdx.x);
    }
  }
  if (warp == kConsumerWarps + 1) bulk_wait_all();   // all y rows have left shared memory and are written
  if (*abort_flag && warp == kConsumerWarps) {
    const uint32_t q = loader.q;
    int never = 0;
    for (uint32_t i = q > kExpandStages ? q - kExpandStages : 0; i < q; ++i)
      mbar_wait(&S.full[i % kExpandStages], (i / kExpandStages) & 1u, &never);
  }
}

// ---- host side -----------------------------------------------------------------
int g_attr_done = 0;

int32_t ensure_attrs() {
  if (g_attr_done) return MINT_OK;
  int32_t st = mint_check_cuda(cudaFuncSetAttribute(shrink_stream_kernel,
                                                    cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kShrinkSmem),
                               "shrink_stream smem attribute");
  if (st) return st;
  st = mint_check_cuda(cudaFuncSetAttribute(expand_stream_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                            (int)kExpandSmem),
                       "expand_stream smem attribute");
  if (st) return st;
  g_attr_done = 1;
  return MINT_OK;
}

struct WorkspaceLayout {
  size_t ticket, v, part, total;
};

WorkspaceLayout workspace_layout(int64_t tiles, int32_t r_max) {
  WorkspaceLayout w;
  const size_t slot_bytes = (size_t)kTileRowsMax * r_max * sizeof(float);
  w.ticket = 0;
  w.v = ((size_t)tiles * 4 + 255) / 256 * 256;
  w.part = w.v + (size_t)tiles * slot_bytes;
  w.total = w.part + (size_t)(tiles + MINT_MAX_LANES) * slot_bytes + 256;
  return w;
}

}  // namespace

bool mint_stream_supported(int32_t r_max_bound) { return r_max_bound <= kStreamRankCap; }

size_t mint_stream_workspace_bytes(int32_t T, int32_t num_slots, int32_t r_max) {
  return workspace_layout(mint_tile_upper_bound(1, T, num_slots), r_max).total;
}

int32_t mint_launch_stream(const DenseArgs *args, int nprob, const TableDev &tab, const void *plan_dev,
                           void *const *workspaces, cudaStream_t s) {
  if (nprob < 1 || nprob > kMaxProblems)
    return mint_fail(MINT_ERR_INVALID_ARG, "grouped apply: 1..%d problems", kMaxProblems);
  int32_t st = ensure_attrs();
  if (st) return st;
  int32_t lanes = 0;
  if ((st = mint_device_lanes(&lanes))) return st;
  const int32_t T = args[0].T;
  const int64_t tiles = mint_tile_upper_bound(1, T, tab.num_slots);
  if (tiles == 0) return MINT_OK;
  StreamParams P = {};
  int cb_s = 0, cb_e = 0;
  for (int i = 0; i < nprob; ++i) {
    const DenseArgs &a = args[i];
    StreamProblem &pb = P.prob[i];
    pb.A = a.A; pb.B = a.B; pb.x = a.x; pb.y = a.y;
    pb.ldx = a.ldx; pb.ldy = a.ldy;
    pb.d = a.d; pb.n = a.n; pb.r_max = a.r_max;
    pb.cb0_shrink = cb_s;
    pb.cb0_expand = cb_e;
    cb_s += (a.d + 15) >> 4;
    cb_e += (a.n + 15) >> 4;
    const WorkspaceLayout w = workspace_layout(tiles, a.r_max);
    uint8_t *base = static_cast<uint8_t *>(workspaces[i]);
    pb.ws_ticket = reinterpret_cast<int32_t *>(base + w.ticket);
    pb.ws_v = reinterpret_cast<float *>(base + w.v);
    pb.ws_part = reinterpret_cast<float *>(base + w.part);
  }
  P.nprob = nprob;
  P.T = T;
  P.lanes = lanes;
  P.cb_shrink = cb_s;
  P.cb_expand = cb_e;
  P.status = args[0].status;
  P.tab = tab;
  P.pv = mint_plan_view(plan_dev, T, tab.num_slots);

  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)lanes);
  cfg.stream = s;
  cfg.attrs = attr;
  cfg.numAttrs = 1;

  cfg.blockDim = dim3(kShrinkThreads);
  cfg.dynamicSmemBytes = kShrinkSmem;
  st = mint_check_cuda(cudaLaunchKernelEx(&cfg, shrink_stream_kernel, P), "shrink_stream launch");
  if (st) return st;
  cfg.blockDim = dim3(kExpandThreads);
  cfg.dynamicSmemBytes = kExpandSmem;
  return mint_check_cuda(cudaLaunchKernelEx(&cfg, expand_stream_kernel, P), "expand_stream launch");
}
