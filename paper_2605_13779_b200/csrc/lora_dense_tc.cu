// Tensor-core kernels for dense segments.  First the shrink:
//   v[128-row tile] = X[tile rows, :] . A_slot^T   (d -> r);
// the expand (r -> n with the update of y) follows further down.
//
// A segmented-prefill batch holds runs of hundreds of tokens of one adapter; for
// those the d -> r contraction is a genuinely dense [128 x d] . [d x r] product
// per 128-token tile, and it runs on the fifth-generation tensor cores:
// tcgen05.mma (M = 128, N = the rank rounded up to 16, K = 16 per instruction,
// bf16 operands, fp32 accumulators in tensor memory), issued by one thread of
// the CTA.  Both operands have the reduction index contiguous in memory (rows
// of x, rows of A[slot][rank][d]), the K-major case of the MMA.
//
// One CTA per 128-row tile walks d in chunks of 64 columns.  A chunk of the token
// rows (128 x 128 bytes) and of the rank rows (N x 128 bytes) is copied into a
// shared-memory stage with 16-byte asynchronous copies, eight consecutive
// threads per row, in the 128-byte-swizzled layout the MMA's shared-memory
// descriptors name (16-byte chunk c of row i at chunk c ^ (i & 7) of its row,
// rows in groups of 8 x 128 bytes).  Four stages are in flight; a stage is
// refilled once the MMAs that read it have signalled an mbarrier
// (tcgen05.commit).  After the last chunk every warp reads its 32 accumulator
// rows out of tensor memory (tcgen05.ld) and writes them, fp32, to the slots of
// the workspace from which the expand kernel takes v: a region of slots of its
// own, one per 32-token sub-tile (the streamed shrink skips these tiles).
//
// Every wait on an mbarrier is bounded; a wait that runs out records
// MINT_ERR_TIMEOUT, and the CTA still frees its tensor memory before it returns.
#include <algorithm>

#include "mint_tc.cuh"

using namespace mint;
using namespace mint::tc;

namespace {

constexpr int kThreads = 128;
constexpr int kTileRows = 128;          // M of the MMA
constexpr int kChunk = 64;              // columns of d per stage: one 128-byte swizzle atom per row
constexpr int kStages = 4;
constexpr int kMaxRank = 64;            // N <= 64
constexpr int kXStageBytes = kTileRows * 128;
constexpr int kAStageBytes = kMaxRank * 128;
constexpr int kStageBytes = kXStageBytes + kAStageBytes;   // 24 KB
constexpr int kTmemCols = 64;
constexpr size_t kDynSmem = (size_t)kStages * kStageBytes + 1024;   // + alignment slack
constexpr int kMaxProblems = MINT_MAX_GROUP;

struct DenseProblem {
  const uint16_t *A;   // [slot][r_max][d]
  const uint16_t *x;
  int64_t ldx;
  int32_t d, r_max;
  int32_t splits;      // CTAs per tile, each over an equal share of the 64-column chunks of d
  int32_t use_tma;     // the two tensor maps below are valid
  float *ws_part;      // slots of 32 * r_max floats, [len][rank] packed fp32
  alignas(64) CUtensorMap x_map;   // x as [T][d], boxes of 128 rows x 64 columns, 128-byte swizzle
  alignas(64) CUtensorMap a_map;   // A as [slots * r_max][d], boxes of 64 rows x 64 columns
};

struct DenseParams {
  DenseProblem prob[kMaxProblems];
  int32_t nprob;
  int32_t T;
  int32_t lanes;
  int32_t dense_slot0;   // part s of the v of dense tile t goes to workspace slot dense_slot0 + s * dense_stride + t
  int32_t dense_stride;
  int32_t withhold;      // self-test only: no MMA is issued and nothing ever signals the barriers, so the waits run out
  uint64_t wait_ns;      // limit of every wait
  int32_t *status;
  TableDev tab;
  PlanView pv;
};


__global__ void __launch_bounds__(kThreads, 2) dense_shrink_kernel(const __grid_constant__ DenseParams P) {
  extern __shared__ uint8_t dyn_raw[];
  __shared__ uint64_t mma_done[kStages];   // a stage's MMAs have read it
  __shared__ uint64_t full[kStages];       // a stage's tiles have landed (tensor-map path)
  __shared__ uint64_t all_done;
  __shared__ uint32_t tmem_base_slot;
  __shared__ int32_t rows[kTileRows];
  __shared__ volatile int32_t failed;   // written after a wait that ran out; read only after a CTA barrier
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  // the grid's second dimension runs over the shares of d of all problems laid end to end
  int split = blockIdx.y, z = 0;
  while (z + 1 < P.nprob && split >= P.prob[z].splits) split -= P.prob[z++].splits;
  const DenseProblem &pb = P.prob[z];

  pdl_launch_dependents();
  // The plan and the pool weights were complete before this call's kernels
  // started; activations and the workspace are touched only after the wait.
  const bool ok = plan_ok(P.pv.header, P.T, 1, P.tab.num_slots, 0, P.tab.gen_lo, P.tab.gen_hi, nullptr) &&
                  P.pv.header[PH_LANES] == P.lanes;
  const int m = blockIdx.x;
  if (!ok || m >= P.pv.header[PH_NUM_DENSE] || split >= pb.splits) {
    pdl_wait();
    return;
  }
  const int ntiles = P.pv.header[PH_NCHUNK1];
  const int listed = P.pv.dense_tile[m];
  const int t0 = listed < 0 ? ~listed : listed;   // (~tile: the plan found its tokens scattered)
  const TileDesc d0 = P.pv.tile_desc[t0];
  // the 128-row tile = up to four consecutive 32-token tiles of the segment
  int nrows = d0.len;
  {
    TileDesc dn[3];   // the three descriptors that may follow, requested together
#pragma unroll
    for (int i = 1; i < 4; ++i) dn[i - 1] = P.pv.tile_desc[min(t0 + i, ntiles - 1)];
#pragma unroll
    for (int i = 1; i < 4; ++i) {
      const TileDesc &di = dn[i - 1];
      if (nrows != 32 * i || t0 + i >= ntiles || !di.dense || di.slot != d0.slot || di.off != d0.off + 32 * i) break;
      nrows += di.len;
    }
  }
  const int r = d0.rank;
  if (r > pb.r_max || r > kMaxRank || r < 1) {
    if (tid == 0) report(P.status, MINT_ERR_RANK_TOO_LARGE, d0.slot);
    pdl_wait();
    return;
  }
  const int n_mma = (r + 15) / 16 * 16;
  for (int i = tid; i < kTileRows; i += kThreads) rows[i] = i < nrows ? P.pv.perm[d0.off + i] : 0;
  if (tid == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(&mma_done[s], 1);
      mbar_init(&full[s], 1);
    }
    mbar_init(&all_done, 1);
    fence_mbar_init();
    failed = 0;
  }
  if (warp == 0) tmem_alloc(&tmem_base_slot, kTmemCols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_d = tmem_base_slot;
  const uint32_t stage0 = (smem_addr(dyn_raw) + 1023u) & ~1023u;   // swizzle atoms are 1024-byte aligned
  const uint16_t *A_rows = pb.A + (int64_t)d0.slot * pb.r_max * pb.d;
  const uint32_t idesc = instr_desc(n_mma);
  // this CTA's share of the chunks of d: [chunk0, chunk0 + nchunks)
  const int all_chunks = (pb.d + kChunk - 1) / kChunk;
  const int chunk0 = (int)((int64_t)all_chunks * split / pb.splits);
  const int nchunks = (int)((int64_t)all_chunks * (split + 1) / pb.splits) - chunk0;

  pdl_wait();

  // A tile whose tokens are consecutive rows of x (a request's tokens usually are) comes in through the
  // tensor maps: one thread asks for the two tiles of a chunk (hardware swizzle, bytes counted on the
  // stage's mbarrier), another issues the MMAs as soon as a stage is full and hands it back when they
  // have read it; nobody computes an address per row and no barrier of the CTA sits in the loop.
  const bool contiguous = pb.use_tma && listed >= 0;
  if (contiguous) {
    if (warp == 0) {
     if (lane == 0) {   // producer
      int kc = 0;
      for (; kc < nchunks; ++kc) {
        const int s = kc % kStages;
        if (kc >= kStages && !mbar_wait(&mma_done[s], ((kc / kStages) - 1) & 1u, P.wait_ns)) {
          failed = 1;
          break;
        }
        const uint32_t xs = stage0 + (uint32_t)(s * kStageBytes), as = xs + kXStageBytes;
        mbar_arrive_expect_tx(&full[s], (uint32_t)kStageBytes);
        const int col = (chunk0 + kc) * kChunk;
        tma_load_2d(xs, &pb.x_map, col, rows[0], &full[s]);
        tma_load_2d(as, &pb.a_map, col, d0.slot * pb.r_max, &full[s]);
      }
      if (failed)   // the tiles still on their way land before this CTA's memory goes away
        for (int j = max(0, kc - kStages); j < kc; ++j) mbar_wait(&full[j % kStages], (j / kStages) & 1u, 100000000ull);
     }
     __syncwarp();
    } else if (warp == 1) {
     if (lane == 0) {   // MMA issuer
      bool ok_mma = true;
      for (int kc = 0; kc < nchunks && ok_mma; ++kc) {
        const int s = kc % kStages;
        if (!mbar_wait(&full[s], (kc / kStages) & 1u, P.wait_ns)) {
          failed = 1;
          ok_mma = false;
          break;
        }
        if (P.withhold) continue;
        tc_fence_after();
        const uint32_t xs = stage0 + (uint32_t)(s * kStageBytes), as = xs + kXStageBytes;
        const uint64_t da = smem_desc_k_sw128(xs), db = smem_desc_k_sw128(as);
#pragma unroll
        for (int ks = 0; ks < kChunk / 16; ++ks)
          umma_bf16(tmem_d, da + (uint64_t)(2 * ks), db + (uint64_t)(2 * ks), idesc, kc > 0 || ks > 0);
        umma_commit(&mma_done[s]);
      }
      if (!P.withhold) umma_commit(&all_done);
     }
     __syncwarp();
    }
  } else {
  // this thread's 16-byte pieces of a stage: row q >> 3, chunk q & 7 for q = tid + 128 i
  auto issue = [&](int kc) {
    if (kc < nchunks) {
      const uint32_t xs = stage0 + (uint32_t)((kc % kStages) * kStageBytes), as = xs + kXStageBytes;
      const int c = tid & 7;
      const int col = (chunk0 + kc) * kChunk + c * 8;
      const bool col_ok = col < pb.d;
#pragma unroll
      for (int i = 0; i < kTileRows / 16; ++i) {
        const int row = (tid >> 3) + 16 * i;
        const bool v = col_ok && row < nrows;
        cp_async16(xs + (uint32_t)((row >> 3) * 1024 + (row & 7) * 128 + ((c ^ (row & 7)) << 4)),
                   v ? pb.x + (int64_t)rows[row] * pb.ldx + col : pb.x, v);
      }
      for (int row = tid >> 3; row < n_mma; row += 16) {
        const bool v = col_ok && row < r;
        cp_async16(as + (uint32_t)((row >> 3) * 1024 + (row & 7) * 128 + ((c ^ (row & 7)) << 4)),
                   v ? A_rows + (int64_t)row * pb.d + col : pb.A, v);
      }
    }
    cp_async_commit();
  };

  for (int kc = 0; kc < kStages - 1; ++kc) issue(kc);
  for (int kc = 0; kc < nchunks; ++kc) {
    const int s = kc % kStages;
    cp_async_wait<kStages - 2>();   // this thread's copies of chunk kc have landed
    fence_async_smem();             // ... and are visible to the tensor core's reads of shared memory
    __syncthreads();
    if (tid == 0 && !failed && !P.withhold) {
      tc_fence_after();
      const uint32_t xs = stage0 + (uint32_t)(s * kStageBytes), as = xs + kXStageBytes;
      const uint64_t da = smem_desc_k_sw128(xs), db = smem_desc_k_sw128(as);
#pragma unroll
      for (int ks = 0; ks < kChunk / 16; ++ks)   // 16 columns = 32 bytes further along the swizzled rows
        umma_bf16(tmem_d, da + (uint64_t)(2 * ks), db + (uint64_t)(2 * ks), idesc, kc > 0 || ks > 0);
      umma_commit(&mma_done[s]);
    }
    // chunk kc + kStages - 1 reuses the stage of chunk kc - 1: wait for the MMAs that read it
    if (!failed && kc >= 1 && kc + kStages - 1 < nchunks) {
      const int sp = (kc - 1) % kStages;
      if (!mbar_wait(&mma_done[sp], ((kc - 1) / kStages) & 1u, P.wait_ns)) failed = 1;
    }
    issue(kc + kStages - 1);
  }
  cp_async_wait<0>();
  if (tid == 0 && !P.withhold) umma_commit(&all_done);
  }
  // Also after an earlier wait ran out: whatever this CTA issued has to be complete (or given up on
  // for a second time) before its tensor memory is freed.
  if (!mbar_wait(&all_done, 0, P.wait_ns)) failed = 1;
  tc_fence_after();
  __syncthreads();
  if (!failed) {
    // warp w owns accumulator rows 32 w .. 32 w + 31 (tensor-memory lanes), one row per thread
    const int row = warp * 32 + lane;
    const size_t slot_floats = (size_t)32 * pb.r_max;
    float *dst = pb.ws_part + (size_t)(P.dense_slot0 + split * P.dense_stride + t0 + (row >> 5)) * slot_floats +
                 (size_t)(row & 31) * r;
    for (int j0 = 0; j0 < n_mma; j0 += 16) {
      float v[16];
      tmem_ld16(tmem_d + ((uint32_t)(warp * 32) << 16) + (uint32_t)j0, v);
      if (row < nrows) {
#pragma unroll
        for (int j = 0; j < 16; ++j)
          if (j0 + j < r) dst[j0 + j] = v[j];
      }
    }
  } else if (tid == 0) {
    report(P.status, MINT_ERR_TIMEOUT, m);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem_d, kTmemCols);
}


// ====================================================================================
// Tensor-core expand for dense segments:  Y[128-row tile, :] += s * v[tile] . B_slot   (r -> n).
//
// One CTA takes a 128-row tile and a range of kColsPerCta columns of n, 128
// columns at a time.  v (fp32, left by the tensor-core shrink in the workspace)
// is scaled by s and split into a bf16 head and a bf16 remainder, both stored
// once as K-major MMA A operands (128 rows x 64 ranks, 128-byte-swizzled).  B
// is [rank][n] in memory, n contiguous, which is the wrong way round for a
// K-major operand: a chunk (64 ranks x 128 columns) is copied as it is into a
// staging buffer (cp.async) and transposed through the registers
// (ldmatrix.trans, 32-bit stores) into the swizzled K-major layout; the next
// chunk's copy starts as soon as the staging buffer has been read.  Two chains
// of tcgen05.mma (head, then remainder, M = 128, N = 128, K = 16 each) leave
// Y's update in 128 columns of tensor memory.  The 128 x 128 tile of y comes
// into shared memory with coalesced 16-byte copies while all that happens;
// every thread then adds its accumulator row (tcgen05.ld) to its row of the
// tile, and the warp writes its 32 rows back to memory, two whole rows per
// store instruction.  (A thread reading and writing its row of y in memory
// directly touches 32 cache lines per instruction; that version ran at a third
// of the speed.)  B is read once per 128 tokens; the streamed expand reads it
// once per 32.  Waits are bounded as in the shrink.
constexpr int kExpChunk = 128;                 // columns of n per MMA (N)
constexpr int kColsPerCta = 16384;
constexpr int kStageRowBytes = kExpChunk * 2 + 16;   // padded: rows of a transposing 8x8 load fall into different banks
constexpr int kBStageBytes = kMaxRank * kStageRowBytes;          // 17408
constexpr int kYRowBytes = kExpChunk * 2 + 16;                   // padded: a warp's 16-byte accesses to 8 rows do not collide
constexpr int kYTileBytes = kTileRows * kYRowBytes;              // 34816
constexpr int kVBytes = kTileRows * 128;                         // one A operand: 16 KB
constexpr int kBkmBytes = kExpChunk * 128;                       // 16 KB
constexpr size_t kExpDynSmem = 2 * kVBytes + kBkmBytes + kBStageBytes + kYTileBytes + 1024;
constexpr int kExpTmemCols = 128;

struct DenseExpandProblem {
  const uint16_t *B;   // [slot][r_max][n]
  uint16_t *y;
  int64_t ldy;
  int32_t n, r_max;
  int32_t splits;      // parts of v per tile (the shrink's split of d)
  int32_t use_tma;     // the two tensor maps below are valid
  const float *ws_part;
  alignas(64) CUtensorMap b_map;   // B as [slots * r_max][n], boxes of 64 rows x 64 columns, 128-byte swizzle
  alignas(64) CUtensorMap y_map;   // y as [T][n], boxes of 128 rows x 64 columns
};
struct DenseExpandParams {
  DenseExpandProblem prob[kMaxProblems];
  int32_t nprob;
  int32_t T;
  int32_t lanes;
  int32_t dense_slot0;
  int32_t dense_stride;
  int32_t *status;
  TableDev tab;
  PlanView pv;
};

// The grid's second dimension runs over the column ranges of all problems laid end to end (a
// narrow problem then brings no CTAs that only exit).  A problem of n columns has
// ceil(n / kColsPerCta) ranges of equal width (a multiple of the 128-column chunk): returns the
// problem of range y and its columns [col_begin, col_end).
__device__ __forceinline__ int expand_range(const DenseExpandParams &P, int y, int &col_begin, int &col_end) {
  int z = 0, ranges = 1;
  for (;; ++z) {
    ranges = (P.prob[z].n + kColsPerCta - 1) / kColsPerCta;
    if (y < ranges || z + 1 >= P.nprob) break;
    y -= ranges;
  }
  const int n = P.prob[z].n;
  const int per = ((n + ranges - 1) / ranges + kExpChunk - 1) / kExpChunk * kExpChunk;
  col_begin = y * per;
  col_end = min(n, col_begin + per);
  return z;
}

__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(addr)
               : "memory");
}
__device__ __forceinline__ void sts32(uint32_t addr, uint32_t v) {
  asm volatile("st.shared.b32 [%0], %1;" ::"r"(addr), "r"(v) : "memory");
}
__device__ __forceinline__ void sts128(uint32_t addr, const uint4 &v) {
  asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};" ::"r"(addr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}
__device__ __forceinline__ uint4 lds128(uint32_t addr) {
  uint4 r;
  asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w) : "r"(addr) : "memory");
  return r;
}
// byte offset of (row, 16-byte chunk c) in a 128-byte-swizzled K-major tile
__device__ __forceinline__ uint32_t sw128(int row, int c) {
  return (uint32_t)((row >> 3) * 1024 + (row & 7) * 128 + ((c ^ (row & 7)) << 4));
}

__global__ void __launch_bounds__(kThreads, 2) dense_expand_kernel(const __grid_constant__ DenseExpandParams P) {
  extern __shared__ uint8_t dyn_raw[];
  __shared__ uint64_t mma_done;
  __shared__ uint64_t drain;            // after a wait ran out: everything issued so far, once more
  __shared__ uint32_t tmem_base_slot;
  __shared__ int32_t rows[kTileRows];
  __shared__ volatile int32_t failed;   // written after a wait that ran out; read only after a CTA barrier
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  int col_begin, col_end;
  const DenseExpandProblem &pb = P.prob[expand_range(P, (int)blockIdx.y, col_begin, col_end)];

  pdl_launch_dependents();
  const bool ok = plan_ok(P.pv.header, P.T, 1, P.tab.num_slots, 0, P.tab.gen_lo, P.tab.gen_hi, nullptr) &&
                  P.pv.header[PH_LANES] == P.lanes;
  const int m = blockIdx.x;
  // (with tensor maps this kernel is left the tiles whose tokens are scattered: usually none)
  if (!ok || m >= P.pv.header[PH_NUM_DENSE] || col_begin >= pb.n ||
      (pb.use_tma && P.pv.header[PH_NUM_SCATTERED] == 0)) {
    pdl_wait();
    return;
  }
  const int ntiles = P.pv.header[PH_NCHUNK1];
  const int listed = P.pv.dense_tile[m];
  if (pb.use_tma && listed >= 0) {   // a tile of consecutive tokens is the tensor-map kernel's
    pdl_wait();
    return;
  }
  const int t0 = listed < 0 ? ~listed : listed;
  const TileDesc d0 = P.pv.tile_desc[t0];
  int nrows = d0.len;
  {
    TileDesc dn[3];   // the three descriptors that may follow, requested together
#pragma unroll
    for (int i = 1; i < 4; ++i) dn[i - 1] = P.pv.tile_desc[min(t0 + i, ntiles - 1)];
#pragma unroll
    for (int i = 1; i < 4; ++i) {
      const TileDesc &di = dn[i - 1];
      if (nrows != 32 * i || t0 + i >= ntiles || !di.dense || di.slot != d0.slot || di.off != d0.off + 32 * i) break;
      nrows += di.len;
    }
  }
  const int r = d0.rank;
  if (r > pb.r_max || r > kMaxRank || r < 1) {   // reported by the shrink
    pdl_wait();
    return;
  }
  const int k_mma = (r + 15) / 16 * 16;
  for (int i = tid; i < kTileRows; i += kThreads) rows[i] = i < nrows ? P.pv.perm[d0.off + i] : 0;
  if (tid == 0) {
    mbar_init(&mma_done, 1);
    mbar_init(&drain, 1);
    fence_mbar_init();
    failed = 0;
  }
  if (warp == 0) tmem_alloc(&tmem_base_slot, kExpTmemCols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_d = tmem_base_slot;
  const uint32_t base = (smem_addr(dyn_raw) + 1023u) & ~1023u;
  const uint32_t v_hi = base, v_lo = base + kVBytes, b_km = base + 2 * kVBytes;
  const uint32_t stage = b_km + kBkmBytes, ytile = stage + kBStageBytes;
  const uint16_t *B_rows = pb.B + (int64_t)d0.slot * pb.r_max * pb.n;
  const uint32_t idesc = instr_desc(kExpChunk);
  const int nchunks = (col_end - col_begin + kExpChunk - 1) / kExpChunk;

  // B chunk kc into the staging buffer: rows k < k_mma (zero beyond the rank), 16 x 16-byte pieces per row
  auto issue_b = [&](int kc) {
    if (kc < nchunks) {
      const int c = tid & 15;
      const int col = col_begin + kc * kExpChunk + c * 8;
      for (int k = tid >> 4; k < k_mma; k += 8) {
        const bool v = k < r && col < col_end;
        cp_async16(stage + (uint32_t)(k * kStageRowBytes + c * 16), v ? B_rows + (int64_t)k * pb.n + col : pb.B, v);
      }
    }
    cp_async_commit();
  };
  // the y tile of chunk kc: 16 consecutive threads copy the 256 bytes of a row
  auto issue_y = [&](int kc) {
    const int c = tid & 15;
    const int col = col_begin + kc * kExpChunk + c * 8;
#pragma unroll 4
    for (int row = tid >> 4; row < kTileRows; row += 8) {
      const bool v = row < nrows && col < col_end;
      cp_async16(ytile + (uint32_t)(row * kYRowBytes + c * 16), v ? pb.y + (int64_t)rows[row] * pb.ldy + col : pb.y, v);
    }
    cp_async_commit();
  };
  issue_b(0);   // weights: not written by any kernel of the stream

  pdl_wait();   // v and y belong to the earlier kernels until here

  // v, scaled, as head and remainder: consecutive threads take consecutive pairs of ranks of a row
  {
    const size_t slot_floats = (size_t)32 * pb.r_max;
    const int pairs = k_mma / 2;
    for (int q0 = tid; q0 < kTileRows * pairs; q0 += 8 * kThreads) {
      float a[8], b[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) a[u] = b[u] = 0.f;
      for (int sp = 0; sp < pb.splits; ++sp) {   // the parts of the shrink's CTAs, in their order; 16 loads go out together
        float pa[8], pbv[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
          const int q = q0 + u * kThreads;
          const int row = q / pairs, k = 2 * (q - row * pairs);
          const bool in = q < kTileRows * pairs && row < nrows;
          const float *src = pb.ws_part + (size_t)(P.dense_slot0 + sp * P.dense_stride + t0 + (row >> 5)) * slot_floats +
                             (size_t)(row & 31) * r;
          pa[u] = (in && k < r) ? __ldcg(src + k) : 0.f;
          pbv[u] = (in && k + 1 < r) ? __ldcg(src + k + 1) : 0.f;
        }
#pragma unroll
        for (int u = 0; u < 8; ++u) {
          a[u] += pa[u];
          b[u] += pbv[u];
        }
      }
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const int q = q0 + u * kThreads;
        if (q < kTileRows * pairs) {
          const int row = q / pairs, k = 2 * (q - row * pairs);
          const float fa = d0.scale * a[u], fb = d0.scale * b[u];
          const uint32_t hi = pack_bf16x2(fa, fb);
          const uint32_t lo = pack_bf16x2(fa - bf16lo(hi), fb - bf16hi(hi));
          const uint32_t off = sw128(row, k >> 3) + (uint32_t)((k & 7) * 2);
          sts32(v_hi + off, hi);
          sts32(v_lo + off, lo);
        }
      }
    }
  }

  for (int kc = 0; kc < nchunks; ++kc) {
    issue_y(kc);          // (the previous chunk's tile was stored and all warps passed a barrier since)
    cp_async_wait<1>();   // this thread's copies of B chunk kc have landed (the y tile may still be on its way)
    __syncthreads();      // ... everybody's; and the MMAs of chunk kc - 1 were waited for by every thread
    // transpose staging [k][128 columns] into the K-major operand [column][k]:
    // a transposed 8x8 block gives lane (g, t) the pair (k0 + 2t, k0 + 2t + 1) of column n0 + g
    {
      const int g = lane >> 2, t = lane & 3;
      for (int blk = warp; blk < (k_mma / 8) * (kExpChunk / 32); blk += kThreads / 32) {
        const int kb = blk / (kExpChunk / 32), nb = blk % (kExpChunk / 32);   // 8 ranks x 32 columns
        uint32_t q4[4];
        // matrix i of the x4 = columns nb*32 + 8 i .. + 7; lane L gives the address of row L % 8 of matrix L / 8
        ldmatrix_x4_trans(q4, stage + (uint32_t)((kb * 8 + (lane & 7)) * kStageRowBytes + (nb * 32 + (lane >> 3) * 8) * 2));
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const int n = nb * 32 + i * 8 + g;
          sts32(b_km + sw128(n, kb) + (uint32_t)(t * 4), q4[i]);
        }
      }
    }
    fence_async_smem();   // the operand writes are visible to the tensor core
    __syncthreads();      // the staging buffer has been read by everybody
    issue_b(kc + 1);
    if (tid == 0 && !failed) {
      tc_fence_after();
      const uint64_t dh = smem_desc_k_sw128(v_hi), dl = smem_desc_k_sw128(v_lo), db = smem_desc_k_sw128(b_km);
      for (int ks = 0; ks < k_mma / 16; ++ks) umma_bf16(tmem_d, dh + (uint64_t)(2 * ks), db + (uint64_t)(2 * ks), idesc, ks > 0);
      for (int ks = 0; ks < k_mma / 16; ++ks) umma_bf16(tmem_d, dl + (uint64_t)(2 * ks), db + (uint64_t)(2 * ks), idesc, true);
      umma_commit(&mma_done);
    }
    cp_async_wait<1>();   // this thread's copies of the y tile have landed (B chunk kc + 1 may still be on its way)
    if (!failed && !mbar_wait(&mma_done, (uint32_t)(kc & 1))) failed = 1;
    tc_fence_after();
    __syncthreads();      // everybody's copies of the y tile have landed
    const int col0 = col_begin + kc * kExpChunk;
    if (!__any_sync(0xffffffffu, failed != 0)) {   // the accumulator loads are warp-wide
      // this thread's row of the tile: y += accumulator
      const uint32_t yr = ytile + (uint32_t)(tid * kYRowBytes);
#pragma unroll
      for (int j0 = 0; j0 < kExpChunk; j0 += 16) {
        float acc[16];
        tmem_ld16(tmem_d + ((uint32_t)(warp * 32) << 16) + (uint32_t)j0, acc);
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          float f[8];
          unpack8(lds128(yr + (uint32_t)((j0 + 8 * h) * 2)), f);
#pragma unroll
          for (int e = 0; e < 8; ++e) f[e] += acc[8 * h + e];
          sts128(yr + (uint32_t)((j0 + 8 * h) * 2), pack8(f));
        }
      }
      __syncwarp();
      // the warp's 32 rows go back to memory, two rows (2 x 256 bytes) per instruction
      const int c = lane & 15;
      if (col0 + c * 8 < col_end) {
#pragma unroll 4
        for (int i = 0; i < 16; ++i) {
          const int row = warp * 32 + 2 * i + (lane >> 4);
          if (row < nrows)
            *reinterpret_cast<uint4 *>(pb.y + (int64_t)rows[row] * pb.ldy + col0 + c * 8) =
                lds128(ytile + (uint32_t)(row * kYRowBytes + c * 16));
        }
      }
    }
    tc_fence_before();   // the accumulator reads are done before the next chunk's MMAs overwrite it
    __syncthreads();      // the y tile is free for the next chunk's copies
  }
  cp_async_wait<0>();
  if (failed) {
    // the MMAs of the chunk whose wait ran out may still be under way: give them one more bounded
    // wait before the tensor memory they write is freed
    if (tid == 0) {
      report(P.status, MINT_ERR_TIMEOUT, m);
      umma_commit(&drain);
    }
    mbar_wait(&drain, 0);
  }
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem_d, kExpTmemCols);
}

// ------------------------------------------------------------------------------------
// The same expand for tiles whose tokens are consecutive rows of y (a request's tokens
// usually are), as a pipeline of three roles over the 128-column chunks of the CTA's
// column range.  One thread asks for the tiles of a chunk through tensor maps: B as two
// boxes of 64 ranks x 64 columns, y as two boxes of 128 rows x 64 columns, all in the
// 128-byte-swizzled layout.  B is used as it lies in memory (columns contiguous): its
// shared-memory descriptor names the MN-major layout, so nothing is transposed.  One
// thread issues the MMAs of a chunk as soon as its B has landed, into one of two
// accumulators in tensor memory.  Eight warps add the accumulator to the y tile in shared
// memory (tcgen05.ld, one row x 64 columns per thread) and store its rows themselves when the
// tile is a segment's last, shorter one (the rows beyond it belong to another CTA); a thread
// of a warp of its own hands full tiles to a tensor-map store and returns the buffer when the
// copy engine has read it, so the epilogue warps never wait for a store.  Three buffers of B and y, two accumulators: the loads and the MMAs of chunk
// kc + 1 run under the epilogue of chunk kc.  Every wait is bounded.
constexpr int kEpiThreads = 256;                   // 8 epilogue warps: warp w takes rows 32 (w % 4) .., columns 64 (w / 4) .. of a chunk
constexpr int kTmaThreads = kEpiThreads + 96;      // + the producer's warp, the MMA warp and the warp that stores
constexpr int kBHalfBytes = kMaxRank * 128;        // 64 ranks x 64 columns
constexpr int kBBufBytes = 2 * kBHalfBytes;        // 16 KB
constexpr int kYHalfBytes = kTileRows * 128;       // 128 rows x 64 columns
constexpr int kYBufBytes = 2 * kYHalfBytes;        // 32 KB
constexpr int kBufs = 4;                            // chunks whose B and y tiles are in shared memory at a time
constexpr size_t kTmaDynSmem = 2 * kVBytes + kBufs * kBBufBytes + kBufs * kYBufBytes + 1024;
constexpr int kTmaTmemCols = 256;                  // two accumulators of 128 columns


__global__ void __launch_bounds__(kTmaThreads, 1) dense_expand_tma_kernel(const __grid_constant__ DenseExpandParams P) {
  extern __shared__ uint8_t dyn_raw[];
  __shared__ uint64_t b_full[kBufs], b_free[kBufs];   // B of a chunk has landed / its MMAs have read it
  __shared__ uint64_t y_full[kBufs], y_free[kBufs];   // the y tile has landed / has gone back to memory
  __shared__ uint64_t acc_full[2], acc_free[2];   // the chunk's MMAs are complete / the accumulator has been read
  __shared__ uint64_t y_written[kBufs];           // every epilogue thread has updated (and, for short tiles, stored) its row
  __shared__ uint64_t drain;
  __shared__ uint32_t tmem_base_slot;
  __shared__ volatile int32_t failed;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  int col_begin, col_end;
  const DenseExpandProblem &pb = P.prob[expand_range(P, (int)blockIdx.y, col_begin, col_end)];

  pdl_launch_dependents();
  const bool ok = plan_ok(P.pv.header, P.T, 1, P.tab.num_slots, 0, P.tab.gen_lo, P.tab.gen_hi, nullptr) &&
                  P.pv.header[PH_LANES] == P.lanes;
  const int m = blockIdx.x;
  if (!ok || !pb.use_tma || m >= P.pv.header[PH_NUM_DENSE] || col_begin >= pb.n) {
    pdl_wait();
    return;
  }
  const int ntiles = P.pv.header[PH_NCHUNK1];
  const int t0 = P.pv.dense_tile[m];
  if (t0 < 0) {   // its tokens are scattered: the other kernel's
    pdl_wait();
    return;
  }
  const TileDesc d0 = P.pv.tile_desc[t0];
  int nrows = d0.len;
  {
    TileDesc dn[3];   // the three descriptors that may follow, requested together
#pragma unroll
    for (int i = 1; i < 4; ++i) dn[i - 1] = P.pv.tile_desc[min(t0 + i, ntiles - 1)];
#pragma unroll
    for (int i = 1; i < 4; ++i) {
      const TileDesc &di = dn[i - 1];
      if (nrows != 32 * i || t0 + i >= ntiles || !di.dense || di.slot != d0.slot || di.off != d0.off + 32 * i) break;
      nrows += di.len;
    }
  }
  const int r = d0.rank;
  const int row0 = P.pv.perm[d0.off];
  if (r > pb.r_max || r > kMaxRank || r < 1) {   // reported by the shrink
    pdl_wait();
    return;
  }
  const int k_mma = (r + 15) / 16 * 16;
  if (tid == 0) {
    for (int b = 0; b < kBufs; ++b) {
      mbar_init(&b_full[b], 1);
      mbar_init(&b_free[b], 1);
      mbar_init(&y_full[b], 1);
      mbar_init(&y_free[b], 1);
      mbar_init(&y_written[b], kEpiThreads);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(&acc_full[b], 1);
      mbar_init(&acc_free[b], kEpiThreads);
    }
    mbar_init(&drain, 1);
    fence_mbar_init();
    failed = 0;
  }
  if (warp == 0) tmem_alloc(&tmem_base_slot, kTmaTmemCols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_d = tmem_base_slot;
  const uint32_t base = (smem_addr(dyn_raw) + 1023u) & ~1023u;
  const uint32_t v_hi = base, v_lo = base + kVBytes;
  const uint32_t b_buf = base + 2 * kVBytes, y_buf = b_buf + kBufs * kBBufBytes;
  const int nchunks = (col_end - col_begin + kExpChunk - 1) / kExpChunk;
  const bool full_tile = nrows == kTileRows;   // (the tile's 128 rows are all this CTA's: whole boxes may be stored)

  pdl_wait();   // v and y belong to the earlier kernels until here

  if (warp == kEpiThreads / 32) {
    // ---- producer ----
    if (lane == 0) {
      int kc = 0;
      for (; kc < nchunks; ++kc) {
        const int b = kc % kBufs;
        const uint32_t par = ((kc / kBufs) & 1u) ^ 1u;   // (the buffers start out free)
        const int col = col_begin + kc * kExpChunk;
        if (!mbar_wait(&b_free[b], par)) { failed = 1; break; }
        mbar_arrive_expect_tx(&b_full[b], (uint32_t)kBBufBytes);
        tma_load_2d(b_buf + (uint32_t)(b * kBBufBytes), &pb.b_map, col, d0.slot * pb.r_max, &b_full[b]);
        tma_load_2d(b_buf + (uint32_t)(b * kBBufBytes + kBHalfBytes), &pb.b_map, col + 64, d0.slot * pb.r_max, &b_full[b]);
        if (!mbar_wait(&y_free[b], par)) { failed = 1; break; }
        mbar_arrive_expect_tx(&y_full[b], (uint32_t)kYBufBytes);
        tma_load_2d(y_buf + (uint32_t)(b * kYBufBytes), &pb.y_map, col, row0, &y_full[b]);
        tma_load_2d(y_buf + (uint32_t)(b * kYBufBytes + kYHalfBytes), &pb.y_map, col + 64, row0, &y_full[b]);
      }
      if (failed)   // the tiles still on their way land before this CTA's memory goes away
        for (int j = max(0, kc - kBufs); j < kc; ++j) {
          mbar_wait(&b_full[j % kBufs], (j / kBufs) & 1u, 100000000ull);
          mbar_wait(&y_full[j % kBufs], (j / kBufs) & 1u, 100000000ull);
        }
    }
    __syncwarp();
  } else if (warp == kEpiThreads / 32 + 1) {
    // ---- MMA issuer (the whole warp clears the rank rows beyond the slot's rank first) ----
    const uint32_t idesc = instr_desc_b_mn(kExpChunk);
    for (int kc = 0; kc < nchunks; ++kc) {
      const int b = kc % kBufs, ab = kc & 1;                          // buffer of B, accumulator
      const uint32_t par = (kc / kBufs) & 1u, apar = (kc >> 1) & 1u;
      bool good = mbar_wait(&b_full[b], par);
      const uint32_t bs = b_buf + (uint32_t)(b * kBBufBytes);
      if (good && r < k_mma) {
        // rows r .. k_mma - 1 of the boxes are whatever follows the slot's rows in the pool: v is zero
        // there, but zero times a NaN is not
        for (int q = lane; q < (k_mma - r) * 16; q += 32) {
          const int row = r + (q >> 4), c = q & 15;
          sts128(bs + (uint32_t)((c >> 3) * kBHalfBytes) + sw128(row, c & 7), make_uint4(0u, 0u, 0u, 0u));
        }
        fence_async_smem();
      }
      __syncwarp();
      if (lane == 0) {
        good = good && mbar_wait(&acc_free[ab], apar);   // (phase 0 of it: v is in place)
        if (!good) failed = 1;
        else {
          tc_fence_after();
          const uint32_t acc = tmem_d + (uint32_t)(ab * kExpChunk);
          const uint64_t dh = smem_desc_k_sw128(v_hi), dl = smem_desc_k_sw128(v_lo);
          const uint64_t db = smem_desc_mn_sw128(bs, (uint32_t)kBHalfBytes);
          // a step of 16 ranks: 32 bytes further along v's rows, two 8-row groups further down B
          for (int ks = 0; ks < k_mma / 16; ++ks)
            umma_bf16(acc, dh + (uint64_t)(2 * ks), db + (uint64_t)(128 * ks), idesc, ks > 0);
          for (int ks = 0; ks < k_mma / 16; ++ks)
            umma_bf16(acc, dl + (uint64_t)(2 * ks), db + (uint64_t)(128 * ks), idesc, true);
          umma_commit(&acc_full[ab]);
          umma_commit(&b_free[b]);
        }
      }
      __syncwarp();
      if (failed) break;
    }
    if (lane == 0 && failed) {   // whatever was issued is complete (or given up on once more) before tensor memory is freed
      umma_commit(&drain);
      mbar_wait(&drain, 0);
    }
    __syncwarp();
  } else if (warp == kEpiThreads / 32 + 2) {
    // ---- storing thread: a finished y tile goes back through the tensor map, and its buffer is handed
    // back once the copy engine has read it (the epilogue warps are on the next chunk meanwhile) ----
    if (lane == 0) {
      for (int kc = 0; kc < nchunks; ++kc) {
        const int b = kc % kBufs;
        const uint32_t par = (kc / kBufs) & 1u;
        if (!mbar_wait(&y_written[b], par)) {
          failed = 1;
          break;
        }
        if (full_tile) {   // (columns beyond n are clipped by the tensor map; short tiles were stored row by row)
          const int col0 = col_begin + kc * kExpChunk;
          const uint32_t yb = y_buf + (uint32_t)(b * kYBufBytes);
          tma_store_2d(&pb.y_map, col0, row0, yb);
          tma_store_2d(&pb.y_map, col0 + 64, row0, yb + (uint32_t)kYHalfBytes);
          bulk_commit();
          bulk_wait_read();   // the tile has been read: the buffer may be refilled
        }
        mbar_arrive(&y_free[b]);
      }
      bulk_wait_all();   // the stores are complete before the kernel ends
    }
    __syncwarp();
  } else {
    // ---- epilogue warps; first v, scaled, as head and remainder (consecutive threads: consecutive rank pairs of a row) ----
    {
      const size_t slot_floats = (size_t)32 * pb.r_max;
      const int pairs = k_mma / 2;
      for (int q0 = tid; q0 < kTileRows * pairs; q0 += 8 * kEpiThreads) {
        float a[8], b[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) a[u] = b[u] = 0.f;
        for (int sp = 0; sp < pb.splits; ++sp) {   // the parts of the shrink's CTAs, in their order; 16 loads go out together
          float pa[8], pbv[8];
#pragma unroll
          for (int u = 0; u < 8; ++u) {
            const int q = q0 + u * kEpiThreads;
            const int row = q / pairs, k = 2 * (q - row * pairs);
            const bool in = q < kTileRows * pairs && row < nrows;
            const float *src = pb.ws_part + (size_t)(P.dense_slot0 + sp * P.dense_stride + t0 + (row >> 5)) * slot_floats +
                               (size_t)(row & 31) * r;
            pa[u] = (in && k < r) ? __ldcg(src + k) : 0.f;
            pbv[u] = (in && k + 1 < r) ? __ldcg(src + k + 1) : 0.f;
          }
#pragma unroll
          for (int u = 0; u < 8; ++u) {
            a[u] += pa[u];
            b[u] += pbv[u];
          }
        }
#pragma unroll
        for (int u = 0; u < 8; ++u) {
          const int q = q0 + u * kEpiThreads;
          if (q < kTileRows * pairs) {
            const int row = q / pairs, k = 2 * (q - row * pairs);
            const float fa = d0.scale * a[u], fb = d0.scale * b[u];
            const uint32_t hi = pack_bf16x2(fa, fb);
            const uint32_t lo = pack_bf16x2(fa - bf16lo(hi), fb - bf16hi(hi));
            const uint32_t off = sw128(row, k >> 3) + (uint32_t)((k & 7) * 2);
            sts32(v_hi + off, hi);
            sts32(v_lo + off, lo);
          }
        }
      }
      fence_async_smem();   // the operand writes are visible to the tensor core
      // (accumulator 0 and 1 are "read" before their first use: this arrival also tells the MMA thread that v is in place)
      mbar_arrive(&acc_free[0]);
      mbar_arrive(&acc_free[1]);
    }
    for (int kc = 0; kc < nchunks; ++kc) {
      const int b = kc % kBufs, ab = kc & 1;
      const uint32_t par = (kc / kBufs) & 1u, apar = (kc >> 1) & 1u;
      if (!mbar_wait(&acc_full[ab], apar) || !mbar_wait(&y_full[b], par)) {
        failed = 1;
        break;
      }
      tc_fence_after();
      const int col0 = col_begin + kc * kExpChunk;
      const uint32_t yb = y_buf + (uint32_t)(b * kYBufBytes);
      // this thread's row of its half of the tile (64 columns): y += accumulator; the four loads of
      // tensor memory go out together
      const int row = (warp & 3) * 32 + lane, half = warp >> 2;
      const uint32_t yh = yb + (uint32_t)(half * kYHalfBytes);
      {
        uint32_t acc[4][16];
#pragma unroll
        for (int q = 0; q < 4; ++q)
          tmem_ld16_issue(tmem_d + ((uint32_t)((warp & 3) * 32) << 16) + (uint32_t)(ab * kExpChunk + half * 64 + q * 16), acc[q]);
        tmem_ld_wait();
#pragma unroll
        for (int q = 0; q < 4; ++q)
#pragma unroll
          for (int h = 0; h < 2; ++h) {
            const uint32_t addr = yh + sw128(row, 2 * q + h);
            float f[8];
            unpack8(lds128(addr), f);
#pragma unroll
            for (int e = 0; e < 8; ++e) f[e] += __uint_as_float(acc[q][8 * h + e]);
            sts128(addr, pack8(f));
          }
      }
      tc_fence_before();
      mbar_arrive(&acc_free[ab]);   // the accumulator may be overwritten
      if (!full_tile) {
        // a short tile: the warp's rows of its half go back to memory row by row (four rows per instruction)
        __syncwarp();
        const int c = lane & 7;
        if (col0 + half * 64 + c * 8 < col_end) {
#pragma unroll 4
          for (int i = 0; i < 8; ++i) {
            const int rr = (warp & 3) * 32 + 4 * i + (lane >> 3);
            if (rr < nrows)
              *reinterpret_cast<uint4 *>(pb.y + (int64_t)(row0 + rr) * pb.ldy + col0 + half * 64 + c * 8) =
                  lds128(yh + sw128(rr, c));
          }
        }
      }
      fence_async_smem();   // this thread's writes to the tile are visible to the store of the storing warp
      mbar_arrive(&y_written[b]);
    }
  }
  __syncthreads();
  if (failed && tid == 0) report(P.status, MINT_ERR_TIMEOUT, m);
  tc_fence_after();
  if (warp == 0) tmem_dealloc(tmem_d, kTmaTmemCols);
}

}  // namespace

int32_t mint_launch_dense_shrink(const DenseArgs *args, int nprob, const TableDev &tab, const void *plan_dev,
                                 void *const *workspaces, int32_t lanes, int32_t dense_slot0, int32_t dense_stride,
                                 cudaStream_t s, bool withhold_for_selftest) {
  static bool attr_set = false;
  if (!attr_set) {
    int32_t st = mint_check_cuda(cudaFuncSetAttribute(dense_shrink_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                      (int)kDynSmem), "dense_shrink shared memory");
    if (st) return st;
    attr_set = true;
  }
  const int32_t T = args[0].T;
  // 128-row tiles of dense segments: a segment of len tokens has at most len / 128 + 1, and there are at
  // most min(slots, T / 128) dense segments
  const int64_t tiles = (int64_t)(T / MINT_DENSE_MIN_SEGMENT) +
                        std::min<int64_t>(tab.num_slots, T / MINT_DENSE_MIN_SEGMENT);
  if (tiles == 0) return MINT_OK;
  DenseParams P = {};
  int32_t shares = 0;
  for (int i = 0; i < nprob; ++i) {
    DenseProblem &pb = P.prob[i];
    pb.A = args[i].A;
    pb.x = args[i].x;
    pb.ldx = args[i].ldx;
    pb.d = args[i].d;
    pb.r_max = args[i].r_max;
    pb.splits = mint_dense_splits(args[i].d);
    shares += pb.splits;
    pb.ws_part = static_cast<float *>(workspaces[i]);
    pb.use_tma = make_map_2d(&pb.x_map, args[i].x, (uint64_t)T, (uint64_t)args[i].d, (uint64_t)args[i].ldx, kTileRows) &&
                 make_map_2d(&pb.a_map, args[i].A, (uint64_t)args[i].num_slots * args[i].r_max, (uint64_t)args[i].d,
                             (uint64_t)args[i].d, kMaxRank);
  }
  P.nprob = nprob;
  P.T = T;
  P.lanes = lanes;
  P.dense_slot0 = dense_slot0;
  P.dense_stride = dense_stride;
  P.withhold = withhold_for_selftest ? 1 : 0;
  P.wait_ns = withhold_for_selftest ? 2000000ull : kWaitLimitNs;   // the self-test gives up after 2 ms
  P.status = args[0].status;
  P.tab = tab;
  P.pv = mint_plan_view(plan_dev, T, tab.num_slots);
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)tiles, (unsigned)shares);
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = kDynSmem;
  cfg.stream = s;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return mint_check_cuda(cudaLaunchKernelEx(&cfg, dense_shrink_kernel, P), "dense_shrink launch");
}


int32_t mint_launch_dense_expand(const DenseArgs *args, int nprob, const TableDev &tab, const void *plan_dev,
                                 void *const *workspaces, int32_t lanes, int32_t dense_slot0, int32_t dense_stride,
                                 cudaStream_t s) {
  static bool attr_set = false;
  if (!attr_set) {
    int32_t st = mint_check_cuda(cudaFuncSetAttribute(dense_expand_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                      (int)kExpDynSmem), "dense_expand shared memory");
    if (st) return st;
    st = mint_check_cuda(cudaFuncSetAttribute(dense_expand_tma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                              (int)kTmaDynSmem), "dense_expand (tensor maps) shared memory");
    if (st) return st;
    attr_set = true;
  }
  const int32_t T = args[0].T;
  // 128-row tiles of dense segments: a segment of len tokens has at most len / 128 + 1, and there are at
  // most min(slots, T / 128) dense segments
  const int64_t tiles = (int64_t)(T / MINT_DENSE_MIN_SEGMENT) +
                        std::min<int64_t>(tab.num_slots, T / MINT_DENSE_MIN_SEGMENT);
  if (tiles == 0) return MINT_OK;
  DenseExpandParams P = {};
  int32_t ranges = 0;
  bool any_tma = false;
  for (int i = 0; i < nprob; ++i) {
    DenseExpandProblem &pb = P.prob[i];
    pb.B = args[i].B;
    pb.y = args[i].y;
    pb.ldy = args[i].ldy;
    pb.n = args[i].n;
    pb.r_max = args[i].r_max;
    pb.splits = mint_dense_splits(args[i].d);
    pb.ws_part = static_cast<const float *>(workspaces[i]);
    pb.use_tma = make_map_2d(&pb.b_map, args[i].B, (uint64_t)args[i].num_slots * args[i].r_max, (uint64_t)args[i].n,
                             (uint64_t)args[i].n, kMaxRank) &&
                 make_map_2d(&pb.y_map, args[i].y, (uint64_t)T, (uint64_t)args[i].n, (uint64_t)args[i].ldy, kTileRows);
    any_tma = any_tma || pb.use_tma;
    ranges += (pb.n + kColsPerCta - 1) / kColsPerCta;
  }
  P.nprob = nprob;
  P.T = T;
  P.lanes = lanes;
  P.dense_slot0 = dense_slot0;
  P.dense_stride = dense_stride;
  P.status = args[0].status;
  P.tab = tab;
  P.pv = mint_plan_view(plan_dev, T, tab.num_slots);
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)tiles, (unsigned)ranges);
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = kExpDynSmem;
  cfg.stream = s;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  int32_t st = mint_check_cuda(cudaLaunchKernelEx(&cfg, dense_expand_kernel, P), "dense_expand launch");
  if (st || !any_tma) return st;
  // the tiles of consecutive tokens: same grid, six warps, one CTA per SM
  cfg.blockDim = dim3(kTmaThreads);
  cfg.dynamicSmemBytes = kTmaDynSmem;
  return mint_check_cuda(cudaLaunchKernelEx(&cfg, dense_expand_tma_kernel, P), "dense_expand (tensor maps) launch");
}
