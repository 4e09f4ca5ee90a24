// Dense-projection LoRA kernels on CUDA cores: shrink, expand and the fused
// apply for batches where most adapters own only a few tokens (decode).
//
//   shrink   v[t, :r] = x[t, :] . A_slot            (d -> r)
//   expand   y[t, :] += s_slot * v[t, :r] . B_slot   (r -> n)
//   fused    both in one launch; v stays in shared memory
//
// Work unit: one tile of the plan's list 0 (at most 8 tokens of one segment).
// In the fused kernel a thread-block cluster of C CTAs owns one tile: CTA c
// shrinks over the c-th part of d, the partial results are exchanged through
// distributed shared memory (plain remote shared-memory reads, no multicast),
// and CTA c then expands into the c-th part of n.  Every byte of x, A, B and y
// is therefore fetched from HBM once per tile and nothing is recomputed.
#include <cooperative_groups.h>

#include "tile_ops.cuh"

namespace cg = cooperative_groups;
using namespace mint;

namespace {

struct TileInfo {
  int len, slot, r;
  float scale;
};

// Loads the tile's rows into shared memory; returns false when the tile index
// is past the plan's tile count or the slot's rank does not fit the pool.
__device__ __forceinline__ bool load_tile(const PlanView &pv, const TableDev &tab, int tile, int r_max,
                                          int32_t *status, TileSmem &sm, TileInfo &ti) {
  if (tile >= pv.header[PH_NCHUNK0]) return false;
  const int seg = pv.tile_seg[0][tile];
  const int off = pv.tile_off[0][tile];
  ti.len = min(kTileRows, pv.seg_start[seg + 1] - off);
  ti.slot = pv.seg_slot[seg];
  ti.r = tab.slot_rank[ti.slot];
  ti.scale = tab.slot_scale[ti.slot];
  if (ti.r > r_max || ti.r > kRankCap) {
    if (threadIdx.x == 0) report(status, MINT_ERR_RANK_TOO_LARGE, ti.slot);
    return false;
  }
  if (threadIdx.x < kTileRows) {
    const int l = threadIdx.x;
    const int row = pv.perm[off + (l < ti.len ? l : 0)];
    sm.row_x[l] = row;
    sm.row_y[l] = l < ti.len ? row : -1;
    sm.scale[l] = ti.scale;
  }
  return true;
}

__device__ __forceinline__ int rows_bucket(int len) { return len <= 1 ? 1 : (len <= 2 ? 2 : (len <= 4 ? 4 : 8)); }

__device__ __forceinline__ void shrink_dispatch(const uint16_t *A_slot, int d, int r, const uint16_t *x,
                                                int64_t ldx, TileSmem &sm, int len, int v0, int v1,
                                                float *out, int r_stride) {
  switch (rows_bucket(len)) {
    case 1: shrink_tile_rd<1>(A_slot, d, r, x, ldx, sm, v0, v1, out, r_stride); break;
    case 2: shrink_tile_rd<2>(A_slot, d, r, x, ldx, sm, v0, v1, out, r_stride); break;
    case 4: shrink_tile_rd<4>(A_slot, d, r, x, ldx, sm, v0, v1, out, r_stride); break;
    default: shrink_tile_rd<8>(A_slot, d, r, x, ldx, sm, v0, v1, out, r_stride); break;
  }
}

__device__ __forceinline__ void expand_dispatch(const uint16_t *B_slot, int n, int r, const float *vs,
                                                int r_stride, uint16_t *y, int64_t ldy,
                                                const TileSmem &sm, int len, int v0, int v1) {
  switch (rows_bucket(len)) {
    case 1: expand_tile<1>(B_slot, n, r, vs, r_stride, y, ldy, sm, v0, v1); break;
    case 2: expand_tile<2>(B_slot, n, r, vs, r_stride, y, ldy, sm, v0, v1); break;
    case 4: expand_tile<4>(B_slot, n, r, vs, r_stride, y, ldy, sm, v0, v1); break;
    default: expand_tile<8>(B_slot, n, r, vs, r_stride, y, ldy, sm, v0, v1); break;
  }
}

__global__ void __launch_bounds__(kTileThreads) shrink_kernel(const DenseArgs a, const TableDev tab,
                                                             const PlanView pv) {
  __shared__ TileSmem sm;
  if (!plan_ok(pv.header, a.T, 1, tab.num_slots, 0, tab.gen_lo, tab.gen_hi, a.status)) return;
  TileInfo ti;
  if (!load_tile(pv, tab, blockIdx.x, a.r_max, a.status, sm, ti)) return;
  __syncthreads();
  const int r_stride = a.r_max;
  shrink_dispatch(a.A + (int64_t)ti.slot * a.r_max * a.d, a.d, ti.r, a.x, a.ldx, sm, ti.len, 0,
                  a.d >> 3, sm.vs, r_stride);
  for (int i = threadIdx.x; i < ti.len * ti.r; i += kTileThreads) {
    const int l = i / ti.r, j = i - l * ti.r;
    a.v[(int64_t)sm.row_y[l] * a.r_max + j] = sm.vs[l * r_stride + j];
  }
}

__global__ void __launch_bounds__(kTileThreads) expand_kernel(const DenseArgs a, const TableDev tab,
                                                             const PlanView pv) {
  __shared__ TileSmem sm;
  if (!plan_ok(pv.header, a.T, 1, tab.num_slots, 0, tab.gen_lo, tab.gen_hi, a.status)) return;
  TileInfo ti;
  if (!load_tile(pv, tab, blockIdx.x, a.r_max, a.status, sm, ti)) return;
  __syncthreads();
  const int r_stride = a.r_max;
  for (int i = threadIdx.x; i < kTileRows * ti.r; i += kTileThreads) {
    const int l = i / ti.r, j = i - l * ti.r;
    sm.vs[l * r_stride + j] = l < ti.len ? a.v[(int64_t)sm.row_x[l] * a.r_max + j] : 0.f;
  }
  __syncthreads();
  const int nv = a.n >> 3;
  const int v0 = (int)((int64_t)nv * blockIdx.y / gridDim.y);
  const int v1 = (int)((int64_t)nv * (blockIdx.y + 1) / gridDim.y);
  expand_dispatch(a.B + (int64_t)ti.slot * a.r_max * a.n, a.n, ti.r, sm.vs, r_stride, a.y, a.ldy, sm,
                  ti.len, v0, v1);
}

__global__ void __launch_bounds__(kTileThreads) fused_kernel(const DenseArgs a, const TableDev tab,
                                                            const PlanView pv) {
  __shared__ TileSmem sm;
  cg::cluster_group cluster = cg::this_cluster();
  const int C = (int)cluster.num_blocks();
  const int crank = (int)cluster.block_rank();
  // Every CTA of a cluster takes the same early exits: they depend only on the
  // plan header and on the tile index, which the whole cluster shares.
  if (!plan_ok(pv.header, a.T, 1, tab.num_slots, 0, tab.gen_lo, tab.gen_hi, a.status)) return;
  TileInfo ti;
  if (!load_tile(pv, tab, blockIdx.x / C, a.r_max, a.status, sm, ti)) return;
  __syncthreads();
  const int r_stride = ti.r;
  const int dv = a.d >> 3;
  const int d0 = (int)((int64_t)dv * crank / C), d1 = (int)((int64_t)dv * (crank + 1) / C);
  shrink_dispatch(a.A + (int64_t)ti.slot * a.r_max * a.d, a.d, ti.r, a.x, a.ldx, sm, ti.len, d0, d1,
                  sm.vpart, r_stride);
  const int cnt = rows_bucket(ti.len) * ti.r;
  if (C > 1) {
    cluster.sync();  // every CTA's partial is complete and visible cluster-wide
    for (int i = threadIdx.x; i < cnt; i += kTileThreads) {
      float s = 0.f;
      for (int q = 0; q < C; ++q) s += cluster.map_shared_rank(sm.vpart, q)[i];
      sm.vs[i] = s;
    }
    cluster.sync();  // no CTA leaves (or reuses vpart) while a peer still reads it
  } else {
    for (int i = threadIdx.x; i < cnt; i += kTileThreads) sm.vs[i] = sm.vpart[i];
    __syncthreads();
  }
  const int nv = a.n >> 3;
  const int n0 = (int)((int64_t)nv * crank / C), n1 = (int)((int64_t)nv * (crank + 1) / C);
  expand_dispatch(a.B + (int64_t)ti.slot * a.r_max * a.n, a.n, ti.r, sm.vs, r_stride, a.y, a.ldy, sm,
                  ti.len, n0, n1);
}

int pick_cluster(int64_t tiles_ub) {
  // Enough CTAs to cover the 148 SMs a few times over; few tiles -> wide clusters.
  if (tiles_ub >= 1024) return 1;
  if (tiles_ub >= 512) return 2;
  if (tiles_ub >= 192) return 4;
  return 8;
}

}  // namespace

int32_t mint_launch_shrink(const DenseArgs &a, const TableDev &tab, const void *plan_dev, cudaStream_t s) {
  const int64_t ub = mint_tile_upper_bound(0, a.T, tab.num_slots);
  if (ub == 0) return MINT_OK;
  shrink_kernel<<<(unsigned)ub, kTileThreads, 0, s>>>(a, tab, mint_plan_view(plan_dev, a.T, tab.num_slots));
  return mint_check_cuda(cudaGetLastError(), "shrink kernel launch");
}

int32_t mint_launch_expand(const DenseArgs &a, const TableDev &tab, const void *plan_dev, cudaStream_t s) {
  const int64_t ub = mint_tile_upper_bound(0, a.T, tab.num_slots);
  if (ub == 0) return MINT_OK;
  int ny = 1;
  while (ub * ny < 592 && ny < 16 && (a.n >> 3) / (ny * 2) >= 32) ny *= 2;
  expand_kernel<<<dim3((unsigned)ub, ny), kTileThreads, 0, s>>>(a, tab, mint_plan_view(plan_dev, a.T, tab.num_slots));
  return mint_check_cuda(cudaGetLastError(), "expand kernel launch");
}

int32_t mint_launch_fused(const DenseArgs &a, const TableDev &tab, const void *plan_dev, cudaStream_t s) {
  const int64_t ub = mint_tile_upper_bound(0, a.T, tab.num_slots);
  if (ub == 0) return MINT_OK;
  int C = pick_cluster(ub);
  while (C > 1 && ((a.d >> 3) / C < 32 || (a.n >> 3) / C < 32)) C >>= 1;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)(ub * C));
  cfg.blockDim = dim3(kTileThreads);
  cfg.dynamicSmemBytes = 0;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = C;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  const PlanView pv = mint_plan_view(plan_dev, a.T, tab.num_slots);
  return mint_check_cuda(cudaLaunchKernelEx(&cfg, fused_kernel, a, tab, pv), "fused kernel launch");
}
