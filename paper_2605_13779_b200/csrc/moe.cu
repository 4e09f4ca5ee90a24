// MoE expert LoRA apply over the packed layout A[slot][expert][d][r_max],
// B[slot][expert][r_max][n].
//
// Per-expert LoRA tensors are keyed by expert id (paper, section "Scale Up",
// Megatron placement) and stacked along an expert axis in the packed serving
// representation.  For pair p = t*K + k with expert e and slot sigma:
//     Y[p, :] += s_sigma * w_p * (X[row(p), :] . A[sigma][e]) . B[sigma][e]
// The plan groups pairs by (expert, slot); a tile (at most 8 pairs of one
// group) is one CTA's work: shrink in two halves of 4 rows, then expand.
#include "tile_ops.cuh"

using namespace mint;

namespace {

template <int LC>
__device__ __forceinline__ void moe_half(const MoEArgs &a, const uint16_t *A_e, const uint16_t *B_e,
                                         int r, TileSmem &sm, int r_stride) {
  shrink_tile_dr<LC>(A_e, a.r_max, r, a.x, a.ldx, sm, 0, a.d, sm.vs, r_stride);
  expand_tile<LC>(B_e, a.n, r, sm.vs, r_stride, a.y, a.ldy, sm, 0, a.n >> 3);
}

__global__ void __launch_bounds__(kTileThreads) moe_kernel(const MoEArgs a, const TableDev tab,
                                                          const PlanView pv) {
  __shared__ TileSmem sm;
  if (!plan_ok(pv.header, a.T, a.K, tab.num_slots, a.num_experts, tab.gen_lo, tab.gen_hi, a.status))
    return;
  const int tile = blockIdx.x;
  if (tile >= pv.header[PH_NCHUNK0]) return;
  const int seg = pv.tile_seg[0][tile];
  const int off = pv.tile_off[0][tile];
  const int len = min(kTileRows, pv.seg_start[seg + 1] - off);
  const int slot = pv.seg_slot[seg];
  const int expert = pv.seg_expert[seg];
  const int r = tab.slot_rank[slot];
  const float scale = tab.slot_scale[slot];
  if (r > a.r_max || r > kRankCap) {
    if (threadIdx.x == 0) report(a.status, MINT_ERR_RANK_TOO_LARGE, slot);
    return;
  }
  const uint16_t *A_e = a.A + ((int64_t)slot * a.num_experts + expert) * (int64_t)a.d * a.r_max;
  const uint16_t *B_e = a.B + ((int64_t)slot * a.num_experts + expert) * (int64_t)a.r_max * a.n;
  const int r_stride = r;
  for (int h = 0; h < len; h += 4) {
    const int hl = min(4, len - h);
    __syncthreads();
    if (threadIdx.x < 4) {
      const int l = threadIdx.x;
      const int p = pv.perm[off + h + (l < hl ? l : 0)];
      int64_t row = a.x_row ? (int64_t)a.x_row[p] : (int64_t)p;
      bool ok = l < hl;
      if (row < 0 || row >= a.x_rows) {
        if (ok) report(a.status, MINT_ERR_BAD_INDEX, p);
        row = 0;
        ok = false;
      }
      sm.row_x[l] = (int)row;
      sm.row_y[l] = ok ? p : -1;
      sm.scale[l] = scale * (a.pair_weight ? a.pair_weight[p] : 1.f);
    }
    __syncthreads();
    switch (hl) {
      case 1: moe_half<1>(a, A_e, B_e, r, sm, r_stride); break;
      case 2: moe_half<2>(a, A_e, B_e, r, sm, r_stride); break;
      default: moe_half<4>(a, A_e, B_e, r, sm, r_stride); break;
    }
  }
}

}  // namespace

int32_t mint_launch_moe(const MoEArgs &a, const TableDev &tab, const void *plan_dev, cudaStream_t s) {
  const int64_t P = (int64_t)a.T * a.K;
  const int64_t ub = mint_tile_upper_bound(0, P, (int64_t)tab.num_slots * a.num_experts);
  if (ub == 0) return MINT_OK;
  moe_kernel<<<(unsigned)ub, kTileThreads, 0, s>>>(a, tab, mint_plan_view(plan_dev, P, (int64_t)tab.num_slots * a.num_experts));
  return mint_check_cuda(cudaGetLastError(), "moe kernel launch");
}
