// Streamed LoRA apply for dense projections: the fused path of
// mint_lora_apply_fused and of its grouped form.
//
//   shrink_stream_kernel : v[tile] = X[tile rows, :] . A_slot           (d -> r)
//   expand_stream_kernel : Y[tile rows, :] += s_slot * v[tile] . B_slot  (r -> n)
//
// Work unit = (tile, slice): a tile is at most 32 tokens of one segment (plan
// tile list 1), a slice is a contiguous range of d (shrink) or n (expand)
// sized so that one unit moves a few tens of KB.  Every row of A, B, x and y
// that a unit touches is a contiguous byte range, so a unit streams its rows
// through shared memory with bulk asynchronous copies (cp.async.bulk) tracked
// by mbarriers, three stages deep; HBM latency is hidden by bytes in flight,
// not by registers.  The arithmetic runs on the warp-level tensor-core MMA
// (m16n8k16, bf16 in, fp32 accumulate) with operands fetched by ldmatrix; tiles
// that are both short and of very low rank (rank <= 4, at most 8 tokens) use
// plain fp32 FMAs instead, because padding them to a 16 x 8 MMA tile would
// multiply the shared-memory reads.
//
// The two kernels are launched back to back.  The expand kernel is launched
// with programmatic stream serialization: its CTAs become resident while the
// shrink kernel still runs, start streaming B and y (neither depends on the
// shrink result) and wait (griddepcontrol.wait) only before they read v.
// v travels through a small L2-resident workspace: [tile][32][r_max] fp32.
// When several slices share a tile, each writes its partial sum and the last
// one to finish (an atomic ticket per tile) adds the partials in slice order,
// so the result does not depend on scheduling.
#include <algorithm>

#include "mint_device.cuh"

using namespace mint;

namespace {

constexpr int kThreads = 128;
constexpr int kWarps = 4;
constexpr int kStages = 3;
constexpr int kStageBytes = 14848;          // 64 rows of 108 bf16 + 16 B of row padding
constexpr int kFrontBytes = 8448;           // [32][64] fp32 + 32 floats in front of the stages
constexpr int kDynSmemBytes = kFrontBytes + kStages * kStageBytes;  // 4 CTAs per SM
constexpr int kTileRowsMax = 32;            // plan tile list 1
constexpr int kStreamRankCap = 64;          // larger ranks take the CUDA-core cluster kernel
constexpr int kMaxChunkElems = 2048;
constexpr uint32_t kWaitLimit = 1u << 22;   // polls before a wait gives up

struct StreamProblem {
  const uint16_t *A;   // [slot][r_max][d]
  const uint16_t *B;   // [slot][r_max][n]
  const uint16_t *x;
  uint16_t *y;
  int64_t ldx, ldy;
  int32_t d, n, r_max;
  int32_t shrink_cap, expand_cap;  // most slices a tile may be cut into
  float *ws_v;         // [tiles_ub][32][r_max]
  float *ws_part;      // [tiles_ub][shrink_cap][32][r_max]
  int32_t *ws_ticket;  // [tiles_ub], zero between launches
};

constexpr int kMaxProblems = 8;
struct StreamParams {
  StreamProblem prob[kMaxProblems];
  int32_t T;
  int32_t target_bytes;  // bytes one unit should move
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
__device__ __forceinline__ void mbar_expect_tx(uint64_t *bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr(bar)), "r"(bytes)
               : "memory");
}
// Bounded wait for the phase with the given parity; false when it gave up.
__device__ __forceinline__ bool mbar_wait(uint64_t *bar, uint32_t parity) {
  const uint32_t a = smem_addr(bar);
  for (uint32_t it = 0; it < kWaitLimit; ++it) {
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done)
        : "r"(a), "r"(parity)
        : "memory");
    if (done) return true;
  }
  return false;
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
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void fence_mbar_init() {
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void pdl_launch_dependents() {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

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

// ---- unit geometry -------------------------------------------------------------
struct Unit {
  int len, slot, r, off;
  float scale;
  bool mma;       // tensor-core path (else fp32 FMA path)
  int r_pad;      // rows reserved for weight rows in a stage
  int m_pad;      // rows reserved for activation rows in a stage
  int pitch;      // bytes between rows of a stage
  int cw;         // chunk width in elements
};

__host__ __device__ inline int round_up(int v, int m) { return (v + m - 1) / m * m; }

__host__ __device__ inline int slices_for(int64_t bytes, int units16, int cap, int target_bytes) {
  int64_t s = (bytes + target_bytes - 1) / target_bytes;
  if (s > cap) s = cap;
  if (s > units16) s = units16;
  if (s < 1) s = 1;
  return (int)s;
}

__device__ __forceinline__ bool decode_unit(const StreamParams &P, int tile, int r_max, Unit &u) {
  if (tile >= P.pv.header[PH_NCHUNK1]) return false;
  const int seg = P.pv.tile_seg[1][tile];
  u.off = P.pv.tile_off[1][tile];
  u.len = min(kTileRowsMax, P.pv.seg_start[seg + 1] - u.off);
  u.slot = P.pv.seg_slot[seg];
  u.r = P.tab.slot_rank[u.slot];
  u.scale = P.tab.slot_scale[u.slot];
  if (u.r > r_max || u.r > kStreamRankCap || u.r < 1) {
    if (threadIdx.x == 0) report(P.status, MINT_ERR_RANK_TOO_LARGE, u.slot);
    return false;
  }
  u.mma = !(u.r <= 4 && u.len <= 8);
  u.r_pad = u.mma ? round_up(u.r, 16) : u.r;
  u.m_pad = u.mma ? round_up(u.len, 16) : u.len;
  const int rows = u.r_pad + u.m_pad;
  int cw = ((kStageBytes / rows) - 16) / 2;
  cw = cw / 16 * 16;
  if (cw > kMaxChunkElems) cw = kMaxChunkElems;
  u.cw = cw;                    // >= 32 for rows <= 96
  u.pitch = cw * 2 + 16;
  return true;
}

// Issue the bulk loads of one chunk: weight rows [0, r) then activation rows.
// Called by warp 0; each lane copies the rows lane, lane + 32, ...
__device__ __forceinline__ void issue_chunk(uint8_t *stage, uint64_t *bar, const Unit &u,
                                            const uint16_t *w_slot, int64_t w_ld, const uint16_t *act,
                                            int64_t act_ld, const int *rows, int col0, int width) {
  const int lane = threadIdx.x & 31;
  const uint32_t row_bytes = (uint32_t)width * 2u;
  if (lane == 0) mbar_expect_tx(bar, row_bytes * (uint32_t)(u.r + u.len));
  __syncwarp();
  for (int i = lane; i < u.r + u.len; i += 32) {
    const uint16_t *src;
    uint8_t *dst;
    if (i < u.r) {
      src = w_slot + (int64_t)i * w_ld + col0;
      dst = stage + (size_t)i * u.pitch;
    } else {
      src = act + (int64_t)rows[i - u.r] * act_ld + col0;
      dst = stage + (size_t)(u.r_pad + i - u.r) * u.pitch;
    }
    bulk_load(dst, src, row_bytes, bar);
  }
}

// ================================================================================
// shrink
// ================================================================================
// Tensor-core body: warps split the k-steps of every chunk; each keeps the full
// [MT*16 x NT*8] accumulator; partial sums meet in shared memory at the end.
template <int MT, int NT>
__device__ __forceinline__ bool shrink_mma_body(const StreamParams &P, const StreamProblem &pb, const Unit &u,
                                                uint8_t *smem, uint64_t *full, const int *rows, int k0,
                                                int k1, float *red /*[len][r]*/) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint16_t *A_slot = pb.A + (int64_t)u.slot * pb.r_max * pb.d;
  const int nchunks = (k1 - k0 + u.cw - 1) / u.cw;
  float acc[MT][NT][4];
#pragma unroll
  for (int mt = 0; mt < MT; ++mt)
#pragma unroll
    for (int nt = 0; nt < NT; ++nt)
#pragma unroll
      for (int q = 0; q < 4; ++q) acc[mt][nt][q] = 0.f;

  if (warp == 0)
    for (int c = 0; c < min(kStages - 1, nchunks); ++c)
      issue_chunk(smem + c * kStageBytes, &full[c], u, A_slot, pb.d, pb.x, pb.ldx, rows, k0 + c * u.cw,
                  min(u.cw, k1 - (k0 + c * u.cw)));
  for (int c = 0; c < nchunks; ++c) {
    const int s = c % kStages;
    if (warp == 0 && c + kStages - 1 < nchunks) {
      const int cn = c + kStages - 1;
      issue_chunk(smem + (cn % kStages) * kStageBytes, &full[cn % kStages], u, A_slot, pb.d, pb.x, pb.ldx,
                  rows, k0 + cn * u.cw, min(u.cw, k1 - (k0 + cn * u.cw)));
    }
    if (!mbar_wait(&full[s], (c / kStages) & 1)) {
      report(P.status, MINT_ERR_TIMEOUT, blockIdx.y);
      return false;
    }
    uint8_t *stage = smem + s * kStageBytes;
    const int width = min(u.cw, k1 - (k0 + c * u.cw));
    if (width & 15) {  // ragged tail of d: pad the last half k-step with zeros
      for (int i = threadIdx.x; i < u.r_pad + u.m_pad; i += kThreads)
        *reinterpret_cast<uint4 *>(stage + (size_t)i * u.pitch + width * 2) = make_uint4(0, 0, 0, 0);
      __syncthreads();
    }
    const int ksteps = (width + 15) >> 4;
    const uint32_t a_base = smem_addr(stage);
    const uint32_t x_base = a_base + (uint32_t)(u.r_pad * u.pitch);
    for (int ks = warp; ks < ksteps; ks += kWarps) {
      uint32_t xa[MT][4];
#pragma unroll
      for (int mt = 0; mt < MT; ++mt)
        ldmatrix_x4(xa[mt], x_base + (uint32_t)((mt * 16 + (lane & 15)) * u.pitch + (ks * 16 + (lane >> 4) * 8) * 2));
#pragma unroll
      for (int jp = 0; jp < NT / 2; ++jp) {
        if (jp * 16 < u.r_pad) {
          uint32_t b[4];
          const int m = lane >> 3;
          ldmatrix_x4(b, a_base + (uint32_t)((jp * 16 + (m >> 1) * 8 + (lane & 7)) * u.pitch +
                                             (ks * 16 + (m & 1) * 8) * 2));
#pragma unroll
          for (int mt = 0; mt < MT; ++mt) {
            mma_bf16(acc[mt][2 * jp], xa[mt], b[0], b[1]);
            mma_bf16(acc[mt][2 * jp + 1], xa[mt], b[2], b[3]);
          }
        }
      }
    }
    __syncthreads();  // stage s may be refilled
  }
  // cross-warp sum through shared memory (stages are idle now)
  float *scratch = reinterpret_cast<float *>(smem);  // [kWarps][MT*16][NT*8]
  const int g = lane >> 2, t = lane & 3;
  constexpr int RW = NT * 8;
#pragma unroll
  for (int mt = 0; mt < MT; ++mt)
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
      float *base = scratch + ((size_t)warp * MT * 16 + mt * 16) * RW + nt * 8 + 2 * t;
      *reinterpret_cast<float2 *>(base + (size_t)g * RW) = make_float2(acc[mt][nt][0], acc[mt][nt][1]);
      *reinterpret_cast<float2 *>(base + (size_t)(g + 8) * RW) = make_float2(acc[mt][nt][2], acc[mt][nt][3]);
    }
  __syncthreads();
  for (int i = threadIdx.x; i < u.len * u.r; i += kThreads) {
    const int l = i / u.r, j = i - l * u.r;
    float s = 0.f;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) s += scratch[((size_t)w * MT * 16 + l) * RW + j];
    red[i] = s;
  }
  return true;
}

// fp32 FMA body for rank <= 4 and at most 8 tokens: only the real rows are read.
__device__ __forceinline__ bool shrink_fma_body(const StreamParams &P, const StreamProblem &pb, const Unit &u,
                                                uint8_t *smem, uint64_t *full, const int *rows, int k0,
                                                int k1, float *red, float *scratch /*[kWarps][32]*/) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint16_t *A_slot = pb.A + (int64_t)u.slot * pb.r_max * pb.d;
  const int nchunks = (k1 - k0 + u.cw - 1) / u.cw;
  float acc[8][4];
#pragma unroll
  for (int l = 0; l < 8; ++l)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[l][j] = 0.f;
  if (warp == 0)
    for (int c = 0; c < min(kStages - 1, nchunks); ++c)
      issue_chunk(smem + c * kStageBytes, &full[c], u, A_slot, pb.d, pb.x, pb.ldx, rows, k0 + c * u.cw,
                  min(u.cw, k1 - (k0 + c * u.cw)));
  for (int c = 0; c < nchunks; ++c) {
    const int s = c % kStages;
    if (warp == 0 && c + kStages - 1 < nchunks) {
      const int cn = c + kStages - 1;
      issue_chunk(smem + (cn % kStages) * kStageBytes, &full[cn % kStages], u, A_slot, pb.d, pb.x, pb.ldx,
                  rows, k0 + cn * u.cw, min(u.cw, k1 - (k0 + cn * u.cw)));
    }
    if (!mbar_wait(&full[s], (c / kStages) & 1)) {
      report(P.status, MINT_ERR_TIMEOUT, blockIdx.y);
      return false;
    }
    const uint8_t *stage = smem + s * kStageBytes;
    const int width = min(u.cw, k1 - (k0 + c * u.cw));
    for (int v = threadIdx.x; v < (width >> 3); v += kThreads) {
      float af[4][8];
#pragma unroll
      for (int j = 0; j < 4; ++j)
        if (j < u.r) unpack8(*reinterpret_cast<const uint4 *>(stage + (size_t)j * u.pitch + v * 16), af[j]);
#pragma unroll
      for (int l = 0; l < 8; ++l) {
        if (l < u.len) {
          float xf[8];
          unpack8(*reinterpret_cast<const uint4 *>(stage + (size_t)(u.r_pad + l) * u.pitch + v * 16), xf);
#pragma unroll
          for (int j = 0; j < 4; ++j)
            if (j < u.r) {
#pragma unroll
              for (int e = 0; e < 8; ++e) acc[l][j] = fmaf(xf[e], af[j][e], acc[l][j]);
            }
        }
      }
    }
    __syncthreads();
  }
#pragma unroll
  for (int l = 0; l < 8; ++l)
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      if (l < u.len && j < u.r) {
        const float s = warp_sum(acc[l][j]);
        if (lane == 0) scratch[warp * 32 + l * 4 + j] = s;
      }
    }
  __syncthreads();
  for (int i = threadIdx.x; i < u.len * u.r; i += kThreads) {
    const int l = i / u.r, j = i - l * u.r;
    float s = 0.f;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) s += scratch[w * 32 + l * 4 + j];
    red[i] = s;
  }
  return true;
}

__global__ void __launch_bounds__(kThreads) shrink_stream_kernel(const StreamParams P) {
  extern __shared__ __align__(128) uint8_t dyn_smem[];
  __shared__ uint64_t full[kStages];
  __shared__ int rows[kTileRowsMax];
  __shared__ float fma_scratch[kWarps * 32];
  __shared__ int is_last;
  float *red = reinterpret_cast<float *>(dyn_smem);  // [len][r] reduced result of this unit
  uint8_t *smem = dyn_smem + kFrontBytes;            // the stages

  pdl_launch_dependents();  // the expand kernel may start streaming B and y now
  const StreamProblem &pb = P.prob[blockIdx.z];
  if (!plan_ok(P.pv.header, P.T, 1, P.tab.num_slots, 0, P.tab.gen_lo, P.tab.gen_hi, P.status)) return;
  Unit u;
  const int tile = blockIdx.y;
  if (!decode_unit(P, tile, pb.r_max, u)) return;
  const int units16 = (pb.d + 15) >> 4;
  const int slices = slices_for((int64_t)(u.r + u.len) * pb.d * 2, units16, pb.shrink_cap, P.target_bytes);
  const int slice = blockIdx.x;
  if (slice >= slices) return;
  const int k0 = (int)((int64_t)units16 * slice / slices) * 16;
  const int k1 = min(pb.d, (int)((int64_t)units16 * (slice + 1) / slices) * 16);

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) mbar_init(&full[s], 1);
    fence_mbar_init();
  }
  if (threadIdx.x < u.len) rows[threadIdx.x] = P.pv.perm[u.off + threadIdx.x];
  __syncthreads();

  bool ok;
  if (!u.mma) {
    ok = shrink_fma_body(P, pb, u, smem, full, rows, k0, k1, red, fma_scratch);
  } else {
    const int mt = u.m_pad >> 4, nt = u.r_pad >> 3;
    if (mt == 1) {
      if (nt <= 2) ok = shrink_mma_body<1, 2>(P, pb, u, smem, full, rows, k0, k1, red);
      else if (nt <= 4) ok = shrink_mma_body<1, 4>(P, pb, u, smem, full, rows, k0, k1, red);
      else ok = shrink_mma_body<1, 8>(P, pb, u, smem, full, rows, k0, k1, red);
    } else {
      if (nt <= 2) ok = shrink_mma_body<2, 2>(P, pb, u, smem, full, rows, k0, k1, red);
      else if (nt <= 4) ok = shrink_mma_body<2, 4>(P, pb, u, smem, full, rows, k0, k1, red);
      else ok = shrink_mma_body<2, 8>(P, pb, u, smem, full, rows, k0, k1, red);
    }
  }
  if (!ok) return;
  __syncthreads();

  // v[tile][l][j], row stride r_max
  float *v_tile = pb.ws_v + (size_t)tile * kTileRowsMax * pb.r_max;
  const int cnt = u.len * u.r;
  if (slices == 1) {
    for (int i = threadIdx.x; i < cnt; i += kThreads) {
      const int l = i / u.r, j = i - l * u.r;
      v_tile[l * pb.r_max + j] = red[i];
    }
    return;
  }
  float *part = pb.ws_part + ((size_t)tile * pb.shrink_cap) * kTileRowsMax * pb.r_max;
  const size_t part_stride = (size_t)kTileRowsMax * pb.r_max;
  for (int i = threadIdx.x; i < cnt; i += kThreads) part[slice * part_stride + i] = red[i];
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) {
    const int ticket = atomicAdd(&pb.ws_ticket[tile], 1);
    is_last = (ticket == slices - 1);
  }
  __syncthreads();
  if (!is_last) return;
  __threadfence();
  for (int i = threadIdx.x; i < cnt; i += kThreads) {
    float s = 0.f;
    for (int q = 0; q < slices; ++q) s += __ldcg(&part[q * part_stride + i]);
    const int l = i / u.r, j = i - l * u.r;
    v_tile[l * pb.r_max + j] = s;
  }
  if (threadIdx.x == 0) pb.ws_ticket[tile] = 0;  // leave the tickets zero for the next launch
}

// ================================================================================
// expand
// ================================================================================
template <int MT, int KS>
__device__ __forceinline__ void expand_mma_chunk(const Unit &u, uint8_t *stage, int width,
                                                 const uint32_t (&vh)[MT][KS][4],
                                                 const uint32_t (&vl)[MT][KS][4]) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, t = lane & 3;
  const uint32_t b_base = smem_addr(stage);
  uint8_t *y_base = stage + (size_t)u.r_pad * u.pitch;
  const int pairs = (width + 15) >> 4;
  for (int p = warp; p < pairs; p += kWarps) {
    float acc[MT][2][4];
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
      for (int nt = 0; nt < 2; ++nt)
#pragma unroll
        for (int q = 0; q < 4; ++q) acc[mt][nt][q] = 0.f;
#pragma unroll
    for (int ks = 0; ks < KS; ++ks) {
      if (ks * 16 < u.r_pad) {
        uint32_t b[4];
        const int m = lane >> 3;
        ldmatrix_x4_trans(b, b_base + (uint32_t)((ks * 16 + (m & 1) * 8 + (lane & 7)) * u.pitch +
                                                 (p * 16 + (m >> 1) * 8) * 2));
#pragma unroll
        for (int mt = 0; mt < MT; ++mt) {
          mma_bf16(acc[mt][0], vh[mt][ks], b[0], b[1]);
          mma_bf16(acc[mt][0], vl[mt][ks], b[0], b[1]);
          mma_bf16(acc[mt][1], vh[mt][ks], b[2], b[3]);
          mma_bf16(acc[mt][1], vl[mt][ks], b[2], b[3]);
        }
      }
    }
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
      for (int nt = 0; nt < 2; ++nt) {
        const int col = p * 16 + nt * 8 + 2 * t;
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          const int row = mt * 16 + g + h * 8;
          if (row < u.len) {
            uint32_t *yp = reinterpret_cast<uint32_t *>(y_base + (size_t)row * u.pitch + col * 2);
            const uint32_t w = *yp;
            *yp = pack_bf16x2(fmaf(u.scale, acc[mt][nt][2 * h], bf16lo(w)),
                              fmaf(u.scale, acc[mt][nt][2 * h + 1], bf16hi(w)));
          }
        }
      }
  }
}

__device__ __forceinline__ void expand_fma_chunk(const Unit &u, uint8_t *stage, int width, const float *vs) {
  // vs: [len][r] fp32 in shared memory
  uint8_t *y_base = stage + (size_t)u.r_pad * u.pitch;
  for (int v = threadIdx.x; v < (width >> 3); v += kThreads) {
    float bf[4][8];
#pragma unroll
    for (int j = 0; j < 4; ++j)
      if (j < u.r) unpack8(*reinterpret_cast<const uint4 *>(stage + (size_t)j * u.pitch + v * 16), bf[j]);
#pragma unroll
    for (int l = 0; l < 8; ++l) {
      if (l < u.len) {
        uint4 *yp = reinterpret_cast<uint4 *>(y_base + (size_t)l * u.pitch + v * 16);
        float yf[8], dl[8];
        unpack8(*yp, yf);
#pragma unroll
        for (int e = 0; e < 8; ++e) dl[e] = 0.f;
#pragma unroll
        for (int j = 0; j < 4; ++j)
          if (j < u.r) {
            const float vv = vs[l * u.r + j];
#pragma unroll
            for (int e = 0; e < 8; ++e) dl[e] = fmaf(vv, bf[j][e], dl[e]);
          }
#pragma unroll
        for (int e = 0; e < 8; ++e) yf[e] = fmaf(u.scale, dl[e], yf[e]);
        *yp = pack8(yf);
      }
    }
  }
}

// Splits v into a bf16 head and a bf16 remainder so that two MMAs carry about
// 16 significant bits of the fp32 shrink result into the expand.
__device__ __forceinline__ void split_pair(float a, float b, uint32_t &hi, uint32_t &lo) {
  hi = pack_bf16x2(a, b);
  lo = pack_bf16x2(a - bf16lo(hi), b - bf16hi(hi));
}

template <int MT, int KS>
__device__ __forceinline__ bool expand_body(const StreamParams &P, const StreamProblem &pb, const Unit &u,
                                            uint8_t *smem, uint64_t *full, const int *rows, int c0, int c1,
                                            const float *vs /*[32][64] fp32, zero beyond len / r*/) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint16_t *B_slot = pb.B + (int64_t)u.slot * pb.r_max * pb.n;
  const int nchunks = (c1 - c0 + u.cw - 1) / u.cw;
  uint32_t vh[MT][KS][4], vl[MT][KS][4];
  if (u.mma) {
    const int g = lane >> 2, t = lane & 3;
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
      for (int ks = 0; ks < KS; ++ks) {
        const float *r0 = vs + (mt * 16 + g) * kStreamRankCap + ks * 16 + 2 * t;
        const float *r1 = r0 + 8 * kStreamRankCap;
        split_pair(r0[0], r0[1], vh[mt][ks][0], vl[mt][ks][0]);
        split_pair(r1[0], r1[1], vh[mt][ks][1], vl[mt][ks][1]);
        split_pair(r0[8], r0[9], vh[mt][ks][2], vl[mt][ks][2]);
        split_pair(r1[8], r1[9], vh[mt][ks][3], vl[mt][ks][3]);
      }
  }
  for (int c = 0; c < nchunks; ++c) {
    const int s = c % kStages;
    uint8_t *stage = smem + s * kStageBytes;
    const int width = min(u.cw, c1 - (c0 + c * u.cw));
    if (!mbar_wait(&full[s], (c / kStages) & 1)) {
      report(P.status, MINT_ERR_TIMEOUT, blockIdx.y);
      return false;
    }
    if (u.mma) expand_mma_chunk<MT, KS>(u, stage, width, vh, vl);
    else expand_fma_chunk(u, stage, width, vs + kTileRowsMax * kStreamRankCap);
    fence_async_smem();  // this thread's y updates become visible to the bulk-copy engine
    __syncthreads();
    if (warp == 0) {
      uint8_t *y_base = stage + (size_t)u.r_pad * u.pitch;
      for (int l = lane; l < u.len; l += 32)
        bulk_store(pb.y + (int64_t)rows[l] * pb.ldy + c0 + c * u.cw, y_base + (size_t)l * u.pitch,
                   (uint32_t)width * 2u);
      bulk_commit();
      const int cn = c + kStages;  // the chunk that reuses this stage
      if (cn < nchunks) {
        bulk_wait_read_all();       // the stores above have read their shared-memory source
        __syncwarp();
        issue_chunk(stage, &full[s], u, B_slot, pb.n, pb.y, pb.ldy, rows, c0 + cn * u.cw,
                    min(u.cw, c1 - (c0 + cn * u.cw)));
      }
    }
  }
  if (warp == 0) bulk_wait_read_all();
  return true;
}

__global__ void __launch_bounds__(kThreads) expand_stream_kernel(const StreamParams P) {
  extern __shared__ __align__(128) uint8_t dyn_smem[];
  __shared__ uint64_t full[kStages];
  __shared__ int rows[kTileRowsMax];
  // [32][64] fp32 laid out for the MMA fragments, then [8][4] compact for the FMA path
  float *vs = reinterpret_cast<float *>(dyn_smem);
  uint8_t *smem = dyn_smem + kFrontBytes;

  const StreamProblem &pb = P.prob[blockIdx.z];
  // The plan, the slot table, B and y were all complete before the shrink kernel
  // started (it is an ordinary in-order launch), so they may be read before the
  // dependency wait; only v is produced by the shrink kernel.
  if (!plan_ok(P.pv.header, P.T, 1, P.tab.num_slots, 0, P.tab.gen_lo, P.tab.gen_hi, nullptr)) return;
  Unit u;
  const int tile = blockIdx.y;
  if (!decode_unit(P, tile, pb.r_max, u)) return;
  const int units16 = (pb.n + 15) >> 4;
  const int slices = slices_for((int64_t)(u.r + 2 * u.len) * pb.n * 2, units16, pb.expand_cap, P.target_bytes);
  const int slice = blockIdx.x;
  if (slice >= slices) return;
  const int c0 = (int)((int64_t)units16 * slice / slices) * 16;
  const int c1 = min(pb.n, (int)((int64_t)units16 * (slice + 1) / slices) * 16);
  const int nchunks = (c1 - c0 + u.cw - 1) / u.cw;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) mbar_init(&full[s], 1);
    fence_mbar_init();
  }
  if (threadIdx.x < u.len) rows[threadIdx.x] = P.pv.perm[u.off + threadIdx.x];
  // weight rows between the rank and its padding to 16 take part in the MMA: keep them zero
  if (u.mma && u.r_pad > u.r) {
    const int vec_per_row = u.pitch >> 4;
    for (int s = 0; s < kStages; ++s)
      for (int i = threadIdx.x; i < (u.r_pad - u.r) * vec_per_row; i += kThreads)
        *reinterpret_cast<uint4 *>(smem + s * kStageBytes + (size_t)(u.r + i / vec_per_row) * u.pitch +
                                   (i % vec_per_row) * 16) = make_uint4(0, 0, 0, 0);
  }
  __syncthreads();
  if ((threadIdx.x >> 5) == 0) {
    const uint16_t *B_slot = pb.B + (int64_t)u.slot * pb.r_max * pb.n;
    for (int c = 0; c < min(kStages, nchunks); ++c)
      issue_chunk(smem + c * kStageBytes, &full[c], u, B_slot, pb.n, pb.y, pb.ldy, rows, c0 + c * u.cw,
                  min(u.cw, c1 - (c0 + c * u.cw)));
  }

  pdl_wait();  // the shrink kernel has completed and its v is visible

  const float *v_tile = pb.ws_v + (size_t)tile * kTileRowsMax * pb.r_max;
  if (u.mma) {
    for (int i = threadIdx.x; i < u.m_pad * u.r_pad; i += kThreads) {
      const int l = i / u.r_pad, j = i - l * u.r_pad;
      vs[l * kStreamRankCap + j] = (l < u.len && j < u.r) ? __ldcg(&v_tile[l * pb.r_max + j]) : 0.f;
    }
  } else {
    for (int i = threadIdx.x; i < u.len * u.r; i += kThreads) {
      const int l = i / u.r, j = i - l * u.r;
      vs[kTileRowsMax * kStreamRankCap + i] = __ldcg(&v_tile[l * pb.r_max + j]);
    }
  }
  __syncthreads();

  const int mt = u.m_pad >> 4, ks = u.r_pad >> 4;
  if (!u.mma || (mt == 1 && ks <= 1)) expand_body<1, 1>(P, pb, u, smem, full, rows, c0, c1, vs);
  else if (mt == 1 && ks == 2) expand_body<1, 2>(P, pb, u, smem, full, rows, c0, c1, vs);
  else if (mt == 1) expand_body<1, 4>(P, pb, u, smem, full, rows, c0, c1, vs);
  else if (ks <= 1) expand_body<2, 1>(P, pb, u, smem, full, rows, c0, c1, vs);
  else if (ks == 2) expand_body<2, 2>(P, pb, u, smem, full, rows, c0, c1, vs);
  else expand_body<2, 4>(P, pb, u, smem, full, rows, c0, c1, vs);
}

// ---- host side -----------------------------------------------------------------
int g_attr_done = 0;

int32_t ensure_attrs() {
  if (g_attr_done) return MINT_OK;
  const int bytes = kDynSmemBytes;
  int32_t st = mint_check_cuda(cudaFuncSetAttribute(shrink_stream_kernel,
                                                    cudaFuncAttributeMaxDynamicSharedMemorySize, bytes),
                               "shrink_stream smem attribute");
  if (st) return st;
  st = mint_check_cuda(cudaFuncSetAttribute(expand_stream_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                            bytes),
                       "expand_stream smem attribute");
  if (st) return st;
  g_attr_done = 1;
  return MINT_OK;
}

int split_cap_for(int64_t tiles_ub) {
  int64_t cap = 2400 / (tiles_ub > 0 ? tiles_ub : 1);
  if (cap < 1) cap = 1;
  if (cap > 32) cap = 32;
  return (int)cap;
}

constexpr int kTargetBytes = 40960;

}  // namespace

bool mint_stream_supported(int32_t r_max_bound) { return r_max_bound <= kStreamRankCap; }

size_t mint_stream_workspace_bytes(int32_t T, int32_t num_slots, int32_t r_max) {
  const int64_t tiles = mint_tile_upper_bound(1, T, num_slots);
  const int cap = split_cap_for(tiles);
  const size_t tile_floats = (size_t)kTileRowsMax * r_max;
  size_t bytes = (size_t)tiles * 4;                       // tickets
  bytes = (bytes + 255) / 256 * 256;
  bytes += (size_t)tiles * tile_floats * 4;               // v
  bytes += (size_t)tiles * cap * tile_floats * 4;         // split partial sums
  return bytes + 256;
}

int32_t mint_launch_stream(const DenseArgs *args, int nprob, const TableDev &tab, const void *plan_dev,
                           void *const *workspaces, cudaStream_t s) {
  if (nprob < 1 || nprob > kMaxProblems) return mint_fail(MINT_ERR_INVALID_ARG, "grouped apply: 1..%d problems", kMaxProblems);
  int32_t st = ensure_attrs();
  if (st) return st;
  const int32_t T = args[0].T;
  const int64_t tiles = mint_tile_upper_bound(1, T, tab.num_slots);
  if (tiles == 0) return MINT_OK;
  const int cap = split_cap_for(tiles);
  StreamParams P = {};
  int gx_shrink = 1, gx_expand = 1;
  for (int i = 0; i < nprob; ++i) {
    const DenseArgs &a = args[i];
    StreamProblem &pb = P.prob[i];
    pb.A = a.A; pb.B = a.B; pb.x = a.x; pb.y = a.y;
    pb.ldx = a.ldx; pb.ldy = a.ldy;
    pb.d = a.d; pb.n = a.n; pb.r_max = a.r_max;
    pb.shrink_cap = cap;
    pb.expand_cap = cap * 2;
    uint8_t *w = static_cast<uint8_t *>(workspaces[i]);
    const size_t tile_floats = (size_t)kTileRowsMax * a.r_max;
    size_t off = ((size_t)tiles * 4 + 255) / 256 * 256;
    pb.ws_ticket = reinterpret_cast<int32_t *>(w);
    pb.ws_v = reinterpret_cast<float *>(w + off);
    off += (size_t)tiles * tile_floats * 4;
    pb.ws_part = reinterpret_cast<float *>(w + off);
    const int rr = a.r_max < kStreamRankCap ? a.r_max : kStreamRankCap;
    gx_shrink = std::max(gx_shrink, slices_for((int64_t)(rr + kTileRowsMax) * a.d * 2, (a.d + 15) >> 4,
                                               pb.shrink_cap, kTargetBytes));
    gx_expand = std::max(gx_expand, slices_for((int64_t)(rr + 2 * kTileRowsMax) * a.n * 2, (a.n + 15) >> 4,
                                               pb.expand_cap, kTargetBytes));
  }
  P.T = T;
  P.target_bytes = kTargetBytes;
  P.status = args[0].status;
  P.tab = tab;
  P.pv = mint_plan_view(plan_dev, T);
  const size_t smem = (size_t)kDynSmemBytes;

  shrink_stream_kernel<<<dim3(gx_shrink, (unsigned)tiles, nprob), kThreads, smem, s>>>(P);
  st = mint_check_cuda(cudaGetLastError(), "shrink_stream launch");
  if (st) return st;

  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(gx_expand, (unsigned)tiles, nprob);
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return mint_check_cuda(cudaLaunchKernelEx(&cfg, expand_stream_kernel, P), "expand_stream launch");
}
