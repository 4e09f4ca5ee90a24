// LoRA backward over padded slots (dense projections).
//
// The paper trains many adapters over one frozen base in time slices and names
// kernels that update several adapters in one batch as the alternative (section
// "Time-Sliced Multi-LoRA Training"); workers hold adapters in slots of a
// configured maximum shape, smaller ranks padded and masked.  This file is that
// alternative for the update the forward path applies,
//   y[t, :] += s * (x[t, :] . A^T) . B          (A: rank x d, B: rank x n of the token's slot):
// for an upstream gradient dy,
//   u = dy . B^T,  v = x . A^T                               (rank values per token)
//   dx[t, :] += s * u[t, :] . A
//   dA[slot][k, :] += s * sum over the slot's tokens of u[t, k] * x[t, :]
//   dB[slot][k, :] += s * sum over the slot's tokens of v[t, k] * dy[t, :]
// with rows k >= rank (the padding) and slots without tokens left untouched.
//
// dx is the forward apply with the pool's tensors in each other's place (B's
// rows are rank rows of n contiguous elements, exactly what the shrink wants of
// A, and A's are what the expand wants of B), u and v are the streamed shrink of
// the same two pools, so those three steps reuse the forward kernels.  What is
// new is the weight gradient: one CTA per (segment, 512 columns of a tensor) walks the
// segment's tokens in plan order and keeps 8 rank rows x 4 columns of fp32
// sums per thread; a thread owns its elements of dA / dB outright, so there are
// no atomics and the sums do not depend on scheduling.
#include "mint_device.cuh"

using namespace mint;

namespace {

constexpr int kThreads = 128;
constexpr int kColsPerThread = 4;
constexpr int kColsPerCta = kThreads * kColsPerThread;   // 512
constexpr int kTokenBatch = 64;
constexpr int kRankChunk = 8;         // rank rows per pass: 32 sums per thread keep eight CTAs on an SM (measured
                                      // on the 4B-dense decode layer: 16 rows 212 us, 8 rows 176 us, 4 rows 166 us;
                                      // with the gradient rows prefetched 8 rows 145 us, 4 rows 142 us; 8 kept for
                                      // segments of many tokens, whose activations are re-read per pass)
constexpr int kBlocksPerCta = 1;      // 512-column blocks of one tensor per CTA (more measured slower: 185 us for 2)

constexpr int kMaxJobs = 2 * MINT_MAX_GROUP;   // dA and dB of every projection of a grouped call

// Programmatic dependent launch: the next kernel of the stream may become resident at once; data of
// earlier kernels is touched only after the wait, which every CTA executes (completion stays
// transitive along the stream).
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

struct GradJob {
  const float *coef;      // [T][r_max] fp32, token order: u (for dA) or v (for dB)
  const uint16_t *act;    // [T][ld] bf16: x (for dA) or dy (for dB)
  int64_t ld;
  float *out;             // [blocks][r_max][width] fp32, accumulated into (packed: [blocks][width][r_max]);
                          // block = slot, or slot * experts + expert
  const int32_t *row_map; // row of act that item p reads (nullptr: p)
  int64_t act_rows;       // rows of act: an item whose row is outside is left out
  int32_t width, r_max;
  int32_t block0;         // first of its groups of kBlocksPerCta column blocks in the grid's second dimension
  int32_t packed;
};

struct GradParams {
  GradJob job[kMaxJobs];
  int32_t njobs, T;
  int32_t K, E;           // items per token and experts of a MoE plan (1, 0: dense)
  int32_t *status;
  TableDev tab;
  PlanView pv;
};

// kGeneral: (slot, expert) blocks, a row map for the activations and the packed layout (MoE pools); the
// dense instantiation carries none of that.
template <bool kGeneral>
__global__ void __launch_bounds__(kThreads) grad_weight_kernel(const __grid_constant__ GradParams P) {
  __shared__ int32_t tok[kTokenBatch];    // staged items (tokens, or (token, k) pairs)
  __shared__ int32_t arow[kTokenBatch];   // the row of act each of them reads
  __shared__ float cf[kTokenBatch][kRankChunk];
  const int tid = threadIdx.x;
  pdl_launch_dependents();
  // (before the wait: the plan and the slot table, complete before this call's first kernel started)
  if (!plan_ok(P.pv.header, P.T, P.K, P.tab.num_slots, P.E, P.tab.gen_lo, P.tab.gen_hi,
               (blockIdx.x == 0 && blockIdx.y == 0) ? P.status : nullptr)) {
    pdl_wait();
    return;
  }
  int ji = 0;   // the job this column block belongs to
  while (ji + 1 < P.njobs && (int)blockIdx.y >= P.job[ji + 1].block0) ++ji;
  const GradJob &p = P.job[ji];
  const int seg = blockIdx.x;
  if (seg >= P.pv.header[PH_NUM_SEGMENTS]) {
    pdl_wait();
    return;
  }
  const int off = P.pv.seg_start[seg], len = P.pv.seg_start[seg + 1] - off;
  const int slot = P.pv.seg_slot[seg];
  const int rank = P.tab.slot_rank[slot];
  const float scale = P.tab.slot_scale[slot];
  if (rank > p.r_max) {
    pdl_wait();
    if (tid == 0) report(P.status, MINT_ERR_RANK_TOO_LARGE, slot);
    return;
  }
  const int block = (kGeneral && P.E > 0) ? slot * P.E + P.pv.seg_expert[seg] : slot;
  float *out_slot = p.out + (size_t)block * p.r_max * p.width;
  const bool one_batch = len <= kTokenBatch;   // the usual case of a decode batch: staged once per rank chunk
  // stages the token indices and the coefficients of tokens [b0, b0 + nb) for ranks k0 .. k0 + kc - 1
  auto stage = [&](int b0, int nb, int k0, int kc) {
    __syncthreads();   // what was staged before has been read
    if (tid < nb) {
      const int item = P.pv.perm[off + b0 + tid];
      tok[tid] = item;
      const int r_ = (kGeneral && p.row_map) ? p.row_map[item] : item;
      arow[tid] = (!kGeneral || (r_ >= 0 && r_ < p.act_rows)) ? r_ : ~0;   // (~0: out of range, reported by the shrink; it counts as zero)
    }
    __syncthreads();
    for (int i = tid; i < nb * kRankChunk; i += kThreads) {
      const int j = i / kRankChunk, k = i - j * kRankChunk;
      cf[j][k] = (k < kc && (!kGeneral || arow[j] >= 0)) ? p.coef[(size_t)tok[j] * p.r_max + k0 + k] : 0.f;
    }
    __syncthreads();
  };
  {
    // the gradient rows this CTA will add to, on their way into L2 while the tokens are walked
    const int col = ((int)blockIdx.y - p.block0) * kBlocksPerCta * kColsPerCta + tid * kColsPerThread;
    if (kGeneral && p.packed) {   // [width][r_max]: this thread's four columns are 4 r_max consecutive floats
      if (col < p.width)
        for (int i = 0; i < 4 * p.r_max; i += 32)
          asm volatile("prefetch.global.L2 [%0];" ::"l"(out_slot + (size_t)col * p.r_max + i));
    } else if ((tid & 7) == 0 && col < p.width)
      for (int k = 0; k < rank; ++k)
        asm volatile("prefetch.global.L2 [%0];" ::"l"(out_slot + (size_t)k * p.width + col));
  }
  pdl_wait();   // the coefficients, the activations and the gradients belong to earlier kernels until here
  for (int k0 = 0; k0 < rank; k0 += kRankChunk) {
    const int kc = min(kRankChunk, rank - k0);
    if (one_batch) stage(0, len, k0, kc);
    for (int cb = 0; cb < kBlocksPerCta; ++cb) {
      const int col = (((int)blockIdx.y - p.block0) * kBlocksPerCta + cb) * kColsPerCta + tid * kColsPerThread;
      if (((int)blockIdx.y - p.block0) * kBlocksPerCta * kColsPerCta + cb * kColsPerCta >= p.width) break;   // (same for all threads)
      const bool col_ok = col < p.width;   // (widths are multiples of 8, so four columns are in or out together)
      float acc[kRankChunk][kColsPerThread];
#pragma unroll
      for (int k = 0; k < kRankChunk; ++k)
#pragma unroll
        for (int e = 0; e < kColsPerThread; ++e) acc[k][e] = 0.f;
      for (int b0 = 0; b0 < len; b0 += kTokenBatch) {
        const int nb = min(kTokenBatch, len - b0);
        if (!one_batch) stage(b0, nb, k0, kc);
        if (col_ok) {
#pragma unroll 4
          for (int j = 0; j < nb; ++j) {
            const uint2 q = __ldg(reinterpret_cast<const uint2 *>(p.act + (int64_t)(kGeneral ? max(arow[j], 0) : tok[j]) * p.ld + col));
            const float a[4] = {bf16lo(q.x), bf16hi(q.x), bf16lo(q.y), bf16hi(q.y)};
#pragma unroll
            for (int k = 0; k < kRankChunk; ++k) {
              const float c = cf[j][k];
#pragma unroll
              for (int e = 0; e < kColsPerThread; ++e) acc[k][e] = fmaf(c, a[e], acc[k][e]);
            }
          }
        }
      }
      if (kGeneral && col_ok && p.packed) {
        // [width][r_max]: the chunk's ranks of a column are eight consecutive floats (r_max is a multiple of
        // 8); ranks at or above the slot's rank are written back as they were read
#pragma unroll
        for (int e = 0; e < kColsPerThread; ++e)
#pragma unroll
          for (int h = 0; h < kRankChunk / 4; ++h)
            if (4 * h < kc) {
              float4 *dst = reinterpret_cast<float4 *>(out_slot + (size_t)(col + e) * p.r_max + k0 + 4 * h);
              float4 o = *dst;
              if (4 * h + 0 < kc) o.x = fmaf(scale, acc[4 * h + 0][e], o.x);
              if (4 * h + 1 < kc) o.y = fmaf(scale, acc[4 * h + 1][e], o.y);
              if (4 * h + 2 < kc) o.z = fmaf(scale, acc[4 * h + 2][e], o.z);
              if (4 * h + 3 < kc) o.w = fmaf(scale, acc[4 * h + 3][e], o.w);
              *dst = o;
            }
      } else if (col_ok) {
#pragma unroll
        for (int k = 0; k < kRankChunk; ++k)
          if (k < kc) {
            float4 *dst = reinterpret_cast<float4 *>(out_slot + (size_t)(k0 + k) * p.width + col);
            float4 o = *dst;
            o.x = fmaf(scale, acc[k][0], o.x);
            o.y = fmaf(scale, acc[k][1], o.y);
            o.z = fmaf(scale, acc[k][2], o.z);
            o.w = fmaf(scale, acc[k][3], o.w);
            *dst = o;
          }
      }
    }
  }
}

// ---- dx of per-expert LoRA tensors in the packed layout -------------------------------
// dx[p, :] += s * u[p, :rank] . A[slot][expert]^T with A stored [d][r_max] (a column of d is r_max
// consecutive values).  One CTA per (tile of at most 32 pairs of one (expert, slot), 1024 columns
// of d): the tile's u (already times the routing weight) waits in shared memory times s, a thread
// holds the r_max weights of its column(s) in registers and walks the tile's pairs.  CUDA cores:
// 2 r_max flops per 2 bytes of dx read and written.
struct MoeDxParams {
  const uint16_t *A;      // [slot][E][d][r_max]
  const float *u;         // [T*K][r_max], pair order
  uint16_t *dx;           // [T*K][lddx] bf16, accumulated into
  int64_t lddx;
  int32_t d, r_max, T, K, E;
  int32_t *status;
  TableDev tab;
  PlanView pv;
};

constexpr int kDxColsPerCta = 1024;

template <int RM>
__global__ void __launch_bounds__(kThreads) moe_dx_kernel(const __grid_constant__ MoeDxParams P) {
  constexpr int kCols = RM <= 16 ? 2 : 1;   // columns per thread
  __shared__ float us[32][RM];
  __shared__ int32_t row[32];
  const int tid = threadIdx.x;
  pdl_launch_dependents();
  if (!plan_ok(P.pv.header, P.T, P.K, P.tab.num_slots, P.E, P.tab.gen_lo, P.tab.gen_hi, nullptr) ||
      (int)blockIdx.x >= P.pv.header[PH_NCHUNK1]) {
    pdl_wait();
    return;
  }
  const TileDesc t = P.pv.tile_desc[blockIdx.x];
  const uint16_t *A_blk = P.A + ((size_t)t.slot * P.E + t.expert) * (size_t)P.d * RM;
  if (tid < 32) row[tid] = tid < t.len ? P.pv.perm[t.off + tid] : 0;
  pdl_wait();   // u and dx belong to earlier kernels until here
  __syncthreads();
  for (int i = tid; i < 32 * RM; i += kThreads) {
    const int l = i / RM, k = i - l * RM;
    us[l][k] = (l < t.len && k < t.rank) ? t.scale * P.u[(size_t)row[l] * RM + k] : 0.f;
  }
  __syncthreads();
  const int c_end = min(P.d, ((int)blockIdx.y + 1) * kDxColsPerCta);
  for (int c = (int)blockIdx.y * kDxColsPerCta + tid * kCols; c < c_end; c += kThreads * kCols) {
    float a[kCols][RM];
#pragma unroll
    for (int e = 0; e < kCols; ++e)
#pragma unroll
      for (int k8 = 0; k8 < RM; k8 += 8) {
        float f[8];
        unpack8(__ldg(reinterpret_cast<const uint4 *>(A_blk + (size_t)(c + e) * RM + k8)), f);
#pragma unroll
        for (int k = 0; k < 8; ++k) a[e][k8 + k] = k8 + k < t.rank ? f[k] : 0.f;   // (padding may hold anything)
      }
    for (int l = 0; l < t.len; ++l) {
      float acc[kCols];
#pragma unroll
      for (int e = 0; e < kCols; ++e) acc[e] = 0.f;
#pragma unroll
      for (int k = 0; k < RM; ++k) {
        const float uk = us[l][k];
#pragma unroll
        for (int e = 0; e < kCols; ++e) acc[e] = fmaf(uk, a[e][k], acc[e]);
      }
      uint16_t *dst = P.dx + (size_t)row[l] * P.lddx + c;
      if (kCols == 2) {
        const uint32_t old = *reinterpret_cast<const uint32_t *>(dst);
        *reinterpret_cast<uint32_t *>(dst) = pack_bf16x2(bf16lo(old) + acc[0], bf16hi(old) + acc[kCols - 1]);
      } else {
        const uint32_t old = (uint32_t)*dst;
        *dst = (uint16_t)(pack_bf16x2(bf16lo(old) + acc[0], 0.f) & 0xffffu);
      }
    }
  }
}

}  // namespace

int32_t mint_launch_grad_weights(const GradJobHost *jobs, int njobs, int32_t T, const TableDev &tab,
                                 const void *plan_dev, int32_t *status, cudaStream_t s, int32_t K, int32_t E) {
  if (T == 0 || njobs == 0) return MINT_OK;
  if (njobs > kMaxJobs) return mint_fail(MINT_ERR_INVALID_ARG, "weight gradients: at most %d tensors per launch", kMaxJobs);
  GradParams P = {};
  int blocks = 0;
  for (int i = 0; i < njobs; ++i) {
    GradJob &j = P.job[i];
    j.coef = jobs[i].coef;
    j.act = jobs[i].act;
    j.ld = jobs[i].ld;
    j.out = jobs[i].out;
    j.width = jobs[i].width;
    j.r_max = jobs[i].r_max;
    j.row_map = jobs[i].row_map;
    j.act_rows = jobs[i].act_rows > 0 ? jobs[i].act_rows : ((int64_t)1 << 40);
    j.packed = jobs[i].packed;
    j.block0 = blocks;
    blocks += (jobs[i].width + kBlocksPerCta * kColsPerCta - 1) / (kBlocksPerCta * kColsPerCta);
  }
  P.njobs = njobs;
  P.T = T;
  P.K = K;
  P.E = E;
  P.status = status;
  P.tab = tab;
  const int64_t items = (int64_t)T * K, key_space = (int64_t)tab.num_slots * (E > 0 ? E : 1);
  P.pv = mint_plan_view(plan_dev, items, key_space);
  const int64_t seg_ub = items < key_space ? items : key_space;
  const dim3 grid((unsigned)seg_ub, (unsigned)blocks);
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = dim3(kThreads);
  cfg.stream = s;
  cfg.attrs = attr;
  // right after a plan or a bind kernel it waits for that kernel in full: it reads the plan at once
  cfg.numAttrs = mint_take_tables_changed() ? 0 : 1;
  bool general = E > 0;
  for (int i = 0; i < njobs; ++i) general = general || jobs[i].row_map != nullptr || jobs[i].packed;
  return mint_check_cuda(general ? cudaLaunchKernelEx(&cfg, grad_weight_kernel<true>, P)
                                 : cudaLaunchKernelEx(&cfg, grad_weight_kernel<false>, P),
                         "grad_weight launch");
}


// dx[p, :] += s * u[p, :] . A[slot][expert]^T for the pairs of a MoE plan (packed A, r_max 8, 16, 32 or 64).
int32_t mint_launch_moe_dx(const uint16_t *A, const float *u, uint16_t *dx, int64_t lddx, int32_t d, int32_t r_max,
                           int32_t T, int32_t K, int32_t E, const TableDev &tab, const void *plan_dev,
                           int32_t *status, cudaStream_t s) {
  const int64_t pairs = (int64_t)T * K, key_space = (int64_t)tab.num_slots * E;
  const int64_t tiles = mint_tile_upper_bound(1, pairs, key_space);
  if (tiles == 0) return MINT_OK;
  MoeDxParams P = {};
  P.A = A; P.u = u; P.dx = dx; P.lddx = lddx;
  P.d = d; P.r_max = r_max; P.T = T; P.K = K; P.E = E;
  P.status = status;
  P.tab = tab;
  P.pv = mint_plan_view(plan_dev, pairs, key_space);
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)tiles, (unsigned)((d + kDxColsPerCta - 1) / kDxColsPerCta));
  cfg.blockDim = dim3(kThreads);
  cfg.stream = s;
  cfg.attrs = attr;
  cfg.numAttrs = mint_take_tables_changed() ? 0 : 1;
  cudaError_t e;
  switch (r_max) {
    case 8: e = cudaLaunchKernelEx(&cfg, moe_dx_kernel<8>, P); break;
    case 16: e = cudaLaunchKernelEx(&cfg, moe_dx_kernel<16>, P); break;
    case 32: e = cudaLaunchKernelEx(&cfg, moe_dx_kernel<32>, P); break;
    case 64: e = cudaLaunchKernelEx(&cfg, moe_dx_kernel<64>, P); break;
    default: return mint_fail(MINT_ERR_UNSUPPORTED, "MoE backward: r_max %d (8, 16, 32 or 64)", r_max);
  }
  return mint_check_cuda(e, "moe_dx launch");
}
