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
  float *out;             // [slots][r_max][width] fp32, accumulated into
  int32_t width, r_max;
  int32_t block0;         // first of its groups of kBlocksPerCta column blocks in the grid's second dimension
  int32_t pad;
};

struct GradParams {
  GradJob job[kMaxJobs];
  int32_t njobs, T;
  int32_t *status;
  TableDev tab;
  PlanView pv;
};

__global__ void __launch_bounds__(kThreads) grad_weight_kernel(const __grid_constant__ GradParams P) {
  __shared__ int32_t tok[kTokenBatch];
  __shared__ float cf[kTokenBatch][kRankChunk];
  const int tid = threadIdx.x;
  pdl_launch_dependents();
  // (before the wait: the plan and the slot table, complete before this call's first kernel started)
  if (!plan_ok(P.pv.header, P.T, 1, P.tab.num_slots, 0, P.tab.gen_lo, P.tab.gen_hi,
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
  float *out_slot = p.out + (size_t)slot * p.r_max * p.width;
  const bool one_batch = len <= kTokenBatch;   // the usual case of a decode batch: staged once per rank chunk
  // stages the token indices and the coefficients of tokens [b0, b0 + nb) for ranks k0 .. k0 + kc - 1
  auto stage = [&](int b0, int nb, int k0, int kc) {
    __syncthreads();   // what was staged before has been read
    if (tid < nb) tok[tid] = P.pv.perm[off + b0 + tid];
    __syncthreads();
    for (int i = tid; i < nb * kRankChunk; i += kThreads) {
      const int j = i / kRankChunk, k = i - j * kRankChunk;
      cf[j][k] = k < kc ? p.coef[(size_t)tok[j] * p.r_max + k0 + k] : 0.f;
    }
    __syncthreads();
  };
  {
    // the gradient rows this CTA will add to, on their way into L2 while the tokens are walked
    const int col = ((int)blockIdx.y - p.block0) * kBlocksPerCta * kColsPerCta + tid * kColsPerThread;
    if ((tid & 7) == 0 && col < p.width)
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
            const uint2 q = __ldg(reinterpret_cast<const uint2 *>(p.act + (int64_t)tok[j] * p.ld + col));
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
      if (col_ok) {
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

}  // namespace

int32_t mint_launch_grad_weights(const GradJobHost *jobs, int njobs, int32_t T, const TableDev &tab,
                                 const void *plan_dev, int32_t *status, cudaStream_t s) {
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
    j.block0 = blocks;
    blocks += (jobs[i].width + kBlocksPerCta * kColsPerCta - 1) / (kBlocksPerCta * kColsPerCta);
  }
  P.njobs = njobs;
  P.T = T;
  P.status = status;
  P.tab = tab;
  P.pv = mint_plan_view(plan_dev, T, tab.num_slots);
  const int64_t seg_ub = T < tab.num_slots ? T : tab.num_slots;
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
  return mint_check_cuda(cudaLaunchKernelEx(&cfg, grad_weight_kernel, P), "grad_weight launch");
}
