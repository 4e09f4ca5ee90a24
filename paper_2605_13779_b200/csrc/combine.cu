// Router-weighted combine of the MoE expert LoRA update.
//
// Per-expert LoRA tensors are keyed by expert id (paper, section "Scale Up",
// Megatron placement); a token's routed experts are combined with the router's
// weights.  For the projection that ends an expert FFN (down), the update of
// token t is
//     Y[t, :] += sum over k of  w[t,k] * s_sigma * (X[p, :] . A[sigma][e_k]) . B[sigma][e_k],   p = t*K + k.
// The pairs of one token belong to different (expert, adapter) groups, which
// different CTAs stream; adding them into one row from there would need atomics
// and leave the order of the sum to the scheduler.  Instead the weighted
// per-pair updates are written to a scratch [T*K][n] (the ordinary MoE apply on
// a zero start), and this kernel adds the K rows of every token in k order in
// fp32 onto y with one round-to-nearest-even store.  A token whose K updates are
// all exactly zero (no resident adapter) keeps its row of y bit for bit.
#include "mint_device.cuh"

namespace {

__global__ void __launch_bounds__(256) combine_kernel(const uint16_t *__restrict__ pair, uint16_t *__restrict__ y,
                                                      int64_t ldy, int32_t T, int32_t K, int32_t n) {
  const int chunks = n >> 3;
  const int64_t total = (int64_t)T * chunks;
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  for (int64_t q = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; q < total; q += stride) {
    const int64_t t = q / chunks;
    const int c = (int)(q - t * chunks);
    float sum[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) sum[e] = 0.f;
    bool any = false;
    for (int k = 0; k < K; ++k) {   // k ascending: the order of the sum is fixed
      const uint4 w = mint::ldg128_stream(pair + ((t * K + k) * (int64_t)n + c * 8));
      any |= ((w.x | w.y | w.z | w.w) & 0x7fff7fffu) != 0u;
      float f[8];
      mint::unpack8(w, f);
#pragma unroll
      for (int e = 0; e < 8; ++e) sum[e] += f[e];
    }
    if (!any) continue;
    uint16_t *yp = y + t * ldy + c * 8;
    float f[8];
    mint::unpack8(*reinterpret_cast<const uint4 *>(yp), f);
#pragma unroll
    for (int e = 0; e < 8; ++e) f[e] += sum[e];
    *reinterpret_cast<uint4 *>(yp) = mint::pack8(f);
  }
}

size_t align256(size_t v) { return (v + 255) & ~(size_t)255; }

}  // namespace

extern "C" size_t mint_moe_lora_apply_combine_workspace_bytes(const mint_pool *pool, int32_t T, int32_t K) {
  if (!pool || T <= 0 || K < 1 || pool->desc.num_experts < 1) return 0;
  return align256(mint_moe_lora_apply_workspace_bytes(pool, T, K)) + align256((size_t)T * K * pool->desc.n * 2);
}

extern "C" int32_t mint_moe_lora_apply_combine(const mint_pool *pool, const mint_slot_table *table, const void *plan_dev,
                                               int32_t T, int32_t K, const void *x_dev, int64_t ldx, int64_t x_rows,
                                               const int32_t *x_row_dev, const float *pair_weight_dev, void *y_dev,
                                               int64_t ldy, void *workspace_dev, size_t workspace_bytes,
                                               int32_t *status_dev, mint_stream_t stream) {
  if (!pool || !y_dev) return mint_fail(MINT_ERR_INVALID_ARG, "moe_apply_combine: null argument");
  if (!pair_weight_dev) return mint_fail(MINT_ERR_INVALID_ARG, "moe_apply_combine: the router's weights are required");
  if (T < 0 || K < 1) return mint_fail(MINT_ERR_INVALID_ARG, "moe_apply_combine: T=%d K=%d", T, K);
  if (T == 0) return MINT_OK;
  if ((reinterpret_cast<uintptr_t>(y_dev) & 15u) || (ldy & 7) || ldy < pool->desc.n)
    return mint_fail(MINT_ERR_MISALIGNED, "moe_apply_combine: y must be 16-byte aligned with a row stride >= n that is a multiple of 8");
  const size_t need = mint_moe_lora_apply_combine_workspace_bytes(pool, T, K);
  if (!workspace_dev || workspace_bytes < need)
    return mint_fail(MINT_ERR_WORKSPACE_TOO_SMALL, "moe_apply_combine: workspace %zu < %zu", workspace_bytes, need);
  if (reinterpret_cast<uintptr_t>(workspace_dev) & 255u)
    return mint_fail(MINT_ERR_MISALIGNED, "moe_apply_combine: workspace must be 256-byte aligned");
  const size_t apply_bytes = align256(mint_moe_lora_apply_workspace_bytes(pool, T, K));
  uint16_t *pair = reinterpret_cast<uint16_t *>(static_cast<char *>(workspace_dev) + apply_bytes);
  const int32_t n = pool->desc.n;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  int32_t st = mint_check_cuda(cudaMemsetAsync(pair, 0, (size_t)T * K * n * 2, s), "moe_apply_combine: clear scratch");
  if (st) return st;
  // (the memset is not a kernel: the apply's first kernel must not start early against it)
  mint_mark_tables_changed();
  st = mint_moe_lora_apply(pool, table, plan_dev, T, K, x_dev, ldx, x_rows, x_row_dev, pair_weight_dev, pair, n,
                           workspace_dev, apply_bytes, status_dev, stream);
  if (st) return st;
  const int64_t total = (int64_t)T * (n >> 3);
  int64_t blocks = (total + 255) / 256;
  if (blocks > 8 * 148) blocks = 8 * 148;
  combine_kernel<<<(unsigned)blocks, 256, 0, s>>>(pair, static_cast<uint16_t *>(y_dev), ldy, T, K, n);
  return mint_check_cuda(cudaGetLastError(), "combine launch");
}
