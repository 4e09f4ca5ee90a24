// Device-side helpers shared by the kernels of libmint_lora.so.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "mint_internal.h"

namespace mint {

// Record the first device-detected problem; later ones keep the first code.
__device__ __forceinline__ void report(int32_t *status, int32_t code, int32_t detail) {
  if (status == nullptr) return;
  if (atomicCAS(status, 0, code) == 0) status[2] = detail;
}

// 128-bit read-only load (weights and activations that are only read).
__device__ __forceinline__ uint4 ldg128(const void *p) {
  return __ldg(reinterpret_cast<const uint4 *>(p));
}
// Streaming variant: weights read once by one CTA need not stay in L1.
__device__ __forceinline__ uint4 ldg128_stream(const void *p) {
  uint4 r;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w)
               : "l"(p));
  return r;
}

// Two bf16 packed in a 32-bit word -> two floats (exact).
__device__ __forceinline__ float bf16lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16hi(uint32_t w) { return __uint_as_float(w & 0xFFFF0000u); }

__device__ __forceinline__ void unpack8(const uint4 &q, float (&f)[8]) {
  f[0] = bf16lo(q.x); f[1] = bf16hi(q.x);
  f[2] = bf16lo(q.y); f[3] = bf16hi(q.y);
  f[4] = bf16lo(q.z); f[5] = bf16hi(q.z);
  f[6] = bf16lo(q.w); f[7] = bf16hi(q.w);
}

// Two floats -> packed bf16x2, round to nearest even (low half = a).
__device__ __forceinline__ uint32_t pack_bf16x2(float a, float b) {
  __nv_bfloat162 h = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<uint32_t *>(&h);
}

__device__ __forceinline__ uint4 pack8(const float (&f)[8]) {
  uint4 q;
  q.x = pack_bf16x2(f[0], f[1]);
  q.y = pack_bf16x2(f[2], f[3]);
  q.z = pack_bf16x2(f[4], f[5]);
  q.w = pack_bf16x2(f[6], f[7]);
  return q;
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// A kernel consuming a plan first checks that the blob is a plan made for the
// same item count and under the slot table's current generation.
__device__ __forceinline__ bool plan_ok(const int32_t *hdr, int32_t T, int32_t K, int32_t num_slots,
                                        int32_t num_experts, int32_t gen_lo, int32_t gen_hi,
                                        int32_t *status) {
  if (hdr[PH_MAGIC] != MINT_PLAN_MAGIC || hdr[PH_T] != T || hdr[PH_K] != K ||
      hdr[PH_NUM_SLOTS] != num_slots || hdr[PH_NUM_EXPERTS] != num_experts) {
    if (threadIdx.x == 0) report(status, MINT_ERR_SHAPE_MISMATCH, hdr[PH_T]);
    return false;
  }
  if (hdr[PH_GEN_LO] != gen_lo || hdr[PH_GEN_HI] != gen_hi) {
    if (threadIdx.x == 0) report(status, MINT_ERR_STALE_PLAN, hdr[PH_GEN_LO]);
    return false;
  }
  return true;
}

}  // namespace mint
