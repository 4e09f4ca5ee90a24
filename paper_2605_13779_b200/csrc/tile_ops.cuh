// CUDA-core tile operations of the skinny (GEMV-like) LoRA path.
//
// A tile is a run of at most kTileRows work items of one segment: all of them
// use the same slot, so the slot's A and B rows are read once per tile and
// reused for every row of the tile from registers.
//
//   shrink: part[l][j] = sum over a range of d of x[row_l, i] * A[i, j]
//   expand: y[row_l, o] += scale_l * sum_j v[l][j] * B[j, o]   over a range of n
//
// Both walk their range in 128-bit vectors (8 bf16), accumulate in fp32 and
// are templated on the number of live rows LC so that short tiles (decode
// batches are mostly one or two tokens per adapter) do no padded work.
#pragma once
#include "mint_device.cuh"

namespace mint {

constexpr int kTileThreads = 256;
constexpr int kTileWarps = 8;
constexpr int kTileRows = 8;      // tile list 0
constexpr int kRankCap = kRankCapHost;  // largest slot rank the skinny path handles

struct TileSmem {
  int row_x[kTileRows];           // row of x read by tile row l
  int row_y[kTileRows];           // row of y updated by tile row l (-1: skip)
  float scale[kTileRows];         // s_slot * pair weight
  float part[kTileWarps][kTileRows][4];
  float vpart[kTileRows * kRankCap];  // this CTA's partial shrink result [l][r_stride]
  float vs[kTileRows * kRankCap];     // complete shrink result
};

// ---------------------------------------------------------------------------
// shrink over d-vectors [v0, v1) with A stored rank-major: A[j][d].
// Warps split (rank block of 4) x (d range); results land in out[l*r_stride+j].
// ---------------------------------------------------------------------------
template <int LC>
__device__ __forceinline__ void shrink_tile_rd(const uint16_t *__restrict__ A_slot, int d, int r,
                                               const uint16_t *__restrict__ x, int64_t ldx,
                                               TileSmem &sm, int v0, int v1, float *out,
                                               int r_stride) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int njb = (r + 3) >> 2;
  int JW = 1;
  while (JW < njb && JW < kTileWarps) JW <<= 1;
  const int DW = kTileWarps / JW;
  const int jw = warp % JW, dw = warp / JW;
  for (int jb0 = 0; jb0 < njb; jb0 += JW) {
    const int j0 = (jb0 + jw) * 4;
    const int nj = min(4, r - j0);
    float acc[LC][4];
#pragma unroll
    for (int l = 0; l < LC; ++l)
#pragma unroll
      for (int jj = 0; jj < 4; ++jj) acc[l][jj] = 0.f;
    if (nj > 0) {
      const uint16_t *a0 = A_slot + (int64_t)j0 * d;
      for (int v = v0 + dw * 32 + lane; v < v1; v += DW * 32) {
        float af[4][8];
#pragma unroll
        for (int jj = 0; jj < 4; ++jj) {
          uint4 q = make_uint4(0, 0, 0, 0);
          if (jj < nj) q = ldg128_stream(a0 + (int64_t)jj * d + v * 8);
          unpack8(q, af[jj]);
        }
#pragma unroll
        for (int l = 0; l < LC; ++l) {
          float xf[8];
          unpack8(ldg128(x + (int64_t)sm.row_x[l] * ldx + v * 8), xf);
#pragma unroll
          for (int jj = 0; jj < 4; ++jj)
#pragma unroll
            for (int e = 0; e < 8; ++e) acc[l][jj] = fmaf(xf[e], af[jj][e], acc[l][jj]);
        }
      }
    }
#pragma unroll
    for (int l = 0; l < LC; ++l)
#pragma unroll
      for (int jj = 0; jj < 4; ++jj) {
        const float s = warp_sum(acc[l][jj]);
        if (lane == 0) sm.part[warp][l][jj] = s;
      }
    __syncthreads();
    {
      const int t = threadIdx.x;
      if (t < JW * LC * 4) {
        const int jj = t & 3, l = (t >> 2) % LC, jq = t / (4 * LC);
        const int j = (jb0 + jq) * 4 + jj;
        if (j < r) {
          float s = 0.f;
          for (int q = 0; q < DW; ++q) s += sm.part[q * JW + jq][l][jj];
          out[l * r_stride + j] = s;
        }
      }
    }
    __syncthreads();
  }
}

// ---------------------------------------------------------------------------
// shrink over d-rows [i0, i1) (multiples of 8) with A stored d-major:
// A[i][r_max] (the packed MoE layout).  Every thread owns groups of 8
// consecutive d-rows; rank columns are taken 8 at a time.
// ---------------------------------------------------------------------------
template <int LC>
__device__ __forceinline__ void shrink_tile_dr(const uint16_t *__restrict__ A_e, int r_max, int r,
                                               const uint16_t *__restrict__ x, int64_t ldx,
                                               TileSmem &sm, int i0, int i1, float *out,
                                               int r_stride) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const bool vec_ok = (r_max & 7) == 0;
  float *red = &sm.part[0][0][0];  // [kTileWarps][LC*8] floats (LC <= 4)
  static_assert(LC * 8 <= kTileRows * 4, "reduction scratch too small");
  for (int j0 = 0; j0 < r; j0 += 8) {
    const int nj = min(8, r - j0);
    float acc[LC][8];
#pragma unroll
    for (int l = 0; l < LC; ++l)
#pragma unroll
      for (int jj = 0; jj < 8; ++jj) acc[l][jj] = 0.f;
    for (int i = i0 + threadIdx.x * 8; i < i1; i += kTileThreads * 8) {
      float xf[LC][8];
#pragma unroll
      for (int l = 0; l < LC; ++l) unpack8(ldg128(x + (int64_t)sm.row_x[l] * ldx + i), xf[l]);
#pragma unroll
      for (int ii = 0; ii < 8; ++ii) {
        float af[8];
        const uint16_t *arow = A_e + (int64_t)(i + ii) * r_max + j0;
        if (vec_ok) {
          // columns at or beyond the rank may be padding: mask them after the load
          unpack8(ldg128_stream(arow), af);
#pragma unroll
          for (int jj = 0; jj < 8; ++jj) if (jj >= nj) af[jj] = 0.f;
        } else {
#pragma unroll
          for (int jj = 0; jj < 8; ++jj)
            af[jj] = (jj < nj) ? __uint_as_float(((uint32_t)__ldg(arow + jj)) << 16) : 0.f;
        }
#pragma unroll
        for (int l = 0; l < LC; ++l)
#pragma unroll
          for (int jj = 0; jj < 8; ++jj) acc[l][jj] = fmaf(xf[l][ii], af[jj], acc[l][jj]);
      }
    }
#pragma unroll
    for (int l = 0; l < LC; ++l)
#pragma unroll
      for (int jj = 0; jj < 8; ++jj) {
        const float s = warp_sum(acc[l][jj]);
        if (lane == 0) red[warp * (LC * 8) + l * 8 + jj] = s;
      }
    __syncthreads();
    if (threadIdx.x < LC * 8) {
      const int l = threadIdx.x >> 3, jj = threadIdx.x & 7;
      if (jj < nj) {
        float s = 0.f;
        for (int w = 0; w < kTileWarps; ++w) s += red[w * (LC * 8) + threadIdx.x];
        out[l * r_stride + j0 + jj] = s;
      }
    }
    __syncthreads();
  }
}

// ---------------------------------------------------------------------------
// expand over n-vectors [v0, v1): B stored [j][n].  One thread owns 8 output
// columns of every tile row; y is read, updated and stored exactly once.
// ---------------------------------------------------------------------------
template <int LC>
__device__ __forceinline__ void expand_tile(const uint16_t *__restrict__ B_slot, int n, int r,
                                            const float *vs, int r_stride, uint16_t *__restrict__ y,
                                            int64_t ldy, const TileSmem &sm, int v0, int v1) {
  for (int v = v0 + threadIdx.x; v < v1; v += kTileThreads) {
    float acc[LC][8];
#pragma unroll
    for (int l = 0; l < LC; ++l)
#pragma unroll
      for (int e = 0; e < 8; ++e) acc[l][e] = 0.f;
    const uint16_t *b0 = B_slot + (int64_t)v * 8;
#pragma unroll 4
    for (int j = 0; j < r; ++j) {
      float bf[8];
      unpack8(ldg128_stream(b0 + (int64_t)j * n), bf);
#pragma unroll
      for (int l = 0; l < LC; ++l) {
        const float vv = vs[l * r_stride + j];
#pragma unroll
        for (int e = 0; e < 8; ++e) acc[l][e] = fmaf(vv, bf[e], acc[l][e]);
      }
    }
#pragma unroll
    for (int l = 0; l < LC; ++l) {
      const int row = sm.row_y[l];
      if (row < 0) continue;
      uint4 *yp = reinterpret_cast<uint4 *>(y + (int64_t)row * ldy + (int64_t)v * 8);
      float yf[8];
      unpack8(*yp, yf);
      const float sc = sm.scale[l];
#pragma unroll
      for (int e = 0; e < 8; ++e) yf[e] = fmaf(sc, acc[l][e], yf[e]);
      *yp = pack8(yf);
    }
  }
}

}  // namespace mint
