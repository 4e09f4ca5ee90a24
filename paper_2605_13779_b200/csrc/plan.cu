// Segment planner: token -> adapter segmentation of one batch.
//
// The paper's serving engine runs a batch that holds several adapters at once
// (at most 64 distinct adapters in the GPU-batch tier, section "Scale Out:
// Policy-Population Serving"); grouping the batch by adapter is the engine's
// job.  This kernel produces the canonical stable grouping: work items (tokens,
// or (token, k) pairs for MoE) ordered by key = slot (dense) or
// expert*num_slots + slot (MoE), ties by item index; one segment per key.
//
// One CTA of 1024 threads.  The order is produced by a least-significant-digit
// radix sort over the key bits with digits of at most 8 bits.  Every pass is
// stable by construction and free of scheduling-dependent choices:
//   - warp w owns the contiguous item range [w*R, (w+1)*R) and walks it in
//     order, 32 items per step;
//   - count walk: per-warp digit histogram (match_any groups equal digits, the
//     group's lowest lane adds the group size);
//   - the histogram is scanned bin-major, warp-minor: items of a smaller digit
//     first, and inside one digit the items of a lower warp first;
//   - scatter walk: position = bin base + warp offset + rank inside the step.
// Items without an adapter get key = key_space (sorted last), so the active
// items form a prefix.  Segment boundaries and the derived tile lists are then
// found with block-wide prefix sums over contiguous runs per thread.
#include "mint_device.cuh"

namespace {

constexpr int kThreads = 1024;
constexpr int kWarps = 32;

struct PlanParams {
  TableDev tab;
  const int64_t *ids;
  const int32_t *expert_ids;
  int32_t T, K, E;
  int32_t P;
  int32_t key_space;   // num_slots * max(E, 1); also the key of inactive items
  int32_t npass;
  int32_t digit_bits;
  int32_t lanes;       // cost lanes G of the lane tables
  int32_t presort_ctas;   // > 0: the grid-wide counting sort has left sorted keys in key_b and the order in perm
  PlanOffsets off;
  char *blob;
  int32_t *status;
};

// Exclusive prefix sum of one int per thread over the block; returns the total.
__device__ int block_exclusive_scan(int val, int *warp_tot /*[kWarps + 1]*/, int &total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int inc = val;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    int nb = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += nb;
  }
  __syncthreads();  // warp_tot may still be read from a previous call
  if (lane == 31) warp_tot[warp] = inc;
  __syncthreads();
  if (warp == 0) {
    int w = warp_tot[lane];
    int winc = w;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      int nb = __shfl_up_sync(0xffffffffu, winc, o);
      if (lane >= o) winc += nb;
    }
    warp_tot[lane] = winc - w;
    if (lane == 31) warp_tot[kWarps] = winc;
  }
  __syncthreads();
  total = warp_tot[kWarps];
  return warp_tot[warp] + inc - val;
}

// Ordered compaction over positions 0 .. n-1 walked 1024 at a time (coalesced): pass A stores, per
// (chunk, warp), how many positions of the warp are flagged; scan_counts turns the counts into exclusive
// prefix sums (and returns the total); pass B then gives every flagged position its rank as
// cnt[chunk * 32 + warp] + the flagged lanes below it.  cnt holds chunks * 32 <= kCompactMax entries.
constexpr int kCompactMax = kWarps * 256;   // the radix sort's histogram array, free once the sort is done
__device__ int scan_counts(int32_t *cnt, int n_cnt, int *warp_tot) {
  constexpr int kPer = kCompactMax / kThreads;   // 8 consecutive entries per thread
  const int base = threadIdx.x * kPer;
  int v[kPer], sum = 0;
#pragma unroll
  for (int q = 0; q < kPer; ++q) {
    v[q] = base + q < n_cnt ? cnt[base + q] : 0;
    sum += v[q];
  }
  int total;
  int run = block_exclusive_scan(sum, warp_tot, total);
#pragma unroll
  for (int q = 0; q < kPer; ++q) {
    if (base + q < n_cnt) cnt[base + q] = run;
    run += v[q];
  }
  __syncthreads();
  return total;
}

// Key of item i (key_space: no adapter, or an error that is counted in cnt: 0 inactive, 1 not
// resident, 2 first missing token, 3 bad expert, 4 first bad item).  kFromZero: the counters started
// at zero (a memset), so the two minima are kept as maxima of 0x7fffffff - index.
template <bool kFromZero>
__device__ __forceinline__ int32_t item_key(const PlanParams &p, int i, int32_t *cnt) {
  const int t = i / p.K;
  const int64_t id = p.ids[t];
  int32_t key = p.key_space;
  if (id != -1) {
    int32_t slot = -1;
    if (id >= 0 && id < p.tab.catalog_size) slot = p.tab.id_to_slot[id];
    if (slot < 0 || slot >= p.tab.num_slots) {
      if (i == t * p.K) {
        atomicAdd(&cnt[1], 1);
        if (kFromZero) atomicMax(&cnt[2], 0x7fffffff - t); else atomicMin(&cnt[2], t);
      }
    } else if (p.expert_ids != nullptr) {
      const int32_t e = p.expert_ids[i];
      if (e < 0 || e >= p.E) {
        atomicAdd(&cnt[3], 1);
        if (kFromZero) atomicMax(&cnt[4], 0x7fffffff - i); else atomicMin(&cnt[4], i);
      } else {
        key = e * p.tab.num_slots + slot;
      }
    } else {
      key = slot;
    }
  }
  if (key == p.key_space) atomicAdd(&cnt[0], 1);
  return key;
}

// Programmatic dependent launch between the kernels of one plan: a kernel lets its successor become
// resident at once, and touches nothing before its own wait (which every CTA executes).
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// ---- grid-wide stable counting sort (many items, small key space) ---------------
// CTA c owns items [1024 c, 1024 c + 1024).  (1) keys and per-CTA key counts; (2) one CTA turns the
// counts into start positions, key-major and CTA-minor; (3) every CTA places its items: the warps
// take turns in warp order, and inside a warp an item's rank among equal keys is the number of
// lower lanes with that key, so equal keys keep their item order whatever the scheduling.
static_assert((mint_tile_tokens(0) & (mint_tile_tokens(0) - 1)) == 0 && (mint_tile_tokens(1) & (mint_tile_tokens(1) - 1)) == 0 &&
                  mint_tile_tokens_rank1(0) == mint_tile_tokens(0) && (mint_tile_tokens_rank1(1) & (mint_tile_tokens_rank1(1) - 1)) == 0,
              "the tile walks take run lengths as powers of two, and list 0 as one length");
constexpr int kPresortMaxKeys = 4096;   // key_space of the counting sort (bins = key_space + 1)

__global__ void __launch_bounds__(kThreads) presort_count_kernel(const PlanParams p) {
  __shared__ int32_t bins[kPresortMaxKeys + 1];
  pdl_launch_dependents();
  pdl_wait();
  int32_t *g = reinterpret_cast<int32_t *>(p.blob + p.off.cta_hist);
  int32_t *key_a = reinterpret_cast<int32_t *>(p.blob + p.off.key_a);
  const int nb = p.key_space + 1;
  for (int b = threadIdx.x; b < nb; b += kThreads) bins[b] = 0;
  __syncthreads();
  const int i = blockIdx.x * kThreads + threadIdx.x;
  if (i < p.P) {
    const int32_t key = item_key<true>(p, i, g);
    key_a[i] = key;
    atomicAdd(&bins[key], 1);
  }
  __syncthreads();
  int32_t *row = g + 16 + (size_t)blockIdx.x * nb;
  for (int b = threadIdx.x; b < nb; b += kThreads) row[b] = bins[b];
}

__global__ void __launch_bounds__(kThreads) presort_scan_kernel(const PlanParams p) {
  __shared__ int32_t base[kPresortMaxKeys + 1 + 8];
  __shared__ int warp_tot[kWarps + 1];
  pdl_launch_dependents();
  pdl_wait();
  int32_t *hist = reinterpret_cast<int32_t *>(p.blob + p.off.cta_hist) + 16;
  const int nb = p.key_space + 1, C = p.presort_ctas;
  for (int b = threadIdx.x; b < nb; b += kThreads) {   // counts -> offsets inside the key, CTA-minor
    int run = 0;
    for (int c0 = 0; c0 < C; c0 += 16) {   // (sixteen loads go out together)
      int v[16];
#pragma unroll
      for (int q = 0; q < 16; ++q) v[q] = c0 + q < C ? __ldcg(hist + (size_t)(c0 + q) * nb + b) : 0;
#pragma unroll
      for (int q = 0; q < 16; ++q) {
        if (c0 + q < C) hist[(size_t)(c0 + q) * nb + b] = run;
        run += v[q];
      }
    }
    base[b] = run;
  }
  __syncthreads();
  constexpr int kPer = (kPresortMaxKeys + 1 + kThreads - 1) / kThreads;   // consecutive keys per thread
  const int b0 = threadIdx.x * kPer;
  int v[kPer], sum = 0;
#pragma unroll
  for (int q = 0; q < kPer; ++q) {
    v[q] = b0 + q < nb ? base[b0 + q] : 0;
    sum += v[q];
  }
  int total;
  int run = block_exclusive_scan(sum, warp_tot, total);
#pragma unroll
  for (int q = 0; q < kPer; ++q) {
    if (b0 + q < nb) base[b0 + q] = run;
    run += v[q];
  }
  __syncthreads();
  // row C of the table: where every key starts; the placing CTAs add it to their own row
  for (int b = threadIdx.x; b < nb; b += kThreads) hist[(size_t)C * nb + b] = base[b];

  // A key that has items is a segment, and its tiles follow from its item count: segments, and per
  // key the segment index and the first tile of either list (rows C + 1 .. C + 3; the placing CTAs
  // write the tile lists from them).  v[q] still holds the item count of key b0 + q.
  int32_t *g = reinterpret_cast<int32_t *>(p.blob + p.off.cta_hist);
  int32_t *seg_start = reinterpret_cast<int32_t *>(p.blob + p.off.seg_start);
  int32_t *seg_key = reinterpret_cast<int32_t *>(p.blob + p.off.seg_key);
  int32_t *seg_slot = reinterpret_cast<int32_t *>(p.blob + p.off.seg_slot);
  int32_t *seg_expert = reinterpret_cast<int32_t *>(p.blob + p.off.seg_expert);
  const bool dense_plan = p.expert_ids == nullptr && p.P >= MINT_DENSE_MIN_BATCH;
  int run1[kPer], n0 = 0, n1 = 0, ns = 0, max_seg = 0, sum_rank = 0;
#pragma unroll
  for (int q = 0; q < kPer; ++q) {
    run1[q] = mint_tile_tokens(1);
    if (b0 + q >= p.key_space || v[q] == 0) {   // (the last bin holds the items without an adapter)
      v[q] = 0;
      continue;
    }
    const int rank = p.tab.slot_rank[(b0 + q) % p.tab.num_slots];
    const bool dense_seg = dense_plan && v[q] >= MINT_DENSE_MIN_SEGMENT;
    if (rank == 1 && !dense_seg) run1[q] = mint_tile_tokens_rank1(1);
    ns += 1;
    n0 += (v[q] + mint_tile_tokens(0) - 1) / mint_tile_tokens(0);
    n1 += (v[q] + run1[q] - 1) / run1[q];
    max_seg = max(max_seg, v[q]);
    sum_rank += rank;
  }
  int S, T0, T1;
  int seg = block_exclusive_scan(ns, warp_tot, S);
  int t0 = block_exclusive_scan(n0, warp_tot, T0);
  int t1 = block_exclusive_scan(n1, warp_tot, T1);
  int32_t *row_seg = hist + (size_t)(C + 1) * nb, *row_t0 = hist + (size_t)(C + 2) * nb,
          *row_t1 = hist + (size_t)(C + 3) * nb;
#pragma unroll
  for (int q = 0; q < kPer; ++q) {
    if (v[q] == 0) continue;
    const int b = b0 + q;
    row_seg[b] = seg;
    row_t0[b] = t0;
    row_t1[b] = t1 | (run1[q] << 24);
    seg_start[seg] = base[b];
    seg_key[seg] = b;
    seg_slot[seg] = b % p.tab.num_slots;
    seg_expert[seg] = b / p.tab.num_slots;
    seg += 1;
    t0 += (v[q] + mint_tile_tokens(0) - 1) / mint_tile_tokens(0);
    t1 += (v[q] + run1[q] - 1) / run1[q];
  }
  if (max_seg > 0) atomicMax(&g[5], max_seg);
  if (sum_rank > 0) atomicAdd(&g[6], sum_rank);
  if (threadIdx.x == 0) {
    seg_start[S] = base[p.key_space];   // the active items
    g[7] = S;
    g[8] = T0;
    g[9] = T1;
  }
}

__global__ void __launch_bounds__(kThreads) presort_place_kernel(const PlanParams p) {
  __shared__ int32_t next[kPresortMaxKeys + 1];
  pdl_launch_dependents();
  pdl_wait();
  const int32_t *hist = reinterpret_cast<const int32_t *>(p.blob + p.off.cta_hist) + 16;
  const int32_t *key_a = reinterpret_cast<const int32_t *>(p.blob + p.off.key_a);
  int32_t *key_b = reinterpret_cast<int32_t *>(p.blob + p.off.key_b);
  int32_t *perm = reinterpret_cast<int32_t *>(p.blob + p.off.perm);
  int32_t *tseg0 = reinterpret_cast<int32_t *>(p.blob + p.off.tile_seg[0]);
  int32_t *toff0 = reinterpret_cast<int32_t *>(p.blob + p.off.tile_off[0]);
  int32_t *tseg1 = reinterpret_cast<int32_t *>(p.blob + p.off.tile_seg[1]);
  int32_t *toff1 = reinterpret_cast<int32_t *>(p.blob + p.off.tile_off[1]);
  const int nb = p.key_space + 1;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  for (int b = threadIdx.x; b < nb; b += kThreads)
    next[b] = hist[(size_t)blockIdx.x * nb + b] + hist[(size_t)p.presort_ctas * nb + b];
  const int i = blockIdx.x * kThreads + threadIdx.x;
  const bool live = i < p.P;
  const int32_t key = live ? key_a[i] : -1;
  const uint32_t grp = __match_any_sync(0xffffffffu, key);
  const int rank = __popc(grp & ((1u << lane) - 1u));
  __syncthreads();
  // the warps take their positions in warp order (shared memory only); the stores follow, all at once
  int pos = 0;
  for (int w = 0; w < kWarps; ++w) {
    if (warp == w && live) pos = next[key] + rank;
    __syncwarp();
    if (warp == w && live && rank == 0) next[key] += __popc(grp);
    __syncthreads();
  }
  if (!live) return;
  key_b[pos] = key;
  perm[pos] = i;
  if (key < p.key_space) {   // the first item of a tile lists the tile
    const int32_t *rows = hist + (size_t)p.presort_ctas * nb + key;   // start, segment, first tiles of the key
    const int off = pos - __ldg(rows);
    const int seg = __ldg(rows + nb), c0 = __ldg(rows + 2 * (size_t)nb), w1 = __ldg(rows + 3 * (size_t)nb);
    const int run1 = w1 >> 24;
    if ((off & (mint_tile_tokens(0) - 1)) == 0) {
      const int c = c0 + off / mint_tile_tokens(0);
      tseg0[c] = seg;
      toff0[c] = pos;
    }
    if ((off & (run1 - 1)) == 0) {
      const int c = (w1 & 0xffffff) + (off >> (31 - __clz(run1)));
      tseg1[c] = seg;
      toff1[c] = pos;
    }
  }
}

__global__ void __launch_bounds__(kThreads, 1) plan_kernel(const PlanParams p) {
  __shared__ int32_t hist[kWarps][256];
  __shared__ int32_t bin_base[256];
  __shared__ int warp_tot[kWarps + 1];
  __shared__ int32_t counters[9];  // 0 inactive, 1 not resident, 2 first missing token, 3 bad expert,
                                   // 4 first bad item, 5 max segment, 6 sum rank, 7 max tile rows,
                                   // 8 dense 128-row tiles whose tokens are not consecutive rows

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int P = p.P;
  pdl_wait();   // (launched programmatically behind the grid-wide sort; otherwise returns at once)
  int32_t *hdr = reinterpret_cast<int32_t *>(p.blob + p.off.header);
  int32_t *perm = reinterpret_cast<int32_t *>(p.blob + p.off.perm);
  int32_t *seg_start = reinterpret_cast<int32_t *>(p.blob + p.off.seg_start);
  int32_t *seg_key = reinterpret_cast<int32_t *>(p.blob + p.off.seg_key);
  int32_t *seg_slot = reinterpret_cast<int32_t *>(p.blob + p.off.seg_slot);
  int32_t *seg_expert = reinterpret_cast<int32_t *>(p.blob + p.off.seg_expert);
  int32_t *key_a = reinterpret_cast<int32_t *>(p.blob + p.off.key_a);
  int32_t *key_b = reinterpret_cast<int32_t *>(p.blob + p.off.key_b);
  int32_t *idx_a = reinterpret_cast<int32_t *>(p.blob + p.off.idx_a);
  int32_t *idx_b = reinterpret_cast<int32_t *>(p.blob + p.off.idx_b);

  if (tid < 9) counters[tid] = (tid == 2 || tid == 4) ? 0x7fffffff : 0;
  __syncthreads();

  // ---- keys: id -> slot through the table, (expert, slot) -> key ----------
  if (p.presort_ctas > 0) {   // done by the grid-wide sort, with its counters
    const int32_t *g = reinterpret_cast<const int32_t *>(p.blob + p.off.cta_hist);
    if (tid < 5) counters[tid] = (tid == 2 || tid == 4) ? 0x7fffffff - g[tid] : g[tid];   // (5, 6: further down)
  } else {
    for (int i = tid; i < P; i += kThreads) key_a[i] = item_key<false>(p, i, counters);
  }
  __syncthreads();

  // ---- stable LSD radix sort of (key, item index) ---------------------------
  const int R = (((P + kWarps - 1) / kWarps + 31) / 32) * 32;  // items per warp, multiple of 32
  const int w_begin = min(P, warp * R), w_end = min(P, (warp + 1) * R);
  const int nbins = 1 << p.digit_bits;
  for (int pass = 0; pass < (p.presort_ctas > 0 ? 0 : p.npass); ++pass) {
    const int32_t *kin = (pass & 1) ? key_b : key_a;
    int32_t *kout = (pass & 1) ? key_a : key_b;
    const int32_t *iin = (pass & 1) ? idx_b : idx_a;  // unused in pass 0 (index = position)
    int32_t *iout = (pass == p.npass - 1) ? perm : ((pass & 1) ? idx_a : idx_b);
    const int shift = pass * p.digit_bits;
    const uint32_t mask = (uint32_t)nbins - 1u;

    for (int i = tid; i < kWarps * 256; i += kThreads) (&hist[0][0])[i] = 0;
    __syncthreads();
    for (int base = w_begin; base < w_end; base += 32) {
      const int i = base + lane;
      const uint32_t dig = (i < w_end) ? (((uint32_t)kin[i] >> shift) & mask) : 0xFFFFFFFFu;
      const uint32_t grp = __match_any_sync(0xffffffffu, dig);
      if (i < w_end && lane == (__ffs(grp) - 1)) hist[warp][dig] += __popc(grp);
      __syncwarp();
    }
    __syncthreads();
    if (tid < nbins) {
      int run = 0;
      for (int w = 0; w < kWarps; ++w) {
        const int c = hist[w][tid];
        hist[w][tid] = run;
        run += c;
      }
      bin_base[tid] = run;
    }
    __syncthreads();
    if (warp == 0) {  // exclusive scan of the (up to 256) bin totals
      int v[8], s = 0;
#pragma unroll
      for (int q = 0; q < 8; ++q) {
        const int b = lane * 8 + q;
        v[q] = (b < nbins) ? bin_base[b] : 0;
        s += v[q];
      }
      int inc = s;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        int nb = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += nb;
      }
      int run = inc - s;
#pragma unroll
      for (int q = 0; q < 8; ++q) {
        const int b = lane * 8 + q;
        if (b < nbins) bin_base[b] = run;
        run += v[q];
      }
    }
    __syncthreads();
    for (int base = w_begin; base < w_end; base += 32) {
      const int i = base + lane;
      const bool live = i < w_end;
      const int32_t key = live ? kin[i] : 0;
      const uint32_t dig = live ? (((uint32_t)key >> shift) & mask) : 0xFFFFFFFFu;
      const uint32_t grp = __match_any_sync(0xffffffffu, dig);
      if (live) {
        const int rank = __popc(grp & ((1u << lane) - 1u));
        const int pos = bin_base[dig] + hist[warp][dig] + rank;
        kout[pos] = key;
        iout[pos] = (pass == 0) ? i : iin[i];
      }
      __syncwarp();
      if (live && lane == (__ffs(grp) - 1)) hist[warp][dig] += __popc(grp);
      __syncwarp();
    }
    __syncthreads();
  }
  const int32_t *skey = (p.presort_ctas > 0 || (p.npass & 1)) ? key_b : key_a;  // keys in sorted order
  const int n_active = P - counters[0];

  // ---- segments and tile lists ------------------------------------------------------
  const int run_len = (P + kThreads - 1) / kThreads;
  const int r_begin = min(n_active, tid * run_len), r_end = min(n_active, (tid + 1) * run_len);
  int S;
  int tile_total[MINT_NUM_TILE_LISTS];
  // dense segments (segmented prefill): dense plans of large batches only
  const bool dense_plan = p.expert_ids == nullptr && P >= MINT_DENSE_MIN_BATCH;
  auto tile_len = [&](int g, int sg) {   // the run length list g cuts segment sg into
    const bool dense_seg = dense_plan && seg_start[sg + 1] - seg_start[sg] >= MINT_DENSE_MIN_SEGMENT;
    return (p.tab.slot_rank[seg_slot[sg]] == 1 && !dense_seg) ? mint_tile_tokens_rank1(g) : mint_tile_tokens(g);
  };
  const int chunks = (n_active + kThreads - 1) / kThreads;
  if (p.presort_ctas > 0) {
    // the grid-wide sort has also written the segments and both tile lists (a key with items is a segment)
    const int32_t *g = reinterpret_cast<const int32_t *>(p.blob + p.off.cta_hist);
    S = g[7];
    tile_total[0] = g[8];
    tile_total[1] = g[9];
    if (tid == 0) {
      counters[5] = g[5];
      counters[6] = g[6];
    }
  } else if (chunks * kWarps <= kCompactMax) {
    // Coalesced walks (every batch of up to 262 144 items): a position is a segment head when its key
    // differs from the one before it, and a tile head of list g when its offset in its segment is a
    // multiple of the segment's run length.  Ordered compaction gives each head its index.
    int32_t *cnt = &hist[0][0];
    int32_t *seg_of = idx_a;   // segment of every position (the sort's scratch is free)
    int32_t *seg_run = idx_b;  // per segment: run length of list 0 | run length of list 1 << 8
    const unsigned below = (1u << lane) - 1u;
    auto is_head = [&](int i) { return i < n_active && (i == 0 || skey[i] != skey[i - 1]); };
    // (kU chunks per step: the loads that decide their flags go out together)
    constexpr int kU = 4;
    for (int c0 = 0; c0 < chunks; c0 += kU) {
      bool f[kU];
#pragma unroll
      for (int q = 0; q < kU; ++q) f[q] = is_head((c0 + q) * kThreads + tid);
#pragma unroll
      for (int q = 0; q < kU; ++q) {
        const unsigned b = __ballot_sync(0xffffffffu, f[q]);
        if (lane == 0 && c0 + q < chunks) cnt[(c0 + q) * kWarps + warp] = __popc(b);
      }
    }
    __syncthreads();
    S = scan_counts(cnt, chunks * kWarps, warp_tot);
    for (int c0 = 0; c0 < chunks; c0 += kU) {
      bool f[kU];
      int32_t k[kU];
#pragma unroll
      for (int q = 0; q < kU; ++q) {
        const int i = (c0 + q) * kThreads + tid;
        f[q] = is_head(i);
        k[q] = i < n_active ? skey[i] : 0;
      }
#pragma unroll
      for (int q = 0; q < kU; ++q) {
        const int i = (c0 + q) * kThreads + tid;
        const unsigned b = __ballot_sync(0xffffffffu, f[q]);
        if (i < n_active) {
          // heads at or before i, less one
          const int seg = cnt[(c0 + q) * kWarps + warp] + __popc(b & below) + (f[q] ? 1 : 0) - 1;
          seg_of[i] = seg;
          if (f[q]) {
            seg_start[seg] = i;
            seg_key[seg] = k[q];
            seg_slot[seg] = k[q] % p.tab.num_slots;
            seg_expert[seg] = k[q] / p.tab.num_slots;
          }
        }
      }
    }
    if (tid == 0) seg_start[S] = n_active;
    __syncthreads();
    for (int sg = tid; sg < S; sg += kThreads) {
      atomicMax(&counters[5], seg_start[sg + 1] - seg_start[sg]);
      atomicAdd(&counters[6], p.tab.slot_rank[seg_slot[sg]]);
      seg_run[sg] = tile_len(0, sg) | (tile_len(1, sg) << 8);
    }
    __syncthreads();
#pragma unroll
    for (int g = 0; g < MINT_NUM_TILE_LISTS; ++g) {
      int32_t *tseg = reinterpret_cast<int32_t *>(p.blob + p.off.tile_seg[g]);
      int32_t *toff = reinterpret_cast<int32_t *>(p.blob + p.off.tile_off[g]);
      auto tile_head = [&](int i, int &sg) {
        if (i >= n_active) return false;
        sg = seg_of[i];
        // (run lengths are powers of two; list 0 cuts every segment alike)
        const int G = g == 0 ? mint_tile_tokens(0) : (seg_run[sg] >> 8) & 255;
        return ((i - seg_start[sg]) & (G - 1)) == 0;
      };
      for (int c0 = 0; c0 < chunks; c0 += kU) {
        bool f[kU];
#pragma unroll
        for (int q = 0; q < kU; ++q) {
          int sg = 0;
          f[q] = tile_head((c0 + q) * kThreads + tid, sg);
        }
#pragma unroll
        for (int q = 0; q < kU; ++q) {
          const unsigned b = __ballot_sync(0xffffffffu, f[q]);
          if (lane == 0 && c0 + q < chunks) cnt[(c0 + q) * kWarps + warp] = __popc(b);
        }
      }
      __syncthreads();
      tile_total[g] = scan_counts(cnt, chunks * kWarps, warp_tot);
      for (int c0 = 0; c0 < chunks; c0 += kU) {
        bool f[kU];
        int sg[kU];
#pragma unroll
        for (int q = 0; q < kU; ++q) {
          sg[q] = 0;
          f[q] = tile_head((c0 + q) * kThreads + tid, sg[q]);
        }
#pragma unroll
        for (int q = 0; q < kU; ++q) {
          const unsigned b = __ballot_sync(0xffffffffu, f[q]);
          if (f[q]) {
            const int pos = cnt[(c0 + q) * kWarps + warp] + __popc(b & below);
            tseg[pos] = sg[q];
            toff[pos] = (c0 + q) * kThreads + tid;
          }
        }
      }
      __syncthreads();   // cnt is rewritten for the next list
    }
  } else {
  // (larger batches: every thread walks a contiguous run of positions)
  int heads = 0;
  for (int i = r_begin; i < r_end; ++i) heads += (i == 0 || skey[i] != skey[i - 1]);
  int seg = block_exclusive_scan(heads, warp_tot, S);
  for (int i = r_begin; i < r_end; ++i) {
    const int32_t k = skey[i];
    if (i == 0 || k != skey[i - 1]) {
      seg_start[seg] = i;
      seg_key[seg] = k;
      seg_slot[seg] = k % p.tab.num_slots;
      seg_expert[seg] = k / p.tab.num_slots;
      ++seg;
    }
  }
  if (tid == 0) seg_start[S] = n_active;
  __syncthreads();

  for (int s = tid; s < S; s += kThreads) {
    atomicMax(&counters[5], seg_start[s + 1] - seg_start[s]);
    atomicAdd(&counters[6], p.tab.slot_rank[seg_slot[s]]);
  }

  // Position i starts a tile of list g when (i - start of its segment) % G == 0.
  int s0 = 0;
  if (r_begin < r_end) {  // segment containing r_begin: last s with seg_start[s] <= r_begin
    int lo = 0, hi = S - 1;
    while (lo < hi) {
      const int mid = (lo + hi + 1) >> 1;
      if (seg_start[mid] <= r_begin) lo = mid; else hi = mid - 1;
    }
    s0 = lo;
  }
#pragma unroll
  for (int g = 0; g < MINT_NUM_TILE_LISTS; ++g) {
    int cnt = 0, s = s0;
    int G = r_begin < r_end ? tile_len(g, s) : 1;
    for (int i = r_begin; i < r_end; ++i) {
      while (i >= seg_start[s + 1]) {
        ++s;
        G = tile_len(g, s);
      }
      cnt += ((i - seg_start[s]) % G) == 0;
    }
    int pos = block_exclusive_scan(cnt, warp_tot, tile_total[g]);
    int32_t *tseg = reinterpret_cast<int32_t *>(p.blob + p.off.tile_seg[g]);
    int32_t *toff = reinterpret_cast<int32_t *>(p.blob + p.off.tile_off[g]);
    s = s0;
    G = r_begin < r_end ? tile_len(g, s) : 1;
    for (int i = r_begin; i < r_end; ++i) {
      while (i >= seg_start[s + 1]) {
        ++s;
        G = tile_len(g, s);
      }
      if (((i - seg_start[s]) % G) == 0) {
        tseg[pos] = s;
        toff[pos] = i;
        ++pos;
      }
    }
  }
  }
  __syncthreads();

  // ---- list-1 tile descriptors, their row prefix sums and the lane tables ----
  // A streaming kernel splits the rows x columns area of its work evenly over
  // G lanes; lane j starts inside the tile t with rows[t]*G <= j*rows_total,
  // which does not depend on the projection's width, so it is tabulated here.
  TileDesc *desc = reinterpret_cast<TileDesc *>(p.blob + p.off.tile_desc);
  LaneStart *lane_tab[2] = {reinterpret_cast<LaneStart *>(p.blob + p.off.lane_shrink),
                            reinterpret_cast<LaneStart *>(p.blob + p.off.lane_expand)};
  int rows_total[2];
  int num_dense = 0;
  {
    const int32_t *tseg = reinterpret_cast<const int32_t *>(p.blob + p.off.tile_seg[1]);
    const int32_t *toff = reinterpret_cast<const int32_t *>(p.blob + p.off.tile_off[1]);
    const int ntile = tile_total[1];
    const int per = (ntile + kThreads - 1) / kThreads;
    const int c_begin = min(ntile, tid * per), c_end = min(ntile, (tid + 1) * per);
    const bool dense_on = dense_plan;
    auto is_dense = [&](int sg) { return dense_on && seg_start[sg + 1] - seg_start[sg] >= MINT_DENSE_MIN_SEGMENT; };
    int sum_s = 0, sum_e = 0, sum_m = 0;
    for (int c = c_begin; c < c_end; ++c) {
      const int sg = tseg[c];
      const int len = min(tile_len(1, sg), seg_start[sg + 1] - toff[c]);
      const int r = p.tab.slot_rank[seg_slot[sg]];
      if (is_dense(sg)) {
        sum_m += ((toff[c] - seg_start[sg]) % 128) == 0;
      } else {
        sum_s += mint_tile_rows_shrink(r, len);
        atomicMax(&counters[7], mint_tile_rows_shrink(r, len));
      }
      if (!is_dense(sg)) sum_e += mint_tile_rows_expand(r, len);
    }
    int run_s = block_exclusive_scan(sum_s, warp_tot, rows_total[0]);
    int run_e = block_exclusive_scan(sum_e, warp_tot, rows_total[1]);
    int run_m = block_exclusive_scan(sum_m, warp_tot, num_dense);
    int32_t *dense_tile = reinterpret_cast<int32_t *>(p.blob + p.off.dense_tile);
    const int64_t G = p.lanes;
    for (int c = c_begin; c < c_end; ++c) {
      const int sg = tseg[c];
      const int slot = seg_slot[sg];
      TileDesc dsc;
      dsc.off = toff[c];
      dsc.len = min(tile_len(1, sg), seg_start[sg + 1] - toff[c]);
      dsc.slot = slot;
      dsc.expert = seg_expert[sg];
      dsc.rank = p.tab.slot_rank[slot];
      dsc.scale = p.tab.slot_scale[slot];
      dsc.rows_shrink = run_s;
      dsc.rows_expand = run_e;
      dsc.dense = is_dense(sg) ? 1 : 0;
      if (dsc.dense && ((toff[c] - seg_start[sg]) % 128) == 0) {
        // a 128-row tile of a dense segment; its tokens are consecutive rows (a request's tokens
        // usually are) when the last index is the first plus the count: then the tensor-core kernels
        // fetch it through tensor maps.  Scattered tiles are listed as ~c.
        const int rows128 = min(128, seg_start[sg + 1] - toff[c]);
        const bool scattered = perm[toff[c] + rows128 - 1] - perm[toff[c]] != rows128 - 1;
        if (scattered) atomicAdd(&counters[8], 1);
        dense_tile[run_m++] = scattered ? ~c : c;
      }
      const int begin[2] = {run_s, run_e};
      const int end[2] = {run_s + (dsc.dense ? 0 : mint_tile_rows_shrink(dsc.rank, dsc.len)),
                          run_e + (dsc.dense ? 0 : mint_tile_rows_expand(dsc.rank, dsc.len))};
      // shrink lanes that can meet this tile: from the last lane starting at or
      // before the tile's first row to the last lane starting before its end
      dsc.lane_lo = dsc.lane_hi = 0;
      if (!dsc.dense) {
        dsc.lane_lo = (int32_t)(begin[0] * G / rows_total[0]);
        dsc.lane_hi = (int32_t)min(G - 1, (end[0] * G - 1) / rows_total[0]);
      }
      dsc.pad1 = 0;
      desc[c] = dsc;
      // lanes whose start falls inside this tile: rows[c]*G <= j*total < rows[c+1]*G
#pragma unroll
      for (int q = 0; q < 2; ++q) {
        const int64_t tot = rows_total[q];
        if (tot == 0 || begin[q] == end[q]) continue;
        const int64_t j_lo = (begin[q] * G + tot - 1) / tot;
        const int64_t j_hi = (end[q] * G + tot - 1) / tot;   // exclusive
        for (int64_t j = j_lo; j < j_hi && j < G; ++j) {
          lane_tab[q][j].tile = c;
          lane_tab[q][j].rows = begin[q];
          lane_tab[q][j].w = end[q] - begin[q];
        }
      }
      run_s = end[0];
      run_e = end[1];
    }
    for (int j = tid; j <= p.lanes; j += kThreads) {
#pragma unroll
      for (int q = 0; q < 2; ++q) {
        const int64_t jw = (int64_t)j * rows_total[q];
        lane_tab[q][j].q = (int32_t)(jw / G);
        lane_tab[q][j].r = (int32_t)(jw % G);
        lane_tab[q][j].pad[0] = lane_tab[q][j].pad[1] = lane_tab[q][j].pad[2] = 0;
        if (j == p.lanes || rows_total[q] == 0) {
          lane_tab[q][j].tile = (j == p.lanes) ? ntile : 0;
          lane_tab[q][j].rows = 0;
          lane_tab[q][j].w = 1;
        }
      }
    }
  }
  __syncthreads();

  if (tid == 0) {
    hdr[PH_MAGIC] = MINT_PLAN_MAGIC;
    hdr[PH_T] = p.T;
    hdr[PH_K] = p.K;
    hdr[PH_NUM_ITEMS] = P;
    hdr[PH_NUM_SLOTS] = p.tab.num_slots;
    hdr[PH_NUM_EXPERTS] = p.E;
    hdr[PH_NUM_ACTIVE] = n_active;
    hdr[PH_NUM_SEGMENTS] = S;
    hdr[PH_MAX_SEGMENT] = counters[5];
    hdr[PH_SUM_RANK] = counters[6];
    hdr[PH_NOT_RESIDENT] = counters[1];
    hdr[PH_BAD_EXPERT] = counters[3];
    hdr[PH_GEN_LO] = p.tab.gen_lo;
    hdr[PH_GEN_HI] = p.tab.gen_hi;
    hdr[PH_NCHUNK0] = tile_total[0];
    hdr[PH_NCHUNK1] = tile_total[1];
    hdr[PH_LANES] = p.lanes;
    hdr[PH_ROWS_SHRINK] = rows_total[0];
    hdr[PH_ROWS_EXPAND] = rows_total[1];
    hdr[PH_MAX_TILE_ROWS] = counters[7];
    hdr[PH_NUM_DENSE] = num_dense;
    hdr[PH_NUM_SCATTERED] = counters[8];
    for (int w = PH_NUM_SCATTERED + 1; w < PH_WORDS; ++w) hdr[w] = 0;
    if (counters[1] > 0) {
      mint::report(p.status, MINT_ERR_NOT_RESIDENT, counters[2]);
      if (p.status) atomicAdd(&p.status[1], counters[1]);
    }
    if (counters[3] > 0) mint::report(p.status, MINT_ERR_BAD_INDEX, counters[4]);
  }
}

int64_t align_up(int64_t v, int64_t a) { return (v + a - 1) / a * a; }

}  // namespace

PlanOffsets mint_plan_offsets(int64_t P, int64_t key_space) {
  PlanOffsets o;
  const int64_t n = (P > 0 ? P : 1);
  int64_t cur = 0;
  auto take = [&](int64_t count) {
    int64_t at = cur;
    cur = align_up(cur + count * 4, 256);
    return at;
  };
  o.header = take(PH_WORDS);
  o.perm = take(n);
  o.seg_start = take(n + 1);
  o.seg_key = take(n);
  o.seg_slot = take(n);
  o.seg_expert = take(n);
  for (int g = 0; g < MINT_NUM_TILE_LISTS; ++g) {
    o.tile_seg[g] = take(n);
    o.tile_off[g] = take(n);
  }
  o.tile_desc = take((mint_tile_upper_bound(1, P, key_space) + 1) * (int64_t)(sizeof(TileDesc) / 4));
  o.dense_tile = take(mint_tile_upper_bound(1, P, key_space) + 1);
  o.lane_shrink = take((MINT_MAX_LANES + 1) * (int64_t)(sizeof(LaneStart) / 4));
  o.lane_expand = take((MINT_MAX_LANES + 1) * (int64_t)(sizeof(LaneStart) / 4));
  o.key_a = take(n);
  o.key_b = take(n);
  o.idx_a = take(n);
  o.idx_b = take(n);
  o.cta_hist = cur;
  const int64_t ctas = mint_plan_presort_ctas(P, key_space);
  if (ctas > 0) o.cta_hist = take(16 + (ctas + 4) * (key_space + 1));
  o.total = cur;
  return o;
}

int32_t mint_plan_presort_ctas(int64_t P, int64_t key_space) {
  if (P < 4096 || P > 256 * (int64_t)kThreads || key_space > kPresortMaxKeys) return 0;
  return (int32_t)((P + kThreads - 1) / kThreads);
}

int64_t mint_tile_upper_bound(int g, int64_t P, int64_t key_space) {
  // (list 1 may cut rank-1 segments into runs of mint_tile_tokens_rank1)
  const int64_t G = mint_tile_tokens(g) < mint_tile_tokens_rank1(g) ? mint_tile_tokens(g) : mint_tile_tokens_rank1(g);
  const int64_t max_segments = key_space < P ? key_space : P;
  int64_t ub = P / G + max_segments;
  return ub < P ? ub : P;
}

PlanView mint_plan_view(const void *plan_dev, int64_t P, int64_t key_space) {
  const PlanOffsets o = mint_plan_offsets(P, key_space);
  const char *b = static_cast<const char *>(plan_dev);
  PlanView v;
  v.header = reinterpret_cast<const int32_t *>(b + o.header);
  v.perm = reinterpret_cast<const int32_t *>(b + o.perm);
  v.seg_start = reinterpret_cast<const int32_t *>(b + o.seg_start);
  v.seg_key = reinterpret_cast<const int32_t *>(b + o.seg_key);
  v.seg_slot = reinterpret_cast<const int32_t *>(b + o.seg_slot);
  v.seg_expert = reinterpret_cast<const int32_t *>(b + o.seg_expert);
  for (int g = 0; g < MINT_NUM_TILE_LISTS; ++g) {
    v.tile_seg[g] = reinterpret_cast<const int32_t *>(b + o.tile_seg[g]);
    v.tile_off[g] = reinterpret_cast<const int32_t *>(b + o.tile_off[g]);
  }
  v.tile_desc = reinterpret_cast<const TileDesc *>(b + o.tile_desc);
  v.dense_tile = reinterpret_cast<const int32_t *>(b + o.dense_tile);
  v.lane_shrink = reinterpret_cast<const LaneStart *>(b + o.lane_shrink);
  v.lane_expand = reinterpret_cast<const LaneStart *>(b + o.lane_expand);
  return v;
}

int32_t mint_launch_plan(const TableDev &tab, const int64_t *ids, int32_t T, const int32_t *expert_ids,
                         int32_t K, int32_t num_experts, int32_t lanes, void *plan_dev, int32_t *status,
                         cudaStream_t stream) {
  PlanParams p;
  p.lanes = lanes;
  p.tab = tab;
  p.ids = ids;
  p.expert_ids = expert_ids;
  p.T = T;
  p.K = K;
  p.E = num_experts;
  p.P = T * K;
  p.key_space = tab.num_slots * (num_experts > 0 ? num_experts : 1);
  int nbits = 1;
  while ((1ll << nbits) <= (long long)p.key_space) ++nbits;  // key_space itself must fit
  p.npass = (nbits + 7) / 8;
  p.digit_bits = (nbits + p.npass - 1) / p.npass;
  p.off = mint_plan_offsets(p.P, p.key_space);
  p.blob = static_cast<char *>(plan_dev);
  p.status = status;
  p.presort_ctas = mint_plan_presort_ctas(p.P, p.key_space);
  if (p.presort_ctas > 0) {
    int32_t st = mint_check_cuda(cudaMemsetAsync(p.blob + p.off.cta_hist, 0, 64, stream), "plan counters");
    if (st) return st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.blockDim = dim3(kThreads);
    cfg.stream = stream;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cfg.gridDim = dim3((unsigned)p.presort_ctas);
    if ((st = mint_check_cuda(cudaLaunchKernelEx(&cfg, presort_count_kernel, p), "plan sort (count) launch"))) return st;
    cfg.gridDim = dim3(1);
    if ((st = mint_check_cuda(cudaLaunchKernelEx(&cfg, presort_scan_kernel, p), "plan sort (scan) launch"))) return st;
    cfg.gridDim = dim3((unsigned)p.presort_ctas);
    if ((st = mint_check_cuda(cudaLaunchKernelEx(&cfg, presort_place_kernel, p), "plan sort (place) launch"))) return st;
    cfg.gridDim = dim3(1);
    return mint_check_cuda(cudaLaunchKernelEx(&cfg, plan_kernel, p), "plan kernel launch");
  }
  plan_kernel<<<1, kThreads, 0, stream>>>(p);
  return mint_check_cuda(cudaGetLastError(), "plan kernel launch");
}
