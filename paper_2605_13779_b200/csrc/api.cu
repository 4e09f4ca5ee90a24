// Host side of the C ABI: argument validation, the pool and slot-table
// handles, and the launch of each kernel on the caller's stream.
#include <stdarg.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <atomic>
#include <new>

#include "mint_device.cuh"

// ---------------------------------------------------------------------------
// errors
// ---------------------------------------------------------------------------
static thread_local char g_err[512] = "";

int32_t mint_fail(int32_t code, const char *fmt, ...) {
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(g_err, sizeof g_err, fmt, ap);
  va_end(ap);
  return code;
}

int32_t mint_check_cuda(cudaError_t e, const char *what) {
  if (e == cudaSuccess) return MINT_OK;
  return mint_fail(MINT_ERR_CUDA, "%s: %s", what, cudaGetErrorString(e));
}

int32_t mint_device_lanes(int32_t *lanes_out) {
  static int cached[64] = {0};
  int dev = 0;
  int32_t st = mint_check_cuda(cudaGetDevice(&dev), "cudaGetDevice");
  if (st) return st;
  if (dev < 0 || dev >= 64) return mint_fail(MINT_ERR_UNSUPPORTED, "device ordinal %d", dev);
  if (cached[dev] == 0) {
    int sms = 0;
    st = mint_check_cuda(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev), "SM count");
    if (st) return st;
    if (sms < 1) return mint_fail(MINT_ERR_CUDA, "device reports %d SMs", sms);
    const int lanes = sms * 3;   // three streaming CTAs per SM
    cached[dev] = lanes > MINT_MAX_LANES ? MINT_MAX_LANES : lanes;
  }
  *lanes_out = cached[dev];
  return MINT_OK;
}

static std::atomic<bool> g_tables_changed{false};
void mint_mark_tables_changed() { g_tables_changed.store(true, std::memory_order_release); }
bool mint_take_tables_changed() { return g_tables_changed.exchange(false, std::memory_order_acq_rel); }

extern "C" const char *mint_last_error_string(void) { return g_err; }

extern "C" const char *mint_status_name(int32_t s) {
  switch (s) {
    case MINT_OK: return "MINT_OK";
    case MINT_ERR_INVALID_ARG: return "MINT_ERR_INVALID_ARG";
    case MINT_ERR_NOT_RESIDENT: return "MINT_ERR_NOT_RESIDENT";
    case MINT_ERR_SHAPE_MISMATCH: return "MINT_ERR_SHAPE_MISMATCH";
    case MINT_ERR_RANK_TOO_LARGE: return "MINT_ERR_RANK_TOO_LARGE";
    case MINT_ERR_WORKSPACE_TOO_SMALL: return "MINT_ERR_WORKSPACE_TOO_SMALL";
    case MINT_ERR_MISALIGNED: return "MINT_ERR_MISALIGNED";
    case MINT_ERR_CUDA: return "MINT_ERR_CUDA";
    case MINT_ERR_TIMEOUT: return "MINT_ERR_TIMEOUT";
    case MINT_ERR_UNSUPPORTED: return "MINT_ERR_UNSUPPORTED";
    case MINT_ERR_STALE_PLAN: return "MINT_ERR_STALE_PLAN";
    case MINT_ERR_BAD_INDEX: return "MINT_ERR_BAD_INDEX";
    default: return "MINT_ERR_UNKNOWN";
  }
}

static bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
static const int64_t kMaxItems = 1ll << 24;

// ---------------------------------------------------------------------------
// small device kernels for the slot table
// ---------------------------------------------------------------------------
namespace {

__global__ void table_init_kernel(int32_t *id_to_slot, int64_t catalog_size, int32_t *slot_rank,
                                  float *slot_scale, int32_t num_slots) {
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < catalog_size; i += stride)
    id_to_slot[i] = -1;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < num_slots; i += stride) {
    slot_rank[i] = 0;
    slot_scale[i] = 0.f;
  }
}

// Entries are applied in order by one thread: later entries of a batch may
// rebind a slot an earlier one emptied.
__global__ void bind_kernel(int32_t *id_to_slot, int32_t *slot_rank, float *slot_scale,
                            const BindBatch b) {
  if (blockIdx.x != 0 || threadIdx.x != 0) return;
  for (int i = 0; i < b.count; ++i) {
    if (b.slot[i] < 0) {
      id_to_slot[b.id[i]] = -1;
      slot_rank[b.old_slot[i]] = 0;
      slot_scale[b.old_slot[i]] = 0.f;
    } else {
      id_to_slot[b.id[i]] = b.slot[i];
      slot_rank[b.slot[i]] = b.rank[i];
      slot_scale[b.slot[i]] = b.scale[i];
    }
  }
}

}  // namespace

int32_t mint_launch_table_init(int32_t *id_to_slot, int64_t catalog_size, int32_t *slot_rank,
                               float *slot_scale, int32_t num_slots, cudaStream_t s) {
  int64_t blocks = (catalog_size + 255) / 256;
  if (blocks > 1184) blocks = 1184;
  if (blocks < 1) blocks = 1;
  table_init_kernel<<<(unsigned)blocks, 256, 0, s>>>(id_to_slot, catalog_size, slot_rank, slot_scale,
                                                      num_slots);
  return mint_check_cuda(cudaGetLastError(), "slot table init launch");
}

int32_t mint_launch_bind(int32_t *id_to_slot, int32_t *slot_rank, float *slot_scale,
                         const BindBatch &batch, cudaStream_t s) {
  mint_mark_tables_changed();
  bind_kernel<<<1, 32, 0, s>>>(id_to_slot, slot_rank, slot_scale, batch);
  return mint_check_cuda(cudaGetLastError(), "slot table bind launch");
}

// ---------------------------------------------------------------------------
// pool
// ---------------------------------------------------------------------------
extern "C" int32_t mint_pool_create(mint_pool **out, const mint_pool_desc *desc) {
  if (!out || !desc) return mint_fail(MINT_ERR_INVALID_ARG, "pool_create: null argument");
  *out = nullptr;
  if (desc->d <= 0 || desc->n <= 0 || desc->r_max <= 0 || desc->num_slots <= 0 || desc->num_experts < 0)
    return mint_fail(MINT_ERR_INVALID_ARG, "pool_create: non-positive dimension");
  if ((desc->d & 7) || (desc->n & 7))
    return mint_fail(MINT_ERR_SHAPE_MISMATCH, "pool_create: d=%d and n=%d must be multiples of 8",
                     desc->d, desc->n);
  if (desc->r_max > mint::kRankCapHost)
    return mint_fail(MINT_ERR_RANK_TOO_LARGE, "pool_create: r_max=%d exceeds the supported %d",
                     desc->r_max, mint::kRankCapHost);
  if (desc->layout == MINT_LAYOUT_RANK_MAJOR) {
    if (desc->num_experts != 0)
      return mint_fail(MINT_ERR_UNSUPPORTED, "pool_create: rank-major layout is for dense pools (num_experts=0)");
  } else if (desc->layout == MINT_LAYOUT_PACKED_MOE) {
    if (desc->num_experts < 1)
      return mint_fail(MINT_ERR_INVALID_ARG, "pool_create: packed MoE layout needs num_experts >= 1");
  } else {
    return mint_fail(MINT_ERR_INVALID_ARG, "pool_create: unknown layout %d", desc->layout);
  }
  if (!desc->A_dev || !desc->B_dev) return mint_fail(MINT_ERR_INVALID_ARG, "pool_create: null storage");
  if (!aligned16(desc->A_dev) || !aligned16(desc->B_dev))
    return mint_fail(MINT_ERR_MISALIGNED, "pool_create: A_dev/B_dev must be 16-byte aligned");
  mint_pool *p = new (std::nothrow) mint_pool;
  if (!p) return mint_fail(MINT_ERR_INVALID_ARG, "pool_create: out of host memory");
  p->desc = *desc;
  *out = p;
  return MINT_OK;
}

extern "C" int32_t mint_pool_destroy(mint_pool *pool) {
  delete pool;
  return MINT_OK;
}

extern "C" int32_t mint_pool_write_slot(mint_pool *pool, int32_t slot, int32_t expert, const void *A_src,
                                        const void *B_src, int32_t rank, int32_t src_is_device,
                                        mint_stream_t stream) {
  if (!pool || !A_src || !B_src) return mint_fail(MINT_ERR_INVALID_ARG, "write_slot: null argument");
  const mint_pool_desc &p = pool->desc;
  if (slot < 0 || slot >= p.num_slots) return mint_fail(MINT_ERR_INVALID_ARG, "write_slot: slot %d out of range", slot);
  if (rank < 1) return mint_fail(MINT_ERR_INVALID_ARG, "write_slot: rank %d", rank);
  if (rank > p.r_max) return mint_fail(MINT_ERR_RANK_TOO_LARGE, "write_slot: rank %d > r_max %d", rank, p.r_max);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const cudaMemcpyKind kind = src_is_device ? cudaMemcpyDeviceToDevice : cudaMemcpyHostToDevice;
  uint16_t *A = static_cast<uint16_t *>(p.A_dev);
  uint16_t *B = static_cast<uint16_t *>(p.B_dev);
  if (p.layout == MINT_LAYOUT_RANK_MAJOR) {
    int32_t st = mint_check_cuda(cudaMemcpyAsync(A + (int64_t)slot * p.r_max * p.d, A_src,
                                                 (size_t)rank * p.d * 2, kind, s), "write_slot A");
    if (st) return st;
    return mint_check_cuda(cudaMemcpyAsync(B + (int64_t)slot * p.r_max * p.n, B_src,
                                           (size_t)rank * p.n * 2, kind, s), "write_slot B");
  }
  if (expert < 0 || expert >= p.num_experts)
    return mint_fail(MINT_ERR_INVALID_ARG, "write_slot: expert %d out of range", expert);
  const int64_t se = (int64_t)slot * p.num_experts + expert;
  int32_t st = mint_check_cuda(cudaMemcpy2DAsync(A + se * p.d * p.r_max, (size_t)p.r_max * 2, A_src,
                                                 (size_t)rank * 2, (size_t)rank * 2, (size_t)p.d, kind, s),
                               "write_slot A");
  if (st) return st;
  return mint_check_cuda(cudaMemcpyAsync(B + se * p.r_max * p.n, B_src, (size_t)rank * p.n * 2, kind, s),
                         "write_slot B");
}

// ---------------------------------------------------------------------------
// slot table
// ---------------------------------------------------------------------------
extern "C" int32_t mint_slot_table_create(mint_slot_table **out, int64_t catalog_size, int32_t num_slots,
                                          int32_t *id_to_slot_dev, int32_t *slot_rank_dev,
                                          float *slot_scale_dev, mint_stream_t stream) {
  if (!out) return mint_fail(MINT_ERR_INVALID_ARG, "slot_table_create: null out");
  *out = nullptr;
  if (catalog_size <= 0 || num_slots <= 0 || catalog_size > (1ll << 31) - 1)
    return mint_fail(MINT_ERR_INVALID_ARG, "slot_table_create: catalog_size=%lld num_slots=%d",
                     (long long)catalog_size, num_slots);
  if (!id_to_slot_dev || !slot_rank_dev || !slot_scale_dev)
    return mint_fail(MINT_ERR_INVALID_ARG, "slot_table_create: null device array");
  mint_slot_table *t = new (std::nothrow) mint_slot_table;
  if (!t) return mint_fail(MINT_ERR_INVALID_ARG, "slot_table_create: out of host memory");
  t->catalog_size = catalog_size;
  t->num_slots = num_slots;
  t->id_to_slot_dev = id_to_slot_dev;
  t->slot_rank_dev = slot_rank_dev;
  t->slot_scale_dev = slot_scale_dev;
  t->generation = 1;
  t->max_rank = 0;
  t->id_to_slot_host = static_cast<int32_t *>(malloc(sizeof(int32_t) * (size_t)catalog_size));
  t->slots_host = static_cast<SlotBinding *>(malloc(sizeof(SlotBinding) * (size_t)num_slots));
  if (!t->id_to_slot_host || !t->slots_host) {
    free(t->id_to_slot_host);
    free(t->slots_host);
    delete t;
    return mint_fail(MINT_ERR_INVALID_ARG, "slot_table_create: out of host memory");
  }
  for (int64_t i = 0; i < catalog_size; ++i) t->id_to_slot_host[i] = -1;
  for (int32_t i = 0; i < num_slots; ++i) t->slots_host[i] = SlotBinding{-1, 0, 0.f};
  int32_t st = mint_launch_table_init(id_to_slot_dev, catalog_size, slot_rank_dev, slot_scale_dev, num_slots,
                                      static_cast<cudaStream_t>(stream));
  if (st) {
    free(t->id_to_slot_host);
    free(t->slots_host);
    delete t;
    return st;
  }
  *out = t;
  return MINT_OK;
}

extern "C" int32_t mint_slot_table_destroy(mint_slot_table *t) {
  if (t) {
    free(t->id_to_slot_host);
    free(t->slots_host);
    delete t;
  }
  return MINT_OK;
}

extern "C" int64_t mint_slot_table_generation(const mint_slot_table *t) { return t ? t->generation : -1; }

static int32_t validate_bind(const mint_slot_table *t, int64_t id, int32_t slot, int32_t rank) {
  if (id < 0 || id >= t->catalog_size)
    return mint_fail(MINT_ERR_INVALID_ARG, "bind: catalog id %lld outside [0, %lld)", (long long)id,
                     (long long)t->catalog_size);
  if (slot < 0 || slot >= t->num_slots) return mint_fail(MINT_ERR_INVALID_ARG, "bind: slot %d out of range", slot);
  if (rank < 1) return mint_fail(MINT_ERR_INVALID_ARG, "bind: rank %d", rank);
  if (rank > mint::kRankCapHost) return mint_fail(MINT_ERR_RANK_TOO_LARGE, "bind: rank %d exceeds %d", rank, mint::kRankCapHost);
  if (t->id_to_slot_host[id] >= 0)
    return mint_fail(MINT_ERR_INVALID_ARG, "bind: id %lld is already resident in slot %d", (long long)id,
                     t->id_to_slot_host[id]);
  if (t->slots_host[slot].catalog_id >= 0)
    return mint_fail(MINT_ERR_INVALID_ARG, "bind: slot %d is occupied by id %lld", slot,
                     (long long)t->slots_host[slot].catalog_id);
  return MINT_OK;
}

extern "C" int32_t mint_slot_table_bind_many(mint_slot_table *t, int64_t count, const int64_t *ids,
                                             const int32_t *slots, const int32_t *ranks, const float *scales,
                                             mint_stream_t stream) {
  if (!t || count < 0 || (count > 0 && (!ids || !slots || !ranks || !scales)))
    return mint_fail(MINT_ERR_INVALID_ARG, "bind_many: null argument");
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  BindBatch b;
  b.count = 0;
  int32_t result = MINT_OK;
  auto flush = [&]() -> int32_t {
    if (b.count == 0) return MINT_OK;
    int32_t st = mint_launch_bind(t->id_to_slot_dev, t->slot_rank_dev, t->slot_scale_dev, b, s);
    b.count = 0;
    return st;
  };
  for (int64_t i = 0; i < count; ++i) {
    result = validate_bind(t, ids[i], slots[i], ranks[i]);
    if (result) break;
    t->id_to_slot_host[ids[i]] = slots[i];
    t->slots_host[slots[i]] = SlotBinding{ids[i], ranks[i], scales[i]};
    if (ranks[i] > t->max_rank) t->max_rank = ranks[i];
    ++t->generation;
    const int k = b.count++;
    b.id[k] = ids[i];
    b.slot[k] = slots[i];
    b.old_slot[k] = -1;
    b.rank[k] = ranks[i];
    b.scale[k] = scales[i];
    if (b.count == BindBatch::kMax) {
      int32_t st = flush();
      if (st) return st;
    }
  }
  int32_t st = flush();
  return result ? result : st;
}

extern "C" int32_t mint_slot_table_bind(mint_slot_table *t, int64_t id, int32_t slot, int32_t rank, float scale,
                                        mint_stream_t stream) {
  return mint_slot_table_bind_many(t, 1, &id, &slot, &rank, &scale, stream);
}

extern "C" int32_t mint_slot_table_evict(mint_slot_table *t, int64_t id, mint_stream_t stream) {
  if (!t) return mint_fail(MINT_ERR_INVALID_ARG, "evict: null table");
  if (id < 0 || id >= t->catalog_size)
    return mint_fail(MINT_ERR_INVALID_ARG, "evict: catalog id %lld outside the catalog", (long long)id);
  const int32_t slot = t->id_to_slot_host[id];
  if (slot < 0) return mint_fail(MINT_ERR_NOT_RESIDENT, "evict: id %lld is not resident", (long long)id);
  t->id_to_slot_host[id] = -1;
  t->slots_host[slot] = SlotBinding{-1, 0, 0.f};
  ++t->generation;
  int32_t mr = 0;
  for (int32_t i = 0; i < t->num_slots; ++i)
    if (t->slots_host[i].catalog_id >= 0 && t->slots_host[i].rank > mr) mr = t->slots_host[i].rank;
  t->max_rank = mr;
  BindBatch b;
  b.count = 1;
  b.id[0] = id;
  b.slot[0] = -1;
  b.old_slot[0] = slot;
  b.rank[0] = 0;
  b.scale[0] = 0.f;
  return mint_launch_bind(t->id_to_slot_dev, t->slot_rank_dev, t->slot_scale_dev, b,
                          static_cast<cudaStream_t>(stream));
}

static TableDev table_dev(const mint_slot_table *t) {
  TableDev d;
  d.id_to_slot = t->id_to_slot_dev;
  d.slot_rank = t->slot_rank_dev;
  d.slot_scale = t->slot_scale_dev;
  d.catalog_size = t->catalog_size;
  d.num_slots = t->num_slots;
  d.gen_lo = (int32_t)(t->generation & 0xffffffffll);
  d.gen_hi = (int32_t)(t->generation >> 32);
  return d;
}

// ---------------------------------------------------------------------------
// plan
// ---------------------------------------------------------------------------
static int32_t check_plan_shape(int32_t T, int32_t K, int32_t num_slots, int32_t num_experts, const char *who) {
  if (T < 0 || K < 1 || num_slots < 1 || num_experts < 0)
    return mint_fail(MINT_ERR_INVALID_ARG, "%s: T=%d K=%d num_slots=%d num_experts=%d", who, T, K, num_slots,
                     num_experts);
  if ((int64_t)T * K > kMaxItems)
    return mint_fail(MINT_ERR_UNSUPPORTED, "%s: T*K=%lld exceeds %lld items", who, (long long)T * K,
                     (long long)kMaxItems);
  if ((int64_t)num_slots * (num_experts > 0 ? num_experts : 1) > (1ll << 30))
    return mint_fail(MINT_ERR_UNSUPPORTED, "%s: key space too large", who);
  return MINT_OK;
}

extern "C" size_t mint_lora_plan_bytes(int32_t T, int32_t K, int32_t num_slots, int32_t num_experts) {
  if (check_plan_shape(T, K, num_slots, num_experts, "plan_bytes")) return 0;
  return (size_t)mint_plan_offsets((int64_t)T * K, (int64_t)num_slots * (num_experts > 0 ? num_experts : 1)).total;
}

extern "C" int32_t mint_lora_plan_layout(int32_t T, int32_t K, int32_t num_slots, int32_t num_experts,
                                         mint_plan_layout *out) {
  if (!out) return mint_fail(MINT_ERR_INVALID_ARG, "plan_layout: null out");
  int32_t st = check_plan_shape(T, K, num_slots, num_experts, "plan_layout");
  if (st) return st;
  const PlanOffsets o = mint_plan_offsets((int64_t)T * K, (int64_t)num_slots * (num_experts > 0 ? num_experts : 1));
  out->total_bytes = o.total;
  out->header_off = o.header;
  out->perm_off = o.perm;
  out->seg_start_off = o.seg_start;
  out->seg_key_off = o.seg_key;
  return MINT_OK;
}

extern "C" int32_t mint_lora_plan(const mint_slot_table *table, const int64_t *ids_dev, int32_t T,
                                  const int32_t *expert_ids_dev, int32_t K, int32_t num_experts,
                                  void *plan_dev, size_t plan_bytes, int32_t *status_dev,
                                  mint_stream_t stream) {
  if (!table || !plan_dev || !status_dev || (T > 0 && !ids_dev))
    return mint_fail(MINT_ERR_INVALID_ARG, "plan: null argument");
  int32_t st = check_plan_shape(T, K, table->num_slots, num_experts, "plan");
  if (st) return st;
  if (expert_ids_dev == nullptr && (K != 1 || num_experts != 0))
    return mint_fail(MINT_ERR_INVALID_ARG, "plan: a dense plan has K=1 and num_experts=0");
  if (expert_ids_dev != nullptr && num_experts < 1)
    return mint_fail(MINT_ERR_INVALID_ARG, "plan: a MoE plan needs num_experts >= 1");
  if (!aligned16(plan_dev)) return mint_fail(MINT_ERR_MISALIGNED, "plan: plan_dev must be 16-byte aligned");
  const size_t need = (size_t)mint_plan_offsets((int64_t)T * K, (int64_t)table->num_slots * (num_experts > 0 ? num_experts : 1)).total;
  if (plan_bytes < need)
    return mint_fail(MINT_ERR_WORKSPACE_TOO_SMALL, "plan: plan_bytes=%zu < %zu", plan_bytes, need);
  int32_t lanes = 0;
  if ((st = mint_device_lanes(&lanes))) return st;
  mint_mark_tables_changed();
  return mint_launch_plan(table_dev(table), ids_dev, T, expert_ids_dev, K, num_experts, lanes, plan_dev,
                          status_dev, static_cast<cudaStream_t>(stream));
}

extern "C" int32_t mint_plan_fetch_summary(const void *plan_dev, mint_plan_summary *out, mint_stream_t stream) {
  if (!plan_dev || !out) return mint_fail(MINT_ERR_INVALID_ARG, "fetch_summary: null argument");
  int32_t h[PH_WORDS];
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  int32_t st = mint_check_cuda(cudaMemcpyAsync(h, plan_dev, sizeof h, cudaMemcpyDeviceToHost, s), "fetch_summary copy");
  if (st) return st;
  st = mint_check_cuda(cudaStreamSynchronize(s), "fetch_summary sync");
  if (st) return st;
  if (h[PH_MAGIC] != MINT_PLAN_MAGIC) return mint_fail(MINT_ERR_INVALID_ARG, "fetch_summary: not a plan");
  out->num_items = h[PH_NUM_ITEMS];
  out->num_active = h[PH_NUM_ACTIVE];
  out->num_segments = h[PH_NUM_SEGMENTS];
  out->max_segment = h[PH_MAX_SEGMENT];
  out->sum_rank = h[PH_SUM_RANK];
  out->not_resident = h[PH_NOT_RESIDENT];
  out->bad_expert = h[PH_BAD_EXPERT];
  out->reserved = 0;
  out->generation = ((int64_t)(uint32_t)h[PH_GEN_HI] << 32) | (uint32_t)h[PH_GEN_LO];
  return MINT_OK;
}

// ---------------------------------------------------------------------------
// dense shrink / expand / fused
// ---------------------------------------------------------------------------
static int32_t check_dense(const mint_pool *pool, const mint_slot_table *table, const void *plan_dev, int32_t T,
                           const char *who) {
  if (!pool || !table || !plan_dev) return mint_fail(MINT_ERR_INVALID_ARG, "%s: null argument", who);
  if (T < 0 || T > kMaxItems) return mint_fail(MINT_ERR_INVALID_ARG, "%s: T=%d", who, T);
  if (pool->desc.layout != MINT_LAYOUT_RANK_MAJOR || pool->desc.num_experts != 0)
    return mint_fail(MINT_ERR_UNSUPPORTED, "%s: needs a dense rank-major pool", who);
  if (pool->desc.num_slots != table->num_slots)
    return mint_fail(MINT_ERR_SHAPE_MISMATCH, "%s: pool has %d slots, table has %d", who, pool->desc.num_slots,
                     table->num_slots);
  if (table->max_rank > pool->desc.r_max)
    return mint_fail(MINT_ERR_RANK_TOO_LARGE, "%s: a bound adapter has rank %d > pool r_max %d", who,
                     table->max_rank, pool->desc.r_max);
  return MINT_OK;
}

static int32_t check_act(const void *p, int64_t ld, int32_t width, const char *name, const char *who) {
  if (!p) return mint_fail(MINT_ERR_INVALID_ARG, "%s: null %s", who, name);
  if (!aligned16(p)) return mint_fail(MINT_ERR_MISALIGNED, "%s: %s must be 16-byte aligned", who, name);
  if (ld < width) return mint_fail(MINT_ERR_SHAPE_MISMATCH, "%s: row stride of %s (%lld) < width %d", who, name, (long long)ld, width);
  if (ld & 7) return mint_fail(MINT_ERR_MISALIGNED, "%s: row stride of %s (%lld) must be a multiple of 8", who, name, (long long)ld);
  return MINT_OK;
}

static DenseArgs dense_args(const mint_pool *pool, int32_t T) {
  DenseArgs a = {};
  a.A = static_cast<const uint16_t *>(pool->desc.A_dev);
  a.B = static_cast<const uint16_t *>(pool->desc.B_dev);
  a.d = pool->desc.d;
  a.n = pool->desc.n;
  a.r_max = pool->desc.r_max;
  a.num_slots = pool->desc.num_slots;
  a.T = T;
  return a;
}

extern "C" int32_t mint_lora_shrink(const mint_pool *pool, const mint_slot_table *table, const void *plan_dev,
                                    int32_t T, const void *x_dev, int64_t ldx, float *v_dev, int32_t *status_dev,
                                    mint_stream_t stream) {
  int32_t st = check_dense(pool, table, plan_dev, T, "shrink");
  if (st) return st;
  if (!status_dev) return mint_fail(MINT_ERR_INVALID_ARG, "shrink: null status_dev");
  if (T == 0) return MINT_OK;
  if ((st = check_act(x_dev, ldx, pool->desc.d, "x_dev", "shrink"))) return st;
  if (!v_dev) return mint_fail(MINT_ERR_INVALID_ARG, "shrink: null v_dev");
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  st = mint_check_cuda(cudaMemsetAsync(v_dev, 0, (size_t)T * pool->desc.r_max * sizeof(float), s), "shrink: clear v");
  if (st) return st;
  DenseArgs a = dense_args(pool, T);
  a.x = static_cast<const uint16_t *>(x_dev);
  a.ldx = ldx;
  a.v = v_dev;
  a.status = status_dev;
  return mint_launch_shrink(a, table_dev(table), plan_dev, s);
}

extern "C" int32_t mint_lora_expand(const mint_pool *pool, const mint_slot_table *table, const void *plan_dev,
                                    int32_t T, const float *v_dev, void *y_dev, int64_t ldy, int32_t *status_dev,
                                    mint_stream_t stream) {
  int32_t st = check_dense(pool, table, plan_dev, T, "expand");
  if (st) return st;
  if (!status_dev) return mint_fail(MINT_ERR_INVALID_ARG, "expand: null status_dev");
  if (T == 0) return MINT_OK;
  if ((st = check_act(y_dev, ldy, pool->desc.n, "y_dev", "expand"))) return st;
  if (!v_dev) return mint_fail(MINT_ERR_INVALID_ARG, "expand: null v_dev");
  DenseArgs a = dense_args(pool, T);
  a.y = static_cast<uint16_t *>(y_dev);
  a.ldy = ldy;
  a.v = const_cast<float *>(v_dev);
  a.status = status_dev;
  return mint_launch_expand(a, table_dev(table), plan_dev, static_cast<cudaStream_t>(stream));
}

extern "C" size_t mint_lora_apply_workspace_bytes(const mint_pool *pool, int32_t T) {
  if (!pool || T < 0) return 0;
  return mint_stream_workspace_bytes(T, pool->desc.num_slots, pool->desc.r_max);
}

static int32_t fill_item(const mint_apply_item &it, const mint_slot_table *table, const void *plan_dev, int32_t T,
                         int32_t *status_dev, bool need_ws, DenseArgs &a, const char *who) {
  int32_t st = check_dense(it.pool, table, plan_dev, T, who);
  if (st) return st;
  if ((st = check_act(it.x_dev, it.ldx, it.pool->desc.d, "x_dev", who))) return st;
  if ((st = check_act(it.y_dev, it.ldy, it.pool->desc.n, "y_dev", who))) return st;
  if (need_ws) {
    const size_t need = mint_lora_apply_workspace_bytes(it.pool, T);
    if (!it.workspace_dev || it.workspace_bytes < need)
      return mint_fail(MINT_ERR_WORKSPACE_TOO_SMALL, "%s: workspace %zu < %zu", who, it.workspace_bytes, need);
    if (reinterpret_cast<uintptr_t>(it.workspace_dev) & 255u)
      return mint_fail(MINT_ERR_MISALIGNED, "%s: workspace must be 256-byte aligned", who);
  }
  a = dense_args(it.pool, T);
  a.x = static_cast<const uint16_t *>(it.x_dev);
  a.ldx = it.ldx;
  a.y = static_cast<uint16_t *>(it.y_dev);
  a.ldy = it.ldy;
  a.status = status_dev;
  return MINT_OK;
}

extern "C" int32_t mint_lora_apply_fused_grouped(const mint_apply_item *items, int32_t count,
                                                 const mint_slot_table *table, const void *plan_dev, int32_t T,
                                                 int32_t *status_dev, mint_stream_t stream) {
  if (!items || count < 1 || count > MINT_MAX_GROUP)
    return mint_fail(MINT_ERR_INVALID_ARG, "apply_fused_grouped: count=%d (1..%d)", count, MINT_MAX_GROUP);
  if (!table || !status_dev) return mint_fail(MINT_ERR_INVALID_ARG, "apply_fused_grouped: null argument");
  if (T == 0) {
    for (int i = 0; i < count; ++i) {
      int32_t st = check_dense(items[i].pool, table, plan_dev, T, "apply_fused_grouped");
      if (st) return st;
    }
    return MINT_OK;
  }
  const bool stream_path = mint_stream_supported(table->max_rank);
  DenseArgs args[MINT_MAX_GROUP];
  void *ws[MINT_MAX_GROUP];
  for (int i = 0; i < count; ++i) {
    int32_t st = fill_item(items[i], table, plan_dev, T, status_dev, stream_path, args[i], "apply_fused_grouped");
    if (st) return st;
    ws[i] = items[i].workspace_dev;
  }
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (stream_path) return mint_launch_stream(args, count, table_dev(table), plan_dev, ws, s);
  // ranks above the streamed path's limit: one cluster kernel per projection
  for (int i = 0; i < count; ++i) {
    int32_t st = mint_launch_fused(args[i], table_dev(table), plan_dev, s);
    if (st) return st;
  }
  return MINT_OK;
}

extern "C" int32_t mint_lora_apply_fused(const mint_pool *pool, const mint_slot_table *table, const void *plan_dev,
                                         int32_t T, const void *x_dev, int64_t ldx, void *y_dev, int64_t ldy,
                                         void *workspace_dev, size_t workspace_bytes, int32_t *status_dev,
                                         mint_stream_t stream) {
  mint_apply_item it;
  it.pool = pool;
  it.x_dev = x_dev;
  it.ldx = ldx;
  it.y_dev = y_dev;
  it.ldy = ldy;
  it.workspace_dev = workspace_dev;
  it.workspace_bytes = workspace_bytes;
  return mint_lora_apply_fused_grouped(&it, 1, table, plan_dev, T, status_dev, stream);
}

// Self-test of the bounded device-side waits: the tensor-core shrink of the plan's dense segments
// alone, with its tensor-core work withheld, so that every wait of every CTA that has a tile runs out.
extern "C" int32_t mint_selftest_wait_timeout(const mint_pool *pool, const mint_slot_table *table,
                                              const void *plan_dev, int32_t T, const void *x_dev, int64_t ldx,
                                              void *workspace_dev, size_t workspace_bytes, int32_t *status_dev,
                                              mint_stream_t stream) {
  int32_t st = check_dense(pool, table, plan_dev, T, "selftest_wait_timeout");
  if (st) return st;
  if (!status_dev) return mint_fail(MINT_ERR_INVALID_ARG, "selftest_wait_timeout: null status_dev");
  if (T < MINT_DENSE_MIN_BATCH || !mint_stream_supported(table->max_rank))
    return mint_fail(MINT_ERR_UNSUPPORTED, "selftest_wait_timeout: needs a batch of at least %d tokens and ranks up to 64",
                     MINT_DENSE_MIN_BATCH);
  if ((st = check_act(x_dev, ldx, pool->desc.d, "x_dev", "selftest_wait_timeout"))) return st;
  const size_t need = mint_lora_apply_workspace_bytes(pool, T);
  if (!workspace_dev || workspace_bytes < need)
    return mint_fail(MINT_ERR_WORKSPACE_TOO_SMALL, "selftest_wait_timeout: workspace %zu < %zu", workspace_bytes, need);
  DenseArgs a = dense_args(pool, T);
  a.x = static_cast<const uint16_t *>(x_dev);
  a.ldx = ldx;
  a.status = status_dev;
  int32_t lanes = 0;
  if ((st = mint_device_lanes(&lanes))) return st;
  const int64_t tiles = mint_tile_upper_bound(1, T, table->num_slots);
  void *ws[1] = {workspace_dev};
  return mint_launch_dense_shrink(&a, 1, table_dev(table), plan_dev, ws, lanes, (int32_t)(tiles + MINT_MAX_LANES),
                                  (int32_t)tiles, static_cast<cudaStream_t>(stream), true);
}

// ---------------------------------------------------------------------------
// backward
// ---------------------------------------------------------------------------
static size_t align256(size_t v) { return (v + 255) & ~(size_t)255; }

// The pool with A and B in each other's place: B's rows (rank rows of n elements) are what the shrink
// wants of A, A's rows what the expand wants of B, so the forward kernels compute dy . B^T and (.) . A.
static mint_pool transposed_pool(const mint_pool *pool) {
  mint_pool t = *pool;
  t.desc.A_dev = pool->desc.B_dev;
  t.desc.B_dev = pool->desc.A_dev;
  t.desc.d = pool->desc.n;
  t.desc.n = pool->desc.d;
  return t;
}

extern "C" size_t mint_lora_backward_workspace_bytes(const mint_pool *pool, int32_t T) {
  if (!pool || T < 0) return 0;
  const mint_pool tp = transposed_pool(pool);
  // u and v, the workspace of the forward kernels on the exchanged pool (the shrink of dy, then the apply
  // that makes dx) and the one of the shrink of x on the pool itself
  return 2 * align256((size_t)T * pool->desc.r_max * sizeof(float)) +
         align256(mint_lora_apply_workspace_bytes(&tp, T)) + align256(mint_lora_apply_workspace_bytes(pool, T));
}

extern "C" int32_t mint_lora_backward(const mint_pool *pool, const mint_slot_table *table, const void *plan_dev,
                                      int32_t T, const void *x_dev, int64_t ldx, const void *dy_dev, int64_t lddy,
                                      void *dx_dev, int64_t lddx, float *dA_dev, float *dB_dev,
                                      void *workspace_dev, size_t workspace_bytes, int32_t *status_dev,
                                      mint_stream_t stream) {
  mint_backward_item it;
  it.pool = pool;
  it.x_dev = x_dev;
  it.ldx = ldx;
  it.dy_dev = dy_dev;
  it.lddy = lddy;
  it.dx_dev = dx_dev;
  it.lddx = lddx;
  it.dA_dev = dA_dev;
  it.dB_dev = dB_dev;
  it.workspace_dev = workspace_dev;
  it.workspace_bytes = workspace_bytes;
  return mint_lora_backward_grouped(&it, 1, table, plan_dev, T, status_dev, stream);
}

extern "C" int32_t mint_lora_backward_grouped(const mint_backward_item *items, int32_t count,
                                              const mint_slot_table *table, const void *plan_dev, int32_t T,
                                              int32_t *status_dev, mint_stream_t stream) {
  if (!items || count < 1 || count > MINT_MAX_GROUP)
    return mint_fail(MINT_ERR_INVALID_ARG, "backward: count=%d (1..%d)", count, MINT_MAX_GROUP);
  if (!table || !status_dev) return mint_fail(MINT_ERR_INVALID_ARG, "backward: null argument");
  int32_t st;
  mint_pool tp[MINT_MAX_GROUP];
  for (int i = 0; i < count; ++i) {
    const mint_backward_item &it = items[i];
    if ((st = check_dense(it.pool, table, plan_dev, T, "backward"))) return st;
    if (T == 0) continue;
    if ((st = check_act(it.x_dev, it.ldx, it.pool->desc.d, "x_dev", "backward"))) return st;
    if ((st = check_act(it.dy_dev, it.lddy, it.pool->desc.n, "dy_dev", "backward"))) return st;
    if (it.dx_dev && (st = check_act(it.dx_dev, it.lddx, it.pool->desc.d, "dx_dev", "backward"))) return st;
    if ((it.dA_dev == nullptr) != (it.dB_dev == nullptr))
      return mint_fail(MINT_ERR_INVALID_ARG, "backward: dA_dev and dB_dev come together (both or neither)");
    if ((it.dA_dev && !aligned16(it.dA_dev)) || (it.dB_dev && !aligned16(it.dB_dev)))
      return mint_fail(MINT_ERR_MISALIGNED, "backward: dA_dev and dB_dev must be 16-byte aligned");
    if ((it.pool->desc.d & 7) || (it.pool->desc.n & 7))
      return mint_fail(MINT_ERR_UNSUPPORTED, "backward: d and n must be multiples of 8");
    const size_t need = mint_lora_backward_workspace_bytes(it.pool, T);
    if (!it.workspace_dev || it.workspace_bytes < need)
      return mint_fail(MINT_ERR_WORKSPACE_TOO_SMALL, "backward: workspace %zu < %zu", it.workspace_bytes, need);
    if (reinterpret_cast<uintptr_t>(it.workspace_dev) & 255u)
      return mint_fail(MINT_ERR_MISALIGNED, "backward: workspace must be 256-byte aligned");
    tp[i] = transposed_pool(it.pool);
  }
  if (T == 0) return MINT_OK;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const TableDev tab = table_dev(table);
  // every item's workspace: u, v, the workspace of the kernels on the exchanged pool, the one of the shrink of x
  float *u[MINT_MAX_GROUP], *v[MINT_MAX_GROUP];
  void *ws_t[MINT_MAX_GROUP], *ws_n[MINT_MAX_GROUP];
  size_t ws_t_bytes[MINT_MAX_GROUP];
  for (int i = 0; i < count; ++i) {
    const size_t vbytes = align256((size_t)T * items[i].pool->desc.r_max * sizeof(float));
    char *ws = static_cast<char *>(items[i].workspace_dev);
    u[i] = reinterpret_cast<float *>(ws);
    v[i] = reinterpret_cast<float *>(ws + vbytes);
    ws_t[i] = ws + 2 * vbytes;
    ws_t_bytes[i] = align256(mint_lora_apply_workspace_bytes(&tp[i], T));
    ws_n[i] = ws + 2 * vbytes + ws_t_bytes[i];
  }
  // The usual training step wants everything of every item: then the shrink of dy through B's rows serves
  // twice, as u for dA and as the first half of the apply that makes dx (its parts stay in the workspace).
  bool everything = mint_stream_supported(table->max_rank);
  for (int i = 0; i < count; ++i) everything = everything && items[i].dx_dev && items[i].dA_dev;
  if (everything) {
    DenseArgs pu[MINT_MAX_GROUP], pv_[MINT_MAX_GROUP];
    GradJobHost jobs[2 * MINT_MAX_GROUP];
    for (int i = 0; i < count; ++i) {
      const mint_backward_item &it = items[i];
      pu[i] = dense_args(&tp[i], T);
      pu[i].x = static_cast<const uint16_t *>(it.dy_dev);
      pu[i].ldx = it.lddy;
      pu[i].y = static_cast<uint16_t *>(it.dx_dev);
      pu[i].ldy = it.lddx;
      pu[i].status = status_dev;
      pv_[i] = dense_args(it.pool, T);
      pv_[i].x = static_cast<const uint16_t *>(it.x_dev);
      pv_[i].ldx = it.ldx;
      pv_[i].status = status_dev;
      jobs[2 * i] = GradJobHost{u[i], static_cast<const uint16_t *>(it.x_dev), it.ldx, it.dA_dev, it.pool->desc.d,
                                it.pool->desc.r_max};
      jobs[2 * i + 1] = GradJobHost{v[i], static_cast<const uint16_t *>(it.dy_dev), it.lddy, it.dB_dev,
                                    it.pool->desc.n, it.pool->desc.r_max};
    }
    if ((st = mint_launch_stream_phases(pu, count, tab, plan_dev, ws_t, s, 1, u))) return st;
    if ((st = mint_launch_stream_phases(pv_, count, tab, plan_dev, ws_n, s, 1, v))) return st;
    if ((st = mint_launch_grad_weights(jobs, 2 * count, T, tab, plan_dev, status_dev, s))) return st;
    return mint_launch_stream_phases(pu, count, tab, plan_dev, ws_t, s, 2, nullptr);
  }
  // 1. the rank-space tensors u = dy . B^T and v = x . A^T of every item whose adapters are trained
  DenseArgs probs[2 * MINT_MAX_GROUP];
  void *pws[2 * MINT_MAX_GROUP];
  float *pv[2 * MINT_MAX_GROUP];
  GradJobHost jobs[2 * MINT_MAX_GROUP];
  int np = 0;
  for (int i = 0; i < count; ++i) {
    const mint_backward_item &it = items[i];
    if (!it.dA_dev) continue;
    probs[np] = dense_args(&tp[i], T);
    probs[np].x = static_cast<const uint16_t *>(it.dy_dev);
    probs[np].ldx = it.lddy;
    probs[np].status = status_dev;
    pws[np] = ws_t[i];
    pv[np] = u[i];
    jobs[np] = GradJobHost{u[i], static_cast<const uint16_t *>(it.x_dev), it.ldx, it.dA_dev, it.pool->desc.d,
                           it.pool->desc.r_max};
    ++np;
    probs[np] = dense_args(it.pool, T);
    probs[np].x = static_cast<const uint16_t *>(it.x_dev);
    probs[np].ldx = it.ldx;
    probs[np].status = status_dev;
    pws[np] = ws_n[i];
    pv[np] = v[i];
    jobs[np] = GradJobHost{v[i], static_cast<const uint16_t *>(it.dy_dev), it.lddy, it.dB_dev, it.pool->desc.n,
                           it.pool->desc.r_max};
    ++np;
  }
  if (np > 0) {
    if (mint_stream_supported(table->max_rank)) {
      for (int p0 = 0; p0 < np; p0 += MINT_MAX_GROUP) {   // the streamed shrink takes eight problems a launch
        const int m = np - p0 < MINT_MAX_GROUP ? np - p0 : MINT_MAX_GROUP;
        if ((st = mint_launch_stream_shrink_v(probs + p0, m, tab, plan_dev, pws + p0, pv + p0, s))) return st;
      }
    } else {
      for (int i = 0; i < count; ++i) {
        const mint_backward_item &it = items[i];
        if (!it.dA_dev) continue;
        if ((st = mint_lora_shrink(&tp[i], table, plan_dev, T, it.dy_dev, it.lddy, u[i], status_dev, stream))) return st;
        if ((st = mint_lora_shrink(it.pool, table, plan_dev, T, it.x_dev, it.ldx, v[i], status_dev, stream))) return st;
      }
    }
    // 2. dA and dB of all items in one launch
    if ((st = mint_launch_grad_weights(jobs, np, T, tab, plan_dev, status_dev, s))) return st;
  }
  // 3. dx of all items: the fused apply on the exchanged pools
  mint_apply_item ax[MINT_MAX_GROUP];
  int nx = 0;
  for (int i = 0; i < count; ++i) {
    const mint_backward_item &it = items[i];
    if (!it.dx_dev) continue;
    ax[nx].pool = &tp[i];
    ax[nx].x_dev = it.dy_dev;
    ax[nx].ldx = it.lddy;
    ax[nx].y_dev = it.dx_dev;
    ax[nx].ldy = it.lddx;
    ax[nx].workspace_dev = ws_t[i];
    ax[nx].workspace_bytes = ws_t_bytes[i];
    ++nx;
  }
  if (nx > 0) return mint_lora_apply_fused_grouped(ax, nx, table, plan_dev, T, status_dev, stream);
  return MINT_OK;
}

// ---------------------------------------------------------------------------
// MoE
// ---------------------------------------------------------------------------
extern "C" size_t mint_moe_lora_apply_workspace_bytes(const mint_pool *pool, int32_t T, int32_t K) {
  if (!pool || T <= 0 || K < 1 || pool->desc.num_experts < 1) return 0;
  // pools the streamed kernels do not take (r_max other than 8, 16, 32, 64) need no workspace
  if (!mint_stream_moe_supported(pool->desc.r_max, 0)) return 0;
  return mint_stream_moe_workspace_bytes((int64_t)T * K, (int64_t)pool->desc.num_slots * pool->desc.num_experts,
                                         pool->desc.r_max);
}

// Checks one MoE projection's arguments and fills its launch record.
static int32_t fill_moe(const mint_pool *pool, const mint_slot_table *table, int32_t T, int32_t K, const void *x_dev,
                        int64_t ldx, int64_t x_rows, const int32_t *x_row_dev, const float *pair_weight_dev,
                        void *y_dev, int64_t ldy, void *workspace_dev, size_t workspace_bytes, int32_t *status_dev,
                        const char *who, MoEArgs &a, bool &streamed) {
  if (!pool) return mint_fail(MINT_ERR_INVALID_ARG, "%s: null pool", who);
  if (pool->desc.layout != MINT_LAYOUT_PACKED_MOE || pool->desc.num_experts < 1)
    return mint_fail(MINT_ERR_UNSUPPORTED, "%s: needs a packed MoE pool", who);
  if (pool->desc.num_slots != table->num_slots)
    return mint_fail(MINT_ERR_SHAPE_MISMATCH, "%s: pool has %d slots, table has %d", who, pool->desc.num_slots,
                     table->num_slots);
  if (table->max_rank > pool->desc.r_max)
    return mint_fail(MINT_ERR_RANK_TOO_LARGE, "%s: a bound adapter has rank %d > pool r_max %d", who,
                     table->max_rank, pool->desc.r_max);
  streamed = false;
  if (T == 0) return MINT_OK;
  int32_t st;
  if ((st = check_act(x_dev, ldx, pool->desc.d, "x_dev", who))) return st;
  if ((st = check_act(y_dev, ldy, pool->desc.n, "y_dev", who))) return st;
  if (x_rows < 1) return mint_fail(MINT_ERR_INVALID_ARG, "%s: x_rows=%lld", who, (long long)x_rows);
  if (!x_row_dev && x_rows < (int64_t)T * K)
    return mint_fail(MINT_ERR_SHAPE_MISMATCH, "%s: identity rows need x_rows >= T*K", who);
  const size_t need = mint_moe_lora_apply_workspace_bytes(pool, T, K);
  if (need > 0 && (!workspace_dev || workspace_bytes < need))
    return mint_fail(MINT_ERR_WORKSPACE_TOO_SMALL, "%s: workspace %zu < %zu", who, workspace_bytes, need);
  a = MoEArgs{};
  a.A = static_cast<const uint16_t *>(pool->desc.A_dev);
  a.B = static_cast<const uint16_t *>(pool->desc.B_dev);
  a.d = pool->desc.d;
  a.n = pool->desc.n;
  a.r_max = pool->desc.r_max;
  a.num_slots = pool->desc.num_slots;
  a.num_experts = pool->desc.num_experts;
  a.T = T;
  a.K = K;
  a.x = static_cast<const uint16_t *>(x_dev);
  a.ldx = ldx;
  a.x_rows = x_rows;
  a.x_row = x_row_dev;
  a.pair_weight = pair_weight_dev;
  a.y = static_cast<uint16_t *>(y_dev);
  a.ldy = ldy;
  a.status = status_dev;
  streamed = need > 0 && mint_stream_moe_supported(pool->desc.r_max, table->max_rank);
  if (streamed && (reinterpret_cast<uintptr_t>(workspace_dev) & 15) != 0)
    return mint_fail(MINT_ERR_MISALIGNED, "%s: workspace_dev must be 16-byte aligned", who);
  return MINT_OK;
}

extern "C" int32_t mint_moe_lora_apply(const mint_pool *pool, const mint_slot_table *table, const void *plan_dev,
                                       int32_t T, int32_t K, const void *x_dev, int64_t ldx, int64_t x_rows,
                                       const int32_t *x_row_dev, const float *pair_weight_dev, void *y_dev,
                                       int64_t ldy, void *workspace_dev, size_t workspace_bytes,
                                       int32_t *status_dev, mint_stream_t stream) {
  mint_moe_apply_item it;
  it.pool = pool;
  it.x_dev = x_dev;
  it.ldx = ldx;
  it.y_dev = y_dev;
  it.ldy = ldy;
  it.workspace_dev = workspace_dev;
  it.workspace_bytes = workspace_bytes;
  return mint_moe_lora_apply_grouped(&it, 1, table, plan_dev, T, K, x_rows, x_row_dev, pair_weight_dev, status_dev,
                                     stream);
}

extern "C" int32_t mint_moe_lora_apply_grouped(const mint_moe_apply_item *items, int32_t count,
                                               const mint_slot_table *table, const void *plan_dev, int32_t T,
                                               int32_t K, int64_t x_rows, const int32_t *x_row_dev,
                                               const float *pair_weight_dev, int32_t *status_dev,
                                               mint_stream_t stream) {
  if (!items || count < 1 || count > MINT_MAX_GROUP)
    return mint_fail(MINT_ERR_INVALID_ARG, "moe_apply: count=%d (1..%d)", count, MINT_MAX_GROUP);
  if (!table || !plan_dev || !status_dev) return mint_fail(MINT_ERR_INVALID_ARG, "moe_apply: null argument");
  if (T < 0 || K < 1 || (int64_t)T * K > kMaxItems)
    return mint_fail(MINT_ERR_INVALID_ARG, "moe_apply: T=%d K=%d", T, K);
  MoEArgs args[MINT_MAX_GROUP];
  void *ws[MINT_MAX_GROUP];
  bool streamed[MINT_MAX_GROUP];
  bool all_streamed = true;
  for (int i = 0; i < count; ++i) {
    const mint_moe_apply_item &it = items[i];
    int32_t st = fill_moe(it.pool, table, T, K, it.x_dev, it.ldx, x_rows, x_row_dev, pair_weight_dev, it.y_dev,
                          it.ldy, it.workspace_dev, it.workspace_bytes, status_dev, "moe_apply", args[i], streamed[i]);
    if (st) return st;
    if (it.pool->desc.num_experts != items[0].pool->desc.num_experts)
      return mint_fail(MINT_ERR_SHAPE_MISMATCH, "moe_apply: the pools of a grouped call hold %d and %d experts",
                       items[0].pool->desc.num_experts, it.pool->desc.num_experts);
    ws[i] = it.workspace_dev;
    all_streamed = all_streamed && streamed[i];
  }
  if (T == 0) return MINT_OK;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (all_streamed) return mint_launch_stream_moe(args, count, table_dev(table), plan_dev, ws, s);
  // a pool the streamed kernels do not take: one call per projection
  for (int i = 0; i < count; ++i) {
    int32_t st = streamed[i] ? mint_launch_stream_moe(&args[i], 1, table_dev(table), plan_dev, &ws[i], s)
                             : mint_launch_moe(args[i], table_dev(table), plan_dev, s);
    if (st) return st;
  }
  return MINT_OK;
}

// ---- backward of per-expert LoRA tensors (packed MoE pools) -------------------------------
// Workspace: u and v ([T*K][r_max] fp32, pair order), then the streamed shrink's parts for dy . B^T and
// for x . A.
extern "C" size_t mint_moe_lora_backward_workspace_bytes(const mint_pool *pool, int32_t T, int32_t K) {
  if (!pool || T <= 0 || K < 1 || pool->desc.num_experts < 1) return 0;
  if (!mint_stream_moe_supported(pool->desc.r_max, 0)) return 0;
  const size_t parts = align256(mint_stream_moe_workspace_bytes(
      (int64_t)T * K, (int64_t)pool->desc.num_slots * pool->desc.num_experts, pool->desc.r_max));
  return 2 * align256((size_t)T * K * pool->desc.r_max * sizeof(float)) + 2 * parts;
}

extern "C" int32_t mint_moe_lora_backward(const mint_pool *pool, const mint_slot_table *table, const void *plan_dev,
                                          int32_t T, int32_t K, const void *x_dev, int64_t ldx, int64_t x_rows,
                                          const int32_t *x_row_dev, const float *pair_weight_dev,
                                          const void *dy_dev, int64_t lddy, void *dx_dev, int64_t lddx,
                                          float *dA_dev, float *dB_dev, void *workspace_dev, size_t workspace_bytes,
                                          int32_t *status_dev, mint_stream_t stream) {
  const char *who = "moe_backward";
  if (!pool || !table || !plan_dev || !status_dev) return mint_fail(MINT_ERR_INVALID_ARG, "%s: null argument", who);
  if (T < 0 || K < 1 || (int64_t)T * K > kMaxItems) return mint_fail(MINT_ERR_INVALID_ARG, "%s: T=%d K=%d", who, T, K);
  if ((dA_dev == nullptr) != (dB_dev == nullptr))
    return mint_fail(MINT_ERR_INVALID_ARG, "%s: dA_dev and dB_dev are given together or not at all", who);
  if (!dx_dev && !dA_dev) return mint_fail(MINT_ERR_INVALID_ARG, "%s: nothing to compute", who);
  MoEArgs a;
  bool streamed = false;
  // (the forward checks; y stands for dy here: same width, same row per pair)
  int32_t st = fill_moe(pool, table, T, K, x_dev, ldx, x_rows, x_row_dev, pair_weight_dev, const_cast<void *>(dy_dev),
                        lddy, workspace_dev, workspace_bytes, status_dev, who, a, streamed);
  if (st) return st;
  if (T == 0) return MINT_OK;
  if (!streamed)
    return mint_fail(MINT_ERR_UNSUPPORTED, "%s: pools of r_max 8, 16, 32 or 64 and ranks up to 64 only", who);
  if (dx_dev && (st = check_act(dx_dev, lddx, pool->desc.d, "dx_dev", who))) return st;
  const size_t need = mint_moe_lora_backward_workspace_bytes(pool, T, K);
  if (!workspace_dev || workspace_bytes < need)
    return mint_fail(MINT_ERR_WORKSPACE_TOO_SMALL, "%s: workspace %zu < %zu", who, workspace_bytes, need);
  if ((reinterpret_cast<uintptr_t>(workspace_dev) & 255) != 0)
    return mint_fail(MINT_ERR_MISALIGNED, "%s: workspace_dev must be 256-byte aligned", who);
  const int64_t pairs = (int64_t)T * K;
  const int32_t E = pool->desc.num_experts, r_max = pool->desc.r_max;
  char *w = static_cast<char *>(workspace_dev);
  float *u = reinterpret_cast<float *>(w);
  w += align256((size_t)pairs * r_max * sizeof(float));
  float *v = reinterpret_cast<float *>(w);
  w += align256((size_t)pairs * r_max * sizeof(float));
  void *parts_u = w;
  w += align256(mint_stream_moe_workspace_bytes(pairs, (int64_t)pool->desc.num_slots * E, r_max));
  void *parts_v = w;
  const TableDev tab = table_dev(table);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  // u = w * dy . B^T: B's blocks are rank rows of n elements, and row p of dy belongs to pair p
  MoEArgs au = a;
  au.A = a.B;
  au.d = a.n;
  au.x = static_cast<const uint16_t *>(dy_dev);
  au.ldx = lddy;
  au.x_rows = pairs;
  au.x_row = nullptr;
  if ((st = mint_launch_stream_moe_shrink_v(&au, 1, true, tab, plan_dev, &parts_u, &u, s))) return st;
  if (dx_dev &&
      (st = mint_launch_moe_dx(a.A, u, static_cast<uint16_t *>(dx_dev), lddx, a.d, r_max, T, K, E, tab, plan_dev,
                               status_dev, s)))
    return st;
  if (!dA_dev) return MINT_OK;
  // v = w * x . A, then both weight gradients in one launch
  if ((st = mint_launch_stream_moe_shrink_v(&a, 1, false, tab, plan_dev, &parts_v, &v, s))) return st;
  GradJobHost jobs[2];
  jobs[0].coef = u;
  jobs[0].act = a.x;
  jobs[0].ld = ldx;
  jobs[0].out = dA_dev;
  jobs[0].width = a.d;
  jobs[0].r_max = r_max;
  jobs[0].row_map = x_row_dev;
  jobs[0].act_rows = x_rows;
  jobs[0].packed = 1;
  jobs[1].coef = v;
  jobs[1].act = static_cast<const uint16_t *>(dy_dev);
  jobs[1].ld = lddy;
  jobs[1].out = dB_dev;
  jobs[1].width = a.n;
  jobs[1].r_max = r_max;
  return mint_launch_grad_weights(jobs, 2, T, tab, plan_dev, status_dev, s, K, E);
}
