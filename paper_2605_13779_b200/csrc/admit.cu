// Admission of an adapter revision into a GPU slot from the packed
// representation, and the residency bookkeeping of the slots.
//
// The paper's cold path ends with "admit L_r into a GPU batch slot" before any
// request may use the revision (section "Shared-Base Rollout and Serving"), and
// its serving evaluation finds MoE adapters object-bound on that path: tens of
// thousands of tiny per-expert tensors for about a hundred megabytes.  The
// packed serving representation stacks the per-expert tensors of a projection
// along an expert axis (packed MoE LoRA loader table: 37 248 tensors become
// 672).  Here the whole stacked pair of one projection goes into the slot of a
// pool with ONE kernel: A_packed[E][d][rank] -> A[slot][E][d][r_max] (a strided
// scatter when rank < r_max), B_packed[E][rank][n] -> B[slot][E][r_max][n];
// padding beyond the adapter's rank is left as it is.
//
// The slot manager is host-side bookkeeping over the bounded set of GPU slots
// (at most 64 distinct adapters in a decoding batch, cache-tier table of "Scale
// Out: Policy-Population Serving"; pinned adapters are tracked, "Worker
// admission and eviction"): least-recently-used order over the slots that no
// running step pins.
#include <new>

#include "mint_device.cuh"

namespace {

struct AdmitParams {
  uint16_t *A_dst;         // first element of the slot in the pool's A
  uint16_t *B_dst;
  const uint16_t *A_src;
  const uint16_t *B_src;
  int32_t experts;         // 1 for dense pools
  int32_t d, n, rank, r_max;
  int32_t packed;          // 1: A is [expert][d][r_max] (rank contiguous); 0: A is [r_max][d]
  int64_t a_chunks;        // work items of the A part (16-byte chunks, or elements)
  int64_t b_chunks;        // 16-byte chunks of the B part
  int32_t a_vec;           // 1: the A part moves 16-byte chunks; 0: single elements
};

__global__ void __launch_bounds__(256) admit_packed_kernel(const AdmitParams p) {
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  const int64_t tid = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  // ---- A ----
  if (!p.packed) {
    // rank rows of d elements, contiguous in source and slot
    const uint4 *src = reinterpret_cast<const uint4 *>(p.A_src);
    uint4 *dst = reinterpret_cast<uint4 *>(p.A_dst);
    for (int64_t q = tid; q < p.a_chunks; q += stride) dst[q] = mint::ldg128_stream(src + q);
  } else if (p.a_vec) {
    // rows of `rank` elements (a multiple of 8) into rows of r_max elements
    const int cpr = p.rank >> 3;   // 16-byte chunks per row
    for (int64_t q = tid; q < p.a_chunks; q += stride) {
      const int64_t row = q / cpr;
      const int c = (int)(q - row * cpr);
      *reinterpret_cast<uint4 *>(p.A_dst + row * p.r_max + c * 8) =
          mint::ldg128_stream(p.A_src + row * p.rank + c * 8);
    }
  } else {
    for (int64_t q = tid; q < p.a_chunks; q += stride) {
      const int64_t row = q / p.rank;
      const int j = (int)(q - row * p.rank);
      p.A_dst[row * p.r_max + j] = p.A_src[q];
    }
  }
  // ---- B: per expert, rank rows of n elements into the first rows of an r_max x n block ----
  const int64_t per_expert = (int64_t)p.rank * p.n / 8;
  for (int64_t q = tid; q < p.b_chunks; q += stride) {
    const int64_t e = q / per_expert;
    const int64_t rem = q - e * per_expert;
    *reinterpret_cast<uint4 *>(p.B_dst + e * (int64_t)p.r_max * p.n + rem * 8) =
        mint::ldg128_stream(p.B_src + q * 8);
  }
}

}  // namespace

extern "C" int32_t mint_pool_admit_packed(mint_pool *pool, int32_t slot, const void *A_packed_dev,
                                          const void *B_packed_dev, int32_t rank, mint_stream_t stream) {
  if (!pool || !A_packed_dev || !B_packed_dev) return mint_fail(MINT_ERR_INVALID_ARG, "admit_packed: null argument");
  const mint_pool_desc &p = pool->desc;
  if (slot < 0 || slot >= p.num_slots)
    return mint_fail(MINT_ERR_INVALID_ARG, "admit_packed: slot %d out of range", slot);
  if (rank < 1) return mint_fail(MINT_ERR_INVALID_ARG, "admit_packed: rank %d", rank);
  if (rank > p.r_max)
    return mint_fail(MINT_ERR_RANK_TOO_LARGE, "admit_packed: rank %d > r_max %d", rank, p.r_max);
  if ((reinterpret_cast<uintptr_t>(A_packed_dev) & 15u) || (reinterpret_cast<uintptr_t>(B_packed_dev) & 15u))
    return mint_fail(MINT_ERR_MISALIGNED, "admit_packed: sources must be 16-byte aligned");
  AdmitParams a = {};
  const bool packed = p.layout == MINT_LAYOUT_PACKED_MOE;
  const int64_t E = packed ? p.num_experts : 1;
  a.A_dst = static_cast<uint16_t *>(p.A_dev) + (int64_t)slot * E * p.d * p.r_max;
  a.B_dst = static_cast<uint16_t *>(p.B_dev) + (int64_t)slot * E * p.r_max * p.n;
  a.A_src = static_cast<const uint16_t *>(A_packed_dev);
  a.B_src = static_cast<const uint16_t *>(B_packed_dev);
  a.experts = (int32_t)E;
  a.d = p.d;
  a.n = p.n;
  a.rank = rank;
  a.r_max = p.r_max;
  a.packed = packed ? 1 : 0;
  if (!packed) {
    a.a_vec = 1;
    a.a_chunks = (int64_t)rank * p.d / 8;
  } else if ((rank & 7) == 0 && (p.r_max & 7) == 0) {
    a.a_vec = 1;
    a.a_chunks = E * p.d * (rank / 8);
  } else {
    a.a_vec = 0;
    a.a_chunks = E * p.d * rank;
  }
  a.b_chunks = E * rank * p.n / 8;
  const int64_t work = a.a_chunks > a.b_chunks ? a.a_chunks : a.b_chunks;
  int64_t blocks = (work + 255) / 256;
  if (blocks > 4 * 148) blocks = 4 * 148;
  if (blocks < 1) blocks = 1;
  admit_packed_kernel<<<(unsigned)blocks, 256, 0, static_cast<cudaStream_t>(stream)>>>(a);
  return mint_check_cuda(cudaGetLastError(), "admit_packed launch");
}

// ---------------------------------------------------------------------------
// slot manager
// ---------------------------------------------------------------------------
struct mint_slot_manager {
  mint_slot_table *table;   // may be null: bookkeeping only
  int32_t num_slots;
  int64_t *id_of;           // [num_slots] resident id or -1
  int32_t *pins;            // [num_slots]
  int32_t *prev, *next;     // recency list over occupied slots; head = least recently used
  int32_t head, tail;
  // id -> slot: open addressing over 4 * num_slots entries (ids are sparse in a catalog of up to 10^6 and more)
  int64_t *key;
  int32_t *val;
  int32_t cap;
};

namespace {

uint32_t hash_id(int64_t id, int32_t cap) {
  uint64_t x = (uint64_t)id * 0x9E3779B97F4A7C15ull;
  return (uint32_t)(x >> 33) % (uint32_t)cap;
}
int32_t map_find(const mint_slot_manager *m, int64_t id) {
  for (uint32_t h = hash_id(id, m->cap);; h = (h + 1) % (uint32_t)m->cap) {
    if (m->key[h] == id) return m->val[h];
    if (m->key[h] == -1) return -1;   // (-2 marks a deleted entry: keep probing)
  }
}
void map_put(mint_slot_manager *m, int64_t id, int32_t slot) {
  for (uint32_t h = hash_id(id, m->cap);; h = (h + 1) % (uint32_t)m->cap)
    if (m->key[h] < 0) {
      m->key[h] = id;
      m->val[h] = slot;
      return;
    }
}
void map_erase(mint_slot_manager *m, int64_t id) {
  for (uint32_t h = hash_id(id, m->cap);; h = (h + 1) % (uint32_t)m->cap) {
    if (m->key[h] == id) {
      m->key[h] = -2;
      return;
    }
    if (m->key[h] == -1) return;
  }
}
// Deleted entries pile up with churn: rebuild the map from the slots when a probe could grow long.
void map_rebuild(mint_slot_manager *m) {
  for (int32_t i = 0; i < m->cap; ++i) m->key[i] = -1;
  for (int32_t s = 0; s < m->num_slots; ++s)
    if (m->id_of[s] >= 0) map_put(m, m->id_of[s], s);
}
void list_unlink(mint_slot_manager *m, int32_t s) {
  if (m->prev[s] >= 0) m->next[m->prev[s]] = m->next[s]; else m->head = m->next[s];
  if (m->next[s] >= 0) m->prev[m->next[s]] = m->prev[s]; else m->tail = m->prev[s];
  m->prev[s] = m->next[s] = -1;
}
void list_push_back(mint_slot_manager *m, int32_t s) {
  m->prev[s] = m->tail;
  m->next[s] = -1;
  if (m->tail >= 0) m->next[m->tail] = s; else m->head = s;
  m->tail = s;
}

}  // namespace

extern "C" int32_t mint_slot_manager_create(mint_slot_manager **out, int32_t num_slots, mint_slot_table *table) {
  if (!out) return mint_fail(MINT_ERR_INVALID_ARG, "slot_manager_create: null out");
  *out = nullptr;
  if (num_slots < 1 || num_slots > (1 << 24))
    return mint_fail(MINT_ERR_INVALID_ARG, "slot_manager_create: num_slots=%d", num_slots);
  if (table && table->num_slots != num_slots)
    return mint_fail(MINT_ERR_SHAPE_MISMATCH, "slot_manager_create: the table has %d slots, not %d", table->num_slots,
                     num_slots);
  if (table)
    for (int32_t s = 0; s < num_slots; ++s)
      if (table->slots_host[s].catalog_id >= 0)
        return mint_fail(MINT_ERR_INVALID_ARG, "slot_manager_create: slot %d of the table is already bound", s);
  mint_slot_manager *m = new (std::nothrow) mint_slot_manager;
  if (!m) return mint_fail(MINT_ERR_INVALID_ARG, "slot_manager_create: out of host memory");
  m->table = table;
  m->num_slots = num_slots;
  m->cap = 4 * num_slots + 8;
  m->id_of = new (std::nothrow) int64_t[num_slots];
  m->pins = new (std::nothrow) int32_t[num_slots];
  m->prev = new (std::nothrow) int32_t[num_slots];
  m->next = new (std::nothrow) int32_t[num_slots];
  m->key = new (std::nothrow) int64_t[m->cap];
  m->val = new (std::nothrow) int32_t[m->cap];
  if (!m->id_of || !m->pins || !m->prev || !m->next || !m->key || !m->val) {
    delete[] m->id_of; delete[] m->pins; delete[] m->prev; delete[] m->next; delete[] m->key; delete[] m->val;
    delete m;
    return mint_fail(MINT_ERR_INVALID_ARG, "slot_manager_create: out of host memory");
  }
  for (int32_t s = 0; s < num_slots; ++s) {
    m->id_of[s] = -1;
    m->pins[s] = 0;
    m->prev[s] = m->next[s] = -1;
  }
  for (int32_t i = 0; i < m->cap; ++i) m->key[i] = -1;
  m->head = m->tail = -1;
  *out = m;
  return MINT_OK;
}

extern "C" int32_t mint_slot_manager_destroy(mint_slot_manager *m) {
  if (m) {
    delete[] m->id_of; delete[] m->pins; delete[] m->prev; delete[] m->next; delete[] m->key; delete[] m->val;
    delete m;
  }
  return MINT_OK;
}

extern "C" int32_t mint_slot_manager_acquire(mint_slot_manager *m, int64_t catalog_id, int32_t rank, float scale,
                                             int32_t *slot_out, int32_t *admitted_out, int64_t *evicted_id_out,
                                             mint_stream_t stream) {
  if (!m || !slot_out || !admitted_out || !evicted_id_out)
    return mint_fail(MINT_ERR_INVALID_ARG, "slot_manager_acquire: null argument");
  if (catalog_id < 0) return mint_fail(MINT_ERR_INVALID_ARG, "slot_manager_acquire: id %lld", (long long)catalog_id);
  *evicted_id_out = -1;
  int32_t s = map_find(m, catalog_id);
  if (s >= 0) {   // resident: most recently used from now on
    list_unlink(m, s);
    list_push_back(m, s);
    ++m->pins[s];
    *slot_out = s;
    *admitted_out = 0;
    return MINT_OK;
  }
  // the lowest-numbered empty slot, else the least recently used one that nothing pins
  for (s = 0; s < m->num_slots && m->id_of[s] >= 0; ++s) {
  }
  int64_t victim = -1;
  if (s == m->num_slots) {
    for (s = m->head; s >= 0 && m->pins[s] > 0; s = m->next[s]) {
    }
    if (s < 0)
      return mint_fail(MINT_ERR_NOT_RESIDENT, "slot_manager_acquire: all %d slots are pinned by running steps",
                       m->num_slots);
    victim = m->id_of[s];
  }
  if (m->table) {   // the table checks the id and the rank before anything changes
    if (victim >= 0) {
      int32_t st = mint_slot_table_evict(m->table, victim, stream);
      if (st) return st;
    }
    int32_t st = mint_slot_table_bind(m->table, catalog_id, s, rank, scale, stream);
    if (st) {
      if (victim >= 0) {   // the victim is gone from the table: drop it here too
        map_erase(m, victim);
        list_unlink(m, s);
        m->id_of[s] = -1;
        *evicted_id_out = victim;
      }
      return st;
    }
  }
  if (victim >= 0) {
    map_erase(m, victim);
    list_unlink(m, s);
    m->id_of[s] = -1;
    *evicted_id_out = victim;
  }
  int32_t used = 0;   // entries and deleted entries of the map
  for (int32_t i = 0; i < m->cap; ++i) used += m->key[i] != -1;
  if (used * 2 > m->cap) map_rebuild(m);   // (from the slots as they are: the new id is not in yet)
  m->id_of[s] = catalog_id;
  m->pins[s] = 1;
  map_put(m, catalog_id, s);
  list_push_back(m, s);
  *slot_out = s;
  *admitted_out = 1;
  return MINT_OK;
}

extern "C" int32_t mint_slot_manager_release(mint_slot_manager *m, int64_t catalog_id) {
  if (!m) return mint_fail(MINT_ERR_INVALID_ARG, "slot_manager_release: null manager");
  const int32_t s = map_find(m, catalog_id);
  if (s < 0) return mint_fail(MINT_ERR_NOT_RESIDENT, "slot_manager_release: id %lld is not resident", (long long)catalog_id);
  if (m->pins[s] <= 0) return mint_fail(MINT_ERR_INVALID_ARG, "slot_manager_release: id %lld is not pinned", (long long)catalog_id);
  --m->pins[s];
  return MINT_OK;
}

extern "C" int32_t mint_slot_manager_lookup(const mint_slot_manager *m, int64_t catalog_id) {
  return m ? map_find(m, catalog_id) : -1;
}
