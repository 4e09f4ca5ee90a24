/*
 * mint_lora.h -- C ABI of the mixed-adapter LoRA apply for NVIDIA B200 (sm_100a).
 *
 * One resident base model serves a batch in which every request names its own
 * LoRA adapter revision (paper, section "Shared-Base Rollout and Serving").
 * For every token t with adapter a(t), resident in GPU slot sigma:
 *
 *        y[t, :] += s_sigma * (x[t, :] . A_sigma) . B_sigma
 *
 * A_sigma is d x r_sigma, B_sigma is r_sigma x n, s_sigma a per-adapter scalar.
 * The paper delegates the apply to its serving engine and prints no equation;
 * this is the standard LoRA update it relies on (section "Related Work").
 *
 * General rules for every call
 *  - Returns an int32_t status: MINT_OK or a negative MINT_ERR_* code.  Nothing
 *    is thrown across the boundary; mint_last_error_string() gives the detail
 *    for the calling thread.
 *  - Pointers named *_dev are DEVICE pointers, everything else is HOST memory.
 *  - All device buffers (activations, pools, tables, plans, workspaces, status
 *    words) are allocated and owned by the caller.  The library allocates no
 *    device memory.  Handles (mint_pool, mint_slot_table) are small host
 *    objects freed by their *_destroy call.
 *  - GPU work is enqueued on the caller's stream (a cudaStream_t passed as
 *    void*) and the call returns without synchronising, except
 *    mint_plan_fetch_summary, which waits for the stream.
 *  - bf16 tensors: device pointers 16-byte aligned, d and n multiples of 8,
 *    row strides (ldx, ldy, in elements) multiples of 8; otherwise
 *    MINT_ERR_MISALIGNED / MINT_ERR_SHAPE_MISMATCH and nothing is launched.
 *  - Problems only the device can see (an id that is not resident, an index out
 *    of range, a stale plan, a bounded wait that ran out) are recorded in the
 *    caller's status_dev words and the offending work is skipped; kernels never
 *    trap.  status_dev is MINT_STATUS_WORDS int32 that the caller zeroes:
 *      [0] first error code seen (sticky), [1] number of tokens whose id was
 *      not resident, [2] detail of the first error (token or item index),
 *      [3] reserved.
 */
#ifndef MINT_LORA_H
#define MINT_LORA_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef void *mint_stream_t; /* a cudaStream_t */

enum {
  MINT_OK = 0,
  MINT_ERR_INVALID_ARG = -1,
  MINT_ERR_NOT_RESIDENT = -2,        /* a token names an id bound to no slot          */
  MINT_ERR_SHAPE_MISMATCH = -3,      /* pool / table / plan shapes do not agree       */
  MINT_ERR_RANK_TOO_LARGE = -4,      /* rank exceeds the pool's configured r_max      */
  MINT_ERR_WORKSPACE_TOO_SMALL = -5,
  MINT_ERR_MISALIGNED = -6,
  MINT_ERR_CUDA = -7,                /* a CUDA runtime call failed                    */
  MINT_ERR_TIMEOUT = -8,             /* a bounded device-side wait ran out            */
  MINT_ERR_UNSUPPORTED = -9,
  MINT_ERR_STALE_PLAN = -10,         /* the slot table changed after the plan was made */
  MINT_ERR_BAD_INDEX = -11           /* expert id or row index out of range           */
};

#define MINT_STATUS_WORDS 4

/* Pool weight layouts.  Slots are allocated at the configured maximum rank
 * r_max and smaller adapters are padded (paper, "Time-Sliced Multi-LoRA
 * Training": slots at configured maximum shapes, smaller adapters padded and
 * inactive rows masked).  Only rows/columns below a slot's true rank are ever
 * read; padding may hold anything, NaN included.
 *   MINT_LAYOUT_RANK_MAJOR : A[slot][r_max][d],       B[slot][r_max][n]        dense projections
 *   MINT_LAYOUT_PACKED_MOE : A[slot][expert][d][r_max], B[slot][expert][r_max][n]
 *     the packed MoE representation: the per-expert tensors of one projection
 *     stacked along an expert axis (paper, packed MoE LoRA loader).           */
enum { MINT_LAYOUT_RANK_MAJOR = 0, MINT_LAYOUT_PACKED_MOE = 1 };

typedef struct {
  int32_t d;            /* input width                                    */
  int32_t n;            /* output width                                   */
  int32_t r_max;        /* slot rank stride                               */
  int32_t num_slots;
  int32_t num_experts;  /* 0 for a dense projection                       */
  int32_t layout;       /* MINT_LAYOUT_*                                  */
  void *A_dev;          /* bf16, caller-owned, 16-byte aligned            */
  void *B_dev;          /* bf16, caller-owned, 16-byte aligned            */
} mint_pool_desc;

typedef struct mint_pool mint_pool;
typedef struct mint_slot_table mint_slot_table;

const char *mint_last_error_string(void);
const char *mint_status_name(int32_t status);

/* ---- pool: the packed weights of ONE projection over all GPU slots -------
 * The GPU-batch tier of the paper's three cache tiers (at most 64 distinct
 * adapters resident for a decoding step; "Scale Out: Policy-Population
 * Serving").  create copies the descriptor; the storage stays the caller's. */
int32_t mint_pool_create(mint_pool **out, const mint_pool_desc *desc);
int32_t mint_pool_destroy(mint_pool *pool);

/* Admission of one adapter into a slot (the step that, in the paper's serving
 * path, puts an exported adapter revision into a GPU slot before any request
 * may use it): copy A_src (d x rank) and B_src (rank x n) into the slot, in the
 * pool's layout; expert is ignored (pass -1) for dense pools.  Sources are in
 * the pool's own element order with rank in place of r_max:
 *   RANK_MAJOR: A_src[rank][d], B_src[rank][n];  PACKED_MOE: A_src[d][rank], B_src[rank][n].
 * src_is_device selects host or device sources.  Padding is left untouched.  */
int32_t mint_pool_write_slot(mint_pool *pool, int32_t slot, int32_t expert, const void *A_src,
                             const void *B_src, int32_t rank, int32_t src_is_device,
                             mint_stream_t stream);

/* Admission of a whole adapter projection from the PACKED representation, with
 * one kernel: the paper's packed MoE LoRA serving representation stacks the
 * per-expert tensors of a projection along an expert axis so that a cold load
 * touches few objects (packed MoE LoRA loader table: 37 248 tensors become 672;
 * the load path was object-bound, not byte-bound).  Both sources are DEVICE
 * pointers, 16-byte aligned, bf16:
 *   PACKED_MOE pools: A_packed_dev[expert][d][rank], B_packed_dev[expert][rank][n]
 *                     -> A[slot][expert][d][r_max],  B[slot][expert][r_max][n]
 *   RANK_MAJOR pools: A_packed_dev[rank][d], B_packed_dev[rank][n]
 *                     -> A[slot][r_max][d],    B[slot][r_max][n]
 * Padding beyond the adapter's rank is left untouched.  The call only enqueues
 * the copy; binding the id to the slot is mint_slot_table_bind's job (or the
 * slot manager's, below), and must be enqueued on the same stream.           */
int32_t mint_pool_admit_packed(mint_pool *pool, int32_t slot, const void *A_packed_dev,
                               const void *B_packed_dev, int32_t rank, mint_stream_t stream);

/* ---- slot table: catalog id -> slot, slot -> (rank, scale) ---------------
 * The engine-local adapter id of the paper's serving map: a catalog of up to
 * 10^6 addressable ids of which a bounded subset is resident.  The three device
 * arrays are the caller's; create enqueues their initialisation (all ids
 * unbound, all slots empty) on the stream.  A host mirror validates bind/evict
 * and carries a generation counter that every bind/evict bumps; plans record
 * it and an apply with an older plan reports MINT_ERR_STALE_PLAN.            */
int32_t mint_slot_table_create(mint_slot_table **out, int64_t catalog_size, int32_t num_slots,
                               int32_t *id_to_slot_dev /*[catalog_size]*/,
                               int32_t *slot_rank_dev /*[num_slots]*/,
                               float *slot_scale_dev /*[num_slots]*/, mint_stream_t stream);
int32_t mint_slot_table_bind(mint_slot_table *table, int64_t catalog_id, int32_t slot, int32_t rank,
                             float scale, mint_stream_t stream);
/* count binds from host arrays, in order; stops at the first invalid one.   */
int32_t mint_slot_table_bind_many(mint_slot_table *table, int64_t count, const int64_t *catalog_ids,
                                  const int32_t *slots, const int32_t *ranks, const float *scales,
                                  mint_stream_t stream);
int32_t mint_slot_table_evict(mint_slot_table *table, int64_t catalog_id, mint_stream_t stream);
int32_t mint_slot_table_destroy(mint_slot_table *table);
int64_t mint_slot_table_generation(const mint_slot_table *table);

/* ---- slot manager: which adapters hold the GPU slots ------------------------
 * The GPU-batch tier holds a bounded number of distinct adapters, promoted by
 * the batch scheduler and released at the end of a step (paper, cache-tier
 * table of "Scale Out: Policy-Population Serving"; the service tracks pinned
 * adapters, "Worker admission and eviction").  Host-side bookkeeping:
 * acquire makes catalog_id resident and pins it for the running step:
 *  - already resident: *slot_out is its slot, *admitted_out = 0;
 *  - otherwise it takes the lowest-numbered empty slot, or the slot of the
 *    least recently acquired adapter that no step pins (*evicted_id_out names
 *    it, else -1), and *admitted_out = 1: the caller now admits the weights
 *    into that slot of every pool (mint_pool_admit_packed) on the same stream;
 *  - MINT_ERR_NOT_RESIDENT when every slot is pinned.
 * With a table (created empty, same num_slots) acquire also evicts the victim
 * from the table and binds catalog_id to the slot with (rank, scale), which
 * bumps the table's generation; with table = NULL it only keeps the books
 * (rank, scale and stream are then ignored).  release removes one pin.  lookup
 * returns the slot of a resident id or -1.  (The paper names least-recently-used
 * order for its CPU adapter cache; using it for unpinned GPU slots is this
 * library's choice.)                                                          */
typedef struct mint_slot_manager mint_slot_manager;
int32_t mint_slot_manager_create(mint_slot_manager **out, int32_t num_slots, mint_slot_table *table);
int32_t mint_slot_manager_destroy(mint_slot_manager *manager);
int32_t mint_slot_manager_acquire(mint_slot_manager *manager, int64_t catalog_id, int32_t rank, float scale,
                                  int32_t *slot_out, int32_t *admitted_out, int64_t *evicted_id_out,
                                  mint_stream_t stream);
int32_t mint_slot_manager_release(mint_slot_manager *manager, int64_t catalog_id);
int32_t mint_slot_manager_lookup(const mint_slot_manager *manager, int64_t catalog_id);

/* ---- plan: token -> adapter segmentation, once per batch ------------------
 * Groups the batch's work items by the adapter slot they use (paper: batch
 * construction respects the same-batch adapter limit; a batch holds several
 * adapters).  Items are tokens (dense: expert_ids_dev = NULL, K = 1) or
 * (token, k) pairs p = t*K + k (MoE).  key = slot for dense, expert*num_slots +
 * slot for MoE.  Canonical result: items with an adapter, ordered by key
 * ascending and by item index ascending inside a key (the stable grouping);
 * one segment per distinct key.  ids_dev[t] = -1 means "no adapter": the item
 * is dropped and its output row is never touched.  An id that is not resident
 * is dropped too, counted in status_dev[1], and status_dev[0] becomes
 * MINT_ERR_NOT_RESIDENT.
 *
 * The plan is an opaque device blob of mint_lora_plan_bytes() bytes (plan
 * arrays, derived tile lists for the kernels, and the sort scratch).  It is
 * reused by every layer and projection of the step; the calls that consume it
 * take the same T (and K) it was made with and report MINT_ERR_SHAPE_MISMATCH
 * in status_dev when they differ.  mint_lora_plan_layout
 * gives the byte offsets of the canonical arrays inside the blob:
 *   perm int32[n_active], seg_start int32[S+1], seg_key int32[S].           */
typedef struct {
  int64_t total_bytes;
  int64_t header_off;     /* int32[MINT_PLAN_HEADER_WORDS] */
  int64_t perm_off;
  int64_t seg_start_off;
  int64_t seg_key_off;
} mint_plan_layout;

typedef struct {
  int32_t num_items;      /* T*K                                            */
  int32_t num_active;     /* items with a resident adapter                  */
  int32_t num_segments;   /* S                                              */
  int32_t max_segment;    /* longest segment                                */
  int32_t sum_rank;       /* sum over segments of the slot's true rank      */
  int32_t not_resident;   /* tokens whose id was not resident               */
  int32_t bad_expert;     /* pairs whose expert id was out of range         */
  int32_t reserved;
  int64_t generation;     /* slot-table generation the plan was made under  */
} mint_plan_summary;

size_t mint_lora_plan_bytes(int32_t T, int32_t K, int32_t num_slots, int32_t num_experts);
int32_t mint_lora_plan_layout(int32_t T, int32_t K, int32_t num_slots, int32_t num_experts,
                              mint_plan_layout *out);
int32_t mint_lora_plan(const mint_slot_table *table, const int64_t *ids_dev /*[T]*/, int32_t T,
                       const int32_t *expert_ids_dev /*[T*K] or NULL*/, int32_t K,
                       int32_t num_experts, void *plan_dev, size_t plan_bytes, int32_t *status_dev,
                       mint_stream_t stream);
/* Copies the plan's counters to the host; synchronises the stream.          */
int32_t mint_plan_fetch_summary(const void *plan_dev, mint_plan_summary *host_out,
                                mint_stream_t stream);

/* ---- shrink: v[t, :r] = x[t, :] . A_sigma   (d -> r) ----------------------
 * x_dev: bf16 [T][ldx].  v_dev: fp32 [T][r_max] in ORIGINAL token order; the
 * call defines all of it: columns at or beyond the token's rank and rows of
 * tokens without a resident adapter are written as 0.  Dense pools only.    */
int32_t mint_lora_shrink(const mint_pool *pool, const mint_slot_table *table, const void *plan_dev,
                         int32_t T, const void *x_dev, int64_t ldx, float *v_dev,
                         int32_t *status_dev, mint_stream_t stream);

/* ---- expand: y[t, :] += s_sigma * (v[t, :r] . B_sigma)   (r -> n) ---------
 * y_dev: bf16 [T][ldy], read-modified-written in place: one fp32 add of y and
 * the scaled delta, one round-to-nearest-even store.  Rows of tokens without
 * a resident adapter are neither read nor written.                           */
int32_t mint_lora_expand(const mint_pool *pool, const mint_slot_table *table, const void *plan_dev,
                         int32_t T, const float *v_dev, void *y_dev, int64_t ldy,
                         int32_t *status_dev, mint_stream_t stream);

/* ---- fused apply: shrink + expand in one call -----------------------------------
 * Same result as shrink followed by expand (fp32 accumulation, summation order
 * may differ).  The shrink result never goes to HBM as a tensor of its own: it
 * crosses from the shrink stage to the expand stage through workspace_dev, a
 * few MB that stay in L2.  workspace_dev: at least
 * mint_lora_apply_workspace_bytes(pool, T) bytes, 256-byte aligned; it needs no
 * initialisation (every call writes each entry before it reads it).  Calls
 * that share a workspace must be ordered on one stream.  Batches of 4096 tokens
 * and more whose plan holds runs of 128 and more tokens of one adapter
 * (segmented prefill) run both contractions of those runs (d -> r, and r -> n
 * with the update of y) on the tcgen05 tensor cores in 128-token tiles; the
 * result is the same.                                                         */
size_t mint_lora_apply_workspace_bytes(const mint_pool *pool, int32_t T);
int32_t mint_lora_apply_fused(const mint_pool *pool, const mint_slot_table *table,
                              const void *plan_dev, int32_t T, const void *x_dev, int64_t ldx,
                              void *y_dev, int64_t ldy, void *workspace_dev, size_t workspace_bytes,
                              int32_t *status_dev, mint_stream_t stream);

/* Fused apply for callers that cannot allocate device memory.  (No counterpart
 * in the paper: an addition for embedding this library.)  Some hosts of this
 * code may not call cudaMalloc or any allocator: a plugin running inside an
 * engine that has already claimed all device memory for its own pools, code on
 * a path where allocation is forbidden because it would synchronise the device,
 * or a process whose memory budget was fixed at start-up.  For them the
 * workspace of mint_lora_apply_fused lives inside the library, in a fixed array
 * of MINT_STATIC_WORKSPACE_BYTES that every GPU which loads the library holds
 * until the process exits; the call allocates and frees nothing.  Inputs,
 * outputs, plan and status word are the caller's, exactly as for
 * mint_lora_apply_fused, and the result is the same.
 *  - A batch whose mint_lora_apply_workspace_bytes(pool, T) exceeds
 *    MINT_STATIC_WORKSPACE_BYTES is refused with MINT_ERR_WORKSPACE_TOO_SMALL
 *    and nothing is launched.
 *  - The first call on each device looks up the array's device address (with
 *    that device current); make that first call before any stream capture.
 *  - All calls share the one array, which keeps what the last call left there.
 *    Nothing in it has to start at zero: every call writes each entry before it
 *    reads it.  Calls that may overlap on the GPU (two streams, or two threads
 *    on different streams) race on it: order them on one stream.              */
#define MINT_STATIC_WORKSPACE_BYTES (8u << 20)
int32_t mint_lora_apply_fused_static(const mint_pool *pool, const mint_slot_table *table,
                                     const void *plan_dev, int32_t T, const void *x_dev, int64_t ldx,
                                     void *y_dev, int64_t ldy, int32_t *status_dev, mint_stream_t stream);

/* Self-test of the bounded device-side waits (general rule above: a wait that
 * ran out is recorded as MINT_ERR_TIMEOUT and the kernel returns).  Runs only the
 * tensor-core shrink of the plan's dense segments (batches of 4096 tokens and
 * more with runs of 128 and more tokens of one adapter) with its tensor-core
 * work withheld and a 2 ms limit, so that nothing ever signals the barriers it
 * waits on: every CTA that has a tile gives up, records MINT_ERR_TIMEOUT in
 * status_dev (status_dev[2] = the tile) and writes nothing else; x is only
 * read, workspace_dev (as for mint_lora_apply_fused) is left as it was.  A
 * diagnostic for deployments, not part of the apply path.                     */
int32_t mint_selftest_wait_timeout(const mint_pool *pool, const mint_slot_table *table,
                                   const void *plan_dev, int32_t T, const void *x_dev, int64_t ldx,
                                   void *workspace_dev, size_t workspace_bytes, int32_t *status_dev,
                                   mint_stream_t stream);

/* Grouped form: the fused apply of up to MINT_MAX_GROUP projections that share
 * one plan (for instance q, k and v, which read the same x; or gate and up), in
 * one pair of launches.  An adapter's target modules come as a set (the paper's
 * policy record lists rank and target modules), so one step applies the same
 * batch plan to every targeted projection.  Each item has its own pool, x, y
 * and workspace (rules as above); items must not alias each other's y.        */
#define MINT_MAX_GROUP 8
typedef struct {
  const mint_pool *pool;
  const void *x_dev;
  int64_t ldx;
  void *y_dev;
  int64_t ldy;
  void *workspace_dev;
  size_t workspace_bytes;
} mint_apply_item;
int32_t mint_lora_apply_fused_grouped(const mint_apply_item *items, int32_t count,
                                      const mint_slot_table *table, const void *plan_dev, int32_t T,
                                      int32_t *status_dev, mint_stream_t stream);

/* ---- LoRA backward over padded slots (dense projections) --------------------
 * The derivative of the update the fused apply performs, for the paper's
 * time-sliced training over a shared frozen base ("Time-Sliced Multi-LoRA
 * Training": adapter slots of a configured maximum shape, smaller ranks padded
 * and masked; kernels that update several adapters in one batch are the
 * alternative it names).  With A: rank x d and B: rank x n of the token's slot,
 * u = dy . B^T and v = x . A^T:
 *   dx[t, :]        += s * u[t, :] . A                      bf16 [T][lddx], one RNE store
 *   dA[slot][k, :]  += s * sum over the slot's tokens of u[t, k] * x[t, :]
 *   dB[slot][k, :]  += s * sum over the slot's tokens of v[t, k] * dy[t, :]
 * dA_dev / dB_dev: fp32, device, shaped like the pool's tensors
 * ([num_slots][r_max][d], [num_slots][r_max][n]), caller-owned, accumulated
 * into; rows k >= rank of a slot and slots without tokens are not touched.
 * Tokens with id -1 (or not resident) contribute nothing and keep their dx row
 * bit for bit.  dx_dev may be NULL (no input gradient wanted); dA_dev and dB_dev
 * may both be NULL (frozen adapters).  The sums run in the plan's token order in
 * fp32: bit-identical from run to run.  x_dev [T][ldx] and dy_dev [T][lddy] are
 * bf16; plan_dev, workspace rules and errors as for mint_lora_apply_fused, with
 * mint_lora_backward_workspace_bytes.  Rank-major pools only.                 */
size_t mint_lora_backward_workspace_bytes(const mint_pool *pool, int32_t T);
int32_t mint_lora_backward(const mint_pool *pool, const mint_slot_table *table, const void *plan_dev,
                           int32_t T, const void *x_dev, int64_t ldx, const void *dy_dev, int64_t lddy,
                           void *dx_dev, int64_t lddx, float *dA_dev, float *dB_dev,
                           void *workspace_dev, size_t workspace_bytes, int32_t *status_dev,
                           mint_stream_t stream);
/* Grouped form: the backward of up to MINT_MAX_GROUP projections that share one
 * plan (the projections of a layer) with a handful of launches for all of them.
 * Each item has its own pool, tensors and workspace (rules as above); items
 * must not alias each other's dx, dA or dB.                                   */
typedef struct {
  const mint_pool *pool;
  const void *x_dev;
  int64_t ldx;
  const void *dy_dev;
  int64_t lddy;
  void *dx_dev;        /* may be NULL */
  int64_t lddx;
  float *dA_dev;       /* both NULL or both given */
  float *dB_dev;
  void *workspace_dev;
  size_t workspace_bytes;
} mint_backward_item;
int32_t mint_lora_backward_grouped(const mint_backward_item *items, int32_t count,
                                   const mint_slot_table *table, const void *plan_dev, int32_t T,
                                   int32_t *status_dev, mint_stream_t stream);

/* ---- MoE expert LoRA apply -------------------------------------------------
 * Per-expert LoRA tensors keyed by expert id (paper, "Scale Up", Megatron
 * placement), in the packed layout.  For pair p = t*K + k with expert e and
 * slot sigma of token t:
 *   Y[p, :] += s_sigma * w_p * (X[row(p), :] . A[sigma][e]) . B[sigma][e]
 * row(p) = x_row_dev[p], or p when x_row_dev is NULL (gate/up projections pass
 * row(p) = t, the down projection reads the pair's own intermediate row);
 * w_p = pair_weight_dev[p], or 1 when NULL.  y_dev: bf16 [T*K][ldy].
 * plan_dev must be a MoE plan (expert_ids given) made with the pool's
 * num_experts.  x_rows is the number of rows of x_dev (range check).         */
size_t mint_moe_lora_apply_workspace_bytes(const mint_pool *pool, int32_t T, int32_t K);
int32_t mint_moe_lora_apply(const mint_pool *pool, const mint_slot_table *table,
                            const void *plan_dev, int32_t T, int32_t K, const void *x_dev,
                            int64_t ldx, int64_t x_rows,
                            const int32_t *x_row_dev, const float *pair_weight_dev, void *y_dev,
                            int64_t ldy, void *workspace_dev, size_t workspace_bytes,
                            int32_t *status_dev, mint_stream_t stream);

/* Grouped form: up to MINT_MAX_GROUP MoE projections that share the plan, the
 * row map and the pair weights (the gate and the up projection of an expert
 * FFN: same routed pairs, same hidden rows) in one pair of launches.  Each item
 * has its own pool, x, y and workspace (rules as for mint_moe_lora_apply); all
 * pools hold the same number of experts; items must not alias each other's y.
 * (Paper, "Scale Up": an adapter's per-expert tensors cover each targeted
 * expert projection.)                                                        */
typedef struct {
  const mint_pool *pool;
  const void *x_dev;
  int64_t ldx;
  void *y_dev;
  int64_t ldy;
  void *workspace_dev;
  size_t workspace_bytes;
} mint_moe_apply_item;
int32_t mint_moe_lora_apply_grouped(const mint_moe_apply_item *items, int32_t count,
                                    const mint_slot_table *table, const void *plan_dev, int32_t T,
                                    int32_t K, int64_t x_rows, const int32_t *x_row_dev,
                                    const float *pair_weight_dev, int32_t *status_dev,
                                    mint_stream_t stream);

/* Router-weighted combine: the MoE expert LoRA update of the projection that ends
 * an expert FFN, summed over a token's routed experts into the token's row
 * (paper, "Scale Up": per-expert LoRA tensors keyed by expert id):
 *   Y[t, :] += sum over k of  w[t,k] * s_sigma * (X[row(p), :] . A[sigma][e_k]) . B[sigma][e_k],  p = t*K + k.
 * y_dev: bf16 [T][ldy].  pair_weight_dev is required.  The sum over k runs in k
 * order in fp32 and ends in one round-to-nearest-even store; the weighted
 * per-pair updates pass through workspace_dev as bf16 (T*K*n elements beside the
 * MoE apply's own workspace).  Rows of tokens without a resident adapter keep
 * their bits.  Other arguments as for mint_moe_lora_apply.                    */
size_t mint_moe_lora_apply_combine_workspace_bytes(const mint_pool *pool, int32_t T, int32_t K);
int32_t mint_moe_lora_apply_combine(const mint_pool *pool, const mint_slot_table *table,
                                    const void *plan_dev, int32_t T, int32_t K, const void *x_dev,
                                    int64_t ldx, int64_t x_rows, const int32_t *x_row_dev,
                                    const float *pair_weight_dev, void *y_dev, int64_t ldy,
                                    void *workspace_dev, size_t workspace_bytes, int32_t *status_dev,
                                    mint_stream_t stream);

/* Backward of the MoE expert LoRA apply (paper, "Scale Up": per-expert LoRA tensors
 * keyed by expert id; "Time-Sliced Multi-LoRA Training": adapters padded to the
 * slot's shape and masked).  For pair p = t*K + k with expert e, slot sigma, routing
 * weight w_p and an upstream gradient dy_dev (bf16 [T*K][lddy], one row per pair),
 * with u = B[sigma][e] . dy[p] and v = X[row(p)] . A[sigma][e]:
 *   dx[p, :]             += w_p * s * A[sigma][e] . u          bf16 [T*K][lddx], one row per PAIR, one RNE
 *                                                              store; the rows of the pairs that read one x
 *                                                              row (gate, up: row(p) = t) are the caller's to add
 *   dA[sigma][e][:, k]   += w_p * s * u[k] * X[row(p), :]      fp32 [num_slots][E][d][r_max]
 *   dB[sigma][e][k, :]   += w_p * s * v[k] * dy[p, :]          fp32 [num_slots][E][r_max][n]
 * dA_dev / dB_dev are caller-owned, shaped like the pool's tensors, accumulated into;
 * ranks k >= rank of a slot and (slot, expert) blocks without pairs are not touched;
 * pairs of tokens without a resident adapter, of expert ids out of range (both already
 * reported by the plan) or whose x row is out of range (reported as BAD_INDEX) contribute
 * nothing and keep their dx row.  The routing weights are constants: no gradient with
 * respect to them.  dx_dev may be NULL; dA_dev and dB_dev may both be NULL.  Sums over a
 * block's pairs run in the plan's order in fp32: bit-identical from run to run.
 * Pools of r_max 8, 16, 32 or 64 only (UNSUPPORTED otherwise).  workspace_dev: device,
 * 256-byte aligned, at least mint_moe_lora_backward_workspace_bytes(pool, T, K) bytes,
 * uninitialised.  Other arguments and errors as for mint_moe_lora_apply.           */
size_t mint_moe_lora_backward_workspace_bytes(const mint_pool *pool, int32_t T, int32_t K);
int32_t mint_moe_lora_backward(const mint_pool *pool, const mint_slot_table *table, const void *plan_dev,
                               int32_t T, int32_t K, const void *x_dev, int64_t ldx, int64_t x_rows,
                               const int32_t *x_row_dev, const float *pair_weight_dev,
                               const void *dy_dev, int64_t lddy, void *dx_dev, int64_t lddx,
                               float *dA_dev, float *dB_dev, void *workspace_dev, size_t workspace_bytes,
                               int32_t *status_dev, mint_stream_t stream);

#ifdef __cplusplus
}
#endif
#endif /* MINT_LORA_H */
