/*
 * CPU oracle for the mixed-adapter LoRA apply.  TEST INFRASTRUCTURE ONLY.
 *
 * Plain, slow, fp64, one token at a time.  It shares no code with the CUDA
 * path and is never called by it: only the tests, the smoke check and the
 * bench's cpu_baseline / reference legs may load this file.
 *
 * What it computes.  The paper keeps one base model resident and lets every
 * request in a batch name its own LoRA adapter revision, resident in a GPU
 * batch slot (section "Shared-Base Rollout and Serving"); a catalog name
 * resolves to an engine-local adapter id ("Scale Out: Policy-Population
 * Serving"); slots are allocated at a configured maximum rank and smaller
 * adapters are padded ("Time-Sliced Multi-LoRA Training"); MoE adapters carry
 * per-expert LoRA tensors keyed by expert id ("Scale Up", Megatron placement).
 * The paper prints no equation for the apply itself (it delegates it to the
 * serving engine), so the definition used here is the standard LoRA update it
 * relies on (Related Work: low-rank matrices attached to selected layers):
 *
 *     y[t, :] = y0[t, :] + s_a * (x[t, :] . A_a) . B_a,      a = adapter(t)
 *
 * with A_a of shape d x r_a, B_a of shape r_a x n and a per-adapter scalar
 * s_a.  Tokens whose id is -1 ("no adapter") keep y0 exactly.  Tokens whose id
 * is not resident in any slot are a contract violation: they are counted,
 * reported and left untouched.
 *
 * Pins (tests/test_oracle_*.py): zero-B and id -1 leave y unchanged; rank 1
 * equals an outer-product update; linear in s; equivariant under token
 * permutation; one adapter for every token equals two numpy matrix products;
 * tiny cases equal x.(W + s.A.B) with merged weights; hand-computed integer
 * examples in tests/golden/.  The planner is pinned against an O(T^2)
 * selection, numpy's stable argsort and its counting invariants.
 * Numeric values of a full apply are "parity unpinned" by the paper itself: it
 * prints no worked example; the pins above are identities, library special
 * cases and brute force.
 *
 * All tensors are addressed through explicit element strides so that the
 * same loops read the dense pool layout A[slot][r][d] and the packed MoE
 * layout A[slot][expert][d][r] without any repacking.
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* bfloat16 bit pattern -> double (exact: bf16 is the top half of an fp32). */
static double bf16_to_f64(uint16_t h) {
    uint32_t u = ((uint32_t)h) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

int oracle_max_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* id -> slot.  -1 = no adapter; -2 = id names no resident adapter (out of the
 * catalog range, unbound, or bound to a slot outside the pool). */
static int32_t lookup_slot(int64_t id, const int32_t *id_to_slot, int64_t catalog_size,
                           int32_t num_slots) {
    if (id == -1) return -1;
    if (id < 0 || id >= catalog_size) return -2;
    int32_t s = id_to_slot[id];
    if (s < 0 || s >= num_slots) return -2;
    return s;
}

/* ------------------------------------------------------------------------
 * Segment plan.
 *
 * Work items are tokens (dense: K = 1, expert_ids = NULL) or (token, k) pairs
 * p = t*K + k (MoE).  key(p) = slot(t) for dense, expert(p)*num_slots +
 * slot(t) for MoE.  Items with no adapter or a non-resident adapter are
 * dropped.  The plan lists the remaining items ordered by key ascending, ties
 * by item index ascending (the stable grouping), and one segment per distinct
 * key: seg_key[S], seg_start[S+1].
 *
 * (key, index) pairs are all distinct, so sorting them with a total-order
 * comparator gives the stable grouping whatever algorithm qsort uses.
 * Returns 0; *n_not_resident counts tokens whose id was not resident.
 * ---------------------------------------------------------------------- */
typedef struct { int64_t key; int64_t index; } key_index;

static int cmp_key_index(const void *a, const void *b) {
    const key_index *p = (const key_index *)a, *q = (const key_index *)b;
    if (p->key != q->key) return p->key < q->key ? -1 : 1;
    if (p->index != q->index) return p->index < q->index ? -1 : 1;
    return 0;
}

int oracle_plan(const int64_t *ids, int32_t T,
                const int32_t *expert_ids, int32_t K, int32_t num_experts,
                const int32_t *id_to_slot, int64_t catalog_size, int32_t num_slots,
                int32_t *perm,       /* [T*K]   out: item indices, grouped   */
                int32_t *seg_key,    /* [T*K]   out: key of each segment     */
                int32_t *seg_start,  /* [T*K+1] out: first position of each  */
                int32_t *S_out, int32_t *n_active_out, int32_t *n_not_resident,
                int32_t *n_bad_expert) {
    if (K < 1) K = 1;
    int64_t P = (int64_t)T * K;
    key_index *items = (key_index *)malloc(sizeof(key_index) * (size_t)(P > 0 ? P : 1));
    int64_t m = 0;
    int32_t missing = 0, bad_expert = 0;
    for (int32_t t = 0; t < T; ++t) {
        int32_t slot = lookup_slot(ids[t], id_to_slot, catalog_size, num_slots);
        if (slot == -2) ++missing;
        if (slot < 0) continue;
        for (int32_t k = 0; k < K; ++k) {
            int64_t p = (int64_t)t * K + k;
            int64_t key = slot;
            if (expert_ids) {
                int32_t e = expert_ids[p];
                if (e < 0 || e >= num_experts) { ++bad_expert; continue; }
                key = (int64_t)e * num_slots + slot;
            }
            items[m].key = key;
            items[m].index = p;
            ++m;
        }
    }
    qsort(items, (size_t)m, sizeof(key_index), cmp_key_index);
    int32_t S = 0;
    for (int64_t i = 0; i < m; ++i) {
        perm[i] = (int32_t)items[i].index;
        if (i == 0 || items[i].key != items[i - 1].key) {
            seg_key[S] = (int32_t)items[i].key;
            seg_start[S] = (int32_t)i;
            ++S;
        }
    }
    seg_start[S] = (int32_t)m;
    *S_out = S;
    *n_active_out = (int32_t)m;
    *n_not_resident = missing;
    if (n_bad_expert) *n_bad_expert = bad_expert;
    free(items);
    return 0;
}

/* ------------------------------------------------------------------------
 * Dense apply, one token at a time.
 *
 *   v[j]      = sum_{i<d} x[t,i] * A_slot[i,j]                 j < r_slot
 *   y_ref[t,o] = y0[t,o] + s_slot * sum_{j<r} v[j] * B_slot[j,o]
 *
 * A element (slot, i, j) lives at A[slot*A_slot_stride + i*A_i_stride +
 * j*A_j_stride]; B element (slot, j, o) at B[slot*B_slot_stride +
 * j*B_j_stride + o*B_o_stride].  Only j < rank[slot] is ever read.
 * y_ref is [T][n] doubles, never rounded.  v_out, if not NULL, is
 * [T][r_max] doubles: the shrink result, zero beyond the rank and for
 * tokens without a resident adapter.
 * Returns the number of tokens whose id was not resident.
 * ---------------------------------------------------------------------- */
int32_t oracle_lora_apply(int32_t T, int32_t d, int32_t n, int32_t r_max,
                          const int64_t *ids, const int32_t *id_to_slot, int64_t catalog_size,
                          int32_t num_slots, const int32_t *slot_rank, const float *slot_scale,
                          const uint16_t *A, int64_t A_slot_stride, int64_t A_i_stride, int64_t A_j_stride,
                          const uint16_t *B, int64_t B_slot_stride, int64_t B_j_stride, int64_t B_o_stride,
                          const uint16_t *x, int64_t ldx,
                          const uint16_t *y0, int64_t ldy,
                          double *y_ref, double *v_out, int32_t num_threads) {
    int32_t missing = 0;
#ifdef _OPENMP
    if (num_threads > 0) omp_set_num_threads(num_threads);
#endif
    #pragma omp parallel for schedule(dynamic, 1) reduction(+:missing)
    for (int32_t t = 0; t < T; ++t) {
        double *yr = y_ref + (int64_t)t * n;
        for (int32_t o = 0; o < n; ++o) yr[o] = bf16_to_f64(y0[(int64_t)t * ldy + o]);
        if (v_out) for (int32_t j = 0; j < r_max; ++j) v_out[(int64_t)t * r_max + j] = 0.0;
        int32_t slot = lookup_slot(ids[t], id_to_slot, catalog_size, num_slots);
        if (slot == -2) ++missing;
        if (slot < 0) continue;
        int32_t r = slot_rank[slot];
        double s = (double)slot_scale[slot];
        double *v = (double *)malloc(sizeof(double) * (size_t)(r > 0 ? r : 1));
        for (int32_t j = 0; j < r; ++j) {
            double acc = 0.0;
            for (int32_t i = 0; i < d; ++i)
                acc += bf16_to_f64(x[(int64_t)t * ldx + i]) *
                       bf16_to_f64(A[slot * A_slot_stride + i * A_i_stride + j * A_j_stride]);
            v[j] = acc;
            if (v_out) v_out[(int64_t)t * r_max + j] = acc;
        }
        for (int32_t o = 0; o < n; ++o) {
            double acc = 0.0;
            for (int32_t j = 0; j < r; ++j)
                acc += v[j] * bf16_to_f64(B[slot * B_slot_stride + j * B_j_stride + o * B_o_stride]);
            yr[o] += s * acc;
        }
        free(v);
    }
    return missing;
}

/* ------------------------------------------------------------------------
 * MoE expert LoRA apply, one (token, k) pair at a time.
 *
 *   p = t*K + k,  e = expert[p],  slot = slot(t),  row = x_row ? x_row[p] : p
 *   Y_ref[p,:] = Y0[p,:] + s_slot * w_p * (X[row,:] . A[slot][e]) . B[slot][e]
 *
 * w_p = 1 when pair_weight is NULL.  A element (slot, e, i, j) at
 * slot*A_slot_stride + e*A_e_stride + i*A_i_stride + j*A_j_stride, B likewise.
 * Returns the number of tokens whose id was not resident.
 * ---------------------------------------------------------------------- */
int32_t oracle_moe_lora_apply(int32_t T, int32_t K, int32_t num_experts, int32_t d, int32_t n,
                              const int64_t *ids, const int32_t *expert_ids,
                              const int32_t *id_to_slot, int64_t catalog_size, int32_t num_slots,
                              const int32_t *slot_rank, const float *slot_scale,
                              const uint16_t *A, int64_t A_slot_stride, int64_t A_e_stride,
                              int64_t A_i_stride, int64_t A_j_stride,
                              const uint16_t *B, int64_t B_slot_stride, int64_t B_e_stride,
                              int64_t B_j_stride, int64_t B_o_stride,
                              const uint16_t *x, int64_t ldx, const int32_t *x_row,
                              const float *pair_weight,
                              const uint16_t *y0, int64_t ldy,
                              double *y_ref, int32_t num_threads) {
    int32_t missing = 0;
    int64_t P = (int64_t)T * K;
#ifdef _OPENMP
    if (num_threads > 0) omp_set_num_threads(num_threads);
#endif
    #pragma omp parallel for schedule(dynamic, 8) reduction(+:missing)
    for (int64_t p = 0; p < P; ++p) {
        int32_t t = (int32_t)(p / K);
        double *yr = y_ref + p * n;
        for (int32_t o = 0; o < n; ++o) yr[o] = bf16_to_f64(y0[p * ldy + o]);
        int32_t slot = lookup_slot(ids[t], id_to_slot, catalog_size, num_slots);
        if (slot == -2 && p % K == 0) ++missing;
        if (slot < 0) continue;
        int32_t e = expert_ids[p];
        if (e < 0 || e >= num_experts) continue;
        int32_t r = slot_rank[slot];
        double s = (double)slot_scale[slot];
        double w = pair_weight ? (double)pair_weight[p] : 1.0;
        int64_t row = x_row ? (int64_t)x_row[p] : p;
        const uint16_t *Ae = A + slot * A_slot_stride + e * A_e_stride;
        const uint16_t *Be = B + slot * B_slot_stride + e * B_e_stride;
        double *v = (double *)malloc(sizeof(double) * (size_t)(r > 0 ? r : 1));
        for (int32_t j = 0; j < r; ++j) {
            double acc = 0.0;
            for (int32_t i = 0; i < d; ++i)
                acc += bf16_to_f64(x[row * ldx + i]) * bf16_to_f64(Ae[i * A_i_stride + j * A_j_stride]);
            v[j] = acc;
        }
        for (int32_t o = 0; o < n; ++o) {
            double acc = 0.0;
            for (int32_t j = 0; j < r; ++j)
                acc += v[j] * bf16_to_f64(Be[j * B_j_stride + o * B_o_stride]);
            yr[o] += s * w * acc;
        }
        free(v);
    }
    return missing;
}
