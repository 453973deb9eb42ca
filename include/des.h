/*
 * des.h — C ABI of the single-GPU hot path of Distributed Equivalent
 * Substitution (DES) training (arXiv 1909.04823).
 *
 * What the library computes
 * -------------------------
 * The weights-rich sparse operators of CTR models, each rewritten as S
 * per-shard sub-operators M_j over a partition of the weights, an
 * aggregation (+) over shards and a substitution operator F (Algorithm 1,
 * Eq. 1).  The S "processes" of the paper are S logical shards resident on
 * one GPU; the aggregation is an in-device reduction in fixed shard order.
 *
 *   LR      M_1 = sum_{j in shard} w_j x_j                (Section 4.1)
 *   FM      M_1 = sum v_j x_j (k-vector),
 *           M_2 = sum <v_j x_j, v_j x_j> (scalar),
 *           F   = 1/2 <(+)M_1,(+)M_1> - 1/2 (+)M_2        (Section 4.2)
 *   POOL    sum-pooled latent vectors per (sample, field) (Section 4.3,
 *           embedding layer; same field on the same shard under FIELD)
 *   DENSE1  V^T W = sum_s V_s^T W_s, the first FC layer split over the
 *           rows of W by owning shard                      (Section 4.3)
 *   table   lookup / insert / update on a dynamic hash table of
 *           uint64 keys and float32 weights               (Section 5)
 *   backward: the aggregated gradient flows back into each shard's own
 *           sub-operator, no cross-shard term             (Section 3.2,
 *           "Back-propagation Phase"); one optimizer application per
 *           unique key per step, state local to the shard (Section 4.3,
 *           last paragraph before "Extending to General Models").
 *
 * Conventions
 * -----------
 * - Every function returns des_status_t; nothing throws, nothing aborts.
 * - Pointers named d_* (and every pointer inside des_batch_t, des_partials_t,
 *   des_outputs_t, des_grads_t) are DEVICE pointers owned by the caller; they
 *   must stay valid until the stream has passed the call.  Pointers named h_*
 *   are HOST pointers.  The library owns only what des_table_create allocates
 *   and frees it in des_table_destroy.
 * - All device work is enqueued on the caller's stream (a cudaStream_t passed
 *   as void*; NULL = the legacy default stream).  Only des_table_status,
 *   des_table_size, des_table_export, des_dense1_get/set on host pointers,
 *   des_step_host and des_step_host_wait synchronise.
 * - One table, one order: every call on a table reuses workspace that the table
 *   owns (routing arrays, the gradient buffer, hot-key lists), so all calls on
 *   one table must be ordered — the same stream, or streams ordered by events.
 *   Two calls on one table that overlap on the GPU race.  Different tables are
 *   independent.  A table belongs to the device that was current when it was
 *   created; calls with another device current return DES_ERR_INVALID_ARG where
 *   the library can tell, and are undefined otherwise.
 * - Reproducibility: the integer outputs (shards, rows, unique indices, the key
 *   set) and the forward's floating-point results are identical from run to
 *   run.  The backward sums a key's gradient terms with floating-point atomics
 *   in an order that changes from run to run: updated weights agree between
 *   runs within rounding (the tolerance of the parity tests), not bit for bit.
 * - Device-side problems (reserved key, full shard) never fault: the
 *   offending occurrences get row DES_ROW_NONE, are skipped by every later
 *   kernel, and a sticky error word is raised that des_table_status returns.
 * - There is no CPU fallback: without a CUDA device every call that would
 *   launch returns DES_ERR_CUDA.
 *
 * Batch layout (CSR over bags): bag (b, f) = sample b, field f, holds the
 * occurrences offsets[b*F+f] .. offsets[b*F+f+1]-1 of ids[] / vals[].
 * An id that appears twice in a bag is two terms of every sum.
 */
#ifndef DES_H_
#define DES_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  DES_OK = 0,
  DES_ERR_INVALID_ARG = 1,   /* bad argument, found on the host before any launch      */
  DES_ERR_RESERVED_KEY = 2,  /* an id equals DES_KEY_EMPTY (sticky, device-side)        */
  DES_ERR_CAPACITY = 3,      /* a shard ran out of slots or rows (sticky, device-side)  */
  DES_ERR_UNSUPPORTED = 4,
  DES_ERR_CUDA = 5,          /* a CUDA runtime call failed, or no device                */
  DES_ERR_NOT_FOUND = 6,
  DES_ERR_TOO_LARGE = 7,     /* problem exceeds the fixed scratch of a no-allocation entry point */
  DES_ERR_RANGE = 8          /* checking build only (libdes_debug.so): a kernel met an index outside the
                                table's bounds, skipped the access and raised this (sticky, device-side) */
} des_status_t;

/* operator kind bitmask */
enum { DES_OP_LR = 1, DES_OP_FM = 2, DES_OP_POOL = 4, DES_OP_DENSE1 = 8 };
/* modifier, des_forward_fused only: keep the shard-by-shard form (see there) */
enum { DES_FUSED_SHARD_ORDER = 16 };
/* weight placement: HASH = mix64(id) mod S (Section 4.2 allows any partition
 * that keeps the shards balanced); FIELD = field mod S (the rule of Section 5,
 * paragraph on large-scale sparse features; required for a weight-disjoint row
 * split, Section 4.3). */
enum { DES_PART_HASH = 0, DES_PART_FIELD = 1 };
/* optimizer of the latent vectors and of the first dense layer; the order-1
 * (linear) weights follow it unless lin_optimizer says FTRL (Section 6,
 * parameter settings: the paper trains the order-1 parts with FTRL and the
 * embeddings and dense layers with Adagrad or Adam). */
enum { DES_OPT_SGD = 0, DES_OPT_ADAGRAD = 1, DES_OPT_ADAM = 2 };
enum { DES_LIN_SAME = 0, DES_LIN_FTRL = 1 };

#define DES_KEY_EMPTY 0xFFFFFFFFFFFFFFFFull /* reserved id                         */
#define DES_ROW_NONE  0xFFFFFFFFu           /* "no row": missing key / failed insert */

typedef struct des_table des_table_t;

typedef struct {
  uint32_t num_shards;   /* S, 1..64                                                  */
  uint32_t num_fields;   /* F >= 1                                                    */
  uint32_t emb_dim;      /* k, a multiple of 4, 4..64                                 */
  uint32_t hidden;       /* H of the first dense layer, multiple of 4; 0 = no DENSE1  */
  uint32_t partition;    /* DES_PART_*                                                */
  uint32_t optimizer;    /* DES_OPT_*                                                 */
  uint64_t max_rows;     /* total key capacity over all shards, < 2^32 - 1            */
  float    max_load;     /* slots per shard = rows of the shard / max_load; (0, 0.9]  */
  const uint64_t* h_rows_per_shard; /* optional host [S] row capacity per shard; NULL =
                                       max_rows/S * 1.05 + 1024 each                  */
  uint64_t seed;         /* seed of the counter-based row initialiser                 */
  float    init_scale;   /* new latent vectors ~ U[-init_scale, init_scale)           */
  float    lr, eps, init_acc; /* theta -= lr*G            (SGD)
                                 a += G*G; theta -= lr*G/(sqrt(a)+eps)   (Adagrad),
                                 a starts at init_acc                                */
  uint32_t lin_optimizer;/* DES_LIN_*: optimizer of the order-1 weights                */
  float    beta1, beta2; /* Adam (lazy: only the keys of the batch move; one global step
                            count t per backward call):  m = b1 m + (1-b1) G;
                            v = b2 v + (1-b2) G*G;
                            theta -= lr * (m/(1-b1^t)) / (sqrt(v/(1-b2^t)) + eps)       */
  float    ftrl_alpha, ftrl_beta, ftrl_l1, ftrl_l2; /* FTRL-Proximal per coordinate:
                            sigma = (sqrt(n+G*G) - sqrt(n))/alpha; z += G - sigma*w;
                            n += G*G; w = |z| <= l1 ? 0 :
                            -(z - sign(z) l1) / ((beta + sqrt(n))/alpha + l2)           */
  uint32_t shard_world, shard_rank; /* multi-GPU (Algorithm 1: each process holds W_i): this
                            table owns the shards s with s mod shard_world == shard_rank
                            and ignores every other key (row DES_ROW_NONE, never inserted);
                            shard_world 0 or 1 = owns all.  max_rows is spread over the
                            owned shards only                                           */
  int64_t  max_nnz;      /* largest nnz of any batch (sizes the workspace)            */
  int32_t  max_batch;    /* largest B of any batch                                    */
  int64_t  max_uniq;     /* largest number of distinct keys in one batch (sizes the
                            gradient buffer: max_uniq*(k+4)*4 bytes); 0 = max_nnz     */
  /* optional device allocator (e.g. backed by the caller's caching allocator);
   * NULL = cudaMalloc / cudaFree.  alloc must return 256-byte aligned memory.   */
  void* (*alloc)(size_t bytes, void* ctx);
  void  (*dealloc)(void* ptr, void* ctx);
  void*  alloc_ctx;
} des_config_t;

/* One batch.  find_or_insert reads offsets/ids and fills rows, shards, uidx,
 * uniq_rows, n_uniq; the other calls read them. */
typedef struct {
  int32_t         batch;      /* B                                                    */
  int64_t         nnz;        /* occurrences, < 2^31                                  */
  const int32_t*  offsets;    /* [B*F+1]                                              */
  const uint64_t* ids;        /* [nnz]                                                */
  const float*    vals;       /* [nnz] feature values x_j, or NULL = all 1.0          */
  uint32_t*       rows;       /* [nnz] shard-local row of each occurrence             */
  uint8_t*        shards;     /* [nnz] owning shard of each occurrence                */
  uint32_t*       uidx;       /* [nnz] batch-unique index of the occurrence's key:
                                 keys numbered 0..U-1 by first occurrence in CSR order */
  uint32_t*       uniq_rows;  /* [nnz] (first U used) table-global row of unique key u
                                 = des_table_row_base()[shard] + shard-local row      */
  uint32_t*       n_uniq;     /* [1]   U                                              */
} des_batch_t;

/* Per-shard partial results (the paper's intermediate results S_M).
 * SMALL_STRIDE(k) = k + 4 floats per (shard, sample):
 *   [0..k)  M_1 of FM   (sum v x)
 *   [k]     M_1 of LR   (sum w x)
 *   [k+1]   M_2 of FM   (sum <v x, v x>)
 *   [k+2], [k+3]  zero padding (keeps rows 16-byte aligned). */
typedef struct {
  float* part_small;   /* [S][B][k+4], required for LR / FM                            */
  float* pooled;       /* [B][F*k] sum-pooled field embeddings, already aggregated over
                          shards on chip; required for POOL / DENSE1                   */
  float* part_pooled;  /* optional [S][B][F*k] dense per-shard pooled partials
                          (parity / inspection at small sizes), or NULL                */
  float* part_dense;   /* optional [S][B][H] per-shard partial products P_s = V_s W_s,
                          or NULL (then only Z is produced by des_aggregate)           */
} des_partials_t;

/* Aggregated results.  out_small has k + 4 floats per sample:
 *   [0..k) A = (+)M_1 ; [k] R_lr = (+)M_1^lr ; [k+1] fm2 = F ; [k+2] Q = (+)M_2 ;
 *   [k+3] zero. */
typedef struct {
  float* out_small;    /* [B][k+4]                                                     */
  float* pooled;       /* [B][F*k]; may alias des_partials_t.pooled                    */
  float* Z;            /* [B][H] = sum_s P_s (DENSE1), fp32                            */
} des_outputs_t;

/* Upstream gradients of the aggregated results (what the rest of the model
 * sends back).  Any pointer may be NULL when its operator is not in `ops`. */
typedef struct {
  const float* gL;     /* [B]      dLoss/dR_lr                                         */
  const float* gF;     /* [B]      dLoss/dfm2                                          */
  const float* gE;     /* [B][F*k] dLoss/dpooled (direct consumers of pooled), or NULL */
  const float* gZ;     /* [B][H]   dLoss/dZ (DENSE1), or NULL                          */
  float*       gE_work;/* [B][F*k] scratch, required with DENSE1: receives
                          gE + gZ * W1^T                                               */
} des_grads_t;

/* ---- table life cycle (Section 5, "Dynamic Hash Table") ------------------- */

/* Allocates slots, rows, optimizer state and the per-call workspace on the
 * current device.  *out is NULL on failure. */
des_status_t des_table_create(const des_config_t* cfg, des_table_t** out);
des_status_t des_table_destroy(des_table_t* t);

/* lookup + insert (Section 5).  insert != 0: ids not yet in the table are
 * inserted; a new key gets the next shard-local row, numbered in order of the
 * key's first occurrence in CSR order within this call, its latent vector is
 * initialised from a counter-based generator keyed on (seed, id) — so row
 * contents never depend on insertion order —, its linear weight is 0 and its
 * optimizer state init_acc.  insert == 0: lookup only; missing ids get
 * DES_ROW_NONE, and uidx / uniq_rows / n_uniq are not written.
 * Errors: DES_ERR_INVALID_ARG (nnz > max_nnz, batch > max_batch, NULL
 * pointers); device-side sticky DES_ERR_RESERVED_KEY / DES_ERR_CAPACITY. */
des_status_t des_find_or_insert(des_table_t* t, const des_batch_t* batch, int insert, void* stream);

/* Sub-operators M_j of every shard (Eq. of Sections 4.1-4.3), see
 * des_partials_t.  `batch` must have been through des_find_or_insert.  (Under
 * DES_PART_FIELD with pooling among the operators a shard's sub-operators are formed
 * as the sums over the bags of its own fields, from the same pass that pools them;
 * otherwise shard by shard from the shard's own occurrences.) */
des_status_t des_forward_partials(des_table_t* t, uint32_t ops, const des_batch_t* batch,
                                  const des_partials_t* part, void* stream);

/* Aggregation (+) over shards in the fixed order s = 0..S-1 (Eq. 1) and the
 * substitution operator F (Algorithm 1, R = F(f_1..f_m)): out_small from
 * part_small; Z from pooled and W1 in one product on the tensor cores (its K loop
 * runs over the columns of pooled in field order; under the FIELD partition that
 * visits every shard's block once, not shard by shard — inside the 2e-2 bound of
 * bf16 operands) or, when part->part_dense is given, P_s materialised first (K
 * slices in shard order, CUDA-core kernel) and Z = sum_s P_s. */
des_status_t des_aggregate(des_table_t* t, uint32_t ops, const des_batch_t* batch,
                           const des_partials_t* part, const des_outputs_t* out, void* stream);

/* des_forward_partials + des_aggregate in one call, with the per-shard partial
 * results of LR / FM kept on chip (Algorithm 1 with the aggregation made an
 * on-chip reduction).  Two forms:
 *  - `ops` holds LR / FM only, or part->part_small is given (to receive the
 *    partials as well): every sample's partials are formed shard by shard in
 *    registers, aggregated in the same fixed shard order and passed through F
 *    without being written; results are bit-identical to the two-call path.
 *  - `ops` holds LR / FM together with POOL / DENSE1, part->part_small is
 *    NULL and DES_FUSED_SHARD_ORDER is not set in `ops`: every occurrence's row
 *    is gathered once; the pass that pools a bag
 *    also sums its linear weights and squared norms, and (+)M_1, (+)M_1^lr,
 *    (+)M_2 are the sums over a sample's bags, taken in double in field order.
 *    The per-shard partials are never formed — Eq. 1's sum over a sample's
 *    occurrences grouped by field instead of by shard — so the results agree
 *    with the two-call path within the float32 tolerance, not bit for bit.
 * part->part_pooled and part->part_dense must be NULL. */
des_status_t des_forward_fused(des_table_t* t, uint32_t ops, const des_batch_t* batch,
                               const des_partials_t* part, const des_outputs_t* out, void* stream);

/* Mirror of the forward (Section 3.2): per-occurrence gradients
 *   g_w(j) = x_j gL[b],  g_v(j) = x_j ( gF[b] (A[b] - v_j x_j) + gE[b][f] ),
 * summed per unique key, then one SGD / Adagrad application per key with the
 * state kept in the shard.  With DENSE1: gE_work = gE + gZ W1^T (each shard's
 * own column block), gW1 = pooled^T gZ, and the same optimizer on W1.
 * `out` supplies A (out_small) and pooled. */
des_status_t des_backward_update(des_table_t* t, uint32_t ops, const des_batch_t* batch,
                                 const des_outputs_t* out, const des_grads_t* grads, void* stream);

/* ---- aggregation across processes (Algorithm 1, the exchange step) ---------- */

/* With the shards spread over several tables (shard_world > 1, one table per GPU, the
 * same batch on every GPU as in Section 6), (+) runs in two levels.  des_rank_partial
 * adds this table's per-shard small partials (des_forward_partials' part_small) in
 * shard order into d_rank_part [B][k+4], same column layout as one shard's block:
 * that is the message a process sends.  After the processes have exchanged their
 * messages (an all-gather into [world][B][k+4] in rank order: NCCL, or peer copies),
 * des_aggregate_ranks adds them in rank order and applies F (Eq. 8), writing
 * out_small [B][k+4] exactly as des_aggregate does; every process computes the same
 * bits.  Pooled blocks and first-layer partials Z are plain element-wise sums over
 * processes (an all-reduce of des_aggregate's local outputs).  The backward needs no
 * exchange (Section 3.2): every table updates the keys it owns. */
des_status_t des_rank_partial(des_table_t* t, int32_t batch, const float* d_part_small, float* d_rank_part,
                              void* stream);
des_status_t des_aggregate_ranks(des_table_t* t, uint32_t ops, int32_t batch, int32_t world,
                                 const float* d_rank_parts, float* d_out_small, void* stream);

/* ---- first dense layer weights W1 [F*k][H], fp32 master (Section 4.3) ----- */
des_status_t des_dense1_set(des_table_t* t, const float* d_W1, void* stream);
des_status_t des_dense1_get(des_table_t* t, float* d_W1, void* stream);
/* Optimizer state of W1, same shape as W1: state1 = Adagrad accumulator or Adam
 * first moment, state2 = Adam second moment.  Either pointer may be NULL; a
 * non-NULL pointer for a state the configured optimizer does not keep is
 * DES_ERR_INVALID_ARG.  Device pointers; copies are enqueued on `stream`. */
des_status_t des_dense1_get_state(des_table_t* t, float* d_state1, float* d_state2, void* stream);
des_status_t des_dense1_set_state(des_table_t* t, const float* d_state1, const float* d_state2, void* stream);

/* Row-split first layer for callers that must not allocate.  (The paper has no
 * counterpart: this is a packaging variant of des_aggregate's DENSE1 step, same
 * arithmetic, same result.)
 *
 * Who needs it: code that is handed a stream and some buffers but is not allowed
 * to call cudaMalloc — a serving loop with a frozen memory budget, a plug-in
 * running inside someone else's framework, anything between the begin and end
 * of a latency-critical section where an allocation would synchronise the
 * device.  des_aggregate normally wants the caller to bring the [S][B][H]
 * buffer for the per-shard partial products P_s = V_s W_s; here that buffer is
 * a fixed array inside the library image instead.
 *
 * Computes Z[B][H] = sum over shards s = 0..S-1 of P_s from d_pooled [B][F*k]
 * and the table's W1 (FIELD partition only).  The partial products live in a
 * static device array of DES_NOALLOC_SCRATCH_FLOATS floats (8 MiB, reserved on
 * every GPU that loads the library until the process exits); the call is
 * rejected with DES_ERR_TOO_LARGE when S*B*H exceeds that.  It calls no
 * cudaMalloc / cudaFree and no allocating routine of any library.
 *
 * The first call on a device looks up the array's device address (one runtime
 * query, result cached per device); make that first call outside any stream
 * capture.  All calls share the one array and it keeps the last call's
 * contents: every element a call reads is written by that same call first, so
 * stale contents are harmless, but two calls whose kernels overlap on the GPU
 * (different streams, no ordering) race on it. */
#define DES_NOALLOC_SCRATCH_FLOATS (2u * 1024u * 1024u)
des_status_t des_dense1_forward_noalloc(des_table_t* t, const float* d_pooled, int32_t batch, float* d_Z,
                                        void* stream);

/* ---- inspection (synchronising) ------------------------------------------ */

/* Synchronises the device and returns the sticky device-side error, if any. */
des_status_t des_table_status(des_table_t* t);
/* Number of keys per shard, host array [S]. */
des_status_t des_table_size(des_table_t* t, uint64_t* h_rows_per_shard);
/* First table-global row of each shard and the grand total, host array [S+1]. */
des_status_t des_table_row_base(des_table_t* t, uint64_t* h_row_base);
/* Dumps up to `cap` keys (device arrays, any order): key, shard, shard-local
 * row, latent vector [k], linear weight and their optimizer state (each of the
 * four float arrays may be NULL: not written).  *h_n_out = number of keys in
 * the table (may exceed cap; then only cap are written). */
des_status_t des_table_export(des_table_t* t, uint64_t* d_keys, uint8_t* d_shards, uint32_t* d_rows,
                              float* d_emb, float* d_lin, float* d_acc_emb, float* d_acc_lin,
                              uint64_t cap, uint64_t* h_n_out);
/* Copies the rows (latent vector, linear weight, optimizer state) of the n
 * table-global rows d_global_rows[] into dense device arrays; any output
 * pointer may be NULL. */
des_status_t des_table_read_rows(des_table_t* t, const uint32_t* d_global_rows, int64_t n,
                                 float* d_emb, float* d_lin, float* d_acc_emb, float* d_acc_lin,
                                 void* stream);

/* Inverse of des_table_read_rows (restore from a checkpoint, re-seeding rows):
 * overwrites the rows of the n table-global rows d_global_rows[] from dense
 * device arrays; NULL inputs leave that part untouched.  Rows must exist. */
des_status_t des_table_write_rows(des_table_t* t, const uint32_t* d_global_rows, int64_t n,
                                  const float* d_emb, const float* d_lin, const float* d_acc_emb,
                                  const float* d_acc_lin, void* stream);

/* ---- eviction (Section 1, "Dynamic Features": the live feature set of a streaming model
 * changes over time; the paper's table — Section 5 — has no delete, this is the reading) --- */

/* Removes keys from the table.  A removed key looks up as DES_ROW_NONE; inserting it again
 * makes a new key of it (fresh initial weights and state).  Every other key keeps its
 * contents.  Row numbers: a shard's rows stay 0 .. n-1 — the rows freed below the shard's
 * new size are taken, in ascending order, by the surviving rows from beyond it, in
 * ascending order; all other rows keep their numbers.  Row numbers, unique indices and
 * anything else derived from a batch before the call are stale afterwards: run
 * des_find_or_insert again.
 *   des_table_evict_keys   the n keys of the device array d_keys (unknown or repeated keys
 *                          are ignored; under DES_PART_FIELD a key is removed from every
 *                          shard that holds it);
 *   des_table_evict_stale  every key whose row was neither inserted nor updated by
 *                          des_backward_update since the table's clock read min_clock.  The
 *                          clock (des_table_clock) counts the inserting des_find_or_insert
 *                          calls that had at least one occurrence.
 * *h_n_evicted (optional) = number of rows removed.  Maintenance calls: they synchronise the
 * device, allocate temporaries with cudaMalloc (4 bytes per table row, 16 bytes per surviving
 * key of the shards that lose a key) and free them before returning; not for use inside a
 * stream capture.  Errors: DES_ERR_INVALID_ARG, DES_ERR_CUDA (also: out of memory). */
des_status_t des_table_evict_keys(des_table_t* t, const uint64_t* d_keys, int64_t n, uint64_t* h_n_evicted);
des_status_t des_table_evict_stale(des_table_t* t, uint64_t min_clock, uint64_t* h_n_evicted);
des_status_t des_table_clock(des_table_t* t, uint64_t* h_clock);

/* Second optimizer-state slot of the same rows (what des_table_read_rows /
 * write_rows do for the first): Adam's v of the latent vectors [n][k] and the
 * second state word of the linear weight [n] (Adam's v, FTRL's z; the first
 * word — Adagrad's accumulator, Adam's m, FTRL's n — is `acc_lin`).  Any
 * pointer may be NULL; parts the configured optimizers do not keep read as 0. */
des_status_t des_table_read_state2(des_table_t* t, const uint32_t* d_global_rows, int64_t n,
                                   float* d_acc2_emb, float* d_lin2, void* stream);
des_status_t des_table_write_state2(des_table_t* t, const uint32_t* d_global_rows, int64_t n,
                                    const float* d_acc2_emb, const float* d_lin2, void* stream);

/* ---- whole step from host buffers ---------------------------------------- */

/* One full step — find_or_insert, forward partials, aggregate, backward
 * update — on a batch that lives in HOST memory (pinned for full speed):
 * offsets/ids/vals are copied to device staging owned by the table, the step
 * runs on `stream`, out_small [B][k+4] is copied back to h_out_small and the
 * call returns after synchronising.  Upstream gradients stay device resident
 * (they come from the rest of the model, which lives on the GPU).  d_pooled
 * [B][F*k] is device scratch/output for POOL.  Requires max_nnz/max_batch
 * workspace like the other calls. */
des_status_t des_step_host(des_table_t* t, uint32_t ops, int32_t batch, int64_t nnz,
                           const int32_t* h_offsets, const uint64_t* h_ids, const float* h_vals,
                           const des_grads_t* d_grads, float* d_pooled, float* d_Z,
                           float* h_out_small, void* stream);

/* The same step for callers that feed batches back to back (Section 5: batch
 * building and the optimizer phase follow each other every iteration).
 * des_step_host_submit returns as soon as the step is enqueued: the host
 * buffers are copied on a stream of the table's own into one of two staging
 * slots, the kernels and the read-back of out_small run on `stream` once the
 * copy has landed, so the copy of step i+1 overlaps the kernels of step i.
 * *ticket names the slot; des_step_host_wait(ticket) blocks until that step is
 * over (h_out_small written).  At most two steps are in flight: a third submit
 * first waits for the step that used its slot.  Host buffers (inputs and
 * h_out_small) must stay untouched until the step's wait returns, and must be
 * pinned for the overlap to happen; all submits of a table must use the same
 * `stream`, which orders the steps.  Results are those of des_step_host. */
des_status_t des_step_host_submit(des_table_t* t, uint32_t ops, int32_t batch, int64_t nnz,
                                  const int32_t* h_offsets, const uint64_t* h_ids, const float* h_vals,
                                  const des_grads_t* d_grads, float* d_pooled, float* d_Z,
                                  float* h_out_small, void* stream, int32_t* ticket);
des_status_t des_step_host_wait(des_table_t* t, int32_t ticket);

/* ---- a fixed read-out in place of the rest of the model ---------------------- */

/* The sparse path ends at the aggregated results (R_lr, fm2, pooled, Z); the layers above them (Section 4.3,
 * Fig. 4: the rest of the DNN, the output unit, the loss) are not part of it.  So that multi-step runs and
 * closed-loop measurements need no gradients from outside, des_head stands in for them with a read-out
 * whose constants are given and never trained (the paper has no counterpart for its particular form):
 *   logit = b0 + c_lr R_lr + c_fm fm2 + <u, relu(Z + b1)> + <q, pooled> + <d, xdense>
 *   p = sigmoid(logit);  loss_b = -(y_b log p + (1 - y_b) log(1 - p));  g = (p - y_b) / batch
 *   gL = c_lr g;  gF = c_fm g;  gZ = g u [Z + b1 > 0];  gE = g q
 * Terms follow `ops`: R_lr with DES_OP_LR, fm2 with DES_OP_FM, the Z term with DES_OP_DENSE1 (then there
 * is no pooled term: pooled feeds the first layer), the pooled term with DES_OP_POOL alone, the xdense term
 * when d and d_xdense [batch][n_dense] are given.  All pointers are device pointers; u, b1 [H]; q [F*k];
 * d [n_dense]; d_y [batch] labels in [0, 1]; d_logit, d_loss [batch] outputs; the gradient arrays are what
 * des_grads_t expects (gL, gF [batch]; gE [batch][F*k]; gZ [batch][H]).  Enqueued on `stream`. */
typedef struct {
  float b0, c_lr, c_fm;
  const float* u; const float* b1; const float* q; const float* d;
  int32_t n_dense;
} des_head_t;
typedef struct { float* gL; float* gF; float* gE; float* gZ; } des_head_grads_t;
des_status_t des_head(des_table_t* t, uint32_t ops, int32_t batch, const des_head_t* head, const des_outputs_t* out,
                      const float* d_xdense, const float* d_y, float* d_logit, float* d_loss,
                      const des_head_grads_t* g, void* stream);

/* ---- DCN cross layer under DES (Section 4.4, paragraph on DCN) --------------- */

/* y = x0 * (+)_s <x[slice s], w[slice s]> + b + x  for x0, x, y [B][d] and w, b [d]
 * (all float32, device, row-major).  w is split along d into num_shards contiguous
 * slices (slice s = columns floor(s d / S) .. floor((s+1) d / S) - 1); each shard's
 * partial is one scalar per sample, (+) adds them in shard order.  d_part [S][B]
 * (optional, may be NULL) receives the per-shard scalars, d_P [B] the aggregate
 * (needed by the backward), d_y the layer output.  No table is involved; the call
 * only enqueues kernels on `stream`.  DES_ERR_INVALID_ARG for NULL / non-positive
 * arguments or num_shards > d. */
des_status_t des_cross_forward(int32_t batch, int32_t dim, int32_t num_shards, const float* d_x0,
                               const float* d_x, const float* d_w, const float* d_b, float* d_part,
                               float* d_P, float* d_y, void* stream);

/* Backward of the same layer for an upstream gradient d_gY [B][d]: every shard can form
 * t_b = <gY_b, x0_b> by itself (x0 and gY are replicated), so no exchange is needed:
 *   gx = gY + t w,  gx0 = gY P,  gw = sum_b t_b x_b,  gb = sum_b gY_b.
 * d_gx0, d_gx [B][d]; d_gw, d_gb [d]; d_ws = caller's scratch of
 * des_cross_workspace_floats(batch, dim) floats.  The batch sums are taken in a fixed
 * order (run-to-run identical).  Applying gw / gb is the caller's dense optimizer. */
des_status_t des_cross_backward(int32_t batch, int32_t dim, const float* d_x0, const float* d_x,
                                const float* d_w, const float* d_P, const float* d_gY, float* d_gx0,
                                float* d_gx, float* d_gw, float* d_gb, float* d_ws, void* stream);
int64_t des_cross_workspace_floats(int32_t batch, int32_t dim);

/* ---- transfer volumes (Sections 4.1-4.3) ------------------------------------ */

/* Bytes one worker moves per iteration under the mesh strategy, Q = (N-1)/N (S_f + S_x),
 * and under DES, Q = 2 (N-1)/N S_M, with the saving ratio 1 - Q_DES / Q_Mesh, for
 * [0] LR, [1] FM order 2, [2] the DNN first layer.  S_f = key_bytes * uniq; S_w, S_V from
 * value_bytes, emb_dim and uniq; S_W = first_layer_bytes; the partials are B, B (k + 1)
 * and B * hidden values.  Host only, no GPU needed. */
typedef struct {
  int32_t workers;            /* N >= 2                                   */
  int64_t batch, uniq;        /* samples and unique features per batch   */
  int32_t emb_dim, hidden;    /* k and the first layer's width H         */
  int32_t key_bytes, value_bytes;   /* 8 and 4 in the paper             */
  double  first_layer_bytes;  /* S_W                                     */
} des_comm_model_t;
typedef struct { double q_mesh[3], q_des[3], saving[3]; } des_comm_volume_t;
des_status_t des_comm_volume(const des_comm_model_t* m, des_comm_volume_t* out);

/* Per-launch timing for benchmarks.  While enabled, the library records a CUDA
 * event on the call's stream behind every kernel it launches (and one at the
 * entry of every call); des_profile_read synchronises and returns, in launch
 * order, each kernel's name (static string) and the milliseconds between its
 * event and the previous one, then clears the record.  At most 16384 events
 * are kept between reads.  Off by default; costs one event record per launch. */
des_status_t des_profile_enable(des_table_t* t, int on);
des_status_t des_profile_read(des_table_t* t, const char** h_names, float* h_ms, int cap, int* h_n);

/* Number of kernel launches the library has issued for this table so far. */
uint64_t des_table_launch_count(des_table_t* t);

/* 1 when the library was built with the tcgen05 tensor-core GEMMs of the first dense
 * layer (Section 4.3), 0 when the header tree they need was missing at build time and
 * only the CUDA-core kernel exists.  des_table_uses_tensor_cores: 1 when this table's
 * first layer runs on them (built in, and F*k and H multiples of 8), else 0. */
int des_build_has_tensor_cores(void);
int des_table_uses_tensor_cores(des_table_t* t);
/* 1 in the checking build (libdes_debug.so), 0 in the product library. */
int des_build_is_debug(void);

const char* des_status_string(des_status_t s);

#ifdef __cplusplus
}
#endif
#endif /* DES_H_ */
