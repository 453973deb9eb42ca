// Internal declarations of the DES CUDA library (sm_100a).  Nothing in here is
// shared with the CPU oracle.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "des.h"

#define DES_MAX_SHARDS 64
#define DES_SLOT_NONE 0xFFFFFFFFu
#define HOT_RCHUNK 16u     // replica rows of a hot key summed by one warp of the backward's replica reduction

// The few keys that own a large share of a skewed batch ("super" keys) are counted instead of scattered in the
// backward: a tagged occurrence carries SUPER_TAG | slot where other occurrences carry a gradient row number.
#define SUPER_T 16u             // slots
#define SUPER_TAG 0xFFFFFF00u   // tag | slot; DES_ROW_NONE (low byte 0xFF) is not a tag
// Layout of the hot-key counter block (des_table::hot_ctr, 64 words):
//   [0] hot keys  [1] replica rows  [2] work items  [3] super slots claimed
//   [4 + t]   hot index of super slot t (DES_ROW_NONE: slot unused)
#define HOT_CTR_WORDS 64
#define HOT_CTR_SLOT 4

// One open-addressing slot: 16 bytes, read with a single vector load.
//   key        DES_KEY_EMPTY until claimed by a 64-bit CAS; never changes after.
//   row        shard-local row, DES_ROW_NONE until the key's insert call numbers it.
//   first_occ  scratch of find_or_insert: scratch_base + (smallest occurrence index of
//              the key in the call's batch).  Every call works scratch_base - nnz below the
//              call before it, so what earlier calls left behind is larger than anything
//              the running call writes and never needs to be cleared; when the base runs
//              out (every few billion occurrences) the call that used its last part resets
//              all slots to DES_ROW_NONE, the value of a slot that was never touched, once
//              it has read them.
struct __align__(16) Slot {
  unsigned long long key;
  uint32_t row;
  uint32_t first_occ;
};

// Per-table metadata that kernels read through a pointer (broadcast loads).
struct DevMeta {
  unsigned long long row_base[DES_MAX_SHARDS + 1];   // first table-global row of shard s
  unsigned long long slot_base[DES_MAX_SHARDS + 1];  // first slot of shard s's region
  uint32_t row_cap[DES_MAX_SHARDS];                  // row capacity of shard s
  uint32_t n_rows[DES_MAX_SHARDS];                   // rows in use
  uint32_t new_total[DES_MAX_SHARDS];                // new keys of the running insert call
  uint32_t n_uniq;                                   // unique keys of the running insert call
  uint32_t err;                                      // sticky des_status_t raised on device
  uint32_t any_new;                                  // the running insert call has at least one new key
  uint32_t scratch_base;                             // see Slot::first_occ: the last insert call's base
  uint32_t field_order[1024];                        // fields sorted by (owning shard, field)
  unsigned long long clock;                          // inserting find_or_insert calls so far: the age clock that
                                                     // stamps a row when it is inserted or updated (eviction by age)
  unsigned long long opt_step;                       // backward calls so far (Adam's t), advanced on device
  float adam_c1, adam_c2;                            // 1 - beta1^t, 1 - beta2^t for the running step
};

// Checking build (-DDES_DEBUG, libdes_debug.so): the bounds every gather, scatter and probe is held to.
struct DbgBounds {
  unsigned long long rows;        // table rows + 1 (the all-zero row behind the table is a legal gather target)
  unsigned long long slots;       // slots of all shards
  unsigned long long grad_rows;   // gradient rows: unique keys + replica rows
  unsigned long long nnz;         // occurrences the workspace holds
  DevMeta* meta;                  // where DES_ERR_RANGE is raised
};

struct des_table {
  des_config_t cfg;
  DbgBounds dbg;
  int device;
  uint32_t S, F, k, H, stride;       // stride = k + 4 floats per row
  uint64_t total_rows, total_slots;
  uint64_t h_row_base[DES_MAX_SHARDS + 1], h_slot_base[DES_MAX_SHARDS + 1];
  int64_t max_nnz; int32_t max_batch; int64_t max_uniq;
  uint32_t nblk_max;                 // scan-block capacity of the workspace
  // device memory
  Slot* slots;
  float* W;                          // [total_rows][stride]: latent vector v[k], linear weight, |v|^2, 2 pad
  float* A;                          // same shape, first optimizer-state word: Adagrad accumulator / Adam m;
                                     // tail = (linear weight's state 1, state 2): Adagrad acc | Adam m, v | FTRL n, z
  float* A2;                         // same shape, second state word of the latent vector (Adam v); NULL otherwise
  DevMeta* meta;
  // find_or_insert workspace
  uint32_t* slot_of;                 // [max_nnz]
  uint8_t* flags;                    // [max_nnz]
  uint32_t* uslot;                   // [max_nnz]
  uint32_t* blk_cnt;                 // [(S+1)][nblk_max]
  int32_t* seg_off;                  // [max_batch][S+1] forward routing: (sample, shard) segment bounds
  // backward workspace
  float* Gbuf;                       // [max_uniq + rep_max][stride]: per-unique gradient rows, then
                                     // hot-key replica rows; all zero between calls
  uint32_t* hinfo;                   // [max_uniq] sampled count, then hot index; zero between calls
  uint32_t* dest;                    // [max_nnz] gradient row of each occurrence (or SUPER_TAG | slot), made by the
                                     // hot-key pass that opens the backward; scratch of find_or_insert before that
  float* x_sorted;                   // [max_nnz] forward routing: feature values in shard-major order
  float2* bag_tail;                  // [max_batch * F] single-gather forward: per-bag sums of (w x, |v|^2 x^2)
  // which batch the tags in dest[] / the hot lists belong to (they are rebuilt when another batch comes)
  const void* tag_uidx; long long tag_nnz; int tag_valid; int tag_super;
  uint32_t *hot_base, *hot_R, *hot_u, *hot_ctr;   // hot list [hot_max] and its two counters
  uint32_t* hot_work;                // [work_max] (hot index << 18 | chunk) items of the replica reduction
  double* hot_acc;                   // [hot_max][stride] double sums of the replicas; zero between calls
  float* super_cnt;                  // [max_batch * F][16] per-bag counts of the register-summed keys (k > 28 only)
  uint32_t hot_max, rep_max, work_max;
  // first dense layer
  float* W1; float* accW1;           // [F*k][H] fp32 master and state
  float* acc2W1;                     // Adam's second moment of W1 (NULL otherwise)
  __nv_bfloat16* W1b;                // bf16 shadow
  float* gW1_part; int gw1_splits;   // [splits][F*k][H]
  int use_tc;                        // tensor-core GEMM path usable for this table's shapes
  __nv_bfloat16 *pooled_b, *gZ_b;    // bf16 copies of V [max_batch][F*k] and gZ [max_batch][H]
  const float* pooled_b_src;         // the pooled array whose bf16 copy the pooling kernel has just left in pooled_b
                                     // (consumed, once, by the first-layer product that follows); NULL otherwise
  void* gemm_ws; size_t gemm_ws_bytes;
  // host-step staging
  int32_t* st_offsets[2]; unsigned long long* st_ids[2]; float* st_vals[2];   // two input slots (pipelined submit)
  cudaStream_t st_copy_stream; cudaEvent_t st_copied[2], st_done[2]; int st_busy[2]; uint64_t st_next;
  int st_ready;                      // staging, copy stream and events all exist
  uint32_t* st_rows; uint8_t* st_shards; uint32_t* st_uidx; uint32_t* st_uniq_rows; uint32_t* st_n_uniq;
  float* st_part_small; float* st_out_small;
  uint64_t launches;
  int sm_count;
  // optional per-launch timing (des_profile_*): one event after every launch, and one at API entry
  int prof_on, prof_n;
  cudaStream_t cur_stream;
  cudaEvent_t* prof_ev;              // [DES_PROF_MAX]
  const char** prof_name;            // [DES_PROF_MAX], NULL = API-entry marker
};
#define DES_PROF_MAX 16384

#define DES_CUDA(x) do { cudaError_t e_ = (x); if (e_ != cudaSuccess) return DES_ERR_CUDA; } while (0)
// after every kernel launch: count it, check the launch, and (when profiling) drop an event behind it
int des_prof_mark(des_table* t, const char* name, int check);
void des_api_begin(des_table* t, cudaStream_t cs);
#define DES_LAUNCH_CHECK(t, name) do { if (des_prof_mark((t), (name), 1)) return DES_ERR_CUDA; } while (0)

// ---- device helpers ---------------------------------------------------------

// Table mixer: the three xor-shift / odd-multiply rounds of the splitmix64
// finaliser; a bijection on 64-bit words.
__host__ __device__ __forceinline__ unsigned long long des_mix64(unsigned long long z) {
  z ^= z >> 30; z *= 0xBF58476D1CE4E5B9ull;
  z ^= z >> 27; z *= 0x94D049BB133111EBull;
  z ^= z >> 31;
  return z;
}

// x mod S for a 32-bit x and a small S, exactly, without a division: with M = floor(2^32 / S) + 1 the
// quotient estimate q = floor(x M / 2^32) is floor(x / S) or one more, so x - q S is the remainder or the
// remainder minus S (x M / 2^32 = x / S + x e / 2^32 with 0 < e <= 1, i.e. less than x / S + 1).
__device__ __forceinline__ uint32_t des_mod32(uint32_t x, uint32_t S, uint32_t M) {
  const int r = (int)(x - __umulhi(x, M) * S);
  return (uint32_t)(r < 0 ? r + (int)S : r);
}

// h mod S for a small S (<= 64), exactly:
// h = hi * 2^32 + lo  =>  h mod S = ((hi mod S) * (2^32 mod S) + lo mod S) mod S,
// with M = floor(2^32 / S) + 1 and two32 = 2^32 mod S computed once on the host (des_mod_consts).
__device__ __forceinline__ uint32_t des_mod_small(unsigned long long h, uint32_t S, uint32_t M, uint32_t two32) {
  if (S == 1u) return 0u;                              // (M does not fit 32 bits for S = 1)
  const uint32_t hi = (uint32_t)(h >> 32), lo = (uint32_t)h;
  return des_mod32(des_mod32(hi, S, M) * two32 + des_mod32(lo, S, M), S, M);
}
static inline void des_mod_consts(uint32_t S, uint32_t* M, uint32_t* two32) {
  *M = (uint32_t)((1ull << 32) / S + 1ull);
  *two32 = (uint32_t)((1ull << 32) % S);
}

// Philox4x32-10 block function.
__device__ __forceinline__ uint4 des_philox(uint4 c, uint2 key) {
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    uint32_t hi0 = __umulhi(0xD2511F53u, c.x), lo0 = 0xD2511F53u * c.x;
    uint32_t hi1 = __umulhi(0xCD9E8D57u, c.z), lo1 = 0xCD9E8D57u * c.z;
    c = make_uint4(hi1 ^ c.y ^ key.x, lo1, hi0 ^ c.w ^ key.y, lo0);
    key.x += 0x9E3779B9u; key.y += 0xBB67AE85u;
  }
  return c;
}

// Uniform in [-scale, scale) from the top 24 bits; exact up to the last multiply.
__device__ __forceinline__ float des_u24(uint32_t r, float scale) {
  float x = __fmul_rn(__uint2float_rn(r >> 8), 1.0f / 8388608.0f);
  return __fmul_rn(__fsub_rn(x, 1.0f), scale);
}

// Four consecutive components 4q..4q+3 of the initial latent vector of `id`.
__device__ __forceinline__ float4 des_init4(unsigned long long seed, unsigned long long id, uint32_t q, float scale) {
  uint4 r = des_philox(make_uint4(q, 0u, (uint32_t)seed, (uint32_t)(seed >> 32)),
                       make_uint2((uint32_t)id, (uint32_t)(id >> 32)));
  return make_float4(des_u24(r.x, scale), des_u24(r.y, scale), des_u24(r.z, scale), des_u24(r.w, scale));
}

// Index of the bag that holds occurrence j: largest i with offsets[i] <= j
// among bags that are not past the end (handles empty bags).
__device__ __forceinline__ int des_bag_of(const int32_t* __restrict__ offsets, int nbags, int j) {
  int lo = 0, hi = nbags;             // invariant: offsets[lo] <= j < offsets[hi]
  while (hi - lo > 1) {
    int mid = (lo + hi) >> 1;
    if (__ldg(offsets + mid) <= j) lo = mid; else hi = mid;
  }
  return lo;
}

__device__ __forceinline__ void des_raise(DevMeta* meta, uint32_t code) { atomicCAS(&meta->err, 0u, code); }

// First slot a key is looked for in, inside its shard's region of n slots starting at lo: the top bits of an odd
// multiple of the mixed key (the shard is the same word's residue mod S, so the two are independent).
__device__ __forceinline__ uint32_t des_slot_home(unsigned long long mixed, uint32_t lo, uint32_t n) {
  return lo + (uint32_t)__umul64hi(mixed * 0x9E3779B97F4A7C15ull, (unsigned long long)n);
}
// The age stamp lives in the third word of a row's 16-byte tail, stored as raw bits.
__device__ __forceinline__ float des_stamp_bits(unsigned long long clock) { return __uint_as_float((uint32_t)clock); }

// Optimizer parameters handed to the update kernels by value.
struct OptParams {
  int optimizer, lin_optimizer;
  float lr, eps;
  float beta1, beta2, c1, c2;          // Adam: c1 = 1 - beta1^t, c2 = 1 - beta2^t (filled on device, see des_opt_load)
  float ftrl_alpha, ftrl_beta, ftrl_l1, ftrl_l2;
};

// One application of SGD / Adagrad / Adam to one parameter.  s1, s2: first and
// second state word (Adagrad: accumulator, -; Adam: m, v).
__device__ __forceinline__ void des_opt_step(const OptParams& o, float& theta, float& s1, float& s2, float G) {
  if (o.optimizer == DES_OPT_ADAGRAD) {
    s1 = s1 + G * G;
    theta = theta - o.lr * G / (sqrtf(s1) + o.eps);
  } else if (o.optimizer == DES_OPT_ADAM) {
    s1 = o.beta1 * s1 + (1.f - o.beta1) * G;
    s2 = o.beta2 * s2 + (1.f - o.beta2) * G * G;
    theta = theta - o.lr * (s1 / o.c1) / (sqrtf(s2 / o.c2) + o.eps);
  } else {
    theta = theta - o.lr * G;
  }
}

// FTRL-Proximal on one coordinate: state n (sum of squared gradients) and z.
__device__ __forceinline__ void des_ftrl_step(const OptParams& o, float& w, float& n, float& z, float G) {
  const float n1 = n + G * G;
  const float sigma = (sqrtf(n1) - sqrtf(n)) / o.ftrl_alpha;
  z = z + G - sigma * w;
  n = n1;
  if (fabsf(z) <= o.ftrl_l1) { w = 0.f; return; }
  const float sgn = z > 0.f ? 1.f : -1.f;
  w = -(z - sgn * o.ftrl_l1) / ((o.ftrl_beta + sqrtf(n1)) / o.ftrl_alpha + o.ftrl_l2);
}

OptParams des_opt_params(des_table* t);

// The launch carries the configured constants; Adam's bias corrections live in
// device memory (advanced by one small kernel per backward call) so that a
// backward captured into a CUDA graph keeps counting steps when replayed.
__device__ __forceinline__ OptParams des_opt_load(const OptParams& o, const DevMeta* __restrict__ meta) {
  OptParams r = o;
  if (o.optimizer == DES_OPT_ADAM) { r.c1 = meta->adam_c1; r.c2 = meta->adam_c2; }
  return r;
}

// ---- checking build -----------------------------------------------------------
// In the product library these macros cost nothing.  In the checking build every translation unit keeps a
// copy of the running table's bounds in device memory (armed at the entry of every call that launches
// gathers or scatters); an index outside them raises the table's sticky status word and the access is
// skipped or redirected to the all-zero row — never performed.
#ifdef DES_DEBUG
static __device__ DbgBounds g_dbg;
__device__ __forceinline__ bool des_dbg_in(unsigned long long i, unsigned long long n) {
  if (i < n) return true;
  if (g_dbg.meta) atomicCAS(&g_dbg.meta->err, 0u, (uint32_t)DES_ERR_RANGE);
  return false;
}
#define DES_DBG_ROW(g) (des_dbg_in((unsigned long long)(g), g_dbg.rows) ? (g) : (uint32_t)(g_dbg.rows - 1ull))
#define DES_DBG_SLOT_OK(i) des_dbg_in((unsigned long long)(i), g_dbg.slots)
#define DES_DBG_GRAD_OK(d) des_dbg_in((unsigned long long)(d), g_dbg.grad_rows)
#define DES_DBG_OCC_OK(j) des_dbg_in((unsigned long long)(j), g_dbg.nnz)
#define DES_DBG_ARM(t, cs)                                                                                            \
  do {                                                                                                                \
    if (cudaMemcpyToSymbolAsync(g_dbg, &(t)->dbg, sizeof(DbgBounds), 0, cudaMemcpyHostToDevice, (cs)) != cudaSuccess) \
      return DES_ERR_CUDA;                                                                                            \
  } while (0)
#else
#define DES_DBG_ROW(g) (g)
#define DES_DBG_SLOT_OK(i) true
#define DES_DBG_GRAD_OK(d) true
#define DES_DBG_OCC_OK(j) true
#define DES_DBG_ARM(t, cs) do { } while (0)
#endif

// shared declarations across translation units
des_status_t des_check_batch(const des_table* t, const des_batch_t* b, int need_dedup);
des_status_t des_dense1_forward(des_table* t, const float* pooled, int B, float* Z, float* part_dense,
                                const float* part_pooled, cudaStream_t st);
des_status_t des_dense1_backward(des_table* t, const float* pooled, const float* gE, const float* gZ,
                                 float* gE_work, int B, cudaStream_t st);
// Hot-key pass over a batch's unique indices (sampled counts, hot list, replica assignment, dest[] with
// the super-key tags); a no-op when dest[] already belongs to this batch (a second backward over it).
des_status_t des_tags_ensure(des_table* t, const des_batch_t* b, cudaStream_t st);
