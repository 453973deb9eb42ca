// Eviction for streaming tables (Section 1, "Dynamic Features": under an endless stream the set of live
// features changes over time; Section 5, "Dynamic Hash Table").  The paper's table has lookup, insert and
// update; a table that can only grow fits no memory for long, so keys can be removed here: by list, or by
// age (rows carry the table's clock value of their insertion / last update).
//
// A maintenance operation, not part of the training step: it synchronises, allocates its temporaries
// (4 bytes per row, 16 bytes per surviving key of the shards it touches) and frees them again.
//   mark      every row to go gets fate = GONE (by probing the listed keys, or by comparing age stamps)
//   count     rows to go per shard -> the shard's new size m
//   pair      the freed rows below m (ascending) are paired with the surviving rows at or beyond m
//             (ascending): one block per shard walks the shard's rows in order
//   move      the surviving row's weights and state are copied into the freed row; fate = new row + 1
//   collect   the slots of the touched shards are read once: (key, new row) of every surviving key
//   clear + reinsert   the touched shards' slot regions are emptied and the survivors put back, so that
//             linear probing never meets a deleted slot (no tombstones; the probe of the step is untouched)
// Every loop is bounded (probes by the region size); a full region raises the sticky status word.
#include "des_internal.cuh"

#define FATE_GONE 0xFFFFFFFFu

struct __align__(16) LiveKey { unsigned long long key; uint32_t row, shard; };

__device__ __forceinline__ int shard_of_pos(const unsigned long long* __restrict__ base, int S, unsigned long long i) {
  int lo = 0, hi = S;                                  // base[lo] <= i < base[hi]
  while (hi - lo > 1) { const int mid = (lo + hi) >> 1; if (base[mid] <= i) lo = mid; else hi = mid; }
  return lo;
}

// by list: one thread per (key, candidate shard); HASH: the key's own shard, FIELD: any shard may hold it
__global__ void __launch_bounds__(256) evict_mark_keys_kernel(const unsigned long long* __restrict__ keys, long long n, int S,
                                                             int partition, uint32_t mod_M, uint32_t mod_two32,
                                                             const Slot* __restrict__ slots, const DevMeta* __restrict__ meta,
                                                             uint32_t* __restrict__ fate) {
  const long long per = partition == DES_PART_HASH ? 1 : S;
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n * per) return;
  const unsigned long long key = keys[i / per];
  if (key == DES_KEY_EMPTY) return;
  const unsigned long long h = des_mix64(key);
  const uint32_t s = partition == DES_PART_HASH ? des_mod_small(h, (uint32_t)S, mod_M, mod_two32) : (uint32_t)(i % per);
  const uint32_t lo = (uint32_t)meta->slot_base[s], hi = (uint32_t)meta->slot_base[s + 1], cnt = hi - lo;
  uint32_t cur = des_slot_home(h, lo, cnt);
  for (uint32_t probe = 0; probe < cnt; ++probe) {
    const Slot sl = slots[cur];
    if (sl.key == key) {
      if (sl.row != DES_ROW_NONE && sl.row < meta->n_rows[s]) fate[meta->row_base[s] + sl.row] = FATE_GONE;
      return;
    }
    if (sl.key == DES_KEY_EMPTY) return;
    cur = cur + 1 == hi ? lo : cur + 1;
  }
}

// by age: one thread per row
__global__ void __launch_bounds__(256) evict_mark_stale_kernel(const float* __restrict__ W, int k, int stride, int S,
                                                              unsigned long long total_rows, uint32_t min_clock,
                                                              const DevMeta* __restrict__ meta, uint32_t* __restrict__ fate) {
  const unsigned long long g = (unsigned long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (g >= total_rows) return;
  const int s = shard_of_pos(meta->row_base, S, g);
  if (g - meta->row_base[s] >= meta->n_rows[s]) return;
  if (__float_as_uint(W[g * stride + k + 2]) < min_clock) fate[g] = FATE_GONE;
}

// one block per shard: rows to go
__global__ void __launch_bounds__(1024) evict_count_kernel(const uint32_t* __restrict__ fate, const DevMeta* __restrict__ meta,
                                                           uint32_t* __restrict__ gone) {
  __shared__ uint32_t total;
  const int s = blockIdx.x;
  if (threadIdx.x == 0) total = 0;
  __syncthreads();
  const uint32_t n = meta->n_rows[s];
  const unsigned long long base = meta->row_base[s];
  uint32_t c = 0;
  for (uint32_t r = threadIdx.x; r < n; r += blockDim.x) c += fate[base + r] == FATE_GONE;
#pragma unroll
  for (int d = 16; d > 0; d >>= 1) c += __shfl_xor_sync(0xFFFFFFFFu, c, d);
  if ((threadIdx.x & 31) == 0 && c) atomicAdd(&total, c);
  __syncthreads();
  if (threadIdx.x == 0) gone[s] = total;
}

// one block per shard walks its rows in ascending order, 1024 at a time: freed rows below the new size and
// surviving rows at or beyond it, each list in ascending order (list_off[s] = where the shard's lists start)
__global__ void __launch_bounds__(1024) evict_pair_kernel(const uint32_t* __restrict__ fate, const DevMeta* __restrict__ meta,
                                                          const uint32_t* __restrict__ gone,
                                                          const unsigned long long* __restrict__ list_off,
                                                          uint32_t* __restrict__ holes, uint32_t* __restrict__ movers,
                                                          uint32_t* __restrict__ n_pairs) {
  __shared__ uint32_t wh[32], wm[32], carry_h, carry_m;
  const int s = blockIdx.x, lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const uint32_t e = gone[s];
  if (e == 0) { if (threadIdx.x == 0) n_pairs[s] = 0; return; }
  const uint32_t n = meta->n_rows[s], m = n - e;
  const unsigned long long base = meta->row_base[s], off = list_off[s];
  if (threadIdx.x == 0) { carry_h = 0; carry_m = 0; }
  __syncthreads();
  const unsigned lt = (1u << lane) - 1u;
  for (uint32_t chunk = 0; chunk < n; chunk += 1024) {
    const uint32_t r = chunk + threadIdx.x;
    const bool dead = r < n && fate[base + r] == FATE_GONE;
    const bool is_hole = dead && r < m, is_mover = !dead && r >= m && r < n;
    const unsigned bh = __ballot_sync(0xFFFFFFFFu, is_hole), bm = __ballot_sync(0xFFFFFFFFu, is_mover);
    if (lane == 0) { wh[warp] = __popc(bh); wm[warp] = __popc(bm); }
    __syncthreads();
    uint32_t ph = carry_h, pm = carry_m;
    for (int w2 = 0; w2 < warp; ++w2) { ph += wh[w2]; pm += wm[w2]; }
    if (is_hole) holes[off + ph + __popc(bh & lt)] = r;
    if (is_mover) movers[off + pm + __popc(bm & lt)] = r;
    __syncthreads();
    if (threadIdx.x == 0) {
      uint32_t th = 0, tm = 0;
      for (int w2 = 0; w2 < 32; ++w2) { th += wh[w2]; tm += wm[w2]; }
      carry_h += th; carry_m += tm;
    }
    __syncthreads();
  }
  if (threadIdx.x == 0) n_pairs[s] = carry_h;          // (= carry_m: as many freed rows below m as survivors beyond it)
}

// one warp per pair: the surviving row's weights and state move into the freed row
__global__ void __launch_bounds__(256) evict_move_kernel(const DevMeta* __restrict__ meta,
                                                         const unsigned long long* __restrict__ list_off,
                                                         const uint32_t* __restrict__ holes, const uint32_t* __restrict__ movers,
                                                         const uint32_t* __restrict__ n_pairs, int stride, float* W, float* A,
                                                         float* A2, uint32_t* __restrict__ fate) {
  const int s = blockIdx.y, lane = threadIdx.x & 31;
  const uint32_t np = n_pairs[s];
  const unsigned long long base = meta->row_base[s], off = list_off[s];
  for (uint32_t i = blockIdx.x * 8 + (threadIdx.x >> 5); i < np; i += gridDim.x * 8) {
    const unsigned long long to = base + holes[off + i], from = base + movers[off + i];
    for (int c = lane; c < stride; c += 32) {
      W[to * stride + c] = W[from * stride + c];
      if (A) A[to * stride + c] = A[from * stride + c];
      if (A2) A2[to * stride + c] = A2[from * stride + c];
    }
    if (lane == 0) fate[from] = holes[off + i] + 1u;
  }
}

// every slot of a touched shard: the surviving keys with their (possibly new) rows
__global__ void __launch_bounds__(256) evict_collect_kernel(const Slot* __restrict__ slots, unsigned long long total_slots,
                                                            int S, const DevMeta* __restrict__ meta,
                                                            const uint32_t* __restrict__ gone, const uint32_t* __restrict__ fate,
                                                            LiveKey* __restrict__ live, unsigned long long* __restrict__ n_live) {
  unsigned long long i = (unsigned long long)blockIdx.x * blockDim.x + threadIdx.x;
  const unsigned long long st = (unsigned long long)gridDim.x * blockDim.x;
  for (; i < total_slots; i += st) {
    const int s = shard_of_pos(meta->slot_base, S, i);
    if (gone[s] == 0) continue;
    const Slot sl = slots[i];
    if (sl.key == DES_KEY_EMPTY || sl.row == DES_ROW_NONE) continue;
    const uint32_t f = fate[meta->row_base[s] + sl.row];
    if (f == FATE_GONE) continue;
    LiveKey lk; lk.key = sl.key; lk.row = f ? f - 1u : sl.row; lk.shard = (uint32_t)s;
    live[atomicAdd(n_live, 1ull)] = lk;
  }
}

__global__ void __launch_bounds__(256) evict_clear_kernel(Slot* slots, unsigned long long total_slots, int S,
                                                          const DevMeta* __restrict__ meta, const uint32_t* __restrict__ gone) {
  unsigned long long i = (unsigned long long)blockIdx.x * blockDim.x + threadIdx.x;
  const unsigned long long st = (unsigned long long)gridDim.x * blockDim.x;
  for (; i < total_slots; i += st) {
    if (gone[shard_of_pos(meta->slot_base, S, i)] == 0) continue;
    Slot e; e.key = DES_KEY_EMPTY; e.row = DES_ROW_NONE; e.first_occ = DES_ROW_NONE;
    slots[i] = e;
  }
}

__global__ void __launch_bounds__(256) evict_reinsert_kernel(Slot* slots, DevMeta* meta, const LiveKey* __restrict__ live,
                                                             const unsigned long long* __restrict__ n_live) {
  const unsigned long long n = *n_live;
  unsigned long long i = (unsigned long long)blockIdx.x * blockDim.x + threadIdx.x;
  const unsigned long long st = (unsigned long long)gridDim.x * blockDim.x;
  for (; i < n; i += st) {
    const LiveKey lk = live[i];
    const uint32_t lo = (uint32_t)meta->slot_base[lk.shard], hi = (uint32_t)meta->slot_base[lk.shard + 1], cnt = hi - lo;
    uint32_t cur = des_slot_home(des_mix64(lk.key), lo, cnt);
    bool placed = false;
    for (uint32_t probe = 0; probe < cnt && !placed; ++probe) {
      if (atomicCAS(&slots[cur].key, DES_KEY_EMPTY, lk.key) == DES_KEY_EMPTY) {
        slots[cur].row = lk.row;                       // (first_occ stays at "never touched")
        placed = true;
      }
      cur = cur + 1 == hi ? lo : cur + 1;
    }
    if (!placed) des_raise(meta, DES_ERR_CAPACITY);      // cannot happen: the region held these keys before
  }
}

__global__ void evict_finish_kernel(DevMeta* meta, const uint32_t* __restrict__ gone, int S) {
  if ((int)threadIdx.x < S) meta->n_rows[threadIdx.x] -= gone[threadIdx.x];
}

static des_status_t evict_run(des_table_t* t, const uint64_t* d_keys, int64_t n, uint64_t min_clock, int by_age,
                              uint64_t* h_n_evicted) {
  if (h_n_evicted) *h_n_evicted = 0;
  int dev = 0;
  DES_CUDA(cudaGetDevice(&dev));
  if (dev != t->device) return DES_ERR_INVALID_ARG;
  DES_CUDA(cudaDeviceSynchronize());
  t->tag_valid = 0;                                    // rows move: whatever was derived from a batch is stale
  des_api_begin(t, 0);
  const int S = (int)t->S;
  uint32_t *fate = nullptr, *gone = nullptr, *n_pairs = nullptr, *holes = nullptr, *movers = nullptr;
  unsigned long long *list_off = nullptr, *n_live = nullptr;
  LiveKey* live = nullptr;
  des_status_t rc = DES_OK;
  uint32_t h_gone[DES_MAX_SHARDS];
  unsigned long long h_off[DES_MAX_SHARDS + 1], total_gone = 0, survivors = 0;
  uint64_t h_rows[DES_MAX_SHARDS];
  auto bail = [&](des_status_t code) {
    cudaDeviceSynchronize();
    cudaFree(fate); cudaFree(gone); cudaFree(n_pairs); cudaFree(holes); cudaFree(movers); cudaFree(list_off);
    cudaFree(n_live); cudaFree(live);
    if (code == DES_ERR_CUDA) cudaGetLastError();
    return code;
  };
#define EV_CUDA(x) do { if ((x) != cudaSuccess) return bail(DES_ERR_CUDA); } while (0)
#define EV_LAUNCH(name) do { if (des_prof_mark(t, name, 1)) return bail(DES_ERR_CUDA); } while (0)
  EV_CUDA(cudaMalloc(&fate, (t->total_rows + 1) * 4));
  EV_CUDA(cudaMalloc(&gone, DES_MAX_SHARDS * 4));
  EV_CUDA(cudaMalloc(&n_pairs, DES_MAX_SHARDS * 4));
  EV_CUDA(cudaMalloc(&list_off, (DES_MAX_SHARDS + 1) * 8));
  EV_CUDA(cudaMalloc(&n_live, 8));
  EV_CUDA(cudaMemset(fate, 0, (t->total_rows + 1) * 4));
  EV_CUDA(cudaMemset(n_live, 0, 8));
  if (by_age) {
    const unsigned long long rows = t->total_rows;
    const uint32_t mc = min_clock > 0xFFFFFFFFull ? 0xFFFFFFFFu : (uint32_t)min_clock;
    evict_mark_stale_kernel<<<(unsigned)((rows + 255) / 256), 256>>>(t->W, (int)t->k, (int)t->stride, S, rows, mc, t->meta, fate);
    EV_LAUNCH("evict_mark_stale_kernel");
  } else if (n > 0) {
    uint32_t M, two32;
    des_mod_consts(t->S, &M, &two32);
    const long long threads = n * (t->cfg.partition == DES_PART_HASH ? 1 : S);
    evict_mark_keys_kernel<<<(unsigned)((threads + 255) / 256), 256>>>((const unsigned long long*)d_keys, n, S,
                                                                      (int)t->cfg.partition, M, two32, t->slots, t->meta, fate);
    EV_LAUNCH("evict_mark_keys_kernel");
  }
  evict_count_kernel<<<S, 1024>>>(fate, t->meta, gone);
  EV_LAUNCH("evict_count_kernel");
  EV_CUDA(cudaMemcpy(h_gone, gone, S * 4, cudaMemcpyDeviceToHost));
  if ((rc = des_table_size(t, h_rows)) != DES_OK) return bail(rc);
  for (int s = 0; s < S; ++s) {
    h_off[s] = total_gone;
    total_gone += h_gone[s];
    if (h_gone[s]) survivors += h_rows[s] - h_gone[s];
  }
  h_off[S] = total_gone;
  if (total_gone == 0) return bail(DES_OK);
  EV_CUDA(cudaMemcpy(list_off, h_off, (S + 1) * 8, cudaMemcpyHostToDevice));
  EV_CUDA(cudaMalloc(&holes, total_gone * 4));
  EV_CUDA(cudaMalloc(&movers, total_gone * 4));
  EV_CUDA(cudaMalloc(&live, (survivors + 1) * sizeof(LiveKey)));
  evict_pair_kernel<<<S, 1024>>>(fate, t->meta, gone, list_off, holes, movers, n_pairs);
  EV_LAUNCH("evict_pair_kernel");
  evict_move_kernel<<<dim3((unsigned)(t->sm_count * 4), (unsigned)S), 256>>>(t->meta, list_off, holes, movers, n_pairs,
                                                                             (int)t->stride, t->W, t->A, t->A2, fate);
  EV_LAUNCH("evict_move_kernel");
  evict_collect_kernel<<<t->sm_count * 8, 256>>>(t->slots, t->total_slots, S, t->meta, gone, fate, live, n_live);
  EV_LAUNCH("evict_collect_kernel");
  evict_clear_kernel<<<t->sm_count * 8, 256>>>(t->slots, t->total_slots, S, t->meta, gone);
  EV_LAUNCH("evict_clear_kernel");
  evict_reinsert_kernel<<<t->sm_count * 8, 256>>>(t->slots, t->meta, live, n_live);
  EV_LAUNCH("evict_reinsert_kernel");
  evict_finish_kernel<<<1, DES_MAX_SHARDS>>>(t->meta, gone, S);
  EV_LAUNCH("evict_finish_kernel");
  EV_CUDA(cudaDeviceSynchronize());
#undef EV_CUDA
#undef EV_LAUNCH
  if (h_n_evicted) *h_n_evicted = total_gone;
  return bail(DES_OK);
}

extern "C" des_status_t des_table_evict_keys(des_table_t* t, const uint64_t* d_keys, int64_t n, uint64_t* h_n_evicted) {
  if (!t || n < 0 || (n > 0 && !d_keys)) return DES_ERR_INVALID_ARG;
  return evict_run(t, d_keys, n, 0, 0, h_n_evicted);
}

extern "C" des_status_t des_table_evict_stale(des_table_t* t, uint64_t min_clock, uint64_t* h_n_evicted) {
  if (!t) return DES_ERR_INVALID_ARG;
  return evict_run(t, nullptr, 0, min_clock, 1, h_n_evicted);
}

extern "C" des_status_t des_table_clock(des_table_t* t, uint64_t* h_clock) {
  if (!t || !h_clock) return DES_ERR_INVALID_ARG;
  DES_CUDA(cudaDeviceSynchronize());
  unsigned long long c = 0;
  DES_CUDA(cudaMemcpy(&c, &t->meta->clock, 8, cudaMemcpyDeviceToHost));
  *h_clock = c;
  return DES_OK;
}
