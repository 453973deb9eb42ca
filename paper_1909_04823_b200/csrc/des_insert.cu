// lookup + insert on the dynamic hash table (Section 5, "Dynamic Hash Table"),
// including shard routing (Section 5, "Large-scale Sparse Features": weights of
// field f live on node f mod N; Section 4.2: any balanced partition).
//
// One call = nine short kernels, none of which waits on another thread; the table's slots are read
// once per occurrence by the probe and once more by flag_count, and written only for new keys:
//   probe_claim   every occurrence finds its key's slot in the owning shard's
//                 region (linear probing) or claims an empty one with a 64-bit
//                 CAS; the slot remembers the smallest occurrence index.
//   flag_count    occurrence j is the FIRST of its key iff the slot remembers j,
//                 and the key is NEW iff its slot has no row yet; per-block
//                 counts of firsts and of new keys per shard.  Leaves the
//                 slot's row and the first occurrence's index per occurrence.
//   scan          exclusive scan of those counts over blocks.
//   assign        first occurrences get the batch-unique index (rank among
//                 firsts) and, for new keys, the next shard-local row (rank
//                 among the shard's new keys): both in CSR order, so the result
//                 does not depend on thread scheduling.  Two kernels: the ranks
//                 among firsts always, the new-key numbering only when the
//                 batch has a new key at all (that kernel also clears the slots'
//                 scratch words when their range runs out, see Slot::first_occ).
//   apply_first   one thread per unique key: the key's unique index (and a new
//                 key's row) at its first occurrence, a new key's row into its
//                 slot; init_new_rows then fills the new keys' rows from the
//                 counter-based generator (a lane group per row).
//   resolve       every other occurrence takes row and unique index from its
//                 key's first occurrence.
//   finish        shard sizes advance, the call's scratch range is retired.
#include "des_internal.cuh"

#define IB 1024  // occurrences per block (tile) in every per-occurrence kernel of this file

// A probe may read a slot through L1 although other SMs claim slots meanwhile: a key never changes once
// it is set, so a stale line can only show EMPTY where a key now is (the CAS that follows returns the
// truth) or a too-large scratch word (the atomicMin that follows is then merely redundant).
// (One 16-byte load; "volatile" keeps the compiler from reusing an earlier read of the same slot.)
__device__ __forceinline__ Slot load_slot(const Slot* p) {
  unsigned long long a, b;
  asm volatile("ld.global.ca.v2.u64 {%0, %1}, [%2];" : "=l"(a), "=l"(b) : "l"(p));
  Slot s;
  s.key = a; s.row = (uint32_t)b; s.first_occ = (uint32_t)(b >> 32);
  return s;
}

// Occurrences per thread and resident blocks per SM: one probe chain per thread at full occupancy
// measured fastest (more chains per thread cost registers, hence warps in flight; electing one lane
// per distinct key of a warp costs more in match instructions than the cached slot loads it saves).
#ifndef PROBE_ILP
#define PROBE_ILP 1
#endif
#ifndef PROBE_MINB
#define PROBE_MINB 8
#endif

struct SlotGeom {
  unsigned long long slot_base[DES_MAX_SHARDS + 1];
  uint32_t mod_M, mod_two32;        // constants of the division-free mod S (des_mod_consts)
};   // kernel parameter: constant-bank reads

__global__ void __launch_bounds__(256, PROBE_MINB) probe_claim_kernel(
    const unsigned long long* __restrict__ ids, const int32_t* __restrict__ offsets, int nnz, int nbags,
    int S, int F, int partition, int insert, uint32_t world, uint32_t rank, Slot* slots, DevMeta* meta,
    const __grid_constant__ SlotGeom geom, uint32_t* __restrict__ slot_of, uint8_t* __restrict__ shards,
    uint32_t* __restrict__ rows) {
  // occurrence j = tile * (256 * PROBE_ILP) + q * 256 + thread: every access of a warp is contiguous.
  // Per occurrence the probe keeps its key, the table-global slot it looks at (DES_SLOT_NONE once it
  // is done) and the bounds of the owning shard's slot region: all 32-bit but the key.
  // the bounds of the shards' slot regions, staged once per block: indexing the kernel parameter by a
  // per-lane shard would replay the constant-bank read once per distinct shard of the warp
  __shared__ uint32_t s_base[DES_MAX_SHARDS + 1];
  if (threadIdx.x <= (unsigned)S) s_base[threadIdx.x] = (uint32_t)geom.slot_base[threadIdx.x];
  __syncthreads();
  const uint32_t base = meta->scratch_base - (uint32_t)nnz;   // this call's scratch range (Slot::first_occ)
  const int j0 = blockIdx.x * (256 * PROBE_ILP) + threadIdx.x;
  unsigned long long id[PROBE_ILP];
  uint32_t cur[PROBE_ILP], lo[PROBE_ILP], hi[PROBE_ILP], found[PROBE_ILP], row[PROBE_ILP], seen_fo[PROBE_ILP];
  uint32_t nmax = 0;
#pragma unroll
  for (int q = 0; q < PROBE_ILP; ++q) {
    const int j = j0 + q * 256;
    cur[q] = DES_SLOT_NONE; found[q] = DES_SLOT_NONE; row[q] = DES_ROW_NONE; seen_fo[q] = DES_ROW_NONE;
    id[q] = 0; lo[q] = 0; hi[q] = 0;
    if (j < nnz) {
      id[q] = ids[j];
      uint32_t s;
      const unsigned long long h = des_mix64(id[q]);
      if (partition == DES_PART_HASH) s = des_mod_small(h, (uint32_t)S, geom.mod_M, geom.mod_two32);
      else s = (uint32_t)(des_bag_of(offsets, nbags, j) % F) % (unsigned)S;
      shards[j] = (uint8_t)s;
      if (id[q] == DES_KEY_EMPTY) {
        des_raise(meta, DES_ERR_RESERVED_KEY);
      } else if (world > 1 && s % world != rank) {
        // another process holds this shard: the occurrence has no row here
      } else {
        lo[q] = s_base[s];
        hi[q] = s_base[s + 1];
        const uint32_t n = hi[q] - lo[q];
        // position inside the region: the top bits of an odd multiple of the same mixed word (the shard is its
        // residue mod S; a second full mixing round bought nothing measurable in probe lengths)
        cur[q] = des_slot_home(h, lo[q], n);
        nmax = max(nmax, n);
      }
    }
  }
  for (uint32_t probe = 0; probe < nmax; ++probe) {
    Slot sl[PROBE_ILP];
    bool any = false;
#pragma unroll
    for (int q = 0; q < PROBE_ILP; ++q) {
      if (cur[q] != DES_SLOT_NONE && !DES_DBG_SLOT_OK(cur[q])) cur[q] = DES_SLOT_NONE;   // (checking build)
      if (cur[q] != DES_SLOT_NONE) { sl[q] = load_slot(slots + cur[q]); any = true; }
    }
    if (!any) break;
#pragma unroll
    for (int q = 0; q < PROBE_ILP; ++q) {
      if (cur[q] == DES_SLOT_NONE) continue;
      bool done = false;
      if (sl[q].key == id[q]) {
        found[q] = cur[q]; row[q] = sl[q].row; seen_fo[q] = sl[q].first_occ;
        done = true;
      } else if (sl[q].key == DES_KEY_EMPTY) {
        if (!insert) {
          done = true;
        } else {
          const unsigned long long old = atomicCAS(&slots[cur[q]].key, DES_KEY_EMPTY, id[q]);
          if (old == DES_KEY_EMPTY || old == id[q]) { found[q] = cur[q]; done = true; }
        }
      }
      if (!done && probe + 1 >= hi[q] - lo[q]) {       // region is full
        done = true;
        if (insert) des_raise(meta, DES_ERR_CAPACITY);
      }
      cur[q] = done ? DES_SLOT_NONE : (cur[q] + 1 == hi[q] ? lo[q] : cur[q] + 1);
    }
  }
#pragma unroll
  for (int q = 0; q < PROBE_ILP; ++q) {
    const int j = j0 + q * 256;
    if (j >= nnz) continue;
    // the slot's scratch word as seen by the probe may be stale (or an earlier call's), but only ever
    // too LARGE: skipping the atomic when it is already smaller than this occurrence's is safe
    if (found[q] != DES_SLOT_NONE && insert && seen_fo[q] > base + (uint32_t)j)
      atomicMin(&slots[found[q]].first_occ, base + (uint32_t)j);
    if (insert) slot_of[j] = found[q];
    else rows[j] = row[q];
  }
}

// flags: bit0 = first occurrence of its key in the batch, bit1 = key is new.  This is the only pass
// that reads every occurrence's slot after the claims: it also leaves the slot's row (DES_ROW_NONE for a
// new key) in rows[] and the index of the key's first occurrence in first_of[], which is all that the
// later passes need.
__global__ void __launch_bounds__(IB / 4) flag_count_kernel(
    int nnz, int S, const Slot* __restrict__ slots, const DevMeta* __restrict__ meta,
    const uint32_t* __restrict__ slot_of, const uint8_t* __restrict__ shards, uint8_t* __restrict__ flags,
    uint32_t* __restrict__ rows, uint32_t* __restrict__ first_of, uint32_t* __restrict__ blk_cnt, int nblk_max) {
  // IB occurrences per block, IB / 4 threads: a thread's four slot look-ups are in flight together
  __shared__ uint32_t cnt[DES_MAX_SHARDS + 1];
  if (threadIdx.x <= DES_MAX_SHARDS) cnt[threadIdx.x] = 0;
  __syncthreads();
  const uint32_t base = meta->scratch_base - (uint32_t)nnz;
  const int j0 = blockIdx.x * IB + threadIdx.x;
  uint32_t so[4];
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    const int j = j0 + q * (IB / 4);
    so[q] = (j < nnz) ? slot_of[j] : DES_SLOT_NONE;
    if (so[q] != DES_SLOT_NONE && !DES_DBG_SLOT_OK(so[q])) so[q] = DES_SLOT_NONE;              // (checking build)
  }
  uint2 rf[4];                                         // (row, first_occ): the slot's second half
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    rf[q] = make_uint2(DES_ROW_NONE, DES_ROW_NONE);
    if (so[q] != DES_SLOT_NONE) rf[q] = reinterpret_cast<const uint2*>(slots + so[q])[1];
  }
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    const int j = j0 + q * (IB / 4);
    uint8_t fl = 0;
    if (j < nnz) {
      const bool mapped = so[q] != DES_SLOT_NONE;
      if (mapped && rf[q].y == base + (uint32_t)j) fl = (rf[q].x == DES_ROW_NONE) ? 3 : 1;
      flags[j] = fl;
      rows[j] = rf[q].x;
      first_of[j] = mapped ? rf[q].y - base : DES_ROW_NONE;
    }
    const unsigned firsts = __ballot_sync(0xFFFFFFFFu, fl & 1);
    if ((threadIdx.x & 31) == 0 && firsts) atomicAdd(&cnt[0], __popc(firsts));
    if (fl & 2) atomicAdd(&cnt[1 + shards[j]], 1u);
  }
  __syncthreads();
  if (threadIdx.x <= S) blk_cnt[(size_t)threadIdx.x * nblk_max + blockIdx.x] = cnt[threadIdx.x];
}

// One block per sequence (sequence 0 = firsts, 1 + s = new keys of shard s):
// in-place exclusive scan over the blocks of the batch, total to meta.
__global__ void __launch_bounds__(1024) scan_blocks_kernel(uint32_t* blk_cnt, int nblk, int nblk_max, DevMeta* meta) {
  // Warp w owns the contiguous chunk [w * per, (w + 1) * per) of the sequence and walks it 32 entries at a
  // time (coalesced loads and stores, a warp scan per row, a running carry); the 32 warp totals are scanned
  // in between, and sequences that are all zero (new keys of a shard in a populated table) are not rewritten.
  __shared__ uint32_t wsum[32];
  __shared__ uint32_t s_total;
  uint32_t* seq = blk_cnt + (size_t)blockIdx.x * nblk_max;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int per = ((nblk + 31) / 32 + 31) / 32 * 32;          // entries per warp, a multiple of 32
  const int lo = warp * per, hi = min(nblk, lo + per);
  uint32_t sum = 0;
  for (int i = lo + lane; i < hi; i += 32) sum += seq[i];
#pragma unroll
  for (int d = 16; d > 0; d >>= 1) sum += __shfl_xor_sync(0xFFFFFFFFu, sum, d);
  if (lane == 0) wsum[warp] = sum;
  __syncthreads();
  if (threadIdx.x < 32) {
    uint32_t w = wsum[threadIdx.x], wi = w;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      uint32_t v = __shfl_up_sync(0xFFFFFFFFu, wi, d);
      if (threadIdx.x >= d) wi += v;
    }
    wsum[threadIdx.x] = wi - w;
    if (threadIdx.x == 31) {
      s_total = wi;
      if (blockIdx.x == 0) meta->n_uniq = wi;
      else { meta->new_total[blockIdx.x - 1] = wi; if (wi) atomicOr(&meta->any_new, 1u); }
    }
  }
  __syncthreads();
  if (s_total == 0u) return;                                  // an all-zero sequence is its own exclusive scan
  uint32_t carry = wsum[warp];
  for (int base = lo; base < hi; base += 32) {
    const int i = base + lane;
    const uint32_t v = (i < hi) ? seq[i] : 0u;
    uint32_t incl = v;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      const uint32_t o = __shfl_up_sync(0xFFFFFFFFu, incl, d);
      if (lane >= d) incl += o;
    }
    if (i < hi) seq[i] = carry + incl - v;
    carry += __shfl_sync(0xFFFFFFFFu, incl, 31);
  }
}

// The common case of assign_kernel below — a batch without a single new key — needs the rank among the
// first occurrences only: IB occurrences per block, four consecutive ones per thread (their flags are one
// 32-bit load), one block-wide scan.  Runs always; when the batch does have new keys, assign_kernel
// rewrites first_j with the new-key marks.
__global__ void __launch_bounds__(IB / 4) assign_firsts_kernel(int nnz, const uint8_t* __restrict__ flags,
                                                               const uint32_t* __restrict__ blk_cnt,
                                                               uint32_t* __restrict__ first_j) {
  __shared__ uint32_t wsum[IB / 128];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int j0 = blockIdx.x * IB + threadIdx.x * 4;
  uint32_t w = 0;
  if (j0 + 3 < nnz) w = *reinterpret_cast<const uint32_t*>(flags + j0);
  else for (int q = 0; q < 4; ++q) if (j0 + q < nnz) w |= (uint32_t)flags[j0 + q] << (8 * q);
  w &= 0x01010101u;                                           // bit 0 of each flag: first occurrence of its key
  const uint32_t cnt = __popc(w);
  uint32_t incl = cnt;
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    const uint32_t v = __shfl_up_sync(0xFFFFFFFFu, incl, d);
    if (lane >= d) incl += v;
  }
  if (lane == 31) wsum[warp] = incl;
  __syncthreads();
  uint32_t before = 0;
  for (int i = 0; i < warp; ++i) before += wsum[i];
  uint32_t u = blk_cnt[blockIdx.x] + before + incl - cnt;
#pragma unroll
  for (int q = 0; q < 4; ++q)
    if ((w >> (8 * q)) & 1u) first_j[u++] = (uint32_t)(j0 + q);
}

// New keys only: first_j[u] gets bit 31 and uniq_rows[u] the key's shard-local row (rank among the
// shard's new keys on top of the shard's size).  The random slot
// accesses are left to apply_first_kernel, which runs one thread per unique key.
__global__ void __launch_bounds__(IB) assign_kernel(
    int nnz, int nblk, int S, DevMeta* meta, const uint8_t* __restrict__ shards, const uint8_t* __restrict__ flags,
    const uint32_t* __restrict__ blk_cnt, int nblk_max, uint32_t* __restrict__ first_j,
    uint32_t* __restrict__ uniq_rows, Slot* slots, unsigned long long total_slots, uint32_t max_nnz) {
  __shared__ uint32_t wfirst[32];
  __shared__ uint16_t wnew[32][DES_MAX_SHARDS];
  // The slots' scratch range ends with this call (see Slot::first_occ; finish_kernel then starts a new one):
  // nothing reads the scratch words after flag_count_kernel, so this kernel — a few blocks that are idle
  // in the steady state — clears them all, once every few billion occurrences.
  if (meta->scratch_base - (uint32_t)nnz < max_nnz)
    for (unsigned long long i = (unsigned long long)blockIdx.x * blockDim.x + threadIdx.x; i < total_slots;
         i += (unsigned long long)gridDim.x * blockDim.x)
      slots[i].first_occ = DES_ROW_NONE;
  // steady state of a populated table: no new key in the whole batch (settled by scan_blocks_kernel, which
  // ran before this kernel), and assign_firsts_kernel has done all there is to do
  if (meta->any_new == 0u) return;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const unsigned lt = (1u << lane) - 1u;
  for (int tile = blockIdx.x; tile < nblk; tile += gridDim.x) {   // a few resident blocks walk the tiles
    const int j = tile * IB + threadIdx.x;
    const uint8_t fl = (j < nnz) ? flags[j] : 0;
    const uint32_t s = (j < nnz) ? shards[j] : 0;
    for (int i = threadIdx.x; i < 32 * DES_MAX_SHARDS; i += IB) (&wnew[0][0])[i] = 0;
    __syncthreads();
    // rank among firsts / among the shard's new keys inside the warp (lane order = CSR order)
    const unsigned fmask = __ballot_sync(0xFFFFFFFFu, fl & 1);
    const uint32_t frank = __popc(fmask & lt);
    const unsigned nmask_all = __ballot_sync(0xFFFFFFFFu, fl & 2);
    uint32_t nrank = 0;
    if (fl & 2) {
      unsigned same = __match_any_sync(nmask_all, s);
      nrank = __popc(same & lt);
      if ((same >> lane) == 1u) wnew[warp][s] = (uint16_t)__popc(same);   // highest lane of the group
    }
    if (lane == 0) wfirst[warp] = __popc(fmask);
    __syncthreads();
    // exclusive prefix over warps
    if (threadIdx.x < 32) {
      uint32_t v = wfirst[threadIdx.x], in = v;
#pragma unroll
      for (int d = 1; d < 32; d <<= 1) {
        uint32_t o = __shfl_up_sync(0xFFFFFFFFu, in, d);
        if (threadIdx.x >= d) in += o;
      }
      wfirst[threadIdx.x] = in - v;
    } else if (threadIdx.x >= 64 && threadIdx.x < 64 + S) {
      const int sh = threadIdx.x - 64;
      uint32_t run = 0;
      for (int w = 0; w < 32; ++w) { uint16_t v = wnew[w][sh]; wnew[w][sh] = (uint16_t)run; run += v; }
    }
    __syncthreads();
    if (fl & 2) {                                     // (first_j of the other firsts is already in place)
      const uint32_t u = blk_cnt[tile] + wfirst[warp] + frank;
      uint32_t local = meta->n_rows[s] + blk_cnt[(size_t)(1 + s) * nblk_max + tile] + wnew[warp][s] + nrank;
      if (local >= meta->row_cap[s]) { local = DES_ROW_NONE; des_raise(meta, DES_ERR_CAPACITY); }
      uniq_rows[u] = local;
      first_j[u] = (uint32_t)j | 0x80000000u;
    }
    __syncthreads();                                  // the shared tables are reused by the next tile
  }
}

// One thread per unique key of the batch: a new key's row number goes into its slot (the only slot
// access) and into rows[] at its first occurrence; the first occurrence also takes the key's batch-unique
// index (resolve_kernel hands both on to the key's other occurrences); uniq_rows gets the table-global row.
__global__ void __launch_bounds__(256) apply_first_kernel(
    Slot* slots, const DevMeta* __restrict__ meta, const uint32_t* __restrict__ slot_of,
    const uint8_t* __restrict__ shards, const uint32_t* __restrict__ first_j, uint32_t* __restrict__ rows,
    uint32_t* __restrict__ uidx, uint32_t* __restrict__ uniq_rows) {
  const uint32_t U = meta->n_uniq;
  for (uint32_t u = blockIdx.x * blockDim.x + threadIdx.x; u < U; u += gridDim.x * blockDim.x) {
    const uint32_t fj = first_j[u];
    const bool is_new = fj >> 31;
    const uint32_t j = fj & 0x7FFFFFFFu;
    if (!DES_DBG_OCC_OK(j)) continue;                  // (checking build)
    const uint32_t s = shards[j];
    uint32_t local;
    if (is_new) {
      local = uniq_rows[u];                            // DES_ROW_NONE: the shard is full
      if (local != DES_ROW_NONE && DES_DBG_SLOT_OK(slot_of[j])) slots[slot_of[j]].row = local;
      rows[j] = local;
    } else {
      local = rows[j];
    }
    uidx[j] = (local == DES_ROW_NONE) ? DES_ROW_NONE : u;
    const unsigned long long g = meta->row_base[s] + local;
    uniq_rows[u] = (local == DES_ROW_NONE) ? DES_ROW_NONE : (uint32_t)g;
  }
}

// Rows of the batch's new keys: weights from the counter-based generator keyed on the id, optimizer state
// at its start value.  G lanes per unique key (one 16-byte column each); keys that are not new cost one
// load.  uniq_rows[u] already holds the table-global row (apply_first_kernel).
template <int G>
__global__ void __launch_bounds__(256) init_new_rows_kernel(
    const unsigned long long* __restrict__ ids, int k, int stride, const DevMeta* __restrict__ meta,
    const uint32_t* __restrict__ first_j, const uint32_t* __restrict__ uniq_rows, float* __restrict__ W,
    float* __restrict__ A, float* __restrict__ A2, unsigned long long seed, float init_scale, float state_init,
    float lin_state_init) {
  if (meta->any_new == 0u) return;                     // steady state of a populated table: nothing to initialise
  const uint32_t U = meta->n_uniq;
  const int K4 = k >> 2, c4 = threadIdx.x % G;
  const long long gstep = (long long)gridDim.x * (256 / G);
  // every lane of a warp runs the same number of rounds (the squared norm is a warp-level sum)
  const long long rounds = ((long long)U + gstep - 1) / gstep;
  long long u = (long long)blockIdx.x * (256 / G) + threadIdx.x / G;
  for (long long r = 0; r < rounds; ++r, u += gstep) {
    uint32_t fj = 0, grow = DES_ROW_NONE;
    if (u < U) { fj = first_j[u]; if (fj >> 31) grow = uniq_rows[u]; }
    const bool init = grow != DES_ROW_NONE;
    float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
    if (init && c4 < K4) v = des_init4(seed, ids[fj & 0x7FFFFFFFu], (uint32_t)c4, init_scale);
    float n2 = v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
#pragma unroll
    for (int d = 1; d < G; d <<= 1) n2 += __shfl_xor_sync(0xFFFFFFFFu, n2, d);
    if (!init || DES_DBG_ROW(grow) != grow) continue;
    float4* w = reinterpret_cast<float4*>(W + (size_t)grow * stride);
    if (c4 < K4) w[c4] = v;
    // linear weight, squared norm of the latent vector, age stamp (the clock value this call ends with)
    if (c4 == 0) w[K4] = make_float4(0.f, n2, des_stamp_bits(meta->clock + 1ull), 0.f);
    if (A) {
      float4* a = reinterpret_cast<float4*>(A + (size_t)grow * stride);
      if (c4 < K4) a[c4] = make_float4(state_init, state_init, state_init, state_init);
      if (c4 == 0) a[K4] = make_float4(lin_state_init, 0.f, 0.f, 0.f);
    }
    if (A2) {
      float4* a2 = reinterpret_cast<float4*>(A2 + (size_t)grow * stride);
      if (c4 < K4) a2[c4] = make_float4(0.f, 0.f, 0.f, 0.f);
      if (c4 == 0) a2[K4] = make_float4(0.f, 0.f, 0.f, 0.f);
    }
  }
}

// Every occurrence that is not its key's first one takes the unique index — and, for a key that was new,
// the row — from the first one (a look-up in the batch's own arrays, not in the table).  IB occurrences per
// block, IB / 4 threads: a thread's four look-ups are in flight together.  First occurrences are only read
// here (apply_first_kernel wrote them), the others only written.
__global__ void __launch_bounds__(IB / 4) resolve_kernel(int nnz, const uint32_t* __restrict__ first_of,
                                                         uint32_t* rows, uint32_t* uidx, DevMeta* meta) {
  const int j0 = blockIdx.x * IB + threadIdx.x;
  uint32_t f[4], r[4], u[4];
  bool newrow[4];                                      // the occurrence's row comes from the first occurrence
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    const int j = j0 + q * (IB / 4);
    f[q] = DES_ROW_NONE; r[q] = DES_ROW_NONE; newrow[q] = false;
    if (j < nnz) { f[q] = first_of[j]; r[q] = rows[j]; }
    // (a first-occurrence index is an index into this batch; anything else would be a broken scratch word)
    if (f[q] != DES_ROW_NONE && f[q] >= (uint32_t)nnz) {
      f[q] = DES_ROW_NONE; r[q] = DES_ROW_NONE; newrow[q] = true; des_raise(meta, DES_ERR_CUDA);
    }
  }
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    const int j = j0 + q * (IB / 4);
    u[q] = DES_ROW_NONE;
    if (f[q] != DES_ROW_NONE && f[q] != (uint32_t)j) {
      u[q] = uidx[f[q]];
      if (r[q] == DES_ROW_NONE) { r[q] = rows[f[q]]; newrow[q] = true; }
    }
  }
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    const int j = j0 + q * (IB / 4);
    if (j >= nnz || f[q] == (uint32_t)j) continue;
    if (newrow[q]) rows[j] = r[q];                     // (every other row is in place since flag_count_kernel)
    uidx[j] = u[q];
  }
}

// One block: shard sizes advance, the call's scratch range is retired.
__global__ void __launch_bounds__(DES_MAX_SHARDS) finish_kernel(int S, int nnz, uint32_t max_nnz, DevMeta* meta,
                                                                uint32_t* n_uniq_out) {
  if ((int)threadIdx.x < S) {
    uint32_t n = meta->n_rows[threadIdx.x] + meta->new_total[threadIdx.x];
    meta->n_rows[threadIdx.x] = min(n, meta->row_cap[threadIdx.x]);
  }
  if (threadIdx.x == 0) {
    *n_uniq_out = meta->n_uniq;
    meta->any_new = 0u;
    meta->clock += 1ull;
    const uint32_t base = meta->scratch_base - (uint32_t)nnz;
    // the next call may need up to max_nnz below the base; if that is not left, assign_kernel has
    // cleared every slot's scratch word in this call and the range starts again at the top
    meta->scratch_base = base < max_nnz ? 0xFFFFFFFFu : base;
  }
}

extern "C" des_status_t des_find_or_insert(des_table_t* t, const des_batch_t* b, int insert, void* stream) {
  des_status_t st = des_check_batch(t, b, insert);
  if (st != DES_OK) return st;
  cudaStream_t cs = (cudaStream_t)stream;
  des_api_begin(t, cs);
  DES_DBG_ARM(t, cs);
  t->tag_valid = 0;                                    // dest[] is scratch of this call: the backward rebuilds its tags
  const int nnz = (int)b->nnz;
  const int nbags = b->batch * (int)t->F;
  if (nnz == 0) {
    if (insert) DES_CUDA(cudaMemsetAsync(b->n_uniq, 0, 4, cs));
    return DES_OK;
  }
  const int nblk = (nnz + IB - 1) / IB;
  SlotGeom geom;
  for (uint32_t s = 0; s <= t->S; ++s) geom.slot_base[s] = t->h_slot_base[s];
  des_mod_consts(t->S, &geom.mod_M, &geom.mod_two32);
  probe_claim_kernel<<<(nnz + 256 * PROBE_ILP - 1) / (256 * PROBE_ILP), 256, 0, cs>>>((const unsigned long long*)b->ids, b->offsets, nnz, nbags, t->S, t->F,
                                          t->cfg.partition, insert, t->cfg.shard_world, t->cfg.shard_rank, t->slots, t->meta, geom,
                                          t->slot_of, b->shards, b->rows);
  DES_LAUNCH_CHECK(t, "probe_claim_kernel");
  if (!insert) return DES_OK;
  uint32_t* first_of = t->uslot;
  flag_count_kernel<<<nblk, IB / 4, 0, cs>>>(nnz, t->S, t->slots, t->meta, t->slot_of, b->shards, t->flags, b->rows,
                                             first_of, t->blk_cnt, t->nblk_max);
  DES_LAUNCH_CHECK(t, "flag_count_kernel");
  scan_blocks_kernel<<<t->S + 1, 1024, 0, cs>>>(t->blk_cnt, nblk, t->nblk_max, t->meta);
  DES_LAUNCH_CHECK(t, "scan_blocks_kernel");
  assign_firsts_kernel<<<nblk, IB / 4, 0, cs>>>(nnz, t->flags, t->blk_cnt, t->dest);
  DES_LAUNCH_CHECK(t, "assign_firsts_kernel");
  assign_kernel<<<nblk < t->sm_count * 2 ? nblk : t->sm_count * 2, IB, 0, cs>>>(nnz, nblk, t->S, t->meta, b->shards, t->flags,
                                                                                t->blk_cnt, t->nblk_max, t->dest, b->uniq_rows,
                                                                                t->slots, t->total_slots, (uint32_t)t->max_nnz);
  DES_LAUNCH_CHECK(t, "assign_kernel");
  apply_first_kernel<<<t->sm_count * 8, 256, 0, cs>>>(t->slots, t->meta, t->slot_of, b->shards, t->dest, b->rows,
                                                      b->uidx, b->uniq_rows);
  DES_LAUNCH_CHECK(t, "apply_first_kernel");
  {
    const float state_init = t->cfg.optimizer == DES_OPT_ADAGRAD ? t->cfg.init_acc : 0.f;
    const float lin_state_init =
        (t->cfg.lin_optimizer == DES_LIN_FTRL || t->cfg.optimizer != DES_OPT_ADAGRAD) ? 0.f : t->cfg.init_acc;
    int G = 1;
    while (G < (int)t->k / 4) G <<= 1;
#define INIT(GG) init_new_rows_kernel<GG><<<t->sm_count * 8, 256, 0, cs>>>(                                            \
        (const unsigned long long*)b->ids, t->k, t->stride, t->meta, t->dest, b->uniq_rows, t->W, t->A, t->A2,         \
        t->cfg.seed, t->cfg.init_scale, state_init, lin_state_init)
    switch (G) { case 1: INIT(1); break; case 2: INIT(2); break; case 4: INIT(4); break; case 8: INIT(8); break; default: INIT(16); }
#undef INIT
    DES_LAUNCH_CHECK(t, "init_new_rows_kernel");
  }
  resolve_kernel<<<nblk, IB / 4, 0, cs>>>(nnz, first_of, b->rows, b->uidx, t->meta);
  DES_LAUNCH_CHECK(t, "resolve_kernel");
  finish_kernel<<<1, DES_MAX_SHARDS, 0, cs>>>(t->S, nnz, (uint32_t)t->max_nnz, t->meta, b->n_uniq);
  DES_LAUNCH_CHECK(t, "finish_kernel");
  return DES_OK;
}
