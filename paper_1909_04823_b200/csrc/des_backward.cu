// Backward of the DES sparse operators and the table update (Section 3.2,
// "Back-propagation Phase"; Section 5, `update`).
//
// The aggregation hands every shard the same upstream gradient, so each
// occurrence j of bag (b, f) contributes, to its own key only,
//   g_w(j) = x_j gL[b]
//   g_v(j) = x_j ( gF[b] (A[b] - v_j x_j) + gE[b][f] )
// Summed over a key's occurrences (v is the same row for all of them):
//   G_v = sum_j x_j c_bag(j)  -  v * sum_j x_j^2 gF[b_j],   c_bag = gF[b] A[b] + gE[b][f]
// so the kernel walks the batch in BAG order — c_bag is formed once per bag
// from rows that stream through exactly once — and scatter-adds x_j c_bag into
// the gradient row of the key's batch-unique index (dedup by the index that
// find_or_insert assigned).  A second kernel visits every unique key once:
// it finishes G_v with the key's own row, applies SGD / Adagrad to weights and
// state in place, and clears the gradient row for the next step.
//
// Hot keys.  CTR ids are Zipf distributed: a handful of keys own most of a
// batch's occurrences.  Millions of float atomics on one gradient row would
// serialise in L2 and, summed one after the other in fp32, lose the 1e-5
// accuracy the step must keep.  So before the scatter, occurrences are counted
// per unique key on a sample of the batch; a key whose estimated count reaches
// HOT_MIN gets R = count / CHAIN private replica rows, every occurrence is sent
// to replica hash(j) mod R, and after the scatter the replicas of a key are
// summed in double into its gradient row.  No accumulator ever takes more than
// a few hundred float additions, and no address is shared by more than that
// many atomics.
#include "des_internal.cuh"

#define HOT_MIN 512u      // estimated occurrences from which a key is treated as hot
#define HOT_CHAIN 256u    // target number of additions per replica row
#define SUPER_R 64u       // replica rows of a super key (they only take one partial sum per lane group)
#ifndef SC_BLOCKS_PER_SM
#define SC_BLOCKS_PER_SM 64     // grid cap of the scatter (it strides over the bags)
#endif

__device__ __forceinline__ uint32_t hash_u32(uint32_t x) {
  x ^= x >> 16; x *= 0x7FEB352Du; x ^= x >> 15; x *= 0x846CA68Bu; x ^= x >> 16;
  return x;
}

// hinfo[u] += 1 for a 1 / 2^shift sample of the occurrences.  A hot key would draw tens of
// thousands of atomics on one word, which L2 serialises; so counts are first merged per warp
// (lanes holding the same key), then per block in a small shared-memory table keyed by a hash of
// the key (a slot taken by another key sends the count straight to memory), and each block adds
// its table to hinfo once.
#define SC_THREADS 1024
#define SC_SLOTS 1024
#ifndef SC_PER
#define SC_PER 4
#endif
__global__ void __launch_bounds__(SC_THREADS) sample_count_kernel(const uint32_t* __restrict__ uidx, int nnz, int shift,
                                                                  long long max_uniq, uint32_t* hinfo) {
  __shared__ uint32_t s_key[SC_SLOTS], s_cnt[SC_SLOTS];
  for (int i = threadIdx.x; i < SC_SLOTS; i += SC_THREADS) { s_key[i] = DES_ROW_NONE; s_cnt[i] = 0u; }
  __syncthreads();
  // SC_PER samples per thread, their loads in flight together
  uint32_t u[SC_PER];
#pragma unroll
  for (int q = 0; q < SC_PER; ++q) {
    const long long i = ((long long)blockIdx.x * SC_PER + q) * SC_THREADS + threadIdx.x;
    const long long j = (i << shift) + (shift ? (hash_u32((uint32_t)i) & ((1u << shift) - 1u)) : 0u);
    u[q] = DES_ROW_NONE;
    if (j < nnz) u[q] = __ldg(uidx + j);
  }
#pragma unroll
  for (int q = 0; q < SC_PER; ++q) {
    const bool ok = u[q] != DES_ROW_NONE && (long long)u[q] < max_uniq;
    const unsigned act = __ballot_sync(0xFFFFFFFFu, ok);
    if (ok) {
      const unsigned same = __match_any_sync(act, u[q]);
      if ((threadIdx.x & 31) == __ffs(same) - 1) {
        const uint32_t c = (uint32_t)__popc(same), slot = hash_u32(u[q]) & (SC_SLOTS - 1);
        const uint32_t old = atomicCAS(&s_key[slot], DES_ROW_NONE, u[q]);
        if (old == DES_ROW_NONE || old == u[q]) atomicAdd(&s_cnt[slot], c);
        else atomicAdd(hinfo + u[q], c);
      }
    }
  }
  __syncthreads();
  for (int s = threadIdx.x; s < SC_SLOTS; s += SC_THREADS)
    if (s_cnt[s]) atomicAdd(hinfo + s_key[s], s_cnt[s]);
}

// Turns the sampled counts into the hot list: hinfo[u] becomes the key's hot
// index, or DES_ROW_NONE for a cold key.  ctr[0] = hot keys, ctr[1] = replica rows.
__global__ void __launch_bounds__(256) hot_select_kernel(uint32_t* hinfo, const uint32_t* __restrict__ n_uniq,
                                                         long long max_uniq, int shift, uint32_t* hot_base,
                                                         uint32_t* hot_R, uint32_t* hot_u, uint32_t* ctr,
                                                         uint32_t h_max, uint32_t rep_max, DevMeta* meta,
                                                         uint32_t* hot_work, uint32_t work_max, uint32_t super_min) {
  long long U = *n_uniq;
  if (U > max_uniq) U = max_uniq;   // more unique keys than the gradient buffer holds: the backward reports it
  for (long long u = (long long)blockIdx.x * blockDim.x + threadIdx.x; u < U; u += (long long)gridDim.x * blockDim.x) {
    const uint32_t est = hinfo[u] << shift;
    uint32_t h = DES_ROW_NONE;
    if (est >= HOT_MIN) {
      // the few keys that own a large share of the batch (super_min = 0: feature off) take one of
      // SUPER_T slots: ctr[3] = slots claimed, ctr[4 + slot] = hot index; hinfo carries slot + 1 in bits 24..
      bool sup = false;
      uint32_t ts = 0;
      if (super_min && est >= super_min) { ts = atomicAdd(&ctr[3], 1u); sup = ts < SUPER_T; }
      // (capped so that a key's chunk number fits the 18 bits of a work item; longer chains only cost accuracy)
      const uint32_t R = sup ? SUPER_R : min((est + HOT_CHAIN - 1) / HOT_CHAIN, 0x3FFFFu * HOT_RCHUNK);
      const uint32_t hh = atomicAdd(&ctr[0], 1u);
      if (hh < h_max) {
        const uint32_t base = atomicAdd(&ctr[1], R);
        const uint32_t nchunk = (R + HOT_RCHUNK - 1) / HOT_RCHUNK;
        bool ok = base + R <= rep_max;
        uint32_t wbase = 0;
        if (ok) { wbase = atomicAdd(&ctr[2], nchunk); ok = wbase + nchunk <= work_max; }
        if (ok) {
          hot_base[hh] = base; hot_R[hh] = R; hot_u[hh] = (uint32_t)u;
          h = hh | (sup ? (ts + 1u) << 24 : 0u);
          for (uint32_t i = 0; i < nchunk; ++i) hot_work[wbase + i] = (hh << 18) | i;
        } else {
          hot_R[hh] = 0;
        }
      }
      if (sup) ctr[HOT_CTR_SLOT + ts] = (h == DES_ROW_NONE) ? DES_ROW_NONE : (h & 0xFFFFFFu);
    }
    hinfo[u] = h;
  }
}

// dest[j] = gradient row of occurrence j: the key's own row, one of its replicas, or the tag of a
// register-summed key.  Four occurrences per thread: their look-up chains are in flight together.
__global__ void __launch_bounds__(256) make_dest_kernel(const uint32_t* __restrict__ uidx, int nnz,
                                                        const uint32_t* __restrict__ hinfo,
                                                        const uint32_t* __restrict__ hot_base,
                                                        const uint32_t* __restrict__ hot_R, long long max_uniq,
                                                        uint32_t* __restrict__ dest) {
  const int j0 = blockIdx.x * 1024 + threadIdx.x;
  uint32_t u[4], hv[4], d[4];
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    const int j = j0 + q * 256;
    u[q] = (j < nnz) ? __ldg(uidx + j) : DES_ROW_NONE;
    if (u[q] != DES_ROW_NONE && (long long)u[q] >= max_uniq) u[q] = DES_ROW_NONE;
  }
#pragma unroll
  for (int q = 0; q < 4; ++q) hv[q] = (u[q] != DES_ROW_NONE) ? __ldg(hinfo + u[q]) : DES_ROW_NONE;
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    const int j = j0 + q * 256;
    d[q] = u[q];                                          // cold key (or no row)
    if (u[q] != DES_ROW_NONE && hv[q] != DES_ROW_NONE) {
      if (hv[q] >> 24) d[q] = SUPER_TAG | ((hv[q] >> 24) - 1u);
      else   // replica floor(hash * R / 2^32): uniform over the R replicas without a division
        d[q] = (uint32_t)max_uniq + __ldg(hot_base + hv[q]) + __umulhi(hash_u32((uint32_t)j), __ldg(hot_R + hv[q]));
    }
  }
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    const int j = j0 + q * 256;
    if (j < nnz) dest[j] = d[q];
  }
}

// Replica reduction, stage 1: one warp per work item = HOT_RCHUNK replica rows
// of one hot key.  Columns are spread over the lanes, sums are taken in double
// and added (double atomics, a few hundred per key at most) to the key's row of
// hot_acc; the replica rows are cleared for the next step.
__global__ void __launch_bounds__(256) hot_reduce_kernel(const uint32_t* __restrict__ ctr, uint32_t work_max,
                                                         const uint32_t* __restrict__ hot_work,
                                                         const uint32_t* __restrict__ hot_base,
                                                         const uint32_t* __restrict__ hot_R, long long max_uniq,
                                                         int k, float* __restrict__ Gbuf, double* __restrict__ hot_acc) {
  const int stride = k + 4, lane = threadIdx.x & 31;
  uint32_t nw = ctr[2];
  if (nw > work_max) nw = work_max;
  const uint32_t wstep = gridDim.x * (blockDim.x >> 5);
  for (uint32_t wi = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5); wi < nw; wi += wstep) {
    const uint32_t item = hot_work[wi], h = item >> 18, chunk = item & 0x3FFFFu;
    const uint32_t R = hot_R[h];
    const uint32_t r_lo = chunk * HOT_RCHUNK, r_hi = min(R, r_lo + HOT_RCHUNK);
    float* rep = Gbuf + ((size_t)max_uniq + hot_base[h]) * stride;
    double a0 = 0.0, a1 = 0.0, a2 = 0.0;
    const bool c0 = lane < stride, c1 = lane + 32 < stride, c2 = lane + 64 < stride;
    uint32_t r = r_lo;
    for (; r + 4 <= r_hi; r += 4) {                    // four rows in flight
      float v0[4], v1[4], v2[4];
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const float* row = rep + (size_t)(r + q) * stride;
        v0[q] = c0 ? row[lane] : 0.f; v1[q] = c1 ? row[lane + 32] : 0.f; v2[q] = c2 ? row[lane + 64] : 0.f;
      }
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        float* row = rep + (size_t)(r + q) * stride;
        a0 += (double)v0[q]; a1 += (double)v1[q]; a2 += (double)v2[q];
        if (c0) row[lane] = 0.f;
        if (c1) row[lane + 32] = 0.f;
        if (c2) row[lane + 64] = 0.f;
      }
    }
    for (; r < r_hi; ++r) {
      float* row = rep + (size_t)r * stride;
      if (c0) { a0 += (double)row[lane]; row[lane] = 0.f; }
      if (c1) { a1 += (double)row[lane + 32]; row[lane + 32] = 0.f; }
      if (c2) { a2 += (double)row[lane + 64]; row[lane + 64] = 0.f; }
    }
    double* dst = hot_acc + (size_t)h * stride;
    if (lane < stride) atomicAdd(dst + lane, a0);
    if (lane + 32 < stride) atomicAdd(dst + lane + 32, a1);
    if (lane + 64 < stride) atomicAdd(dst + lane + 64, a2);
  }
}

// Stage 2: the double sums go into the hot keys' gradient rows; hot_acc is cleared.
__global__ void __launch_bounds__(256) hot_finish_kernel(const uint32_t* __restrict__ ctr, uint32_t h_max,
                                                         const uint32_t* __restrict__ hot_R,
                                                         const uint32_t* __restrict__ hot_u, int k,
                                                         float* __restrict__ Gbuf, double* __restrict__ hot_acc) {
  const int stride = k + 4;
  uint32_t nh = ctr[0];
  if (nh > h_max) nh = h_max;
  const long long n = (long long)nh * stride;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x) {
    const uint32_t h = (uint32_t)(i / stride), c = (uint32_t)(i % stride);
    if (hot_R[h] == 0) continue;
    Gbuf[(size_t)hot_u[h] * stride + c] += (float)hot_acc[i];
    hot_acc[i] = 0.0;
  }
}

// U occurrences i, i + P, ... of a bag: one vector atomic per lane into the occurrence's gradient
// row (lane 0 of the sub-group also adds the linear-weight tail).  SUPER: occurrences marked
// dest = SUPER_TAG | slot send nothing; lane t counts those of slot t.
template <int U, int P, bool HAS_VALS, bool SUPER>
__device__ __forceinline__ void scatter_step(const uint32_t* __restrict__ dest, const float* __restrict__ vals, int i,
                                             char* gcol, char* gtail, unsigned rowB, bool col, bool lead,
                                             const float4& c, float gl, float gf, uint32_t mine, uint32_t& cnt) {
  uint32_t d[U]; float x[U];
#pragma unroll
  for (int u = 0; u < U; ++u) {
    d[u] = __ldg(dest + i + u * P);
    if (HAS_VALS) x[u] = __ldg(vals + i + u * P);
  }
#pragma unroll
  for (int u = 0; u < U; ++u) {
    if (SUPER) cnt += (d[u] == mine);
    bool ok = SUPER ? d[u] < SUPER_TAG : d[u] != DES_ROW_NONE;   // SUPER_TAG.. also covers "no row"
    if (ok && !DES_DBG_GRAD_OK(d[u])) ok = false;                     // (checking build)
    if (ok) {
      const size_t off = (size_t)d[u] * rowB;
      if (HAS_VALS) {
        const float xx = x[u];
        if (col) atomicAdd(reinterpret_cast<float4*>(gcol + off), make_float4(xx * c.x, xx * c.y, xx * c.z, xx * c.w));
        if (lead) atomicAdd(reinterpret_cast<float4*>(gtail + off), make_float4(xx * gl, xx * xx * gf, 0.f, 0.f));
      } else {
        if (col) atomicAdd(reinterpret_cast<float4*>(gcol + off), c);
        if (lead) atomicAdd(reinterpret_cast<float4*>(gtail + off), make_float4(gl, gf, 0.f, 0.f));
      }
    }
  }
}

// One bag per G * P lanes: P sub-groups of G lanes (one 16-byte column each) take alternate
// occurrences of the bag.  c_bag is formed once per bag; the loop body is the destination load
// and the atomics.  SUPER (G = 16 only): occurrences of the few keys that own a large share of a
// skewed batch send no atomics; lane t counts the bag's occurrences of slot t and the counts go
// to super_cnt[bag][16]; super_dense_kernel turns them into the keys' gradient sums.
template <int G, int P, bool HAS_VALS, bool SUPER>
__global__ void __launch_bounds__(256) grad_scatter_kernel(
    const int32_t* __restrict__ offsets, const float* __restrict__ vals, const uint32_t* __restrict__ dest,
    long long nbags, int F, int k, uint32_t ops, const float* __restrict__ out_small,
    const float* __restrict__ gL, const float* __restrict__ gF, const float* __restrict__ gE, float* Gbuf,
    float* __restrict__ super_cnt) {
  constexpr int LB = G * P;
  const int K4 = k >> 2, stride = k + 4;
  const int sub = threadIdx.x % LB, c4 = sub % G, p = sub / G;
  const bool col = c4 < K4, lead = c4 == 0;
  const unsigned rowB = (unsigned)stride * 4u;
  char* gcol = reinterpret_cast<char*>(Gbuf) + c4 * 16;
  char* gtail = reinterpret_cast<char*>(Gbuf + k);
  const uint32_t mine = SUPER_TAG | (uint32_t)c4;
  // grid-stride over bags (every lane of a warp runs the same number of rounds); the next bag's bounds are
  // fetched while the current bag is scattered, so only the destination loads wait on them
  const long long slots = (long long)gridDim.x * (256 / LB);
  const long long rounds = (nbags + slots - 1) / slots;
  long long bag = (long long)blockIdx.x * (256 / LB) + threadIdx.x / LB;
  int lo_n = 0, hi_n = 0;
  if (bag < nbags) { lo_n = __ldg(offsets + bag); hi_n = __ldg(offsets + bag + 1); }
  for (long long r = 0; r < rounds; ++r, bag += slots) {
    const bool live = bag < nbags;
    const int lo = lo_n, hi = hi_n;
    lo_n = 0; hi_n = 0;
    if (bag + slots < nbags) { lo_n = __ldg(offsets + bag + slots); hi_n = __ldg(offsets + bag + slots + 1); }
    float4 c = make_float4(0.f, 0.f, 0.f, 0.f);
    float gf = 0.f, gl = 0.f;
    if (lo < hi) {
      const long long b = (long long)((unsigned)bag / (unsigned)F);   // bags < 2^31: no 64-bit division
      if (ops & DES_OP_FM) gf = __ldg(gF + b);
      if (ops & DES_OP_LR) gl = __ldg(gL + b);
      if (col) {
        if (ops & DES_OP_FM) {
          const float4 a = __ldg(reinterpret_cast<const float4*>(out_small + b * stride) + c4);
          c = make_float4(gf * a.x, gf * a.y, gf * a.z, gf * a.w);
        }
        if (gE) {
          const float4 e = __ldg(reinterpret_cast<const float4*>(gE + bag * k) + c4);
          c.x += e.x; c.y += e.y; c.z += e.z; c.w += e.w;
        }
      }
    }
    uint32_t cnt = 0;
    int i0 = lo;
#define SC_STEP(U) scatter_step<U, P, HAS_VALS, SUPER>(dest, vals, i0 + p, gcol, gtail, rowB, col, lead, c, gl, gf, mine, cnt)
    for (; i0 + 4 * P <= hi; i0 += 4 * P) SC_STEP(4);
    if (i0 + 2 * P <= hi) { SC_STEP(2); i0 += 2 * P; }
    if (i0 + P <= hi) { SC_STEP(1); i0 += P; }
    if (i0 + p < hi) SC_STEP(1);
#undef SC_STEP
    if (SUPER) {
#pragma unroll
      for (int d = G; d < LB; d <<= 1) cnt += __shfl_xor_sync(0xFFFFFFFFu, cnt, d);
      if (live && p == 0) super_cnt[bag * 16 + c4] = (float)cnt;
    }
  }
}

// Gradient sums of the SUPER_T marked keys as a dense product:
//   G_t = sum over bags of count[bag][t] * c_bag,   tail_t = sum of count * (gL[b], gF[b]),
// with c_bag rebuilt from gE and the aggregated forward exactly as in the scatter.  A CTA
// stages SD_TILE bags (c_bag rows, counts, gL / gF) in shared memory; thread (t, c4) owns the
// accumulator of key t, 16-byte column c4.  Each CTA adds its sums to one replica row per key
// (summed in double by hot_reduce).  All feature values are 1 on this path.
#define SD_TILE 32
#define SD_STAGES 4
#define SD_THREADS 288   // 256 column threads + one warp for the linear-weight tails

__device__ __forceinline__ void sd_cp_async16(void* smem, const void* gmem) {
  const unsigned sa = (unsigned)__cvta_generic_to_shared(smem);
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(sa), "l"(gmem));
}
__device__ __forceinline__ void sd_cp_async4(void* smem, const void* gmem) {
  const unsigned sa = (unsigned)__cvta_generic_to_shared(smem);
  asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(sa), "l"(gmem));
}
__device__ __forceinline__ void sd_cp_commit() { asm volatile("cp.async.commit_group;"); }
template <int N>
__device__ __forceinline__ void sd_cp_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N)); }

// The kernel is one stream over gE.  Per tile of SD_TILE bags a ring of SD_STAGES shared-memory stages takes,
// by asynchronous copies, the bags' rows of gE, their samples' rows of A and (gL, gF), and the counts; thread
// (c4, kg, sub) multiplies column c4 of c_bag = gE row + gF A by the counts of keys 8 kg .. 8 kg + 7 for
// bags sub, sub + 8, ... of the tile; the extra warp sums the linear-weight tails.  One barrier per tile:
// behind it every thread has finished the previous tile, whose stage the next copies overwrite.
__global__ void __launch_bounds__(SD_THREADS) super_dense_kernel(
    const float* __restrict__ super_cnt, int nbags, int F, int k, uint32_t ops,
    const float* __restrict__ out_small, const float* __restrict__ gL, const float* __restrict__ gF,
    const float* __restrict__ gE, float* Gbuf, const uint32_t* __restrict__ ctr,
    const uint32_t* __restrict__ hot_base, const uint32_t* __restrict__ hot_R, long long max_uniq) {
  uint32_t ns = __ldg(ctr + 3);
  if (ns == 0) return;
  if (ns > SUPER_T) ns = SUPER_T;
  extern __shared__ __align__(16) unsigned char sd_smem[];
  typedef float4 (*tile_t)[SD_TILE][16];
  tile_t s_c = reinterpret_cast<tile_t>(sd_smem);                                      // gE rows
  tile_t s_a = s_c + SD_STAGES;                                                        // A rows
  float (*s_n)[SD_TILE][16] = reinterpret_cast<float (*)[SD_TILE][16]>(s_a + SD_STAGES);   // counts
  float2 (*s_g)[SD_TILE] = reinterpret_cast<float2 (*)[SD_TILE]>(s_n + SD_STAGES);     // (gL, gF) per bag
  const int K4 = k >> 2, stride = k + 4;
  const int tid = threadIdx.x;
  const bool tailw = tid >= 256;                       // the extra warp
  const int c4 = tid & 15, tk = (tid >> 4) & 15;       // copy role: column c4 of bags tk and tk + 16 of a tile
  const int kg = (tid >> 4) & 1, sub = (tid >> 5) & 7; // multiply role
  const int tt = tid & 15, th = (tid >> 4) & 1;        // tail role: key tt, bags th, th + 2, ...
  const bool col = c4 < K4, fm = ops & DES_OP_FM, lr = ops & DES_OP_LR;
  const float4 zero = make_float4(0.f, 0.f, 0.f, 0.f);
  float4 acc[8] = {zero, zero, zero, zero, zero, zero, zero, zero};
  float tw = 0.f, tq = 0.f;
  const int tstep = gridDim.x * SD_TILE;
  const int base0 = blockIdx.x * SD_TILE;
  // one group of asynchronous copies per tile and thread (an empty one past the end)
  auto issue = [&](int base, int stage) {
    if (base < nbags) {
      if (!tailw) {
#pragma unroll
        for (int r = 0; r < 2; ++r) {
          const int i = r * 16 + tk, bag = base + i;
          const bool in = bag < nbags && col;
          if (in && gE) sd_cp_async16(&s_c[stage][i][c4], gE + (size_t)bag * k + c4 * 4);
          else s_c[stage][i][c4] = zero;
          if (in && fm) sd_cp_async16(&s_a[stage][i][c4], out_small + (size_t)(bag / F) * stride + c4 * 4);
          else s_a[stage][i][c4] = zero;
        }
        if (tid < 128) {                               // 32 bags x 16 counts: 128 copies of 16 bytes
          const int i = tid >> 2, q = tid & 3, bag = base + i;
          if (bag < nbags) sd_cp_async16(&s_n[stage][i][q * 4], super_cnt + (size_t)bag * 16 + q * 4);
          else *reinterpret_cast<float4*>(&s_n[stage][i][q * 4]) = zero;
        }
      } else {
        const int i = tid - 256, bag = base + i;
        const int b = bag / F;                         // (a plain store and a copy never target the same word)
        if (bag < nbags && lr) sd_cp_async4(&s_g[stage][i].x, gL + b); else s_g[stage][i].x = 0.f;
        if (bag < nbags && fm) sd_cp_async4(&s_g[stage][i].y, gF + b); else s_g[stage][i].y = 0.f;
      }
    }
    sd_cp_commit();
  };
#pragma unroll
  for (int p = 0; p < SD_STAGES - 1; ++p) issue(base0 + p * tstep, p);
  int it = 0;
  for (int base = base0; base < nbags; base += tstep, ++it) {
    const int stage = it % SD_STAGES;
    sd_cp_wait<SD_STAGES - 2>();                       // this thread's copies of the tile have landed
    __syncthreads();                                   // ... and everybody's; the previous tile is consumed
    issue(base + (SD_STAGES - 1) * tstep, (it + SD_STAGES - 1) % SD_STAGES);
    if (tailw) {
#pragma unroll 4
      for (int i = th; i < SD_TILE; i += 2) {
        const float f = s_n[stage][i][tt];
        const float2 gg = s_g[stage][i];
        tw = fmaf(f, gg.x, tw);
        tq = fmaf(f, gg.y, tq);
      }
    } else {
#pragma unroll
      for (int i = sub; i < SD_TILE; i += 8) {
        const float4 f0 = *reinterpret_cast<const float4*>(&s_n[stage][i][kg * 8]);
        const float4 f1 = *reinterpret_cast<const float4*>(&s_n[stage][i][kg * 8 + 4]);
        float4 c = s_c[stage][i][c4];
        if (fm) {
          const float4 a = s_a[stage][i][c4];
          const float gf = s_g[stage][i].y;
          c.x = fmaf(gf, a.x, c.x); c.y = fmaf(gf, a.y, c.y); c.z = fmaf(gf, a.z, c.z); c.w = fmaf(gf, a.w, c.w);
        }
#define SD_FMA(q, f) acc[q].x = fmaf(f, c.x, acc[q].x); acc[q].y = fmaf(f, c.y, acc[q].y); \
                     acc[q].z = fmaf(f, c.z, acc[q].z); acc[q].w = fmaf(f, c.w, acc[q].w)
        SD_FMA(0, f0.x); SD_FMA(1, f0.y); SD_FMA(2, f0.z); SD_FMA(3, f0.w);
        SD_FMA(4, f1.x); SD_FMA(5, f1.y); SD_FMA(6, f1.z); SD_FMA(7, f1.w);
#undef SD_FMA
      }
    }
  }
  sd_cp_wait<0>();
  // each (CTA, bag subset) hands its sums to one replica row per key
  const uint32_t salt = hash_u32(blockIdx.x * 8u + (uint32_t)(tailw ? th : sub));
  if (tailw) {
    if ((uint32_t)tt >= ns) return;
    const uint32_t hh = __ldg(ctr + HOT_CTR_SLOT + tt);
    if (hh == DES_ROW_NONE) return;
    const uint32_t R = __ldg(hot_R + hh);
    if (R == 0) return;
    float* row = Gbuf + ((size_t)max_uniq + __ldg(hot_base + hh) + salt % R) * stride;
    atomicAdd(reinterpret_cast<float4*>(row) + K4, make_float4(tw, tq, 0.f, 0.f));
    return;
  }
#pragma unroll
  for (int q = 0; q < 8; ++q) {
    const uint32_t key = (uint32_t)(kg * 8 + q);
    if (key >= ns || !col) continue;
    const uint32_t hh = __ldg(ctr + HOT_CTR_SLOT + key);
    if (hh == DES_ROW_NONE) continue;
    const uint32_t R = __ldg(hot_R + hh);
    if (R == 0) continue;
    float* row = Gbuf + ((size_t)max_uniq + __ldg(hot_base + hh) + salt % R) * stride;
    atomicAdd(reinterpret_cast<float4*>(row) + c4, acc[q]);
  }
}

#ifndef UP_MINB
#define UP_MINB 2
#endif
#ifndef UP_UNROLL
#define UP_UNROLL 4
#endif

// Advances Adam's step count and recomputes the bias corrections 1 - beta^t in double.
__global__ void adam_tick_kernel(DevMeta* meta, float beta1, float beta2) {
  const unsigned long long t = meta->opt_step + 1;
  meta->opt_step = t;
  meta->adam_c1 = (float)(1.0 - pow((double)beta1, (double)t));
  meta->adam_c2 = (float)(1.0 - pow((double)beta2, (double)t));
}

// One optimizer application per unique key.  A group of G lanes owns a key (one
// 16-byte column each, lane 0 also the linear weight); it works on UP_UNROLL
// keys at a time so that their gradient rows, row numbers, weights and state
// are all in flight together: the kernel is a pure stream of 272-byte rows.
template <int G, bool ADAM>
__global__ void __launch_bounds__(256, UP_MINB) update_rows_kernel(
    const uint32_t* __restrict__ uniq_rows, const uint32_t* __restrict__ n_uniq, long long max_uniq, int k,
    uint32_t ops, const OptParams opt_in, DevMeta* __restrict__ meta, float* __restrict__ Gbuf,
    float* __restrict__ W, float* __restrict__ A, float* __restrict__ A2) {
  const int K4 = k >> 2, stride = k + 4;
  const OptParams opt = des_opt_load(opt_in, meta);
  const float stamp = des_stamp_bits(meta->clock);     // "updated in the step of the current batch" (eviction by age)
  long long U = *n_uniq;
  if (U > max_uniq) {           // the gradient buffer cannot hold this batch: report, update what fits
    if (blockIdx.x == 0 && threadIdx.x == 0) des_raise(meta, DES_ERR_CAPACITY);
    U = max_uniq;
  }
  const int c4 = (int)(threadIdx.x % G);
  const bool col = c4 < K4, lead = c4 == 0;
  const bool upd_v = ops & (DES_OP_FM | DES_OP_POOL | DES_OP_DENSE1), upd_w = ops & DES_OP_LR;
  const long long gstep = (long long)gridDim.x * (blockDim.x / G);
  const float4 zero = make_float4(0.f, 0.f, 0.f, 0.f);
  // every lane of a warp runs the same number of iterations (keys past U are masked off)
  const long long iters = (U + gstep * UP_UNROLL - 1) / (gstep * UP_UNROLL);
  long long u0 = (long long)blockIdx.x * (blockDim.x / G) + threadIdx.x / G;
  for (long long it = 0; it < iters; ++it, u0 += gstep * UP_UNROLL) {
    uint32_t r[UP_UNROLL];
    float4 g[UP_UNROLL], v[UP_UNROLL], s[UP_UNROLL], s2[ADAM ? UP_UNROLL : 1];
    float2 tail[UP_UNROLL], st[UP_UNROLL];   // gradient tail (G_w, sum x^2 gF); linear weight's two state words
    float lw[UP_UNROLL];                      // linear weight (lead lane)
#pragma unroll
    for (int q = 0; q < UP_UNROLL; ++q) {
      const long long u = u0 + q * gstep;
      r[q] = (u < U) ? __ldg(uniq_rows + u) : DES_ROW_NONE;
      if (r[q] != DES_ROW_NONE && DES_DBG_ROW(r[q]) != r[q]) r[q] = DES_ROW_NONE;   // (checking build)
      g[q] = zero; tail[q] = make_float2(0.f, 0.f);
      if (u < U) {
        const float4* grow = reinterpret_cast<const float4*>(Gbuf + (size_t)u * stride);
        if (col) g[q] = grow[c4];
        tail[q] = *reinterpret_cast<const float2*>(grow + K4);
      }
    }
#pragma unroll
    for (int q = 0; q < UP_UNROLL; ++q) {
      v[q] = zero; s[q] = zero; lw[q] = 0.f; st[q] = make_float2(0.f, 0.f);
      if (ADAM) s2[ADAM ? q : 0] = zero;
      if (r[q] != DES_ROW_NONE) {
        const float4* w = reinterpret_cast<const float4*>(W + (size_t)r[q] * stride);
        const float4* a = A ? reinterpret_cast<const float4*>(A + (size_t)r[q] * stride) : nullptr;
        if (col) {
          v[q] = w[c4];
          if (a && upd_v) s[q] = a[c4];
          if (ADAM && upd_v) s2[ADAM ? q : 0] = reinterpret_cast<const float4*>(A2 + (size_t)r[q] * stride)[c4];
        }
        if (lead) {
          lw[q] = *reinterpret_cast<const float*>(w + K4);
          if (a && upd_w) st[q] = *reinterpret_cast<const float2*>(a + K4);
        }
      }
    }
    __syncwarp();   // all lanes of a group have read the gradient row before its lead lane clears it
#pragma unroll
    for (int q = 0; q < UP_UNROLL; ++q) {
      const long long u = u0 + q * gstep;
      const bool live = u < U, mapped = r[q] != DES_ROW_NONE;
      if (live) {
        float4* grow = reinterpret_cast<float4*>(Gbuf + (size_t)u * stride);
        if (col) grow[c4] = zero;
        if (lead) grow[K4] = zero;
      }
      float4& m2 = s2[ADAM ? q : 0];            // Adam's second moment (unused otherwise)
      if (mapped && col && upd_v) {
        const float t1 = tail[q].y;
        des_opt_step(opt, v[q].x, s[q].x, m2.x, g[q].x - v[q].x * t1);
        des_opt_step(opt, v[q].y, s[q].y, m2.y, g[q].y - v[q].y * t1);
        des_opt_step(opt, v[q].z, s[q].z, m2.z, g[q].z - v[q].z * t1);
        des_opt_step(opt, v[q].w, s[q].w, m2.w, g[q].w - v[q].w * t1);
      }
      // squared norm of the (new) latent vector, kept in the row's tail for the forward's M_2
      float n2 = v[q].x * v[q].x + v[q].y * v[q].y + v[q].z * v[q].z + v[q].w * v[q].w;
#pragma unroll
      for (int d = 1; d < G; d <<= 1) n2 += __shfl_xor_sync(0xFFFFFFFFu, n2, d);
      if (!mapped) continue;
      float4* w = reinterpret_cast<float4*>(W + (size_t)r[q] * stride);
      float4* a = A ? reinterpret_cast<float4*>(A + (size_t)r[q] * stride) : nullptr;
      if (col && upd_v) {
        w[c4] = v[q];
        if (a) a[c4] = s[q];
        if (ADAM) reinterpret_cast<float4*>(A2 + (size_t)r[q] * stride)[c4] = m2;
      }
      if (lead) {
        if (upd_w) {     // linear weight: its two state words sit side by side in the state row's tail
          if (opt.lin_optimizer == DES_LIN_FTRL) des_ftrl_step(opt, lw[q], st[q].x, st[q].y, tail[q].x);
          else des_opt_step(opt, lw[q], st[q].x, st[q].y, tail[q].x);
        }
        w[K4] = make_float4(lw[q], n2, stamp, 0.f);
        if (a && upd_w) a[K4] = make_float4(st[q].x, st[q].y, 0.f, 0.f);
      }
    }
  }
}

static int group_for(int k) { int K4 = k / 4, G = 1; while (G < K4) G <<= 1; return G; }

// Skewed-batch path: 16-lane groups, unit feature values, batches large enough to fill a persistent grid.
// The dense product of the backward costs time per BAG, the atomics it replaces per OCCURRENCE: it pays from
// about ten ids per bag on (measured: 20 ids per bag 1.50 -> 0.85 + 0.25 ms; 4 ids per bag 0.43 -> 0.39 + 0.29 ms).
static bool super_path(const des_table* t, const des_batch_t* b) {
  const long long nbags = (long long)b->batch * t->F;
  return group_for(t->k) == 16 && !b->vals && b->nnz >= (1 << 20) && t->super_cnt && b->nnz >= 8 * nbags;
}

des_status_t des_tags_ensure(des_table* t, const des_batch_t* b, cudaStream_t cs) {
  if (t->tag_valid && t->tag_uidx == (const void*)b->uidx && t->tag_nnz == (long long)b->nnz) return DES_OK;
  t->tag_valid = 0;
  if (b->nnz == 0) return DES_OK;
  const int nnz = (int)b->nnz;
  int shift = 0;
  while (shift < 6 && ((long long)nnz >> shift) > (1ll << 20)) ++shift;
  DES_CUDA(cudaMemsetAsync(t->hot_ctr, 0, HOT_CTR_WORDS * 4, cs));
  DES_CUDA(cudaMemsetAsync(t->hinfo, 0, (size_t)t->max_uniq * 4, cs));
  const bool use_super = super_path(t, b);
  const uint32_t super_min = use_super ? (uint32_t)(nnz >> 7) : 0u;
  const int n = (nnz >> shift) + 1;
  sample_count_kernel<<<(n + SC_THREADS * SC_PER - 1) / (SC_THREADS * SC_PER), SC_THREADS, 0, cs>>>(b->uidx, nnz, shift, t->max_uniq, t->hinfo);
  DES_LAUNCH_CHECK(t, "sample_count_kernel");
  hot_select_kernel<<<t->sm_count * 4, 256, 0, cs>>>(t->hinfo, b->n_uniq, t->max_uniq, shift, t->hot_base, t->hot_R,
                                                     t->hot_u, t->hot_ctr, t->hot_max, t->rep_max, t->meta,
                                                     t->hot_work, t->work_max, super_min);
  DES_LAUNCH_CHECK(t, "hot_select_kernel");
  make_dest_kernel<<<(nnz + 1023) / 1024, 256, 0, cs>>>(b->uidx, nnz, t->hinfo, t->hot_base, t->hot_R, t->max_uniq,
                                                      t->dest);
  DES_LAUNCH_CHECK(t, "make_dest_kernel");
  t->tag_uidx = b->uidx; t->tag_nnz = (long long)b->nnz; t->tag_super = use_super ? 1 : 0; t->tag_valid = 1;
  return DES_OK;
}

extern "C" des_status_t des_backward_update(des_table_t* t, uint32_t ops, const des_batch_t* b,
                                            const des_outputs_t* out, const des_grads_t* gr, void* stream) {
  des_status_t st = des_check_batch(t, b, 1);
  if (st != DES_OK) return st;
  if (!out || !gr || (ops & ~15u) || ops == 0) return DES_ERR_INVALID_ARG;
  if ((ops & DES_OP_LR) && !gr->gL) return DES_ERR_INVALID_ARG;
  if ((ops & DES_OP_FM) && (!gr->gF || !out->out_small)) return DES_ERR_INVALID_ARG;
  if ((ops & DES_OP_POOL) && !(ops & DES_OP_DENSE1) && !gr->gE) return DES_ERR_INVALID_ARG;
  if ((ops & DES_OP_DENSE1) && (!t->H || !gr->gZ || !gr->gE_work || !out->pooled)) return DES_ERR_INVALID_ARG;
  cudaStream_t cs = (cudaStream_t)stream;
  des_api_begin(t, cs);
  DES_DBG_ARM(t, cs);
  const int B = b->batch;
  const OptParams opt = des_opt_params(t);
  if (opt.optimizer == DES_OPT_ADAM) {               // one optimizer step per backward call (Adam's t)
    adam_tick_kernel<<<1, 1, 0, cs>>>(t->meta, opt.beta1, opt.beta2);
    DES_LAUNCH_CHECK(t, "adam_tick_kernel");
  }
  const float* gE = (ops & DES_OP_POOL) ? gr->gE : nullptr;
  if (ops & DES_OP_DENSE1) {
    st = des_dense1_backward(t, out->pooled, gE, gr->gZ, gr->gE_work, B, cs);
    if (st != DES_OK) return st;
    gE = gr->gE_work;
  }
  if (b->nnz == 0) return DES_OK;
  const int G = group_for(t->k);
  const int nnz = (int)b->nnz;
  const long long nbags = (long long)B * t->F;
  // hot-key detection on a sample, replica assignment, per-occurrence destination row (kept if this very batch
  // has been through it since its find_or_insert)
  if ((st = des_tags_ensure(t, b, cs)) != DES_OK) return st;
  const bool use_super = t->tag_super;
  {
    // long bags: a whole warp per bag (its sub-groups take alternate occurrences); short bags: G lanes per bag
    const bool wide = (long long)nnz >= 8 * nbags;   // (at 4 ids per bag the narrow form measured faster)
    const long long threads = nbags * (wide ? 32 : G);
    long long blocks = (threads + 255) / 256;
    if (blocks > (long long)t->sm_count * SC_BLOCKS_PER_SM) blocks = (long long)t->sm_count * SC_BLOCKS_PER_SM;
    const unsigned grid = (unsigned)blocks;
#define SC4(GG, PP, HV, SU) grad_scatter_kernel<GG, PP, HV, SU><<<grid, 256, 0, cs>>>(                                  \
        b->offsets, b->vals, t->dest, nbags, t->F, t->k, ops, out->out_small, gr->gL, gr->gF, gE, t->Gbuf, t->super_cnt)
#define SC3(GG, HV) do { if (wide) SC4(GG, 32 / GG, HV, false); else SC4(GG, 1, HV, false); } while (0)
#define SC(GG) do { if (b->vals) SC3(GG, true); else SC3(GG, false); } while (0)
    if (use_super) {
      if (wide) SC4(16, 2, false, true); else SC4(16, 1, false, true);
    } else {
      switch (G) { case 1: SC(1); break; case 2: SC(2); break; case 4: SC(4); break; case 8: SC(8); break; default: SC(16); }
    }
#undef SC
#undef SC3
#undef SC4
    DES_LAUNCH_CHECK(t, "grad_scatter_kernel");
  }
  if (use_super) {
    const int sd_smem = SD_STAGES * SD_TILE * (2 * 16 * (int)sizeof(float4) + 16 * (int)sizeof(float) + (int)sizeof(float2));
    // (an attribute of the function on the current device, not a stream operation: legal under capture)
    if (cudaFuncSetAttribute(super_dense_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, sd_smem) != cudaSuccess)
      return DES_ERR_CUDA;
    super_dense_kernel<<<t->sm_count * 3, SD_THREADS, sd_smem, cs>>>(t->super_cnt, (int)nbags, t->F, t->k, ops, out->out_small,
                                                               gr->gL, gr->gF, gE, t->Gbuf, t->hot_ctr, t->hot_base,
                                                               t->hot_R, t->max_uniq);
    DES_LAUNCH_CHECK(t, "super_dense_kernel");
  }
  hot_reduce_kernel<<<t->sm_count * 8, 256, 0, cs>>>(t->hot_ctr, t->work_max, t->hot_work, t->hot_base, t->hot_R,
                                                     t->max_uniq, t->k, t->Gbuf, t->hot_acc);
  DES_LAUNCH_CHECK(t, "hot_reduce_kernel");
  hot_finish_kernel<<<t->sm_count * 2, 256, 0, cs>>>(t->hot_ctr, t->hot_max, t->hot_R, t->hot_u, t->k, t->Gbuf,
                                                     t->hot_acc);
  DES_LAUNCH_CHECK(t, "hot_finish_kernel");
  {
#ifndef UP_GRID
#define UP_GRID 8
#endif
    const unsigned grid = (unsigned)(t->sm_count * UP_GRID);
#define UP2(GG, AD) update_rows_kernel<GG, AD><<<grid, 256, 0, cs>>>(b->uniq_rows, b->n_uniq, t->max_uniq, t->k, ops, \
                                                                   opt, t->meta, t->Gbuf, t->W, t->A, t->A2)
#define UP(GG) do { if (t->A2) UP2(GG, true); else UP2(GG, false); } while (0)
    switch (G) { case 1: UP(1); break; case 2: UP(2); break; case 4: UP(4); break; case 8: UP(8); break; default: UP(16); }
#undef UP
#undef UP2
    DES_LAUNCH_CHECK(t, "update_rows_kernel");
  }
  return DES_OK;
}

// ---- whole step from host buffers ---------------------------------------------
static void* st_alloc(des_table* t, size_t bytes) {
  if (t->cfg.alloc) return t->cfg.alloc(bytes ? bytes : 256, t->cfg.alloc_ctx);
  void* p = nullptr;
  if (cudaMalloc(&p, bytes ? bytes : 256) != cudaSuccess) { cudaGetLastError(); return nullptr; }
  return p;
}

// Device staging of the host-buffer step, sized for the largest batch (first call: allocates, synchronises).
// The batch inputs (offsets, ids, values) have two slots so that the copy of one step can overlap the
// kernels of the step before; everything the kernels produce is single (kernels of consecutive steps run
// in order on the caller's stream).
static des_status_t st_prepare(des_table* t) {
  if (t->st_ready) return DES_OK;
  if (t->st_ids[0]) return DES_ERR_CUDA;               // an earlier attempt ran out of memory half-way
  const size_t nb = (size_t)t->max_batch * t->F + 1;
  for (int s = 0; s < 2; ++s) {
    t->st_offsets[s] = (int32_t*)st_alloc(t, nb * 4);
    t->st_ids[s] = (unsigned long long*)st_alloc(t, (size_t)t->max_nnz * 8);
    t->st_vals[s] = (float*)st_alloc(t, (size_t)t->max_nnz * 4);
    if (!t->st_offsets[s] || !t->st_ids[s] || !t->st_vals[s]) return DES_ERR_CUDA;
  }
  t->st_rows = (uint32_t*)st_alloc(t, (size_t)t->max_nnz * 4);
  t->st_shards = (uint8_t*)st_alloc(t, (size_t)t->max_nnz);
  t->st_uidx = (uint32_t*)st_alloc(t, (size_t)t->max_nnz * 4);
  t->st_uniq_rows = (uint32_t*)st_alloc(t, (size_t)t->max_nnz * 4);
  t->st_n_uniq = (uint32_t*)st_alloc(t, 256);
  t->st_part_small = (float*)st_alloc(t, (size_t)t->S * t->max_batch * t->stride * 4);
  t->st_out_small = (float*)st_alloc(t, (size_t)t->max_batch * t->stride * 4);
  if (!t->st_rows || !t->st_shards || !t->st_uidx || !t->st_uniq_rows || !t->st_n_uniq || !t->st_part_small ||
      !t->st_out_small)
    return DES_ERR_CUDA;
  if (cudaStreamCreateWithFlags(&t->st_copy_stream, cudaStreamNonBlocking) != cudaSuccess) return DES_ERR_CUDA;
  for (int s = 0; s < 2; ++s) {
    if (cudaEventCreateWithFlags(&t->st_copied[s], cudaEventDisableTiming) != cudaSuccess) return DES_ERR_CUDA;
    if (cudaEventCreateWithFlags(&t->st_done[s], cudaEventDisableTiming) != cudaSuccess) return DES_ERR_CUDA;
    t->st_busy[s] = 0;
  }
  t->st_ready = 1;
  return DES_OK;
}

// Enqueues one whole step from host buffers: inputs go to staging slot `slot` on `copy` (the caller's
// stream itself, or the table's copy stream), the kernels and the read-back of out_small on `cs`.
static des_status_t st_enqueue(des_table* t, int slot, cudaStream_t copy, uint32_t ops, int32_t batch, int64_t nnz,
                               const int32_t* h_offsets, const uint64_t* h_ids, const float* h_vals,
                               const des_grads_t* d_grads, float* d_pooled, float* d_Z, float* h_out_small,
                               cudaStream_t cs) {
  const size_t nb = (size_t)batch * t->F + 1;
  DES_CUDA(cudaMemcpyAsync(t->st_offsets[slot], h_offsets, nb * 4, cudaMemcpyHostToDevice, copy));
  if (nnz) DES_CUDA(cudaMemcpyAsync(t->st_ids[slot], h_ids, (size_t)nnz * 8, cudaMemcpyHostToDevice, copy));
  if (h_vals && nnz) DES_CUDA(cudaMemcpyAsync(t->st_vals[slot], h_vals, (size_t)nnz * 4, cudaMemcpyHostToDevice, copy));
  if (copy != cs) {
    DES_CUDA(cudaEventRecord(t->st_copied[slot], copy));
    DES_CUDA(cudaStreamWaitEvent(cs, t->st_copied[slot], 0));
  }
  des_batch_t b;
  b.batch = batch; b.nnz = nnz; b.offsets = t->st_offsets[slot]; b.ids = (const uint64_t*)t->st_ids[slot];
  b.vals = h_vals ? t->st_vals[slot] : nullptr; b.rows = t->st_rows; b.shards = t->st_shards; b.uidx = t->st_uidx;
  b.uniq_rows = t->st_uniq_rows; b.n_uniq = t->st_n_uniq;
  des_partials_t p; p.part_small = t->st_part_small; p.pooled = d_pooled; p.part_pooled = nullptr; p.part_dense = nullptr;
  des_outputs_t o; o.out_small = t->st_out_small; o.pooled = d_pooled; o.Z = d_Z;
  des_status_t st;
  if ((st = des_find_or_insert(t, &b, 1, cs)) != DES_OK) return st;
  if ((st = des_forward_partials(t, ops, &b, &p, cs)) != DES_OK) return st;
  if ((st = des_aggregate(t, ops, &b, &p, &o, cs)) != DES_OK) return st;
  if ((st = des_backward_update(t, ops, &b, &o, d_grads, cs)) != DES_OK) return st;
  DES_CUDA(cudaMemcpyAsync(h_out_small, t->st_out_small, (size_t)batch * t->stride * 4, cudaMemcpyDeviceToHost, cs));
  return DES_OK;
}

static des_status_t st_check_args(des_table* t, int32_t batch, int64_t nnz, const int32_t* h_offsets,
                                  const uint64_t* h_ids, const des_grads_t* d_grads, const float* h_out_small) {
  if (!t || !h_offsets || (nnz > 0 && !h_ids) || !d_grads || !h_out_small) return DES_ERR_INVALID_ARG;
  if (batch <= 0 || batch > t->max_batch || nnz < 0 || nnz > t->max_nnz) return DES_ERR_INVALID_ARG;
  return DES_OK;
}

extern "C" des_status_t des_step_host(des_table_t* t, uint32_t ops, int32_t batch, int64_t nnz,
                                      const int32_t* h_offsets, const uint64_t* h_ids, const float* h_vals,
                                      const des_grads_t* d_grads, float* d_pooled, float* d_Z, float* h_out_small,
                                      void* stream) {
  des_status_t st = st_check_args(t, batch, nnz, h_offsets, h_ids, d_grads, h_out_small);
  if (st != DES_OK) return st;
  if ((st = st_prepare(t)) != DES_OK) return st;
  cudaStream_t cs = (cudaStream_t)stream;
  for (int s = 0; s < 2; ++s)          // steps submitted earlier own the staging slots until they finish
    if (t->st_busy[s]) { DES_CUDA(cudaEventSynchronize(t->st_done[s])); t->st_busy[s] = 0; }
  if ((st = st_enqueue(t, 0, cs, ops, batch, nnz, h_offsets, h_ids, h_vals, d_grads, d_pooled, d_Z, h_out_small, cs)) != DES_OK)
    return st;
  DES_CUDA(cudaStreamSynchronize(cs));
  return DES_OK;
}

extern "C" des_status_t des_step_host_submit(des_table_t* t, uint32_t ops, int32_t batch, int64_t nnz,
                                             const int32_t* h_offsets, const uint64_t* h_ids, const float* h_vals,
                                             const des_grads_t* d_grads, float* d_pooled, float* d_Z,
                                             float* h_out_small, void* stream, int32_t* ticket) {
  des_status_t st = st_check_args(t, batch, nnz, h_offsets, h_ids, d_grads, h_out_small);
  if (st != DES_OK) return st;
  if (!ticket) return DES_ERR_INVALID_ARG;
  if ((st = st_prepare(t)) != DES_OK) return st;
  cudaStream_t cs = (cudaStream_t)stream;
  const int slot = (int)(t->st_next & 1);
  if (t->st_busy[slot]) {              // the step that last used this slot must be over before it is overwritten
    DES_CUDA(cudaEventSynchronize(t->st_done[slot]));
    t->st_busy[slot] = 0;
  }
  if ((st = st_enqueue(t, slot, t->st_copy_stream, ops, batch, nnz, h_offsets, h_ids, h_vals, d_grads, d_pooled, d_Z,
                       h_out_small, cs)) != DES_OK)
    return st;
  DES_CUDA(cudaEventRecord(t->st_done[slot], cs));
  t->st_busy[slot] = 1;
  t->st_next += 1;
  *ticket = slot;
  return DES_OK;
}

extern "C" des_status_t des_step_host_wait(des_table_t* t, int32_t ticket) {
  if (!t || ticket < 0 || ticket > 1) return DES_ERR_INVALID_ARG;
  if (!t->st_ready || !t->st_busy[ticket]) return DES_OK;
  DES_CUDA(cudaEventSynchronize(t->st_done[ticket]));
  t->st_busy[ticket] = 0;
  return DES_OK;
}
