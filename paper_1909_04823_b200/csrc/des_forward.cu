// Forward of the DES sparse operators.
//
// des_forward_partials: the sub-operators M_j of every shard —
//   LR   M_1 = sum_{j in shard} w_j x_j                       (Eq. 2)
//   FM   M_1 = sum v_j x_j,  M_2 = sum <v_j x_j, v_j x_j>      (Eq. 7)
//   POOL per-field sum pooling of the latent vectors          (Section 4.3)
// des_aggregate: (+) over shards in the order s = 0..S-1 (Eq. 1) and the
// substitution operator F = 1/2 <(+)M_1,(+)M_1> - 1/2 (+)M_2 (Eq. 8).
//
// Kernels.
//  route_kernel   every shard gets the ids it owns: one warp per sample buckets
//                 the sample's occurrences by owning shard with a stable counting
//                 sort (warp match + running cursors), writing the table-global
//                 row of every occurrence in shard-major order, the segment
//                 bounds [B][S+1], and the same rows in CSR order for pooling.
//  shard_partials_kernel   one warp per sample (32 / G sub-groups of G = k/4
//                 lanes, rounded up to a power of two) walks the sample's
//                 (sample, shard) segments in shard order: it streams a segment's
//                 rows with 16-byte loads and keeps
//                 M_1, M_1^lr, M_2 in registers until the segment ends — no shared
//                 memory, no atomics, a fixed summation order (deterministic).  M_2 uses the |v|^2 cached in the
//                 row's 16-byte tail.  Fused variant: (+) over shards and F on chip.
//  pool_kernel    one group per bag: sum pooling of the latent vectors in
//                 registers.  The per-shard pooled partial [S][B][F*k] is only
//                 materialised (with atomics) when the caller asks for it.
//
// FIELD partition (field f on shard f mod S): a bag belongs to one shard, so when pooling is among the
// operators one gather pass (single_gather_kernel: pooled vectors and per-bag sums of the linear weights and
// squared norms) feeds everything, and field_partials_kernel forms shard s's sub-operators as the sums over
// the bags of its own fields — no routing pass, no second gather.
//
// Accuracy.  A lane never adds more than a few dozen terms into one float32 accumulator (long
// segments are summed in two levels), and the sum over shards is taken in double and rounded once, so
// every per-sample sum keeps the stated float32 tolerance even when one key contributes
// hundreds of equal terms that the other terms cancel.
#include "des_internal.cuh"

#ifndef POOL_BLOCKS_PER_SM
#define POOL_BLOCKS_PER_SM 64   // grid cap of the pooling kernel (it strides over the bags)
#endif


#ifndef ROUTE_PF
#define ROUTE_PF 8    // batches of 32 occurrences whose loads a warp keeps in flight
#endif
__global__ void __launch_bounds__(256) route_kernel(
    const int32_t* __restrict__ offsets, const float* __restrict__ vals, const uint32_t* __restrict__ rows,
    const uint8_t* __restrict__ shards, int B, int F, int S, const DevMeta* __restrict__ meta, uint32_t null_row,
    uint32_t* __restrict__ grow_csr, uint32_t* __restrict__ grow_sorted, float* __restrict__ x_sorted,
    int32_t* __restrict__ seg_off) {
  __shared__ uint32_t row_base[DES_MAX_SHARDS];
  __shared__ int cursor[8][DES_MAX_SHARDS];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if (threadIdx.x < S) row_base[threadIdx.x] = (uint32_t)meta->row_base[threadIdx.x];
  __syncthreads();
  int* cur = cursor[warp];
  const unsigned lt = (1u << lane) - 1u;
  for (int b = blockIdx.x * 8 + warp; b < B; b += gridDim.x * 8) {
    const int lo = __ldg(offsets + (size_t)b * F), hi = __ldg(offsets + (size_t)(b + 1) * F);
    for (int s = lane; s < S; s += 32) cur[s] = 0;
    __syncwarp();
    // pass 1: occurrences per shard (mapped rows only); CSR-order rows for the pooling kernel.
    // Both passes keep the loads of the next ROUTE_PF x 32 occurrences in flight while they work on the
    // current ones (a warp is one dependent chain per sample; what it waits for is memory latency).
    {
      uint32_t rq[ROUTE_PF]; int sq[ROUTE_PF];
#pragma unroll
      for (int q = 0; q < ROUTE_PF; ++q) {
        const int j = lo + q * 32 + lane;
        rq[q] = DES_ROW_NONE; sq[q] = 0;
        if (j < hi) { rq[q] = __ldg(rows + j); sq[q] = __ldg(shards + j); }
      }
      for (int base = lo; base < hi; base += 32 * ROUTE_PF) {
#pragma unroll
        for (int q = 0; q < ROUTE_PF; ++q) {
          const int j = base + q * 32 + lane;
          const uint32_t r = rq[q]; const int s = sq[q];
          if (j + 32 * ROUTE_PF < hi) { rq[q] = __ldg(rows + j + 32 * ROUTE_PF); sq[q] = __ldg(shards + j + 32 * ROUTE_PF); }
          if (j < hi) {
            grow_csr[j] = (r == DES_ROW_NONE) ? null_row : row_base[s] + r;
            if (r != DES_ROW_NONE) atomicAdd(&cur[s], 1);   // counting only: order does not matter here
          }
        }
      }
      __syncwarp();
    }
    // exclusive scan over shards -> segment starts (two counters per lane, S <= 64, warp scans)
    {
      static_assert(DES_MAX_SHARDS <= 64, "two counters per lane");
      const int c0 = lane < S ? cur[lane] : 0, c1 = lane + 32 < S ? cur[lane + 32] : 0;
      int i0 = c0, i1 = c1;
#pragma unroll
      for (int d = 1; d < 32; d <<= 1) {
        const int v0 = __shfl_up_sync(0xFFFFFFFFu, i0, d), v1 = __shfl_up_sync(0xFFFFFFFFu, i1, d);
        if (lane >= d) { i0 += v0; i1 += v1; }
      }
      const int t0 = __shfl_sync(0xFFFFFFFFu, i0, 31), t1 = __shfl_sync(0xFFFFFFFFu, i1, 31);
      int32_t* so = seg_off + (size_t)b * (S + 1);
      __syncwarp();
      if (lane < S) { cur[lane] = lo + i0 - c0; so[lane] = lo + i0 - c0; }
      if (lane + 32 < S) { cur[lane + 32] = lo + t0 + i1 - c1; so[lane + 32] = lo + t0 + i1 - c1; }
      if (lane == 0) so[S] = lo + t0 + t1;
    }
    __syncwarp();
    // pass 2: stable placement
    {
      uint32_t rq[ROUTE_PF]; int sq[ROUTE_PF]; float xq[ROUTE_PF];
#pragma unroll
      for (int q = 0; q < ROUTE_PF; ++q) {
        const int j = lo + q * 32 + lane;
        rq[q] = DES_ROW_NONE; sq[q] = 0; xq[q] = 1.f;
        if (j < hi) {
          rq[q] = __ldg(rows + j); sq[q] = __ldg(shards + j);
          if (vals) xq[q] = __ldg(vals + j);
        }
      }
      for (int base = lo; base < hi; base += 32 * ROUTE_PF) {
#pragma unroll
        for (int q = 0; q < ROUTE_PF; ++q) {
          if (base + q * 32 >= hi) break;                  // whole warp
          const int j = base + q * 32 + lane;
          const uint32_t r = rq[q]; const int s = sq[q]; const float x = xq[q];
          if (j + 32 * ROUTE_PF < hi) {
            rq[q] = __ldg(rows + j + 32 * ROUTE_PF); sq[q] = __ldg(shards + j + 32 * ROUTE_PF);
            if (vals) xq[q] = __ldg(vals + j + 32 * ROUTE_PF);
          }
          int key = -1 - lane; uint32_t gr = 0;
          if (j < hi && r != DES_ROW_NONE) { key = s; gr = row_base[s] + r; }
          // the first lane of every group of equal shards advances the shard's cursor (a warp's
          // shared-memory atomics execute in program order, so successive batches stay ordered) and
          // hands the old value to its group
          const unsigned same = __match_any_sync(0xFFFFFFFFu, key);
          const int leader = __ffs(same) - 1;
          int first = 0;
          if (key >= 0 && lane == leader) first = atomicAdd(&cur[key], __popc(same));
          first = __shfl_sync(0xFFFFFFFFu, first, leader);
          if (key >= 0) {
            const int pos = first + __popc(same & lt);
            grow_sorted[pos] = gr;
            if (vals) x_sorted[pos] = x;
          }
        }
      }
    }
  }
}

// One round of a (sample, shard) segment: U rows per lane in flight, occurrences i, i + P, ... below `hi`;
// positions past the segment's end read the all-zero row behind the table, so a round has no branch.
template <int U, int P, bool HAS_VALS>
__device__ __forceinline__ void sp_round(const uint32_t* __restrict__ grow_sorted, const float* __restrict__ x_sorted,
                                         int i, int hi, uint32_t null_row, const char* __restrict__ Wc,
                                         const char* __restrict__ Wt, unsigned rowB, float4& acc, float& m1lr, float& m2) {
  float4 v[U]; float2 tl[U]; float x[U]; uint32_t g[U];
#pragma unroll
  for (int u = 0; u < U; ++u) {
    const bool in = i + u * P < hi;
    g[u] = in ? __ldg(grow_sorted + i + u * P) : null_row;
    if (HAS_VALS) x[u] = in ? __ldg(x_sorted + i + u * P) : 0.f;
  }
#pragma unroll
  for (int u = 0; u < U; ++u) {
    const size_t off = (size_t)DES_DBG_ROW(g[u]) * rowB;
    v[u] = __ldg(reinterpret_cast<const float4*>(Wc + off));
    tl[u] = __ldg(reinterpret_cast<const float2*>(Wt + off));
  }
#pragma unroll
  for (int u = 0; u < U; ++u) {
    if (HAS_VALS) {
      acc.x += v[u].x * x[u]; acc.y += v[u].y * x[u]; acc.z += v[u].z * x[u]; acc.w += v[u].w * x[u];
      m1lr += tl[u].x * x[u]; m2 += tl[u].y * x[u] * x[u];
    } else {
      acc.x += v[u].x; acc.y += v[u].y; acc.z += v[u].z; acc.w += v[u].w;
      m1lr += tl[u].x; m2 += tl[u].y;
    }
  }
}

// Same for a bag: U rows per lane, optionally also added to the per-shard copy of the pooled sum
// (MATERIALISE, tests only).
template <int U, int P, bool HAS_VALS, bool MATERIALISE>
__device__ __forceinline__ void pool_step(const uint32_t* __restrict__ grow_csr, const float* __restrict__ vals,
                                          const uint8_t* __restrict__ shards, int i, const char* __restrict__ Wc,
                                          unsigned rowB, uint32_t null_row, float* __restrict__ part_block, size_t shard_pitch,
                                          bool col, float4& acc) {
  float4 v[U]; float x[U]; uint32_t gr[U];
#pragma unroll
  for (int u = 0; u < U; ++u) {
    gr[u] = DES_DBG_ROW(__ldg(grow_csr + i + u * P));
    if (HAS_VALS) x[u] = __ldg(vals + i + u * P);
    v[u] = __ldg(reinterpret_cast<const float4*>(Wc + (size_t)gr[u] * rowB));
  }
#pragma unroll
  for (int u = 0; u < U; ++u) {
    float4 vx = v[u];
    if (HAS_VALS) { vx.x *= x[u]; vx.y *= x[u]; vx.z *= x[u]; vx.w *= x[u]; }
    acc.x += vx.x; acc.y += vx.y; acc.z += vx.z; acc.w += vx.w;
    if (MATERIALISE && col && gr[u] != null_row)
      atomicAdd(reinterpret_cast<float4*>(part_block + (size_t)__ldg(shards + i + u * P) * shard_pitch), vx);
  }
}

// One WARP per sample walks the sample's S segments in shard order.  The warp is
// split into P = 32 / G sub-groups of G lanes (one 16-byte column per lane);
// sub-group p takes occurrences p, p + P, ... of a segment, SP_U of them in
// flight per round, and the sub-groups' sums are combined by a butterfly when the
// segment ends — so both halves of a warp always run the same trip counts, whatever
// the skew between shards, and every warp has the same amount of work (a sample's
// occurrences).  What a warp waits for is memory latency, one dependent chain per
// sample, so the chain is kept short: the sample's S + 1 segment bounds are read
// once (two per lane) and handed round by shuffles, and a round's row numbers are
// all fetched before its rows (positions past the segment's end name the all-zero
// row: no branch).  Lanes without a column of their own (k not a multiple of 4 G)
// re-read column 0 instead of branching.  A lane's float32 sums move on into a
// second set of accumulators every SP_FLUSH rounds, so that no accumulator takes more
// than a few dozen additions; the sum over shards runs in double.  part_small
// (optional) receives each segment's partial sums, rounded to float32, as soon as
// the segment ends; with FUSED the aggregation (+) over shards and the substitution
// operator F are applied on chip, in the same shard order and with the same
// arithmetic as aggregate_small_kernel (the sum of the float32-rounded partials in
// double), and out_small is written directly — the per-shard partials then never
// touch memory.
#define SP_U 4
#define SP_FLUSH 4
template <int G, bool HAS_VALS, bool FUSED>
__global__ void __launch_bounds__(256) shard_partials_kernel(
    const uint32_t* __restrict__ grow_sorted, const float* __restrict__ x_sorted, const int32_t* __restrict__ seg_off,
    int B, int S, int k, uint32_t ops, const float* __restrict__ W, uint32_t null_row, float* __restrict__ part_small,
    float* __restrict__ out_small) {
  constexpr int P = 32 / G;
  const int K4 = k >> 2, stride = k + 4;
  const int lane = threadIdx.x & 31;
  const int b = blockIdx.x * 8 + (threadIdx.x >> 5);
  if (b >= B) return;                                  // whole warp
  const int c4 = lane % G, p = lane / G;
  const bool col = c4 < K4;
  const bool lr = ops & DES_OP_LR, fm = ops & DES_OP_FM;
  const float4 zero4 = make_float4(0.f, 0.f, 0.f, 0.f);
  const unsigned rowB = (unsigned)stride * 4u;         // bytes per row
  const char* Wc = reinterpret_cast<const char*>(W) + (col ? c4 : 0) * 16;
  const char* Wt = reinterpret_cast<const char*>(W + k);                       // (w, |v|^2)
  double Ax = 0.0, Ay = 0.0, Az = 0.0, Aw = 0.0, R = 0.0, Q = 0.0;   // FUSED: (+)M_1, (+)M_1^lr, (+)M_2
  // the sample's segment bounds: lane l holds bounds l and l + 32, lane 0 also bound 64 (S <= 64)
  const int32_t* so = seg_off + (size_t)b * (S + 1);
  static_assert(DES_MAX_SHARDS <= 64, "three bounds per lane");
  const int o0 = lane <= S ? __ldg(so + lane) : 0, o1 = lane + 32 <= S ? __ldg(so + lane + 32) : 0;
  const int o2 = (lane == 0 && S == 64) ? __ldg(so + 64) : 0;
  auto bound = [&](int s) { return s < 32 ? __shfl_sync(0xFFFFFFFFu, o0, s) : s < 64 ? __shfl_sync(0xFFFFFFFFu, o1, s - 32)
                                                                                     : __shfl_sync(0xFFFFFFFFu, o2, 0); };
  int hi = bound(0);
  for (int s = 0; s < S; ++s) {
    const int lo = hi;
    hi = bound(s + 1);
    float4 acc = zero4, up = zero4;
    float m1lr = 0.f, m2 = 0.f, up_l = 0.f, up_q = 0.f;
    int round = 0;
    for (int i0 = lo; i0 < hi; i0 += SP_U * P) {
      sp_round<SP_U, P, HAS_VALS>(grow_sorted, x_sorted, i0 + p, hi, null_row, Wc, Wt, rowB, acc, m1lr, m2);
      if ((++round & (SP_FLUSH - 1)) == 0) {           // (a long segment: one hot id, hundreds of times in the sample)
        up.x += acc.x; up.y += acc.y; up.z += acc.z; up.w += acc.w; up_l += m1lr; up_q += m2;
        acc = zero4; m1lr = 0.f; m2 = 0.f;
      }
    }
    acc.x += up.x; acc.y += up.y; acc.z += up.z; acc.w += up.w; m1lr += up_l; m2 += up_q;
#pragma unroll
    for (int d = G; d < 32; d <<= 1) {                 // combine the sub-groups (same result in every lane)
      acc.x += __shfl_xor_sync(0xFFFFFFFFu, acc.x, d); acc.y += __shfl_xor_sync(0xFFFFFFFFu, acc.y, d);
      acc.z += __shfl_xor_sync(0xFFFFFFFFu, acc.z, d); acc.w += __shfl_xor_sync(0xFFFFFFFFu, acc.w, d);
      m1lr += __shfl_xor_sync(0xFFFFFFFFu, m1lr, d); m2 += __shfl_xor_sync(0xFFFFFFFFu, m2, d);
    }
    if (!fm) { acc = zero4; m2 = 0.f; }
    if (!lr) m1lr = 0.f;
    if (part_small && p == 0) {
      float4* dst = reinterpret_cast<float4*>(part_small + ((size_t)s * B + b) * stride);
      if (col) dst[c4] = acc;
      if (c4 == 0) dst[K4] = make_float4(m1lr, m2, 0.f, 0.f);
    }
    if (FUSED) {
      Ax += (double)acc.x; Ay += (double)acc.y; Az += (double)acc.z; Aw += (double)acc.w;
      R += (double)m1lr; Q += (double)m2;
    }
  }
  if (FUSED) {
    double aa = col ? Ax * Ax + Ay * Ay + Az * Az + Aw * Aw : 0.0;
#pragma unroll
    for (int d = 1; d < G; d <<= 1) aa += __shfl_xor_sync(0xFFFFFFFFu, aa, d);
    float4* o = reinterpret_cast<float4*>(out_small + (size_t)b * stride);
    if (p == 0 && col) o[c4] = make_float4((float)Ax, (float)Ay, (float)Az, (float)Aw);
    if (lane == 0) o[K4] = make_float4((float)R, fm ? (float)(0.5 * aa - 0.5 * Q) : 0.f, (float)Q, 0.f);
  }
}

// four floats rounded to bfloat16 (RNE), one 8-byte store
__device__ __forceinline__ void store_bf16x4(__nv_bfloat16* dst, const float4& v) {
  const __nv_bfloat162 a = __floats2bfloat162_rn(v.x, v.y), b = __floats2bfloat162_rn(v.z, v.w);
  *reinterpret_cast<uint2*>(dst) = make_uint2(*reinterpret_cast<const uint32_t*>(&a), *reinterpret_cast<const uint32_t*>(&b));
}

template <int G, int P, bool HAS_VALS, bool MATERIALISE, bool BF16OUT>
__global__ void __launch_bounds__(256) pool_kernel(
    const int32_t* __restrict__ offsets, const float* __restrict__ vals, const uint32_t* __restrict__ grow_csr,
    const uint8_t* __restrict__ shards, long long nbags, int B, int F, int k, const float* __restrict__ W,
    uint32_t null_row, float* __restrict__ pooled, float* __restrict__ part_pooled, __nv_bfloat16* __restrict__ pooled_b) {
  constexpr int LB = G * P;                            // lanes per bag
  const int K4 = k >> 2, stride = k + 4;
  const int sub = threadIdx.x % LB, c4 = sub % G, p = sub / G;
  const bool col = c4 < K4;
  const unsigned rowB = (unsigned)stride * 4u;
  const char* Wc = reinterpret_cast<const char*>(W) + (col ? c4 : 0) * 16;
  const size_t shard_pitch = (size_t)B * F * k;
  // grid-stride over bags (every lane of a warp runs the same number of rounds); the next bag's bounds are
  // fetched while the current bag is summed
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
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    // MATERIALISE: this lane's column of block (shard 0, sample, field) of part_pooled [S][B][F*k]
    float* part_block = nullptr;
    if (MATERIALISE && live) part_block = part_pooled + (size_t)bag * k + (col ? c4 : 0) * 4;
    int i0 = lo;
#define POOL_STEP(U) pool_step<U, P, HAS_VALS, MATERIALISE>(grow_csr, vals, shards, i0 + p, Wc, rowB, null_row, part_block, \
                                                           shard_pitch, col, acc)
    for (; i0 + 4 * P <= hi; i0 += 4 * P) POOL_STEP(4);
    if (i0 + 2 * P <= hi) { POOL_STEP(2); i0 += 2 * P; }
    if (i0 + P <= hi) { POOL_STEP(1); i0 += P; }
    if (i0 + p < hi) POOL_STEP(1);
#undef POOL_STEP
#pragma unroll
    for (int d = G; d < LB; d <<= 1) {                 // combine the bag's sub-groups
      acc.x += __shfl_xor_sync(0xFFFFFFFFu, acc.x, d); acc.y += __shfl_xor_sync(0xFFFFFFFFu, acc.y, d);
      acc.z += __shfl_xor_sync(0xFFFFFFFFu, acc.z, d); acc.w += __shfl_xor_sync(0xFFFFFFFFu, acc.w, d);
    }
    if (live && p == 0 && col) {
      reinterpret_cast<float4*>(pooled + bag * k)[c4] = acc;
      if (BF16OUT) store_bf16x4(pooled_b + bag * k + c4 * 4, acc);    // operand of the first-layer product
    }
  }
}

// (+) over shards and F.  G lanes per sample, one float4 column each; lane 0 of
// the group also carries the tail (R_lr, Q).  The float32 partials are added in
// double in shard order and rounded once; <A, A> is taken on the double sums.
template <int G>
__global__ void __launch_bounds__(256) aggregate_small_kernel(const float* __restrict__ part_small, int B, int S, int k,
                                                              uint32_t ops, float* __restrict__ out_small) {
  const int K4 = k >> 2, stride = k + 4;
  const int t = blockIdx.x * blockDim.x + threadIdx.x;
  const int b = t / G, c4 = t % G;
  const bool live = b < B;
  double ax = 0.0, ay = 0.0, az = 0.0, aw = 0.0, tr = 0.0, tq = 0.0;
  if (live) {
    for (int s = 0; s < S; ++s) {
      const float4* p = reinterpret_cast<const float4*>(part_small + ((size_t)s * B + b) * stride);
      if (c4 < K4) { float4 v = __ldg(p + c4); ax += (double)v.x; ay += (double)v.y; az += (double)v.z; aw += (double)v.w; }
      if (c4 == 0) { float4 v = __ldg(p + K4); tr += (double)v.x; tq += (double)v.y; }
    }
  }
  double aa = ax * ax + ay * ay + az * az + aw * aw;
#pragma unroll
  for (int d = 1; d < G; d <<= 1) aa += __shfl_xor_sync(0xFFFFFFFFu, aa, d);
  if (!live) return;
  float4* o = reinterpret_cast<float4*>(out_small + (size_t)b * stride);
  if (c4 < K4) o[c4] = make_float4((float)ax, (float)ay, (float)az, (float)aw);
  if (c4 == 0) {
    const float fm2 = (ops & DES_OP_FM) ? (float)(0.5 * aa - 0.5 * tq) : 0.f;
    o[K4] = make_float4((float)tr, fm2, (float)tq, 0.f);
  }
}

// ---- single-gather forward (des_forward_fused with pooling in `ops`) -----------------------------------
// Every occurrence's row is read ONCE: the group that pools a bag also sums the bag's linear weights and
// cached squared norms, and a second, small kernel adds a sample's bags up in double: A = sum over fields of
// the pooled vectors, R_lr and Q = the sums of the bag tails.  The per-shard partials are never formed (the
// sum over a sample's occurrences is taken field by field instead of shard by shard — Eq. 1 with (+) = +
// allows any grouping), so the results agree with the two-call path within the float32 tolerance, not bit
// for bit.  Reads the batch as find_or_insert left it (shard-local rows + shards): no routing pass.
template <int U, int P, bool HAS_VALS>
__device__ __forceinline__ void sg_step(const uint32_t* __restrict__ rows, const uint8_t* __restrict__ shards,
                                        const float* __restrict__ vals, const uint32_t* __restrict__ s_base, int i,
                                        const char* __restrict__ Wc, const char* __restrict__ Wt, unsigned rowB,
                                        uint32_t null_row, float4& acc, float& bl, float& bq) {
  float4 v[U]; float2 tl[U]; float x[U];
#pragma unroll
  for (int u = 0; u < U; ++u) {
    const uint32_t r = __ldg(rows + i + u * P);
    const uint32_t g = (r == DES_ROW_NONE) ? null_row : s_base[__ldg(shards + i + u * P)] + r;
    const size_t off = (size_t)DES_DBG_ROW(g) * rowB;
    if (HAS_VALS) x[u] = __ldg(vals + i + u * P);
    v[u] = __ldg(reinterpret_cast<const float4*>(Wc + off));
    tl[u] = __ldg(reinterpret_cast<const float2*>(Wt + off));
  }
#pragma unroll
  for (int u = 0; u < U; ++u) {
    if (HAS_VALS) {
      acc.x += v[u].x * x[u]; acc.y += v[u].y * x[u]; acc.z += v[u].z * x[u]; acc.w += v[u].w * x[u];
      bl += tl[u].x * x[u]; bq += tl[u].y * x[u] * x[u];
    } else {
      acc.x += v[u].x; acc.y += v[u].y; acc.z += v[u].z; acc.w += v[u].w;
      bl += tl[u].x; bq += tl[u].y;
    }
  }
}

template <int G, int P, bool HAS_VALS>
__global__ void __launch_bounds__(256) single_gather_kernel(
    const int32_t* __restrict__ offsets, const float* __restrict__ vals, const uint32_t* __restrict__ rows,
    const uint8_t* __restrict__ shards, long long nbags, int S, int k, const float* __restrict__ W,
    const DevMeta* __restrict__ meta, uint32_t null_row, float* __restrict__ pooled, float2* __restrict__ bag_tail,
    __nv_bfloat16* __restrict__ pooled_b) {
  constexpr int LB = G * P;                            // lanes per bag
  __shared__ uint32_t s_base[DES_MAX_SHARDS];
  if (threadIdx.x < S) s_base[threadIdx.x] = (uint32_t)meta->row_base[threadIdx.x];
  __syncthreads();
  const int K4 = k >> 2, stride = k + 4;
  const int sub = threadIdx.x % LB, c4 = sub % G, p = sub / G;
  const bool col = c4 < K4;
  const unsigned rowB = (unsigned)stride * 4u;
  const char* Wc = reinterpret_cast<const char*>(W) + (col ? c4 : 0) * 16;
  const char* Wt = reinterpret_cast<const char*>(W + k);
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
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    float bl = 0.f, bq = 0.f;
    int i0 = lo;
#define SG_STEP(U) sg_step<U, P, HAS_VALS>(rows, shards, vals, s_base, i0 + p, Wc, Wt, rowB, null_row, acc, bl, bq)
    for (; i0 + 4 * P <= hi; i0 += 4 * P) SG_STEP(4);
    if (i0 + 2 * P <= hi) { SG_STEP(2); i0 += 2 * P; }
    if (i0 + P <= hi) { SG_STEP(1); i0 += P; }
    if (i0 + p < hi) SG_STEP(1);
#undef SG_STEP
#pragma unroll
    for (int d = G; d < LB; d <<= 1) {                 // combine the bag's sub-groups
      acc.x += __shfl_xor_sync(0xFFFFFFFFu, acc.x, d); acc.y += __shfl_xor_sync(0xFFFFFFFFu, acc.y, d);
      acc.z += __shfl_xor_sync(0xFFFFFFFFu, acc.z, d); acc.w += __shfl_xor_sync(0xFFFFFFFFu, acc.w, d);
      bl += __shfl_xor_sync(0xFFFFFFFFu, bl, d); bq += __shfl_xor_sync(0xFFFFFFFFu, bq, d);
    }
    if (live && p == 0) {
      if (col) {
        reinterpret_cast<float4*>(pooled + bag * k)[c4] = acc;
        if (pooled_b) store_bf16x4(pooled_b + bag * k + c4 * 4, acc);
      }
      if (c4 == 0) bag_tail[bag] = make_float2(bl, bq);
    }
  }
}

// A, R_lr, Q and F per sample from the pooled vectors and bag tails of its F bags, added in double in field
// order.  G lanes per sample, one float4 column each; lane 0 of the group carries the tails.
template <int G>
__global__ void __launch_bounds__(256) fused_finish_kernel(const float* __restrict__ pooled, const float2* __restrict__ bag_tail,
                                                           int B, int F, int k, uint32_t ops, float* __restrict__ out_small) {
  const int K4 = k >> 2, stride = k + 4;
  const int t = blockIdx.x * blockDim.x + threadIdx.x;
  const int b = t / G, c4 = t % G;
  const bool live = b < B;
  const bool lr = ops & DES_OP_LR, fm = ops & DES_OP_FM;
  double ax = 0.0, ay = 0.0, az = 0.0, aw = 0.0, tr = 0.0, tq = 0.0;
  if (live) {
    const float4* pb = reinterpret_cast<const float4*>(pooled + (size_t)b * F * k) + c4;
    const float2* tb = bag_tail + (size_t)b * F;
    int f = 0;
    for (; f + 4 <= F; f += 4) {                       // four bags in flight
      float4 v[4]; float2 tl[4];
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        v[q] = (c4 < K4 && fm) ? __ldg(pb + (size_t)(f + q) * K4) : make_float4(0.f, 0.f, 0.f, 0.f);
        tl[q] = (c4 == 0) ? __ldg(tb + f + q) : make_float2(0.f, 0.f);
      }
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        ax += (double)v[q].x; ay += (double)v[q].y; az += (double)v[q].z; aw += (double)v[q].w;
        tr += (double)tl[q].x; tq += (double)tl[q].y;
      }
    }
    for (; f < F; ++f) {
      if (c4 < K4 && fm) { const float4 v = __ldg(pb + (size_t)f * K4); ax += (double)v.x; ay += (double)v.y; az += (double)v.z; aw += (double)v.w; }
      if (c4 == 0) { const float2 tl = __ldg(tb + f); tr += (double)tl.x; tq += (double)tl.y; }
    }
  }
  if (!lr) tr = 0.0;
  if (!fm) tq = 0.0;
  double aa = ax * ax + ay * ay + az * az + aw * aw;
#pragma unroll
  for (int d = 1; d < G; d <<= 1) aa += __shfl_xor_sync(0xFFFFFFFFu, aa, d);
  if (!live) return;
  float4* o = reinterpret_cast<float4*>(out_small + (size_t)b * stride);
  if (c4 < K4) o[c4] = make_float4((float)ax, (float)ay, (float)az, (float)aw);
  if (c4 == 0) o[K4] = make_float4((float)tr, fm ? (float)(0.5 * aa - 0.5 * tq) : 0.f, (float)tq, 0.f);
}

// FIELD partition: a bag belongs to one shard (field f lives on shard f mod S), so the sub-operators of shard s
// are sums over the bags of its own fields — which the pooling pass has already formed (pooled vectors, bag
// tails).  G lanes per sample walk the shards in order; shard s adds its fields f = s, s + S, ... in field order
// (float32, a handful of terms), part_small receives the partial, and with FUSED the partials are added in
// double in shard order and passed through F exactly as aggregate_small_kernel does.
template <int G, bool FUSED>
__global__ void __launch_bounds__(256) field_partials_kernel(const float* __restrict__ pooled, const float2* __restrict__ bag_tail,
                                                             int B, int F, int S, int k, uint32_t ops,
                                                             float* __restrict__ part_small, float* __restrict__ out_small) {
  const int K4 = k >> 2, stride = k + 4;
  const int t = blockIdx.x * blockDim.x + threadIdx.x;
  const int b = t / G, c4 = t % G;
  const bool live = b < B, col = c4 < K4;
  const bool lr = ops & DES_OP_LR, fm = ops & DES_OP_FM;
  double Ax = 0.0, Ay = 0.0, Az = 0.0, Aw = 0.0, R = 0.0, Q = 0.0;
  if (live) {
    const float4* pb = reinterpret_cast<const float4*>(pooled + (size_t)b * F * k) + c4;
    const float2* tb = bag_tail + (size_t)b * F;
    for (int s = 0; s < S; ++s) {
      float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
      float m1lr = 0.f, m2 = 0.f;
      for (int f = s; f < F; f += S) {
        if (col && fm) { const float4 v = __ldg(pb + (size_t)f * K4); acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w; }
        if (c4 == 0) { const float2 tl = __ldg(tb + f); m1lr += tl.x; m2 += tl.y; }
      }
      if (!fm) m2 = 0.f;
      if (!lr) m1lr = 0.f;
      if (part_small) {
        float4* dst = reinterpret_cast<float4*>(part_small + ((size_t)s * B + b) * stride);
        if (col) dst[c4] = acc;
        if (c4 == 0) dst[K4] = make_float4(m1lr, m2, 0.f, 0.f);
      }
      if (FUSED) {
        Ax += (double)acc.x; Ay += (double)acc.y; Az += (double)acc.z; Aw += (double)acc.w;
        R += (double)m1lr; Q += (double)m2;
      }
    }
  }
  if (FUSED) {
    double aa = col ? Ax * Ax + Ay * Ay + Az * Az + Aw * Aw : 0.0;
#pragma unroll
    for (int d = 1; d < G; d <<= 1) aa += __shfl_xor_sync(0xFFFFFFFFu, aa, d);
    if (!live) return;
    float4* o = reinterpret_cast<float4*>(out_small + (size_t)b * stride);
    if (col) o[c4] = make_float4((float)Ax, (float)Ay, (float)Az, (float)Aw);
    if (c4 == 0) o[K4] = make_float4((float)R, fm ? (float)(0.5 * aa - 0.5 * Q) : 0.f, (float)Q, 0.f);
  }
}

// sum over shards of a dense [S][B][n] tensor (materialised pooled / dense partials)
__global__ void reduce_shards_kernel(const float* __restrict__ part, size_t per_shard, int S, float* __restrict__ out) {
  size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x, st = (size_t)gridDim.x * blockDim.x;
  for (; i < per_shard; i += st) {
    float a = 0.f;
    for (int s = 0; s < S; ++s) a += __ldg(part + (size_t)s * per_shard + i);
    out[i] = a;
  }
}

static int group_for(int k) { int K4 = k / 4, G = 1; while (G < K4) G <<= 1; return G; }

static des_status_t launch_single_gather(des_table_t* t, uint32_t ops, const des_batch_t* b, float* pooled, cudaStream_t cs);

// shared by des_forward_partials (fused_out == NULL) and des_forward_fused
static des_status_t forward_impl(des_table_t* t, uint32_t ops, const des_batch_t* b, const des_partials_t* part,
                                 float* fused_out, void* stream) {
  des_status_t st = des_check_batch(t, b, 0);
  if (st != DES_OK) return st;
  if (!part || (ops & ~15u) || ops == 0) return DES_ERR_INVALID_ARG;
  const bool small = ops & (DES_OP_LR | DES_OP_FM), pool = ops & (DES_OP_POOL | DES_OP_DENSE1);
  if (small && !part->part_small && !fused_out) return DES_ERR_INVALID_ARG;
  if (!small) fused_out = nullptr;
  if (pool && !part->pooled) return DES_ERR_INVALID_ARG;
  if ((ops & DES_OP_DENSE1) && !t->H) return DES_ERR_INVALID_ARG;
  cudaStream_t cs = (cudaStream_t)stream;
  des_api_begin(t, cs);
  DES_DBG_ARM(t, cs);
  const int B = b->batch;
  float* ps = small ? part->part_small : nullptr;
  float* pl = pool ? part->pooled : nullptr;
  float* pp = pool ? part->part_pooled : nullptr;
  if (pp) DES_CUDA(cudaMemsetAsync(pp, 0, (size_t)t->S * B * t->F * t->k * 4, cs));
  const int G = group_for(t->k);
  if (t->cfg.partition == DES_PART_FIELD && pl && !pp && (ps || fused_out)) {
    // FIELD partition with pooling among the operators: one gather pass (pooled vectors + bag tails), then the
    // per-shard sub-operators as sums over each shard's own fields — no routing pass, no second gather
    if ((st = launch_single_gather(t, ops, b, pl, cs)) != DES_OK) return st;
    const int grid = (int)(((long long)B * G + 255) / 256);
#define FP2(GG, FU) field_partials_kernel<GG, FU><<<grid, 256, 0, cs>>>(pl, t->bag_tail, B, (int)t->F, (int)t->S, t->k, ops, ps, fused_out)
#define FP(GG) do { if (fused_out) FP2(GG, true); else FP2(GG, false); } while (0)
    switch (G) { case 1: FP(1); break; case 2: FP(2); break; case 4: FP(4); break; case 8: FP(8); break; default: FP(16); }
#undef FP
#undef FP2
    DES_LAUNCH_CHECK(t, "field_partials_kernel");
    return DES_OK;
  }
  // routing: rows of every occurrence in shard-major order per sample (workspace shared with find_or_insert,
  // which has finished with it by the time a forward can run on the same stream)
  uint32_t* grow_csr = t->uslot;
  uint32_t* grow_sorted = t->slot_of;
  float* x_sorted = t->x_sorted;
  route_kernel<<<(B + 7) / 8 < t->sm_count * 8 ? (B + 7) / 8 : t->sm_count * 8, 256, 0, cs>>>(
      b->offsets, b->vals, b->rows, b->shards, B, t->F, t->S, t->meta, (uint32_t)t->total_rows, grow_csr, grow_sorted,
      x_sorted, t->seg_off);
  DES_LAUNCH_CHECK(t, "route_kernel");
  if (ps || fused_out) {
    const unsigned grid = (unsigned)((B + 7) / 8);      // one warp per sample
#define SP3(GG, HV, FU) shard_partials_kernel<GG, HV, FU><<<grid, 256, 0, cs>>>(grow_sorted, x_sorted, t->seg_off, B, t->S, \
                                                                              t->k, ops, t->W, (uint32_t)t->total_rows, ps, fused_out)
#define SP(GG) do { if (fused_out) { if (b->vals) SP3(GG, true, true); else SP3(GG, false, true); } \
                    else { if (b->vals) SP3(GG, true, false); else SP3(GG, false, false); } } while (0)
    switch (G) { case 1: SP(1); break; case 2: SP(2); break; case 4: SP(4); break; case 8: SP(8); break; default: SP(16); }
#undef SP
#undef SP3
    DES_LAUNCH_CHECK(t, "shard_partials_kernel");
  }
  if (pl) {
    const long long nbags = (long long)B * t->F;
    // long bags: a whole warp per bag (its halves take alternate occurrences); short bags: G lanes per bag
    const bool wide = b->nnz >= 8 * nbags;            // (at 4 ids per bag the narrow form measured faster)
    const long long threads = nbags * (wide ? 32 : G);
    long long blocks = (threads + 255) / 256;
    if (blocks > (long long)t->sm_count * POOL_BLOCKS_PER_SM) blocks = (long long)t->sm_count * POOL_BLOCKS_PER_SM;
    const unsigned grid = (unsigned)blocks;
    // with the first layer among the operators the pooled vectors are also left as bfloat16, the operand
    // format of the tensor-core product that follows (one conversion pass less)
    __nv_bfloat16* pb = ((ops & DES_OP_DENSE1) && t->use_tc && !pp) ? t->pooled_b : nullptr;
#define PK5(GG, PP, HV, MT, BO) pool_kernel<GG, PP, HV, MT, BO><<<grid, 256, 0, cs>>>(                                 \
        b->offsets, b->vals, grow_csr, b->shards, nbags, B, t->F, t->k, t->W, (uint32_t)t->total_rows, pl, pp, pb)
#define PK3(GG, HV, MT, BO) do { if (wide) PK5(GG, 32 / GG, HV, MT, BO); else PK5(GG, 1, HV, MT, BO); } while (0)
#define PK2(GG, HV) do { if (pp) PK3(GG, HV, true, false); else if (pb) PK3(GG, HV, false, true); else PK3(GG, HV, false, false); } while (0)
#define PK(GG) do { if (b->vals) PK2(GG, true); else PK2(GG, false); } while (0)
    switch (G) { case 1: PK(1); break; case 2: PK(2); break; case 4: PK(4); break; case 8: PK(8); break; default: PK(16); }
#undef PK
#undef PK2
#undef PK3
#undef PK5
    DES_LAUNCH_CHECK(t, "pool_kernel");
    t->pooled_b_src = pb ? pl : nullptr;
  }
  return DES_OK;
}
extern "C" des_status_t des_forward_partials(des_table_t* t, uint32_t ops, const des_batch_t* b,
                                             const des_partials_t* part, void* stream) {
  return forward_impl(t, ops, b, part, nullptr, stream);
}

// the gather pass of the single-gather forms: pooled vectors (and their bfloat16 copy when the first layer
// follows) and per-bag sums of the linear weights and squared norms
static des_status_t launch_single_gather(des_table_t* t, uint32_t ops, const des_batch_t* b, float* pooled, cudaStream_t cs) {
  const int B = b->batch, G = group_for(t->k);
  const long long nbags = (long long)B * t->F;
  const bool wide = b->nnz >= 8 * nbags;
  const long long threads = nbags * (wide ? 32 : G);
  long long blocks = (threads + 255) / 256;
  if (blocks > (long long)t->sm_count * POOL_BLOCKS_PER_SM) blocks = (long long)t->sm_count * POOL_BLOCKS_PER_SM;
  const unsigned grid = (unsigned)blocks;
  __nv_bfloat16* pb = ((ops & DES_OP_DENSE1) && t->use_tc) ? t->pooled_b : nullptr;
#define SG3(GG, PP, HV) single_gather_kernel<GG, PP, HV><<<grid, 256, 0, cs>>>(b->offsets, b->vals, b->rows, b->shards, nbags,   \
                                                                              (int)t->S, t->k, t->W, t->meta,                 \
                                                                              (uint32_t)t->total_rows, pooled, t->bag_tail, pb)
#define SG2(GG, HV) do { if (wide) SG3(GG, 32 / GG, HV); else SG3(GG, 1, HV); } while (0)
#define SG(GG) do { if (b->vals) SG2(GG, true); else SG2(GG, false); } while (0)
  switch (G) { case 1: SG(1); break; case 2: SG(2); break; case 4: SG(4); break; case 8: SG(8); break; default: SG(16); }
#undef SG
#undef SG2
#undef SG3
  DES_LAUNCH_CHECK(t, "single_gather_kernel");
  t->pooled_b_src = pb ? pooled : nullptr;
  return DES_OK;
}

// des_forward_fused with pooling among the operators: one gather pass for everything.
static des_status_t forward_single_gather(des_table_t* t, uint32_t ops, const des_batch_t* b, float* pooled,
                                          float* out_small, cudaStream_t cs) {
  des_status_t st = launch_single_gather(t, ops, b, pooled, cs);
  if (st != DES_OK) return st;
  const int B = b->batch, G = group_for(t->k);
  const int grid = (int)(((long long)B * G + 255) / 256);
#define FF(GG) fused_finish_kernel<GG><<<grid, 256, 0, cs>>>(pooled, t->bag_tail, B, (int)t->F, t->k, ops, out_small)
  switch (G) { case 1: FF(1); break; case 2: FF(2); break; case 4: FF(4); break; case 8: FF(8); break; default: FF(16); }
#undef FF
  DES_LAUNCH_CHECK(t, "fused_finish_kernel");
  return DES_OK;
}

extern "C" des_status_t des_forward_fused(des_table_t* t, uint32_t ops, const des_batch_t* b,
                                          const des_partials_t* part, const des_outputs_t* out, void* stream) {
  if (!t || !part || !out || (ops & ~31u) || (ops & 15u) == 0) return DES_ERR_INVALID_ARG;
  const bool shard_order = ops & DES_FUSED_SHARD_ORDER;   // the shard-by-shard form even where one gather pass would do
  ops &= 15u;
  if ((ops & (DES_OP_LR | DES_OP_FM)) && !out->out_small) return DES_ERR_INVALID_ARG;
  if (part->part_pooled || part->part_dense) return DES_ERR_INVALID_ARG;      // materialised partials: use the two-call path
  const uint32_t rest = ops & ~(uint32_t)(DES_OP_LR | DES_OP_FM);
  des_status_t st;
  if ((ops & (DES_OP_LR | DES_OP_FM)) && rest && !part->part_small && !shard_order) {
    // LR / FM together with pooling and no request for the per-shard partials: one gather pass
    st = des_check_batch(t, b, 0);
    if (st != DES_OK) return st;
    if (!part->pooled || ((ops & DES_OP_DENSE1) && !t->H)) return DES_ERR_INVALID_ARG;
    des_api_begin(t, (cudaStream_t)stream);
    DES_DBG_ARM(t, (cudaStream_t)stream);
    st = forward_single_gather(t, ops, b, part->pooled, out->out_small, (cudaStream_t)stream);
  } else {
    st = forward_impl(t, ops, b, part, out->out_small, stream);
  }
  if (st != DES_OK) return st;
  // what is left of the aggregation: hand the pooled block over and run the first layer
  return rest ? des_aggregate(t, rest, b, part, out, stream) : DES_OK;
}

extern "C" des_status_t des_aggregate(des_table_t* t, uint32_t ops, const des_batch_t* b, const des_partials_t* part,
                                      const des_outputs_t* out, void* stream) {
  if (!t || !b || !part || !out || (ops & ~15u) || ops == 0) return DES_ERR_INVALID_ARG;
  if (b->batch <= 0 || b->batch > t->max_batch) return DES_ERR_INVALID_ARG;
  cudaStream_t cs = (cudaStream_t)stream;
  des_api_begin(t, cs);
  const int B = b->batch;
  if (ops & (DES_OP_LR | DES_OP_FM)) {
    if (!part->part_small || !out->out_small) return DES_ERR_INVALID_ARG;
    const int G = group_for(t->k);
    const long long threads = (long long)B * G;
    const int grid = (int)((threads + 255) / 256);
    switch (G) {
      case 1: aggregate_small_kernel<1><<<grid, 256, 0, cs>>>(part->part_small, B, t->S, t->k, ops, out->out_small); break;
      case 2: aggregate_small_kernel<2><<<grid, 256, 0, cs>>>(part->part_small, B, t->S, t->k, ops, out->out_small); break;
      case 4: aggregate_small_kernel<4><<<grid, 256, 0, cs>>>(part->part_small, B, t->S, t->k, ops, out->out_small); break;
      case 8: aggregate_small_kernel<8><<<grid, 256, 0, cs>>>(part->part_small, B, t->S, t->k, ops, out->out_small); break;
      default: aggregate_small_kernel<16><<<grid, 256, 0, cs>>>(part->part_small, B, t->S, t->k, ops, out->out_small); break;
    }
    DES_LAUNCH_CHECK(t, "aggregate_small_kernel");
  }
  if (ops & (DES_OP_POOL | DES_OP_DENSE1)) {
    if (!part->pooled || !out->pooled) return DES_ERR_INVALID_ARG;
    const size_t n = (size_t)B * t->F * t->k;
    if (part->part_pooled) {
      // materialised per-shard pooled partials: aggregate them in shard order
      reduce_shards_kernel<<<t->sm_count * 4, 256, 0, cs>>>(part->part_pooled, n, t->S, out->pooled);
      DES_LAUNCH_CHECK(t, "reduce_shards_kernel");
      t->pooled_b_src = nullptr;
    } else if (out->pooled != part->pooled) {
      DES_CUDA(cudaMemcpyAsync(out->pooled, part->pooled, n * 4, cudaMemcpyDeviceToDevice, cs));
    }
  }
  if (ops & DES_OP_DENSE1) {
    if (!t->H || !out->Z) return DES_ERR_INVALID_ARG;
    des_status_t st = des_dense1_forward(t, out->pooled, B, out->Z, part->part_dense, part->part_pooled, cs);
    if (st != DES_OK) return st;
    if (part->part_dense) {
      reduce_shards_kernel<<<t->sm_count * 4, 256, 0, cs>>>(part->part_dense, (size_t)B * t->H, t->S, out->Z);
      DES_LAUNCH_CHECK(t, "reduce_shards_kernel");
    }
  }
  return DES_OK;
}

// ---- two-level (+) for shards spread over several processes -------------------
extern "C" des_status_t des_rank_partial(des_table_t* t, int32_t batch, const float* d_part_small,
                                         float* d_rank_part, void* stream) {
  if (!t || !d_part_small || !d_rank_part || batch <= 0 || batch > t->max_batch) return DES_ERR_INVALID_ARG;
  cudaStream_t cs = (cudaStream_t)stream;
  des_api_begin(t, cs);
  reduce_shards_kernel<<<t->sm_count * 4, 256, 0, cs>>>(d_part_small, (size_t)batch * t->stride, t->S, d_rank_part);
  DES_LAUNCH_CHECK(t, "reduce_shards_kernel");
  return DES_OK;
}

extern "C" des_status_t des_aggregate_ranks(des_table_t* t, uint32_t ops, int32_t batch, int32_t world,
                                            const float* d_rank_parts, float* d_out_small, void* stream) {
  if (!t || !d_rank_parts || !d_out_small || batch <= 0 || batch > t->max_batch || world < 1 || (ops & ~15u) ||
      !(ops & (DES_OP_LR | DES_OP_FM)))
    return DES_ERR_INVALID_ARG;
  cudaStream_t cs = (cudaStream_t)stream;
  des_api_begin(t, cs);
  const int G = group_for(t->k);
  const int grid = (int)(((long long)batch * G + 255) / 256);
  switch (G) {   // the processes' messages are added like shards' partials: fixed (rank) order, then F
    case 1: aggregate_small_kernel<1><<<grid, 256, 0, cs>>>(d_rank_parts, batch, world, t->k, ops, d_out_small); break;
    case 2: aggregate_small_kernel<2><<<grid, 256, 0, cs>>>(d_rank_parts, batch, world, t->k, ops, d_out_small); break;
    case 4: aggregate_small_kernel<4><<<grid, 256, 0, cs>>>(d_rank_parts, batch, world, t->k, ops, d_out_small); break;
    case 8: aggregate_small_kernel<8><<<grid, 256, 0, cs>>>(d_rank_parts, batch, world, t->k, ops, d_out_small); break;
    default: aggregate_small_kernel<16><<<grid, 256, 0, cs>>>(d_rank_parts, batch, world, t->k, ops, d_out_small); break;
  }
  DES_LAUNCH_CHECK(t, "aggregate_small_kernel");
  return DES_OK;
}
