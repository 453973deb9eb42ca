// Forward of the DES sparse operators.
//
// des_forward_partials: the sub-operators M_j of every shard —
//   LR   M_1 = sum_{j in shard} w_j x_j                       (Eq. 2)
//   FM   M_1 = sum v_j x_j,  M_2 = sum <v_j x_j, v_j x_j>      (Eq. 7)
//   POOL per-field sum pooling of the latent vectors          (Section 4.3)
// des_aggregate: (+) over shards in the order s = 0..S-1 (Eq. 1) and the
// substitution operator F = 1/2 <(+)M_1,(+)M_1> - 1/2 (+)M_2 (Eq. 8).
//
// Kernel shape.  One warp walks one sample, bag by bag.  A row (k floats + the
// linear weight) is read by a group of G = k/4 lanes (rounded up to a power of
// two) with one 16-byte load per lane; the NG = 32/G groups of the warp split
// the occurrences of a bag BY SHARD: group g takes the occurrences whose shard
// is congruent to g modulo NG.  The per-(shard, sample) partials live in shared
// memory, S x (k+4) floats per warp, and because a shard's accumulator row is
// only ever touched by its owning group, in occurrence order, there are no
// conflicts to resolve and the result is deterministic.  A bag's pooled sum is
// the sum of the groups' partial sums (a few shuffles per bag).  Each group
// keeps FW_UNROLL row loads in flight.  M_2 needs |v|^2 of every row: the table
// keeps it next to the linear weight in the row's 16-byte tail (refreshed by the
// update kernel), so the forward adds x^2 |v|^2 without a cross-lane reduction.
#include "des_internal.cuh"

#define FW_UNROLL 4

template <int G, bool HAS_VALS, bool MATERIALISE>
__global__ void __launch_bounds__(384) forward_partials_kernel(
    const int32_t* __restrict__ offsets, const float* __restrict__ vals, const uint32_t* __restrict__ rows,
    const uint8_t* __restrict__ shards, int B, int F, int S, int k, uint32_t ops, const float* __restrict__ W,
    const DevMeta* __restrict__ meta, float* __restrict__ part_small, float* __restrict__ pooled,
    float* __restrict__ part_pooled) {
  extern __shared__ __align__(16) float smem[];
  __shared__ uint32_t row_base[DES_MAX_SHARDS];
  constexpr int NG = 32 / G;
  const int K4 = k >> 2, stride = k + 4;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, wpb = blockDim.x >> 5;
  const int g = lane / G, c4 = lane % G;
  const bool col = c4 < K4, lead = c4 == 0;
  const bool want_small = part_small != nullptr;
  float* acc = smem + (size_t)warp * S * stride;
  const int acc_f4 = S * (K4 + 1);
  if (threadIdx.x < S) row_base[threadIdx.x] = (uint32_t)meta->row_base[threadIdx.x];
  if (want_small)
    for (int i = lane; i < acc_f4; i += 32) reinterpret_cast<float4*>(acc)[i] = make_float4(0.f, 0.f, 0.f, 0.f);
  __syncthreads();

  for (int b = blockIdx.x * wpb + warp; b < B; b += gridDim.x * wpb) {
    for (int f = 0; f < F; ++f) {
      const int lo = __ldg(offsets + (size_t)b * F + f), hi = __ldg(offsets + (size_t)b * F + f + 1);
      float4 pacc = make_float4(0.f, 0.f, 0.f, 0.f);
      for (int base = lo; base < hi; base += 32) {
        // every lane fetches one occurrence of the chunk; groups then pick their shards' entries
        const int j = base + lane;
        uint32_t my_grow = DES_ROW_NONE; int my_s = 0; float my_x = 1.f;
        if (j < hi) {
          const uint32_t r = __ldg(rows + j);
          my_s = __ldg(shards + j);
          if (r != DES_ROW_NONE) my_grow = row_base[my_s] + r;      // table-global row
          if (HAS_VALS) my_x = __ldg(vals + j);
        }
        const int key = (my_grow == DES_ROW_NONE) ? -1 : ((want_small ? my_s : lane) & (NG - 1));
        unsigned m = 0;
#pragma unroll
        for (int q = 0; q < NG; ++q) {
          const unsigned mq = __ballot_sync(0xFFFFFFFFu, key == q);
          if (q == g) m = mq;
        }
        while (__any_sync(0xFFFFFFFFu, m != 0)) {
          float4 v[FW_UNROLL], tl[FW_UNROLL]; float x[FW_UNROLL]; int sh[FW_UNROLL];
#pragma unroll
          for (int u = 0; u < FW_UNROLL; ++u) {
            const bool have = m != 0;
            const int src = have ? (__ffs(m) - 1) : 0;
            m &= m - 1;                                     // 0 stays 0
            const uint32_t gr = __shfl_sync(0xFFFFFFFFu, my_grow, src);
            const int s = __shfl_sync(0xFFFFFFFFu, my_s, src);
            x[u] = HAS_VALS ? __shfl_sync(0xFFFFFFFFu, my_x, src) : 1.f;
            sh[u] = have ? s : -1;
            v[u] = make_float4(0.f, 0.f, 0.f, 0.f); tl[u] = v[u];
            if (have) {
              const float4* wr = reinterpret_cast<const float4*>(W + (size_t)gr * stride);
              if (col) v[u] = __ldg(wr + c4);
              if (lead && want_small) tl[u] = __ldg(wr + K4);      // (linear weight, |v|^2, 0, 0)
            }
          }
#pragma unroll
          for (int u = 0; u < FW_UNROLL; ++u) {
            float4 vx = v[u];
            if (HAS_VALS) { vx.x *= x[u]; vx.y *= x[u]; vx.z *= x[u]; vx.w *= x[u]; }
            pacc.x += vx.x; pacc.y += vx.y; pacc.z += vx.z; pacc.w += vx.w;
            if (sh[u] >= 0) {
              if (MATERIALISE && col)
                atomicAdd(reinterpret_cast<float4*>(part_pooled + ((size_t)sh[u] * B + b) * ((size_t)F * k) +
                                                    (size_t)f * k) + c4, vx);
              if (want_small) {
                float* a = acc + sh[u] * stride;             // row owned by this group
                if (col) {
                  float4 t = reinterpret_cast<float4*>(a)[c4];
                  t.x += vx.x; t.y += vx.y; t.z += vx.z; t.w += vx.w;
                  reinterpret_cast<float4*>(a)[c4] = t;
                }
                if (lead) {
                  float2 t = *reinterpret_cast<float2*>(a + k);
                  t.x += tl[u].x * x[u]; t.y += tl[u].y * x[u] * x[u];
                  *reinterpret_cast<float2*>(a + k) = t;
                }
              }
            }
          }
        }
      }
      if (pooled) {
#pragma unroll
        for (int d = G; d < 32; d <<= 1) {
          pacc.x += __shfl_xor_sync(0xFFFFFFFFu, pacc.x, d); pacc.y += __shfl_xor_sync(0xFFFFFFFFu, pacc.y, d);
          pacc.z += __shfl_xor_sync(0xFFFFFFFFu, pacc.z, d); pacc.w += __shfl_xor_sync(0xFFFFFFFFu, pacc.w, d);
        }
        if (g == 0 && col) reinterpret_cast<float4*>(pooled + ((size_t)b * F + f) * k)[c4] = pacc;
      }
    }
    if (want_small) {
      __syncwarp();
      const bool lr = ops & DES_OP_LR, fm = ops & DES_OP_FM;
      for (int i = lane; i < acc_f4; i += 32) {
        const int s = i / (K4 + 1), q = i % (K4 + 1);
        float4 t = reinterpret_cast<float4*>(acc)[i];
        reinterpret_cast<float4*>(acc)[i] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (q == K4) { if (!lr) t.x = 0.f; if (!fm) t.y = 0.f; }
        else if (!fm) t = make_float4(0.f, 0.f, 0.f, 0.f);
        reinterpret_cast<float4*>(part_small + ((size_t)s * B + b) * stride)[q] = t;
      }
      __syncwarp();
    }
  }
}

// (+) over shards and F.  G lanes per sample, one float4 column each; lane 0 of
// the group also carries the tail (R_lr, Q).  <A, A> is taken in double.
template <int G>
__global__ void __launch_bounds__(256) aggregate_small_kernel(const float* __restrict__ part_small, int B, int S, int k,
                                                              uint32_t ops, float* __restrict__ out_small) {
  const int K4 = k >> 2, stride = k + 4;
  const int t = blockIdx.x * blockDim.x + threadIdx.x;
  const int b = t / G, c4 = t % G;
  const bool live = b < B;
  float4 a = make_float4(0.f, 0.f, 0.f, 0.f), tail = a;
  if (live) {
    for (int s = 0; s < S; ++s) {
      const float4* p = reinterpret_cast<const float4*>(part_small + ((size_t)s * B + b) * stride);
      if (c4 < K4) { float4 v = __ldg(p + c4); a.x += v.x; a.y += v.y; a.z += v.z; a.w += v.w; }
      if (c4 == 0) { float4 v = __ldg(p + K4); tail.x += v.x; tail.y += v.y; }
    }
  }
  double aa = (double)a.x * a.x + (double)a.y * a.y + (double)a.z * a.z + (double)a.w * a.w;
#pragma unroll
  for (int d = 1; d < G; d <<= 1) aa += __shfl_xor_sync(0xFFFFFFFFu, aa, d);
  if (!live) return;
  float4* o = reinterpret_cast<float4*>(out_small + (size_t)b * stride);
  if (c4 < K4) o[c4] = a;
  if (c4 == 0) {
    const float fm2 = (ops & DES_OP_FM) ? (float)(0.5 * aa - 0.5 * (double)tail.y) : 0.f;
    o[K4] = make_float4(tail.x, fm2, tail.y, 0.f);
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

extern "C" des_status_t des_forward_partials(des_table_t* t, uint32_t ops, const des_batch_t* b,
                                             const des_partials_t* part, void* stream) {
  des_status_t st = des_check_batch(t, b, 0);
  if (st != DES_OK) return st;
  if (!part || (ops & ~15u) || ops == 0) return DES_ERR_INVALID_ARG;
  const bool small = ops & (DES_OP_LR | DES_OP_FM), pool = ops & (DES_OP_POOL | DES_OP_DENSE1);
  if (small && !part->part_small) return DES_ERR_INVALID_ARG;
  if (pool && !part->pooled) return DES_ERR_INVALID_ARG;
  if ((ops & DES_OP_DENSE1) && !t->H) return DES_ERR_INVALID_ARG;
  cudaStream_t cs = (cudaStream_t)stream;
  des_api_begin(t, cs);
  const int B = b->batch;
  float* ps = small ? part->part_small : nullptr;
  float* pl = pool ? part->pooled : nullptr;
  float* pp = pool ? part->part_pooled : nullptr;
  if (pp) DES_CUDA(cudaMemsetAsync(pp, 0, (size_t)t->S * B * t->F * t->k * 4, cs));
  const size_t per_warp = small ? (size_t)t->S * t->stride * 4 : 0;
  int wpb = 12;
  while (wpb > 1 && per_warp * wpb > 208 * 1024) --wpb;
  const size_t smem = per_warp * wpb;
  int grid = (B + wpb - 1) / wpb;
  const int G = group_for(t->k);
#define FWD3(GG, HV, MT)                                                                                          \
  do {                                                                                                            \
    if (smem > 48 * 1024)                                                                                         \
      DES_CUDA(cudaFuncSetAttribute(forward_partials_kernel<GG, HV, MT>,                                          \
                                    cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));                     \
    forward_partials_kernel<GG, HV, MT><<<grid, wpb * 32, smem, cs>>>(                                            \
        b->offsets, b->vals, b->rows, b->shards, B, t->F, t->S, t->k, ops, t->W, t->meta, ps, pl, pp);            \
  } while (0)
#define FWD(GG)                                                                                                   \
  do {                                                                                                            \
    if (pp) { if (b->vals) FWD3(GG, true, true); else FWD3(GG, false, true); }                                    \
    else { if (b->vals) FWD3(GG, true, false); else FWD3(GG, false, false); }                                     \
  } while (0)
  switch (G) {
    case 1: FWD(1); break;
    case 2: FWD(2); break;
    case 4: FWD(4); break;
    case 8: FWD(8); break;
    default: FWD(16); break;
  }
#undef FWD3
#undef FWD
  DES_LAUNCH_CHECK(t, "forward_partials_kernel");
  return DES_OK;
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
