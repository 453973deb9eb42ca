// Row-split first dense layer (Section 4.3): V^T W = sum_s V_s^T W_s, where
// V_s are the pooled blocks of the fields shard s owns and W_s the matching
// rows of W1 (Eq. 9); its backward needs no cross-shard term (Section 3.2):
// gE = gZ W1^T block by block, gW1 = V^T gZ.
//
// Operands are rounded to bfloat16 (RNE) and accumulated in fp32.  The K loop
// of the forward runs over fields in (owning shard, field) order, so the
// accumulator sees P_0, P_1, ... in shard order; with `part_dense` the K range
// of every shard is a separate slice of the launch and P_s is stored.
//
// Fast path: the three GEMMs (Z = V W, gE = gZ W1^T, gW1 = V^T gZ) run on the
// tcgen05 tensor cores (des_tc_gemm*.cu: bf16 operands by TMA, fp32 accumulators
// in tensor memory) after a float -> bf16 pass over V and gZ.  The kernel in
// this file is the plain shared-memory tiled CUDA-core version (64x64x16 tiles,
// 4x4 outputs per thread): it serves the materialised per-shard partials P_s
// (slices of the K range) and shapes the TMA path cannot take (a K or N extent
// that is not a multiple of 8).
#include "des_internal.cuh"
#define DES_TC_GEMM_DECL_ONLY
#include "des_tc_gemm.cuh"

#define TM 64
#define TN 64
#define TK 16

enum { GEMM_FWD = 0, GEMM_DGRAD = 1, GEMM_WGRAD = 2 };

struct GemmArgs {
  int M, N, K;                 // problem
  const float* A32;            // fwd: pooled [B][FK]   dgrad: gZ [B][H]    wgrad: pooled [B][FK]
  const __nv_bfloat16* Bb;     // fwd/dgrad: W1 bf16 [FK][H]
  const float* B32;            // wgrad: gZ [B][H]
  const float* add;            // dgrad: gE [B][FK] or NULL
  float* out;                  // [slices][M][N]
  int k_emb, FK, H;
  const DevMeta* meta;
  int slices;                  // grid.z
  int slice_by_shard;          // fwd: slice z = K range of shard z (FIELD) / all K of part_pooled[z] (HASH)
  int partition, S, F;
  size_t a_slice_stride;       // fwd + HASH materialise: part_pooled slice stride
};

__device__ __forceinline__ float bf16r(float x) { return __bfloat162float(__float2bfloat16_rn(x)); }

template <int MODE>
__global__ void __launch_bounds__(256) gemm_kernel(GemmArgs g) {
  __shared__ float As[TK][TM + 4];
  __shared__ float Bs[TK][TN + 4];
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  const int m0 = blockIdx.y * TM, n0 = blockIdx.x * TN, z = blockIdx.z;
  int k_lo = 0, k_hi = g.K;
  const float* A32 = g.A32;
  if (MODE == GEMM_FWD && g.slice_by_shard) {
    if (g.partition == DES_PART_FIELD) {
      // fields are K-ordered by owning shard: shard z owns a contiguous K range
      int before = 0, mine = 0;
      for (int f = 0; f < g.F; ++f) { int s = f % g.S; if (s < z) ++before; else if (s == z) ++mine; }
      k_lo = before * g.k_emb; k_hi = k_lo + mine * g.k_emb;
    } else {
      A32 += (size_t)z * g.a_slice_stride;
    }
  } else if (MODE == GEMM_WGRAD) {
    const int per = (g.K + g.slices - 1) / g.slices;
    k_lo = z * per; k_hi = min(g.K, k_lo + per);
  }
  float acc[4][4] = {};
  for (int kb = k_lo; kb < k_hi; kb += TK) {
    // stage A tile [TM][TK] and B tile [TK][TN], 4 elements per thread each
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const int idx = threadIdx.x + e * 256;
      float av = 0.f, bv = 0.f;
      if (MODE == GEMM_FWD) {
        const int kk = kb + (idx & 15), m = m0 + (idx >> 4);
        if (kk < k_hi && m < g.M) {
          const int col = g.meta->field_order[kk / g.k_emb] * g.k_emb + kk % g.k_emb;
          av = bf16r(__ldg(A32 + (size_t)m * g.FK + col));
        }
        As[idx & 15][idx >> 4] = av;
        const int kk2 = kb + (idx >> 6), n = n0 + (idx & 63);
        if (kk2 < k_hi && n < g.N) {
          const int row = g.meta->field_order[kk2 / g.k_emb] * g.k_emb + kk2 % g.k_emb;
          bv = __bfloat162float(g.Bb[(size_t)row * g.H + n]);
        }
        Bs[idx >> 6][idx & 63] = bv;
      } else if (MODE == GEMM_DGRAD) {
        const int kk = kb + (idx & 15), m = m0 + (idx >> 4);
        if (kk < k_hi && m < g.M) av = __ldg(A32 + (size_t)m * g.H + kk);
        As[idx & 15][idx >> 4] = av;
        const int kk2 = kb + (idx & 15), n = n0 + (idx >> 4);       // W1^T: read along H
        if (kk2 < k_hi && n < g.N) bv = __bfloat162float(g.Bb[(size_t)n * g.H + kk2]);
        Bs[idx & 15][idx >> 4] = bv;
      } else {
        const int kk = kb + (idx >> 6), m = m0 + (idx & 63);        // pooled^T: read along FK
        if (kk < k_hi && m < g.M) av = bf16r(__ldg(A32 + (size_t)kk * g.FK + m));
        As[idx >> 6][idx & 63] = av;
        const int kk2 = kb + (idx >> 6), n = n0 + (idx & 63);
        if (kk2 < k_hi && n < g.N) bv = __ldg(g.B32 + (size_t)kk2 * g.H + n);
        Bs[idx >> 6][idx & 63] = bv;
      }
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < TK; ++kk) {
      float a[4], b[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) { a[i] = As[kk][ty * 4 + i]; b[i] = Bs[kk][tx * 4 + i]; }
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
    }
    __syncthreads();
  }
  float* out = g.out + (size_t)z * g.M * g.N;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int m = m0 + ty * 4 + i;
    if (m >= g.M) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int n = n0 + tx * 4 + j;
      if (n >= g.N) continue;
      float v = acc[i][j];
      if (MODE == GEMM_DGRAD && g.add) v += __ldg(g.add + (size_t)m * g.N + n);
      out[(size_t)m * g.N + n] = v;
    }
  }
}

// Sum the split-K slices of gW1 in slice order, apply the optimizer to the
// fp32 master weights, refresh the bf16 shadow.
__global__ void w1_update_kernel(const float* __restrict__ part, int slices, size_t n, float* W1, float* acc,
                                 float* acc2, __nv_bfloat16* W1b, const OptParams opt_in,
                                 const DevMeta* __restrict__ meta) {
  const OptParams opt = des_opt_load(opt_in, meta);
  size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x, st = (size_t)gridDim.x * blockDim.x;
  for (; i < n; i += st) {
    float G = 0.f;
    for (int z = 0; z < slices; ++z) G += __ldg(part + (size_t)z * n + i);
    float w = W1[i];
    float s1 = acc[i], s2 = acc2 ? acc2[i] : 0.f;
    des_opt_step(opt, w, s1, s2, G);
    acc[i] = s1;
    if (acc2) acc2[i] = s2;
    W1[i] = w;
    W1b[i] = __float2bfloat16_rn(w);
  }
}

__global__ void cvt_bf16_kernel(const float* __restrict__ src, __nv_bfloat16* __restrict__ dst, size_t n) {
  size_t i = ((size_t)blockIdx.x * blockDim.x + threadIdx.x) * 4, st = (size_t)gridDim.x * blockDim.x * 4;
  for (; i + 3 < n; i += st) {
    const float4 v = *reinterpret_cast<const float4*>(src + i);
    __nv_bfloat162 a = __floats2bfloat162_rn(v.x, v.y), b = __floats2bfloat162_rn(v.z, v.w);
    *reinterpret_cast<uint2*>(dst + i) = make_uint2(*reinterpret_cast<uint32_t*>(&a), *reinterpret_cast<uint32_t*>(&b));
  }
}

// two arrays in one launch (the backward's two operands)
__global__ void cvt_bf16_pair_kernel(const float* __restrict__ s1, __nv_bfloat16* __restrict__ d1, size_t n1,
                                     const float* __restrict__ s2, __nv_bfloat16* __restrict__ d2, size_t n2) {
  size_t i = ((size_t)blockIdx.x * blockDim.x + threadIdx.x) * 4;
  const size_t st = (size_t)gridDim.x * blockDim.x * 4;
  for (; i + 3 < n1 + n2; i += st) {                   // n1 and n2 are multiples of 4
    const float* src = i < n1 ? s1 + i : s2 + (i - n1);
    __nv_bfloat16* dst = i < n1 ? d1 + i : d2 + (i - n1);
    const float4 v = *reinterpret_cast<const float4*>(src);
    __nv_bfloat162 a = __floats2bfloat162_rn(v.x, v.y), b = __floats2bfloat162_rn(v.z, v.w);
    *reinterpret_cast<uint2*>(dst) = make_uint2(*reinterpret_cast<uint32_t*>(&a), *reinterpret_cast<uint32_t*>(&b));
  }
}

static des_status_t to_bf16(des_table* t, const float* src, __nv_bfloat16* dst, size_t n, cudaStream_t st) {
  cvt_bf16_kernel<<<t->sm_count * 4, 256, 0, st>>>(src, dst, n);     // n is a multiple of 4 (k and H are)
  DES_LAUNCH_CHECK(t, "cvt_bf16_kernel");
  return DES_OK;
}

des_status_t des_dense1_forward(des_table* t, const float* pooled, int B, float* Z, float* part_dense,
                                const float* part_pooled, cudaStream_t st) {
  if (!part_dense && t->use_tc) {
    const int FK = t->F * t->k;
    // the pooling kernel of the same forward has usually left the bfloat16 copy already
    const bool have = t->pooled_b_src == pooled;
    t->pooled_b_src = nullptr;                         // good for one product only
    if (!have) {
      des_status_t e = to_bf16(t, pooled, t->pooled_b, (size_t)B * FK, st);
      if (e != DES_OK) return e;
    }
    const int rc = des_tc_gemm_fwd(B, t->H, FK, 1, t->pooled_b, t->W1b, Z, Z, 0.f, t->gemm_ws, t->gemm_ws_bytes, st);
    if (rc == 0) { DES_LAUNCH_CHECK(t, "tc_gemm_fwd"); return DES_OK; }
    if (rc != 1) return DES_ERR_CUDA;
  }
  GemmArgs g; memset(&g, 0, sizeof(g));
  g.M = B; g.N = t->H; g.K = t->F * t->k; g.A32 = pooled; g.Bb = t->W1b; g.k_emb = t->k; g.FK = g.K; g.H = t->H;
  g.meta = t->meta; g.partition = t->cfg.partition; g.S = t->S; g.F = t->F;
  g.out = Z; g.slices = 1; g.slice_by_shard = 0;
  if (part_dense) {
    if (t->cfg.partition == DES_PART_HASH && !part_pooled) return DES_ERR_INVALID_ARG;
    g.out = part_dense; g.slices = t->S; g.slice_by_shard = 1;
    if (t->cfg.partition == DES_PART_HASH) { g.A32 = part_pooled; g.a_slice_stride = (size_t)B * g.FK; }
  }
  dim3 grid((g.N + TN - 1) / TN, (g.M + TM - 1) / TM, g.slices);
  gemm_kernel<GEMM_FWD><<<grid, 256, 0, st>>>(g);
  DES_LAUNCH_CHECK(t, "gemm_kernel");
  return DES_OK;
}

des_status_t des_dense1_backward(des_table* t, const float* pooled, const float* gE, const float* gZ,
                                 float* gE_work, int B, cudaStream_t st) {
  const int FK = t->F * t->k;
  if (t->use_tc) {
    t->pooled_b_src = nullptr;
    cvt_bf16_pair_kernel<<<t->sm_count * 4, 256, 0, st>>>(gZ, t->gZ_b, (size_t)B * t->H, pooled, t->pooled_b, (size_t)B * FK);
    DES_LAUNCH_CHECK(t, "cvt_bf16_kernel");
    const int rc1 = des_tc_gemm_dgrad(B, FK, t->H, 1, t->gZ_b, t->W1b, gE ? gE : gE_work, gE_work, gE ? 1.f : 0.f,
                                      t->gemm_ws, t->gemm_ws_bytes, st);
    if (rc1 == 0) {
      DES_LAUNCH_CHECK(t, "tc_gemm_dgrad");
      // The product has few output tiles (F*k x H) and a long contraction (the batch): cut the batch into L
      // pieces so that every SM gets tiles (L partial products, added in piece order by w1_update_kernel).
      const int tiles = ((FK + 127) / 128) * ((t->H + 127) / 128);
      int L = 1;
      while (L < t->gw1_splits && tiles * L < 2 * t->sm_count && B % (2 * L * 64) == 0) L *= 2;
      const int rc2 = des_tc_gemm_wgrad(FK, t->H, B / L, L, t->pooled_b, t->gZ_b, t->gW1_part, t->gW1_part, 0.f,
                                        t->gemm_ws, t->gemm_ws_bytes, st);
      if (rc2 != 0) return DES_ERR_CUDA;           // same alignment rules as the dgrad: cannot differ
      DES_LAUNCH_CHECK(t, "tc_gemm_wgrad");
      w1_update_kernel<<<t->sm_count * 2, 256, 0, st>>>(t->gW1_part, L, (size_t)FK * t->H, t->W1, t->accW1, t->acc2W1,
                                                        t->W1b, des_opt_params(t), t->meta);
      DES_LAUNCH_CHECK(t, "w1_update_kernel");
      return DES_OK;
    }
    if (rc1 != 1) return DES_ERR_CUDA;
  }
  {  // gE_work = gE + gZ W1^T
    GemmArgs g; memset(&g, 0, sizeof(g));
    g.M = B; g.N = FK; g.K = t->H; g.A32 = gZ; g.Bb = t->W1b; g.add = gE; g.out = gE_work;
    g.k_emb = t->k; g.FK = FK; g.H = t->H; g.meta = t->meta; g.slices = 1;
    dim3 grid((g.N + TN - 1) / TN, (g.M + TM - 1) / TM, 1);
    gemm_kernel<GEMM_DGRAD><<<grid, 256, 0, st>>>(g);
    DES_LAUNCH_CHECK(t, "gemm_kernel");
  }
  {  // gW1 = pooled^T gZ, split over the batch
    GemmArgs g; memset(&g, 0, sizeof(g));
    g.M = FK; g.N = t->H; g.K = B; g.A32 = pooled; g.B32 = gZ; g.out = t->gW1_part;
    g.k_emb = t->k; g.FK = FK; g.H = t->H; g.meta = t->meta; g.slices = t->gw1_splits;
    dim3 grid((g.N + TN - 1) / TN, (g.M + TM - 1) / TM, g.slices);
    gemm_kernel<GEMM_WGRAD><<<grid, 256, 0, st>>>(g);
    DES_LAUNCH_CHECK(t, "gemm_kernel");
    const size_t n = (size_t)FK * t->H;
    w1_update_kernel<<<t->sm_count * 2, 256, 0, st>>>(t->gW1_part, g.slices, n, t->W1, t->accW1, t->acc2W1,
                                                      t->W1b, des_opt_params(t), t->meta);
    DES_LAUNCH_CHECK(t, "w1_update_kernel");
  }
  return DES_OK;
}

// ---- no-allocation variant of the row-split forward ---------------------------
// The per-shard partial products live in this file-scope array.  In host code
// the symbol below is only a handle: its device address is obtained once per
// device with cudaGetSymbolAddress and that pointer is what the kernels get.
static __device__ __align__(256) float g_noalloc_partials[DES_NOALLOC_SCRATCH_FLOATS];
static float* g_noalloc_ptr[64];   // per device ordinal, filled on first use

__global__ void noalloc_reduce_kernel(const float* __restrict__ part, size_t per_shard, int S, float* __restrict__ out) {
  size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x, st = (size_t)gridDim.x * blockDim.x;
  for (; i < per_shard; i += st) {
    float a = 0.f;
    for (int s = 0; s < S; ++s) a += part[(size_t)s * per_shard + i];
    out[i] = a;
  }
}

extern "C" des_status_t des_dense1_forward_noalloc(des_table_t* t, const float* d_pooled, int32_t batch, float* d_Z,
                                                   void* stream) {
  if (!t || !d_pooled || !d_Z || batch <= 0 || !t->H) return DES_ERR_INVALID_ARG;
  if (t->cfg.partition != DES_PART_FIELD) return DES_ERR_UNSUPPORTED;
  const size_t need = (size_t)t->S * (size_t)batch * t->H;
  if (need > (size_t)DES_NOALLOC_SCRATCH_FLOATS) return DES_ERR_TOO_LARGE;
  int dev = 0;
  DES_CUDA(cudaGetDevice(&dev));
  if (dev < 0 || dev >= 64) return DES_ERR_UNSUPPORTED;
  // the scratch array is this device's copy; the table's weights must live on the same device
  if (dev != t->device) return DES_ERR_INVALID_ARG;
  // (two host threads making the first call on a device at the same time both store the same address:
  // the unlocked write below is benign)
  if (!g_noalloc_ptr[dev]) {          // set-up, once per device, with that device current
    float* p = nullptr;
    if (cudaGetSymbolAddress((void**)&p, g_noalloc_partials) != cudaSuccess || !p) { cudaGetLastError(); return DES_ERR_CUDA; }
    g_noalloc_ptr[dev] = p;
  }
  float* part = g_noalloc_ptr[dev];
  cudaStream_t cs = (cudaStream_t)stream;
  des_api_begin(t, cs);
  GemmArgs g; memset(&g, 0, sizeof(g));
  g.M = batch; g.N = t->H; g.K = t->F * t->k; g.A32 = d_pooled; g.Bb = t->W1b; g.k_emb = t->k; g.FK = g.K; g.H = t->H;
  g.meta = t->meta; g.partition = t->cfg.partition; g.S = t->S; g.F = t->F;
  g.out = part; g.slices = t->S; g.slice_by_shard = 1;     // every element of every slice is written
  dim3 grid((g.N + TN - 1) / TN, (g.M + TM - 1) / TM, g.slices);
  gemm_kernel<GEMM_FWD><<<grid, 256, 0, cs>>>(g);
  DES_LAUNCH_CHECK(t, "gemm_kernel");
  noalloc_reduce_kernel<<<t->sm_count * 4, 256, 0, cs>>>(part, (size_t)batch * t->H, t->S, d_Z);
  DES_LAUNCH_CHECK(t, "noalloc_reduce_kernel");
  return DES_OK;
}
