// DCN cross layer under DES (Section 4.4, the paragraph on DCN) and the
// transfer-volume formulas of Sections 4.1-4.3.
//
// Cross layer: w is split along its long dimension d into S contiguous slices;
// shard s forms the scalar p_s = <x[slice s], w[slice s]> per sample, (+) adds
// the scalars in shard order, and y = x0 * (+)p + b + x.  Both passes are plain
// streams over [B][d] rows: one warp per sample, 16-byte loads where d allows.
#include "des_internal.cuh"

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int d = 16; d > 0; d >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, d);
  return v;
}

// part[s][b] (optional), P[b], y[b][:].  Slice s = columns floor(s d / S) .. floor((s+1) d / S) - 1.
__global__ void __launch_bounds__(256) cross_forward_kernel(int B, int d, int S, const float* __restrict__ x0,
                                                            const float* __restrict__ x, const float* __restrict__ w,
                                                            const float* __restrict__ bias, float* __restrict__ part,
                                                            float* __restrict__ P, float* __restrict__ y) {
  const int lane = threadIdx.x & 31;
  const int b = blockIdx.x * 8 + (threadIdx.x >> 5);
  if (b >= B) return;
  const float* xr = x + (size_t)b * d;
  float tot = 0.f;
  for (int s = 0; s < S; ++s) {
    const int lo = (int)((long long)s * d / S), hi = (int)((long long)(s + 1) * d / S);
    float ps = 0.f;
    for (int i = lo + lane; i < hi; i += 32) ps = fmaf(__ldg(xr + i), __ldg(w + i), ps);
    ps = warp_sum(ps);
    if (part && lane == 0) part[(size_t)s * B + b] = ps;
    tot += ps;                                          // (+): shard order
  }
  if (lane == 0) P[b] = tot;
  const float* x0r = x0 + (size_t)b * d;
  float* yr = y + (size_t)b * d;
  for (int i = lane; i < d; i += 32) yr[i] = fmaf(__ldg(x0r + i), tot, __ldg(bias + i) + __ldg(xr + i));
}

// t[b] = <gY_b, x0_b>;  gx = gY + t w;  gx0 = gY P.
__global__ void __launch_bounds__(256) cross_backward_rows_kernel(int B, int d, const float* __restrict__ x0,
                                                                  const float* __restrict__ w,
                                                                  const float* __restrict__ P,
                                                                  const float* __restrict__ gY, float* __restrict__ gx0,
                                                                  float* __restrict__ gx, float* __restrict__ t_out) {
  const int lane = threadIdx.x & 31;
  const int b = blockIdx.x * 8 + (threadIdx.x >> 5);
  if (b >= B) return;
  const float* gr = gY + (size_t)b * d;
  const float* x0r = x0 + (size_t)b * d;
  float t = 0.f;
  for (int i = lane; i < d; i += 32) t = fmaf(__ldg(gr + i), __ldg(x0r + i), t);
  t = warp_sum(t);
  if (lane == 0) t_out[b] = t;
  const float p = __ldg(P + b);
  for (int i = lane; i < d; i += 32) {
    const float g = __ldg(gr + i);
    gx[(size_t)b * d + i] = fmaf(t, __ldg(w + i), g);
    gx0[(size_t)b * d + i] = g * p;
  }
}

// Column sums over a chunk of the batch: pw[c][i] = sum_b t_b x[b][i], pb[c][i] = sum_b gY[b][i].
#define CROSS_CHUNKS 64
__global__ void __launch_bounds__(128) cross_backward_cols_kernel(int B, int d, const float* __restrict__ x,
                                                                  const float* __restrict__ gY,
                                                                  const float* __restrict__ t, float* __restrict__ pw,
                                                                  float* __restrict__ pb) {
  const int i = blockIdx.x * 128 + threadIdx.x;
  const int c = blockIdx.y;
  const int per = (B + CROSS_CHUNKS - 1) / CROSS_CHUNKS;
  const int b_lo = c * per, b_hi = min(B, b_lo + per);
  if (i >= d) return;
  float aw = 0.f, ab = 0.f;
  for (int b = b_lo; b < b_hi; ++b) {
    aw = fmaf(__ldg(t + b), __ldg(x + (size_t)b * d + i), aw);
    ab += __ldg(gY + (size_t)b * d + i);
  }
  pw[(size_t)c * d + i] = aw;
  pb[(size_t)c * d + i] = ab;
}

// Chunks added in chunk order (deterministic).
__global__ void __launch_bounds__(256) cross_backward_finish_kernel(int d, const float* __restrict__ pw,
                                                                    const float* __restrict__ pb, float* __restrict__ gw,
                                                                    float* __restrict__ gb) {
  const int i = blockIdx.x * 256 + threadIdx.x;
  if (i >= d) return;
  float aw = 0.f, ab = 0.f;
  for (int c = 0; c < CROSS_CHUNKS; ++c) { aw += pw[(size_t)c * d + i]; ab += pb[(size_t)c * d + i]; }
  gw[i] = aw; gb[i] = ab;
}

extern "C" int64_t des_cross_workspace_floats(int32_t batch, int32_t dim) {
  if (batch <= 0 || dim <= 0) return 0;
  return (int64_t)batch + 2ll * CROSS_CHUNKS * dim;
}

extern "C" des_status_t des_cross_forward(int32_t batch, int32_t dim, int32_t num_shards, const float* d_x0,
                                          const float* d_x, const float* d_w, const float* d_b, float* d_part,
                                          float* d_P, float* d_y, void* stream) {
  if (batch <= 0 || dim <= 0 || num_shards <= 0 || num_shards > dim || !d_x0 || !d_x || !d_w || !d_b || !d_P || !d_y)
    return DES_ERR_INVALID_ARG;
  cross_forward_kernel<<<(batch + 7) / 8, 256, 0, (cudaStream_t)stream>>>(batch, dim, num_shards, d_x0, d_x, d_w, d_b,
                                                                         d_part, d_P, d_y);
  return cudaGetLastError() == cudaSuccess ? DES_OK : DES_ERR_CUDA;
}

extern "C" des_status_t des_cross_backward(int32_t batch, int32_t dim, const float* d_x0, const float* d_x,
                                           const float* d_w, const float* d_P, const float* d_gY, float* d_gx0,
                                           float* d_gx, float* d_gw, float* d_gb, float* d_ws, void* stream) {
  if (batch <= 0 || dim <= 0 || !d_x0 || !d_x || !d_w || !d_P || !d_gY || !d_gx0 || !d_gx || !d_gw || !d_gb || !d_ws)
    return DES_ERR_INVALID_ARG;
  cudaStream_t cs = (cudaStream_t)stream;
  float* t = d_ws;
  float* pw = d_ws + batch;
  float* pb = pw + (size_t)CROSS_CHUNKS * dim;
  cross_backward_rows_kernel<<<(batch + 7) / 8, 256, 0, cs>>>(batch, dim, d_x0, d_w, d_P, d_gY, d_gx0, d_gx, t);
  cross_backward_cols_kernel<<<dim3((dim + 127) / 128, CROSS_CHUNKS), 128, 0, cs>>>(batch, dim, d_x, d_gY, t, pw, pb);
  cross_backward_finish_kernel<<<(dim + 255) / 256, 256, 0, cs>>>(dim, pw, pb, d_gw, d_gb);
  return cudaGetLastError() == cudaSuccess ? DES_OK : DES_ERR_CUDA;
}

// Bytes a worker moves per iteration under the mesh strategy and under DES, and the saving
// ratio 1 - Q_DES / Q_Mesh, for LR, FM order 2 and the DNN first layer (Sections 4.1-4.3).
extern "C" des_status_t des_comm_volume(const des_comm_model_t* m, des_comm_volume_t* out) {
  if (!m || !out || m->workers < 2 || m->batch <= 0 || m->uniq <= 0 || m->emb_dim <= 0 || m->hidden < 0 ||
      m->key_bytes <= 0 || m->value_bytes <= 0 || m->first_layer_bytes < 0)
    return DES_ERR_INVALID_ARG;
  const double frac = (double)(m->workers - 1) / (double)m->workers;     // share held by the other workers
  const double keys = (double)m->key_bytes * (double)m->uniq;            // S_f
  const double vb = (double)m->value_bytes;
  const double weights[3] = {vb * (double)m->uniq,                                       // S_w
                             vb * (double)m->emb_dim * (double)m->uniq,                  // S_V
                             vb * (double)m->emb_dim * (double)m->uniq + m->first_layer_bytes};  // S_V + S_W
  const double partials[3] = {vb * (double)m->batch,                                     // M_1: a scalar per sample
                              vb * (double)m->batch * ((double)m->emb_dim + 1.0),        // M_1 (k-vector) + M_2
                              vb * (double)m->batch * (double)m->hidden};                // M_1 = V_i^T W_i
  for (int i = 0; i < 3; ++i) {
    out->q_mesh[i] = frac * (keys + weights[i]);
    out->q_des[i] = 2.0 * frac * partials[i];
    out->saving[i] = 1.0 - out->q_des[i] / out->q_mesh[i];
  }
  return DES_OK;
}
