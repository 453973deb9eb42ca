// A fixed read-out that stands for the rest of the model — the layers above the first FC layer in Section
// 4.3 / Fig. 4, which the sparse path does not contain.  It turns the aggregated results of one forward into
// one logit per sample and the log loss into the upstream gradients des_backward_update consumes, so that
// multi-step runs and the closed-loop benchmark need no gradients from outside.  Nothing in it is trained.
//   logit = b0 + c_lr R_lr + c_fm fm2 + <u, relu(Z + b1)> + <q, pooled> + <d, xdense>
//   p = sigmoid(logit);  loss_b = -(y log p + (1 - y) log(1 - p));  g = (p - y) / B
//   gL = c_lr g;  gF = c_fm g;  gZ = g u [Z + b1 > 0];  gE = g q
// One warp per sample: the dot products are taken in double (lanes stride over the row, then a butterfly),
// the gradient rows are written with 16-byte stores.
#include "des_internal.cuh"

__global__ void __launch_bounds__(256) head_kernel(
    int B, int k, int H, int FK, int nd, uint32_t ops, float b0, float c_lr, float c_fm, const float* __restrict__ u,
    const float* __restrict__ b1, const float* __restrict__ q, const float* __restrict__ d,
    const float* __restrict__ out_small, const float* __restrict__ Z, const float* __restrict__ pooled,
    const float* __restrict__ xdense, const float* __restrict__ y, float* __restrict__ logit, float* __restrict__ loss,
    float* __restrict__ gL, float* __restrict__ gF, float* __restrict__ gZ, float* __restrict__ gE) {
  const int lane = threadIdx.x & 31;
  const int b = blockIdx.x * 8 + (threadIdx.x >> 5);
  if (b >= B) return;                                  // whole warp
  const int stride = k + 4;
  const bool use_z = (ops & DES_OP_DENSE1) && Z && u && b1;
  const bool use_p = (ops & DES_OP_POOL) && !(ops & DES_OP_DENSE1) && pooled && q;
  double acc = 0.0;
  if (use_z) {
    const float* z = Z + (size_t)b * H;
    for (int h = lane; h < H; h += 32) {
      const float a = z[h] + __ldg(b1 + h);
      if (a > 0.f) acc += (double)__ldg(u + h) * (double)a;
    }
  }
  if (use_p) {
    const float4* p4 = reinterpret_cast<const float4*>(pooled + (size_t)b * FK);
    const float4* q4 = reinterpret_cast<const float4*>(q);
    for (int i = lane; i < FK / 4; i += 32) {
      const float4 v = p4[i], w = __ldg(q4 + i);
      acc += (double)v.x * (double)w.x + (double)v.y * (double)w.y + (double)v.z * (double)w.z + (double)v.w * (double)w.w;
    }
  }
  if (d && xdense)
    for (int i = lane; i < nd; i += 32) acc += (double)__ldg(d + i) * (double)xdense[(size_t)b * nd + i];
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, o);
  double zl = (double)b0 + acc;
  if (ops & DES_OP_LR) zl += (double)c_lr * (double)out_small[(size_t)b * stride + k];
  if (ops & DES_OP_FM) zl += (double)c_fm * (double)out_small[(size_t)b * stride + k + 1];
  const double yy = (double)y[b];
  const double sp_neg = log1p(exp(-fabs(zl))) + (zl < 0.0 ? -zl : 0.0);   // -log p, without overflow
  const double p = 1.0 / (1.0 + exp(-zl));
  const float g = (float)((p - yy) / (double)B);
  if (lane == 0) {
    logit[b] = (float)zl;
    loss[b] = (float)(yy * sp_neg + (1.0 - yy) * (sp_neg + zl));
    if (gL) gL[b] = (ops & DES_OP_LR) ? c_lr * g : 0.f;
    if (gF) gF[b] = (ops & DES_OP_FM) ? c_fm * g : 0.f;
  }
  if (use_z && gZ) {
    const float* z = Z + (size_t)b * H;
    float* o = gZ + (size_t)b * H;
    for (int h = lane; h < H; h += 32) o[h] = (z[h] + __ldg(b1 + h) > 0.f) ? g * __ldg(u + h) : 0.f;
  }
  if (use_p && gE) {
    const float4* q4 = reinterpret_cast<const float4*>(q);
    float4* o = reinterpret_cast<float4*>(gE + (size_t)b * FK);
    for (int i = lane; i < FK / 4; i += 32) {
      const float4 w = __ldg(q4 + i);
      o[i] = make_float4(g * w.x, g * w.y, g * w.z, g * w.w);
    }
  }
}

extern "C" des_status_t des_head(des_table_t* t, uint32_t ops, int32_t batch, const des_head_t* head,
                                 const des_outputs_t* out, const float* d_xdense, const float* d_y, float* d_logit,
                                 float* d_loss, const des_head_grads_t* g, void* stream) {
  if (!t || !head || !out || !d_y || !d_logit || !d_loss || !g || (ops & ~15u) || ops == 0) return DES_ERR_INVALID_ARG;
  if (batch <= 0 || batch > t->max_batch) return DES_ERR_INVALID_ARG;
  if ((ops & (DES_OP_LR | DES_OP_FM)) && !out->out_small) return DES_ERR_INVALID_ARG;
  if ((ops & DES_OP_LR) && !g->gL) return DES_ERR_INVALID_ARG;
  if ((ops & DES_OP_FM) && !g->gF) return DES_ERR_INVALID_ARG;
  if ((ops & DES_OP_DENSE1) && (!t->H || !out->Z || !head->u || !head->b1 || !g->gZ)) return DES_ERR_INVALID_ARG;
  if ((ops & DES_OP_POOL) && !(ops & DES_OP_DENSE1) && (!out->pooled || !head->q || !g->gE)) return DES_ERR_INVALID_ARG;
  if (head->n_dense < 0 || (head->n_dense > 0 && head->d && !d_xdense)) return DES_ERR_INVALID_ARG;
  cudaStream_t cs = (cudaStream_t)stream;
  des_api_begin(t, cs);
  head_kernel<<<(batch + 7) / 8, 256, 0, cs>>>(batch, (int)t->k, (int)t->H, (int)(t->F * t->k), head->n_dense, ops, head->b0,
                                               head->c_lr, head->c_fm, head->u, head->b1, head->q,
                                               head->n_dense > 0 ? head->d : nullptr, out->out_small, out->Z, out->pooled,
                                               d_xdense, d_y, d_logit, d_loss, g->gL, g->gF, g->gZ, g->gE);
  DES_LAUNCH_CHECK(t, "head_kernel");
  return DES_OK;
}
