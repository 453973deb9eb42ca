// Table life cycle and inspection: allocation of slots / rows / state /
// workspace, status, size, export, row read-back (Section 5, "Dynamic Hash
// Table": the storage behind lookup / insert / update).
#include <new>
#include <math.h>
#include <string.h>

#include "des_internal.cuh"
#include <cstdlib>

static void* dalloc(const des_config_t& c, size_t bytes) {
  if (bytes == 0) bytes = 256;
  if (c.alloc) return c.alloc(bytes, c.alloc_ctx);
  void* p = nullptr;
  if (cudaMalloc(&p, bytes) != cudaSuccess) { cudaGetLastError(); return nullptr; }
  return p;
}
static void dfree(const des_config_t& c, void* p) {
  if (!p) return;
  if (c.dealloc) c.dealloc(p, c.alloc_ctx); else cudaFree(p);
}

__global__ void fill_f32_kernel(float* p, size_t n, float v) {
  size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x, st = (size_t)gridDim.x * blockDim.x;
  for (; i < n; i += st) p[i] = v;
}

OptParams des_opt_params(des_table* t) {
  OptParams o;
  const des_config_t& c = t->cfg;
  o.optimizer = (int)c.optimizer; o.lin_optimizer = (int)c.lin_optimizer;
  o.lr = c.lr; o.eps = c.eps; o.beta1 = c.beta1; o.beta2 = c.beta2;
  o.c1 = 1.f; o.c2 = 1.f;
  o.ftrl_alpha = c.ftrl_alpha; o.ftrl_beta = c.ftrl_beta; o.ftrl_l1 = c.ftrl_l1; o.ftrl_l2 = c.ftrl_l2;
  return o;
}

int des_prof_mark(des_table* t, const char* name, int check) {
  if (name) t->launches++;
  if (check && cudaGetLastError() != cudaSuccess) return 1;
  if (t->prof_on && t->prof_n < DES_PROF_MAX) {
    t->prof_name[t->prof_n] = name;
    cudaEventRecord(t->prof_ev[t->prof_n], t->cur_stream);
    t->prof_n++;
  }
  return 0;
}

void des_api_begin(des_table* t, cudaStream_t cs) {
  t->cur_stream = cs;
  if (t->prof_on) des_prof_mark(t, nullptr, 0);
}

extern "C" des_status_t des_profile_enable(des_table_t* t, int on) {
  if (!t) return DES_ERR_INVALID_ARG;
  if (on && !t->prof_ev) {
    t->prof_ev = new (std::nothrow) cudaEvent_t[DES_PROF_MAX];
    t->prof_name = new (std::nothrow) const char*[DES_PROF_MAX];
    if (!t->prof_ev || !t->prof_name) return DES_ERR_CUDA;
    for (int i = 0; i < DES_PROF_MAX; ++i) DES_CUDA(cudaEventCreate(&t->prof_ev[i]));
  }
  t->prof_on = on ? 1 : 0;
  t->prof_n = 0;
  return DES_OK;
}

extern "C" des_status_t des_profile_read(des_table_t* t, const char** h_names, float* h_ms, int cap, int* h_n) {
  if (!t || !h_n || !t->prof_ev) return DES_ERR_INVALID_ARG;
  DES_CUDA(cudaDeviceSynchronize());
  int n = 0;
  for (int i = 1; i < t->prof_n; ++i) {
    if (!t->prof_name[i]) continue;
    float ms = 0.f;
    DES_CUDA(cudaEventElapsedTime(&ms, t->prof_ev[i - 1], t->prof_ev[i]));
    if (n < cap) { if (h_names) h_names[n] = t->prof_name[i]; if (h_ms) h_ms[n] = ms; }
    ++n;
  }
  *h_n = n;
  t->prof_n = 0;
  return DES_OK;
}

extern "C" const char* des_status_string(des_status_t s) {
  switch (s) {
    case DES_OK: return "ok";
    case DES_ERR_INVALID_ARG: return "invalid argument";
    case DES_ERR_RESERVED_KEY: return "reserved key (all ones) in the batch";
    case DES_ERR_CAPACITY: return "a shard is out of slots or rows";
    case DES_ERR_UNSUPPORTED: return "unsupported";
    case DES_ERR_CUDA: return "CUDA runtime error or no device";
    case DES_ERR_NOT_FOUND: return "not found";
    case DES_ERR_TOO_LARGE: return "problem exceeds the fixed scratch of the no-allocation entry point";
    case DES_ERR_RANGE: return "checking build: an index outside the table's bounds was met and skipped";
  }
  return "?";
}

extern "C" des_status_t des_table_destroy(des_table_t* t) {
  if (!t) return DES_OK;
  int caller_dev = -1;                                   // the caller's current device is put back at the end
  if (cudaGetDevice(&caller_dev) != cudaSuccess) { cudaGetLastError(); caller_dev = -1; }
  cudaSetDevice(t->device);
  cudaDeviceSynchronize();
  void* ptrs[] = {t->slots, t->W, t->A, t->A2, t->acc2W1, t->meta, t->slot_of, t->flags, t->uslot, t->blk_cnt, t->seg_off, t->Gbuf, t->hinfo, t->dest, t->hot_base,
                  t->hot_R, t->hot_u, t->hot_ctr, t->hot_work, t->hot_acc, t->super_cnt, t->x_sorted, t->bag_tail,
                  t->W1, t->accW1, t->W1b, t->gW1_part, t->pooled_b, t->gZ_b, t->gemm_ws, t->st_offsets[0], t->st_ids[0], t->st_vals[0], t->st_offsets[1], t->st_ids[1], t->st_vals[1], t->st_rows,
                  t->st_shards, t->st_uidx, t->st_uniq_rows, t->st_n_uniq, t->st_part_small, t->st_out_small};
  for (void* p : ptrs) dfree(t->cfg, p);
  if (t->st_copy_stream) {
    cudaStreamDestroy(t->st_copy_stream);
    for (int s = 0; s < 2; ++s) { if (t->st_copied[s]) cudaEventDestroy(t->st_copied[s]); if (t->st_done[s]) cudaEventDestroy(t->st_done[s]); }
  }
  if (t->prof_ev) { for (int i = 0; i < DES_PROF_MAX; ++i) cudaEventDestroy(t->prof_ev[i]); delete[] t->prof_ev; }
  delete[] t->prof_name;
  const int own_dev = t->device;
  delete t;
  if (caller_dev >= 0 && caller_dev != own_dev) cudaSetDevice(caller_dev);
  return DES_OK;
}

extern "C" des_status_t des_table_create(const des_config_t* cfg, des_table_t** out) {
  if (!out) return DES_ERR_INVALID_ARG;
  *out = nullptr;
  if (!cfg) return DES_ERR_INVALID_ARG;
  const des_config_t& c = *cfg;
  if (c.num_shards < 1 || c.num_shards > DES_MAX_SHARDS || c.num_fields < 1 || c.num_fields > 1024 ||
      c.emb_dim < 4 || c.emb_dim > 64 || (c.emb_dim & 3) || (c.hidden & 3) || c.partition > DES_PART_FIELD ||
      c.optimizer > DES_OPT_ADAM || c.lin_optimizer > DES_LIN_FTRL || c.max_rows == 0 || !(c.max_load > 0.f && c.max_load <= 0.9f) ||
      c.max_nnz <= 0 || c.max_nnz >= (1ll << 31) || c.max_batch <= 0 || c.max_uniq < 0 ||
      (int64_t)c.max_batch * c.num_fields >= (1ll << 31))
    return DES_ERR_INVALID_ARG;
  if ((c.alloc == nullptr) != (c.dealloc == nullptr)) return DES_ERR_INVALID_ARG;
  if (c.shard_world > 1 && c.shard_rank >= c.shard_world) return DES_ERR_INVALID_ARG;
  if (c.shard_world <= 1 && c.shard_rank != 0) return DES_ERR_INVALID_ARG;
  if (c.optimizer == DES_OPT_ADAM && !(c.beta1 >= 0.f && c.beta1 < 1.f && c.beta2 >= 0.f && c.beta2 < 1.f))
    return DES_ERR_INVALID_ARG;
  if (c.lin_optimizer == DES_LIN_FTRL && !(c.ftrl_alpha > 0.f && c.ftrl_beta >= 0.f && c.ftrl_l1 >= 0.f && c.ftrl_l2 >= 0.f))
    return DES_ERR_INVALID_ARG;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return DES_ERR_CUDA; }
  des_table* t = new (std::nothrow) des_table();
  if (!t) return DES_ERR_CUDA;
  memset(t, 0, sizeof(*t));
  t->cfg = c; t->cfg.h_rows_per_shard = nullptr; t->device = dev;
  t->S = c.num_shards; t->F = c.num_fields; t->k = c.emb_dim; t->H = c.hidden; t->stride = c.emb_dim + 4;
  t->max_nnz = c.max_nnz; t->max_batch = c.max_batch; t->max_uniq = c.max_uniq ? c.max_uniq : c.max_nnz;
  if (t->max_uniq > t->max_nnz) t->max_uniq = t->max_nnz;
  cudaDeviceGetAttribute(&t->sm_count, cudaDevAttrMultiProcessorCount, dev);
  DevMeta hm; memset(&hm, 0, sizeof(hm));
  hm.scratch_base = 0xFFFFFFFFu;                      // top of the insert calls' scratch range (Slot::first_occ)
#ifdef DES_DEBUG
  if (const char* e = getenv("DES_DEBUG_SCRATCH_BASE")) {   // checking build only — tests start near the end of the
    const unsigned long long v = strtoull(e, nullptr, 0);   // range, so that the rare reset pass runs within a few calls
    if (v >= (unsigned long long)t->max_nnz && v <= 0xFFFFFFFFull) hm.scratch_base = (uint32_t)v;
  }
#endif
  uint64_t rows = 0, slots = 0;
  const uint32_t world = c.shard_world > 1 ? c.shard_world : 1;
  uint32_t owned = 0;
  for (uint32_t s = 0; s < t->S; ++s) owned += (s % world == c.shard_rank);
  for (uint32_t s = 0; s < t->S; ++s) {
    uint64_t cap = c.h_rows_per_shard ? c.h_rows_per_shard[s]
                                      : (uint64_t)((double)(c.max_rows / (owned ? owned : 1)) * 1.05) + 1024;
    if (s % world != c.shard_rank) cap = 0;            // another process holds this shard
    if (cap == 0) cap = 1;
    uint64_t ns = (uint64_t)((double)cap / (double)c.max_load) + 1;
    if (cap >= 0xFFFFFFF0ull) { delete t; return DES_ERR_INVALID_ARG; }
    t->h_row_base[s] = rows; t->h_slot_base[s] = slots;
    hm.row_base[s] = rows; hm.slot_base[s] = slots; hm.row_cap[s] = (uint32_t)cap;
    rows += cap; slots += ns;
  }
  t->h_row_base[t->S] = rows; t->h_slot_base[t->S] = slots;
  hm.row_base[t->S] = rows; hm.slot_base[t->S] = slots;
  if (rows >= 0xFFFFFFF0ull || slots >= 0xFFFFFFF0ull) { delete t; return DES_ERR_INVALID_ARG; }
  t->total_rows = rows; t->total_slots = slots;
  // fields sorted by (owning shard under FIELD, field): the K order of the row-split GEMM
  {
    uint32_t n = 0;
    for (uint32_t s = 0; s < t->S; ++s)
      for (uint32_t f = 0; f < t->F; ++f)
        if (f % t->S == s) hm.field_order[n++] = f;
  }
  t->nblk_max = (uint32_t)((t->max_nnz + 1023) / 1024) + 1;
  const size_t rowbytes = (size_t)t->stride * 4;
  const size_t FKH = (size_t)t->F * t->k * t->H;
  bool ok = true;
  auto A = [&](auto*& p, size_t bytes) {
    p = (typename std::remove_reference<decltype(p)>::type)dalloc(c, bytes);
    if (!p) ok = false;
  };
  A(t->slots, slots * sizeof(Slot));
  A(t->W, (rows + 1) * rowbytes);          // one all-zero row behind the table stands for "no row" in gathers
  if (c.optimizer != DES_OPT_SGD || c.lin_optimizer == DES_LIN_FTRL) A(t->A, rows * rowbytes);
  if (c.optimizer == DES_OPT_ADAM) A(t->A2, rows * rowbytes);
  A(t->meta, sizeof(DevMeta));
  A(t->slot_of, (size_t)t->max_nnz * 4);
  A(t->flags, (size_t)t->max_nnz);
  A(t->uslot, (size_t)t->max_nnz * 4);
  A(t->blk_cnt, (size_t)(t->S + 1) * t->nblk_max * 4);
  A(t->seg_off, (size_t)t->max_batch * (t->S + 1) * 4);
  t->hot_max = 16384;
  t->rep_max = (uint32_t)(t->max_nnz / 256 + t->hot_max + 1024);
  A(t->Gbuf, ((size_t)t->max_uniq + t->rep_max) * rowbytes);
  A(t->hinfo, (size_t)t->max_uniq * 4);
  A(t->dest, (size_t)t->max_nnz * 4);
  A(t->x_sorted, (size_t)t->max_nnz * 4);
  A(t->bag_tail, (size_t)t->max_batch * t->F * sizeof(float2));
  A(t->hot_base, (size_t)t->hot_max * 4);
  A(t->hot_R, (size_t)t->hot_max * 4);
  A(t->hot_u, (size_t)t->hot_max * 4);
  A(t->hot_ctr, HOT_CTR_WORDS * 4);
  t->work_max = t->rep_max / HOT_RCHUNK + t->hot_max;
  A(t->hot_work, (size_t)t->work_max * 4);
  A(t->hot_acc, (size_t)t->hot_max * t->stride * 8);
  if (t->k > 28 && t->max_nnz >= (1 << 20)) A(t->super_cnt, (size_t)t->max_batch * t->F * 16 * sizeof(float));
  if (t->H) {
    A(t->W1, FKH * 4); A(t->accW1, FKH * 4); A(t->W1b, FKH * 2);
    if (c.optimizer == DES_OPT_ADAM) A(t->acc2W1, FKH * 4);
    t->gw1_splits = 32;
    A(t->gW1_part, (size_t)t->gw1_splits * FKH * 4);
    // TMA needs 16-byte rows: every contiguous extent of a bf16 operand a multiple of 8
    t->use_tc = ((t->F * t->k) % 8 == 0) && (t->H % 8 == 0);
    A(t->pooled_b, (size_t)t->max_batch * t->F * t->k * 2);
    A(t->gZ_b, (size_t)t->max_batch * t->H * 2);
    t->gemm_ws_bytes = 8u << 20;
    A(t->gemm_ws, t->gemm_ws_bytes);
  }
  if (!ok) { des_table_destroy(t); return DES_ERR_CUDA; }
  t->dbg.rows = rows + 1; t->dbg.slots = slots; t->dbg.grad_rows = (unsigned long long)t->max_uniq + t->rep_max;
  t->dbg.nnz = (unsigned long long)t->max_nnz; t->dbg.meta = t->meta;
  bool cu = true;
  cu &= cudaMemset(t->slots, 0xFF, slots * sizeof(Slot)) == cudaSuccess;
  cu &= cudaMemset(t->W + rows * t->stride, 0, rowbytes) == cudaSuccess;
  cu &= cudaMemset(t->Gbuf, 0, ((size_t)t->max_uniq + t->rep_max) * rowbytes) == cudaSuccess;
  cu &= cudaMemset(t->hinfo, 0, (size_t)t->max_uniq * 4) == cudaSuccess;
  cu &= cudaMemset(t->hot_acc, 0, (size_t)t->hot_max * t->stride * 8) == cudaSuccess;
  cu &= cudaMemcpy(t->meta, &hm, sizeof(hm), cudaMemcpyHostToDevice) == cudaSuccess;
  if (t->H) {
    cu &= cudaMemset(t->W1, 0, FKH * 4) == cudaSuccess;
    cu &= cudaMemset(t->W1b, 0, FKH * 2) == cudaSuccess;
    fill_f32_kernel<<<256, 256>>>(t->accW1, FKH, c.optimizer == DES_OPT_ADAGRAD ? c.init_acc : 0.f);
    if (t->acc2W1) cu &= cudaMemset(t->acc2W1, 0, FKH * 4) == cudaSuccess;
    cu &= cudaGetLastError() == cudaSuccess;
  }
  cu &= cudaDeviceSynchronize() == cudaSuccess;
  if (!cu) { cudaGetLastError(); des_table_destroy(t); return DES_ERR_CUDA; }
  *out = t;
  return DES_OK;
}

extern "C" des_status_t des_table_status(des_table_t* t) {
  if (!t) return DES_ERR_INVALID_ARG;
  if (cudaDeviceSynchronize() != cudaSuccess) return DES_ERR_CUDA;
  uint32_t e = 0;
  DES_CUDA(cudaMemcpy(&e, &t->meta->err, 4, cudaMemcpyDeviceToHost));
  return (des_status_t)e;
}

extern "C" des_status_t des_table_size(des_table_t* t, uint64_t* h) {
  if (!t || !h) return DES_ERR_INVALID_ARG;
  uint32_t n[DES_MAX_SHARDS];
  DES_CUDA(cudaDeviceSynchronize());
  DES_CUDA(cudaMemcpy(n, t->meta->n_rows, sizeof(n), cudaMemcpyDeviceToHost));
  for (uint32_t s = 0; s < t->S; ++s) h[s] = n[s];
  return DES_OK;
}

extern "C" des_status_t des_table_row_base(des_table_t* t, uint64_t* h) {
  if (!t || !h) return DES_ERR_INVALID_ARG;
  for (uint32_t s = 0; s <= t->S; ++s) h[s] = t->h_row_base[s];
  return DES_OK;
}

extern "C" uint64_t des_table_launch_count(des_table_t* t) { return t ? t->launches : 0; }

extern "C" int des_build_has_tensor_cores(void) {
#ifdef DES_NO_CUTLASS
  return 0;
#else
  return 1;
#endif
}
extern "C" int des_table_uses_tensor_cores(des_table_t* t) { return (t && t->H && t->use_tc && des_build_has_tensor_cores()) ? 1 : 0; }
extern "C" int des_build_is_debug(void) {
#ifdef DES_DEBUG
  return 1;
#else
  return 0;
#endif
}

__global__ void export_kernel(const Slot* __restrict__ slots, unsigned long long nslots, const DevMeta* __restrict__ meta,
                              int S, int k, int stride, const float* __restrict__ W, const float* __restrict__ A,
                              unsigned long long* keys, uint8_t* shards, uint32_t* rows, float* emb, float* lin,
                              float* acc_emb, float* acc_lin, unsigned long long cap, unsigned long long* counter) {
  unsigned long long i = (unsigned long long)blockIdx.x * blockDim.x + threadIdx.x;
  unsigned long long st = (unsigned long long)gridDim.x * blockDim.x;
  for (; i < nslots; i += st) {
    Slot sl = slots[i];
    if (sl.key == DES_KEY_EMPTY || sl.row == DES_ROW_NONE) continue;
    int s = 0;
    while (s + 1 < S && meta->slot_base[s + 1] <= i) ++s;
    unsigned long long o = atomicAdd(counter, 1ull);
    if (o >= cap) continue;
    unsigned long long g = meta->row_base[s] + sl.row;
    if (keys) keys[o] = sl.key;
    if (shards) shards[o] = (uint8_t)s;
    if (rows) rows[o] = sl.row;
    for (int c = 0; c < k; ++c) {
      if (emb) emb[o * k + c] = W[g * stride + c];
      if (acc_emb) acc_emb[o * k + c] = A ? A[g * stride + c] : 0.f;
    }
    if (lin) lin[o] = W[g * stride + k];
    if (acc_lin) acc_lin[o] = A ? A[g * stride + k] : 0.f;
  }
}

extern "C" des_status_t des_table_export(des_table_t* t, uint64_t* d_keys, uint8_t* d_shards, uint32_t* d_rows,
                                         float* d_emb, float* d_lin, float* d_acc_emb, float* d_acc_lin,
                                         uint64_t cap, uint64_t* h_n_out) {
  if (!t || !h_n_out) return DES_ERR_INVALID_ARG;
  unsigned long long* ctr = nullptr;
  DES_CUDA(cudaMalloc(&ctr, 8));
  cudaMemset(ctr, 0, 8);
  des_api_begin(t, 0);
  export_kernel<<<t->sm_count * 8, 256>>>(t->slots, t->total_slots, t->meta, t->S, t->k, t->stride, t->W, t->A,
                                          (unsigned long long*)d_keys, d_shards, d_rows, d_emb, d_lin, d_acc_emb,
                                          d_acc_lin, cap, ctr);
  des_prof_mark(t, "export_kernel", 0);
  cudaError_t e = cudaDeviceSynchronize();
  unsigned long long n = 0;
  if (e == cudaSuccess) e = cudaMemcpy(&n, ctr, 8, cudaMemcpyDeviceToHost);
  cudaFree(ctr);
  if (e != cudaSuccess) return DES_ERR_CUDA;
  *h_n_out = n;
  return DES_OK;
}

__global__ void read_rows_kernel(const uint32_t* __restrict__ grows, long long n, int k, int stride,
                                 unsigned long long total_rows, const float* __restrict__ W,
                                 const float* __restrict__ A, float* emb, float* lin, float* acc_emb, float* acc_lin) {
  long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n) return;
  uint32_t g = grows[i];
  bool ok = g != DES_ROW_NONE && g < total_rows;
  for (int c = 0; c < k; ++c) {
    if (emb) emb[i * k + c] = ok ? W[(size_t)g * stride + c] : 0.f;
    if (acc_emb) acc_emb[i * k + c] = (ok && A) ? A[(size_t)g * stride + c] : 0.f;
  }
  if (lin) lin[i] = ok ? W[(size_t)g * stride + k] : 0.f;
  if (acc_lin) acc_lin[i] = (ok && A) ? A[(size_t)g * stride + k] : 0.f;
}

extern "C" des_status_t des_table_read_rows(des_table_t* t, const uint32_t* d_global_rows, int64_t n, float* d_emb,
                                            float* d_lin, float* d_acc_emb, float* d_acc_lin, void* stream) {
  if (!t || n < 0) return DES_ERR_INVALID_ARG;
  if (n == 0) return DES_OK;                 // nothing to do, whatever the pointers
  if (!d_global_rows) return DES_ERR_INVALID_ARG;
  des_api_begin(t, (cudaStream_t)stream);
  read_rows_kernel<<<(unsigned)((n + 255) / 256), 256, 0, (cudaStream_t)stream>>>(
      d_global_rows, n, t->k, t->stride, t->total_rows, t->W, t->A, d_emb, d_lin, d_acc_emb, d_acc_lin);
  DES_LAUNCH_CHECK(t, "read_rows_kernel");
  return DES_OK;
}

__global__ void write_rows_kernel(const uint32_t* __restrict__ grows, long long n, int k, int stride,
                                  unsigned long long total_rows, float* W, float* A, const float* __restrict__ emb,
                                  const float* __restrict__ lin, const float* __restrict__ acc_emb,
                                  const float* __restrict__ acc_lin) {
  long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n) return;
  uint32_t g = grows[i];
  if (g == DES_ROW_NONE || g >= total_rows) return;
  float n2 = 0.f;
  for (int c = 0; c < k; ++c) {
    if (emb) W[(size_t)g * stride + c] = emb[i * k + c];
    if (acc_emb && A) A[(size_t)g * stride + c] = acc_emb[i * k + c];
    const float v = W[(size_t)g * stride + c];
    n2 += v * v;
  }
  W[(size_t)g * stride + k + 1] = n2;
  if (lin) W[(size_t)g * stride + k] = lin[i];
  if (acc_lin && A) A[(size_t)g * stride + k] = acc_lin[i];
}

extern "C" des_status_t des_table_write_rows(des_table_t* t, const uint32_t* d_global_rows, int64_t n,
                                             const float* d_emb, const float* d_lin, const float* d_acc_emb,
                                             const float* d_acc_lin, void* stream) {
  if (!t || n < 0) return DES_ERR_INVALID_ARG;
  if (n == 0) return DES_OK;                 // nothing to do, whatever the pointers
  if (!d_global_rows) return DES_ERR_INVALID_ARG;
  des_api_begin(t, (cudaStream_t)stream);
  write_rows_kernel<<<(unsigned)((n + 255) / 256), 256, 0, (cudaStream_t)stream>>>(
      d_global_rows, n, t->k, t->stride, t->total_rows, t->W, t->A, d_emb, d_lin, d_acc_emb, d_acc_lin);
  DES_LAUNCH_CHECK(t, "write_rows_kernel");
  return DES_OK;
}

__global__ void state2_kernel(const uint32_t* __restrict__ grows, long long n, int k, int stride,
                              unsigned long long total_rows, float* A, float* A2, float* acc2_emb, float* lin2,
                              int write) {
  long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n) return;
  uint32_t g = grows[i];
  const bool ok = g != DES_ROW_NONE && g < total_rows;
  if (write) {
    if (!ok) return;
    if (acc2_emb && A2) for (int c = 0; c < k; ++c) A2[(size_t)g * stride + c] = acc2_emb[i * k + c];
    if (lin2 && A) A[(size_t)g * stride + k + 1] = lin2[i];
  } else {
    if (acc2_emb) for (int c = 0; c < k; ++c) acc2_emb[i * k + c] = (ok && A2) ? A2[(size_t)g * stride + c] : 0.f;
    if (lin2) lin2[i] = (ok && A) ? A[(size_t)g * stride + k + 1] : 0.f;
  }
}

extern "C" des_status_t des_table_read_state2(des_table_t* t, const uint32_t* d_global_rows, int64_t n,
                                              float* d_acc2_emb, float* d_lin2, void* stream) {
  if (!t || n < 0) return DES_ERR_INVALID_ARG;
  if (n == 0) return DES_OK;                 // nothing to do, whatever the pointers
  if (!d_global_rows) return DES_ERR_INVALID_ARG;
  des_api_begin(t, (cudaStream_t)stream);
  state2_kernel<<<(unsigned)((n + 255) / 256), 256, 0, (cudaStream_t)stream>>>(
      d_global_rows, n, t->k, t->stride, t->total_rows, t->A, t->A2, d_acc2_emb, d_lin2, 0);
  DES_LAUNCH_CHECK(t, "state2_kernel");
  return DES_OK;
}

extern "C" des_status_t des_table_write_state2(des_table_t* t, const uint32_t* d_global_rows, int64_t n,
                                               const float* d_acc2_emb, const float* d_lin2, void* stream) {
  if (!t || n < 0) return DES_ERR_INVALID_ARG;
  if (n == 0) return DES_OK;                 // nothing to do, whatever the pointers
  if (!d_global_rows) return DES_ERR_INVALID_ARG;
  des_api_begin(t, (cudaStream_t)stream);
  state2_kernel<<<(unsigned)((n + 255) / 256), 256, 0, (cudaStream_t)stream>>>(
      d_global_rows, n, t->k, t->stride, t->total_rows, t->A, t->A2, const_cast<float*>(d_acc2_emb),
      const_cast<float*>(d_lin2), 1);
  DES_LAUNCH_CHECK(t, "state2_kernel");
  return DES_OK;
}

// ---- first dense layer weights ----------------------------------------------
__global__ void w1_shadow_kernel(const float* __restrict__ W1, __nv_bfloat16* __restrict__ W1b, size_t n) {
  size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x, st = (size_t)gridDim.x * blockDim.x;
  for (; i < n; i += st) W1b[i] = __float2bfloat16_rn(W1[i]);
}

extern "C" des_status_t des_dense1_set(des_table_t* t, const float* d_W1, void* stream) {
  if (!t || !d_W1 || !t->H) return DES_ERR_INVALID_ARG;
  size_t n = (size_t)t->F * t->k * t->H;
  des_api_begin(t, (cudaStream_t)stream);
  DES_CUDA(cudaMemcpyAsync(t->W1, d_W1, n * 4, cudaMemcpyDeviceToDevice, (cudaStream_t)stream));
  w1_shadow_kernel<<<256, 256, 0, (cudaStream_t)stream>>>(t->W1, t->W1b, n);
  DES_LAUNCH_CHECK(t, "w1_shadow_kernel");
  return DES_OK;
}

extern "C" des_status_t des_dense1_get(des_table_t* t, float* d_W1, void* stream) {
  if (!t || !d_W1 || !t->H) return DES_ERR_INVALID_ARG;
  size_t n = (size_t)t->F * t->k * t->H;
  DES_CUDA(cudaMemcpyAsync(d_W1, t->W1, n * 4, cudaMemcpyDeviceToDevice, (cudaStream_t)stream));
  return DES_OK;
}

// Optimizer state of W1: first word (Adagrad accumulator / Adam m) and second word (Adam v).
extern "C" des_status_t des_dense1_get_state(des_table_t* t, float* d_state1, float* d_state2, void* stream) {
  if (!t || !t->H) return DES_ERR_INVALID_ARG;
  if ((d_state1 && !t->accW1) || (d_state2 && !t->acc2W1)) return DES_ERR_INVALID_ARG;
  size_t n = (size_t)t->F * t->k * t->H;
  if (d_state1) DES_CUDA(cudaMemcpyAsync(d_state1, t->accW1, n * 4, cudaMemcpyDeviceToDevice, (cudaStream_t)stream));
  if (d_state2) DES_CUDA(cudaMemcpyAsync(d_state2, t->acc2W1, n * 4, cudaMemcpyDeviceToDevice, (cudaStream_t)stream));
  return DES_OK;
}

extern "C" des_status_t des_dense1_set_state(des_table_t* t, const float* d_state1, const float* d_state2, void* stream) {
  if (!t || !t->H) return DES_ERR_INVALID_ARG;
  if ((d_state1 && !t->accW1) || (d_state2 && !t->acc2W1)) return DES_ERR_INVALID_ARG;
  size_t n = (size_t)t->F * t->k * t->H;
  if (d_state1) DES_CUDA(cudaMemcpyAsync(t->accW1, d_state1, n * 4, cudaMemcpyDeviceToDevice, (cudaStream_t)stream));
  if (d_state2) DES_CUDA(cudaMemcpyAsync(t->acc2W1, d_state2, n * 4, cudaMemcpyDeviceToDevice, (cudaStream_t)stream));
  return DES_OK;
}

des_status_t des_check_batch(const des_table* t, const des_batch_t* b, int need_dedup) {
  if (!t || !b) return DES_ERR_INVALID_ARG;
  if (b->batch <= 0 || b->batch > t->max_batch || b->nnz < 0 || b->nnz > t->max_nnz) return DES_ERR_INVALID_ARG;
  if (!b->offsets || !b->rows || !b->shards || (b->nnz > 0 && !b->ids)) return DES_ERR_INVALID_ARG;
  if (need_dedup && (!b->uidx || !b->uniq_rows || !b->n_uniq)) return DES_ERR_INVALID_ARG;
  return DES_OK;
}
