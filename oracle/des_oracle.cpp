// CPU oracle of the DES sparse step (arXiv 1909.04823).
//
// TEST INFRASTRUCTURE ONLY: a plain, slow, sequential implementation that the
// tests, the smoke check and the benchmark's cpu_baseline leg compare the CUDA
// path against.  The product never calls it; it shares no code, header, table
// or constant generator with the CUDA sources.
//
// What it computes, and from which passage:
//   * the ORIGINAL (unsubstituted) operators F — LR's W^T X (Section 4.1), FM's
//     order-2 sum in both its O(n^2) pair form and its linear form (Eq. 5),
//     the embedding layer's per-field pooling and the first FC layer V^T W
//     (Eq. 6) — looked up by key with no notion of shards;
//   * the DES form — per-shard sub-operators M_j (Eqs. 2, 7, and
//     M_1(V_i,W_i) = V_i^T W_i of Section 4.3), aggregation (+) in shard order
//     (Eq. 1), and the substitution operator F (Eqs. 3, 8, 10; Algorithm 1);
//   * the backward rule of Section 3.2 ("Back-propagation Phase"): the
//     gradient of the aggregate flows unchanged into each shard's own
//     sub-operator; one optimizer application per unique key on the summed
//     gradient, state local to the shard (Section 4.3, closing paragraph);
//   * the dynamic hash table's lookup / insert / update (Section 5).
// Where the paper is silent (which hash, how a new weight is initialised, how
// rows are numbered, Adagrad's exact form) it takes one fixed reading; each is
// marked "reading" below.
//
// All-cores build: compiled a second time with -fopenmp, the per-sample loops of
// the forward, the per-element loops of the first layer's backward and the
// per-unique-key loops of the update run as `omp parallel for`; every sum keeps
// the order of the sequential build (a key's occurrences are added in CSR order
// either way), so both builds return the same bits.  Without -fopenmp the
// pragmas and the grouped form of the gradient sum below are compiled out.
//
// Arithmetic: weights and optimizer state are float32 (the paper's storage
// type, Section 4.1); every sum is accumulated in double and rounded once.
//
// Pins (tests/, marked not-gpu): Philox known-answer vectors; mix64 inverse;
// FM pair form == linear form; DES form == original for any S and both
// partitions; S = 1 == any S; gradients == central finite differences;
// dedup/Adagrad special cases; row-split GEMM == one dense matmul; canonical
// row numbering vs a dictionary walk; Adagrad / Adam / FTRL vs library optimizers
// and closed forms; eviction vs a brute-force model of its rule; the read-out head
// vs the library's log loss and autograd.  Fixed by no passage of the paper, hence
// "parity unpinned" by it: the hash / shard rule (pinned only by bijectivity and
// balance), the eviction rule, the read-out head.
#ifdef _OPENMP
#include <omp.h>
#endif
#include <cmath>
#include <cstdint>
#include <cstring>
#include <unordered_map>
#include <vector>

namespace {

const uint32_t ROW_NONE = 0xFFFFFFFFu;
enum { OP_LR = 1, OP_FM = 2, OP_POOL = 4, OP_DENSE1 = 8 };
enum { PART_HASH = 0, PART_FIELD = 1 };
enum { OPT_SGD = 0, OPT_ADAGRAD = 1, OPT_ADAM = 2 };
enum { LIN_SAME = 0, LIN_FTRL = 1 };

// reading: the table's 64-bit mixer (splitmix64 finaliser steps)
uint64_t mix64(uint64_t z) {
  z ^= z >> 30; z *= 0xBF58476D1CE4E5B9ull;
  z ^= z >> 27; z *= 0x94D049BB133111EBull;
  z ^= z >> 31;
  return z;
}

// Philox4x32-10 (Salmon et al., SC'11): ten rounds of two 32x32->64
// multiplies with the key bumped by the Weyl constants each round.
void philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]) {
  uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
  uint32_t k0 = key[0], k1 = key[1];
  for (int r = 0; r < 10; ++r) {
    uint64_t p0 = (uint64_t)0xD2511F53u * c0;
    uint64_t p1 = (uint64_t)0xCD9E8D57u * c2;
    uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
    uint32_t n1 = (uint32_t)p1;
    uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
    uint32_t n3 = (uint32_t)p0;
    c0 = n0; c1 = n1; c2 = n2; c3 = n3;
    k0 += 0x9E3779B9u; k1 += 0xBB67AE85u;
  }
  out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

// reading: component c of a new key's latent vector is
//   ((r >> 8) * 2^-23 - 1) * init_scale,   r = word (c mod 4) of
//   Philox4x32-10(counter = (c/4, 0, seed_lo, seed_hi), key = (id_lo, id_hi)).
// Everything before the final multiply is exact in float32.
float init_value(uint64_t seed, uint64_t id, uint32_t c, float init_scale) {
  uint32_t ctr[4] = {c / 4u, 0u, (uint32_t)seed, (uint32_t)(seed >> 32)};
  uint32_t key[2] = {(uint32_t)id, (uint32_t)(id >> 32)};
  uint32_t r[4];
  philox4x32_10(ctr, key, r);
  float u = (float)(r[c % 4u] >> 8);          // 24 bits, exact
  float x = u * (1.0f / 8388608.0f);          // * 2^-23, exact, in [0, 2)
  float y = x - 1.0f;                          // exact, in [-1, 1)
  volatile float z = y * init_scale;           // one rounding (no contraction)
  return z;
}

float bf16_round(float x) {                    // round-to-nearest-even to bfloat16
  uint32_t u; std::memcpy(&u, &x, 4);
  if ((u & 0x7F800000u) == 0x7F800000u) return x;
  uint32_t lsb = (u >> 16) & 1u;
  u += 0x7FFFu + lsb;
  u &= 0xFFFF0000u;
  float y; std::memcpy(&y, &u, 4);
  return y;
}

struct Shard {
  std::unordered_map<uint64_t, uint32_t> map;   // key -> shard-local row
  std::vector<uint64_t> keys;                   // row -> key
  std::vector<float> emb, lin, acc_emb, acc_lin;
  std::vector<float> acc2_emb, lin2;            // second state word: Adam's v; linear weight: Adam's v / FTRL's z
  std::vector<uint64_t> stamp;                  // table clock when the row was inserted or last updated
};

struct Table {
  uint32_t S, F, k, H, partition, optimizer;
  uint64_t seed; float init_scale, lr, eps, init_acc;
  std::vector<Shard> sh;
  std::vector<float> W1, accW1, acc2W1;         // [F*k][H]
  uint32_t lin_optimizer = LIN_SAME;
  float beta1 = 0.9f, beta2 = 0.999f, ftrl_alpha = 0.05f, ftrl_beta = 1.0f, ftrl_l1 = 0.f, ftrl_l2 = 0.f;
  int64_t step = 0;                             // backward calls so far (Adam's t)
  uint64_t clock = 0;                           // inserting find_or_insert calls so far (the age clock of eviction)
  float state_init() const { return optimizer == OPT_ADAGRAD ? init_acc : 0.0f; }
  float lin_state_init() const { return (lin_optimizer == LIN_FTRL || optimizer != OPT_ADAGRAD) ? 0.0f : init_acc; }
  uint32_t shard_of(uint64_t id, uint32_t field) const {
    return partition == PART_HASH ? (uint32_t)(mix64(id) % S) : field % S;
  }
  uint32_t insert(uint32_t s, uint64_t id) {
    Shard& h = sh[s];
    uint32_t row = (uint32_t)h.keys.size();
    h.map.emplace(id, row);
    h.keys.push_back(id);
    for (uint32_t c = 0; c < k; ++c) h.emb.push_back(init_value(seed, id, c, init_scale));
    h.lin.push_back(0.0f);
    for (uint32_t c = 0; c < k; ++c) { h.acc_emb.push_back(state_init()); h.acc2_emb.push_back(0.0f); }
    h.acc_lin.push_back(lin_state_init());
    h.lin2.push_back(0.0f);
    h.stamp.push_back(clock);
    return row;
  }
};

// FTRL-Proximal per coordinate (McMahan et al. 2013, "Ad Click Prediction"), the
// optimizer the paper runs on the order-1 weights (Section 6, "Parameter
// Settings"): state n (sum of squared gradients) and z.
inline void apply_ftrl(const Table& t, float& w, float& n, float& z, double Gd) {
  const double G = (double)(float)Gd, n0 = (double)n;
  const double sigma = (std::sqrt(n0 + G * G) - std::sqrt(n0)) / (double)t.ftrl_alpha;
  const float zf = (float)((double)z + G - sigma * (double)w);
  const float nf = (float)(n0 + G * G);
  z = zf; n = nf;
  const double zz = (double)zf, l1 = (double)t.ftrl_l1;
  if (std::fabs(zz) <= l1) { w = 0.0f; return; }
  const double sgn = zz > 0 ? 1.0 : -1.0;
  w = (float)(-(zz - sgn * l1) / (((double)t.ftrl_beta + std::sqrt((double)nf)) / (double)t.ftrl_alpha + (double)t.ftrl_l2));
}

// acc / acc2: first and second state word (Adagrad: accumulator / unused; Adam: m / v).
inline void apply_opt(const Table& t, float& theta, float& acc, float& acc2, double Gd) {
  float G = (float)Gd;                          // summed gradient, rounded once
  if (t.optimizer == OPT_SGD) {
    theta = (float)((double)theta - (double)t.lr * (double)G);
  } else if (t.optimizer == OPT_ADAM) {         // reading: lazy Adam, one global step count per backward call
    const double b1 = (double)t.beta1, b2 = (double)t.beta2;
    const float m = (float)(b1 * (double)acc + (1.0 - b1) * (double)G);
    const float v = (float)(b2 * (double)acc2 + (1.0 - b2) * (double)G * (double)G);
    acc = m; acc2 = v;
    const double c1 = 1.0 - std::pow(b1, (double)t.step), c2 = 1.0 - std::pow(b2, (double)t.step);
    theta = (float)((double)theta - (double)t.lr * ((double)m / c1) / (std::sqrt((double)v / c2) + (double)t.eps));
  } else {                                      // reading: eps outside the root
    float a = (float)((double)acc + (double)G * (double)G);
    acc = a;
    theta = (float)((double)theta - (double)t.lr * (double)G / (std::sqrt((double)a) + (double)t.eps));
  }
}

}  // namespace

extern "C" {

// threads the parallel loops of this build use (1 without -fopenmp)
int orc_num_threads() {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

uint64_t orc_mix64(uint64_t x) { return mix64(x); }
void orc_philox4x32_10(const uint32_t* ctr, const uint32_t* key, uint32_t* out) { philox4x32_10(ctr, key, out); }
float orc_init_value(uint64_t seed, uint64_t id, uint32_t c, float scale) { return init_value(seed, id, c, scale); }
float orc_bf16_round(float x) { return bf16_round(x); }

void orc_shard_of_many(const uint64_t* ids, int64_t n, uint32_t S, uint8_t* out) {
  for (int64_t i = 0; i < n; ++i) out[i] = (uint8_t)(mix64(ids[i]) % S);
}

// Communication-saving ratios of Section 4 (R_lr, R_fm(2), R_dnn) from the
// byte sizes of what DES exchanges (the per-shard partials above: B, B*k + B
// and B*H float32 values) against the mesh strategy's keys + weights for U
// unique features (uint64 keys, float32 weights, k-vectors; S_W = bytes of the
// first FC layer's weights).
void orc_comm_saving(int64_t B, int64_t U, int64_t k, int64_t H, double S_W, double* out3) {
  double S_key = 8.0 * U, S_w = 4.0 * U, S_V = 4.0 * k * U;
  double S_M1_lr = 4.0 * B, S_M1_fm = 4.0 * B * k, S_M2_fm = 4.0 * B, S_M1_dnn = 4.0 * B * H;
  out3[0] = 1.0 - 2.0 * S_M1_lr / (S_key + S_w);
  out3[1] = 1.0 - 2.0 * (S_M1_fm + S_M2_fm) / (S_key + S_V);
  out3[2] = 1.0 - 2.0 * S_M1_dnn / (S_key + S_V + S_W);
}

void* orc_create(uint32_t S, uint32_t F, uint32_t k, uint32_t H, uint32_t partition, uint32_t optimizer,
                 uint64_t seed, float init_scale, float lr, float eps, float init_acc) {
  Table* t = new Table();
  t->S = S; t->F = F; t->k = k; t->H = H; t->partition = partition; t->optimizer = optimizer;
  t->seed = seed; t->init_scale = init_scale; t->lr = lr; t->eps = eps; t->init_acc = init_acc;
  t->sh.resize(S);
  if (H) {
    t->W1.assign((size_t)F * k * H, 0.0f);
    t->accW1.assign((size_t)F * k * H, t->state_init());
    t->acc2W1.assign((size_t)F * k * H, 0.0f);
  }
  return t;
}
void orc_destroy(void* p) { delete (Table*)p; }

// Optimizer settings beyond the constructor's (call before the first insert).
void orc_set_opt(void* p, uint32_t lin_optimizer, float beta1, float beta2, float ftrl_alpha, float ftrl_beta,
                 float ftrl_l1, float ftrl_l2) {
  Table* t = (Table*)p;
  t->lin_optimizer = lin_optimizer; t->beta1 = beta1; t->beta2 = beta2;
  t->ftrl_alpha = ftrl_alpha; t->ftrl_beta = ftrl_beta; t->ftrl_l1 = ftrl_l1; t->ftrl_l2 = ftrl_l2;
}

void orc_dense1_set(void* p, const float* W1) { Table* t = (Table*)p; std::memcpy(t->W1.data(), W1, t->W1.size() * 4); }
void orc_dense1_get(void* p, float* W1, float* acc) {
  Table* t = (Table*)p;
  if (W1) std::memcpy(W1, t->W1.data(), t->W1.size() * 4);
  if (acc) std::memcpy(acc, t->accW1.data(), t->accW1.size() * 4);
}

void orc_size(void* p, uint64_t* per_shard) {
  Table* t = (Table*)p;
  for (uint32_t s = 0; s < t->S; ++s) per_shard[s] = t->sh[s].keys.size();
}

// lookup + insert (Section 5).  Rows are numbered per shard in order of first
// occurrence in CSR order (reading); batch-unique indices likewise over the
// whole batch.  Outputs: rows[nnz], shards[nnz], uidx[nnz], and for each
// unique key u its (shard, row) in uniq_shard/uniq_row; returns U.
int64_t orc_find_or_insert(void* p, const int32_t* offsets, const uint64_t* ids, int32_t B, int insert,
                           uint32_t* rows, uint8_t* shards, uint32_t* uidx,
                           uint8_t* uniq_shard, uint32_t* uniq_row) {
  Table* t = (Table*)p;
  if (insert && offsets[(int64_t)B * t->F] > 0) t->clock += 1;   // reading: the table's age clock counts the inserting calls (with at least one occurrence)
  std::unordered_map<uint64_t, uint32_t> seen;   // (shard<<32 | row) -> u
  int64_t U = 0;
  for (int64_t bag = 0; bag < (int64_t)B * t->F; ++bag) {
    uint32_t f = (uint32_t)(bag % t->F);
    for (int32_t j = offsets[bag]; j < offsets[bag + 1]; ++j) {
      uint64_t id = ids[j];
      uint32_t s = t->shard_of(id, f);
      shards[j] = (uint8_t)s;
      auto it = t->sh[s].map.find(id);
      uint32_t row;
      if (it != t->sh[s].map.end()) row = it->second;
      else if (insert) row = t->insert(s, id);
      else row = ROW_NONE;
      rows[j] = row;
      if (row == ROW_NONE) { if (uidx) uidx[j] = ROW_NONE; continue; }
      uint64_t gk = ((uint64_t)s << 32) | row;
      auto iu = seen.find(gk);
      uint32_t u;
      if (iu == seen.end()) {
        u = (uint32_t)U++;
        seen.emplace(gk, u);
        if (uniq_shard) uniq_shard[u] = (uint8_t)s;
        if (uniq_row) uniq_row[u] = row;
      } else u = iu->second;
      if (uidx) uidx[j] = u;
    }
  }
  return U;
}

// The ORIGINAL operators, per sample, over all of the sample's occurrences
// regardless of shard.  Outputs (double): lr0[B] = W^T X (Section 4.1);
// A0[B][k] = sum v x, Q0[B] = sum <vx,vx>, fm2[B] linear form (Eq. 5, last
// line); pooled0[B][F*k] (embedding layer, Section 4.3); Z0[B][H] = V^T W
// (Eq. 6) on bfloat16-rounded operands (reading), accumulated in double.
// Sabs[B][k+1] (optional): sums of the absolute values of the terms of A0 and
// lr0, the scale of a float32 summation error when the terms cancel.
void orc_forward_original(void* p, uint32_t ops, const int32_t* offsets, const uint64_t* ids,
                          const float* vals, int32_t B, double* lr0, double* A0, double* Q0,
                          double* fm2, double* pooled0, double* Z0, double* Sabs) {
  Table* t = (Table*)p;
  const uint32_t F = t->F, k = t->k, H = t->H;
#pragma omp parallel for schedule(dynamic, 16)
  for (int32_t b = 0; b < B; ++b) {
    std::vector<double> A(k, 0.0), pool((size_t)F * k, 0.0);
    double lr = 0, Q = 0;
    for (uint32_t f = 0; f < F; ++f) {
      int64_t bag = (int64_t)b * F + f;
      for (int32_t j = offsets[bag]; j < offsets[bag + 1]; ++j) {
        uint32_t s = t->shard_of(ids[j], f);
        auto it = t->sh[s].map.find(ids[j]);
        if (it == t->sh[s].map.end()) continue;            // unknown key: no weight
        const Shard& h = t->sh[s];
        uint32_t row = it->second;
        double x = vals ? (double)vals[j] : 1.0;
        lr += (double)h.lin[row] * x;
        if (Sabs) Sabs[(size_t)b * (k + 1) + k] += std::fabs((double)h.lin[row] * x);
        for (uint32_t c = 0; c < k; ++c) {
          double vx = (double)h.emb[(size_t)row * k + c] * x;
          A[c] += vx; Q += vx * vx; pool[(size_t)f * k + c] += vx;
          if (Sabs) Sabs[(size_t)b * (k + 1) + c] += std::fabs(vx);
        }
      }
    }
    if (lr0) lr0[b] = lr;
    double AA = 0;
    for (uint32_t c = 0; c < k; ++c) { if (A0) A0[(size_t)b * k + c] = A[c]; AA += A[c] * A[c]; }
    if (Q0) Q0[b] = Q;
    if (fm2) fm2[b] = 0.5 * AA - 0.5 * Q;
    if (pooled0) for (size_t i = 0; i < (size_t)F * k; ++i) pooled0[(size_t)b * F * k + i] = pool[i];
    if ((ops & OP_DENSE1) && Z0) {
      for (uint32_t h2 = 0; h2 < H; ++h2) {
        double z = 0;
        for (size_t i = 0; i < (size_t)F * k; ++i)
          z += (double)bf16_round((float)pool[i]) * (double)bf16_round(t->W1[i * H + h2]);
        Z0[(size_t)b * H + h2] = z;
      }
    }
  }
}

// FM order-2 in its defining pair form, sum_{i<i'} <v_i, v_i'> x_i x_i'
// (Eq. 5, first line): O(n^2 k), tiny inputs only.
void orc_fm_pairs(void* p, const int32_t* offsets, const uint64_t* ids, const float* vals,
                  int32_t B, double* fm_pairs) {
  Table* t = (Table*)p;
  const uint32_t F = t->F, k = t->k;
  for (int32_t b = 0; b < B; ++b) {
    std::vector<const float*> v; std::vector<double> x;
    for (uint32_t f = 0; f < F; ++f) {
      int64_t bag = (int64_t)b * F + f;
      for (int32_t j = offsets[bag]; j < offsets[bag + 1]; ++j) {
        uint32_t s = t->shard_of(ids[j], f);
        auto it = t->sh[s].map.find(ids[j]);
        if (it == t->sh[s].map.end()) continue;
        v.push_back(&t->sh[s].emb[(size_t)it->second * k]);
        x.push_back(vals ? (double)vals[j] : 1.0);
      }
    }
    double acc = 0;
    for (size_t i = 0; i < v.size(); ++i)
      for (size_t i2 = i + 1; i2 < v.size(); ++i2) {
        double dot = 0;
        for (uint32_t c = 0; c < k; ++c) dot += (double)v[i][c] * (double)v[i2][c];
        acc += dot * x[i] * x[i2];
      }
    fm_pairs[b] = acc;
  }
}

// Sub-operators of every shard (Eqs. 2 and 7; pooled per-field partials;
// M_1(V_s, W_s) = V_s^T W_s).  Shard s only ever touches the keys it owns and
// finds them through the (shard, row) pair that find_or_insert returned.
//   part_small[S][B][k+2] = (M1_fm[0..k), M1_lr, M2_fm)
//   part_pooled[S][B][F*k]  (optional)
//   part_dense[S][B][H]     (optional; needs part_pooled semantics internally)
void orc_forward_partials(void* p, uint32_t ops, const int32_t* offsets, const float* vals,
                          const uint32_t* rows, const uint8_t* shards, int32_t B,
                          double* part_small, double* part_pooled, double* part_dense) {
  Table* t = (Table*)p;
  const uint32_t S = t->S, F = t->F, k = t->k, H = t->H;
  const size_t FK = (size_t)F * k;
  for (uint32_t s = 0; s < S; ++s) {
    const Shard& h = t->sh[s];
#pragma omp parallel for schedule(dynamic, 16)
    for (int32_t b = 0; b < B; ++b) {
      std::vector<double> pool(FK, 0.0);
      double* ps = part_small ? part_small + ((size_t)s * B + b) * (k + 2) : nullptr;
      if (ps) for (uint32_t c = 0; c < k + 2; ++c) ps[c] = 0;
      for (uint32_t f = 0; f < F; ++f) {
        int64_t bag = (int64_t)b * F + f;
        for (int32_t j = offsets[bag]; j < offsets[bag + 1]; ++j) {
          if (shards[j] != s || rows[j] == ROW_NONE) continue;
          uint32_t row = rows[j];
          double x = vals ? (double)vals[j] : 1.0;
          if (ps) ps[k] += (double)h.lin[row] * x;
          for (uint32_t c = 0; c < k; ++c) {
            double vx = (double)h.emb[(size_t)row * k + c] * x;
            if (ps) { ps[c] += vx; ps[k + 1] += vx * vx; }
            pool[(size_t)f * k + c] += vx;
          }
        }
      }
      if (part_pooled) std::memcpy(part_pooled + ((size_t)s * B + b) * FK, pool.data(), FK * 8);
      if ((ops & OP_DENSE1) && part_dense) {
        for (uint32_t h2 = 0; h2 < H; ++h2) {
          double z = 0;
          for (size_t i = 0; i < FK; ++i)
            if (pool[i] != 0.0) z += (double)bf16_round((float)pool[i]) * (double)bf16_round(t->W1[i * H + h2]);
          part_dense[((size_t)s * B + b) * H + h2] = z;
        }
      }
    }
  }
}

// Aggregation over shards s = 0..S-1 (Eq. 1) and substitution operator F
// (Eqs. 3 without sigma/bias, 8, 10).  out_small[B][k+3] = (A[0..k), R_lr, fm2, Q).
void orc_aggregate(void* p, int32_t B, const double* part_small, const double* part_pooled,
                   const double* part_dense, double* out_small, double* pooled, double* Z) {
  Table* t = (Table*)p;
  const uint32_t S = t->S, F = t->F, k = t->k, H = t->H;
  const size_t FK = (size_t)F * k;
#pragma omp parallel for schedule(static)
  for (int32_t b = 0; b < B; ++b) {
    if (part_small && out_small) {
      double* o = out_small + (size_t)b * (k + 3);
      for (uint32_t c = 0; c < k + 3; ++c) o[c] = 0;
      double Q = 0;
      for (uint32_t s = 0; s < S; ++s) {
        const double* ps = part_small + ((size_t)s * B + b) * (k + 2);
        for (uint32_t c = 0; c < k; ++c) o[c] += ps[c];
        o[k] += ps[k]; Q += ps[k + 1];
      }
      double AA = 0;
      for (uint32_t c = 0; c < k; ++c) AA += o[c] * o[c];
      o[k + 1] = 0.5 * AA - 0.5 * Q; o[k + 2] = Q;
    }
    if (part_pooled && pooled)
      for (size_t i = 0; i < FK; ++i) {
        double a = 0;
        for (uint32_t s = 0; s < S; ++s) a += part_pooled[((size_t)s * B + b) * FK + i];
        pooled[(size_t)b * FK + i] = a;
      }
    if (part_dense && Z)
      for (uint32_t h2 = 0; h2 < H; ++h2) {
        double a = 0;
        for (uint32_t s = 0; s < S; ++s) a += part_dense[((size_t)s * B + b) * H + h2];
        Z[(size_t)b * H + h2] = a;
      }
  }
}

// Backward + update.  Per occurrence j of bag (b, f), owned by shard s:
//   g_w(j) = x_j gL[b]                                   (d/dw of Eq. 3's sum)
//   g_v(j) = x_j ( gF[b] (A[b] - v_j x_j) + gE[b][f] )   (d/dv of Eq. 8 + pooling)
// evaluated with the PRE-update weights; with DENSE1, gE += gZ bf16(W1)^T first
// (each shard only needs its own column block: no cross-shard term, Section
// 3.2) and gW1 = bf16(pooled)^T gZ.  Then one optimizer application per unique
// key on the summed gradient.  A is the aggregated (+)M_1 the caller got from
// the forward (float32).  Optional outputs: Gw[U], Gv[U][k] (the summed
// gradients, rounded to float32), gE_total[B][F*k], and Sw[U], Sv[U][k]: the sums
// of the ABSOLUTE values of the same per-occurrence terms (the scale against
// which a float32 summation error is measured when the terms cancel); gW1[F*k][H]:
// the first layer's weight gradient before the optimizer.
void orc_backward_update(void* p, uint32_t ops, const int32_t* offsets, const float* vals,
                         const uint32_t* rows, const uint8_t* shards, const uint32_t* uidx,
                         int32_t B, int64_t U, const float* A, const float* pooled,
                         const float* gL, const float* gF, const float* gE, const float* gZ,
                         float* Gw_out, float* Gv_out, float* gE_total_out, double* Sw_out, double* Sv_out,
                         float* gW1_out) {
  Table* t = (Table*)p;
  const uint32_t F = t->F, k = t->k, H = t->H;
  const size_t FK = (size_t)F * k;
  std::vector<float> gEt;
  const bool use_pool = (ops & (OP_POOL | OP_DENSE1)) != 0;
  if (use_pool) {
    gEt.assign((size_t)B * FK, 0.0f);
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < (int64_t)((size_t)B * FK); ++i) {
      double a = ((ops & OP_POOL) && gE) ? (double)gE[i] : 0.0;
      if ((ops & OP_DENSE1) && gZ) {
        size_t b = i / FK, col = i % FK;
        for (uint32_t h2 = 0; h2 < H; ++h2)
          a += (double)gZ[b * H + h2] * (double)bf16_round(t->W1[col * H + h2]);
      }
      gEt[i] = (float)a;
    }
    if (gE_total_out) std::memcpy(gE_total_out, gEt.data(), gEt.size() * 4);
  }
  t->step += 1;                                  // Adam's global step count
  std::vector<double> Gw((size_t)U, 0.0), Gv((size_t)U * k, 0.0);
  std::vector<double> Sw((size_t)U, 0.0), Sv((size_t)U * k, 0.0);
  std::vector<uint8_t> us((size_t)U); std::vector<uint32_t> ur((size_t)U);
  // the per-occurrence terms of one key, added in CSR order
  auto add_occurrence = [&](int32_t b, uint32_t f, int32_t j) {
    uint32_t u = uidx[j], s = shards[j], row = rows[j];
    us[u] = (uint8_t)s; ur[u] = row;
    const Shard& h = t->sh[s];
    double x = vals ? (double)vals[j] : 1.0;
    if (ops & OP_LR) { Gw[u] += x * (double)gL[b]; Sw[u] += std::fabs(x * (double)gL[b]); }
    for (uint32_t c = 0; c < k; ++c) {
      double g = 0;
      if (ops & OP_FM) g += (double)gF[b] * ((double)A[(size_t)b * k + c] - (double)h.emb[(size_t)row * k + c] * x);
      if (use_pool) g += (double)gEt[(size_t)b * FK + (size_t)f * k + c];
      Gv[(size_t)u * k + c] += x * g;
      Sv[(size_t)u * k + c] += std::fabs(x * g);
    }
  };
#ifndef _OPENMP
  for (int32_t b = 0; b < B; ++b)
    for (uint32_t f = 0; f < F; ++f) {
      int64_t bag = (int64_t)b * F + f;
      for (int32_t j = offsets[bag]; j < offsets[bag + 1]; ++j)
        if (rows[j] != ROW_NONE) add_occurrence(b, f, j);
    }
#else
  {
    // all-cores build: the same sums grouped by key first (a counting sort of the occurrences by
    // unique index that keeps CSR order inside a key), then one thread per key
    std::vector<int64_t> start((size_t)U + 1, 0);
    const int64_t nnz = offsets[(int64_t)B * F];
    for (int64_t j = 0; j < nnz; ++j) if (rows[j] != ROW_NONE) start[uidx[j] + 1]++;
    for (int64_t u = 0; u < U; ++u) start[u + 1] += start[u];
    std::vector<int32_t> occ((size_t)start[U]), bag_of((size_t)start[U]);
    std::vector<int64_t> fill(start.begin(), start.end() - 1);
    for (int64_t bag = 0; bag < (int64_t)B * F; ++bag)
      for (int32_t j = offsets[bag]; j < offsets[bag + 1]; ++j)
        if (rows[j] != ROW_NONE) { int64_t p_ = fill[uidx[j]]++; occ[p_] = j; bag_of[p_] = (int32_t)bag; }
#pragma omp parallel for schedule(dynamic, 64)
    for (int64_t u = 0; u < U; ++u)
      for (int64_t p_ = start[u]; p_ < start[u + 1]; ++p_)
        add_occurrence((int32_t)(bag_of[p_] / F), (uint32_t)(bag_of[p_] % F), occ[p_]);
  }
#endif
#pragma omp parallel for schedule(dynamic, 64)
  for (int64_t u = 0; u < U; ++u) {
    Shard& h = t->sh[us[u]];
    uint32_t row = ur[u];
    h.stamp[row] = t->clock;                     // updated in the step of the current batch
    if (ops & OP_LR) {
      if (t->lin_optimizer == LIN_FTRL) apply_ftrl(*t, h.lin[row], h.acc_lin[row], h.lin2[row], Gw[u]);
      else apply_opt(*t, h.lin[row], h.acc_lin[row], h.lin2[row], Gw[u]);
    }
    if (ops & (OP_FM | OP_POOL | OP_DENSE1))
      for (uint32_t c = 0; c < k; ++c)
        apply_opt(*t, h.emb[(size_t)row * k + c], h.acc_emb[(size_t)row * k + c], h.acc2_emb[(size_t)row * k + c],
                  Gv[(size_t)u * k + c]);
    if (Sw_out) Sw_out[u] = Sw[u];
    if (Sv_out) for (uint32_t c = 0; c < k; ++c) Sv_out[(size_t)u * k + c] = Sv[(size_t)u * k + c];
    if (Gw_out) Gw_out[u] = (float)Gw[u];
    if (Gv_out) for (uint32_t c = 0; c < k; ++c) Gv_out[(size_t)u * k + c] = (float)Gv[(size_t)u * k + c];
  }
  if ((ops & OP_DENSE1) && gZ && pooled) {
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < (int64_t)FK; ++i)
      for (uint32_t h2 = 0; h2 < H; ++h2) {
        double g = 0;
        for (int32_t b = 0; b < B; ++b)
          g += (double)bf16_round(pooled[(size_t)b * FK + i]) * (double)gZ[(size_t)b * H + h2];
        if (gW1_out) gW1_out[i * H + h2] = (float)g;
        apply_opt(*t, t->W1[i * H + h2], t->accW1[i * H + h2], t->acc2W1[i * H + h2], g);
      }
  }
}

// Row contents by (shard, row).  Any output may be NULL.
void orc_read_rows(void* p, int64_t n, const uint8_t* shard, const uint32_t* row,
                   uint64_t* keys, float* emb, float* lin, float* acc_emb, float* acc_lin) {
  Table* t = (Table*)p;
  const uint32_t k = t->k;
  for (int64_t i = 0; i < n; ++i) {
    const Shard& h = t->sh[shard[i]];
    uint32_t r = row[i];
    if (keys) keys[i] = h.keys[r];
    if (emb) std::memcpy(emb + (size_t)i * k, &h.emb[(size_t)r * k], k * 4);
    if (lin) lin[i] = h.lin[r];
    if (acc_emb) std::memcpy(acc_emb + (size_t)i * k, &h.acc_emb[(size_t)r * k], k * 4);
    if (acc_lin) acc_lin[i] = h.acc_lin[r];
  }
}

// Second optimizer-state word of rows given by (shard, row).
void orc_read_state2(void* p, int64_t n, const uint8_t* shard, const uint32_t* row, float* acc2_emb, float* lin2) {
  Table* t = (Table*)p;
  const uint32_t k = t->k;
  for (int64_t i = 0; i < n; ++i) {
    const Shard& h = t->sh[shard[i]];
    uint32_t r = row[i];
    if (acc2_emb) std::memcpy(acc2_emb + (size_t)i * k, &h.acc2_emb[(size_t)r * k], k * 4);
    if (lin2) lin2[i] = h.lin2[r];
  }
}

void orc_dense1_get_state2(void* p, float* acc2) {
  Table* t = (Table*)p;
  std::memcpy(acc2, t->acc2W1.data(), t->acc2W1.size() * 4);
}

// Eviction for streaming tables (Section 1, "Dynamic Features": under an endless stream the set of live
// features changes with time, so a table that can only grow would not fit any memory).  The paper's three
// table operations (Section 5) do not include a delete; reading: a key is removed from its shard, its row is
// freed, and the shard's rows stay the numbers 0 .. n-1 by moving the surviving rows that lie beyond the
// shard's new size into the freed rows below it — the i-th freed row (ascending) takes the i-th such survivor
// (ascending).  Rows that are not moved keep their numbers.  A removed key looks up as "no row"; inserting
// it again makes a new key of it (fresh initial weights).
static int64_t evict_rows(Table* t, uint32_t s, const std::vector<uint8_t>& dead) {
  Shard& h = t->sh[s];
  const uint32_t n = (uint32_t)h.keys.size(), k = t->k;
  uint32_t e = 0;
  for (uint32_t r = 0; r < n; ++r) e += dead[r];
  if (!e) return 0;
  const uint32_t m = n - e;
  std::vector<uint32_t> holes, movers;
  for (uint32_t r = 0; r < m; ++r) if (dead[r]) holes.push_back(r);
  for (uint32_t r = m; r < n; ++r) if (!dead[r]) movers.push_back(r);
  for (uint32_t r = 0; r < n; ++r) if (dead[r]) h.map.erase(h.keys[r]);
  for (size_t i = 0; i < holes.size(); ++i) {
    const uint32_t to = holes[i], from = movers[i];
    h.keys[to] = h.keys[from];
    h.map[h.keys[to]] = to;
    std::memcpy(&h.emb[(size_t)to * k], &h.emb[(size_t)from * k], k * 4);
    std::memcpy(&h.acc_emb[(size_t)to * k], &h.acc_emb[(size_t)from * k], k * 4);
    std::memcpy(&h.acc2_emb[(size_t)to * k], &h.acc2_emb[(size_t)from * k], k * 4);
    h.lin[to] = h.lin[from]; h.acc_lin[to] = h.acc_lin[from]; h.lin2[to] = h.lin2[from]; h.stamp[to] = h.stamp[from];
  }
  h.keys.resize(m); h.lin.resize(m); h.acc_lin.resize(m); h.lin2.resize(m); h.stamp.resize(m);
  h.emb.resize((size_t)m * k); h.acc_emb.resize((size_t)m * k); h.acc2_emb.resize((size_t)m * k);
  return e;
}

// Removes the listed keys (keys that are not in the table, or listed twice, count once or not at all).
// Under the FIELD partition a key may live in several shards (one per field that uses it): all go.
int64_t orc_evict_keys(void* p, const uint64_t* keys, int64_t n) {
  Table* t = (Table*)p;
  int64_t total = 0;
  for (uint32_t s = 0; s < t->S; ++s) {
    Shard& h = t->sh[s];
    std::vector<uint8_t> dead(h.keys.size(), 0);
    for (int64_t i = 0; i < n; ++i) {
      if (t->partition == PART_HASH && (uint32_t)(mix64(keys[i]) % t->S) != s) continue;
      auto it = h.map.find(keys[i]);
      if (it != h.map.end()) dead[it->second] = 1;
    }
    total += evict_rows(t, s, dead);
  }
  return total;
}

// Removes every key that was neither inserted nor updated since the table's clock showed min_clock.
int64_t orc_evict_stale(void* p, uint64_t min_clock) {
  Table* t = (Table*)p;
  int64_t total = 0;
  for (uint32_t s = 0; s < t->S; ++s) {
    Shard& h = t->sh[s];
    std::vector<uint8_t> dead(h.keys.size(), 0);
    for (size_t r = 0; r < h.keys.size(); ++r) dead[r] = h.stamp[r] < min_clock;
    total += evict_rows(t, s, dead);
  }
  return total;
}

uint64_t orc_clock(void* p) { return ((Table*)p)->clock; }

// A fixed read-out that stands for the rest of the model (the layers above the first FC layer in Section
// 4.3 / Fig. 4, which the sparse path does not contain): it turns the aggregated results into one logit
// per sample and the log loss into upstream gradients, so that multi-step runs are closed loops.  Nothing
// in it is trained; b0, c_lr, c_fm, u[H], b1[H], q[F*k], d[n_dense] are seeded constants.
//   logit = b0 + c_lr R_lr + c_fm fm2 + <u, relu(Z + b1)> + <q, pooled> + <d, xdense>
//           (each term only when its input pointer is given)
//   p = 1 / (1 + exp(-logit));  loss_b = -(y log p + (1 - y) log(1 - p));  L = mean_b loss_b
//   g = dL/dlogit = (p - y) / B;  gL = c_lr g;  gF = c_fm g;  gZ = g u (Z + b1 > 0);  gE = g q
// The paper fixes none of this: parity unpinned by the paper; pinned against the library's
// binary_cross_entropy_with_logits and autograd in the tests.
void orc_head(int64_t B, int64_t H, int64_t FK, int64_t nd, double b0, double c_lr, double c_fm,
              const float* u, const float* b1, const float* q, const float* d,
              const double* R_lr, const double* fm2, const double* Z, const double* pooled, const float* xdense,
              const float* y, double* logit, double* loss, double* gL, double* gF, double* gZ, double* gE) {
  for (int64_t b = 0; b < B; ++b) {
    double z = b0;
    if (R_lr) z += c_lr * R_lr[b];
    if (fm2) z += c_fm * fm2[b];
    if (Z) for (int64_t h = 0; h < H; ++h) { double a = Z[b * H + h] + (double)b1[h]; if (a > 0) z += (double)u[h] * a; }
    if (pooled) for (int64_t i = 0; i < FK; ++i) z += (double)q[i] * pooled[b * FK + i];
    if (xdense) for (int64_t i = 0; i < nd; ++i) z += (double)d[i] * (double)xdense[b * nd + i];
    // log(1 + exp(-|z|)) + max(-z, 0) = -log sigmoid(z), without overflow
    const double sp_neg = std::log1p(std::exp(-std::fabs(z))) + (z < 0 ? -z : 0.0);   // -log p
    const double sp_pos = sp_neg + z;                                                   // -log (1 - p)
    const double yy = (double)y[b], p = 1.0 / (1.0 + std::exp(-z));
    logit[b] = z;
    loss[b] = yy * sp_neg + (1.0 - yy) * sp_pos;
    const double g = (p - yy) / (double)B;
    if (gL) gL[b] = c_lr * g;
    if (gF) gF[b] = c_fm * g;
    if (gZ) for (int64_t h = 0; h < H; ++h) gZ[b * H + h] = (Z[b * H + h] + (double)b1[h] > 0) ? g * (double)u[h] : 0.0;
    if (gE) for (int64_t i = 0; i < FK; ++i) gE[b * FK + i] = g * (double)q[i];
  }
}

// Test hook: add delta to one stored weight (col < k: latent component,
// col == k: linear weight).  Used by the finite-difference pins.
void orc_poke(void* p, uint32_t shard, uint32_t row, uint32_t col, float value, int set) {
  Table* t = (Table*)p;
  Shard& h = t->sh[shard];
  float& w = (col < t->k) ? h.emb[(size_t)row * t->k + col] : h.lin[row];
  w = set ? value : w + value;
}

// DCN cross layer under DES (Section 4.4, the paragraph on DCN): the weight
// vector w is split along its long dimension d into S contiguous slices, shard
// s forms the scalar p_s = <x[slice s], w[slice s]> per sample, (+) adds the
// scalars in shard order, and  y = x0 * (+)p + b + x.  Slice s holds columns
// floor(s d / S) .. floor((s + 1) d / S) - 1.  Sabs (optional) = sum |x_i w_i|.
void orc_cross_forward(int64_t B, int64_t d, int64_t S, const float* x0, const float* x, const float* w,
                       const float* bias, double* part, double* P, double* y, double* Sabs) {
  for (int64_t b = 0; b < B; ++b) {
    double tot = 0.0, sa = 0.0;
    for (int64_t s = 0; s < S; ++s) {
      const int64_t lo = s * d / S, hi = (s + 1) * d / S;
      double ps = 0.0;
      for (int64_t i = lo; i < hi; ++i) {
        ps += (double)x[b * d + i] * (double)w[i];
        sa += std::fabs((double)x[b * d + i] * (double)w[i]);
      }
      if (part) part[s * B + b] = ps;
      tot += ps;
    }
    P[b] = tot;
    if (Sabs) Sabs[b] = sa;
    for (int64_t i = 0; i < d; ++i)
      y[b * d + i] = (double)x0[b * d + i] * tot + (double)bias[i] + (double)x[b * d + i];
  }
}

// Its backward for an upstream gradient gY: with t_b = <gY_b, x0_b> (the gradient of the
// aggregated scalar, which every shard can form by itself),
//   gx = gY + t w,   gx0 = gY P,   gw = sum_b t_b x_b,   gb = sum_b gY_b.
void orc_cross_backward(int64_t B, int64_t d, const float* x0, const float* x, const float* w, const float* P,
                        const float* gY, double* gx0, double* gx, double* gw, double* gb, double* t_out) {
  for (int64_t i = 0; i < d; ++i) { gw[i] = 0.0; gb[i] = 0.0; }
  for (int64_t b = 0; b < B; ++b) {
    double t = 0.0;
    for (int64_t i = 0; i < d; ++i) t += (double)gY[b * d + i] * (double)x0[b * d + i];
    if (t_out) t_out[b] = t;
    for (int64_t i = 0; i < d; ++i) {
      gx[b * d + i] = (double)gY[b * d + i] + t * (double)w[i];
      gx0[b * d + i] = (double)gY[b * d + i] * (double)P[b];
      gw[i] += t * (double)x[b * d + i];
      gb[i] += (double)gY[b * d + i];
    }
  }
}

}  // extern "C"
