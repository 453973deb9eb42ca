"""Seeded synthetic CTR-shaped inputs (numpy only).

This module feeds BOTH the CPU oracle and the CUDA path with identical
batches.  It contains input generation only — none of the method's
arithmetic (no table, no sub-operator, no optimizer) — and imports neither
side.

The five workloads stand in for the paper's Criteo (13 continuous + 26
categorical features, Section 6 "Dataset") and private production datasets
(~950 feature values per sample), which are not available here: shapes,
bag-length laws and Zipf-skewed id popularity follow the benchmark configs.

Batch layout (CSR over bags): bag (b, f) holds occurrences
offsets[b*F+f] .. offsets[b*F+f+1]-1 of ids[].
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace
from typing import Optional

import numpy as np

OP_LR, OP_FM, OP_POOL, OP_DENSE1 = 1, 2, 4, 8
PART_HASH, PART_FIELD = 0, 1
OPT_SGD, OPT_ADAGRAD, OPT_ADAM = 0, 1, 2
LIN_SAME, LIN_FTRL = 0, 1

_U64 = np.uint64


def fmix64(x: np.ndarray) -> np.ndarray:
    """Bijective 64-bit finaliser used ONLY to turn ranks into ids (the
    MurmurHash3 fmix64 steps).  It is deliberately not the table's mixer."""
    x = np.asarray(x, dtype=np.uint64).copy()
    with np.errstate(over="ignore"):
        x ^= x >> _U64(33)
        x *= _U64(0xFF51AFD7ED558CCD)
        x ^= x >> _U64(33)
        x *= _U64(0xC4CEB9FE1A85EC53)
        x ^= x >> _U64(33)
    return x


# ---------------------------------------------------------------------------
# Truncated Zipf sampler: P(r) ∝ r^-s, r = 1..n, by rejection-inversion
# (Hörmann & Derflinger 1996): invert the integral of the continuous hat
# h(x) = x^-s over [1.5 - 1, n + 0.5] and accept when the draw falls under
# the histogram bar of the rounded rank.  O(1) memory for any n.
# ---------------------------------------------------------------------------
def _zipf_H(x, s):
    # integral of t^-s, normalised so that H(1) = 0 (s != 1)
    return (np.power(x, 1.0 - s) - 1.0) / (1.0 - s)


def _zipf_Hinv(y, s):
    return np.power(1.0 + y * (1.0 - s), 1.0 / (1.0 - s))


def zipf_truncated(rng: np.random.Generator, s: float, n: int, size: int) -> np.ndarray:
    """`size` ranks in [1, n], int64, exactly Zipf(s) truncated to n."""
    assert s > 0 and s != 1.0 and n >= 1
    out = np.empty(size, dtype=np.int64)
    if n == 1:
        out[:] = 1
        return out
    h_x1 = _zipf_H(1.5, s) - 1.0          # H(1.5) - h(1)
    h_n = _zipf_H(n + 0.5, s)
    # shortcut width: ranks whose bar surely contains the draw
    sw = 2.0 - _zipf_Hinv(_zipf_H(2.5, s) - 2.0 ** (-s), s)
    todo = np.arange(size)
    while todo.size:
        m = todo.size
        u = h_n + rng.random(m) * (h_x1 - h_n)
        x = _zipf_Hinv(u, s)
        k = np.clip(np.rint(x), 1, n)
        acc = (k - x <= sw) | (u >= _zipf_H(k + 0.5, s) - np.power(k, -s))
        out[todo[acc]] = k[acc].astype(np.int64)
        todo = todo[~acc]
    return out


# ---------------------------------------------------------------------------
@dataclass(frozen=True)
class Workload:
    name: str
    batch: int                 # B
    fields: int                # F
    emb_dim: int               # k
    shards: int                # S
    partition: int
    optimizer: int
    ops: int
    hidden: int = 0            # H
    lr: float = 0.01
    eps: float = 1e-8
    init_acc: float = 0.0
    lin_optimizer: int = 0     # LIN_SAME: order-1 weights follow `optimizer`; LIN_FTRL
    beta1: float = 0.9
    beta2: float = 0.999
    ftrl_alpha: float = 0.05
    ftrl_beta: float = 1.0
    ftrl_l1: float = 0.0
    ftrl_l2: float = 0.0
    init_scale: float = 0.01
    steps: int = 1
    # id law
    zipf_s: float = 1.1
    vocab: int = 100_000       # per field (FIELD-style) or shared
    shared_vocab: bool = True
    bucket_fields: int = 0     # leading fields that are 64-bin bucketised N(0,1)
    # bag-length law: "uniform" (lo..hi), "onehot", "poisson1" (Poisson(lam)+1),
    # "geometric" (p, capped)
    len_law: str = "onehot"
    len_a: float = 1.0
    len_b: float = 1.0
    # streaming: probability that an occurrence is a never-seen id
    p_new: float = 0.0
    prepopulate: int = 0       # keys already in the table before step 0
    seed: int = 0

    def scaled(self, **kw) -> "Workload":
        return replace(self, **kw)


def config(i: int) -> Workload:
    """The five benchmark workloads, numbered from 1."""
    if i == 1:
        return Workload("cfg1_tiny_lr_fm", 512, 8, 8, 4, PART_HASH, OPT_SGD, OP_LR | OP_FM,
                        zipf_s=1.1, vocab=100_000, shared_vocab=True,
                        len_law="uniform", len_a=1, len_b=4, steps=1, seed=1)
    if i == 2:
        return Workload("cfg2_wide_deep", 8192, 26, 16, 8, PART_FIELD, OPT_ADAGRAD,
                        OP_LR | OP_POOL | OP_DENSE1, hidden=256,
                        zipf_s=1.05, vocab=10_000_000, shared_vocab=False,
                        len_law="onehot", steps=10, seed=2)
    if i == 3:
        return Workload("cfg3_deepfm", 16384, 39, 32, 16, PART_FIELD, OPT_ADAGRAD,
                        OP_LR | OP_FM | OP_POOL | OP_DENSE1, hidden=400,
                        zipf_s=1.1, vocab=30_000_000, shared_vocab=False, bucket_fields=13,
                        len_law="onehot", steps=20, seed=3)
    if i == 4:
        return Workload("cfg4_streaming", 65536, 30, 64, 32, PART_HASH, OPT_ADAGRAD,
                        OP_LR | OP_FM | OP_POOL,
                        zipf_s=1.1, vocab=0, shared_vocab=True,
                        len_law="poisson1", len_a=3.0, p_new=0.0625,
                        prepopulate=1_000_000, steps=100, seed=4)
    if i == 5:
        return Workload("cfg5_large_multihot", 16384, 100, 64, 64, PART_HASH, OPT_ADAGRAD,
                        OP_LR | OP_FM | OP_POOL,
                        zipf_s=1.2, vocab=200_000_000, shared_vocab=True,
                        len_law="geometric", len_a=0.05, len_b=100,
                        prepopulate=200_000_000, steps=1, seed=5)
    raise ValueError(i)


@dataclass
class Batch:
    batch: int
    fields: int
    offsets: np.ndarray          # int32 [B*F+1]
    ids: np.ndarray              # uint64 [nnz]
    vals: Optional[np.ndarray]   # float32 [nnz] or None (= all ones)

    @property
    def nnz(self) -> int:
        return int(self.ids.shape[0])


class Stream:
    """Stateful generator of the batches of one workload (state = number of
    ids seen so far, which only the streaming workload changes)."""

    def __init__(self, w: Workload, with_vals: bool = False):
        self.w = w
        self.rng = np.random.default_rng(w.seed)
        self.n_seen = int(w.prepopulate) if w.p_new > 0 else 0
        self.with_vals = with_vals

    # keys present before step 0, in insertion order, chunked
    def prepopulation_ids(self, chunk: int = 1 << 24):
        n = int(self.w.prepopulate)
        for lo in range(0, n, chunk):
            hi = min(n, lo + chunk)
            yield fmix64(np.arange(lo, hi, dtype=np.uint64))

    def _lengths(self, nbags: int) -> np.ndarray:
        w, rng = self.w, self.rng
        if w.len_law == "onehot":
            return np.ones(nbags, dtype=np.int64)
        if w.len_law == "uniform":
            return rng.integers(int(w.len_a), int(w.len_b) + 1, size=nbags, dtype=np.int64)
        if w.len_law == "poisson1":
            return rng.poisson(w.len_a, size=nbags).astype(np.int64) + 1
        if w.len_law == "geometric":
            return np.minimum(rng.geometric(w.len_a, size=nbags), int(w.len_b)).astype(np.int64)
        raise ValueError(w.len_law)

    def next_batch(self) -> Batch:
        w, rng = self.w, self.rng
        B, F = w.batch, w.fields
        lens = self._lengths(B * F)
        offsets = np.zeros(B * F + 1, dtype=np.int64)
        np.cumsum(lens, out=offsets[1:])
        nnz = int(offsets[-1])
        assert nnz < 2 ** 31
        field_of = np.repeat(np.tile(np.arange(F, dtype=np.int64), B), lens)
        if w.p_new > 0:                                   # streaming workload
            fresh = rng.random(nnz) < w.p_new
            ranks = zipf_truncated(rng, w.zipf_s, max(self.n_seen, 1), nnz) - 1
            nf = int(fresh.sum())
            ranks[fresh] = self.n_seen + np.arange(nf, dtype=np.int64)
            self.n_seen += nf
            ids = fmix64(ranks.astype(np.uint64))
        else:
            ranks = zipf_truncated(rng, w.zipf_s, w.vocab, nnz) - 1
            if w.bucket_fields:
                isb = field_of < w.bucket_fields
                x = rng.standard_normal(nnz)
                bins = np.clip(np.floor((x + 4.0) * 8.0), 0, 63).astype(np.int64)
                ranks = np.where(isb, bins, ranks)
            if w.shared_vocab:
                ids = fmix64(ranks.astype(np.uint64))
            else:
                ids = fmix64((field_of.astype(np.uint64) + _U64(1)) << _U64(40) | ranks.astype(np.uint64))
        assert not np.any(ids == _U64(0xFFFFFFFFFFFFFFFF))
        vals = None
        if self.with_vals:
            vals = rng.uniform(0.5, 1.5, size=nnz).astype(np.float32)
        return Batch(B, F, offsets.astype(np.int32), ids, vals)


def prepopulation_batch(ids: np.ndarray, fields: int) -> Batch:
    """Wraps a flat id array as one-id bags (trailing bags empty) so that a
    plain find-or-insert call inserts the ids in array order."""
    n = int(ids.shape[0])
    B = (n + fields - 1) // fields
    offsets = np.minimum(np.arange(B * fields + 1, dtype=np.int64), n).astype(np.int32)
    return Batch(B, fields, offsets, np.ascontiguousarray(ids, dtype=np.uint64), None)


def upstream_grads(w: Workload, batch: int, step: int, std: float = 1.0):
    """Seeded stand-ins for what the rest of the model sends back:
    gL [B], gF [B], gE [B][F*k], gZ [B][H] (float32)."""
    rng = np.random.default_rng([w.seed, 7919, step])
    g = {
        "gL": (rng.standard_normal(batch) * std).astype(np.float32),
        "gF": (rng.standard_normal(batch) * std).astype(np.float32),
        "gE": (rng.standard_normal((batch, w.fields * w.emb_dim)) * std).astype(np.float32),
    }
    if w.hidden:
        g["gZ"] = (rng.standard_normal((batch, w.hidden)) * std).astype(np.float32)
    return g


def dense1_weights(w: Workload) -> np.ndarray:
    """Seeded first-layer weights W1 [F*k][H] (float32), Glorot-like scale."""
    rng = np.random.default_rng([w.seed, 104729])
    K = w.fields * w.emb_dim
    return (rng.standard_normal((K, w.hidden)) / np.sqrt(K)).astype(np.float32)


def head_constants(w: Workload, n_dense: int = 0):
    """Seeded constants of the fixed read-out that closes the loop in multi-step runs (not trained):
    b0, c_lr, c_fm, u [H], b1 [H], q [F*k], d [n_dense], float32.  Scales are chosen from the workload's shape
    so that the logit of the first step is of order one (c_fm shrinks with the square of the number of ids
    per sample, which is how the order-2 term grows when a hot id repeats)."""
    rng = np.random.default_rng([w.seed, 15485863])
    K = w.fields * w.emb_dim
    mean_len = {"onehot": 1.0, "uniform": 0.5 * (w.len_a + w.len_b), "poisson1": w.len_a + 1.0,
                "geometric": min(1.0 / max(w.len_a, 1e-9), w.len_b)}[w.len_law]
    n_occ = w.fields * mean_len
    hc = {"b0": np.float32(-1.0), "c_lr": np.float32(1.0),
          "c_fm": np.float32(1.0 / (1.0 + 0.01 * n_occ * n_occ * w.emb_dim * w.init_scale ** 2)),
          "u": None, "b1": None, "q": None, "d": None}
    if w.hidden:
        hc["u"] = (rng.standard_normal(w.hidden) / np.sqrt(w.hidden)).astype(np.float32)
        hc["b1"] = (0.1 * rng.standard_normal(w.hidden)).astype(np.float32)
    elif w.ops & OP_POOL:
        hc["q"] = (rng.standard_normal(K) / (np.sqrt(K) * max(w.init_scale * np.sqrt(mean_len), 1e-6))).astype(np.float32)
    if n_dense:
        hc["d"] = (rng.standard_normal(n_dense) / np.sqrt(n_dense)).astype(np.float32)
    return hc


def labels(w: Workload, batch: int, step: int, p: float = 0.25) -> np.ndarray:
    """Seeded Bernoulli(p) click labels, float32 [B]."""
    rng = np.random.default_rng([w.seed, 32452843, step])
    return (rng.random(batch) < p).astype(np.float32)


def dense_features(w: Workload, batch: int, step: int, n_dense: int) -> np.ndarray:
    """Seeded N(0, 1) continuous features [B][n_dense], float32 (the 13 continuous Criteo columns)."""
    rng = np.random.default_rng([w.seed, 49979687, step])
    return rng.standard_normal((batch, n_dense)).astype(np.float32)
