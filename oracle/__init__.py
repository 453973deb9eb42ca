"""ctypes front end of the CPU oracle (test infrastructure, never used by the
product path).  `build()` compiles des_oracle.cpp with g++; `Oracle` wraps one
table.  Arrays are numpy; floating-point results come back as float64."""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "des_oracle.cpp")
_LIB = os.path.join(_HERE, "libdes_oracle.so")
_LIB_OMP = os.path.join(_HERE, "libdes_oracle_omp.so")   # the same source with -fopenmp (all host cores)
_lib = None
_lib_omp = None

ROW_NONE = 0xFFFFFFFF


def build(force: bool = False, omp: bool = False) -> str:
    """Compiles the oracle: the plain sequential build (the parity oracle) or, with omp=True, the same
    source with -fopenmp (used only to time the oracle on all host cores)."""
    out = _LIB_OMP if omp else _LIB
    if force or not os.path.exists(out) or os.path.getmtime(out) < os.path.getmtime(_SRC):
        subprocess.check_call(["g++", "-O2", "-std=c++17", "-ffp-contract=off", "-fPIC", "-shared"]
                              + (["-fopenmp"] if omp else []) + ["-o", out, _SRC])
    return out


def _p(a, t):
    if a is None:
        return None
    return a.ctypes.data_as(C.POINTER(t))


def lib(omp: bool = False):
    global _lib, _lib_omp
    if omp:
        if _lib_omp is None:
            _lib_omp = _declare(C.CDLL(build(omp=True)))
        return _lib_omp
    if _lib is None:
        _lib = _declare(C.CDLL(build()))
    return _lib


def _declare(L):
    L.orc_mix64.restype = C.c_uint64
    L.orc_mix64.argtypes = [C.c_uint64]
    L.orc_init_value.restype = C.c_float
    L.orc_init_value.argtypes = [C.c_uint64, C.c_uint64, C.c_uint32, C.c_float]
    L.orc_bf16_round.restype = C.c_float
    L.orc_bf16_round.argtypes = [C.c_float]
    L.orc_create.restype = C.c_void_p
    L.orc_create.argtypes = [C.c_uint32] * 6 + [C.c_uint64] + [C.c_float] * 4
    L.orc_destroy.argtypes = [C.c_void_p]
    L.orc_find_or_insert.restype = C.c_int64
    L.orc_evict_keys.restype = C.c_int64
    L.orc_evict_stale.restype = C.c_int64
    L.orc_clock.restype = C.c_uint64
    for name in ("orc_dense1_set", "orc_dense1_get", "orc_size", "orc_find_or_insert",
                 "orc_forward_original", "orc_fm_pairs", "orc_forward_partials", "orc_aggregate",
                 "orc_backward_update", "orc_read_rows", "orc_poke", "orc_philox4x32_10",
                 "orc_shard_of_many", "orc_comm_saving", "orc_set_opt", "orc_read_state2",
                 "orc_dense1_get_state2"):
        getattr(L, name).argtypes = None
    return L


def num_threads(omp: bool = False) -> int:
    """Threads the oracle's parallel loops use: 1 for the plain build, the OpenMP default for the other."""
    return int(lib(omp).orc_num_threads())


def mix64(x: int) -> int:
    return int(lib().orc_mix64(C.c_uint64(x)))


def philox4x32_10(ctr, key):
    c = (C.c_uint32 * 4)(*ctr)
    k = (C.c_uint32 * 2)(*key)
    o = (C.c_uint32 * 4)()
    lib().orc_philox4x32_10(c, k, o)
    return [int(v) for v in o]


def init_value(seed: int, key: int, c: int, scale: float) -> np.float32:
    return np.float32(lib().orc_init_value(seed, key, c, C.c_float(scale)))


def bf16_round(x: float) -> float:
    return float(lib().orc_bf16_round(C.c_float(x)))


def shard_of_many(ids: np.ndarray, S: int) -> np.ndarray:
    ids = np.ascontiguousarray(ids, dtype=np.uint64)
    out = np.empty(ids.shape[0], dtype=np.uint8)
    lib().orc_shard_of_many(_p(ids, C.c_uint64), C.c_int64(ids.shape[0]), C.c_uint32(S), _p(out, C.c_uint8))
    return out


def comm_saving(B, U, k, H, S_W):
    out = np.zeros(3)
    lib().orc_comm_saving(C.c_int64(B), C.c_int64(U), C.c_int64(k), C.c_int64(H), C.c_double(S_W),
                          _p(out, C.c_double))
    return out


def cross_forward(x0, x, w, bias, S):
    """DCN cross layer under DES -> dict(part [S][B], P [B], y [B][d], Sabs [B]) in float64."""
    x0 = np.ascontiguousarray(x0, np.float32); x = np.ascontiguousarray(x, np.float32)
    w = np.ascontiguousarray(w, np.float32); bias = np.ascontiguousarray(bias, np.float32)
    B, d = x.shape
    part = np.zeros((S, B)); P = np.zeros(B); y = np.zeros((B, d)); sabs = np.zeros(B)
    lib().orc_cross_forward(C.c_int64(B), C.c_int64(d), C.c_int64(S), _p(x0, C.c_float), _p(x, C.c_float),
                            _p(w, C.c_float), _p(bias, C.c_float), _p(part, C.c_double), _p(P, C.c_double),
                            _p(y, C.c_double), _p(sabs, C.c_double))
    return dict(part=part, P=P, y=y, Sabs=sabs)


def cross_backward(x0, x, w, P, gY):
    """-> dict(gx0, gx [B][d], gw, gb [d], t [B]) in float64."""
    x0 = np.ascontiguousarray(x0, np.float32); x = np.ascontiguousarray(x, np.float32)
    w = np.ascontiguousarray(w, np.float32); P = np.ascontiguousarray(P, np.float32)
    gY = np.ascontiguousarray(gY, np.float32)
    B, d = x.shape
    gx0 = np.zeros((B, d)); gx = np.zeros((B, d)); gw = np.zeros(d); gb = np.zeros(d); t = np.zeros(B)
    lib().orc_cross_backward(C.c_int64(B), C.c_int64(d), _p(x0, C.c_float), _p(x, C.c_float), _p(w, C.c_float),
                             _p(P, C.c_float), _p(gY, C.c_float), _p(gx0, C.c_double), _p(gx, C.c_double),
                             _p(gw, C.c_double), _p(gb, C.c_double), _p(t, C.c_double))
    return dict(gx0=gx0, gx=gx, gw=gw, gb=gb, t=t)


def head(hc, R_lr=None, fm2=None, Z=None, pooled=None, xdense=None, y=None):
    """The fixed read-out (see des_oracle.cpp: orc_head).  hc: dict(b0, c_lr, c_fm, u, b1, q, d) of float32
    constants; inputs float64 (the oracle's aggregates) except xdense / y (float32).  Terms whose input is
    None are left out.  -> dict(logit, loss [B], gL, gF, gZ, gE) in float64 (None where not applicable)."""
    B = int(y.shape[0])
    f64 = lambda a: None if a is None else np.ascontiguousarray(a, dtype=np.float64)
    f32 = lambda a: None if a is None else np.ascontiguousarray(a, dtype=np.float32)
    R_lr, fm2, Z, pooled = map(f64, (R_lr, fm2, Z, pooled))
    xdense, y = f32(xdense), f32(y)
    u, b1, q, d = f32(hc.get("u")), f32(hc.get("b1")), f32(hc.get("q")), f32(hc.get("d"))
    H = 0 if Z is None else Z.shape[1]
    FK = 0 if pooled is None else pooled.shape[1]
    nd = 0 if xdense is None else xdense.shape[1]
    logit = np.zeros(B); loss = np.zeros(B)
    gL = np.zeros(B) if R_lr is not None else None
    gF = np.zeros(B) if fm2 is not None else None
    gZ = np.zeros((B, H)) if Z is not None else None
    gE = np.zeros((B, FK)) if pooled is not None else None
    lib().orc_head(C.c_int64(B), C.c_int64(H), C.c_int64(FK), C.c_int64(nd), C.c_double(float(hc["b0"])),
                   C.c_double(float(hc["c_lr"])), C.c_double(float(hc["c_fm"])), _p(u, C.c_float), _p(b1, C.c_float),
                   _p(q, C.c_float), _p(d, C.c_float), _p(R_lr, C.c_double), _p(fm2, C.c_double), _p(Z, C.c_double),
                   _p(pooled, C.c_double), _p(xdense, C.c_float), _p(y, C.c_float), _p(logit, C.c_double),
                   _p(loss, C.c_double), _p(gL, C.c_double), _p(gF, C.c_double), _p(gZ, C.c_double), _p(gE, C.c_double))
    return dict(logit=logit, loss=loss, gL=gL, gF=gF, gZ=gZ, gE=gE)


class Oracle:
    def __init__(self, S, F, k, H=0, partition=0, optimizer=0, seed=0, init_scale=0.01,
                 lr=0.01, eps=1e-8, init_acc=0.0, omp=False):
        self.S, self.F, self.k, self.H = S, F, k, H
        self.L = lib(omp)
        self.h = C.c_void_p(self.L.orc_create(S, F, k, H, partition, optimizer, C.c_uint64(seed),
                                              C.c_float(init_scale), C.c_float(lr), C.c_float(eps),
                                              C.c_float(init_acc)))

    def set_opt(self, lin_optimizer=0, beta1=0.9, beta2=0.999, ftrl_alpha=0.05, ftrl_beta=1.0, ftrl_l1=0.0,
                ftrl_l2=0.0):
        """Optimizer settings beyond the constructor's; call before the first insert."""
        self.L.orc_set_opt(self.h, C.c_uint32(lin_optimizer), C.c_float(beta1), C.c_float(beta2),
                           C.c_float(ftrl_alpha), C.c_float(ftrl_beta), C.c_float(ftrl_l1), C.c_float(ftrl_l2))

    @classmethod
    def for_workload(cls, w, omp=False):
        o = cls(w.shards, w.fields, w.emb_dim, w.hidden, w.partition, w.optimizer, w.seed,
                w.init_scale, w.lr, w.eps, w.init_acc, omp=omp)
        o.set_opt(getattr(w, "lin_optimizer", 0), getattr(w, "beta1", 0.9), getattr(w, "beta2", 0.999),
                  getattr(w, "ftrl_alpha", 0.05), getattr(w, "ftrl_beta", 1.0), getattr(w, "ftrl_l1", 0.0),
                  getattr(w, "ftrl_l2", 0.0))
        return o

    def close(self):
        if self.h:
            self.L.orc_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- table ---------------------------------------------------------------
    def size(self):
        out = np.zeros(self.S, dtype=np.uint64)
        self.L.orc_size(self.h, _p(out, C.c_uint64))
        return out

    # -- eviction --------------------------------------------------------------
    def evict_keys(self, keys) -> int:
        keys = np.ascontiguousarray(keys, dtype=np.uint64)
        return int(self.L.orc_evict_keys(self.h, _p(keys, C.c_uint64), C.c_int64(keys.shape[0])))

    def evict_stale(self, min_clock: int) -> int:
        return int(self.L.orc_evict_stale(self.h, C.c_uint64(min_clock)))

    def clock(self) -> int:
        return int(self.L.orc_clock(self.h))

    def dense1_set(self, W1):
        W1 = np.ascontiguousarray(W1, dtype=np.float32)
        assert W1.shape == (self.F * self.k, self.H)
        self.L.orc_dense1_set(self.h, _p(W1, C.c_float))

    def dense1_get(self):
        W1 = np.empty((self.F * self.k, self.H), dtype=np.float32)
        acc = np.empty_like(W1)
        self.L.orc_dense1_get(self.h, _p(W1, C.c_float), _p(acc, C.c_float))
        return W1, acc

    def find_or_insert(self, batch, insert=True):
        """-> dict(rows, shards, uidx, uniq_shard, uniq_row, U)"""
        nnz = batch.nnz
        rows = np.empty(nnz, dtype=np.uint32)
        shards = np.empty(nnz, dtype=np.uint8)
        uidx = np.empty(nnz, dtype=np.uint32)
        us = np.empty(nnz, dtype=np.uint8)
        ur = np.empty(nnz, dtype=np.uint32)
        U = self.L.orc_find_or_insert(self.h, _p(batch.offsets, C.c_int32), _p(batch.ids, C.c_uint64),
                                      C.c_int32(batch.batch), C.c_int(1 if insert else 0),
                                      _p(rows, C.c_uint32), _p(shards, C.c_uint8), _p(uidx, C.c_uint32),
                                      _p(us, C.c_uint8), _p(ur, C.c_uint32))
        return dict(rows=rows, shards=shards, uidx=uidx, uniq_shard=us[:U].copy(),
                    uniq_row=ur[:U].copy(), U=int(U))

    # -- forward ---------------------------------------------------------------
    def forward_original(self, ops, batch):
        B, k, F, H = batch.batch, self.k, self.F, self.H
        lr0 = np.zeros(B); A0 = np.zeros((B, k)); Q0 = np.zeros(B); fm2 = np.zeros(B)
        pooled0 = np.zeros((B, F * k))
        Z0 = np.zeros((B, H)) if H else None
        Sabs = np.zeros((B, k + 1))
        self.L.orc_forward_original(self.h, C.c_uint32(ops), _p(batch.offsets, C.c_int32),
                                    _p(batch.ids, C.c_uint64), _p(batch.vals, C.c_float), C.c_int32(B),
                                    _p(lr0, C.c_double), _p(A0, C.c_double), _p(Q0, C.c_double),
                                    _p(fm2, C.c_double), _p(pooled0, C.c_double), _p(Z0, C.c_double),
                                    _p(Sabs, C.c_double))
        return dict(lr=lr0, A=A0, Q=Q0, fm2=fm2, pooled=pooled0, Z=Z0, Sabs=Sabs)

    def fm_pairs(self, batch):
        out = np.zeros(batch.batch)
        self.L.orc_fm_pairs(self.h, _p(batch.offsets, C.c_int32), _p(batch.ids, C.c_uint64),
                            _p(batch.vals, C.c_float), C.c_int32(batch.batch), _p(out, C.c_double))
        return out

    def forward_partials(self, ops, batch, fi, want_pooled=True, want_dense=False):
        B, k, F, H, S = batch.batch, self.k, self.F, self.H, self.S
        ps = np.zeros((S, B, k + 2))
        pp = np.zeros((S, B, F * k)) if want_pooled else None
        pd = np.zeros((S, B, H)) if (want_dense and H) else None
        self.L.orc_forward_partials(self.h, C.c_uint32(ops), _p(batch.offsets, C.c_int32),
                                    _p(batch.vals, C.c_float), _p(fi["rows"], C.c_uint32),
                                    _p(fi["shards"], C.c_uint8), C.c_int32(B),
                                    _p(ps, C.c_double), _p(pp, C.c_double), _p(pd, C.c_double))
        return dict(part_small=ps, part_pooled=pp, part_dense=pd)

    def aggregate(self, B, part):
        k, F, H = self.k, self.F, self.H
        out_small = np.zeros((B, k + 3))
        pooled = np.zeros((B, F * k)) if part["part_pooled"] is not None else None
        Z = np.zeros((B, H)) if part["part_dense"] is not None else None
        self.L.orc_aggregate(self.h, C.c_int32(B), _p(part["part_small"], C.c_double),
                             _p(part["part_pooled"], C.c_double), _p(part["part_dense"], C.c_double),
                             _p(out_small, C.c_double), _p(pooled, C.c_double), _p(Z, C.c_double))
        return dict(out_small=out_small, A=out_small[:, :k], lr=out_small[:, k], fm2=out_small[:, k + 1],
                    Q=out_small[:, k + 2], pooled=pooled, Z=Z)

    # -- backward ----------------------------------------------------------------
    def backward_update(self, ops, batch, fi, A, pooled=None, gL=None, gF=None, gE=None, gZ=None):
        """A, pooled: float32 aggregated forward results.  Returns the summed
        per-unique-key gradients (float32) and the total pooled gradient."""
        B, k, F = batch.batch, self.k, self.F
        U = fi["U"]
        f32 = lambda a: None if a is None else np.ascontiguousarray(a, dtype=np.float32)
        A, pooled, gL, gF, gE, gZ = map(f32, (A, pooled, gL, gF, gE, gZ))
        Gw = np.zeros(U, dtype=np.float32)
        Gv = np.zeros((U, k), dtype=np.float32)
        gEt = np.zeros((B, F * k), dtype=np.float32)
        Sw = np.zeros(U); Sv = np.zeros((U, k))
        gW1 = np.zeros((F * k, self.H), dtype=np.float32) if (self.H and gZ is not None) else None
        self.L.orc_backward_update(self.h, C.c_uint32(ops), _p(batch.offsets, C.c_int32),
                                   _p(batch.vals, C.c_float), _p(fi["rows"], C.c_uint32),
                                   _p(fi["shards"], C.c_uint8), _p(fi["uidx"], C.c_uint32),
                                   C.c_int32(B), C.c_int64(U), _p(A, C.c_float), _p(pooled, C.c_float),
                                   _p(gL, C.c_float), _p(gF, C.c_float), _p(gE, C.c_float), _p(gZ, C.c_float),
                                   _p(Gw, C.c_float), _p(Gv, C.c_float), _p(gEt, C.c_float),
                                   _p(Sw, C.c_double), _p(Sv, C.c_double), _p(gW1, C.c_float))
        return dict(Gw=Gw, Gv=Gv, gE_total=gEt, Sw=Sw, Sv=Sv, gW1=gW1)

    def read_rows(self, shard, row):
        shard = np.ascontiguousarray(shard, dtype=np.uint8)
        row = np.ascontiguousarray(row, dtype=np.uint32)
        n, k = shard.shape[0], self.k
        keys = np.empty(n, dtype=np.uint64)
        emb = np.empty((n, k), dtype=np.float32); lin = np.empty(n, dtype=np.float32)
        ae = np.empty((n, k), dtype=np.float32); al = np.empty(n, dtype=np.float32)
        self.L.orc_read_rows(self.h, C.c_int64(n), _p(shard, C.c_uint8), _p(row, C.c_uint32),
                             _p(keys, C.c_uint64), _p(emb, C.c_float), _p(lin, C.c_float),
                             _p(ae, C.c_float), _p(al, C.c_float))
        return dict(keys=keys, emb=emb, lin=lin, acc_emb=ae, acc_lin=al)

    def read_state2(self, shard, row):
        shard = np.ascontiguousarray(shard, dtype=np.uint8)
        row = np.ascontiguousarray(row, dtype=np.uint32)
        n, k = shard.shape[0], self.k
        a2 = np.empty((n, k), dtype=np.float32); l2 = np.empty(n, dtype=np.float32)
        self.L.orc_read_state2(self.h, C.c_int64(n), _p(shard, C.c_uint8), _p(row, C.c_uint32),
                               _p(a2, C.c_float), _p(l2, C.c_float))
        return dict(acc2_emb=a2, lin2=l2)

    def dense1_get_state2(self):
        a2 = np.empty((self.F * self.k, self.H), dtype=np.float32)
        self.L.orc_dense1_get_state2(self.h, _p(a2, C.c_float))
        return a2

    def poke(self, shard, row, col, value, set_=False):
        self.L.orc_poke(self.h, C.c_uint32(shard), C.c_uint32(row), C.c_uint32(col), C.c_float(value),
                        C.c_int(1 if set_ else 0))
