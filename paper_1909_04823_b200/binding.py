"""Thin ctypes binding of libdes.so — argument marshalling only.

Every step of the path runs in the library's CUDA kernels; torch is used for
device memory and streams.  If the library cannot be loaded this module raises:
there is no CPU fallback."""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional

import torch

from . import build as _build

OP_LR, OP_FM, OP_POOL, OP_DENSE1 = 1, 2, 4, 8
FUSED_SHARD_ORDER = 16        # des_forward_fused: keep the shard-by-shard form
PART_HASH, PART_FIELD = 0, 1
OPT_SGD, OPT_ADAGRAD, OPT_ADAM = 0, 1, 2
LIN_SAME, LIN_FTRL = 0, 1
ROW_NONE = 0xFFFFFFFF
KEY_EMPTY = 0xFFFFFFFFFFFFFFFF

STATUS = {0: "DES_OK", 1: "DES_ERR_INVALID_ARG", 2: "DES_ERR_RESERVED_KEY", 3: "DES_ERR_CAPACITY",
          4: "DES_ERR_UNSUPPORTED", 5: "DES_ERR_CUDA", 6: "DES_ERR_NOT_FOUND",
          7: "DES_ERR_TOO_LARGE", 8: "DES_ERR_RANGE"}

EXPORTS = ["des_table_create", "des_table_destroy", "des_find_or_insert", "des_forward_partials",
           "des_aggregate", "des_rank_partial", "des_aggregate_ranks", "des_forward_fused", "des_backward_update", "des_dense1_set", "des_dense1_get", "des_dense1_get_state", "des_dense1_set_state", "des_dense1_forward_noalloc", "des_table_status",
           "des_table_size", "des_table_row_base", "des_table_export", "des_table_read_rows", "des_table_write_rows",
           "des_table_read_state2", "des_table_write_state2",
           "des_step_host", "des_step_host_submit", "des_step_host_wait", "des_cross_forward", "des_cross_backward",
           "des_cross_workspace_floats", "des_comm_volume", "des_profile_enable", "des_profile_read", "des_table_launch_count", "des_status_string",
           "des_build_has_tensor_cores", "des_table_uses_tensor_cores", "des_build_is_debug",
           "des_table_evict_keys", "des_table_evict_stale", "des_table_clock", "des_head"]


class des_comm_model_t(C.Structure):
    _fields_ = [("workers", C.c_int32), ("batch", C.c_int64), ("uniq", C.c_int64), ("emb_dim", C.c_int32),
                ("hidden", C.c_int32), ("key_bytes", C.c_int32), ("value_bytes", C.c_int32),
                ("first_layer_bytes", C.c_double)]


class des_comm_volume_t(C.Structure):
    _fields_ = [("q_mesh", C.c_double * 3), ("q_des", C.c_double * 3), ("saving", C.c_double * 3)]


class DesError(RuntimeError):
    def __init__(self, code, where):
        super().__init__(f"{where}: {STATUS.get(code, code)}")
        self.code = code


class des_config_t(C.Structure):
    _fields_ = [("num_shards", C.c_uint32), ("num_fields", C.c_uint32), ("emb_dim", C.c_uint32),
                ("hidden", C.c_uint32), ("partition", C.c_uint32), ("optimizer", C.c_uint32),
                ("max_rows", C.c_uint64), ("max_load", C.c_float),
                ("h_rows_per_shard", C.POINTER(C.c_uint64)),
                ("seed", C.c_uint64), ("init_scale", C.c_float),
                ("lr", C.c_float), ("eps", C.c_float), ("init_acc", C.c_float),
                ("lin_optimizer", C.c_uint32), ("beta1", C.c_float), ("beta2", C.c_float),
                ("ftrl_alpha", C.c_float), ("ftrl_beta", C.c_float), ("ftrl_l1", C.c_float), ("ftrl_l2", C.c_float),
                ("shard_world", C.c_uint32), ("shard_rank", C.c_uint32),
                ("max_nnz", C.c_int64), ("max_batch", C.c_int32), ("max_uniq", C.c_int64),
                ("alloc", C.c_void_p), ("dealloc", C.c_void_p), ("alloc_ctx", C.c_void_p)]


class des_batch_t(C.Structure):
    _fields_ = [("batch", C.c_int32), ("nnz", C.c_int64), ("offsets", C.c_void_p), ("ids", C.c_void_p),
                ("vals", C.c_void_p), ("rows", C.c_void_p), ("shards", C.c_void_p), ("uidx", C.c_void_p),
                ("uniq_rows", C.c_void_p), ("n_uniq", C.c_void_p)]


class des_partials_t(C.Structure):
    _fields_ = [("part_small", C.c_void_p), ("pooled", C.c_void_p), ("part_pooled", C.c_void_p),
                ("part_dense", C.c_void_p)]


class des_outputs_t(C.Structure):
    _fields_ = [("out_small", C.c_void_p), ("pooled", C.c_void_p), ("Z", C.c_void_p)]


class des_head_t(C.Structure):
    _fields_ = [("b0", C.c_float), ("c_lr", C.c_float), ("c_fm", C.c_float), ("u", C.c_void_p), ("b1", C.c_void_p),
                ("q", C.c_void_p), ("d", C.c_void_p), ("n_dense", C.c_int32)]


class des_head_grads_t(C.Structure):
    _fields_ = [("gL", C.c_void_p), ("gF", C.c_void_p), ("gE", C.c_void_p), ("gZ", C.c_void_p)]


class des_grads_t(C.Structure):
    _fields_ = [("gL", C.c_void_p), ("gF", C.c_void_p), ("gE", C.c_void_p), ("gZ", C.c_void_p),
                ("gE_work", C.c_void_p)]


_lib = None
_lib_debug = None
_use_debug = False


def lib_path() -> str:
    return _build.LIB_DEBUG if _use_debug else _build.LIB


def use_debug_library(on: bool = True) -> bool:
    """Tables created from now on use the checking build (libdes_debug.so: index range checks in every
    gather / scatter / probe, test hooks) instead of the product library.  Returns the previous setting."""
    global _use_debug
    prev, _use_debug = _use_debug, bool(on)
    return prev


def uses_tensor_cores() -> bool:
    """True when the loaded library carries the tcgen05 GEMMs of the first dense layer."""
    return bool(load().des_build_has_tensor_cores())


def load():
    """Loads (building first if the sources are newer) the CUDA library."""
    global _lib, _lib_debug
    if _use_debug:
        if _lib_debug is None:
            _lib_debug = _declare(C.CDLL(_build.build(debug=True)))
        return _lib_debug
    if _lib is None:
        _lib = _declare(C.CDLL(_build.build()))
    return _lib


def _declare(L):
    for name in EXPORTS:
        getattr(L, name)  # fail loudly on a missing symbol
    L.des_table_create.argtypes = [C.POINTER(des_config_t), C.POINTER(C.c_void_p)]
    L.des_table_destroy.argtypes = [C.c_void_p]
    L.des_find_or_insert.argtypes = [C.c_void_p, C.POINTER(des_batch_t), C.c_int, C.c_void_p]
    L.des_forward_partials.argtypes = [C.c_void_p, C.c_uint32, C.POINTER(des_batch_t),
                                       C.POINTER(des_partials_t), C.c_void_p]
    L.des_aggregate.argtypes = [C.c_void_p, C.c_uint32, C.POINTER(des_batch_t), C.POINTER(des_partials_t),
                                C.POINTER(des_outputs_t), C.c_void_p]
    L.des_forward_fused.argtypes = [C.c_void_p, C.c_uint32, C.POINTER(des_batch_t), C.POINTER(des_partials_t),
                                    C.POINTER(des_outputs_t), C.c_void_p]
    L.des_backward_update.argtypes = [C.c_void_p, C.c_uint32, C.POINTER(des_batch_t),
                                      C.POINTER(des_outputs_t), C.POINTER(des_grads_t), C.c_void_p]
    L.des_dense1_set.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p]
    L.des_dense1_get.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p]
    L.des_dense1_get_state.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
    L.des_dense1_set_state.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
    L.des_dense1_forward_noalloc.argtypes = [C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p]
    L.des_table_status.argtypes = [C.c_void_p]
    L.des_table_size.argtypes = [C.c_void_p, C.POINTER(C.c_uint64)]
    L.des_table_row_base.argtypes = [C.c_void_p, C.POINTER(C.c_uint64)]
    L.des_table_export.argtypes = [C.c_void_p] + [C.c_void_p] * 7 + [C.c_uint64, C.POINTER(C.c_uint64)]
    L.des_table_read_rows.argtypes = [C.c_void_p, C.c_void_p, C.c_int64] + [C.c_void_p] * 4 + [C.c_void_p]
    L.des_table_write_rows.argtypes = [C.c_void_p, C.c_void_p, C.c_int64] + [C.c_void_p] * 4 + [C.c_void_p]
    L.des_table_read_state2.argtypes = [C.c_void_p, C.c_void_p, C.c_int64, C.c_void_p, C.c_void_p, C.c_void_p]
    L.des_table_write_state2.argtypes = [C.c_void_p, C.c_void_p, C.c_int64, C.c_void_p, C.c_void_p, C.c_void_p]
    L.des_step_host.argtypes = [C.c_void_p, C.c_uint32, C.c_int32, C.c_int64, C.c_void_p, C.c_void_p,
                                C.c_void_p, C.POINTER(des_grads_t), C.c_void_p, C.c_void_p, C.c_void_p,
                                C.c_void_p]
    L.des_step_host_submit.argtypes = [C.c_void_p, C.c_uint32, C.c_int32, C.c_int64, C.c_void_p, C.c_void_p,
                                       C.c_void_p, C.POINTER(des_grads_t), C.c_void_p, C.c_void_p, C.c_void_p,
                                       C.c_void_p, C.POINTER(C.c_int32)]
    L.des_step_host_wait.argtypes = [C.c_void_p, C.c_int32]
    L.des_rank_partial.argtypes = [C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p]
    L.des_aggregate_ranks.argtypes = [C.c_void_p, C.c_uint32, C.c_int32, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p]
    L.des_cross_forward.argtypes = [C.c_int32, C.c_int32, C.c_int32] + [C.c_void_p] * 8
    L.des_cross_backward.argtypes = [C.c_int32, C.c_int32] + [C.c_void_p] * 11
    L.des_cross_workspace_floats.argtypes = [C.c_int32, C.c_int32]
    L.des_cross_workspace_floats.restype = C.c_int64
    L.des_comm_volume.argtypes = [C.POINTER(des_comm_model_t), C.POINTER(des_comm_volume_t)]
    L.des_table_launch_count.argtypes = [C.c_void_p]
    L.des_profile_enable.argtypes = [C.c_void_p, C.c_int]
    L.des_profile_read.argtypes = [C.c_void_p, C.POINTER(C.c_char_p), C.POINTER(C.c_float), C.c_int,
                                   C.POINTER(C.c_int)]
    L.des_table_launch_count.restype = C.c_uint64
    L.des_status_string.restype = C.c_char_p
    L.des_build_has_tensor_cores.argtypes = []
    L.des_table_uses_tensor_cores.argtypes = [C.c_void_p]
    L.des_build_is_debug.argtypes = []
    L.des_table_evict_keys.argtypes = [C.c_void_p, C.c_void_p, C.c_int64, C.POINTER(C.c_uint64)]
    L.des_table_evict_stale.argtypes = [C.c_void_p, C.c_uint64, C.POINTER(C.c_uint64)]
    L.des_table_clock.argtypes = [C.c_void_p, C.POINTER(C.c_uint64)]
    L.des_head.argtypes = [C.c_void_p, C.c_uint32, C.c_int32, C.POINTER(des_head_t), C.POINTER(des_outputs_t),
                           C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.POINTER(des_head_grads_t), C.c_void_p]
    return L


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


class DeviceBatch:
    """Device-resident batch plus the index arrays find_or_insert fills."""

    def __init__(self, offsets, ids, vals, batch, device="cuda"):
        as_dev = lambda a, dt: a.to(device=device, dtype=dt) if isinstance(a, torch.Tensor) else \
            torch.from_numpy(a).to(device=device, dtype=dt)
        self.batch = int(batch)
        self.offsets = as_dev(offsets, torch.int32).contiguous()
        if isinstance(ids, torch.Tensor):
            self.ids = ids.to(device).contiguous()
        else:
            self.ids = torch.from_numpy(ids.view("int64")).to(device).contiguous()
        self.vals = None if vals is None else as_dev(vals, torch.float32).contiguous()
        self.nnz = int(self.ids.numel())
        n = max(self.nnz, 1)
        self.rows = torch.empty(n, dtype=torch.int32, device=device)      # uint32 payload
        self.shards = torch.empty(n, dtype=torch.uint8, device=device)
        self.uidx = torch.empty(n, dtype=torch.int32, device=device)
        self.uniq_rows = torch.empty(n, dtype=torch.int32, device=device)
        self.n_uniq = torch.zeros(1, dtype=torch.int32, device=device)

    @classmethod
    def from_synth(cls, b, device="cuda"):
        return cls(b.offsets, b.ids, b.vals, b.batch, device)

    def c(self) -> des_batch_t:
        return des_batch_t(self.batch, self.nnz, _ptr(self.offsets), _ptr(self.ids), _ptr(self.vals),
                           _ptr(self.rows), _ptr(self.shards), _ptr(self.uidx), _ptr(self.uniq_rows),
                           _ptr(self.n_uniq))


class Table:
    """Owner of one des_table_t.  Methods have the names of the C entry points
    and only marshal arguments."""

    def __init__(self, num_shards, num_fields, emb_dim, hidden=0, partition=PART_HASH, optimizer=OPT_SGD,
                 max_rows=1 << 20, max_load=0.5, rows_per_shard=None, seed=0, init_scale=0.01, lr=0.01,
                 eps=1e-8, init_acc=0.0, max_nnz=1 << 20, max_batch=1 << 16, max_uniq=0, lin_optimizer=LIN_SAME,
                 beta1=0.9, beta2=0.999, ftrl_alpha=0.05, ftrl_beta=1.0, ftrl_l1=0.0, ftrl_l2=0.0, shard_world=0,
                 shard_rank=0):
        if not torch.cuda.is_available():
            raise RuntimeError("paper_1909_04823_b200 needs a CUDA device; there is no CPU path")
        self.L = load()
        self.S, self.F, self.k, self.H = num_shards, num_fields, emb_dim, hidden
        self.partition, self.max_nnz, self.max_batch = partition, int(max_nnz), int(max_batch)
        self.stride = emb_dim + 4
        cfg = des_config_t()
        cfg.num_shards, cfg.num_fields, cfg.emb_dim, cfg.hidden = num_shards, num_fields, emb_dim, hidden
        cfg.partition, cfg.optimizer = partition, optimizer
        cfg.max_rows, cfg.max_load = int(max_rows), max_load
        self._rps = None
        if rows_per_shard is not None:
            self._rps = (C.c_uint64 * num_shards)(*[int(v) for v in rows_per_shard])
            cfg.h_rows_per_shard = C.cast(self._rps, C.POINTER(C.c_uint64))
        cfg.seed, cfg.init_scale, cfg.lr, cfg.eps, cfg.init_acc = int(seed), init_scale, lr, eps, init_acc
        cfg.lin_optimizer, cfg.beta1, cfg.beta2 = lin_optimizer, beta1, beta2
        cfg.ftrl_alpha, cfg.ftrl_beta, cfg.ftrl_l1, cfg.ftrl_l2 = ftrl_alpha, ftrl_beta, ftrl_l1, ftrl_l2
        cfg.shard_world, cfg.shard_rank = shard_world, shard_rank
        cfg.max_nnz, cfg.max_batch, cfg.max_uniq = int(max_nnz), int(max_batch), int(max_uniq)
        self.h = C.c_void_p()
        self._check(self.L.des_table_create(C.byref(cfg), C.byref(self.h)), "des_table_create")

    @classmethod
    def for_workload(cls, w, max_rows, max_nnz, max_batch=None, rows_per_shard=None, max_uniq=0, max_load=0.5,
                     shard_world=0, shard_rank=0):
        return cls(w.shards, w.fields, w.emb_dim, w.hidden, w.partition, w.optimizer, max_rows=max_rows,
                   max_load=max_load, rows_per_shard=rows_per_shard, seed=w.seed, init_scale=w.init_scale,
                   lr=w.lr, eps=w.eps, init_acc=w.init_acc, lin_optimizer=w.lin_optimizer, beta1=w.beta1,
                   beta2=w.beta2, ftrl_alpha=w.ftrl_alpha, ftrl_beta=w.ftrl_beta, ftrl_l1=w.ftrl_l1,
                   ftrl_l2=w.ftrl_l2, max_nnz=max_nnz,
                   max_batch=max_batch or w.batch, max_uniq=max_uniq, shard_world=shard_world, shard_rank=shard_rank)

    def _check(self, code, where):
        if code != 0:
            raise DesError(code, where)

    def close(self):
        if getattr(self, "h", None) and self.h.value:
            self.L.des_table_destroy(self.h)
            self.h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- the five calls of the path -------------------------------------------
    def find_or_insert(self, batch: DeviceBatch, insert: bool = True):
        cb = batch.c()
        self._check(self.L.des_find_or_insert(self.h, C.byref(cb), 1 if insert else 0, _stream()),
                    "des_find_or_insert")

    def forward_partials(self, ops, batch, part_small=None, pooled=None, part_pooled=None, part_dense=None):
        cb = batch.c()
        p = des_partials_t(_ptr(part_small), _ptr(pooled), _ptr(part_pooled), _ptr(part_dense))
        self._check(self.L.des_forward_partials(self.h, ops, C.byref(cb), C.byref(p), _stream()),
                    "des_forward_partials")

    def aggregate(self, ops, batch, part_small=None, pooled=None, part_pooled=None, part_dense=None,
                  out_small=None, out_pooled=None, Z=None):
        cb = batch.c()
        p = des_partials_t(_ptr(part_small), _ptr(pooled), _ptr(part_pooled), _ptr(part_dense))
        o = des_outputs_t(_ptr(out_small), _ptr(out_pooled if out_pooled is not None else pooled), _ptr(Z))
        self._check(self.L.des_aggregate(self.h, ops, C.byref(cb), C.byref(p), C.byref(o), _stream()),
                    "des_aggregate")

    def forward_fused(self, ops, batch, part_small=None, pooled=None, out_small=None, Z=None):
        cb = batch.c()
        p = des_partials_t(_ptr(part_small), _ptr(pooled), None, None)
        o = des_outputs_t(_ptr(out_small), _ptr(pooled), _ptr(Z))
        self._check(self.L.des_forward_fused(self.h, ops, C.byref(cb), C.byref(p), C.byref(o), _stream()),
                    "des_forward_fused")

    def backward_update(self, ops, batch, out_small=None, pooled=None, Z=None, gL=None, gF=None, gE=None,
                        gZ=None, gE_work=None):
        cb = batch.c()
        o = des_outputs_t(_ptr(out_small), _ptr(pooled), _ptr(Z))
        g = des_grads_t(_ptr(gL), _ptr(gF), _ptr(gE), _ptr(gZ), _ptr(gE_work))
        self._check(self.L.des_backward_update(self.h, ops, C.byref(cb), C.byref(o), C.byref(g), _stream()),
                    "des_backward_update")

    def step_host(self, ops, batch_size, nnz, h_offsets, h_ids, h_vals, h_out_small, d_pooled=None, d_Z=None,
                  gL=None, gF=None, gE=None, gZ=None, gE_work=None):
        g = des_grads_t(_ptr(gL), _ptr(gF), _ptr(gE), _ptr(gZ), _ptr(gE_work))
        self._check(self.L.des_step_host(self.h, ops, batch_size, nnz, _ptr(h_offsets), _ptr(h_ids),
                                         _ptr(h_vals), C.byref(g), _ptr(d_pooled), _ptr(d_Z),
                                         _ptr(h_out_small), _stream()), "des_step_host")

    # -- (+) across processes -----------------------------------------------------------
    def rank_partial(self, batch_size: int, part_small: torch.Tensor, rank_part: torch.Tensor):
        self._check(self.L.des_rank_partial(self.h, batch_size, _ptr(part_small), _ptr(rank_part), _stream()),
                    "des_rank_partial")

    def aggregate_ranks(self, ops: int, batch_size: int, world: int, rank_parts: torch.Tensor, out_small: torch.Tensor):
        self._check(self.L.des_aggregate_ranks(self.h, ops, batch_size, world, _ptr(rank_parts), _ptr(out_small),
                                               _stream()), "des_aggregate_ranks")

    def step_host_submit(self, ops, batch_size, nnz, h_offsets, h_ids, h_vals, h_out_small, d_pooled=None, d_Z=None,
                         gL=None, gF=None, gE=None, gZ=None, gE_work=None) -> int:
        """Pipelined des_step_host: returns a ticket for step_host_wait."""
        g = des_grads_t(_ptr(gL), _ptr(gF), _ptr(gE), _ptr(gZ), _ptr(gE_work))
        ticket = C.c_int32(-1)
        self._check(self.L.des_step_host_submit(self.h, ops, batch_size, nnz, _ptr(h_offsets), _ptr(h_ids),
                                                _ptr(h_vals), C.byref(g), _ptr(d_pooled), _ptr(d_Z),
                                                _ptr(h_out_small), _stream(), C.byref(ticket)), "des_step_host_submit")
        return int(ticket.value)

    def step_host_wait(self, ticket: int):
        self._check(self.L.des_step_host_wait(self.h, ticket), "des_step_host_wait")

    # -- first dense layer ----------------------------------------------------------
    def dense1_set(self, W1: torch.Tensor):
        assert W1.is_cuda and W1.dtype == torch.float32 and W1.shape == (self.F * self.k, self.H)
        self._check(self.L.des_dense1_set(self.h, _ptr(W1.contiguous()), _stream()), "des_dense1_set")
        torch.cuda.current_stream().synchronize()

    def dense1_get(self) -> torch.Tensor:
        W1 = torch.empty((self.F * self.k, self.H), dtype=torch.float32, device="cuda")
        self._check(self.L.des_dense1_get(self.h, _ptr(W1), _stream()), "des_dense1_get")
        return W1

    # -- inspection -------------------------------------------------------------------
    def status(self) -> int:
        return int(self.L.des_table_status(self.h))

    def check_status(self):
        self._check(self.status(), "des_table_status")

    def size(self):
        out = (C.c_uint64 * self.S)()
        self._check(self.L.des_table_size(self.h, out), "des_table_size")
        return [int(v) for v in out]

    def row_base(self):
        out = (C.c_uint64 * (self.S + 1))()
        self._check(self.L.des_table_row_base(self.h, out), "des_table_row_base")
        return [int(v) for v in out]

    def head(self, ops, batch_size, hc, out_small=None, pooled=None, Z=None, xdense=None, y=None, logit=None, loss=None,
             gL=None, gF=None, gE=None, gZ=None):
        """hc: dict(b0, c_lr, c_fm, u, b1, q, d) with device tensors (or None) for the vectors."""
        h = des_head_t(float(hc["b0"]), float(hc["c_lr"]), float(hc["c_fm"]), _ptr(hc.get("u")), _ptr(hc.get("b1")),
                       _ptr(hc.get("q")), _ptr(hc.get("d")), 0 if hc.get("d") is None else int(hc["d"].numel()))
        o = des_outputs_t(_ptr(out_small), _ptr(pooled), _ptr(Z))
        g = des_head_grads_t(_ptr(gL), _ptr(gF), _ptr(gE), _ptr(gZ))
        self._check(self.L.des_head(self.h, ops, int(batch_size), C.byref(h), C.byref(o), _ptr(xdense), _ptr(y),
                                    _ptr(logit), _ptr(loss), C.byref(g), _stream()), "des_head")

    def evict_keys(self, keys: torch.Tensor) -> int:
        """keys: int64 / uint64 device tensor of ids to remove.  Returns the number of rows removed."""
        n = C.c_uint64(0)
        self._check(self.L.des_table_evict_keys(self.h, _ptr(keys), int(keys.numel()), C.byref(n)), "des_table_evict_keys")
        return int(n.value)

    def evict_stale(self, min_clock: int) -> int:
        n = C.c_uint64(0)
        self._check(self.L.des_table_evict_stale(self.h, int(min_clock), C.byref(n)), "des_table_evict_stale")
        return int(n.value)

    def clock(self) -> int:
        c = C.c_uint64(0)
        self._check(self.L.des_table_clock(self.h, C.byref(c)), "des_table_clock")
        return int(c.value)

    def uses_tensor_cores(self) -> bool:
        return bool(self.L.des_table_uses_tensor_cores(self.h))

    def launch_count(self) -> int:
        return int(self.L.des_table_launch_count(self.h))

    def export(self, cap: int, weights: bool = True):
        """Dump of up to `cap` keys with their shard and shard-local row; with `weights`, also the
        rows' weights and first optimizer state (several times the size of the keys)."""
        dev = "cuda"
        keys = torch.empty(cap, dtype=torch.int64, device=dev)
        shards = torch.empty(cap, dtype=torch.uint8, device=dev)
        rows = torch.empty(cap, dtype=torch.int32, device=dev)
        emb = torch.empty((cap, self.k), dtype=torch.float32, device=dev) if weights else None
        lin = torch.empty(cap, dtype=torch.float32, device=dev) if weights else None
        ae = torch.empty((cap, self.k), dtype=torch.float32, device=dev) if weights else None
        al = torch.empty(cap, dtype=torch.float32, device=dev) if weights else None
        n = C.c_uint64(0)
        torch.cuda.synchronize()
        self._check(self.L.des_table_export(self.h, _ptr(keys), _ptr(shards), _ptr(rows), _ptr(emb), _ptr(lin),
                                            _ptr(ae), _ptr(al), cap, C.byref(n)), "des_table_export")
        m = min(int(n.value), cap)
        out = dict(n=int(n.value), keys=keys[:m], shards=shards[:m], rows=rows[:m])
        if weights:
            out.update(emb=emb[:m], lin=lin[:m], acc_emb=ae[:m], acc_lin=al[:m])
        return out

    def import_rows(self, keys: torch.Tensor, shards: torch.Tensor, emb=None, lin=None, acc_emb=None, acc_lin=None):
        """Restores a dump made by `export` (of this or another table with the same S, partition, k):
        inserts the keys — their rows get new numbers, a key's contents are what count — and writes
        weights and state over the freshly initialised rows.  Plumbing over find_or_insert + write_rows:
        one key per sample, in the bag of field 0 (HASH) or of the field that its shard owns (FIELD)."""
        n, F = int(keys.numel()), self.F
        chunk = max(1, min(self.max_batch, self.max_nnz))
        base = torch.tensor(self.row_base()[:-1], dtype=torch.int64, device="cuda")
        for lo in range(0, n, chunk):
            hi = min(n, lo + chunk)
            m = hi - lo
            fb = shards[lo:hi].to(torch.int64) if self.partition == PART_FIELD else torch.zeros(m, dtype=torch.int64, device="cuda")
            f = torch.arange(F, dtype=torch.int64, device="cuda")[None, :]
            off = (torch.arange(m, dtype=torch.int64, device="cuda")[:, None] + (f > fb[:, None])).reshape(-1)
            off = torch.cat([off, torch.tensor([m], dtype=torch.int64, device="cuda")]).to(torch.int32)
            db = DeviceBatch(off, keys[lo:hi].contiguous(), None, m)
            self.find_or_insert(db, True)
            grow = (base[db.shards[:m].to(torch.int64)] + db.rows[:m].to(torch.int64)).to(torch.int32)
            sl = slice(lo, hi)
            pick = lambda a: None if a is None else a[sl].contiguous()
            self.write_rows(grow, pick(emb), pick(lin), pick(acc_emb), pick(acc_lin))
        torch.cuda.current_stream().synchronize()

    def read_rows(self, global_rows: torch.Tensor):
        n = int(global_rows.numel())
        dev = "cuda"
        emb = torch.empty((n, self.k), dtype=torch.float32, device=dev)
        lin = torch.empty(n, dtype=torch.float32, device=dev)
        ae = torch.empty((n, self.k), dtype=torch.float32, device=dev)
        al = torch.empty(n, dtype=torch.float32, device=dev)
        self._check(self.L.des_table_read_rows(self.h, _ptr(global_rows), n, _ptr(emb), _ptr(lin), _ptr(ae),
                                               _ptr(al), _stream()), "des_table_read_rows")
        return dict(emb=emb, lin=lin, acc_emb=ae, acc_lin=al)

    def write_rows(self, global_rows: torch.Tensor, emb=None, lin=None, acc_emb=None, acc_lin=None):
        n = int(global_rows.numel())
        self._check(self.L.des_table_write_rows(self.h, _ptr(global_rows), n, _ptr(emb), _ptr(lin), _ptr(acc_emb),
                                                _ptr(acc_lin), _stream()), "des_table_write_rows")

    def profile_enable(self, on: bool = True):
        self._check(self.L.des_profile_enable(self.h, 1 if on else 0), "des_profile_enable")

    def profile_read(self):
        """-> list of (kernel name, ms) in launch order since the last read."""
        cap = 16384
        names = (C.c_char_p * cap)()
        ms = (C.c_float * cap)()
        n = C.c_int(0)
        self._check(self.L.des_profile_read(self.h, names, ms, cap, C.byref(n)), "des_profile_read")
        return [(names[i].decode(), float(ms[i])) for i in range(min(n.value, cap))]

    def dense1_forward_noalloc(self, pooled: torch.Tensor, Z: torch.Tensor):
        """Z = sum_s P_s with the per-shard partial products kept in the library's
        static device array: no allocation anywhere in the call."""
        self._check(self.L.des_dense1_forward_noalloc(self.h, _ptr(pooled), int(pooled.shape[0]), _ptr(Z), _stream()),
                    "des_dense1_forward_noalloc")

    def read_state2(self, global_rows: torch.Tensor):
        n = int(global_rows.numel())
        a2 = torch.empty((n, self.k), dtype=torch.float32, device="cuda")
        l2 = torch.empty(n, dtype=torch.float32, device="cuda")
        self._check(self.L.des_table_read_state2(self.h, _ptr(global_rows), n, _ptr(a2), _ptr(l2), _stream()),
                    "des_table_read_state2")
        return dict(acc2_emb=a2, lin2=l2)

    def write_state2(self, global_rows: torch.Tensor, acc2_emb=None, lin2=None):
        n = int(global_rows.numel())
        self._check(self.L.des_table_write_state2(self.h, _ptr(global_rows), n, _ptr(acc2_emb), _ptr(lin2), _stream()),
                    "des_table_write_state2")

    def dense1_get_state(self, want2=False):
        n = (self.F * self.k, self.H)
        s1 = torch.empty(n, dtype=torch.float32, device="cuda")
        s2 = torch.empty(n, dtype=torch.float32, device="cuda") if want2 else None
        self._check(self.L.des_dense1_get_state(self.h, _ptr(s1), _ptr(s2), _stream()), "des_dense1_get_state")
        return s1, s2

    def dense1_set_state(self, s1=None, s2=None):
        self._check(self.L.des_dense1_set_state(self.h, _ptr(s1), _ptr(s2), _stream()), "des_dense1_set_state")


# ---- DCN cross layer (no table) and transfer volumes ---------------------------------------------
def _check_free(code, where):
    if code != 0:
        raise DesError(code, where)


def cross_forward(x0: torch.Tensor, x: torch.Tensor, w: torch.Tensor, b: torch.Tensor, num_shards: int,
                  want_part: bool = False):
    """-> (y [B][d], P [B], part [S][B] or None)"""
    B, d = x.shape
    y = torch.empty_like(x)
    P = torch.empty(B, dtype=torch.float32, device=x.device)
    part = torch.empty((num_shards, B), dtype=torch.float32, device=x.device) if want_part else None
    _check_free(load().des_cross_forward(B, d, num_shards, _ptr(x0), _ptr(x), _ptr(w), _ptr(b), _ptr(part), _ptr(P),
                                        _ptr(y), _stream()), "des_cross_forward")
    return y, P, part


def cross_backward(x0, x, w, P, gY):
    """-> (gx0, gx [B][d], gw, gb [d])"""
    B, d = x.shape
    gx0 = torch.empty_like(x); gx = torch.empty_like(x)
    gw = torch.empty(d, dtype=torch.float32, device=x.device); gb = torch.empty_like(gw)
    ws = torch.empty(int(load().des_cross_workspace_floats(B, d)), dtype=torch.float32, device=x.device)
    _check_free(load().des_cross_backward(B, d, _ptr(x0), _ptr(x), _ptr(w), _ptr(P), _ptr(gY), _ptr(gx0), _ptr(gx),
                                         _ptr(gw), _ptr(gb), _ptr(ws), _stream()), "des_cross_backward")
    return gx0, gx, gw, gb


def comm_volume(workers, batch, uniq, emb_dim, hidden, first_layer_bytes, key_bytes=8, value_bytes=4):
    """Per-worker bytes under the mesh strategy and under DES, and the saving ratios: dict of 3-lists
    (LR, FM order 2, DNN first layer).  Host only."""
    m = des_comm_model_t(workers, batch, uniq, emb_dim, hidden, key_bytes, value_bytes, float(first_layer_bytes))
    o = des_comm_volume_t()
    _check_free(load().des_comm_volume(C.byref(m), C.byref(o)), "des_comm_volume")
    return dict(q_mesh=list(o.q_mesh), q_des=list(o.q_des), saving=list(o.saving))
