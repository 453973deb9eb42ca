"""The no-allocation entry point (des_dense1_forward_noalloc) against the
regular one (des_aggregate with a caller-provided partial-product buffer).

It exists for callers that may not allocate device memory — a serving loop with
a frozen memory budget, a plug-in inside another framework, a latency-critical
section — so its per-shard partial products sit in a static device array of the
library instead of a buffer the caller brings.  Two calls in a row share that
array; the second must not see anything of the first.  This file sorts last on
purpose: a run that stops at the first failure has then run every other test."""
import numpy as np
import pytest
import torch

from paper_1909_04823_b200 import synth
from paper_1909_04823_b200.synth import OP_DENSE1, OP_LR, OP_POOL, OPT_ADAGRAD, PART_FIELD, PART_HASH

pytestmark = pytest.mark.gpu


def _table(S=8, F=26, k=16, H=64, B=512, partition=PART_FIELD):
    from paper_1909_04823_b200.binding import Table
    w = synth.Workload("noalloc", B, F, k, S, partition, OPT_ADAGRAD, OP_LR | OP_POOL | OP_DENSE1, hidden=H, seed=21)
    t = Table.for_workload(w, max_rows=1000, max_nnz=B * F, rows_per_shard=[200] * S if partition == PART_FIELD else None)
    t.dense1_set(torch.from_numpy(synth.dense1_weights(w)).cuda())
    return w, t


def test_noalloc_matches_regular_entry_point_twice():
    from paper_1909_04823_b200.binding import DeviceBatch
    w, t = _table()
    try:
        B, F, k, S, H = w.batch, w.fields, w.emb_dim, w.shards, w.hidden
        db = DeviceBatch(np.zeros(B * F + 1, np.int32), np.zeros(0, np.uint64), None, B)   # des_aggregate reads B only
        gen = torch.Generator(device="cuda").manual_seed(3)
        for call in range(2):
            scale = 1.0 if call == 0 else 7.0         # the second call uses different data and a ragged batch
            Bc = B if call == 0 else B - 37
            pooled = torch.randn((Bc, F * k), device="cuda", generator=gen) * scale
            dbc = DeviceBatch(np.zeros(Bc * F + 1, np.int32), np.zeros(0, np.uint64), None, Bc)
            part_dense = torch.empty((S, Bc, H), device="cuda")
            Z_ref = torch.full((Bc, H), float("nan"), device="cuda")
            t.aggregate(OP_DENSE1, dbc, pooled=pooled, part_dense=part_dense, out_pooled=pooled, Z=Z_ref)
            Z = torch.full((Bc, H), float("nan"), device="cuda")
            t.dense1_forward_noalloc(pooled, Z)
            torch.cuda.synchronize()
            assert t.status() == 0
            ref, got = Z_ref.cpu().numpy().astype(np.float64), Z.cpu().numpy().astype(np.float64)
            assert np.isfinite(got).all()
            tol = 2e-2 * np.abs(ref) + 1e-3 * np.abs(ref).max()      # the GEMM tolerance of the parity tests
            assert np.all(np.abs(got - ref) <= tol)
            # same kernels, same order of summation: in fact bit-identical
            assert np.array_equal(Z_ref.cpu().numpy().view(np.uint32), Z.cpu().numpy().view(np.uint32))
            # and both agree with a plain matmul of the bf16-rounded operands
            W1 = t.dense1_get()
            want = pooled.to(torch.bfloat16).to(torch.float64) @ W1.to(torch.bfloat16).to(torch.float64)
            assert np.all(np.abs(got - want.cpu().numpy()) <= tol)
    finally:
        t.close()


def test_noalloc_rejects_what_does_not_fit():
    from paper_1909_04823_b200.binding import DesError
    w, t = _table(H=256, B=2048)                       # 8 * 2048 * 256 floats = 16 MiB > the 8 MiB array
    try:
        pooled = torch.zeros((w.batch, w.fields * w.emb_dim), device="cuda")
        Z = torch.zeros((w.batch, w.hidden), device="cuda")
        with pytest.raises(DesError) as e:
            t.dense1_forward_noalloc(pooled, Z)
        assert e.value.code == 7                       # DES_ERR_TOO_LARGE
        t.dense1_forward_noalloc(pooled[:1024], Z[:1024])   # exactly at the limit is accepted
        torch.cuda.synchronize()
        assert t.status() == 0
    finally:
        t.close()
    w, t = _table(partition=PART_HASH)
    try:
        with pytest.raises(DesError) as e:
            t.dense1_forward_noalloc(torch.zeros((4, w.fields * w.emb_dim), device="cuda"), torch.zeros((4, w.hidden), device="cuda"))
        assert e.value.code == 4                       # DES_ERR_UNSUPPORTED: needs the FIELD placement
    finally:
        t.close()
