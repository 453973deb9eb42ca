"""The checking build of the library (libdes_debug.so, -DDES_DEBUG): every gather, scatter and probe checks its
index against the table's bounds and raises the sticky status DES_ERR_RANGE instead of touching memory
outside them — the stand-in for a memory checker.  A handful of small workloads must run clean under it
(same results, status 0), and an index that is out of range must be reported, not followed.  Needs a B200."""
import numpy as np
import pytest
import torch

from paper_1909_04823_b200 import synth
from paper_1909_04823_b200.synth import OP_FM, OP_LR, OP_POOL, OPT_ADAGRAD, PART_HASH

pytestmark = pytest.mark.gpu


@pytest.fixture
def checking_build():
    from paper_1909_04823_b200 import binding
    prev = binding.use_debug_library(True)
    try:
        assert binding.load().des_build_is_debug() == 1
        yield binding
    finally:
        binding.use_debug_library(prev)


def _steps(w, steps, max_rows, prepop=False, **kw):
    from harness import Pair
    st = synth.Stream(w)
    b = st.next_batch()
    p = Pair(w, max_rows, max_nnz=int(b.nnz * 1.5) + 1024)
    try:
        assert p.t.L.des_build_is_debug() == 1
        if prepop:
            per_call = w.batch * w.fields
            for ids in st.prepopulation_ids(chunk=1 << 18):
                for lo in range(0, ids.size, per_call):
                    p.insert_only(synth.prepopulation_batch(ids[lo:lo + per_call], w.fields))
        for s in range(steps):
            p.step(b, synth.upstream_grads(w, b.batch, s), **kw)
            b = st.next_batch()
        assert p.t.status() == 0
    finally:
        p.close()


def test_small_workloads_run_clean(checking_build):
    _steps(synth.config(1).scaled(init_scale=0.05), 2, 20000, materialise=True)
    _steps(synth.config(3).scaled(batch=300, vocab=5000, hidden=80, init_scale=0.05), 2, 300000)
    _steps(synth.config(4).scaled(batch=512, prepopulate=5000, init_scale=0.05), 3, 200000, prepop=True)
    # above a million occurrences: sampled hot-key counts, replica rows, the counted keys of the backward
    _steps(synth.config(5).scaled(batch=640, vocab=50000, prepopulate=0, init_scale=0.05), 1, 120000)


def test_out_of_range_row_is_reported_not_followed(checking_build):
    from paper_1909_04823_b200.binding import DeviceBatch, Table
    w = synth.Workload("range", 64, 4, 8, 3, PART_HASH, OPT_ADAGRAD, OP_LR | OP_FM | OP_POOL, zipf_s=1.1, vocab=300,
                       shared_vocab=True, len_law="uniform", len_a=1, len_b=3, seed=9, init_scale=0.05)
    b = synth.Stream(w).next_batch()
    t = Table.for_workload(w, max_rows=2000, max_nnz=b.nnz + 64)
    try:
        B, F, k, S = w.batch, w.fields, w.emb_dim, w.shards
        db = DeviceBatch.from_synth(b)
        t.find_or_insert(db, True)
        ps = torch.zeros((S, B, k + 4), device="cuda"); pooled = torch.zeros((B, F * k), device="cuda")
        t.forward_partials(w.ops, db, ps, pooled)
        assert t.status() == 0
        good = (ps.clone(), pooled.clone())
        # a row number a few rows past the end of the table (still next to the table in memory, should a check
        # ever be missing): every kernel that would gather it must skip it and raise the status word
        base = t.row_base()
        shards = db.shards.cpu().numpy()
        rows = db.rows.cpu().numpy().view(np.uint32).copy()
        j = 5
        rows[j] = np.uint32(base[-1] + 5 - base[int(shards[j])])
        db.rows.copy_(torch.from_numpy(rows.view(np.int32)).view(db.rows.dtype))
        t.forward_partials(w.ops, db, ps, pooled)
        torch.cuda.synchronize()
        assert t.status() == 8                                   # DES_ERR_RANGE, sticky
        assert bool(torch.isfinite(ps).all()) and bool(torch.isfinite(pooled).all())
        # the skipped occurrence reads as the all-zero row: every other sample is unchanged
        bad_sample = int(np.searchsorted(b.offsets, j, side="right") - 1) // F
        keep = torch.ones(B, dtype=torch.bool, device="cuda"); keep[bad_sample] = False
        assert torch.equal(ps[:, keep], good[0][:, keep]) and torch.equal(pooled[keep], good[1][keep])
    finally:
        t.close()
