"""Parity of the CUDA path (through the C ABI) against the CPU oracle, element
by element, on the same seeded batches.  Needs a B200."""
import numpy as np
import pytest
import torch

from paper_1909_04823_b200 import synth
from paper_1909_04823_b200.synth import (OP_DENSE1, OP_FM, OP_LR, OP_POOL, OPT_ADAGRAD, OPT_SGD, PART_FIELD,
                                          PART_HASH)

pytestmark = pytest.mark.gpu


def _pair(w, max_rows, max_nnz, **kw):
    from harness import Pair
    return Pair(w, max_rows, max_nnz, **kw)


def _run(w, steps, max_rows, materialise=False, with_vals=False, prepop=0, ops=None, check_init=True):
    st = synth.Stream(w, with_vals=with_vals)
    first = st.next_batch()
    p = _pair(w, max_rows, max_nnz=int(first.nnz * 1.5) + 1024)
    try:
        if prepop:
            per_call = min(w.batch * w.fields, first.nnz)
            for ids in st.prepopulation_ids(chunk=1 << 18):
                for lo in range(0, ids.size, per_call):
                    p.insert_only(synth.prepopulation_batch(ids[lo:lo + per_call], w.fields))
        b = first
        for s in range(steps):
            g = synth.upstream_grads(w, b.batch, s)
            p.step(b, g, ops=ops, materialise=materialise, check_init=check_init and s == 0 and not prepop)
            if s + 1 < steps:
                b = st.next_batch()
    finally:
        p.close()


# ------------------------------------------------------------------ config 1 (full size)
@pytest.mark.parametrize("partition", [PART_HASH, PART_FIELD])
@pytest.mark.parametrize("S", [1, 2, 3, 4, 7])
def test_cfg1_tiny_lr_fm(S, partition):
    w = synth.config(1).scaled(shards=S, partition=partition, shared_vocab=(partition == PART_HASH),
                               ops=OP_LR | OP_FM | OP_POOL, init_scale=0.05)
    _run(w, 1, max_rows=20000, materialise=True)


def test_cfg1_exact_ops_and_vals():
    _run(synth.config(1), 2, max_rows=20000, materialise=False)
    _run(synth.config(1).scaled(init_scale=0.05), 2, max_rows=20000, with_vals=True, materialise=True)


# ------------------------------------------------------------------ config 2 (W&D)
def test_cfg2_wide_deep_scaled_materialised():
    w = synth.config(2).scaled(batch=640, vocab=20000, hidden=72, init_scale=0.05)
    _run(w, 3, max_rows=400000, materialise=True)


def test_adagrad_nonzero_initial_accumulator():
    # accumulators that start at init_acc = 0.1 (rows, linear weights and the first layer), three steps
    w = synth.config(2).scaled(batch=512, vocab=3000, hidden=64, init_scale=0.05, init_acc=0.1)
    _run(w, 3, max_rows=200000)
    w = synth.config(4).scaled(batch=256, prepopulate=2000, init_scale=0.05, init_acc=0.1)
    _run(w, 3, max_rows=200000, prepop=1)


# ------------------------------------------------------------------ config 3 (DeepFM)
def test_cfg3_deepfm_scaled_materialised():
    w = synth.config(3).scaled(batch=300, vocab=5000, hidden=80, init_scale=0.05)
    _run(w, 3, max_rows=300000, materialise=True)


def test_cfg3_deepfm_wide_hidden():
    w = synth.config(3).scaled(batch=1024, vocab=200000)
    _run(w, 2, max_rows=1_500_000)


# ------------------------------------------------------------------ config 4 (streaming, scaled)
def test_cfg4_streaming_scaled_growth():
    w = synth.config(4).scaled(batch=1024, prepopulate=20000, init_scale=0.05)
    _run(w, 6, max_rows=400000, prepop=1)


# ------------------------------------------------------------------ config 5 (multi-hot, scaled)
def test_cfg5_multihot_scaled():
    w = synth.config(5).scaled(batch=192, vocab=50000, prepopulate=50000, init_scale=0.05)
    _run(w, 2, max_rows=120000, prepop=1)


@pytest.mark.parametrize("k", [4, 8, 12, 24, 48, 64])
def test_embedding_dims(k):
    w = synth.config(1).scaled(emb_dim=k, shards=5, ops=OP_LR | OP_FM | OP_POOL, optimizer=OPT_ADAGRAD,
                               init_scale=0.05, batch=200)
    _run(w, 2, max_rows=20000, materialise=True, with_vals=True)


# ------------------------------------------------------------------ edge cases
def _mk(S=4, F=3, k=8, partition=PART_HASH, optimizer=OPT_ADAGRAD, ops=OP_LR | OP_FM | OP_POOL, batch=8):
    return synth.Workload("edge", batch, F, k, S, partition, optimizer, ops, init_scale=0.1, seed=77)


@pytest.mark.parametrize("S,partition", [(4, PART_HASH), (5, PART_FIELD)])
def test_empty_bags_duplicates_and_all_seen(S, partition):
    # (FIELD with more shards than fields: two shards own no field at all)
    w = _mk(S=S, partition=partition)
    F, B = w.fields, w.batch
    rng = np.random.default_rng(5)
    lens = rng.integers(0, 4, size=B * F)
    lens[:F] = 0                                  # a sample with no occurrence at all
    offsets = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    ids = synth.fmix64(rng.integers(0, 6, size=int(offsets[-1])).astype(np.uint64))   # heavy duplication
    vals = rng.uniform(0.5, 2.0, size=ids.size).astype(np.float32)
    b = synth.Batch(B, F, offsets, ids, vals)
    p = _pair(w, 1000, 4096)
    try:
        p.step(b, synth.upstream_grads(w, B, 0), materialise=True, check_init=True)
        # the same batch again: every key already known (no insert), state carries over (this time without
        # materialised per-shard pooled partials: the fast paths, fused forms included)
        p.step(b, synth.upstream_grads(w, B, 1), materialise=False)
    finally:
        p.close()


def test_empty_batch_and_lookup_only():
    from paper_1909_04823_b200.binding import DeviceBatch
    w = _mk()
    p = _pair(w, 1000, 4096)
    try:
        e = synth.Batch(2, w.fields, np.zeros(2 * w.fields + 1, np.int32), np.zeros(0, np.uint64), None)
        db = DeviceBatch.from_synth(e)
        p.t.find_or_insert(db, True)
        torch.cuda.synchronize()
        assert int(db.n_uniq.item()) == 0 and p.t.status() == 0 and sum(p.t.size()) == 0
        # insert some, then look up a mix of known and unknown ids without inserting
        b = synth.Stream(w.scaled(vocab=50, len_law="uniform", len_a=1, len_b=3)).next_batch()
        fi, _ = p.insert_only(b)
        b2 = synth.Batch(b.batch, b.fields, b.offsets, b.ids.copy(), None)
        b2.ids[::3] ^= np.uint64(1 << 40)
        f2 = p.o.find_or_insert(b2, insert=False)
        d2 = DeviceBatch.from_synth(b2)
        p.t.find_or_insert(d2, False)
        torch.cuda.synchronize()
        assert np.array_equal(d2.rows.cpu().numpy().view(np.uint32)[:b2.nnz], f2["rows"])
        assert np.array_equal(d2.shards.cpu().numpy()[:b2.nnz], f2["shards"])
        assert p.t.size() == [int(v) for v in p.o.size()]
        assert (f2["rows"] == 0xFFFFFFFF).any() and (f2["rows"] != 0xFFFFFFFF).any()
        # forward over a batch with unknown keys skips them exactly like the oracle
        S, B, k, F = w.shards, b2.batch, w.emb_dim, w.fields
        part_small = torch.zeros((S, B, k + 4), device="cuda"); pooled = torch.zeros((B, F * k), device="cuda")
        out_small = torch.zeros((B, k + 4), device="cuda")
        p.t.forward_partials(w.ops, d2, part_small, pooled)
        p.t.aggregate(w.ops, d2, part_small, pooled, out_small=out_small)
        torch.cuda.synchronize()
        ref = p.o.forward_original(w.ops, b2)
        from harness import close32
        close32(out_small.cpu().numpy()[:, :k], ref["A"], "A with unknown keys")
        close32(pooled.cpu().numpy(), ref["pooled"], "pooled with unknown keys")
    finally:
        p.close()


def test_capacity_and_reserved_key_are_reported_not_faulted():
    from paper_1909_04823_b200.binding import DeviceBatch, Table
    w = _mk(S=2)
    t = Table.for_workload(w, max_rows=8, max_nnz=8192, rows_per_shard=[4, 4])
    try:
        ids = synth.fmix64(np.arange(600, dtype=np.uint64))
        b = synth.prepopulation_batch(ids[:w.batch * w.fields], w.fields)
        db = DeviceBatch.from_synth(b)
        t.find_or_insert(db, True)
        assert t.status() == 3                                  # DES_ERR_CAPACITY, sticky
        assert all(n <= 4 for n in t.size())
        rows = db.rows.cpu().numpy().view(np.uint32)[:b.nnz]
        assert (rows == 0xFFFFFFFF).any() and (rows[rows != 0xFFFFFFFF] < 4).all()
        # later kernels skip the unmapped occurrences
        S, B, k, F = w.shards, b.batch, w.emb_dim, w.fields
        ps = torch.zeros((S, B, k + 4), device="cuda"); pooled = torch.zeros((B, F * k), device="cuda")
        t.forward_partials(w.ops, db, ps, pooled)
        torch.cuda.synchronize()
        assert torch.isfinite(pooled).all()
    finally:
        t.close()
    t = Table.for_workload(w, max_rows=100, max_nnz=8192)
    try:
        ids = synth.fmix64(np.arange(6, dtype=np.uint64))
        ids[2] = np.uint64(0xFFFFFFFFFFFFFFFF)
        db = DeviceBatch.from_synth(synth.prepopulation_batch(ids, w.fields))
        t.find_or_insert(db, True)
        assert t.status() == 2                                  # DES_ERR_RESERVED_KEY
        rows = db.rows.cpu().numpy().view(np.uint32)
        assert rows[2] == 0xFFFFFFFF and (rows[[0, 1, 3, 4, 5]] != 0xFFFFFFFF).all()
    finally:
        t.close()


def test_gradient_buffer_capacity_is_reported_by_the_backward_only():
    # max_uniq sizes the gradient buffer: a batch with more distinct keys than that inserts and forwards fine
    # (pre-population, inference); only a backward over it raises DES_ERR_CAPACITY — and faults nothing
    from paper_1909_04823_b200.binding import DeviceBatch, Table
    w = _mk(S=3)
    ids = synth.fmix64(np.arange(600, dtype=np.uint64))
    b = synth.prepopulation_batch(ids, w.fields)
    t = Table.for_workload(w, max_rows=2000, max_nnz=1024, max_batch=b.batch, max_uniq=100)
    try:
        db = DeviceBatch.from_synth(b)
        t.find_or_insert(db, True)
        S, B, k, F = w.shards, b.batch, w.emb_dim, w.fields
        ps = torch.zeros((S, B, k + 4), device="cuda"); pooled = torch.zeros((B, F * k), device="cuda")
        out = torch.zeros((B, k + 4), device="cuda")
        t.forward_partials(w.ops, db, ps, pooled)
        t.aggregate(w.ops, db, ps, pooled, out_small=out)
        assert t.status() == 0 and sum(t.size()) == 600
        g = {n: torch.from_numpy(v).cuda() for n, v in synth.upstream_grads(w, B, 0).items()}
        t.backward_update(w.ops, db, out, pooled, None, g["gL"], g["gF"], g["gE"], None, None)
        assert t.status() == 3
    finally:
        t.close()


def test_invalid_arguments_are_rejected_on_the_host():
    from paper_1909_04823_b200.binding import DesError, DeviceBatch, Table
    w = _mk()
    with pytest.raises(DesError):
        Table(4, 3, 7)                                          # k not a multiple of 4
    with pytest.raises(DesError):
        Table(65, 3, 8)                                         # S > 64
    t = Table.for_workload(w, max_rows=100, max_nnz=16)
    try:
        b = synth.prepopulation_batch(synth.fmix64(np.arange(24, dtype=np.uint64)), w.fields)
        with pytest.raises(DesError):
            t.find_or_insert(DeviceBatch.from_synth(b), True)   # nnz > max_nnz
        small = DeviceBatch.from_synth(synth.prepopulation_batch(synth.fmix64(np.arange(6, dtype=np.uint64)), w.fields))
        t.find_or_insert(small, True)
        with pytest.raises(DesError):
            t.forward_partials(OP_DENSE1, small, None, torch.zeros(1, device="cuda"))   # no hidden layer
        with pytest.raises(DesError):
            t.forward_partials(OP_LR, small, None, None)        # missing output
    finally:
        t.close()


def test_integer_outputs_are_run_to_run_identical():
    from paper_1909_04823_b200.binding import DeviceBatch, Table
    w = synth.config(4).scaled(batch=2048, prepopulate=1000)
    b = synth.Stream(w).next_batch()
    outs = []
    for _ in range(3):
        t = Table.for_workload(w, max_rows=200000, max_nnz=b.nnz)
        db = DeviceBatch.from_synth(b)
        t.find_or_insert(db, True)
        torch.cuda.synchronize()
        outs.append((db.rows.cpu().numpy().copy(), db.uidx.cpu().numpy().copy(), db.uniq_rows.cpu().numpy()[:int(db.n_uniq.item())].copy(), t.size()))
        t.close()
    for o in outs[1:]:
        assert all(np.array_equal(a, c) if isinstance(a, np.ndarray) else a == c for a, c in zip(o, outs[0]))


def test_multi_step_without_resync_stays_close():
    # no re-seeding of the CUDA table from the oracle between steps: tolerated
    # differences may compound, so later steps are held to the looser bound
    from harness import Pair
    w = synth.config(1).scaled(batch=256, optimizer=OPT_ADAGRAD, ops=OP_LR | OP_FM | OP_POOL, init_scale=0.05)
    st = synth.Stream(w)
    b = st.next_batch()
    p = Pair(w, 50000, b.nnz * 2, resync=False)
    try:
        for s in range(5):
            p.step(b, synth.upstream_grads(w, b.batch, s))
            b = st.next_batch()
    finally:
        p.close()


def test_cfg5_multihot_million_occurrences():
    # a batch above one million occurrences: the backward samples its hot-key counts (1 in 2)
    # instead of counting every occurrence, and every kernel runs several waves
    w = synth.config(5).scaled(batch=640, vocab=50000, prepopulate=50000, init_scale=0.05)
    assert synth.Stream(w).next_batch().nnz > (1 << 20)
    _run(w, 2, max_rows=120000, prepop=1)


@pytest.mark.parametrize("ops", [OP_LR | OP_FM, OP_POOL])
def test_million_occurrences_operator_subsets(ops):
    # the counted-and-multiplied path of the keys that own the batch, without the pooling gradient (LR + FM
    # only) and without the per-sample gradients (pooling only)
    w = synth.config(5).scaled(batch=640, vocab=50000, prepopulate=0, init_scale=0.05, ops=ops)
    assert synth.Stream(w).next_batch().nnz > (1 << 20)
    _run(w, 1, max_rows=120000, ops=ops)


def test_forward_is_run_to_run_identical():
    # the forward has no atomics on its fast path and a fixed order of additions: same bits every time,
    # also across two tables built the same way
    from paper_1909_04823_b200.binding import DeviceBatch, Table
    w = synth.config(5).scaled(batch=256, vocab=50000, prepopulate=0, init_scale=0.05)
    b = synth.Stream(w).next_batch()
    B, F, k, S = b.batch, w.fields, w.emb_dim, w.shards
    res = []
    for rep in range(2):
        t = Table.for_workload(w, max_rows=200000, max_nnz=b.nnz)
        try:
            db = DeviceBatch.from_synth(b)
            t.find_or_insert(db, True)
            for again in range(2):
                part = torch.full((S, B, k + 4), float("nan"), device="cuda")
                out = torch.full((B, k + 4), float("nan"), device="cuda")
                pooled = torch.full((B, F * k), float("nan"), device="cuda")
                t.forward_partials(w.ops, db, part, pooled, None, None)
                t.aggregate(w.ops, db, part, pooled, None, None, out, pooled, None)
                torch.cuda.synchronize()
                res.append((part.clone(), out.clone(), pooled.clone()))
            assert t.status() == 0
        finally:
            t.close()
    for r in res[1:]:
        for a, c in zip(r, res[0]):
            assert torch.equal(a.view(torch.int32), c.view(torch.int32))


@pytest.mark.parametrize("k", [8, 32, 64])
def test_long_bags_with_feature_values(k):
    # bags of about 20 ids (a whole warp per bag in pooling and scatter, 32 / (k/4) sub-groups taking alternate
    # occurrences) together with real feature values and materialised per-shard partials
    w = synth.config(5).scaled(batch=48, vocab=20000, prepopulate=0, emb_dim=k, shards=7, init_scale=0.05)
    _run(w, 2, max_rows=120000, materialise=True, with_vals=True)


def test_long_bags_field_partition():
    w = synth.config(5).scaled(batch=48, vocab=3000, prepopulate=0, emb_dim=16, shards=6, fields=40, partition=PART_FIELD,
                               shared_vocab=False, init_scale=0.05)
    _run(w, 2, max_rows=150000, materialise=False)


@pytest.mark.parametrize("partition", [PART_HASH, PART_FIELD])
def test_maximum_fields_and_shards(partition):
    # the largest field count and shard count the library accepts (1024 fields, 64 shards)
    w = synth.Workload("max_fields", 6, 1024, 4, 64, partition, OPT_ADAGRAD, OP_LR | OP_FM | OP_POOL, zipf_s=1.1, vocab=500,
                       shared_vocab=(partition == PART_HASH), len_law="uniform", len_a=0, len_b=2, seed=31, init_scale=0.05)
    _run(w, 2, max_rows=80000, materialise=True)


@pytest.mark.parametrize("ops", [OP_LR, OP_FM, OP_POOL, OP_LR | OP_POOL, OP_FM | OP_POOL])
def test_long_bags_operator_subsets(ops):
    w = synth.config(5).scaled(batch=40, vocab=20000, prepopulate=0, shards=9, init_scale=0.05, ops=ops)
    _run(w, 2, max_rows=120000, ops=ops)


def test_insert_scratch_range_wraps(monkeypatch):
    """The slots' scratch word works in a range that moves down with every insert call and is reset by
    one pass over the table when it runs out (every few billion occurrences).  Started three calls
    before the end of the range, the reset must happen unnoticed: every step matches the oracle."""
    w = synth.config(1).scaled(batch=256, ops=OP_LR | OP_FM | OP_POOL, init_scale=0.05, optimizer=OPT_ADAGRAD)
    st = synth.Stream(w)
    first = st.next_batch()
    max_nnz = int(first.nnz * 1.5) + 1024
    # the starting point of the range can only be moved in the checking build of the library
    from paper_1909_04823_b200 import binding
    monkeypatch.setenv("DES_DEBUG_SCRATCH_BASE", str(max_nnz + 3 * first.nnz))
    prev = binding.use_debug_library(True)
    try:
        p = _pair(w, 60000, max_nnz=max_nnz)
        assert p.t.L.des_build_is_debug() == 1
    finally:
        binding.use_debug_library(prev)
    monkeypatch.delenv("DES_DEBUG_SCRATCH_BASE")
    try:
        b = first
        for s in range(8):
            p.step(b, synth.upstream_grads(w, b.batch, s), check_init=(s == 0))
            b = st.next_batch()
    finally:
        p.close()
