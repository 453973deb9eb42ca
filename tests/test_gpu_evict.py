"""Eviction on the CUDA table against the oracle's: same surviving key set, same row of every key
(the compaction rule is deterministic), same contents, removed keys look up as "no row" and come
back as new keys; and the streaming workload run past the capacity of its table with eviction by age.
Needs a B200."""
import numpy as np
import pytest
import torch

from paper_1909_04823_b200 import synth
from paper_1909_04823_b200.synth import OP_FM, OP_LR, OP_POOL, OPT_ADAGRAD, PART_FIELD, PART_HASH

pytestmark = pytest.mark.gpu


def _export_by_key(t, n):
    d = t.export(n + 8)
    assert d["n"] == n
    keys = d["keys"].cpu().numpy().view(np.uint64)
    shards = d["shards"].cpu().numpy()
    rows = d["rows"].cpu().numpy().view(np.uint32)
    emb = d["emb"].cpu().numpy(); lin = d["lin"].cpu().numpy()
    ae = d["acc_emb"].cpu().numpy(); al = d["acc_lin"].cpu().numpy()
    return {(int(s), int(k)): (int(r), emb[i].tobytes(), float(lin[i]), ae[i].tobytes(), float(al[i]))
            for i, (s, k, r) in enumerate(zip(shards, keys, rows))}


def _oracle_by_key(o):
    out = {}
    for s, n in enumerate(o.size()):
        n = int(n)
        if n:
            r = o.read_rows(np.full(n, s, np.uint8), np.arange(n, dtype=np.uint32))
            for i in range(n):
                out[(s, int(r["keys"][i]))] = (i, r["emb"][i].tobytes(), float(r["lin"][i]), r["acc_emb"][i].tobytes(),
                                               float(r["acc_lin"][i]))
    return out


@pytest.mark.parametrize("partition", [PART_HASH, PART_FIELD])
def test_evict_keys_matches_oracle(partition):
    from harness import Pair
    w = synth.config(4).scaled(batch=512, prepopulate=3000, init_scale=0.05, shards=5, partition=partition,
                               shared_vocab=(partition == PART_HASH))
    st = synth.Stream(w)
    b = st.next_batch()
    p = Pair(w, max_rows=200000, max_nnz=int(b.nnz * 1.3) + 1024)
    try:
        for s in range(2):
            p.step(b, synth.upstream_grads(w, b.batch, s))
            b = st.next_batch()
        n0 = sum(p.t.size())
        assert _export_by_key(p.t, n0) == _oracle_by_key(p.o)          # rows were re-seeded from the oracle: same bits
        rng = np.random.default_rng(3)
        all_keys = np.array(sorted({k for (_, k) in _oracle_by_key(p.o)}), dtype=np.uint64)
        gone = rng.choice(all_keys, size=all_keys.size // 3, replace=False)
        lst = np.concatenate([gone, gone[:7], synth.fmix64(np.arange(1 << 40, (1 << 40) + 5, dtype=np.uint64))])
        n_o = p.o.evict_keys(lst)
        n_g = p.t.evict_keys(torch.from_numpy(lst.view(np.int64)).cuda())
        assert n_g == n_o > 0 and p.t.status() == 0
        assert p.t.size() == [int(v) for v in p.o.size()]
        assert _export_by_key(p.t, n0 - n_g) == _oracle_by_key(p.o)     # key set, row of every key, contents
        # the table keeps working: removed keys look up as "no row", then come back as new keys, and the
        # next steps match the oracle in every stage (row numbers of the re-inserted keys included)
        from paper_1909_04823_b200.binding import DeviceBatch
        prev = synth.Stream(w).next_batch()
        look = p.o.find_or_insert(prev, insert=False)
        db = DeviceBatch.from_synth(prev)
        p.t.find_or_insert(db, False)
        torch.cuda.synchronize()
        assert np.array_equal(db.rows.cpu().numpy().view(np.uint32)[:prev.nnz], look["rows"])
        assert (look["rows"] == 0xFFFFFFFF).any()
        p.step(prev, synth.upstream_grads(w, prev.batch, 7), check_init=False)
        p.step(b, synth.upstream_grads(w, b.batch, 8))
        assert _export_by_key(p.t, sum(p.t.size())) == _oracle_by_key(p.o)
    finally:
        p.close()


@pytest.mark.parametrize("optimizer", [OPT_ADAGRAD, synth.OPT_ADAM])
def test_evict_stale_matches_oracle(optimizer):
    # (Adam: a second state array moves with the rows; the steps after the eviction would not match otherwise)
    from harness import Pair
    w = synth.config(4).scaled(batch=384, prepopulate=0, init_scale=0.05, shards=7, optimizer=optimizer)
    st = synth.Stream(w)
    b = st.next_batch()
    p = Pair(w, max_rows=200000, max_nnz=int(b.nnz * 1.3) + 1024)
    try:
        for s in range(5):
            p.step(b, synth.upstream_grads(w, b.batch, s))
            assert p.t.clock() == p.o.clock() == s + 1
            b = st.next_batch()
        n0 = sum(p.t.size())
        n_o = p.o.evict_stale(4)
        n_g = p.t.evict_stale(4)
        assert n_g == n_o and 0 < n_g < n0
        assert _export_by_key(p.t, n0 - n_g) == _oracle_by_key(p.o)
        assert p.t.evict_stale(4) == 0
        for s in range(2):
            p.step(b, synth.upstream_grads(w, b.batch, 9 + s))
            b = st.next_batch()
    finally:
        p.close()


def test_streaming_runs_past_table_capacity_with_eviction():
    """The streaming workload on a table too small for all the keys it will ever see: without eviction the
    run ends in DES_ERR_CAPACITY; evicting the keys that have not been touched for a few steps keeps it going,
    the table's size stays bounded, and its rows stay 0 .. n-1 per shard."""
    from paper_1909_04823_b200.binding import DeviceBatch, Table
    w = synth.config(4).scaled(batch=8192, prepopulate=50_000)
    steps, keep = 26, 3
    st = synth.Stream(w)
    first = st.next_batch()
    B, F, k = w.batch, w.fields, w.emb_dim
    new_per_step = int(first.nnz * w.p_new)
    cap = w.prepopulate + 16 * new_per_step                          # room for about sixteen steps of new keys
    batches = [first] + [st.next_batch() for _ in range(steps - 1)]

    def run(evict):
        t = Table.for_workload(w, max_rows=cap, max_nnz=int(first.nnz * 1.2))
        try:
            for ids in synth.Stream(w).prepopulation_ids(chunk=1 << 18):
                for lo in range(0, ids.size, B * F):
                    t.find_or_insert(DeviceBatch.from_synth(synth.prepopulation_batch(ids[lo:lo + B * F], F)), True)
            out_small = torch.empty((B, k + 4), device="cuda")
            pooled = torch.empty((B, F * k), device="cuda")
            sizes = []
            for s, b in enumerate(batches):
                g = {n: torch.from_numpy(v).cuda() for n, v in synth.upstream_grads(w, B, s % 4).items()}
                db = DeviceBatch.from_synth(b)
                t.find_or_insert(db, True)
                if t.status() != 0:
                    return t.status(), sizes, None
                t.forward_fused(w.ops, db, None, pooled, out_small, None)
                t.backward_update(w.ops, db, out_small, pooled, None, g["gL"], g["gF"], g["gE"], None, None)
                assert bool(torch.isfinite(out_small[:, :k + 3]).all())
                if evict and t.clock() > keep:
                    t.evict_stale(t.clock() - keep + 1)              # keep what was touched in the last `keep` calls
                sizes.append(sum(t.size()))
            n = sum(t.size())
            d = t.export(n + 8, weights=False)
            return t.status(), sizes, (d, t.size())
        finally:
            t.close()

    status, sizes, _ = run(evict=False)
    assert status == 3 and len(sizes) < steps                        # DES_ERR_CAPACITY part of the way through
    status, sizes, (d, per_shard) = run(evict=True)
    assert status == 0 and len(sizes) == steps
    assert max(sizes) < 0.9 * cap, (max(sizes), cap)
    shards = d["shards"].cpu().numpy(); rows = d["rows"].cpu().numpy().view(np.uint32)
    for s in range(w.shards):
        r = np.sort(rows[shards == s])
        assert r.size == per_shard[s] and np.array_equal(r, np.arange(r.size, dtype=np.uint32))
