"""Checkpoint / resume through the C ABI: des_table_export dumps every key with its weights and
optimizer state; a fresh table that re-inserts the keys and takes the rows over computes the same
forward bit for bit and the same next update.  Needs a B200."""
import numpy as np
import pytest
import torch

from paper_1909_04823_b200 import synth
from paper_1909_04823_b200.synth import OP_FM, OP_LR, OP_POOL, OPT_ADAGRAD, PART_FIELD, PART_HASH

pytestmark = pytest.mark.gpu


def _forward(t, w, db):
    B, F, k = db.batch, w.fields, w.emb_dim
    out = torch.empty((B, k + 4), device="cuda")
    pooled = torch.empty((B, F * k), device="cuda")
    t.forward_fused(w.ops, db, None, pooled, out, None)
    return out, pooled


@pytest.mark.parametrize("partition", [PART_HASH, PART_FIELD])
def test_export_import_resumes_training(partition):
    from harness import rows_per_shard_for
    from paper_1909_04823_b200.binding import DeviceBatch, Table
    w = synth.config(1).scaled(shards=5, partition=partition, shared_vocab=(partition == PART_HASH), batch=256,
                               ops=OP_LR | OP_FM | OP_POOL, optimizer=OPT_ADAGRAD, init_scale=0.05, lr=1e-3)
    st = synth.Stream(w)
    batches = [st.next_batch() for _ in range(3)]
    mx = max(b.nnz for b in batches)
    mk = lambda: Table.for_workload(w, max_rows=60000, max_nnz=mx + 1024, rows_per_shard=rows_per_shard_for(w, 60000),
                                    max_batch=4096)
    a = mk()
    b2 = mk()
    try:
        g = [{n: torch.from_numpy(v).cuda() for n, v in synth.upstream_grads(w, w.batch, s).items()} for s in range(3)]
        for s in range(2):                                   # train two steps on the first table
            db = DeviceBatch.from_synth(batches[s])
            a.find_or_insert(db, True)
            out, pooled = _forward(a, w, db)
            a.backward_update(w.ops, db, out, pooled, None, g[s]["gL"], g[s]["gF"], g[s]["gE"], None, None)
        torch.cuda.synchronize()
        n_keys = sum(a.size())
        dump = a.export(n_keys + 10)
        assert dump["n"] == n_keys and len(torch.unique(dump["keys"])) == n_keys
        b2.import_rows(dump["keys"], dump["shards"], dump["emb"], dump["lin"], dump["acc_emb"], dump["acc_lin"])
        assert b2.status() == 0 and b2.size() == a.size()
        # same third step on both
        outs = []
        for t in (a, b2):
            db = DeviceBatch.from_synth(batches[2])
            t.find_or_insert(db, True)
            out, pooled = _forward(t, w, db)
            torch.cuda.synchronize()
            outs.append((out.clone(), pooled.clone(), db))
            t.backward_update(w.ops, db, out, pooled, None, g[2]["gL"], g[2]["gF"], g[2]["gE"], None, None)
        torch.cuda.synchronize()
        assert a.status() == 0 and b2.status() == 0
        # the forward walks a sample's rows in an order that does not depend on row numbers: same bits for
        # everything summed from the weights themselves; M_2 uses the rows' cached |v|^2, which the import
        # recomputes in another order of additions than the update kernel (last-bit differences)
        k = w.emb_dim
        assert torch.equal(outs[0][0][:, :k + 1].view(torch.int32), outs[1][0][:, :k + 1].view(torch.int32))
        assert torch.equal(outs[0][1].view(torch.int32), outs[1][1].view(torch.int32))
        torch.testing.assert_close(outs[0][0][:, k + 1:], outs[1][0][:, k + 1:], rtol=1e-5, atol=1e-6)
        assert np.array_equal(outs[0][2].shards.cpu().numpy(), outs[1][2].shards.cpu().numpy())
        # and the tables agree key by key after the update (gradient atomics may differ in order)
        da, dbb = a.export(sum(a.size())), b2.export(sum(b2.size()))
        ia, ib = torch.argsort(da["keys"]), torch.argsort(dbb["keys"])
        assert torch.equal(da["keys"][ia], dbb["keys"][ib]) and torch.equal(da["shards"][ia], dbb["shards"][ib])
        for name in ("emb", "lin", "acc_emb", "acc_lin"):
            x, y = da[name][ia].cpu().numpy().astype(np.float64), dbb[name][ib].cpu().numpy().astype(np.float64)
            off = np.abs(x - y) > 2e-4 * np.abs(y) + 2e-6
            assert off.mean() < 1e-3, (name, int(off.sum()))   # (Adagrad: a cancelling sum may flip a step's sign)
    finally:
        a.close(); b2.close()
