"""The host-buffer step (copies inside the call) against the device-resident call sequence,
and its pipelined submit / wait form against the blocking one.  Needs a B200."""
import numpy as np
import pytest
import torch

from paper_1909_04823_b200 import synth
from paper_1909_04823_b200.synth import OP_FM, OP_LR, OP_POOL, OPT_SGD

pytestmark = pytest.mark.gpu


def _workload():
    # SGD: the update is linear in the summed gradient, so two runs that differ only in the order of the
    # gradient atomics stay within rounding of each other (Adagrad / Adam divide by |G|-sized quantities and
    # can turn a rounding-sized difference of a cancelling sum into an lr-sized one)
    # (and a small step: with O(1) upstream gradients a larger one blows the weights up within three steps)
    return synth.config(4).scaled(batch=512, prepopulate=2000, init_scale=0.05, optimizer=OPT_SGD, lr=1e-5,
                                  ops=OP_LR | OP_FM | OP_POOL)


def _batches(w, n):
    st = synth.Stream(w)
    return [st.next_batch() for _ in range(n)]


def _pinned(b):
    return (torch.from_numpy(b.offsets).pin_memory(), torch.from_numpy(b.ids.view(np.int64)).pin_memory())


def _close(a, b, what=""):
    """Equal up to the order of float32 additions: relative to the element, or to the size of the row's
    largest element where the element itself is a sum that cancels."""
    a = np.asarray(a, dtype=np.float64); b = np.asarray(b, dtype=np.float64)
    scale = np.abs(b).reshape(b.shape[0], -1).max(axis=1).reshape((-1,) + (1,) * (b.ndim - 1)) if b.ndim > 1 else np.abs(b).max()
    bad = np.abs(a - b) > 2e-4 * np.abs(b) + 2e-6 * np.maximum(scale, 1.0)
    assert not bad.any(), (what, int(bad.sum()), float(np.abs(a - b).max()))


def _final_rows(t, keys_batch):
    from paper_1909_04823_b200.binding import DeviceBatch
    db = DeviceBatch.from_synth(keys_batch)
    t.find_or_insert(db, True)          # every key is already present: numbers the batch's unique keys only
    U = int(db.n_uniq.item())
    r = t.read_rows(db.uniq_rows[:U])
    torch.cuda.synchronize()
    return {n: v.cpu().numpy() for n, v in r.items()}


def test_step_host_equals_device_call_sequence():
    from paper_1909_04823_b200.binding import DeviceBatch, Table
    w = _workload()
    bs = _batches(w, 3)
    B, F, k = w.batch, w.fields, w.emb_dim
    mx = max(b.nnz for b in bs)
    grads = [{n: torch.from_numpy(v).cuda() for n, v in synth.upstream_grads(w, B, s).items()} for s in range(3)]
    ta = Table.for_workload(w, max_rows=200000, max_nnz=mx)
    tb = Table.for_workload(w, max_rows=200000, max_nnz=mx)
    try:
        pooled_a = torch.zeros((B, F * k), device="cuda"); pooled_b = torch.zeros((B, F * k), device="cuda")
        for s, b in enumerate(bs):
            g = grads[s]
            h_off, h_ids = _pinned(b)
            h_out = torch.empty((B, k + 4), dtype=torch.float32).pin_memory()
            ta.step_host(w.ops, B, b.nnz, h_off, h_ids, None, h_out, d_pooled=pooled_a, gL=g["gL"], gF=g["gF"], gE=g["gE"])
            db = DeviceBatch.from_synth(b)
            tb.find_or_insert(db, True)
            part = torch.empty((w.shards, B, k + 4), device="cuda")
            out = torch.empty((B, k + 4), device="cuda")
            tb.forward_partials(w.ops, db, part, pooled_b, None, None)
            tb.aggregate(w.ops, db, part, pooled_b, None, None, out, pooled_b, None)
            tb.backward_update(w.ops, db, out, pooled_b, None, g["gL"], g["gF"], g["gE"], None, None)
            torch.cuda.synchronize()
            assert ta.status() == 0 and tb.status() == 0
            # same kernels on the same table state: equal up to the order of the gradient atomics of earlier steps
            _close(h_out.numpy(), out.cpu().numpy(), "out_small")
            _close(pooled_a.cpu().numpy(), pooled_b.cpu().numpy(), "pooled")
        assert ta.size() == tb.size()
        ra, rb = _final_rows(ta, bs[-1]), _final_rows(tb, bs[-1])
        for n in ra:
            _close(ra[n], rb[n], n)
    finally:
        ta.close(); tb.close()


def test_pipelined_submit_wait_equals_blocking_steps():
    from paper_1909_04823_b200.binding import Table
    w = _workload()
    n = 6
    bs = _batches(w, n)
    B, F, k = w.batch, w.fields, w.emb_dim
    mx = max(b.nnz for b in bs)
    g = {nm: torch.from_numpy(v).cuda() for nm, v in synth.upstream_grads(w, B, 0).items()}
    host = [_pinned(b) for b in bs]
    outs = {}
    for mode in ("blocking", "pipelined"):
        t = Table.for_workload(w, max_rows=300000, max_nnz=mx)
        try:
            pooled = torch.zeros((B, F * k), device="cuda")
            h_out = [torch.full((B, k + 4), float("nan")).pin_memory() for _ in range(n)]
            if mode == "blocking":
                for i, b in enumerate(bs):
                    t.step_host(w.ops, B, b.nnz, host[i][0], host[i][1], None, h_out[i], d_pooled=pooled,
                                gL=g["gL"], gF=g["gF"], gE=g["gE"])
            else:
                tickets = []
                for i, b in enumerate(bs):
                    tickets.append(t.step_host_submit(w.ops, B, b.nnz, host[i][0], host[i][1], None, h_out[i],
                                                      d_pooled=pooled, gL=g["gL"], gF=g["gF"], gE=g["gE"]))
                    if i >= 1:
                        t.step_host_wait(tickets[i - 1])
                        assert not torch.isnan(h_out[i - 1]).any()       # that step's result has landed
                t.step_host_wait(tickets[-1])
                assert tickets == [i & 1 for i in range(n)]
            torch.cuda.synchronize()
            assert t.status() == 0
            outs[mode] = ([o.numpy().copy() for o in h_out], t.size(), _final_rows(t, bs[-1]))
        finally:
            t.close()
    for a, b_ in zip(outs["blocking"][0], outs["pipelined"][0]):
        _close(a, b_, "out_small")
    assert outs["blocking"][1] == outs["pipelined"][1]
    for nm in outs["blocking"][2]:
        _close(outs["blocking"][2][nm], outs["pipelined"][2][nm], nm)


def test_blocking_step_after_submits_waits_for_them():
    from paper_1909_04823_b200.binding import Table
    w = _workload()
    bs = _batches(w, 3)
    B, F, k = w.batch, w.fields, w.emb_dim
    g = {nm: torch.from_numpy(v).cuda() for nm, v in synth.upstream_grads(w, B, 0).items()}
    t = Table.for_workload(w, max_rows=200000, max_nnz=max(b.nnz for b in bs))
    try:
        pooled = torch.zeros((B, F * k), device="cuda")
        host = [_pinned(b) for b in bs]
        h_out = [torch.full((B, k + 4), float("nan")).pin_memory() for _ in range(3)]
        for i in range(2):
            t.step_host_submit(w.ops, B, bs[i].nnz, host[i][0], host[i][1], None, h_out[i], d_pooled=pooled,
                               gL=g["gL"], gF=g["gF"], gE=g["gE"])
        t.step_host(w.ops, B, bs[2].nnz, host[2][0], host[2][1], None, h_out[2], d_pooled=pooled,
                    gL=g["gL"], gF=g["gF"], gE=g["gE"])
        for o in h_out:
            assert not torch.isnan(o).any()
        t.step_host_wait(0); t.step_host_wait(1)        # nothing left to wait for: returns at once
        assert t.status() == 0
    finally:
        t.close()
