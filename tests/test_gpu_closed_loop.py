"""Closed-loop runs: the upstream gradients of every step come from a fixed read-out (des_head) applied to
that step's own forward results, so the table updated in step t feeds the loss whose gradient drives step
t + 1.  Parity against the oracle's closed loop on scaled Wide&Deep- and DeepFM-shaped workloads, and a
check that the loss falls when the labels carry a planted signal.  Needs a B200."""
import numpy as np
import pytest
import torch

from paper_1909_04823_b200 import synth
from paper_1909_04823_b200.synth import OP_FM, OP_LR, OP_POOL, OPT_ADAGRAD, PART_HASH

pytestmark = pytest.mark.gpu


def _closed_loop(w, steps, max_rows, resync, n_dense=0, prepop=False):
    from harness import Pair
    st = synth.Stream(w)
    b = st.next_batch()
    p = Pair(w, max_rows, max_nnz=int(b.nnz * 1.5) + 1024, resync=resync)
    hc = synth.head_constants(w, n_dense)
    losses = []
    try:
        if prepop:
            per_call = w.batch * w.fields
            for ids in st.prepopulation_ids(chunk=1 << 18):
                for lo in range(0, ids.size, per_call):
                    p.insert_only(synth.prepopulation_batch(ids[lo:lo + per_call], w.fields))
        for s in range(steps):
            head = dict(hc=hc, y=synth.labels(w, b.batch, s),
                        xdense=synth.dense_features(w, b.batch, s, n_dense) if n_dense else None)
            r = p.step(b, None, check_init=(s == 0 and not prepop), head=head)
            losses.append((r["head"]["loss"], r["head"]["gpu_loss"]))
            b = st.next_batch()
    finally:
        p.close()
    return losses


@pytest.mark.parametrize("resync", [True, False])
def test_closed_loop_wide_deep_scaled(resync):
    # Criteo-shaped: 26 categorical fields, 13 continuous features that enter the read-out only
    # (accumulators start at 0.1, the value the paper's framework uses by default: from 0 the first Adagrad step
    # of a weight is lr * sign(G), and in a free-running loop a gradient of rounding size then moves the two
    # sides 2 lr apart)
    w = synth.config(2).scaled(batch=512, vocab=3000, hidden=64, init_scale=0.05, lr=0.5, init_acc=0.1)
    losses = _closed_loop(w, 6, max_rows=300000, resync=resync, n_dense=13)
    assert all(abs(a - g) <= 2e-2 * abs(a) + 1e-3 for a, g in losses)


@pytest.mark.parametrize("resync", [True, False])
def test_closed_loop_deepfm_scaled(resync):
    w = synth.config(3).scaled(batch=384, vocab=3000, hidden=80, init_scale=0.05, lr=0.5, init_acc=0.1)
    losses = _closed_loop(w, 6, max_rows=300000, resync=resync)
    assert all(abs(a - g) <= 2e-2 * abs(a) + 1e-3 for a, g in losses)


def test_closed_loop_multihot_pooled_readout():
    # no first layer: the pooled vectors themselves feed the read-out (gE = g q), LR + FM beside them
    w = synth.config(4).scaled(batch=256, prepopulate=2000, init_scale=0.05, lr=0.5, init_acc=0.1)
    _closed_loop(w, 4, max_rows=200000, resync=False, prepop=True)


def test_loss_falls_on_a_planted_signal():
    """CUDA path alone, closed loop, 150 steps: every key carries a hidden score, a sample's label is 1 when the
    scores of its ids add up to more than the median; the linear weights (read-out: logit = b0 + R_lr) must
    pick that up — the mean log loss of the last 25 steps is well below that of the first 25."""
    from paper_1909_04823_b200.binding import DeviceBatch, Table
    w = synth.Workload("planted", 1024, 6, 8, 4, PART_HASH, OPT_ADAGRAD, OP_LR | OP_FM | OP_POOL, zipf_s=1.05, vocab=400,
                       shared_vocab=True, len_law="uniform", len_a=1, len_b=3, seed=21, init_scale=0.01, lr=0.1)
    st = synth.Stream(w)
    B, F, k = w.batch, w.fields, w.emb_dim
    hc = synth.head_constants(w)
    hc["c_fm"] = np.float32(0.0)
    hc["q"] = np.zeros(F * k, np.float32)                 # the signal is linear in the keys: read-out = b0 + R_lr
    hc["b0"] = np.float32(0.0)
    score = lambda ids: ((synth.fmix64(ids ^ np.uint64(0xABCDEF)) >> np.uint64(40)).astype(np.float64) / 2 ** 24 - 0.5)
    t = Table.for_workload(w, max_rows=20000, max_nnz=B * F * 4)
    dev = "cuda"
    try:
        hcd = {n: (torch.from_numpy(v).to(dev) if isinstance(v, np.ndarray) and v.ndim else v) for n, v in hc.items()}
        out_small = torch.empty((B, k + 4), device=dev); pooled = torch.empty((B, F * k), device=dev)
        logit = torch.empty(B, device=dev); loss = torch.empty(B, device=dev)
        gL = torch.empty(B, device=dev); gF = torch.empty(B, device=dev); gE = torch.empty((B, F * k), device=dev)
        hist = []
        for s in range(150):
            b = st.next_batch()
            per_sample = np.add.reduceat(score(b.ids), b.offsets[:-1:F][: B].astype(np.int64))
            y = (per_sample > 0.0).astype(np.float32)
            db = DeviceBatch.from_synth(b)
            t.find_or_insert(db, True)
            t.forward_fused(w.ops, db, None, pooled, out_small, None)
            t.head(w.ops, B, hcd, out_small, pooled, None, None, torch.from_numpy(y).to(dev), logit, loss, gL, gF, gE, None)
            t.backward_update(w.ops, db, out_small, pooled, None, gL * B, gF, gE, None, None)   # (sum, not mean: faster start)
            hist.append(float(loss.mean().item()))
        assert t.status() == 0
        first, last = np.mean(hist[:25]), np.mean(hist[-25:])
        assert abs(hist[0] - np.log(2.0)) < 1e-3          # all weights zero at the start: p = 1/2
        assert last < 0.6 * first, (first, last)
    finally:
        t.close()
