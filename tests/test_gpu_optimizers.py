"""Parity of the Adam (latent vectors, first dense layer) and FTRL-Proximal
(order-1 weights) updates of the CUDA path against the CPU oracle.  Needs a B200."""
import numpy as np
import pytest
import torch

from paper_1909_04823_b200 import synth
from paper_1909_04823_b200.synth import (LIN_FTRL, OP_DENSE1, OP_FM, OP_LR, OP_POOL, OPT_ADAGRAD, OPT_ADAM, OPT_SGD,
                                          PART_FIELD, PART_HASH)

pytestmark = pytest.mark.gpu


def _run(w, steps, max_rows, with_vals=False, repeat_first=0):
    """`repeat_first`: feed the first batch this many extra times, so that every key of it is
    touched on consecutive steps (moments and FTRL sums build up on the same rows)."""
    from harness import Pair
    st = synth.Stream(w, with_vals=with_vals)
    b = st.next_batch()
    p = Pair(w, max_rows, max_nnz=int(b.nnz * 1.5) + 1024)
    try:
        for s in range(steps):
            p.step(b, synth.upstream_grads(w, b.batch, s), check_init=(s == 0))
            if s >= repeat_first:
                b = st.next_batch()
    finally:
        p.close()


@pytest.mark.parametrize("partition", [PART_HASH, PART_FIELD])
def test_adam_lr_fm_pool(partition):
    w = synth.config(1).scaled(optimizer=OPT_ADAM, ops=OP_LR | OP_FM | OP_POOL, init_scale=0.05, lr=0.003,
                               partition=partition, shared_vocab=(partition == PART_HASH), shards=5)
    _run(w, 5, max_rows=30000, repeat_first=2)


@pytest.mark.parametrize("k", [4, 12, 64])
def test_adam_embedding_dims(k):
    w = synth.config(1).scaled(emb_dim=k, optimizer=OPT_ADAM, ops=OP_LR | OP_FM | OP_POOL, init_scale=0.05,
                               lr=0.002, batch=200, beta1=0.8, beta2=0.99)
    _run(w, 3, max_rows=20000, with_vals=True, repeat_first=1)


def test_adam_with_first_dense_layer():
    w = synth.config(3).scaled(batch=300, vocab=5000, hidden=80, init_scale=0.05, optimizer=OPT_ADAM, lr=0.002)
    _run(w, 4, max_rows=300000, repeat_first=2)


@pytest.mark.parametrize("opt", [OPT_SGD, OPT_ADAGRAD, OPT_ADAM])
def test_ftrl_linear_weights(opt):
    # order-1 weights by FTRL-Proximal (with l1 large enough that some stay exactly zero),
    # latent vectors by each of the other optimizers
    w = synth.config(1).scaled(optimizer=opt, lin_optimizer=LIN_FTRL, ops=OP_LR | OP_FM | OP_POOL, init_scale=0.05,
                               lr=0.003, ftrl_alpha=0.1, ftrl_beta=1.0, ftrl_l1=1.0, ftrl_l2=0.01, shards=3)
    _run(w, 5, max_rows=30000, repeat_first=3)


def test_ftrl_wide_and_deep_shape():
    w = synth.config(2).scaled(batch=640, vocab=20000, hidden=72, init_scale=0.05, lin_optimizer=LIN_FTRL,
                               ftrl_alpha=0.05, ftrl_l1=0.5)
    _run(w, 3, max_rows=400000, repeat_first=1)


def test_ftrl_zeroes_and_state_words_are_exact_on_first_touch():
    """First touch of a key with one occurrence: the gradient is a single term, so n = g^2,
    z = g and the thresholded weight are the same float32 operations on both sides."""
    from harness import Pair
    w = synth.Workload("ftrl_first", 64, 1, 4, 2, PART_HASH, OPT_SGD, OP_LR, lin_optimizer=LIN_FTRL,
                       ftrl_alpha=0.1, ftrl_beta=1.0, ftrl_l1=0.7, ftrl_l2=0.0, seed=21, init_scale=0.05)
    keys = synth.fmix64(np.arange(64, dtype=np.uint64) + np.uint64(1000))
    b = synth.Batch(64, 1, np.arange(65, dtype=np.int32), keys, None)
    p = Pair(w, 1000, 256, resync=False)      # keep the CUDA side's own results in its table
    try:
        g = synth.upstream_grads(w, 64, 0)
        r = p.step(b, g)
        rows = p.t.read_rows(r["db"].uniq_rows[:64])
        lin = rows["lin"].cpu().numpy()
        small = np.abs(g["gL"]) <= 0.7
        assert small.any() and (~small).any()
        assert not np.any(lin[small]) and np.all(lin[~small] != 0)
        assert np.all(np.sign(lin[~small]) == -np.sign(g["gL"][~small]))
        assert np.array_equal(rows["acc_lin"].cpu().numpy(), g["gL"] * g["gL"])
        assert np.array_equal(p.t.read_state2(r["db"].uniq_rows[:64])["lin2"].cpu().numpy(), g["gL"])
    finally:
        p.close()


def test_adam_step_count_survives_graph_replay():
    """Adam's bias correction counts backward calls on the device, so replaying a captured
    backward advances it exactly like separate calls do."""
    from paper_1909_04823_b200.binding import DeviceBatch, Table
    w = synth.config(1).scaled(optimizer=OPT_ADAM, ops=OP_LR | OP_FM | OP_POOL, init_scale=0.05, lr=0.003, batch=128)
    b = synth.Stream(w).next_batch()
    g = {n: torch.from_numpy(v).cuda() for n, v in synth.upstream_grads(w, b.batch, 0).items()}
    B, F, k = b.batch, w.fields, w.emb_dim
    res = []
    for use_graph in (False, True):
        t = Table.for_workload(w, max_rows=20000, max_nnz=b.nnz)
        try:
            db = DeviceBatch.from_synth(b)
            t.find_or_insert(db, True)
            out_small = torch.zeros((B, k + 4), device="cuda")
            pooled = torch.zeros((B, F * k), device="cuda")
            t.forward_fused(w.ops, db, None, pooled, out_small, None)
            call = lambda: t.backward_update(w.ops, db, out_small, pooled, None, g["gL"], g["gF"], g["gE"], None, None)
            torch.cuda.synchronize()
            if use_graph:
                call()                                       # step 1, outside the capture
                torch.cuda.synchronize()
                gr = torch.cuda.CUDAGraph()
                with torch.cuda.graph(gr):                   # capturing launches nothing
                    call()
                gr.replay(); gr.replay()                     # steps 2 and 3
            else:
                for _ in range(3):
                    call()
            torch.cuda.synchronize()
            assert t.status() == 0
            U = int(db.n_uniq.item())
            rows = t.read_rows(db.uniq_rows[:U])
            res.append({n: v.cpu().numpy().copy() for n, v in rows.items()})
        finally:
            t.close()
    # the forward results fed to the three backward calls are the same stale ones on both sides,
    # so the two runs execute identical arithmetic except for atomic summation order
    # (a sum that cancels to rounding size can come out with the other sign in another order, and Adam then
    # moves the weight by lr the other way: allow a handful of such elements)
    for n in ("emb", "lin", "acc_emb"):
        a, c = res[0][n].astype(np.float64), res[1][n].astype(np.float64)
        off = np.abs(a - c) > 2e-4 * np.abs(c) + 2e-6
        assert off.mean() < 1e-3, (n, int(off.sum()), off.size)
    # (a bias correction frozen at the captured step would shift EVERY weight of steps 2 and 3)
