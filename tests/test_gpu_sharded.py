"""Shards spread over several tables (one per process in production, Algorithm 1): on one
GPU the ranks run one after the other and the exchange is a stack / a sum of their messages,
so that every CUDA entry point of the multi-process path is compared with the oracle of the
whole model.  Needs a B200."""
import numpy as np
import pytest
import torch

from harness import SUMTOL, SUMTOL_FWD, close32, close_gemm, rows_per_shard_for, u32
from oracle import Oracle
from paper_1909_04823_b200 import synth
from paper_1909_04823_b200.synth import (OP_DENSE1, OP_FM, OP_LR, OP_POOL, OPT_ADAGRAD, OPT_SGD, PART_FIELD,
                                          PART_HASH)

pytestmark = pytest.mark.gpu


def _run(w, world, steps=2):
    from paper_1909_04823_b200.binding import DeviceBatch, Table
    from paper_1909_04823_b200.sharded import ShardedTable, owned_shards
    B, F, k, S, H = w.batch, w.fields, w.emb_dim, w.shards, w.hidden
    ops = w.ops
    st = synth.Stream(w)
    batch = st.next_batch()
    o = Oracle.for_workload(w)
    stack = {}
    ranks = []
    for r in range(world):
        t = Table.for_workload(w, max_rows=200000, max_nnz=int(batch.nnz * 1.5) + 1024,
                               rows_per_shard=rows_per_shard_for(w, 200000), shard_world=world, shard_rank=r)
        # the "network": gather = the stack of all ranks' messages, reduce = the sum of all ranks' tensors
        ranks.append(ShardedTable(t, world, r, gather=lambda local, n: stack["msgs"],
                                  reduce=lambda x: x.copy_(stack["sum"])))
    if H:
        W1 = synth.dense1_weights(w)
        o.dense1_set(W1)
        for rk in ranks:
            rk.t.dense1_set(torch.from_numpy(W1).cuda())
    try:
        for step in range(steps):
            g = synth.upstream_grads(w, B, step)
            gd = {n: torch.from_numpy(v).cuda() for n, v in g.items()}
            fi = o.find_or_insert(batch)
            op = o.forward_partials(ops, batch, fi, want_pooled=True, want_dense=bool(ops & OP_DENSE1))
            oa = o.aggregate(B, op)
            sabs = o.forward_original(ops & ~OP_DENSE1, batch)["Sabs"]
            dbs, msgs, pooled, Zs = [], [], [], []
            for r, rk in enumerate(ranks):
                db = DeviceBatch.from_synth(batch)
                rk.t.find_or_insert(db, True)
                assert rk.t.status() == 0
                mine = np.isin(fi["shards"], owned_shards(S, world, r))
                rows = u32(db.rows)[:batch.nnz]
                assert np.array_equal(rows[mine], fi["rows"][mine]) and np.all(rows[~mine] == 0xFFFFFFFF)
                assert int(db.n_uniq.item()) == int(np.isin(fi["uniq_shard"], owned_shards(S, world, r)).sum())
                pl = torch.zeros((B, F * k), device="cuda")
                Z = torch.zeros((B, max(H, 1)), device="cuda")
                msgs.append(rk.forward_local(ops, db, pl, Z))
                dbs.append(db); pooled.append(pl); Zs.append(Z)
            # exchange, then the rest of the forward on every rank
            outs = []
            if ops & (OP_LR | OP_FM):
                stack["msgs"] = torch.stack(msgs)
            for r, rk in enumerate(ranks):
                out_small = torch.full((B, k + 4), float("nan"), device="cuda")
                pl_all = None
                if ops & OP_POOL:
                    stack["sum"] = torch.stack(pooled).sum(0)
                    pl_all = rk.forward_finish(ops & ~OP_DENSE1, B, msgs[r], out_small, pooled[r], None)
                else:
                    rk.forward_finish(ops & ~(OP_DENSE1 | OP_POOL), B, msgs[r], out_small)
                if ops & OP_DENSE1:
                    stack["sum"] = torch.stack(Zs).sum(0)
                outs.append((out_small, pl_all))
            torch.cuda.synchronize()
            if ops & OP_DENSE1:
                Zsum = torch.stack(Zs).sum(0)
                close_gemm(Zsum.cpu().numpy(), oa["Z"], "Z")
            xa, xl = SUMTOL_FWD * sabs[:, :k], SUMTOL_FWD * sabs[:, k]
            for r, (out_small, pl_all) in enumerate(outs):
                if ops & (OP_LR | OP_FM):
                    assert torch.equal(out_small.view(torch.int32), outs[0][0].view(torch.int32)), "every rank: same bits"
                    osm = out_small.cpu().numpy()
                    if ops & OP_FM:
                        close32(osm[:, :k], oa["A"], "A", extra=xa)
                        close32(osm[:, k + 2], oa["Q"], "Q", extra=SUMTOL_FWD * oa["Q"])
                        AA = np.sum(oa["A"] ** 2, axis=1)
                        close32(osm[:, k + 1], oa["fm2"], "fm2",
                                extra=SUMTOL_FWD * (AA + np.abs(oa["Q"])) + np.sum(np.abs(oa["A"]) * xa, axis=1))
                    if ops & OP_LR:
                        close32(osm[:, k], oa["lr"], "R_lr", extra=xl)
                if pl_all is not None:
                    close32(pl_all.cpu().numpy(), oa["pooled"], "pooled (summed over ranks)")
            # backward: no exchange; stage-wise from the oracle's aggregate
            ob = o.backward_update(ops, batch, fi, oa["A"].astype(np.float32),
                                   oa["pooled"].astype(np.float32) if oa["pooled"] is not None else None,
                                   g.get("gL"), g.get("gF"), g.get("gE") if (ops & OP_POOL) else None,
                                   g.get("gZ") if (ops & OP_DENSE1) else None)
            o32 = np.zeros((B, k + 4), dtype=np.float32)
            o32[:, :k] = oa["A"].astype(np.float32)
            gemm = bool(ops & OP_DENSE1)
            for r, rk in enumerate(ranks):
                own = owned_shards(S, world, r)
                gE_work = torch.empty((B, F * k), device="cuda") if gemm else None
                # the wgrad of the row-split layer wants this rank's own pooled blocks (zero elsewhere)
                pl_local = torch.from_numpy(np.where(np.isin(np.arange(F) % S, own).repeat(k)[None],
                                                     oa["pooled"].astype(np.float32), 0.0).astype(np.float32)).cuda() \
                    if (w.partition == PART_FIELD and oa["pooled"] is not None) else pooled[r]
                rk.backward_update(ops, dbs[r], torch.from_numpy(o32).cuda(), pl_local, Zs[r], gd.get("gL"), gd.get("gF"),
                                   gd.get("gE") if (ops & OP_POOL) else None, gd.get("gZ") if gemm else None, gE_work)
                torch.cuda.synchronize()
                assert rk.t.status() == 0
                sel = np.nonzero(np.isin(fi["uniq_shard"], own))[0]
                U = len(sel)
                ref = o.read_rows(fi["uniq_shard"][sel], fi["uniq_row"][sel])
                got = rk.t.read_rows(dbs[r].uniq_rows[:U])
                Gv, Gw = ob["Gv"][sel].astype(np.float64), ob["Gw"][sel].astype(np.float64)
                for name, Gk, Sk in (("emb", Gv, ob["Sv"][sel]), ("lin", Gw, ob["Sw"][sel])):
                    dG = 1e-5 * np.abs(Gk) + 1e-6 + SUMTOL * Sk
                    if gemm:
                        dG = dG + 2e-2 * np.abs(Gk) + 1e-3 * max(float(np.abs(Gk).max()), 1e-30)
                    if w.optimizer == OPT_SGD:
                        extra = w.lr * dG
                    else:
                        acc = ref["acc_" + name].astype(np.float64)
                        extra = w.lr * np.minimum(2.0, 2.0 * dG / (np.sqrt(acc) + w.eps))
                    (close_gemm if gemm else close32)(got[name].cpu().numpy(), ref[name], f"rank {r} {name}", extra=extra)
                # resync this rank's rows (and W1) from the oracle so that the next step starts equal
                td = lambda a: torch.from_numpy(np.ascontiguousarray(a)).cuda()
                sgd = w.optimizer == OPT_SGD
                rk.t.write_rows(dbs[r].uniq_rows[:U], td(ref["emb"]), td(ref["lin"]),
                                None if sgd else td(ref["acc_emb"]), None if sgd else td(ref["acc_lin"]))
            if gemm:
                W1o, accW1o = o.dense1_get()
                blk = np.arange(F * k) // k                       # field of every row of W1
                for r, rk in enumerate(ranks):
                    rows_own = np.isin(blk % S, owned_shards(S, world, r))
                    Gk = ob["gW1"].astype(np.float64)
                    dG = 2e-2 * np.abs(Gk) + 1e-3 * max(float(np.abs(Gk).max()), 1e-30)
                    extra = w.lr * dG if w.optimizer == OPT_SGD else \
                        w.lr * np.minimum(2.0, 2.0 * dG / (np.sqrt(accW1o.astype(np.float64)) + w.eps))
                    got = rk.t.dense1_get().cpu().numpy()
                    close_gemm(got[rows_own], W1o[rows_own], f"rank {r} W1 (own rows)", extra=extra[rows_own])
                    rk.t.dense1_set(torch.from_numpy(W1o).cuda())
                    rk.t.dense1_set_state(torch.from_numpy(accW1o).cuda(), None)
            batch = st.next_batch()
    finally:
        for rk in ranks:
            rk.t.close()
        o.close()


@pytest.mark.parametrize("world", [2, 3])
@pytest.mark.parametrize("partition", [PART_HASH, PART_FIELD])
def test_lr_fm_pool_over_ranks(world, partition):
    w = synth.config(1).scaled(shards=7, partition=partition, shared_vocab=(partition == PART_HASH),
                               ops=OP_LR | OP_FM | OP_POOL, init_scale=0.05, optimizer=OPT_ADAGRAD, batch=256)
    _run(w, world)


def test_more_ranks_than_shards_leaves_idle_ranks():
    w = synth.config(1).scaled(shards=2, ops=OP_LR | OP_FM, init_scale=0.05, batch=64)
    _run(w, 3, steps=1)


def test_deepfm_first_layer_over_ranks():
    w = synth.config(3).scaled(batch=256, vocab=5000, hidden=80, init_scale=0.05)
    _run(w, 4)
