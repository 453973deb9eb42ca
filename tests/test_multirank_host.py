"""Host-side logic of the N > 1 benchmark path on CPU (gloo, world_size 2):
replicas get distinct data streams, the job time is the slowest rank's, and
the reported throughput is the aggregate over ranks."""
import os
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    import bench
    from paper_1909_04823_b200 import synth
    dist.init_process_group("gloo", rank=rank, world_size=world)
    w = bench.per_rank_workload(synth.config(1), rank, world)
    b = synth.Stream(w).next_batch()
    ms = 10.0 + 5.0 * rank                       # rank 1 is the slow one
    slow = bench.max_over_ranks(ms, world)
    digest = torch.tensor([float(np.bitwise_xor.reduce(b.ids) % (1 << 40))], dtype=torch.float64)
    both = [torch.zeros_like(digest) for _ in range(world)]
    dist.all_gather(both, digest)
    out[rank] = (slow, bench.job_throughput(w.batch, world, slow), [float(x.item()) for x in both], b.nnz)
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_gloo():
    world, port = 2, 29617
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
    assert set(out.keys()) == {0, 1}
    for r in range(world):
        slow, thr, digests, nnz = out[r]
        assert slow == 15.0                                   # max over ranks on every rank
        assert abs(thr - 2 * 512 / 0.015) < 1e-6              # whole-job samples/s
        assert digests[0] != digests[1]                       # replicas see different batches
    assert out[0][2] == out[1][2]


# ---- shards spread over processes: the exchange step of Algorithm 1 over gloo ----------------
def _shard_worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    from oracle import Oracle
    from paper_1909_04823_b200 import synth
    from paper_1909_04823_b200.sharded import _dist_gather, _dist_reduce, owned_shards
    dist.init_process_group("gloo", rank=rank, world_size=world)
    w = synth.config(1).scaled(shards=5, ops=7, batch=64, init_scale=0.5)
    b = synth.Stream(w).next_batch()                    # the same batch on every process (Section 6)
    o = Oracle.for_workload(w)
    fi = o.find_or_insert(b)
    op = o.forward_partials(w.ops, b, fi)
    own = owned_shards(w.shards, world, rank)
    # this process's message: its own shards' partials added in shard order (M_1, M_1^lr, M_2 columns)
    msg = torch.from_numpy(op["part_small"][own].sum(0))
    allmsg = _dist_gather(msg, world)                   # [world][B][k+4], rank order
    tot = allmsg.sum(0).numpy()
    pooled_own = torch.from_numpy(op["part_pooled"][own].sum(0))
    pooled = _dist_reduce(pooled_own.clone()).numpy()
    agg = o.aggregate(w.batch, op)
    k = w.emb_dim
    A, lr, Q = tot[:, :k], tot[:, k], tot[:, k + 1]
    out[rank] = (float(np.abs(A - agg["A"]).max()), float(np.abs(lr - agg["lr"]).max()),
                 float(np.abs(0.5 * (np.sum(A * A, 1) - Q) - agg["fm2"]).max()),
                 float(np.abs(pooled - agg["pooled"]).max()), own, allmsg.numpy().tobytes())
    dist.barrier()
    dist.destroy_process_group()


def test_two_level_aggregation_over_two_gloo_ranks_equals_the_single_process_aggregate():
    world, port = 2, 29641
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_shard_worker, args=(world, port, out), nprocs=world, join=True)
    assert sorted(out[0][4] + out[1][4]) == [0, 1, 2, 3, 4] and not set(out[0][4]) & set(out[1][4])
    for r in range(world):
        assert max(out[r][:4]) < 1e-9                    # (+) over ranks of (+) over own shards = (+) over all shards
    assert out[0][5] == out[1][5]                        # every process holds the same gathered messages
