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
