"""World-size-2 CPU (gloo) test of the data-parallel host logic bench.py uses at N > 1:
rank-sharded batches with replicated weights, no data-path collective, max-over-ranks timing."""
import hashlib
import os
import socket
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _digest(t: torch.Tensor) -> int:
    return int.from_bytes(hashlib.sha256(t.numpy().tobytes()).digest()[:7], "little")


def _worker(rank, world, port, ret):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    import oracle
    from paper_1609_07061_b200 import workloads
    plan = bench.shard_plan(world, rank, batch_per_gpu=6)
    assert plan["stream"] == rank and plan["global_rows"] == 6 * world
    dims = (64, 512, 256, 10)      # wide enough that thresholds in [-64, 64] do not saturate
    wl = workloads.mnist_mlp(M=plan["rows"], dims=dims, seed=1, stream=plan["stream"])
    # replicated weights / thresholds, rank-specific inputs
    wd = torch.tensor([_digest(w) for w in wl.Ws] + [_digest(t) for t in wl.Ts], dtype=torch.int64)
    xd = torch.tensor([_digest(wl.X)], dtype=torch.int64)
    wall = [torch.zeros_like(wd) for _ in range(world)]
    xall = [torch.zeros_like(xd) for _ in range(world)]
    dist.all_gather(wall, wd)
    dist.all_gather(xall, xd)
    assert all(torch.equal(w, wall[0]) for w in wall)
    assert len({int(x.item()) for x in xall}) == world
    # every rank's shard result equals the oracle on that shard alone (no cross-rank dependence)
    scores = oracle.mlp_forward(wl.X.numpy().astype(np.int32), [oracle.sign(w.numpy()) for w in wl.Ws],
                                [t.numpy() for t in wl.Ts])
    assert scores.shape == (plan["rows"], dims[-1])
    # timing reduction: max over ranks
    t = torch.tensor([1.0 + rank, 10.0 - rank], dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    assert t.tolist() == [float(world), 10.0]
    # whole-job throughput = units of all ranks / max time
    ops = sum(bench._ops(plan["rows"]))
    value = world * ops / t[0].item()
    ret[rank] = (value, _digest(torch.from_numpy(scores)))
    dist.barrier()
    dist.destroy_process_group()


def test_two_rank_sharding_gloo():
    world = 2
    port = _free_port()
    ctx = mp.get_context("spawn")
    ret = ctx.Manager().dict()
    procs = [ctx.Process(target=_worker, args=(r, world, port, ret)) for r in range(world)]
    for p in procs:
        p.start()
    for p in procs:
        p.join(timeout=180)
        assert p.exitcode == 0
    assert len(ret) == world
    assert ret[0][0] == ret[1][0]              # both ranks agree on the whole-job figure
    assert ret[0][1] != ret[1][1]              # different shards give different scores
