"""Multi-GPU is replicas only (requests are independent; no collective on the data path).  The host
logic the benchmark uses for N > 1 -- sharding the documents of a batch over ranks and reducing the
per-rank timings with MAX / the per-rank throughputs with SUM -- is exercised here with two gloo
ranks on CPU."""
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


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import workloads as wl
    from paper_2607_29678_b200.sharding import shard_documents
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    lens = wl.batch_lengths(7, 64, 350_000, 1.0, 10_000, 3_000_000)
    mine = shard_documents(lens, world)[rank]
    t = torch.tensor([float(sum(lens[i] for i in mine))], dtype=torch.float64)     # stand-in for a per-rank time
    tmax = t.clone(); dist.all_reduce(tmax, op=dist.ReduceOp.MAX)
    tsum = t.clone(); dist.all_reduce(tsum, op=dist.ReduceOp.SUM)
    gathered = [None] * world
    dist.all_gather_object(gathered, sorted(mine))
    if rank == 0:
        np.save(out, np.array([tmax.item(), tsum.item(), float(lens.sum())] + [float(len(g)) for g in gathered]))
        flat = sorted(i for g in gathered for i in g)
        assert flat == list(range(64))
    dist.destroy_process_group()


def test_two_rank_sharding_and_reductions(tmp_path):
    out = str(tmp_path / "r.npy")
    mp.spawn(_worker, args=(2, _free_port(), out), nprocs=2, join=True)
    tmax, tsum, total, n0, n1 = np.load(out)
    assert tsum == total                        # every document on exactly one rank
    assert tmax <= 0.6 * total                  # longest-first greedy split is balanced
    assert n0 + n1 == 64
