"""World-size-2 check (gloo, CPU) of the multi-rank plumbing the benchmark
uses: ranks hold independent column shards / replicas, Eq. 3 needs no
exchange between them, timings combine by MAX and the work by SUM."""
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
    port = s.getsockname()[1]
    s.close()
    return port


def _worker(rank, world, port, out_dir):
    sys.path.insert(0, ROOT)
    import oracle
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    N, P, S, R = 6, 1000, 4, 2
    g = torch.Generator().manual_seed(0)
    x = (torch.randn(N, P, generator=g) * 0.05).numpy()
    idx = oracle.select_peers(1, 0, N, S, R)          # every rank derives the same table from the seed
    # column shard of this rank, cut at an arbitrary column (not a segment boundary)
    cut = [0, 437, P]
    a, b = cut[rank], cut[rank + 1]
    shard = np.ascontiguousarray(x[:, a:b])
    part = oracle.segment_aggregate(shard, idx, S, R, P=P, p_begin=a, p_end=b)
    # timing and work reductions as the benchmark does them
    t = torch.tensor([10.0 + rank], dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    units = torch.tensor([float(N * (b - a))], dtype=torch.float64)
    dist.all_reduce(units, op=dist.ReduceOp.SUM)
    np.save(os.path.join(out_dir, "part%d.npy" % rank), part)
    if rank == 0:
        np.save(os.path.join(out_dir, "meta.npy"), np.array([float(t), float(units)]))
    dist.barrier()
    dist.destroy_process_group()


def test_column_shards_over_two_ranks(tmp_path):
    import oracle
    port = _free_port()
    mp.spawn(_worker, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    N, P, S, R = 6, 1000, 4, 2
    g = torch.Generator().manual_seed(0)
    x = (torch.randn(N, P, generator=g) * 0.05).numpy()
    idx = oracle.select_peers(1, 0, N, S, R)
    full = oracle.segment_aggregate(x, idx, S, R)
    got = np.concatenate([np.load(tmp_path / "part0.npy"), np.load(tmp_path / "part1.npy")], axis=1)
    assert (got == full).all()
    t_max, units = np.load(tmp_path / "meta.npy")
    assert t_max == 11.0 and units == N * P


def _worker_sharded(rank, world, port, out_dir):
    """Worker-sharded round over two ranks: each rank hosts half of the workers, the rows
    it pulls come from the owning rank (here: an all_gather stands in for the NVLink loads),
    and the traffic matrix each rank derives from the shared peer table agrees."""
    sys.path.insert(0, ROOT)
    import oracle
    from paper_1908_07782_b200 import sharding
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    N, P, S, R = 7, 501, 3, 2                               # uneven shares: 4 and 3 workers
    a, b = sharding.worker_range(rank, world, N)
    g = torch.Generator().manual_seed(100 + rank)
    mine = torch.randn(b - a, P, generator=g) * 0.05        # only the hosted rows exist here
    idx = oracle.select_peers(1, 0, N, S, R)
    # the pull: every rank obtains the rows its hosted workers' tables name
    sizes = [sharding.worker_range(r, world, N) for r in range(world)]
    m = max(hi - lo for lo, hi in sizes)                    # uneven shares: pad to the largest
    padded = torch.zeros(m, P)
    padded[: b - a] = mine
    got = [torch.empty(m, P) for _ in range(world)]
    dist.all_gather(got, padded)
    parts = [got[r][: sizes[r][1] - sizes[r][0]] for r in range(world)]
    rows = torch.cat(parts).numpy()
    full = oracle.segment_aggregate(rows, idx, S, R)        # every worker; this rank keeps its own
    np.save(os.path.join(out_dir, "hosted%d.npy" % rank), full[a:b])
    np.save(os.path.join(out_dir, "rows%d.npy" % rank), mine.numpy())
    t = torch.from_numpy(sharding.pull_traffic(idx, world, P, 4))
    ref = t.clone()
    dist.broadcast(ref, src=0)
    assert torch.equal(t, ref)
    dist.barrier()
    dist.destroy_process_group()


def test_worker_shards_over_two_ranks(tmp_path):
    import oracle
    from paper_1908_07782_b200 import sharding
    port = _free_port()
    mp.spawn(_worker_sharded, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    N, P, S, R = 7, 501, 3, 2
    rows = np.concatenate([np.load(tmp_path / "rows0.npy"), np.load(tmp_path / "rows1.npy")])
    assert rows.shape == (N, P)
    idx = oracle.select_peers(1, 0, N, S, R)
    full = oracle.segment_aggregate(rows, idx, S, R)
    got = np.concatenate([np.load(tmp_path / "hosted0.npy"), np.load(tmp_path / "hosted1.npy")])
    assert (got == full).all()
    assert sharding.worker_range(0, 2, N) == (0, 4) and sharding.worker_range(1, 2, N) == (4, 7)
