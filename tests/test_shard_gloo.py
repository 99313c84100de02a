"""The multi-GPU path on CPU: two gloo ranks shard a workload by whole batch entries (rows are
independent, nothing is exchanged on the data path), each computes its shard, and the pieces put
together equal the unsharded result.  The oracle stands in for the device here; what is tested is
the host logic that bench.py's N > 1 mode relies on: the partition, the head index of a shard that
starts mid-tensor, and the max-over-ranks timing reduction."""
import os
import socket

import numpy as np
import pytest


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out_dir):
    import torch
    import torch.distributed as dist
    from oracle import hccs_oracle as orc
    from paper_2604_02292_b200 import workloads
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    wl = workloads.make_config(3, batch=5)                       # causal, 8 heads, odd batch count
    Bt, H, Lq, Lk = wl.shape
    r0, r1 = workloads.shard_rows(wl.rows, world, rank, granule=H * Lq)
    assert r0 % (H * Lq) == 0 and (r1 % (H * Lq) == 0 or r1 == wl.rows)
    b0, b1 = r0 // (H * Lq), r1 // (H * Lq)
    mine = orc.forward(wl.logits[b0:b1], wl.theta, orc.MODE_CAUSAL)   # a shard is a tensor of its own
    # every rank reports its time; the job's time is the slowest rank's
    t = torch.tensor([float(rank + 1)])
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    assert t.item() == float(world)
    counts = torch.tensor([r1 - r0])
    dist.all_reduce(counts)
    assert counts.item() == wl.rows                               # the shards cover every row once
    np.save(os.path.join(out_dir, f"part{rank}.npy"), mine)
    dist.barrier()
    if rank == 0:
        whole = orc.forward(wl.logits, wl.theta, orc.MODE_CAUSAL)
        parts = np.concatenate([np.load(os.path.join(out_dir, f"part{r}.npy")) for r in range(world)])
        assert parts.shape == whole.shape and (parts == whole).all()
    dist.destroy_process_group()


def test_two_ranks_shard_without_exchange(tmp_path):
    import torch.multiprocessing as mp
    from oracle import hccs_oracle
    hccs_oracle.build()
    mp.spawn(_worker, args=(2, _free_port(), str(tmp_path)), nprocs=2, join=True)


def test_shard_rows_partition():
    from paper_2604_02292_b200.workloads import shard_rows
    for total, world, g in ((1000, 3, 1), (1048576, 8, 256), (7, 4, 2), (5 * 1024, 2, 1024), (0, 2, 4)):
        cuts = [shard_rows(total, world, r, g) for r in range(world)]
        assert cuts[0][0] == 0 and cuts[-1][1] == total
        for (a0, a1), (b0, b1) in zip(cuts, cuts[1:]):
            assert a1 == b0 and a0 <= a1
        assert all(c[0] % g == 0 for c in cuts)
