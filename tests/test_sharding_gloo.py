"""Multi-process sharding of the gate (CPU, gloo, world_size 2): groups are
independent, so every rank gates a contiguous range of groups and the only exchange
is an optional gather of the per-group results.  The per-rank computation here is
the oracle (no GPU on this machine); what is tested is the host-side partition and
gather logic that bench.py and a multi-GPU caller use."""
import os
import socket
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out_dir):
    sys.path.insert(0, ROOT)
    import oracle
    import paper_2605_05802_b200 as sr
    from paper_2605_05802_b200 import workloads as W

    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    w = W.agent_gate(K=15, n_groups=101)          # odd count: ranks get 51 and 50 groups
    lo, hi = sr.shard_groups(w.n_groups, world, rank)
    _, ps, mean, stop = oracle.gate(w.seqs[lo:hi], w.lens[lo:hi], w.K, 0.5, w.norm_mode)
    # gather the 1-byte masks (padded to the largest shard) on every rank
    cap = (w.n_groups + world - 1) // world
    mine = torch.full((cap,), 255, dtype=torch.uint8)
    mine[: hi - lo] = torch.from_numpy(stop)
    gathered = [torch.empty(cap, dtype=torch.uint8) for _ in range(world)]
    dist.all_gather(gathered, mine)
    full = np.concatenate([gathered[r].numpy()[: np.subtract(*sr.shard_groups(w.n_groups, world, r)[::-1])]
                           for r in range(world)])
    # timing reduction used by the benchmark: max over ranks
    t = torch.tensor([float(rank + 1)], dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    np.save(os.path.join(out_dir, f"mask_{rank}.npy"), full)
    np.save(os.path.join(out_dir, f"tmax_{rank}.npy"), t.numpy())
    dist.destroy_process_group()


def test_two_ranks_cover_all_groups_and_agree(tmp_path):
    sys.path.insert(0, ROOT)
    import oracle
    from paper_2605_05802_b200 import workloads as W

    world, port = 2, _free_port()
    mp.start_processes(_worker, args=(world, port, str(tmp_path)), nprocs=world, join=True,
                       start_method="spawn")
    w = W.agent_gate(K=15, n_groups=101)
    _, _, _, want = oracle.gate(w.seqs, w.lens, w.K, 0.5, w.norm_mode)
    for r in range(world):
        got = np.load(tmp_path / f"mask_{r}.npy")
        assert np.array_equal(got, want)
        assert np.load(tmp_path / f"tmax_{r}.npy")[0] == float(world)
    assert 0 < want.sum() < 101
