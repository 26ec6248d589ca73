"""Host logic of the N > 1 benchmark path on two CPU ranks (gloo): events are sharded by sequence with no
data-path collective, the timed value is the max over ranks and the throughput counts every rank's events."""
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


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    import bench
    from paper_2605_14292_b200 import synth
    dist.init_process_group("gloo", rank=rank, world_size=world)
    assert bench.dist_env() == (rank, rank, world)
    # every rank draws its own batch (seed = rank), as bench.py does: shards differ, nothing is exchanged
    ev = synth.make_c3(seed=rank, B=1, L=2, H=2)
    digest = float(ev.V.astype(np.float64).sum())
    ms = 10.0 * (rank + 1)                              # rank 1 is the slow one
    worst = bench.reduce_max(ms, world, torch.device("cpu"))
    value = bench.events_per_second(ev.n_events, world, 4, worst)
    gathered = [None] * world
    dist.all_gather_object(gathered, (digest, ev.n_events))
    if rank == 0:
        torch.save({"worst": worst, "value": value, "gathered": gathered}, out)
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_shard_events_and_time_is_max_over_ranks(tmp_path):
    out = str(tmp_path / "r0.pt")
    mp.spawn(_worker, args=(2, _free_port(), out), nprocs=2, join=True)
    r = torch.load(out, weights_only=False)
    assert r["worst"] == 20.0
    (d0, e0), (d1, e1) = r["gathered"]
    assert d0 != d1 and e0 == e1 == 4                   # different shards of equal size
    assert abs(r["value"] - (e0 + e1) * 4 / 20e-3) < 1e-6


def test_single_rank_reduce_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.reduce_max(3.5, 1, torch.device("cpu")) == 3.5
    assert bench.events_per_second(4096, 1, 10, 1000.0) == 40960.0
