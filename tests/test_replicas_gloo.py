"""The N > 1 path of the benchmark is "replicas only": every rank runs an independent step on
its own seeded batch and the job's time is the maximum over ranks.  This covers that host
logic with two gloo ranks on the CPU (no GPU, no data-path collective)."""
import os
import socket
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _worker(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    sys.path.insert(0, ROOT)
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    import bench
    import oracle
    from paper_2511_18868_b200 import workloads as wl
    dist.init_process_group("gloo", rank=rank, world_size=world)
    cfg = wl.scaled(wl.CONFIGS["tiny"], N=64)
    inp = wl.make_inputs(cfg, seed=bench.replica_seed(cfg, rank))
    # each replica is a complete, independent step (here: the oracle's, on the CPU)
    out = oracle.bandit_step(inp, cfg.iters)
    my_ms = 10.0 * (rank + 1)                      # pretend rank 1 is the slowest replica
    total_ms, = bench.reduce_max([my_ms], dist, torch.device("cpu"))
    # the batches differ between ranks, the reduced time does not
    digest = torch.tensor([float(np.abs(inp["x"]).sum()), float(out["best_arm"][0]), total_ms], dtype=torch.float64)
    gathered = [torch.zeros_like(digest) for _ in range(world)]
    dist.all_gather(gathered, digest)
    if rank == 0:
        np.save(os.path.join(out_dir, "gathered.npy"), torch.stack(gathered).numpy())
        with open(os.path.join(out_dir, "value.txt"), "w") as fh:
            fh.write(repr(bench.job_value(world, cfg.arms, total_ms)))
    dist.barrier()
    dist.destroy_process_group()


def test_two_replicas_max_over_ranks(tmp_path):
    world = 2
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    g = np.load(tmp_path / "gathered.npy")
    assert g.shape == (2, 3)
    assert g[0, 0] != g[1, 0]                      # independent batches
    assert g[0, 2] == g[1, 2] == 20.0              # max over ranks, seen by both
    value = float(open(tmp_path / "value.txt").read())
    assert value == 2 * 64 * 8 / 20e-3             # arms of both replicas / slowest time
