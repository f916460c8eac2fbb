"""The N > 1 path of the benchmark is "replicas only": ranks work independently and only their figures are combined.
This runs that combination on two CPU processes over gloo (no GPU)."""
import os
import socket
import sys

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
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    ms, e2e_s = (100.0, 2.0) if rank == 0 else (140.0, 1.5)      # rank 1 is the slower replica on the device-timed arm
    got = bench.reduce_over_replicas(ms, e2e_s, 512 * (rank + 1), 1024, 2010 + rank, torch.device("cpu"), world)
    dist.barrier()
    if rank == 0:
        torch.save(got, out)
    dist.destroy_process_group()


def test_replica_figures_combine_as_max_time_and_summed_work(tmp_path):
    out = str(tmp_path / "got.pt")
    mp.spawn(_worker, args=(2, _free_port(), out), nprocs=2, join=True)
    ms, e2e_s, tokens, e2e_tokens, launches = torch.load(out)
    assert (ms, e2e_s) == (140.0, 2.0)                  # slowest replica sets each time
    assert (tokens, e2e_tokens, launches) == (512 + 1024, 2048, 2010 + 2011)


def test_single_replica_is_passed_through():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.reduce_over_replicas(1.0, 2.0, 3, 4, 5, torch.device("cpu"), 1) == (1.0, 2.0, 3, 4, 5)
