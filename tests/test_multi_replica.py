"""The N > 1 path of bench.py (independent replicas, no data-path collective): two gloo ranks on
the CPU agree on the job time (the slowest rank's) and on the aggregate value."""
import os
import socket
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank: int, world: int, port: int, out):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    seconds = 2.0 if rank == 0 else 3.0               # rank 1 is the slow replica
    t, value = bench.job_time_and_value(dist, seconds, 300.0, world, "cpu")
    dist.barrier()
    out.put((rank, t, value))
    dist.destroy_process_group()


def test_two_replicas_report_max_time_and_summed_units():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, t, value in res:
        assert t == 3.0 and value == 2 * 300.0 / 3.0


def test_single_process_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.job_time_and_value(None, 2.0, 100.0, 1, "cpu") == (2.0, 50.0)
