"""The N > 1 leg of bench.py without GPUs: ranks are independent replicas (the path has no exchange step), and the
only communication is the reduction of the timing (max over ranks) and of the units processed (sum).  Two gloo
ranks on the CPU run that reduction."""
import os
import socket
import sys

import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world),
                      LOCAL_RANK=str(rank))
    sys.path.insert(0, ROOT)
    import torch.distributed as dist
    import bench
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        assert bench.dist_env() == (rank, rank, world)
        # rank r took (3 + r) ms for its 9 * (r + 1) positions
        ms, units = bench.reduce_max_and_sum(3.0 + rank, 9.0 * (rank + 1), world, device="cpu")
        out[rank] = (ms, units)
    finally:
        dist.destroy_process_group()


def test_two_replicas_report_the_slowest_time_and_the_summed_work():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    out = mp.Manager().dict()
    mp.spawn(_worker, args=(2, port, out), nprocs=2, join=True)
    assert out[0] == out[1] == (4.0, 27.0)          # max(3, 4) ms, 9 + 18 positions: value = 27 / 4 ms


def test_a_single_replica_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.reduce_max_and_sum(2.5, 9.0, 1) == (2.5, 9.0)
