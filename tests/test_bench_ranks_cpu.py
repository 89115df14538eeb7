"""The multi-rank timing logic of bench.py on CPU: two gloo ranks, the slowest rank sets the
time and the reported value is the whole job's (independent replicas, no data-path collective)."""
import os
import socket
import sys

import pytest
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import torch.distributed as dist
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        ms_local, e2e_local = (2.0, 9.0) if rank == 0 else (3.0, 7.0)
        dist.barrier()
        ms, e2e = bench.max_over_ranks([ms_local, e2e_local], dist, "cpu")
        out.put((rank, ms, e2e, bench.whole_job_value(1e12, world, ms)))
    finally:
        dist.destroy_process_group()


def test_two_ranks_take_the_slowest_time_and_sum_the_work():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, ms, e2e, value in res:
        assert ms == 3.0 and e2e == 9.0                    # max over ranks, per quantity
        assert value == pytest.approx(2 * 1e12 / 3e-3)     # both replicas' work over the slowest time


def test_single_process_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks([1.5, 2.5]) == [1.5, 2.5]
    assert bench.whole_job_value(10.0, 1, 2.0) == pytest.approx(5000.0)
