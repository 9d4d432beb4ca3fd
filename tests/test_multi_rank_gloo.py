"""The N > 1 path of bench.py on CPU: two gloo ranks agree on the slowest rank's time, and the job value is the work of
all replicas over that time (weak scaling, replicas only: no data-path collective exists to test)."""
import os
import socket

import torch.multiprocessing as mp


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    import torch.distributed as dist
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    mine = 2.0 + 3.0 * rank                       # rank 1 is the slow one
    slowest = bench.max_over_ranks(mine)
    out.put((rank, slowest, bench.job_value(1000, world, slowest)))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_report_the_slowest_time_and_the_whole_job_value():
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
    assert [r[0] for r in res] == [0, 1]
    assert all(abs(r[1] - 5.0) < 1e-12 for r in res)
    assert all(abs(r[2] - 2 * 1000 / 5e-3) < 1e-6 for r in res)


def test_single_process_is_identity():
    import bench
    assert bench.max_over_ranks(1.25) == 1.25
    assert bench.job_value(10, 1, 2.0) == 10 / 2e-3
