"""World-size-2 check (gloo, CPU) of the benchmark's cross-rank aggregation."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, q):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_2308_15030_b200.replicas import aggregate_throughput, max_over_ranks
    ms = 10.0 if rank == 0 else 25.0                      # rank 1 is the slow replica
    value, ms_max = aggregate_throughput(2048, 100, ms)
    mx = max_over_ranks([float(rank), 5.0 - rank])
    dist.barrier()
    q.put((rank, value, ms_max, mx))
    dist.destroy_process_group()


def test_two_replicas_report_whole_job_throughput_at_the_slowest_rank():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, value, ms_max, mx in res:
        assert ms_max == 25.0
        assert abs(value - 2 * 2048 * 100 / 25e-3) < 1e-6 * value
        assert mx == [1.0, 5.0]


def test_single_process_is_identity():
    from paper_2308_15030_b200.replicas import aggregate_throughput
    v, ms = aggregate_throughput(10, 4, 2.0)
    assert ms == 2.0 and v == 10 * 4 / 2e-3
