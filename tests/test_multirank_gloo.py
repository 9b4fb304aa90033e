"""The N > 1 path of the benchmark (replicas only): two gloo ranks on CPU agree on
max-over-ranks time and summed work."""
import os
import socket

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
    from paper_2312_08538_b200 import multirank
    ms = 10.0 + 5.0 * rank          # rank 1 is the slow one
    value, used_ms = multirank.throughput(ms, 1000.0)
    q.put((rank, value, used_ms))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_report_whole_job_throughput():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, value, used_ms in got:
        assert used_ms == 15.0                       # the slowest rank
        assert abs(value - 2000.0 / 15e-3) < 1e-6    # both ranks' units over that time


def test_single_process_is_identity():
    from paper_2312_08538_b200 import multirank
    assert multirank.throughput(4.0, 8.0) == (2000.0, 4.0)
