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


# ---------------------------------------------------------------- one worker per rank over gloo
class _OracleEngine:
    """The engine interface of ShardedConEF on top of the CPU oracle with one local worker: lets two
    gloo ranks run the sharded call sequence without a GPU.  Messages are torch views of numpy
    buffers so that the all-reduce works in place."""

    def __init__(self, tensors, q, c, lr):
        import numpy as np
        import torch
        from oracle import conef_oracle as orc
        self.np, self.torch, self.orc = np, torch, orc
        self.o = orc.ConEFOracle(tensors, 1, q, c, lr)
        self.total = 1
        self.res = None
        self.buf = {}

    def set_total_workers(self, n):
        self.total = n

    def message_elems(self, kind):
        return self.buf[kind].numel() if kind in self.buf else (1 if self.res is None else 0)

    def message(self, kind, worker):
        return self.buf[kind]

    def step(self, t, grads, phase):
        np, torch, orc = self.np, self.torch, self.orc
        if phase != 0:
            return
        self.res = self.o.step(t, [grads[0].numpy()])
        cat = lambda xs: torch.from_numpy(np.concatenate(xs).astype(np.float32)) if xs else torch.zeros(0)
        comp = self.o.compressed
        self.buf = {0: cat([self.res[l].msg[0] for l in comp]),
                    3: cat([self.res[l].msg[0] for l in sorted(self.res) if l not in comp])}

    def reduce_messages(self, kind):
        return self.buf[kind].clone()


def _sharded_worker(rank, world, port, q):
    import numpy as np
    import torch
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from oracle import conef_oracle as orc
    from paper_2312_08538_b200 import multirank
    tensors = [(8, 16, 1), (5, 1, 0)]
    qc = orc.QCfg(kind="randk", k_num=1, k_den=4, seed=3)
    cc = orc.CCfg(kind="int8", block=32)
    sh = multirank.ShardedConEF(_OracleEngine(tensors, qc, cc, 0.5), lowrank=False)
    rng = np.random.default_rng(100 + rank)
    outs = []
    for t in range(3):
        g = torch.from_numpy(rng.standard_normal(8 * 16 + 5).astype(np.float32))
        out = sh.step(t, g)
        outs.append({k: v.numpy().copy() for k, v in out.items()})
    q.put((rank, sh.eng.total, outs))
    dist.barrier()
    dist.destroy_process_group()


def test_one_worker_per_rank_matches_two_simulated_workers():
    import numpy as np
    from oracle import conef_oracle as orc
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_sharded_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=180) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    # the same job in one process with two simulated workers
    tensors = [(8, 16, 1), (5, 1, 0)]
    o = orc.ConEFOracle(tensors, 2, orc.QCfg(kind="randk", k_num=1, k_den=4, seed=3), orc.CCfg(kind="int8", block=32), 0.5)
    rngs = [np.random.default_rng(100), np.random.default_rng(101)]
    for t in range(3):
        res = o.step(t, [r.standard_normal(8 * 16 + 5).astype(np.float32) for r in rngs])
        for rank, total, outs in got:
            assert total == 2
            assert np.array_equal(outs[t][0], o.reduced(res, "values"))     # two addends: order does not matter
            assert np.array_equal(outs[t][3], o.reduced(res, "dense1d"))


def _sharded_timing_worker(rank, world, port, q):
    """The --sharded mode of the benchmark on two CPU ranks: the same step driver (one worker per
    rank, messages all-reduced between the phases) and the same timing helper, over the oracle."""
    import numpy as np
    import torch
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from oracle import conef_oracle as orc
    from paper_2312_08538_b200 import multirank
    tensors = [(8, 16, 1), (5, 1, 0)]
    sh = multirank.ShardedConEF(_OracleEngine(tensors, orc.QCfg(kind="randk", k_num=1, k_den=4, seed=3),
                                              orc.CCfg(kind="int8", block=32), 0.5), lowrank=False)
    g = torch.from_numpy(np.random.default_rng(7 + rank).standard_normal(8 * 16 + 5).astype(np.float32))
    calls = []
    ms = multirank.timed_steps(lambda t: calls.append(t) or sh.step(t, g), steps=3, warmup=2,
                               clock=multirank.WallClock(), barrier=dist.barrier)
    value, used_ms = multirank.throughput(ms, 8 * 16)      # one worker's compressed elements per rank
    q.put((rank, calls, ms, value, used_ms, sh.world))
    dist.barrier()
    dist.destroy_process_group()


def test_sharded_benchmark_driver_on_two_gloo_ranks():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_sharded_timing_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=180) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    slowest = max(g[2] for g in got)
    for rank, calls, ms, value, used_ms, world in got:
        assert calls == [0, 1, 2, 3, 4]          # warm-up steps then timed steps, step index advancing
        assert world == 2 and ms > 0
        assert used_ms == slowest                # the job's time is the slowest rank's
        assert abs(value - 2 * 8 * 16 / (slowest * 1e-3)) <= 1e-6 * value   # N = world size workers' elements
