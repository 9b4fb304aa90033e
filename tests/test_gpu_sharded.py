"""One worker per rank (messages all-reduced between the library's calls) on one GPU: two contexts
with one worker each, the all-reduce done by hand, must reproduce one context with two simulated
workers bit for bit; and ShardedConEF with a single rank must reproduce the plain call sequence."""
import numpy as np
import pytest
import torch

from paper_2312_08538_b200 import workloads as wl
from tests import parity_util as pu

pytestmark = pytest.mark.gpu


def _allreduce(engs, kind):
    bufs = [e.message(kind, 0) for e in engs]
    if bufs[0].numel() == 0:
        return
    total = bufs[0].clone()
    for b in bufs[1:]:
        total += b                      # rank order, fp32
    for b in bufs:
        b.copy_(total)


@pytest.mark.parametrize("name", ["tiny", "resnet50-mini", "gpt2-xl-mini"])
def test_two_single_worker_contexts_equal_one_two_worker_context(name):
    from paper_2312_08538_b200 import binding as b
    cfg = wl.config(name)
    cfg["n_workers"] = 2
    lowrank = cfg["q"]["kind"] == "lowrank"
    q0 = wl.q_init(cfg, "cuda") if lowrank else None
    ref = b.ConEF(cfg["tensors"], 2, cfg["q"], cfg["c"], cfg["lr"], q_init=q0)
    ranks = [b.ConEF(cfg["tensors"], 1, cfg["q"], cfg["c"], cfg["lr"], q_init=q0) for _ in range(2)]
    for e in ranks:
        e.set_total_workers(2)
    total = wl.total_elems(cfg["tensors"])
    x_ref = torch.linspace(-1, 1, total, device="cuda")
    xs = [x_ref.clone() for _ in ranks]
    for t in range(3):
        gd = [wl.gradient(cfg, i, t, device="cuda") for i in range(2)]
        out_ref = ref.full_step(t, gd)
        ref.apply_update(x_ref, out_ref)
        outs = [dict() for _ in ranks]
        for i, e in enumerate(ranks):
            e.step(t, [gd[i]], 0)
        _allreduce(ranks, b.MSG_DENSE1D)
        if lowrank:
            _allreduce(ranks, b.MSG_P)
            for i, e in enumerate(ranks):
                outs[i][b.MSG_P] = e.reduce_messages(b.MSG_P)
                e.step(t, [gd[i]], 1)
            _allreduce(ranks, b.MSG_Q)
            for i, e in enumerate(ranks):
                outs[i][b.MSG_Q] = e.reduce_messages(b.MSG_Q)
        else:
            _allreduce(ranks, b.MSG_VALUES)
            for i, e in enumerate(ranks):
                outs[i][b.MSG_VALUES] = e.reduce_messages(b.MSG_VALUES)
        for i, e in enumerate(ranks):
            if e.message_elems(b.MSG_DENSE1D):
                outs[i][b.MSG_DENSE1D] = e.reduce_messages(b.MSG_DENSE1D)
            e.apply_update(xs[i], outs[i])
            for k, v in out_ref.items():
                assert torch.equal(outs[i][k], v), f"step {t} rank {i} message {k}"
            assert torch.equal(xs[i], x_ref), f"step {t} rank {i}: parameters differ"
            for l, (r_, c_, comp) in enumerate(cfg["tensors"]):
                if comp and c_ > 1:
                    a_ref, s_ref = ref.state(i, l)
                    a, s = e.state(0, l)
                    assert torch.equal(a, a_ref) and (s is None or torch.equal(s, s_ref)), f"state of rank {i} tensor {l}"
        assert all(e.last_status() == 0 for e in ranks)


def test_sharded_wrapper_with_one_rank_is_the_plain_sequence():
    from paper_2312_08538_b200 import binding as b
    from paper_2312_08538_b200 import multirank
    cfg = wl.config("gpt2-small-mini")
    q0 = wl.q_init(cfg, "cuda")
    plain = b.ConEF(cfg["tensors"], 1, cfg["q"], cfg["c"], cfg["lr"], q_init=q0)
    sh = multirank.ShardedConEF(b.ConEF(cfg["tensors"], 1, cfg["q"], cfg["c"], cfg["lr"], q_init=q0), lowrank=True,
                                world_size=1, all_reduce=lambda t: None)
    total = wl.total_elems(cfg["tensors"])
    x0, x1 = torch.zeros(total, device="cuda"), torch.zeros(total, device="cuda")
    for t in range(2):
        g = wl.gradient(cfg, 0, t, device="cuda")
        out = plain.full_step(t, [g])
        plain.apply_update(x0, out)
        got = sh.step(t, g, x1)
        for k, v in out.items():
            assert torch.equal(got[k], v)
        assert torch.equal(x0, x1)


def test_sharded_wrapper_over_a_one_rank_nccl_group():
    """The default collective (torch.distributed, NCCL) on the library's message buffers."""
    import os
    import socket
    import torch.distributed as dist
    from paper_2312_08538_b200 import binding as b
    from paper_2312_08538_b200 import multirank
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("nccl", rank=0, world_size=1, device_id=torch.device("cuda", 0))
    try:
        cfg = wl.config("tiny")
        cfg["n_workers"] = 1
        plain = b.ConEF(cfg["tensors"], 1, cfg["q"], cfg["c"], cfg["lr"])
        sh = multirank.ShardedConEF(b.ConEF(cfg["tensors"], 1, cfg["q"], cfg["c"], cfg["lr"]), lowrank=False)
        assert sh.world == 1
        for t in range(3):
            g = wl.gradient(cfg, 0, t, device="cuda")
            out = plain.full_step(t, [g])
            got = sh.step(t, g)
            for k, v in out.items():
                assert torch.equal(got[k], v)
    finally:
        dist.destroy_process_group()
