"""Checkpoint and resume: a fresh context loaded with state_dict() continues bit for bit."""
import pytest
import torch

from paper_2312_08538_b200 import workloads as wl
from tests import parity_util as pu

pytestmark = pytest.mark.gpu


def _cfgs():
    a = wl.config("gpt2-xl-mini")
    b = wl.config("transformer-big-rowsketch-mini")
    c = wl.config("tiny")
    c["tensors"] = [(64, 96, 1), (9, 1, 0), (33, 65, 1)]
    c["c"] = dict(kind="int4", block=64, scale_dtype="fp16", iconef=1)
    d = wl.config("transformer-big-mini")
    e = wl.config("tiny")
    e["tensors"] = [(64, 96, 1), (9, 1, 0), (3, 8192 + 65, 1)]
    e["c"] = dict(kind="int8", block=64, iconef=2)       # e~ as k values: the checkpoint carries its step
    return [a, b, c, d, e]


@pytest.mark.parametrize("k", range(5))
def test_resume_from_a_checkpoint_is_bit_identical(k):
    cfg = _cfgs()[k]
    lowrank = cfg["q"]["kind"] == "lowrank"
    q0 = wl.q_init(cfg, "cuda") if lowrank else None
    N = cfg["n_workers"]
    grads = [[wl.gradient(cfg, i, t, "cuda") for i in range(N)] for t in range(4)]
    ref = pu.make_gpu(cfg, q_init=q0)
    for t in range(2):
        ref.full_step(t, grads[t])
    sd = ref.state_dict()
    assert all(not v.is_cuda for v in sd.values())
    want = [ref.full_step(t, grads[t]) for t in (2, 3)]
    want_err = [ref.decompress_error(i).clone() for i in range(N)]

    again = pu.make_gpu(cfg, q_init=torch.zeros_like(q0) if lowrank else None)   # a different warm start: must be overwritten
    again.load_state_dict(sd)
    got = [again.full_step(t, grads[t]) for t in (2, 3)]
    exact = cfg["c"]["kind"] != "countsketch"      # the flat sketch is built by atomic adds
    for w, g in zip(want, got):
        for kind in w:
            if exact:
                assert torch.equal(w[kind], g[kind])
            else:
                assert pu.rel_err(g[kind].cpu().numpy(), w[kind].cpu().numpy()) <= pu.REL
    if exact:
        for i in range(N):
            assert torch.equal(again.decompress_error(i), want_err[i])
