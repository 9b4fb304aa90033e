"""The model update x <- x - Delta_t (Alg. 2 lines 7-8) on the GPU against the oracle."""
import numpy as np
import pytest
import torch

from paper_2312_08538_b200 import workloads as wl
from tests import parity_util as pu

pytestmark = pytest.mark.gpu

SHAPES = [(37, 53, 1), (19, 1, 0), (1, 7, 1), (64, 129, 1), (300, 1, 0), (5, 1000, 1), (200, 96, 1)]


@pytest.mark.parametrize("qkind", ["identity", "randk"])
def test_update_from_value_messages_is_bit_exact(qkind):
    from paper_2312_08538_b200 import binding as b
    cfg = wl.config("tiny")
    cfg["tensors"] = SHAPES
    cfg["n_workers"] = 3
    cfg["q"] = dict(kind=qkind, k_num=3, k_den=100, seed=5)
    cfg["c"] = dict(kind="int8", block=64, scale_dtype="fp32")
    eng, o = pu.make_gpu(cfg), pu.make_oracle(cfg)
    total = wl.total_elems(cfg["tensors"])
    xh = np.random.default_rng(0).standard_normal(total).astype(np.float32)
    xd = torch.from_numpy(xh).cuda()
    for t in range(3):
        gd, gh = pu.grads_both(cfg, t)
        res = o.step(t, gh)
        out = eng.full_step(t, gd)
        o.apply_update(xh, res)
        eng.apply_update(xd, out)
        assert np.array_equal(xd.cpu().numpy(), xh), f"step {t}"


def test_lowrank_update_with_injected_factors_is_bit_exact():
    from paper_2312_08538_b200 import binding as b
    cfg = wl.config("resnet50-mini")
    q0 = wl.q_init(cfg, "cuda")
    eng = pu.make_gpu(cfg, q_init=q0)
    o = pu.make_oracle(cfg, q_init=q0.cpu().numpy())
    total = wl.total_elems(cfg["tensors"])
    xh = np.random.default_rng(1).standard_normal(total).astype(np.float32)
    xd = torch.from_numpy(xh).cuda()
    for t in range(2):
        pu.load_state_from_oracle(eng, o)
        gd, gh = pu.grads_both(cfg, t)
        res = o.step(t, gh)
        eng.step(t, gd, 0)
        eng.reduce_messages(b.MSG_P)
        for l in o.compressed:
            eng.factors(l, 0)["p_hat"].copy_(torch.from_numpy(res[l].Phat).cuda())
        eng.step(t, gd, 2)
        for l in o.compressed:
            for i in range(o.N):
                eng.factors(l, i)["q_i"].copy_(torch.from_numpy(res[l].Qi[i]).cuda())
        eng.step(t, gd, 3)
        with pytest.raises(b.ConEFError):
            eng.apply_update(xd, {})          # the mean of Q does not exist before its reduction
        eng.reduce_messages(b.MSG_Q)
        s1 = eng.reduce_messages(b.MSG_DENSE1D)
        o.apply_update(xh, res)
        eng.apply_update(xd, {b.MSG_DENSE1D: s1})
        assert np.array_equal(xd.cpu().numpy(), xh), f"step {t}"


def test_free_running_lowrank_update_is_close():
    from paper_2312_08538_b200 import binding as b
    cfg = wl.config("gpt2-xl-mini")
    q0 = wl.q_init(cfg, "cuda")
    eng = pu.make_gpu(cfg, q_init=q0)
    o = pu.make_oracle(cfg, q_init=q0.cpu().numpy())
    total = wl.total_elems(cfg["tensors"])
    xh = np.zeros(total, np.float32)
    xd = torch.zeros(total, device="cuda")
    gd, gh = pu.grads_both(cfg, 0)
    res = o.step(0, gh)
    out = eng.full_step(0, gd)
    o.apply_update(xh, res)
    eng.apply_update(xd, out)
    assert pu.frob_err(xd.cpu().numpy(), xh) <= pu.FROB
