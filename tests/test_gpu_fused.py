"""The fused low-rank passes 2 + 3 (one persistent kernel that takes tiles of Q_i = M_i^T P_hat
and of the residual from one task list; Sec. 5.2, Alg. 2 line 9) against the oracle.

Teacher-forced like the separate passes: both sides start a step from the oracle's state, the
oracle's P_hat and Q_i are injected, and the codes and scales the kernel stores must then be
bit-exact; the Q_i the kernel computes on its way is compared within the factor tolerance.
Tile lengths and CTAs per SM are varied so that small tensors reach every path of the kernel:
many tiles per segment, tiles shorter than the warps of a CTA, the ragged last period, the
scratch that cycles."""
import numpy as np
import pytest
import torch

from paper_2312_08538_b200 import workloads as wl
from tests import parity_util as pu

pytestmark = pytest.mark.gpu


def binding():
    from paper_2312_08538_b200 import binding as b
    return b


def fused_teacher_forced(cfg, steps, tile_periods, ctas_per_sm):
    b = binding()
    q0 = wl.q_init(cfg, "cuda")
    eng = pu.make_gpu(cfg, q_init=q0)
    eng.set_fused(True, tile_periods, ctas_per_sm)
    info = eng.fused_info()
    assert info["active"] == 1, info
    o = pu.make_oracle(cfg, q_init=q0.cpu().numpy())
    worst_q, n_fused = 0.0, 0
    for t in range(steps):
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
        eng.step(t, gd, 4)   # pass 3 by the fused kernel, residual from the injected Q_i
        assert eng.last_status() == 0
        for l in o.compressed:
            for i in range(o.N):
                try:
                    fq = eng.fused_q(l, i)
                except b.ConEFError:
                    continue   # a tensor the fused kernel does not take
                n_fused += 1
                worst_q = max(worst_q, pu.frob_err(fq.cpu().numpy(), res[l].Qi[i]))
        eng.reduce_messages(b.MSG_Q)
        for i in range(o.N):
            for l in o.compressed:
                ga, gs = pu.gpu_state_arrays(eng, o, i, l)
                oa, os_ = pu.oracle_state_arrays(o, i, l)
                frac, mx = pu.compare_codes(ga, gs, oa, os_)
                assert frac == 0 and mx == 0, f"step {t} worker {i} tensor {l}: codes differ ({frac}, {mx})"
    assert n_fused > 0
    assert worst_q <= pu.FROB, f"Q_i of the fused kernel: relative Frobenius error {worst_q}"


@pytest.mark.parametrize("name", ["resnet50-mini", "gpt2-small-mini", "gpt2-xl-mini"])
@pytest.mark.parametrize("tile_periods,ctas_per_sm", [(0, 0), (3, 2), (8, 4), (1000, 3)])
def test_fused_teacher_forced(name, tile_periods, ctas_per_sm):
    cfg = wl.config(name)
    fused_teacher_forced(cfg, 3, tile_periods, ctas_per_sm)


@pytest.mark.parametrize("rank,c", [(4, dict(kind="int4", block=128, scale_dtype="fp16")),
                                    (8, dict(kind="int4", block=128, scale_dtype="fp32")),
                                    (8, dict(kind="int8", block=256, scale_dtype="fp16")),
                                    (4, dict(kind="int8", block=256, scale_dtype="fp32"))])
@pytest.mark.parametrize("tile_periods,ctas_per_sm", [(0, 0), (16, 2)])
def test_fused_large_tensor(rank, c, tile_periods, ctas_per_sm):
    # more tiles than resident CTAs, with a ragged last period (rows not a multiple of the period's rows)
    cfg = wl.config("gpt2-xl-mini")
    cfg["tensors"] = [(4099, 1600, 1), (1600, 1, 0), (515, 4800, 1)]
    cfg["n_workers"] = 2
    cfg["q"] = dict(cfg["q"], rank=rank)
    cfg["c"] = c
    fused_teacher_forced(cfg, 2, tile_periods, ctas_per_sm)


def test_fused_free_running_step_matches_oracle_factors():
    # phase 1 as a user calls it: Q_i, the warm start and the stored error of a whole step
    b = binding()
    cfg = wl.config("gpt2-xl-mini")
    q0 = wl.q_init(cfg, "cuda")
    eng, o = pu.make_gpu(cfg, q_init=q0), pu.make_oracle(cfg, q_init=q0.cpu().numpy())
    eng.set_fused(True)
    assert eng.fused_info()["active"] == 1
    gd, gh = pu.grads_both(cfg, 0)
    res = o.step(0, gh)
    out = eng.full_step(0, gd)
    assert eng.last_status() == 0
    assert pu.frob_err(out[b.MSG_Q].cpu().numpy(), o.reduced(res, "Q")) <= pu.FROB
    for i in range(o.N):
        assert pu.frob_err(eng.decompress_error(i).cpu().numpy(), o.decompress_error(i)) <= 1e-2


def test_fused_off_runs_the_separate_kernels():
    cfg = wl.config("gpt2-xl-mini")
    q0 = wl.q_init(cfg, "cuda")
    eng = pu.make_gpu(cfg, q_init=q0)
    eng.set_fused(False)
    assert eng.fused_info()["active"] == 0
    a = pu.make_gpu(cfg, q_init=q0)
    a.set_fused(True)
    gd, _ = pu.grads_both(cfg, 0)
    ra, rb = a.full_step(0, gd), eng.full_step(0, gd)
    # the factors agree to rounding (different summation orders), the messages to the factor tolerance
    b = binding()
    assert pu.frob_err(ra[b.MSG_Q].cpu().numpy(), rb[b.MSG_Q].cpu().numpy()) <= pu.FROB
