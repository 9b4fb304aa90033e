"""Parity of the stochastic s-level quantiser (Eq. 6) as error compressor with the CPU oracle: both
sides draw the same counter-based variates, so stored levels and scales are compared bit for bit."""
import numpy as np
import pytest

from paper_2312_08538_b200 import workloads as wl
from tests import parity_util as pu
from tests.test_gpu_parity import lowrank_teacher_forced, run_single_phase

pytestmark = pytest.mark.gpu

RAGGED = [(37, 53, 1), (19, 1, 0), (1, 7, 1), (64, 129, 1), (300, 1, 0), (5, 1000, 1), (1, 1, 0), (200, 96, 1)]


@pytest.mark.parametrize("levels,block,beta", [(8, 32, 0.0), (16, 128, 0.0), (64, 256, 0.9), (256, 64, 0.0), (127, 128, 0.5)])
def test_randk_stochquant_bit_exact(levels, block, beta):
    cfg = wl.config("tiny")
    cfg["tensors"] = RAGGED
    cfg["n_workers"] = 3
    cfg["q"] = dict(kind="randk", k_num=3, k_den=100, seed=77)
    cfg["c"] = dict(kind="stochquant", block=block, levels=levels, seed=4242, beta=beta)
    run_single_phase(cfg, 5, exact_values=True)


def test_workers_draw_different_variates():
    cfg = wl.config("tiny")
    cfg["tensors"] = [(64, 256, 1)]
    cfg["n_workers"] = 2
    cfg["q"] = dict(kind="randk", k_num=1, k_den=100, seed=1)
    cfg["c"] = dict(kind="stochquant", block=128, levels=8, seed=5)
    eng = pu.make_gpu(cfg)
    g = wl.gradient(cfg, 0, 0, device="cuda")
    eng.full_step(0, [g, g])                      # same gradient on both workers
    o = pu.make_oracle(cfg)
    a0, _ = pu.gpu_state_arrays(eng, o, 0, 0)
    a1, _ = pu.gpu_state_arrays(eng, o, 1, 0)
    assert not np.array_equal(a0, a1)
    assert np.abs(a0 - a1).max() <= 1             # same residual: levels differ by the rounding direction only


@pytest.mark.parametrize("levels", [16, 256])
def test_lowrank_stochquant_teacher_forced(levels):
    cfg = wl.config("resnet50-mini")
    cfg["c"] = dict(kind="stochquant", block=128, levels=levels, seed=31)
    lowrank_teacher_forced(cfg, 3, fast=True)
