"""Seeded random configurations (shapes, compressors, options) through the C ABI against the oracle:
a net for interactions that the hand-picked cases do not reach."""
import os

import numpy as np
import pytest

from paper_2312_08538_b200 import workloads as wl
from tests.test_gpu_parity import lowrank_teacher_forced, run_single_phase

pytestmark = pytest.mark.gpu

# more cases on demand: CONEF_RANDOM_CASES=400 python -m pytest tests/test_gpu_random_configs.py
N_SINGLE = int(os.environ.get("CONEF_RANDOM_CASES", 24))
N_LOWRANK = max(1, N_SINGLE * 2 // 3)

COLS = [1, 3, 7, 32, 50, 64, 96, 129, 160, 256, 288, 320, 512, 576, 1000, 1024, 1600]


def _tensors(rng, lowrank):
    ts = []
    for _ in range(int(rng.integers(2, 7))):
        cols = int(rng.choice(COLS))
        rows = int(rng.integers(1, 400 if cols < 600 else 120))
        ts.append((rows, cols, int(cols > 1 and rng.random() < 0.9)))
    if lowrank and not any(c % 32 == 0 and k for _, c, k in ts):
        ts.append((int(rng.integers(40, 300)), int(rng.choice([64, 160, 320, 576, 1600])), 1))
    if not any(k and c > 1 for _, c, k in ts):
        ts.append((17, 33, 1))
    return ts


def _c(rng, allow_iconef, sparsifying_q=False):
    kind = str(rng.choice(["identity", "int8", "int4", "rowsketch", "stochquant"]))
    c = dict(kind=kind, seed=int(rng.integers(1, 1 << 30)))
    if kind in ("int8", "int4", "stochquant"):
        c["block"] = int(rng.choice([64, 128, 256] if kind == "int4" else [32, 64, 128, 256]))
    if kind in ("int8", "int4"):
        c["scale_dtype"] = str(rng.choice(["fp32", "fp16"]))
    if kind == "stochquant":
        c["levels"] = int(rng.choice([4, 16, 127, 300]))
    if kind == "rowsketch":
        c["cs_rows"] = int(rng.choice([1, 1, 3]))
        c["cs_col_div"] = int(rng.choice([2, 5, 10]))
        c["scale_dtype"] = str(rng.choice(["fp32", "fp16"]))
    if allow_iconef and kind in ("identity", "int8", "int4") and rng.random() < 0.4:
        c["iconef"] = 2 if sparsifying_q and rng.random() < 0.5 else 1
    elif rng.random() < 0.4:
        c["beta"] = float(rng.choice([0.25, 0.5, 0.9]))
    return c


@pytest.mark.parametrize("seed", range(N_SINGLE))
def test_random_single_phase_configuration(seed):
    rng = np.random.default_rng(1000 + seed)
    cfg = wl.config("tiny")
    cfg["tensors"] = _tensors(rng, False)
    cfg["n_workers"] = int(rng.integers(1, 6))
    qk = str(rng.choice(["randk", "randblock", "identity"]))
    cfg["q"] = dict(kind=qk, k_num=int(rng.choice([1, 3, 10])), k_den=100, seed=int(rng.integers(1, 1 << 30)))
    cfg["c"] = _c(rng, True, qk != "identity")
    cfg["lr"] = float(rng.choice([0.01, 0.1, 1.0]))
    run_single_phase(cfg, 3, exact_values=True)


@pytest.mark.parametrize("seed", range(max(1, N_SINGLE // 2)))
def test_random_count_sketch_configuration(seed):
    """The count sketch, hashed over whole rows or run by run: index sets bit for bit, values within
    the tolerance of sums whose order differs."""
    rng = np.random.default_rng(3000 + seed)
    cfg = wl.config("tiny")
    cfg["tensors"] = _tensors(rng, False) + [(int(rng.integers(3, 40)), 1000, 1)]
    cfg["n_workers"] = int(rng.integers(1, 5))
    qk = str(rng.choice(["randk", "randblock", "identity"]))
    cfg["q"] = dict(kind=qk, k_num=int(rng.choice([1, 3, 10])), k_den=100, seed=int(rng.integers(1, 1 << 30)))
    c = dict(kind="countsketch", cs_rows=int(rng.choice([1, 3, 5, 7])), cs_col_div=int(rng.choice([2, 5, 10])),
             seed=int(rng.integers(1, 1 << 30)), cs_chunk=int(rng.choice([0, 256, 1024, 2048, 8192])))
    if rng.random() < 0.3:
        c["beta"] = float(rng.choice([0.25, 0.5]))
    cfg["c"] = c
    cfg["lr"] = float(rng.choice([0.01, 0.1, 1.0]))
    eng, o = run_single_phase(cfg, 3, exact_values=False)


@pytest.mark.parametrize("seed", range(N_LOWRANK))
def test_random_lowrank_configuration(seed):
    rng = np.random.default_rng(2000 + seed)
    cfg = wl.config("resnet50-mini")
    cfg["tensors"] = _tensors(rng, True)
    cfg["n_workers"] = int(rng.integers(1, 5))
    cfg["q"] = dict(kind="lowrank", rank=int(rng.choice([1, 2, 4, 4, 8, 8])), seed=1)
    cfg["c"] = _c(rng, False)
    if rng.random() < 0.35:
        # the setting of the row-per-lane kernels (rank 4, int4 / 128 / fp16), on widths they take
        cfg["q"]["rank"] = 4
        cfg["c"] = dict(kind="int4", block=128, scale_dtype="fp16", seed=3)
        cfg["tensors"] += [(int(rng.integers(32, 300)), int(rng.choice([64, 128, 192, 320, 1600])), 1)]
    cfg["lr"] = float(rng.choice([0.05, 0.5]))
    lowrank_teacher_forced(cfg, 2, fast=bool(rng.random() < 0.8), scale_with_cond=True)
