"""Random-block-k (Sec. 5.3) and error reset (Sec. 4.2.2) on the GPU against the oracle."""
import numpy as np
import pytest
import torch

from paper_2312_08538_b200 import workloads as wl
from tests import parity_util as pu
from tests.test_gpu_parity import run_single_phase

pytestmark = pytest.mark.gpu

RAGGED = [(37, 53, 1), (19, 1, 0), (1, 7, 1), (64, 129, 1), (300, 1, 0), (5, 1000, 1), (200, 96, 1)]


@pytest.mark.parametrize("c", [dict(kind="int8", block=64, scale_dtype="fp16"), dict(kind="int4", block=128),
                               dict(kind="identity"), dict(kind="rowsketch", cs_rows=1, cs_col_div=5, seed=3, beta=0.9),
                               dict(kind="rowsketch", cs_rows=3, cs_col_div=4, seed=3),
                               dict(kind="stochquant", block=64, levels=16, seed=8)])
def test_randblock_bit_exact(c):
    cfg = wl.config("tiny")
    cfg["tensors"] = RAGGED
    cfg["n_workers"] = 3
    cfg["q"] = dict(kind="randblock", k_num=1, k_den=10, seed=31337)
    cfg["c"] = c
    eng, o = run_single_phase(cfg, 5, exact_values=True)
    # the model update reads the same index buffer
    from paper_2312_08538_b200 import binding as b
    total = wl.total_elems(cfg["tensors"])
    xh = np.zeros(total, np.float32)
    xd = torch.zeros(total, device="cuda")
    gd, gh = pu.grads_both(cfg, 5)
    res = o.step(5, gh)
    out = eng.full_step(5, gd)
    o.apply_update(xh, res)
    eng.apply_update(xd, out)
    assert np.array_equal(xd.cpu().numpy(), xh)


@pytest.mark.parametrize("c", [dict(kind="identity"), dict(kind="rowsketch", cs_rows=1, cs_col_div=5, seed=3, beta=0.9),
                               dict(kind="countsketch", cs_rows=3, cs_col_div=3, seed=4)])
def test_error_reset_matches_oracle(c):
    cfg = wl.config("tiny")
    cfg["tensors"] = RAGGED
    cfg["n_workers"] = 4
    cfg["q"] = dict(kind="randk", k_num=1, k_den=20, seed=5)
    cfg["c"] = c
    exact = c["kind"] != "countsketch"      # the flat sketch is built by atomics: tolerance there
    eng, o = run_single_phase(cfg, 2, exact_values=exact)
    if not exact:
        pu.load_state_from_oracle(eng, o)
    eng.error_reset()
    o.error_reset()
    for i in range(o.N):
        for l in o.compressed:
            ga, _ = pu.gpu_state_arrays(eng, o, i, l)
            oa, _ = pu.oracle_state_arrays(o, i, l)
            assert np.array_equal(ga, oa)
    # and the next step still agrees
    gd, gh = pu.grads_both(cfg, 2)
    res = o.step(2, gh)
    eng.full_step(2, gd)
    assert np.array_equal(eng.indices(o.compressed[0]).cpu().numpy().view(np.uint32), res[o.compressed[0]].idx)


def test_error_reset_refused_for_a_quantiser():
    from paper_2312_08538_b200 import binding as b
    cfg = wl.config("tiny")
    eng = pu.make_gpu(cfg)
    with pytest.raises(b.ConEFError):
        eng.error_reset()
