"""Parity of the row-sketch error state (Sec. 4.2.2, tensor trick) and of partial error feedback
(Alg. 4) with the CPU oracle, through the C ABI.  The row sketch is built by a deterministic
gather in the oracle's accumulation order, so everything here is compared bit for bit."""
import numpy as np
import pytest
import torch

from paper_2312_08538_b200 import workloads as wl
from tests import parity_util as pu
from tests.test_gpu_parity import lowrank_teacher_forced, run_single_phase

pytestmark = pytest.mark.gpu

RAGGED = [(37, 53, 1), (19, 1, 0), (1, 7, 1), (64, 129, 1), (300, 1, 0), (5, 1000, 1), (1, 1, 0),
          (200, 96, 1), (130, 320, 1)]


@pytest.mark.parametrize("v,div,beta", [(1, 10, 0.9), (1, 3, 0.0), (3, 4, 0.5), (5, 7, 0.9), (7, 2, 0.25)])
def test_randk_rowsketch_partial_bit_exact(v, div, beta):
    cfg = wl.config("tiny")
    cfg["tensors"] = RAGGED
    cfg["n_workers"] = 3
    cfg["q"] = dict(kind="randk", k_num=3, k_den=100, seed=515151)
    cfg["c"] = dict(kind="rowsketch", cs_rows=v, cs_col_div=div, seed=77, beta=beta)
    run_single_phase(cfg, 5, exact_values=True)


def test_identity_q_rowsketch_keeps_only_the_decayed_sketch():
    cfg = wl.config("tiny")
    cfg["tensors"] = [(33, 65, 1), (10, 1, 0), (90, 64, 1)]
    cfg["q"] = dict(kind="identity")
    cfg["c"] = dict(kind="rowsketch", cs_rows=1, cs_col_div=5, seed=1, beta=0.5)
    eng, o = run_single_phase(cfg, 3, exact_values=True)
    assert not eng.decompress_error(0).any()


@pytest.mark.parametrize("ckind,block,scale", [("identity", 256, "fp32"), ("int8", 64, "fp16"),
                                               ("int4", 128, "fp32"), ("int4", 64, "fp16")])
def test_partial_error_feedback_with_quantisers(ckind, block, scale):
    cfg = wl.config("tiny")
    cfg["tensors"] = RAGGED
    cfg["n_workers"] = 2
    cfg["q"] = dict(kind="randk", k_num=3, k_den=100, seed=1234)
    cfg["c"] = dict(kind=ckind, block=block, scale_dtype=scale, beta=0.9)
    run_single_phase(cfg, 5, exact_values=True)


def test_partial_error_feedback_with_flat_countsketch():
    cfg = wl.config("transformer-big-mini")
    cfg["tensors"] = [(40, 100, 1), (7, 1, 0), (3, 333, 1)]
    cfg["n_workers"] = 2
    cfg["c"] = dict(kind="countsketch", cs_rows=3, cs_col_div=3, seed=99, beta=0.5)
    run_single_phase(cfg, 3, exact_values=False)


@pytest.mark.parametrize("v,beta", [(1, 0.9), (3, 0.0)])
def test_lowrank_rowsketch_teacher_forced(v, beta):
    cfg = wl.config("resnet50-mini")
    cfg["tensors"] = [(40, 96, 1), (11, 1, 0), (3, 50, 1), (130, 7, 1), (256, 160, 1)]
    cfg["n_workers"] = 2
    cfg["c"] = dict(kind="rowsketch", cs_rows=v, cs_col_div=4, seed=5, beta=beta)
    lowrank_teacher_forced(cfg, 3, fast=True)


def test_lowrank_int4_partial_teacher_forced():
    cfg = wl.config("gpt2-xl-mini")
    cfg["c"] = dict(cfg["c"], beta=0.9)
    lowrank_teacher_forced(cfg, 2, fast=True)   # beta != 0 routes every tensor to the generic kernels


def test_rowsketch_with_gradients_that_are_only_4_byte_aligned():
    """Gradient pointers off a 16-byte boundary switch the kernel to its scalar loads; results
    must not change."""
    cfg = wl.config("tiny")
    cfg["tensors"] = [(200, 96, 1), (10, 1, 0), (130, 320, 1)]
    cfg["n_workers"] = 2
    cfg["q"] = dict(kind="randk", k_num=3, k_den=100, seed=9)
    cfg["c"] = dict(kind="rowsketch", cs_rows=1, cs_col_div=8, seed=7, beta=0.9)
    eng = pu.make_gpu(cfg)
    o = pu.make_oracle(cfg)
    from paper_2312_08538_b200 import binding as b
    for t in range(3):
        gd, gh = pu.grads_both(cfg, t)
        shifted = []
        for g in gd:
            buf = torch.empty(g.numel() + 1, dtype=torch.float32, device="cuda")
            buf[1:].copy_(g)
            shifted.append(buf[1:])
            assert shifted[-1].data_ptr() % 16 == 4
        res = o.step(t, gh)
        out = eng.full_step(t, shifted)
        assert np.array_equal(out[b.MSG_VALUES].cpu().numpy(), o.reduced(res, "values"))
        for i in range(o.N):
            for l in o.compressed:
                ga, _ = pu.gpu_state_arrays(eng, o, i, l)
                assert np.array_equal(ga, o.state[i][l]["T"])
    assert eng.last_status() == 0


@pytest.mark.parametrize("qkind,v,beta", [("randk", 1, 0.9), ("randblock", 3, 0.5), ("identity", 1, 0.0)])
def test_half_precision_sketch_bit_exact(qkind, v, beta):
    cfg = wl.config("tiny")
    cfg["tensors"] = RAGGED
    cfg["n_workers"] = 3
    cfg["q"] = dict(kind=qkind, k_num=3, k_den=100, seed=99)
    cfg["c"] = dict(kind="rowsketch", cs_rows=v, cs_col_div=6, seed=13, beta=beta, scale_dtype="fp16")
    eng, o = run_single_phase(cfg, 5, exact_values=True)
    cfg32 = dict(cfg, c=dict(cfg["c"], scale_dtype="fp32"))
    assert eng.state_bytes_per_worker() * 2 <= pu.make_gpu(cfg32).state_bytes_per_worker() + 256 * len(RAGGED)
    eng.error_reset()
    o.error_reset()
    for i in range(o.N):
        for l in o.compressed:
            ga, _ = pu.gpu_state_arrays(eng, o, i, l)
            assert np.array_equal(ga, o.state[i][l]["T16"])


def test_half_precision_sketch_lowrank_teacher_forced():
    cfg = wl.config("resnet50-mini")
    cfg["tensors"] = [(40, 96, 1), (11, 1, 0), (3, 50, 1), (130, 7, 1), (256, 160, 1)]
    cfg["n_workers"] = 2
    cfg["c"] = dict(kind="rowsketch", cs_rows=1, cs_col_div=4, seed=5, beta=0.9, scale_dtype="fp16")
    lowrank_teacher_forced(cfg, 3, fast=True)
