"""iConEF (Alg. 3, versions 1 and 2) on the GPU against the oracle: both stored states, messages
and the decoded error, bit for bit."""
import numpy as np
import pytest
import torch

from paper_2312_08538_b200 import workloads as wl
from tests import parity_util as pu
from tests.test_gpu_parity import run_single_phase

pytestmark = pytest.mark.gpu

RAGGED = [(37, 53, 1), (19, 1, 0), (1, 7, 1), (64, 129, 1), (300, 1, 0), (5, 1000, 1), (200, 96, 1)]


@pytest.mark.parametrize("qkind", ["randk", "randblock"])
@pytest.mark.parametrize("c", [dict(kind="int8", block=64, scale_dtype="fp16"), dict(kind="int8", block=256),
                               dict(kind="int4", block=128, scale_dtype="fp16"), dict(kind="int4", block=64),
                               dict(kind="identity")])
def test_iconef_v1_bit_exact(qkind, c):
    cfg = wl.config("tiny")
    cfg["tensors"] = RAGGED
    cfg["n_workers"] = 3
    cfg["q"] = dict(kind=qkind, k_num=1, k_den=20, seed=2718)
    cfg["c"] = dict(c, iconef=1)
    eng, o = run_single_phase(cfg, 5, exact_values=True)   # messages, first state, decoded error e~ + q
    for i in range(o.N):
        for l in o.compressed:
            ga, gs = pu.gpu_state_arrays(eng, o, i, l, second=True)
            oa, os_ = pu.oracle_state_arrays(o, i, l, second=True)
            assert np.array_equal(ga, oa), f"second state of worker {i} tensor {l}"
            if gs is not None:
                assert np.array_equal(gs, os_)
    assert eng.state_bytes_per_worker() == 2 * pu.make_gpu(dict(cfg, c=c)).state_bytes_per_worker()


@pytest.mark.parametrize("qkind", ["randk", "randblock", "identity"])
@pytest.mark.parametrize("c", [dict(kind="int8", block=64, scale_dtype="fp16"), dict(kind="int8", block=256),
                               dict(kind="int4", block=128, scale_dtype="fp16"), dict(kind="int4", block=64)])
@pytest.mark.parametrize("fast", [True, False])
def test_iconef_v1_on_the_tuned_fused_step(qkind, c, fast):
    """Shapes the tuned fused step takes (whole 8-element groups, aligned offsets), several selection
    tiles and a ragged last chunk: both states, messages and the decoded error bit for bit, and the
    same with the generic kernel."""
    cfg = wl.config("tiny")
    cfg["tensors"] = [(64, 256, 1), (8, 1, 0), (130, 512, 1), (3, 8192 * 2 + 72, 1), (40, 1000, 1)]
    cfg["n_workers"] = 3
    cfg["q"] = dict(kind=qkind, k_num=1, k_den=20, seed=2718)
    cfg["c"] = dict(c, iconef=1)
    eng, o = run_single_phase(cfg, 4, exact_values=True, fast=fast)
    for i in range(o.N):
        for l in o.compressed:
            ga, gs = pu.gpu_state_arrays(eng, o, i, l, second=True)
            oa, os_ = pu.oracle_state_arrays(o, i, l, second=True)
            assert np.array_equal(ga, oa), f"second state of worker {i} tensor {l}"
            assert np.array_equal(gs, os_)


@pytest.mark.parametrize("qkind", ["randk", "randblock"])
@pytest.mark.parametrize("c", [dict(kind="int8", block=64, scale_dtype="fp16"), dict(kind="int8", block=256),
                               dict(kind="int4", block=128, scale_dtype="fp16"), dict(kind="int4", block=64)])
@pytest.mark.parametrize("fast", [True, False])
def test_iconef_v2_on_the_tuned_fused_step(qkind, c, fast):
    """Version 2 on shapes the tuned fused step takes: index sets, messages, the state q, the decoded
    error e~ + q and the kept values e~ bit for bit, with the tuned and with the generic kernel."""
    cfg = wl.config("tiny")
    cfg["tensors"] = [(64, 256, 1), (8, 1, 0), (130, 512, 1), (3, 8192 * 2 + 72, 1), (40, 1000, 1)]
    cfg["n_workers"] = 3
    cfg["q"] = dict(kind=qkind, k_num=1, k_den=20, seed=2718)
    cfg["c"] = dict(c, iconef=2)
    eng, o = run_single_phase(cfg, 5, exact_values=True, fast=fast)
    assert eng.error_step() == 4
    for i in range(o.N):
        for l in o.compressed:
            ev, none = eng.state(i, l, second=True)
            assert np.array_equal(ev.view(torch.float32).cpu().numpy(), o.ev[i][l][1]), f"e~ of worker {i} tensor {l}"


@pytest.mark.parametrize("qkind", ["randk", "randblock"])
@pytest.mark.parametrize("c", [dict(kind="int8", block=64, scale_dtype="fp16"), dict(kind="int8", block=256),
                               dict(kind="int4", block=128, scale_dtype="fp16"), dict(kind="int4", block=32 * 2),
                               dict(kind="identity")])
def test_iconef_v2_bit_exact(qkind, c):
    """Version 2: e~ = Q(r) as the k values of the step's second draw, q = C(r - e~) as the state."""
    cfg = wl.config("tiny")
    cfg["tensors"] = RAGGED + [(3, 8192 * 2 + 77, 1)]      # the last one spans several selection tiles
    cfg["n_workers"] = 3
    cfg["q"] = dict(kind=qkind, k_num=1, k_den=20, seed=2718)
    cfg["c"] = dict(c, iconef=2)
    eng, o = run_single_phase(cfg, 5, exact_values=True)   # index sets, messages, state q, decoded error e~ + q
    assert eng.error_step() == 4
    for i in range(o.N):
        for l in o.compressed:
            ev, none = eng.state(i, l, second=True)
            assert none is None
            assert np.array_equal(ev.view(torch.float32).cpu().numpy(), o.ev[i][l][1]), f"e~ of worker {i} tensor {l}"
    k_total = sum(o.k_of(l) for l in o.compressed)
    assert eng.state_bytes_per_worker() == pu.make_gpu(dict(cfg, c=c)).state_bytes_per_worker() + 4 * k_total


def test_iconef_v2_needs_a_sparsifying_q():
    from paper_2312_08538_b200 import binding as b
    cfg = wl.config("tiny")
    cfg["c"] = dict(kind="int8", block=64, iconef=2)
    for q in (dict(kind="identity"), dict(kind="lowrank", rank=2, seed=1)):
        cfg["q"] = q
        with pytest.raises(b.ConEFError) as e:
            b.conef_workspace_bytes(cfg["tensors"], cfg["n_workers"], cfg["q"], cfg["c"])
        assert e.value.code == b.ERR_UNSUPPORTED


def test_iconef_v2_refuses_error_reset():
    from paper_2312_08538_b200 import binding as b
    cfg = wl.config("tiny")
    cfg["c"] = dict(kind="identity", iconef=2)      # linear C, but e~ is kept outside the averaged state
    eng = pu.make_gpu(cfg)
    with pytest.raises(b.ConEFError) as e:
        eng.error_reset()
    assert e.value.code == b.ERR_UNSUPPORTED


def test_iconef_lowrank_generic_path_close_to_oracle():
    from paper_2312_08538_b200 import binding as b
    cfg = wl.config("resnet50-mini")
    cfg["c"] = dict(cfg["c"], iconef=1)
    q0 = wl.q_init(cfg, "cuda")
    eng = pu.make_gpu(cfg, q_init=q0)
    o = pu.make_oracle(cfg, q_init=q0.cpu().numpy())
    for t in range(2):
        gd, gh = pu.grads_both(cfg, t)
        res = o.step(t, gh)
        out = eng.full_step(t, gd)
        assert pu.frob_err(out[b.MSG_P].cpu().numpy(), o.reduced(res, "P")) <= pu.FROB
        assert pu.frob_err(out[b.MSG_Q].cpu().numpy(), o.reduced(res, "Q")) <= pu.FROB
    for i in range(o.N):
        assert pu.frob_err(eng.decompress_error(i).cpu().numpy(), o.decompress_error(i)) <= 1e-2


def test_iconef_refused_for_sketches_and_partial():
    from paper_2312_08538_b200 import binding as b
    cfg = wl.config("tiny")
    for c in (dict(kind="countsketch", cs_rows=3, cs_col_div=4, iconef=1), dict(kind="int8", block=64, beta=0.5, iconef=1)):
        cfg["c"] = c
        with pytest.raises(b.ConEFError):
            pu.make_gpu(cfg)
