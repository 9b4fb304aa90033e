"""Count sketch applied run by run (cs_chunk > 0) through the C ABI against the oracle: the
shared-memory step and the generic kernels, every single-phase Q, several sketch heights, partial
error feedback, runs with a remainder, tensors of a single run, and windows too wide for shared
memory.  Indices are bit-exact; bucket sums add terms of random sign in a different order, so
values carry the relative tolerance of the other sketch tests."""
import numpy as np
import pytest

from paper_2312_08538_b200 import workloads as wl
from tests import parity_util as pu

pytestmark = pytest.mark.gpu

TENSORS = [(40, 256, 1),      # 10 240 elements: 5 runs of 2048
           (7, 1, 0),
           (33, 333, 1),      # 10 989: the last run takes a remainder that is not a multiple of 32
           (3, 100, 1),       # one run
           (1, 2048, 1),      # exactly one run
           (1, 4095, 1)]      # one run of almost two chunk lengths


def run(cfg, steps, fast):
    from paper_2312_08538_b200 import binding as b
    eng, o = pu.make_gpu(cfg, fast=fast), pu.make_oracle(cfg)
    for t in range(steps):
        gd, gh = pu.grads_both(cfg, t)
        res = o.step(t, gh)
        out = eng.full_step(t, gd)
        assert eng.last_status() == 0
        if cfg["q"]["kind"] in ("randk", "randblock"):
            for l in o.compressed:
                assert np.array_equal(eng.indices(l).cpu().numpy().view(np.uint32), res[l].idx)
        assert pu.rel_err(out[b.MSG_VALUES].cpu().numpy(), o.reduced(res, "values")) <= pu.REL
        for i in range(o.N):
            mine = np.concatenate([res[l].msg[i] for l in o.compressed])
            assert pu.rel_err(eng.message(b.MSG_VALUES, i).cpu().numpy(), mine) <= pu.REL
            for l in o.compressed:
                ga, _ = pu.gpu_state_arrays(eng, o, i, l)
                oa, _ = pu.oracle_state_arrays(o, i, l)
                assert pu.rel_err(ga, oa) <= pu.REL, f"step {t} worker {i} tensor {l}: sketch differs"
    for i in range(o.N):
        assert pu.rel_err(eng.decompress_error(i).cpu().numpy(), o.decompress_error(i)) <= pu.REL
    return eng, o


def base_cfg(q, c, n_workers=2):
    cfg = wl.config("transformer-big-mini")
    cfg["tensors"] = list(TENSORS)
    cfg["n_workers"] = n_workers
    cfg["q"] = q
    cfg["c"] = c
    return cfg


@pytest.mark.parametrize("fast", [True, False])
@pytest.mark.parametrize("q", [dict(kind="randk", k_num=1, k_den=50, seed=5), dict(kind="identity"),
                               dict(kind="randblock", k_num=1, k_den=20, seed=6)])
@pytest.mark.parametrize("v", [1, 3, 5, 7])
def test_chunked_sketch_matches_the_oracle(q, v, fast):
    c = dict(kind="countsketch", cs_rows=v, cs_col_div=5, seed=31, cs_chunk=2048)
    run(base_cfg(q, c), 3, fast)


@pytest.mark.parametrize("fast", [True, False])
def test_chunked_sketch_with_partial_error_feedback(fast):
    c = dict(kind="countsketch", cs_rows=3, cs_col_div=4, seed=2, cs_chunk=1024, beta=0.5)
    run(base_cfg(dict(kind="randk", k_num=1, k_den=10, seed=1), c, n_workers=3), 4, fast)


def test_chunked_sketch_with_the_low_rank_q():
    # two-phase Q: the generic kernels decode and build the chunked sketch
    cfg = base_cfg(dict(kind="lowrank", rank=2, seed=4), dict(kind="countsketch", cs_rows=3, cs_col_div=4, seed=2, cs_chunk=1024))
    q0 = wl.q_init(cfg, "cuda")
    eng = pu.make_gpu(cfg, q_init=q0)
    o = pu.make_oracle(cfg, q_init=q0.cpu().numpy())
    for t in range(2):
        gd, gh = pu.grads_both(cfg, t)
        o.step(t, gh)
        eng.full_step(t, gd)
        assert eng.last_status() == 0
    for i in range(o.N):
        ge, oe = eng.decompress_error(i).cpu().numpy(), o.decompress_error(i)
        assert pu.frob_err(ge, oe) <= 1e-4


def test_windows_too_wide_for_shared_memory_take_the_generic_kernel():
    # one sketch bucket per element and 7 rows: 2 x 7 x 32 768 floats per run do not fit
    cfg = base_cfg(dict(kind="randk", k_num=1, k_den=100, seed=5),
                   dict(kind="countsketch", cs_rows=7, cs_col_div=1, seed=3, cs_chunk=32768))
    cfg["tensors"] = [(3, 32768, 1), (64, 256, 1)]
    run(cfg, 2, True)


def test_full_size_tensor_sampled_against_the_oracle():
    """One 1024 x 4096 tensor at the benchmark's run length: the oracle finishes it in seconds."""
    cfg = wl.config("transformer-big-chunksketch")
    cfg["tensors"] = [(1024, 4096, 1)]
    cfg["n_workers"] = 2
    run(cfg, 2, True)
