"""Parity at the benchmark's full sizes, in the launch configuration bench.py
times.  The oracle cannot run 1.5 G parameters x 8 workers, so it recomputes a
sample of whole tensors (a low-rank factor needs its whole tensor) from the same
gradients, and the rest is covered by properties that hold at any size."""
import numpy as np
import pytest
import torch

from paper_2312_08538_b200 import workloads as wl
from tests import parity_util as pu

pytestmark = pytest.mark.gpu


def sample_layers(cfg, want):
    """Indices of the first tensor of each requested shape."""
    out = []
    for shape in want:
        for l, (r, c, k) in enumerate(cfg["tensors"]):
            if (r, c) == shape and k:
                out.append(l)
                break
    return out


@pytest.mark.parametrize("name,shapes", [("gpt2-small", [(768, 768), (1024, 768), (768, 3072)]),
                                         ("gpt2-xl", [(1024, 1600), (1600, 4800), (6400, 1600)])])
def test_full_size_step_matches_oracle_on_sampled_tensors(name, shapes):
    from paper_2312_08538_b200 import binding as b
    cfg = wl.config(name)
    N = cfg["n_workers"]
    q0 = wl.q_init(cfg, "cuda")
    eng = pu.make_gpu(cfg, q_init=q0)
    grads = [wl.gradient(cfg, i, 0, "cuda") for i in range(N)]
    out = eng.full_step(0, grads)
    assert eng.last_status() == 0
    offs = np.concatenate([[0], np.cumsum([r * c for r, c, _ in cfg["tensors"]])])
    layers = sample_layers(cfg, shapes)
    assert len(layers) == len(shapes)

    # ---- the oracle on the sampled tensors (same gradient bits, same warm start)
    sub = dict(cfg)
    sub["tensors"] = [cfg["tensors"][l] for l in layers]
    rank = cfg["q"]["rank"]
    qoff = {}
    acc = 0
    for l, (r, c, k) in enumerate(cfg["tensors"]):
        if k and c > 1:
            qoff[l] = acc
            acc += c * min(rank, r, c)
    q0_sub = torch.cat([q0[qoff[l]:qoff[l] + cfg["tensors"][l][1] * rank] for l in layers]).cpu().numpy()
    o = pu.make_oracle(sub, q_init=q0_sub)
    gh = [torch.cat([g[offs[l]:offs[l + 1]] for l in layers]).cpu().numpy() for g in grads]
    res = o.step(0, gh)
    bits = 4
    flips = total = 0
    for j, l in enumerate(layers):
        for i in (0, N - 1):
            f = eng.factors(l, i)
            assert pu.frob_err(f["p_i"].cpu().numpy(), res[j].P[i]) <= pu.FROB
            assert pu.frob_err(f["q_i"].cpu().numpy(), res[j].Qi[i]) <= pu.FROB
            a, s = eng.state(i, l)
            d = cfg["tensors"][l][0] * cfg["tensors"][l][1]
            gc = pu.unpack_codes(a.cpu().numpy(), d, bits)
            gs = s.view(torch.float16).cpu().numpy().astype(np.float32)
            oc, os_ = pu.oracle_state_arrays(o, i, j)
            # factors agree to ~1e-7, so a code can only flip where x*inv sits on a rounding boundary
            diff = np.abs(gc - oc)
            assert diff.max() <= 1
            flips += np.count_nonzero(diff)
            total += diff.size
            assert np.mean(gs != os_) <= 1e-3
        assert pu.frob_err(eng.factors(l, 0)["p_hat"].cpu().numpy(), res[j].Phat) <= pu.FROB
    assert flips / total <= 1e-5, f"{flips} of {total} codes differ"

    # ---- properties that hold at any size, on every tensor
    lr = cfg["lr"]
    e0 = eng.decompress_error(0)
    eoff = 0
    for l, (n, m, k) in enumerate(cfg["tensors"]):
        if not (k and m > 1):
            continue
        d = n * m
        f = eng.factors(l, 0)
        ph = f["p_hat"]
        r = f["rank"]
        gram = ph.double().T @ ph.double()
        assert torch.allclose(gram, torch.eye(r, dtype=torch.float64, device="cuda"), atol=1e-5), f"tensor {l}"
        if l in layers or l % 40 == 0:
            # Delta + r = p with r stored through C: |p - Delta - e_1| <= half a quantisation step
            M = (lr * grads[0][offs[l]:offs[l + 1]]).view(n, m)
            resid = M - ph @ f["q_i"].T
            _, s = eng.state(0, l)
            step = s.view(torch.float16).float().repeat_interleave(128)[:d].view(n, m)
            err = (resid - e0[eoff:eoff + d].view(n, m)).abs()
            assert bool((err <= 0.5 * step * 1.001 + 1e-12).all()), f"tensor {l}"
            # C is contractive on what it was given, Q on p
            assert float((err ** 2).sum()) < float((resid ** 2).sum())
            assert float((resid ** 2).sum()) <= float((M ** 2).sum()) * (1 + 1e-5)
        eoff += d
    assert eoff == eng.error_elems()
    assert eng.state_bytes_per_worker() < 0.14 * 4 * eng.error_elems()   # 80-90 % of the dense error saved


def test_resnet50_full_size_every_tensor_against_the_oracle():
    """The ResNet-50 list is small enough for the oracle to redo the whole first step."""
    from paper_2312_08538_b200 import binding as b
    cfg = wl.config("resnet50")
    N = cfg["n_workers"]
    q0 = wl.q_init(cfg, "cuda")
    eng = pu.make_gpu(cfg, q_init=q0)
    o = pu.make_oracle(cfg, q_init=q0.cpu().numpy())
    gd, gh = pu.grads_both(cfg, 0)
    res = o.step(0, gh)
    out = eng.full_step(0, gd)
    assert eng.last_status() == 0
    assert pu.frob_err(out[b.MSG_P].cpu().numpy(), o.reduced(res, "P")) <= pu.FROB
    assert pu.frob_err(out[b.MSG_Q].cpu().numpy(), o.reduced(res, "Q")) <= pu.FROB
    assert np.array_equal(out[b.MSG_DENSE1D].cpu().numpy(), o.reduced(res, "dense1d"))
    flips = total = 0
    for l in o.compressed:
        assert pu.frob_err(eng.factors(l, 0)["p_hat"].cpu().numpy(), res[l].Phat) <= pu.FROB, f"tensor {l}"
        for i in (0, N - 1):
            gc, gs = pu.gpu_state_arrays(eng, o, i, l)
            oc, os_ = pu.oracle_state_arrays(o, i, l)
            diff = np.abs(gc - oc)
            # factors agree to ~1e-7: a code flips only where x*inv sits on a rounding boundary, a
            # scale only where the block's largest residual differs in its last bits
            assert diff.max() <= 1, f"tensor {l} worker {i}"
            flips += np.count_nonzero(diff)
            total += diff.size
            assert np.mean(np.abs(gs - os_) > 1e-6 * np.abs(os_)) <= 1e-3
    assert flips / total <= 1e-4, f"{flips} of {total} codes differ"


@pytest.mark.parametrize("name", ["transformer-big", "transformer-big-flatsketch"])
def test_transformer_big_full_size_sampled_tensors(name):
    """Random-k with the count sketch at full size (run by run, and hashed over whole rows): index
    sets bit for bit, values and sketch buckets within the tolerance of sums whose order differs
    (atomic adds)."""
    from paper_2312_08538_b200 import binding as b
    cfg = wl.config(name)
    N = cfg["n_workers"]
    eng = pu.make_gpu(cfg)
    grads = [wl.gradient(cfg, i, 0, "cuda") for i in range(N)]
    eng.full_step(0, grads)
    grads1 = [wl.gradient(cfg, i, 1, "cuda") for i in range(N)]
    out = eng.full_step(1, grads1)               # the second step decodes a non-trivial sketch
    assert eng.last_status() == 0
    offs = np.concatenate([[0], np.cumsum([r * c for r, c, _ in cfg["tensors"]])])
    layers = sample_layers(cfg, [(1024, 1024), (1024, 4096)])
    voff, acc = {}, 0
    for l, (r, c, k) in enumerate(cfg["tensors"]):
        if k and c > 1:
            voff[l] = acc
            acc += max(1, r * c * cfg["q"]["k_num"] // cfg["q"]["k_den"])
    from oracle import conef_oracle as orc
    for l in layers:
        r, c, _ = cfg["tensors"][l]
        # the oracle's tensor index enters the hashes: run it on a list that keeps this tensor at index l
        sub = dict(cfg)
        sub["tensors"] = [(1, 1, 0)] * l + [cfg["tensors"][l]]
        o = pu.make_oracle(sub)
        for t, gsrc in ((0, grads), (1, grads1)):
            gh = [np.concatenate([np.zeros(l, np.float32), g[offs[l]:offs[l + 1]].cpu().numpy()]) for g in gsrc]
            res = o.step(t, gh)
        k = o.k_of(l)
        assert np.array_equal(eng.indices(l).cpu().numpy().view(np.uint32), res[l].idx)
        want = orc.sum_workers(res[l].msg)
        got = out[b.MSG_VALUES][voff[l]:voff[l] + k].cpu().numpy()
        assert pu.rel_err(got, want) <= pu.REL
        for i in (0, N - 1):
            ga, _ = pu.gpu_state_arrays(eng, o, i, l)
            assert pu.rel_err(ga, o.state[i][l]["S"]) <= pu.REL


def test_transformer_big_row_sketch_full_size_sampled_tensors():
    """Partial ConEF with the row sketch (the Sec. 5.4 setting) at full size: everything bit for bit
    on sampled tensors, two steps (the second decodes a non-trivial sketch)."""
    from paper_2312_08538_b200 import binding as b
    from oracle import conef_oracle as orc
    cfg = wl.config("transformer-big-rowsketch")
    N = cfg["n_workers"]
    eng = pu.make_gpu(cfg)
    steps = [[wl.gradient(cfg, i, t, "cuda") for i in range(N)] for t in range(2)]
    out = None
    for t in range(2):
        out = eng.full_step(t, steps[t])
    assert eng.last_status() == 0
    offs = np.concatenate([[0], np.cumsum([r * c for r, c, _ in cfg["tensors"]])])
    layers = sample_layers(cfg, [(1024, 1024), (4096, 1024)])
    voff, acc = {}, 0
    for l, (r, c, k) in enumerate(cfg["tensors"]):
        if k and c > 1:
            voff[l] = acc
            acc += max(1, r * c * cfg["q"]["k_num"] // cfg["q"]["k_den"])
    for l in layers:
        sub = dict(cfg)
        sub["tensors"] = [(1, 1, 0)] * l + [cfg["tensors"][l]]      # keeps the tensor's index, which enters the hashes
        o = pu.make_oracle(sub)
        for t in range(2):
            gh = [np.concatenate([np.zeros(l, np.float32), g[offs[l]:offs[l + 1]].cpu().numpy()]) for g in steps[t]]
            res = o.step(t, gh)
        k = o.k_of(l)
        assert np.array_equal(eng.indices(l).cpu().numpy().view(np.uint32), res[l].idx)
        assert np.array_equal(out[b.MSG_VALUES][voff[l]:voff[l] + k].cpu().numpy(), orc.sum_workers(res[l].msg))
        for i in (0, N - 1):
            ga, _ = pu.gpu_state_arrays(eng, o, i, l)
            assert np.array_equal(ga, o.state[i][l]["T"]), f"sketch of worker {i} tensor {l}"
