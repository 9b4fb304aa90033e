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


def second_step_teacher_forced(name, shapes, workers=None):
    """Two steps at full size.  Step 0 runs free on both sides; then the sampled tensors' stored
    error (non-zero codes, binary16 scales) and warm start are loaded from the oracle, and step 1 is
    compared stage by stage: P_i, P_hat and Q_i within the factor tolerance, then, with the oracle's
    P_hat and Q_i injected, the stored codes and scales bit for bit -- in the launch configuration
    the benchmark times (every tensor of the model in the grids, tile lengths of the large
    models).  shapes = None takes every compressed tensor.  workers: the workers the oracle redoes
    (default all).  With a subset the oracle is a job of just those workers: P_i, Q_i and the stored
    error of a worker depend on its own gradient and state and on the shared P_hat and warm start,
    which the GPU takes from the oracle, so those workers are compared exactly as before and only
    the comparison of the GPU's own P_hat (a sum over all its workers) falls away."""
    from paper_2312_08538_b200 import binding as b
    cfg = wl.config(name)
    N = cfg["n_workers"]
    q0 = wl.q_init(cfg, "cuda")
    eng = pu.make_gpu(cfg, q_init=q0)
    offs = np.concatenate([[0], np.cumsum([r * c for r, c, _ in cfg["tensors"]])])
    if shapes is None:
        layers = [l for l, (r, c, k) in enumerate(cfg["tensors"]) if k and c > 1]
    else:
        layers = sample_layers(cfg, shapes)
        assert len(layers) == len(shapes)
    W = list(range(N)) if workers is None else list(workers)
    sub = dict(cfg)
    sub["tensors"] = [cfg["tensors"][l] for l in layers]
    sub["n_workers"] = len(W)
    rank = cfg["q"]["rank"]
    qoff, acc = {}, 0
    for l, (r, c, k) in enumerate(cfg["tensors"]):
        if k and c > 1:
            qoff[l] = acc
            acc += c * min(rank, r, c)
    q0_sub = torch.cat([q0[qoff[l]:qoff[l] + cfg["tensors"][l][1] * min(rank, *cfg["tensors"][l][:2])]
                        for l in layers]).cpu().numpy()
    o = pu.make_oracle(sub, q_init=q0_sub)
    bits = 8 if cfg["c"]["kind"] == "int8" else 4
    half = cfg["c"].get("scale_dtype", "fp32") == "fp16"

    def both(t):
        dev = [wl.gradient(cfg, i, t, "cuda") for i in range(N)]
        host = [torch.cat([dev[i][offs[l]:offs[l + 1]] for l in layers]).cpu().numpy() for i in W]
        return dev, host

    gd, gh = both(0)
    o.step(0, gh)
    eng.full_step(0, gd)
    del gd
    # every sampled tensor's stored error is now non-trivial; the GPU continues from the oracle's
    for j, l in enumerate(layers):
        for wi, i in enumerate(W):
            a, sc = eng.state(i, l)
            st = o.state[wi][j]
            assert np.any(st["codes"]), "the error of step 0 should not be empty"
            a.copy_(torch.from_numpy(st["codes"]).cuda())
            if half:
                sc.view(torch.int16).copy_(torch.from_numpy(st["scales16"].view(np.int16)).cuda())
            else:
                sc.view(torch.float32).copy_(torch.from_numpy(st["scales"]).cuda())
        eng.factors(l, 0)["q_prev"].copy_(torch.from_numpy(o.Qprev[j]).cuda())
    gd, gh = both(1)
    res = o.step(1, gh)
    eng.step(1, gd, 0)
    worst = dict(P=0.0, Phat=0.0, Q=0.0)
    for j, l in enumerate(layers):
        for wi, i in enumerate(W):
            worst["P"] = max(worst["P"], pu.frob_err(eng.factors(l, i)["p_i"].cpu().numpy(), res[j].P[wi]))
    eng.reduce_messages(b.MSG_P)
    for j, l in enumerate(layers):
        f = eng.factors(l, 0)
        if len(W) == N:
            worst["Phat"] = max(worst["Phat"], pu.frob_err(f["p_hat"].cpu().numpy(), res[j].Phat))
        f["p_hat"].copy_(torch.from_numpy(res[j].Phat).cuda())
    eng.step(1, gd, 2)
    for j, l in enumerate(layers):
        for wi, i in enumerate(W):
            f = eng.factors(l, i)
            worst["Q"] = max(worst["Q"], pu.frob_err(f["q_i"].cpu().numpy(), res[j].Qi[wi]))
            f["q_i"].copy_(torch.from_numpy(res[j].Qi[wi]).cuda())
    eng.step(1, gd, 3)
    eng.reduce_messages(b.MSG_Q)
    assert eng.last_status() == 0
    for k_, v in worst.items():
        assert v <= pu.FROB, f"factor {k_}: relative Frobenius error {v}"
    for j, l in enumerate(layers):
        d = cfg["tensors"][l][0] * cfg["tensors"][l][1]
        for wi, i in enumerate(W):
            a, sc = eng.state(i, l)
            gc = pu.unpack_codes(a.cpu().numpy(), d, bits)
            gs = sc.view(torch.float16).cpu().numpy().astype(np.float32) if half else sc.view(torch.float32).cpu().numpy()
            oc, os_ = pu.oracle_state_arrays(o, wi, j)
            assert np.array_equal(gs, os_), f"tensor {l} worker {i}: block scales differ"
            assert np.array_equal(gc, oc), f"tensor {l} worker {i}: {np.count_nonzero(gc != oc)} codes differ"
    return worst


@pytest.mark.parametrize("name,shapes", [
    # the embedding (odd row count, a short last quantisation block at 768 columns), one tensor of every other shape
    ("gpt2-small", [(50257, 768), (1024, 768), (768, 768), (768, 2304), (768, 3072), (3072, 768)]),
    ("gpt2-xl", [(50257, 1600), (1024, 1600), (1600, 1600), (1600, 4800), (1600, 6400), (6400, 1600)]),
])
def test_full_size_second_step_teacher_forced_bit_exact(name, shapes):
    # the oracle redoes the first and the last worker (it takes seconds per 10^8 element-steps)
    cfg = wl.config(name)
    second_step_teacher_forced(name, shapes, workers=[0, cfg["n_workers"] - 1])


def test_resnet50_full_size_second_step_every_tensor_bit_exact():
    second_step_teacher_forced("resnet50", None)


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


@pytest.mark.parametrize("name", ["transformer-big", "transformer-big-chunksketch"])
def test_transformer_big_full_size_sampled_tensors(name):
    """Random-k with the count sketch at full size (hashed over whole rows: configuration 4; and the
    run-by-run variant): index
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
