"""Pins for the oracle's model update (Alg. 2 lines 7-8)."""
import numpy as np

import oracle.conef_oracle as orc


def _run(q, c, tensors, N, steps, lr, seed, dyadic=True):
    o = orc.ConEFOracle(tensors, N, q, c, lr)
    total = sum(a * b for a, b, _ in tensors)
    rng = np.random.default_rng(seed)
    x0 = (rng.integers(-64, 64, size=total) / 4.0).astype(np.float32)
    x = x0.copy()
    gsum = np.zeros(total, np.float64)
    for t in range(steps):
        grads = [(rng.integers(-32, 32, size=total) / 8.0).astype(np.float32) for _ in range(N)]
        res = o.step(t, grads)
        o.apply_update(x, res)
        gsum += np.sum([g.astype(np.float64) for g in grads], axis=0)
    return o, x0, x, gsum


def test_virtual_iterate_of_error_feedback_follows_plain_sgd():
    """With an uncompressed error (Alg. 1) x_t - mean_i e_t^i = x_0 - eta * mean_i sum_t g^i:
    the perturbed iterate of the convergence proofs.  Dyadic data make it exact."""
    tensors = [(8, 16, 1), (5, 1, 0), (4, 32, 1)]
    N, lr = 2, 0.5
    q = orc.QCfg(kind="randk", k_num=1, k_den=4, seed=11)
    o, x0, x, gsum = _run(q, orc.CCfg(kind="identity"), tensors, N, 6, lr, 1)
    e_mean = np.zeros(x.size)
    for l in o.compressed:
        sl = slice(o.offsets[l], o.offsets[l + 1])
        e_mean[sl] = np.mean([o.decode(i, l).astype(np.float64) for i in range(N)], axis=0)
    assert np.array_equal(x.astype(np.float64) - e_mean, x0.astype(np.float64) - lr * gsum / N)


def test_identity_q_is_plain_sgd():
    tensors = [(8, 16, 1), (5, 1, 0)]
    o, x0, x, gsum = _run(orc.QCfg(kind="identity"), orc.CCfg(kind="int8", block=32), tensors, 4, 3, 0.25, 2)
    assert np.array_equal(x.astype(np.float64), x0.astype(np.float64) - 0.25 * gsum / 4)


def test_lowrank_update_is_phat_times_mean_q():
    n, m, r, N = 12, 10, 3, 2
    rng = np.random.default_rng(3)
    q0 = rng.standard_normal(m * r).astype(np.float32)
    o = orc.ConEFOracle([(n, m, 1)], N, orc.QCfg(kind="lowrank", rank=r, q_init=q0), orc.CCfg(kind="identity"), 0.1)
    grads = [rng.standard_normal(n * m).astype(np.float32) for _ in range(N)]
    res = o.step(0, grads)
    x = rng.standard_normal(n * m).astype(np.float32)
    x_before = x.copy()
    o.apply_update(x, res)
    ph = res[0].Phat.astype(np.float64)
    qm = (res[0].Qsum.astype(np.float64) / N)
    want = x_before.astype(np.float64) - (ph @ qm.T).reshape(-1)
    assert np.max(np.abs(x - want)) <= 4 * np.finfo(np.float32).eps * (np.abs(want).max() + 1)
    # and it equals the mean of the workers' own Delta_i = P_hat Q_i^T
    mean_delta = np.mean([ph @ Qi.astype(np.float64).T for Qi in res[0].Qi], axis=0).reshape(-1)
    assert np.allclose(x_before - x, mean_delta, atol=1e-6)


def test_sparse_update_moves_only_the_shared_coordinates():
    tensors = [(16, 16, 1)]
    q = orc.QCfg(kind="randk", k_num=1, k_den=8, seed=5)
    o = orc.ConEFOracle(tensors, 3, q, orc.CCfg(kind="identity"), 1.0)
    rng = np.random.default_rng(4)
    grads = [rng.integers(-8, 8, size=256).astype(np.float32) for _ in range(3)]
    res = o.step(0, grads)
    x = np.zeros(256, np.float32)
    o.apply_update(x, res)
    idx = res[0].idx
    moved = np.flatnonzero(x)
    assert set(moved) <= set(idx.tolist())
    want = -(np.float32(1.0) * (grads[0][idx] + grads[1][idx] + grads[2][idx])) / np.float32(3)
    assert np.array_equal(x[idx], want.astype(np.float32))
