"""Whole-run pins of the oracle driver: Algorithm 2 against Algorithm 1, the
error-feedback conservation law, the bookkeeping identity of the convergence
proof, and the degenerate compressors.  CPU only."""
import numpy as np
import pytest

from oracle import conef_oracle as orc


def rng(seed):
    return np.random.default_rng(seed)


def fma32(a, b, c):
    """round-to-fp32 of a*b + c: the product of two fp32 is exact in fp64."""
    return (np.float64(a) * b.astype(np.float64) + c.astype(np.float64)).astype(np.float32)


TENSORS = [(24, 40, 1), (17, 1, 0), (9, 33, 1)]
OFF = np.cumsum([0] + [a * b for a, b, _ in TENSORS])


def grads(N, t, seed=0):
    return [(rng(1000 * seed + 10 * t + i).standard_normal(OFF[-1]) * 0.01).astype(np.float32)
            for i in range(N)]


def efsgd_reference(q, N, lr, steps):
    """Algorithm 1 written independently in numpy: dense fp32 error vector."""
    e = [[np.zeros(a * b, np.float32) for a, b, _ in TENSORS] for _ in range(N)]
    deltas = []
    for t in range(steps):
        g = grads(N, t)
        step_delta = []
        for i in range(N):
            row = []
            for l, (a, b, cmp) in enumerate(TENSORS):
                gl = g[i][OFF[l]:OFF[l + 1]]
                if not (cmp and b > 1):
                    row.append(np.float32(lr) * gl)
                    continue
                p = fma32(np.float32(lr), gl, e[i][l])                    # line 5
                idx = orc.randk_indices(q.seed, l, t, a * b, max(1, a * b * q.k_num // q.k_den))
                delta = np.zeros_like(p)
                delta[idx] = p[idx]                                        # line 6
                e[i][l] = p - delta                                        # line 9
                row.append(delta)
            step_delta.append(row)
        deltas.append(step_delta)
    return e, deltas


def test_identity_C_reduces_to_efsgd_bitwise():
    N, lr, steps = 3, 0.1, 6
    q = orc.QCfg(kind="randk", k_num=1, k_den=10, seed=77)
    o = orc.ConEFOracle(TENSORS, N, q, orc.CCfg(kind="identity"), lr)
    e_ref, d_ref = efsgd_reference(q, N, lr, steps)
    for t in range(steps):
        res = o.step(t, grads(N, t))
        for i in range(N):
            for l in (0, 2):
                assert np.array_equal(res[l].msg[i], d_ref[t][i][l][res[l].idx])
            assert np.array_equal(res[1].msg[i], d_ref[t][i][1])
    for i in range(N):
        assert np.array_equal(o.decompress_error(i), np.concatenate([e_ref[i][0], e_ref[i][2]]))


def test_error_feedback_conserves_mass_with_identity_C():
    # sum_t Delta_t^i + e_T^i = eta sum_t g_t^i  (nothing is lost, only delayed)
    N, lr, steps = 2, 0.05, 12
    q = orc.QCfg(kind="randk", k_num=1, k_den=8, seed=5)
    o = orc.ConEFOracle(TENSORS, N, q, orc.CCfg(kind="identity"), lr)
    sent = [np.zeros(OFF[1]) for _ in range(N)]
    gsum = [np.zeros(OFF[1]) for _ in range(N)]
    for t in range(steps):
        g = grads(N, t, seed=1)
        res = o.step(t, g)
        for i in range(N):
            sent[i][res[0].idx] += res[0].msg[i]
            gsum[i] += g[i][:OFF[1]]
    for i in range(N):
        e = o.decode(i, 0)
        assert np.allclose(sent[i] + e, lr * gsum[i], rtol=0, atol=1e-7)


@pytest.mark.parametrize("ckind", ["int8", "int4", "countsketch"])
def test_proof_bookkeeping_identity(ckind):
    # zeta_t^i = e_{t+1}^i - (p_t^i - Delta_t^i);  z_{t+1} = z_t - eta/N sum g - 1/N sum zeta
    # with z_t = x_t - 1/N sum_i e_t^i and x_{t+1} = x_t - 1/N sum_i Delta_t^i
    N, lr, steps = 3, 0.1, 5
    q = orc.QCfg(kind="randk", k_num=1, k_den=10, seed=3)
    c = orc.CCfg(kind=ckind, block=64, scale_dtype="fp32", cs_rows=3, cs_col_div=2, seed=9)
    o = orc.ConEFOracle(TENSORS, N, q, c, lr)
    l, d = 0, OFF[1]
    x = np.zeros(d)
    for t in range(steps):
        e_old = np.mean([o.decode(i, l).astype(np.float64) for i in range(N)], axis=0)
        z_old = x - e_old
        g = grads(N, t, seed=2)
        res = o.step(t, g, record=True)
        delta = np.zeros((N, d))
        for i in range(N):
            delta[i, res[l].idx] = res[l].msg[i]
            # residual recorded by the oracle is p - Delta
            assert np.array_equal(res[l].r[i].astype(np.float64), res[l].p[i].astype(np.float64) - delta[i])
        x = x - delta.mean(axis=0)
        e_new = [o.decode(i, l).astype(np.float64) for i in range(N)]
        zeta = np.mean([e_new[i] - res[l].r[i] for i in range(N)], axis=0)
        gbar = np.mean([gi[:d].astype(np.float64) for gi in g], axis=0)
        z_new = x - np.mean(e_new, axis=0)
        assert np.allclose(z_new, z_old - lr * gbar - zeta, rtol=0, atol=1e-8)
        # C is contractive on what it was given
        for i in range(N):
            r2 = np.sum(res[l].r[i].astype(np.float64) ** 2)
            if ckind != "countsketch":
                assert np.sum((e_new[i] - res[l].r[i]) ** 2) < r2


def test_identity_Q_leaves_no_error():
    N, lr = 2, 0.1
    # random-k with k = d
    o = orc.ConEFOracle(TENSORS, N, orc.QCfg(kind="randk", k_num=1, k_den=1, seed=1),
                        orc.CCfg(kind="int8", block=32), lr)
    for t in range(2):
        g = grads(N, t, seed=3)
        res = o.step(t, g)
        for i in range(N):
            assert np.array_equal(res[0].msg[i], np.float32(lr) * g[i][:OFF[1]])  # plain SGD step
            assert not o.state[i][0]["codes"].any() and not o.state[i][0]["scales"].any()
            assert not o.decompress_error(i).any()
    # explicit identity
    o = orc.ConEFOracle(TENSORS, N, orc.QCfg(kind="identity"), orc.CCfg(kind="int4", block=16), lr)
    res = o.step(0, grads(N, 0, seed=3))
    assert not o.decompress_error(0).any()
    # full rank: r = min(n, m) makes P_hat P_hat^T the identity on range(M)
    ts = [(12, 20, 1)]
    q0 = rng(4).standard_normal(20 * 12).astype(np.float32)
    o = orc.ConEFOracle(ts, N, orc.QCfg(kind="lowrank", rank=64, q_init=q0), orc.CCfg(kind="identity"), lr)
    g = [(rng(50 + i).standard_normal(240)).astype(np.float32) for i in range(N)]
    o.step(0, g)
    for i in range(N):
        assert np.linalg.norm(o.decompress_error(i)) <= 1e-5 * np.linalg.norm(lr * g[i])


def test_lowrank_step_wiring():
    # mean_i Delta_i = P_hat Qbar^T; warm start is the mean of the Q_i; ranks clip to the shape
    ts = [(30, 50, 1), (3, 40, 1), (8, 1, 0)]
    N, lr, rank = 3, 0.05, 4
    sizes = [50 * 4, 40 * 3]
    q0 = rng(5).standard_normal(sum(sizes)).astype(np.float32)
    o = orc.ConEFOracle(ts, N, orc.QCfg(kind="lowrank", rank=rank, q_init=q0), orc.CCfg(kind="identity"), lr)
    assert o.rank_of(1) == 3
    tot = sum(a * b for a, b, _ in ts)
    g = [(rng(60 + i).standard_normal(tot) * 0.01).astype(np.float32) for i in range(N)]
    res = o.step(0, g, record=True)
    for l in (0, 1):
        n, m, _ = ts[l]
        ls = res[l]
        assert np.array_equal(ls.Pbar, (ls.P[0] + ls.P[1]) + ls.P[2])
        assert np.allclose(ls.P[1], ls.p[1].reshape(n, m).astype(np.float64) @ o_q0(q0, ts, rank, l), atol=1e-6)
        assert np.array_equal(o.Qprev[l], ((ls.Qi[0] + ls.Qi[1]) + ls.Qi[2]) / np.float32(N))
        for i in range(N):
            delta = ls.Phat.astype(np.float64) @ ls.Qi[i].astype(np.float64).T
            assert np.allclose(ls.p[i].reshape(n, m) - delta, ls.r[i].reshape(n, m), atol=1e-6)
            assert np.array_equal(o.decode(i, l), ls.r[i])
    assert np.array_equal(o.reduced(res, "P"), np.concatenate([res[0].Pbar.ravel(), res[1].Pbar.ravel()]))
    assert o.reduced(res, "dense1d").size == 8


def o_q0(q0, ts, rank, l):
    off = 0
    for j, (n, m, c) in enumerate(ts):
        if not (c and m > 1):
            continue
        r = min(rank, n, m)
        if j == l:
            return q0[off:off + m * r].reshape(m, r).astype(np.float64)
        off += m * r
    raise KeyError(l)
