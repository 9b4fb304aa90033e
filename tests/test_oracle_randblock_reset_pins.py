"""Pins for random-block-k (Sec. 5.3) and for error reset with a linear C (Sec. 4.2.2)."""
import numpy as np

import oracle.conef_oracle as orc


def test_randblock_start_is_the_scaled_top_bits_of_the_pinned_hash():
    d, k = 1000, 37
    for step in range(20):
        got = orc.randblock_indices(9, 4, step, d, k)
        u = orc.h64(9, 4, step, 0) >> 32
        start = (u * (d - k + 1)) >> 32
        assert np.array_equal(got, np.arange(start, start + k, dtype=np.uint32))
        assert 0 <= start <= d - k


def test_randblock_full_and_single():
    assert np.array_equal(orc.randblock_indices(1, 0, 0, 50, 50), np.arange(50, dtype=np.uint32))
    starts = {int(orc.randblock_indices(1, 0, t, 10, 1)[0]) for t in range(400)}
    assert starts == set(range(10))            # every start is reachable, none outside


def test_randblock_starts_are_roughly_uniform():
    d, k, T = 64 + 15, 16, 6400
    counts = np.bincount([int(orc.randblock_indices(3, 1, t, d, k)[0]) for t in range(T)], minlength=d - k + 1)
    expect = T / (d - k + 1)
    assert np.all(np.abs(counts - expect) < 6 * np.sqrt(expect))


def test_randblock_step_is_error_feedback_on_a_block():
    tensors = [(8, 16, 1)]
    o = orc.ConEFOracle(tensors, 2, orc.QCfg(kind="randblock", k_num=1, k_den=4, seed=2), orc.CCfg(kind="identity"), 0.5)
    rng = np.random.default_rng(0)
    g = [(rng.integers(-16, 16, size=128) / 4).astype(np.float32) for _ in range(2)]
    res = o.step(0, g, record=True)
    idx = res[0].idx
    assert idx.size == 32 and np.array_equal(np.diff(idx), np.ones(31, np.uint32))
    for i in range(2):
        p = 0.5 * g[i]
        assert np.array_equal(res[0].msg[i], p[idx])
        r = p.copy()
        r[idx] = 0
        assert np.array_equal(o.decode(i, 0), r)


def test_error_reset_averages_linear_states_and_keeps_their_sum():
    n, m, N = 20, 8, 4
    c = orc.CCfg(kind="rowsketch", cs_rows=1, cs_col_div=4, seed=3, beta=0.5)
    o = orc.ConEFOracle([(n, m, 1)], N, orc.QCfg(kind="randk", k_num=1, k_den=8, seed=1), c, 1.0)
    rng = np.random.default_rng(1)
    for t in range(3):
        o.step(t, [(rng.integers(-8, 8, size=n * m) * 4.0).astype(np.float32) for _ in range(N)])
    before = [o.state[i][0]["T"].astype(np.float64) for i in range(N)]
    dec_before = [o.decode(i, 0).astype(np.float64) for i in range(N)]
    o.error_reset()
    mean = sum(before) / N
    for i in range(N):
        assert np.array_equal(o.state[i][0]["T"].astype(np.float64), mean)       # dyadic data: exact
        # linear C with v = 1: the decode of the mean is the mean of the decodes
        assert np.array_equal(o.decode(i, 0).astype(np.float64), sum(dec_before) / N)
