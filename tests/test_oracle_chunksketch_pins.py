"""Pins for the oracle's chunk-wise count sketch (Sec. 4.2.2 applied to runs of a tensor).

The chunked routines are tied to things other than themselves: window bounds redone with Python's
exact integers, the plain count sketch (pinned elsewhere) of one run at a time, the plain sketch
itself when a single run covers the tensor, linearity, exact recovery of sparse inputs, and
unbiasedness of each row's estimate over hash seeds.
"""
import numpy as np
import pytest

import oracle.conef_oracle as orc


def _windows(d, w, E):
    """Window bounds from the definition, in Python integers."""
    nc = max(1, d // E) if E > 0 else 1
    b = [(w * c * E) // d for c in range(nc)] + [w]
    return nc, b


@pytest.mark.parametrize("d,w,E", [(100_000, 10_000, 8192), (8192 * 3, 2457, 8192), (8192 * 3 + 5000, 2957, 8192),
                                   (50, 5, 8192), (20_000, 1, 8192), (70_001, 7000, 16384), (40_000, 39_999, 8192)])
def test_windows_partition_the_buckets_in_proportion(d, w, E):
    nc, b = _windows(d, w, E)
    assert b[0] == 0 and b[-1] == w and all(b[c] <= b[c + 1] for c in range(nc))
    for j in list(range(0, d, max(1, d // 97))) + [d - 1]:
        c = min(j // E, nc - 1)
        assert orc.chunk_window(d, w, E, j) == (b[c], b[c + 1] - b[c])
    # the last run takes the remainder of the elements: between E and 2E - 1 of them once d >= E
    if d >= E:
        assert E <= d - (nc - 1) * E < 2 * E
    # widths follow the element counts to within one bucket
    for c in range(nc):
        n_c = E if c < nc - 1 else d - (nc - 1) * E
        assert abs((b[c + 1] - b[c]) - w * n_c / d) < 1.0 + 1e-9


def test_one_run_is_the_plain_count_sketch():
    rng = np.random.default_rng(1)
    d, v, w = 5000, 5, 500
    r = rng.standard_normal(d).astype(np.float32)
    plain = orc.sketch_encode(r, v, w, 17, 3)
    for E in (0, 8192, 5000, 4096):     # 4096: floor(5000 / 4096) = 1 run as well
        assert np.array_equal(orc.sketch_encode_chunked(r, v, w, E, 17, 3), plain)
        assert np.array_equal(orc.sketch_decode_chunked(plain, d, v, w, E, 17, 3), orc.sketch_decode(plain, d, v, w, 17, 3))


@pytest.mark.parametrize("d,div,E", [(3 * 1024 + 700, 10, 1024), (4 * 512, 7, 512)])
def test_each_window_is_the_plain_sketch_of_its_run(d, div, E):
    """Run c, with every other element zeroed, sketched by the plain routine at the window's width:
    the hash sees the element's index in the whole tensor in both routines."""
    rng = np.random.default_rng(2)
    v, w = 3, d // div
    r = rng.integers(-40, 40, size=d).astype(np.float32)       # integers: sums are exact in any order
    S = orc.sketch_encode_chunked(r, v, w, E, 5, 1).reshape(v, w)
    nc, b = _windows(d, w, E)
    assert nc >= 3
    for c in range(nc):
        lo = c * E
        hi = d if c == nc - 1 else lo + E
        rc = np.zeros(d, np.float32)
        rc[lo:hi] = r[lo:hi]
        width = b[c + 1] - b[c]
        want = orc.sketch_encode(rc, v, width, 5, 1).reshape(v, width)
        assert np.array_equal(S[:, b[c]:b[c + 1]], want)
    # decode: the same medians as decoding each run from its own window
    e = orc.sketch_decode_chunked(S.reshape(-1), d, v, w, E, 5, 1)
    for c in range(nc):
        lo = c * E
        hi = d if c == nc - 1 else lo + E
        win = np.ascontiguousarray(S[:, b[c]:b[c + 1]]).reshape(-1)
        assert np.array_equal(e[lo:hi], orc.sketch_decode(win, d, v, b[c + 1] - b[c], 5, 1)[lo:hi])


def test_chunked_sketch_is_linear_and_recovers_sparse_inputs():
    rng = np.random.default_rng(3)
    d, v, w, E = 5 * 2048 + 77, 5, 1031, 2048
    a = rng.integers(-30, 30, size=d).astype(np.float32)
    b = rng.integers(-30, 30, size=d).astype(np.float32)
    sa = orc.sketch_encode_chunked(a, v, w, E, 9, 0)
    sb = orc.sketch_encode_chunked(b, v, w, E, 9, 0)
    assert np.array_equal(orc.sketch_encode_chunked(a + b, v, w, E, 9, 0), sa + sb)
    # one non-zero per run decodes exactly: nothing collides with it inside its window
    x = np.zeros(d, np.float32)
    pos = [100, 2048 + 5, 3 * 2048 + 1999, d - 1]
    x[pos] = [1.5, -2.0, 3.25, -4.0]
    e = orc.sketch_decode_chunked(orc.sketch_encode_chunked(x, v, w, E, 9, 0), d, v, w, E, 9, 0)
    assert np.array_equal(e[pos], x[pos])
    # an element of another run never sees it: runs without a non-zero decode to zero everywhere
    assert not e[2 * 2048:3 * 2048].any()


def test_each_row_estimate_is_unbiased_over_seeds():
    d, w, E = 3 * 256, 96, 256
    rng = np.random.default_rng(4)
    x = rng.standard_normal(d).astype(np.float32)
    j = 300                                      # an element of the second run
    est = []
    for seed in range(600):
        S = orc.sketch_encode_chunked(x, 1, w, E, seed, 0)
        est.append(orc.sketch_decode_chunked(S, d, 1, w, E, seed, 0)[j])
    est = np.array(est, np.float64)
    # variance of a one-row estimate: energy of the run's other elements over the window's width
    lo, width = orc.chunk_window(d, w, E, j)
    var = (np.sum(x[256:512].astype(np.float64) ** 2) - float(x[j]) ** 2) / width
    assert abs(est.mean() - x[j]) < 4 * np.sqrt(var / len(est))
    assert 0.7 * var < est.var() < 1.4 * var


def test_whole_step_with_chunked_sketch_conserves_the_update():
    """Alg. 2 with the chunked sketch as C: p = eta g + decode(S); message + residual = p."""
    tensors = [(40, 128, 1)]
    q = orc.QCfg(kind="randk", k_num=1, k_den=10, seed=3)
    c = orc.CCfg(kind="countsketch", cs_rows=3, cs_col_div=4, seed=8, cs_chunk=1024)
    o = orc.ConEFOracle(tensors, 2, q, c, 0.5)
    rng = np.random.default_rng(5)
    for t in range(3):
        grads = [(rng.integers(-64, 64, size=5120) / 8.0).astype(np.float32) for _ in range(2)]
        e_before = [o.decode(i, 0) for i in range(2)]
        res = o.step(t, grads, record=True)
        for i in range(2):
            p = (0.5 * grads[i].astype(np.float64) + e_before[i].astype(np.float64)).astype(np.float32)
            assert np.array_equal(res[0].p[i], p)
            r = p.copy()
            r[res[0].idx] = 0
            assert np.array_equal(o.state[i][0]["S"], orc.sketch_encode_chunked(r, 3, 1280, 1024, 8, 0))
