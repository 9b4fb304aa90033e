"""Pins for the oracle's partial error feedback (Alg. 4) and row-wise count sketch (Sec. 4.2.2).

Each test ties an oracle routine to something other than itself: exact integer
arithmetic redone in numpy from the pinned hash, the flat count sketch (pinned
elsewhere) as the special case of one column, linearity, the closed form of the
error recursion, and the literal Alg. 4 with an uncompressed error when the
sketch is wide enough to be collision-free.
"""
import numpy as np
import pytest

import oracle.conef_oracle as orc


def _buckets(seed, tensor, v, n, w):
    h = np.zeros((v, n), np.int64)
    s = np.zeros((v, n), np.int64)
    for i in range(v):
        for a in range(n):
            h[i, a], s[i, a] = orc.sketch_bucket(seed, tensor, i, a, w)
    return h, s


@pytest.mark.parametrize("v,n,m,w", [(1, 37, 5, 4), (3, 50, 8, 7), (5, 9, 3, 20)])
def test_rowsketch_update_equals_integer_brute_force(v, n, m, w):
    rng = np.random.default_rng(5)
    R = rng.integers(-50, 50, size=(n, m)).astype(np.float32)
    T0 = rng.integers(-8, 8, size=(v, w, m)).astype(np.float32)
    beta = np.float32(0.5)   # halves of small integers stay exact
    h, s = _buckets(11, 3, v, n, w)
    want = 0.5 * T0.astype(np.float64)
    for i in range(v):
        for a in range(n):
            want[i, h[i, a]] += s[i, a] * R[a].astype(np.float64)
    got = orc.rowsketch_update(beta, R, T0.reshape(-1), v, w, 11, 3).reshape(v, w, m)
    assert np.array_equal(got.astype(np.float64), want)


def test_rowsketch_one_column_is_the_flat_count_sketch():
    rng = np.random.default_rng(6)
    n, v, w = 301, 3, 29
    r = rng.integers(-100, 100, size=n).astype(np.float32)
    flat = orc.sketch_encode(r, v, w, 77, 2)
    rows = orc.rowsketch_update(np.float32(0), r.reshape(n, 1), np.zeros(v * w, np.float32), v, w, 77, 2)
    assert np.array_equal(flat, rows)
    assert np.array_equal(orc.sketch_decode(flat, n, v, w, 77, 2), orc.rowsketch_decode(rows, n, 1, v, w, 77, 2))


def test_rowsketch_is_linear():
    rng = np.random.default_rng(7)
    n, m, v, w = 40, 6, 3, 5
    A = rng.integers(-30, 30, size=(n, m)).astype(np.float32)
    B = rng.integers(-30, 30, size=(n, m)).astype(np.float32)
    z = np.zeros(v * w * m, np.float32)
    sa = orc.rowsketch_update(np.float32(0), A, z, v, w, 1, 0)
    sb = orc.rowsketch_update(np.float32(0), B, z, v, w, 1, 0)
    sab = orc.rowsketch_update(np.float32(0), A + B, z, v, w, 1, 0)
    assert np.array_equal(sab, sa + sb)
    # beta T + sketch(B) with T = sketch(A) is the sketch of beta A + B
    both = orc.rowsketch_update(np.float32(0.25), B * 4, sa * 4, v, w, 1, 0)
    assert np.array_equal(both, orc.rowsketch_update(np.float32(0), A + 4 * B, z, v, w, 1, 0))


def test_rowsketch_decode_single_row_and_median():
    n, m, v, w = 64, 4, 3, 16
    R = np.zeros((n, m), np.float32)
    R[10] = [1, -2, 3, -4]
    T = orc.rowsketch_update(np.float32(0), R, np.zeros(v * w * m, np.float32), v, w, 9, 1)
    e = orc.rowsketch_decode(T, n, m, v, w, 9, 1).reshape(n, m)
    assert np.array_equal(e[10], R[10])          # all v estimates agree on the row that was inserted
    h, s = _buckets(9, 1, v, n, w)
    for a in range(n):
        if a == 10:
            continue
        hits = [s[i, a] * s[i, 10] for i in range(v) if h[i, a] == h[i, 10]]
        # the median of v estimates is non-zero only if at least two sketch rows collide with row 10
        est = sorted([float(x) for x in hits] + [0.0] * (v - len(hits)))
        assert np.array_equal(e[a], np.float32(est[v // 2]) * R[10])


def test_form_p_partial_closed_form_and_beta_zero():
    g = np.array([1.0, -2.0, 0.5, 8.0], np.float32)
    e = np.array([4.0, 4.0, -8.0, 0.25], np.float32)
    p = orc.form_p_partial(np.float32(0.5), np.float32(0.25), g, e)
    assert np.array_equal(p, np.array([1.5, 0.0, -1.75, 4.0625], np.float32))
    rng = np.random.default_rng(8)
    g = rng.standard_normal(1000).astype(np.float32)
    e = rng.standard_normal(1000).astype(np.float32)
    assert np.array_equal(orc.form_p_partial(np.float32(0.05), np.float32(1.0), g, e), orc.form_p(np.float32(0.05), g, e))
    # the product (1 - beta) e is rounded before the fused multiply-add
    lr, omb = np.float32(0.05), np.float32(0.1)
    want = (np.float64(lr) * g.astype(np.float64) + (omb * e).astype(np.float64)).astype(np.float32)
    assert np.array_equal(orc.form_p_partial(lr, omb, g, e), want)


def test_partial_keep_is_one_fused_multiply_add():
    rng = np.random.default_rng(9)
    e = rng.standard_normal(1000).astype(np.float32)
    r = rng.standard_normal(1000).astype(np.float32)
    beta = np.float32(0.9)
    want = (np.float64(beta) * e.astype(np.float64) + r.astype(np.float64)).astype(np.float32)
    assert np.array_equal(orc.partial_keep(beta, e, r), want)
    assert np.array_equal(orc.partial_keep(np.float32(0), e, r), r)


def _collision_free_seed(n, w, tensor):
    for seed in range(1, 2000):
        h, _ = _buckets(seed, tensor, 1, n, w)
        if len(set(h[0])) == n:
            return seed
    raise AssertionError("no collision-free seed found")


def test_partial_conef_with_injective_sketch_is_alg4_with_dense_error():
    """With every row in a bucket of its own the sketch stores e exactly, so the oracle's recursion
    (linear update, decode next step) must equal Alg. 4 run literally with an uncompressed error:
    p = eta g + (1-beta) e; Delta = Q(p); e <- beta e + p - Delta.  Dyadic data keep it exact."""
    n, m, w, N = 6, 8, 64, 2
    seed = _collision_free_seed(n, w, 0)
    beta, lr = 0.5, 0.5
    q = orc.QCfg(kind="randk", k_num=1, k_den=4, seed=3)
    c = orc.CCfg(kind="rowsketch", cs_rows=1, cs_col_div=1, seed=seed, beta=beta)
    o = orc.ConEFOracle([(n, m, 1)], N, q, c, lr)
    assert o.w_of(0) == n
    # widen the sketch beyond the number of rows through the state itself
    o.w_of = lambda l: w
    for i in range(N):
        o.state[i][0] = {"T": np.zeros(w * m, np.float32)}
    rng = np.random.default_rng(10)
    e = [np.zeros(n * m) for _ in range(N)]
    for t in range(4):
        grads = [(rng.integers(-64, 64, size=n * m) / 8.0).astype(np.float32) for _ in range(N)]
        res = o.step(t, grads, record=True)
        idx = res[0].idx
        for i in range(N):
            p = lr * grads[i].astype(np.float64) + (1 - beta) * e[i]
            assert np.array_equal(res[0].p[i].astype(np.float64), p)
            assert np.array_equal(res[0].msg[i].astype(np.float64), p[idx])
            r = p.copy()
            r[idx] = 0
            e[i] = beta * e[i] + r
            assert np.array_equal(o.decode(i, 0).astype(np.float64), e[i])


def test_partial_conef_quantiser_path_uses_decoded_error():
    """Alg. 4 with a non-linear C: the state after one more step is C(beta e + r) of the decoded e."""
    n, m, N = 4, 64, 1
    q = orc.QCfg(kind="identity")
    c = orc.CCfg(kind="int8", block=32, beta=0.75)
    o = orc.ConEFOracle([(n, m, 1)], N, q, c, 0.1)
    rng = np.random.default_rng(12)
    codes = rng.integers(-127, 128, size=n * m).astype(np.int8).view(np.uint8)
    scales = (rng.random(n * m // 32).astype(np.float32) + 0.5) / 64
    o.state[0][0] = {"codes": codes.copy(), "scales": scales.copy(), "scales16": None}
    e = o.decode(0, 0)
    g = rng.standard_normal(n * m).astype(np.float32)
    o.step(0, [g])
    # Q = identity sends everything: r = 0 and the new state holds C(beta e)
    want_codes, want_scales, _ = orc.quant_encode((np.float32(0.75) * e).astype(np.float32), 32, 8, False)
    assert np.array_equal(o.state[0][0]["codes"], want_codes)
    assert np.array_equal(o.state[0][0]["scales"], want_scales)


def test_fp16_sketch_equals_fp32_sketch_where_halves_are_exact():
    # small integers are exact in binary16: both storages must hold the same numbers
    rng = np.random.default_rng(21)
    n, m, v, w = 40, 6, 3, 5
    R = rng.integers(-20, 20, size=(n, m)).astype(np.float32)
    T32 = orc.rowsketch_update(np.float32(0), R, np.zeros(v * w * m, np.float32), v, w, 4, 1)
    T16 = orc.rowsketch_update_f16(np.float32(0), R, np.zeros(v * w * m, np.uint16), v, w, 4, 1)
    assert np.array_equal(T16.view(np.float16).astype(np.float32), T32)
    assert np.array_equal(orc.rowsketch_decode_f16(T16, n, m, v, w, 4, 1), orc.rowsketch_decode(T32, n, m, v, w, 4, 1))
    # a second update with beta = 0.5 stays exact as well (halves of small integers)
    T32b = orc.rowsketch_update(np.float32(0.5), R, T32, v, w, 4, 1)
    T16b = orc.rowsketch_update_f16(np.float32(0.5), R, T16, v, w, 4, 1)
    assert np.array_equal(T16b.view(np.float16).astype(np.float32), T32b)


def test_fp16_sketch_rounds_once_and_saturates():
    n, m = 3, 2
    seed = _collision_free_seed(n, 64, 0)
    R = np.array([[1.0 + 2.0 ** -12, 70000.0], [-70000.0, 2.0 ** -26], [0.1, -0.1]], np.float32)
    T16 = orc.rowsketch_update_f16(np.float32(0), R, np.zeros(64 * m, np.uint16), 1, 64, seed, 0)
    e = orc.rowsketch_decode_f16(T16, n, m, 1, 64, seed, 0).reshape(n, m)
    want = np.clip(R, -65504, 65504).astype(np.float16).astype(np.float32)     # numpy's conversion is nearest-even
    assert np.array_equal(e, want)
    assert e[0, 1] == 65504.0 and e[1, 0] == -65504.0 and e[1, 1] == 0.0
