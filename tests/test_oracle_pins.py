"""Pins of the CPU oracle against what the paper and the mathematics fix.

None of these tests touches the CUDA library.  Each one is chosen so that a
plausible mistake in the oracle (a dropped term, a wrong sign or index, a
transposed operand, a wrong rounding) fails it.
"""
import math
import os

import numpy as np
import pytest

from oracle import conef_oracle as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
M64 = 2**64 - 1


def rng(seed):
    return np.random.default_rng(seed)


# ----------------------------------------------------------------- hashing

def test_mixer_matches_published_splitmix64_vectors():
    want = [int(l, 16) for l in open(os.path.join(GOLDEN, "splitmix64_seed0.txt"))
            if l.strip() and not l.startswith("#")]
    got = [orc.mix64((0x9E3779B97F4A7C15 * i) & M64) for i in (1, 2, 3)]
    assert got == want


def test_hash_streams_differ_by_every_key_part():
    base = orc.h64(5, 1, 2, 3)
    assert len({base, orc.h64(6, 1, 2, 3), orc.h64(5, 2, 2, 3), orc.h64(5, 1, 3, 3),
                orc.h64(5, 1, 2, 4), orc.h64(5, 2, 1, 3)}) == 6


# ----------------------------------------------------------------- binary16

def test_fp16_conversion_matches_numpy():
    r = rng(1)
    x = np.concatenate([
        (r.standard_normal(20000) * 10.0 ** r.uniform(-9, 5, 20000)).astype(np.float32),
        np.array([0.0, -0.0, 65504.0, 65519.9, 65520.0, 1e9, 2.0**-24, 2.0**-25, 1.5 * 2.0**-25,
                  2.0**-26, 6.1e-5, 6.097e-5, 5.96e-8, 2.98e-8, 2.99e-8, 1.0, 1.0009765625,
                  1.00048828125, 1.00146484375, np.inf, -np.inf], dtype=np.float32)])
    want = x.astype(np.float16)
    got = np.array([orc.f32_to_f16_bits(float(v)) for v in x], dtype=np.uint16)
    assert np.array_equal(got, want.view(np.uint16))
    back = np.array([orc.f16_bits_to_f32(int(h)) for h in got], dtype=np.float32)
    assert np.array_equal(back, want.astype(np.float32))
    # every half bit pattern decodes as numpy does
    allh = np.arange(65536, dtype=np.uint16)
    dec = np.array([orc.f16_bits_to_f32(int(h)) for h in allh], dtype=np.float32)
    ref = allh.view(np.float16).astype(np.float32)
    assert np.array_equal(np.isnan(dec), np.isnan(ref))
    assert np.array_equal(dec[~np.isnan(ref)], ref[~np.isnan(ref)])


# ----------------------------------------------------------------- line 5

def test_form_p_is_a_single_rounding():
    r = rng(2)
    g = r.standard_normal(5000).astype(np.float32)
    e = (r.standard_normal(5000) * 1e-3).astype(np.float32)
    lr = np.float32(0.1)
    p = orc.form_p(lr, g, e)
    # fp32 products are exact in fp64 and the fp64 sum is far finer than fp32
    want = (lr.astype(np.float64) * g.astype(np.float64) + e.astype(np.float64)).astype(np.float32)
    assert np.array_equal(p, want)
    assert np.array_equal(orc.passthrough(lr, g), lr * g)


# ----------------------------------------------------------------- random-k

@pytest.mark.parametrize("d,k", [(1, 1), (7, 3), (16, 16), (16, 1), (13, 5)])
def test_randk_brute_force_tiny(d, k):
    seed, tensor, step = 99, 3, 17
    idx = orc.randk_indices(seed, tensor, step, d, k)
    keys = sorted(((orc.h64(seed, tensor, step, j) >> 32) << 32 | j) for j in range(d))
    want = sorted(key & 0xFFFFFFFF for key in keys[:k])
    assert idx.tolist() == want


def test_randk_set_properties():
    d, k = 20011, 200
    a = orc.randk_indices(7, 0, 0, d, k)
    assert a.size == k and len(set(a.tolist())) == k
    assert a.min() >= 0 and a.max() < d
    assert np.all(np.diff(a.astype(np.int64)) > 0)
    assert np.array_equal(a, orc.randk_indices(7, 0, 0, d, k))      # same on every worker
    assert not np.array_equal(a, orc.randk_indices(7, 0, 1, d, k))  # new set each step
    assert not np.array_equal(a, orc.randk_indices(7, 1, 0, d, k))  # and per tensor
    assert not np.array_equal(a, orc.randk_indices(8, 0, 0, d, k))


def test_randk_is_uniform_and_contractive_as_assumption_4():
    # E||Q(x)-x||^2 = (1 - k/d) ||x||^2 for the unscaled compressor; every
    # index is kept with probability k/d.
    d, k, trials = 400, 40, 1500
    x = rng(3).standard_normal(d).astype(np.float32)
    counts = np.zeros(d)
    err = 0.0
    for s in range(trials):
        idx = orc.randk_indices(1234, 0, s, d, k)
        counts[idx] += 1
        msg, r = orc.randk_apply(x, idx)
        assert np.array_equal(msg, x[idx])
        e2 = float(np.sum(r.astype(np.float64) ** 2))
        # exact identity ||Q(x)-x||^2 = ||x||^2 - ||x_S||^2
        assert math.isclose(e2, float(np.sum(x.astype(np.float64) ** 2) - np.sum(x[idx].astype(np.float64) ** 2)),
                            rel_tol=1e-12)
        err += e2
    freq = counts / trials
    sigma = math.sqrt(0.1 * 0.9 / trials)
    assert abs(freq.mean() - k / d) < 1e-12
    assert np.max(np.abs(freq - k / d)) < 5 * sigma
    mean_ratio = err / trials / float(np.sum(x.astype(np.float64) ** 2))
    assert abs(mean_ratio - (1 - k / d)) < 0.01


def test_randk_delta_plus_residual_is_p_bitwise():
    d, k = 5000, 50
    p = rng(4).standard_normal(d).astype(np.float32)
    idx = orc.randk_indices(1, 0, 0, d, k)
    msg, r = orc.randk_apply(p, idx)
    delta = np.zeros(d, np.float32)
    delta[idx] = msg
    assert np.array_equal(delta + r, p)
    assert np.all(r[idx] == 0)          # exactly k zeros sit on the transmitted entries
    mask = np.ones(d, bool)
    mask[idx] = False
    assert np.array_equal(r[mask], p[mask])


# ----------------------------------------------------------------- quantiser C

def _unpack(codes, d, bits):
    if bits == 8:
        return codes.view(np.int8).astype(np.int32)[:d]
    lo = (codes & 0xF).astype(np.int32)
    hi = (codes >> 4).astype(np.int32)
    both = np.stack([lo, hi], axis=1).reshape(-1)[:d]
    return np.where(both >= 8, both - 16, both)


@pytest.mark.parametrize("bits,block,half", [(8, 256, False), (4, 128, True), (4, 128, False), (8, 64, True)])
def test_quant_matches_numpy_rint_and_bounds(bits, block, half):
    qmax = 127 if bits == 8 else 7
    d = block * 37 + 19                      # ragged last block
    x = (rng(5).standard_t(3, d) * 1e-3).astype(np.float32)
    codes, s32, s16 = orc.quant_encode(x, block, bits, half)
    nb = (d + block - 1) // block
    assert s32.size == nb
    pad = np.zeros(nb * block, np.float32)
    pad[:d] = np.abs(x)
    a = pad.reshape(nb, block).max(axis=1)
    s = a / np.float32(qmax)
    if half:
        s = s.astype(np.float16)
        assert np.array_equal(s.view(np.uint16), s16)
        s = s.astype(np.float32)
    assert np.array_equal(s, s32)
    inv = np.float32(1.0) / s
    want = np.clip(np.rint(x * np.repeat(inv, block)[:d]), -qmax, qmax).astype(np.int32)
    got = _unpack(codes, d, bits)
    assert np.array_equal(got, want)
    dec = orc.quant_decode(codes, s32, d, block, bits)
    assert np.array_equal(dec, got.astype(np.float32) * np.repeat(s32, block)[:d])
    srep = np.repeat(s32, block)[:d].astype(np.float64)
    err = np.abs(dec.astype(np.float64) - x)
    if not half:
        # no clamp with an fp32 scale: within half a step (plus the rounding of x*inv)
        assert np.all(err <= srep * (0.5 + 1e-5))
        # the absmax element takes code +-qmax
        mx = np.abs(got).reshape(-1)
        full = np.abs(got[: (d // block) * block]).reshape(-1, block).max(axis=1)
        assert np.all(full == qmax)
    # contraction of C (Assumption 3's second part): per block ||C(x)-x||^2 <= B/(4 qmax^2) a^2
    theta_blk = block / (4.0 * qmax * qmax)
    e2 = np.zeros(nb * block)
    e2[:d] = err ** 2
    x2 = np.zeros(nb * block)
    x2[:d] = x.astype(np.float64) ** 2
    slack = 1.01 if not half else 1.6       # a rounded-down half scale adds clamp error
    assert np.all(e2.reshape(nb, block).sum(1) <= slack * theta_blk * (a.astype(np.float64) ** 2) + 1e-30)
    assert e2.sum() < x2.sum()               # theta < 1 overall: contractive


def test_quant_nibble_order_ties_clamp_and_zero_block():
    # block of 4, int4: scale = 7/7 = 1 -> codes are the rounded inputs
    x = np.array([7.0, -7.0, 0.5, 1.5, 0.0, 0.0, 0.0, 0.0, 3.5, -2.5, 2.5, -0.5], np.float32)
    codes, s32, _ = orc.quant_encode(x, 4, 4, False)
    assert s32.tolist() == [1.0, 0.0, 0.5]
    # ties to even: 0.5 -> 0, 1.5 -> 2; third block scale 0.5: 7, -5, 5, -1
    want = [7, -7, 0, 2, 0, 0, 0, 0, 7, -5, 5, -1]
    assert _unpack(codes, 12, 4).tolist() == want
    # low nibble holds the even element
    assert codes[0] == ((7 & 0xF) | ((-7 & 0xF) << 4))
    assert codes[1] == ((0 & 0xF) | ((2 & 0xF) << 4))
    # int8, odd length
    y = np.array([127.0, -63.5, 64.5], np.float32)
    c8, s8, _ = orc.quant_encode(y, 256, 8, False)
    assert s8.tolist() == [1.0] and c8.view(np.int8).tolist() == [127, -64, 64]
    # a scale that underflows binary16 to zero drops the block
    z = np.full(8, 1e-9, np.float32)
    cz, sz, hz = orc.quant_encode(z, 8, 4, True)
    assert sz.tolist() == [0.0] and hz.tolist() == [0] and not cz.any()
    # a half scale rounded down makes |x/s| exceed qmax: clamped
    v = np.array([7 * 1.0004, 1.0], np.float32)
    cv, sv, _ = orc.quant_encode(v, 2, 4, True)
    assert sv[0] == np.float32(np.float16(v[0] / np.float32(7))) and sv[0] < v[0] / 7
    assert _unpack(cv, 2, 4).tolist() == [7, 1]


def test_quant_codes_idempotent_with_fp32_scales():
    x = rng(6).standard_normal(256 * 20).astype(np.float32)
    codes, s32, _ = orc.quant_encode(x, 256, 8, False)
    dec = orc.quant_decode(codes, s32, x.size, 256, 8)
    codes2, s2, _ = orc.quant_encode(dec, 256, 8, False)
    assert np.array_equal(codes, codes2)
    assert np.allclose(s32, s2, rtol=2e-7, atol=0)


# ----------------------------------------------------------------- count sketch C

def test_sketch_buckets_in_range_and_signs_balanced():
    w = 37
    bs = [orc.sketch_bucket(11, 2, i, j, w) for i in range(3) for j in range(4000)]
    b = np.array([x[0] for x in bs])
    s = np.array([x[1] for x in bs])
    assert b.min() == 0 and b.max() == w - 1
    assert set(s.tolist()) == {-1, 1}
    assert abs(s.mean()) < 0.05
    cnt = np.bincount(b, minlength=w) / b.size
    assert np.max(np.abs(cnt - 1 / w)) < 0.01


def test_sketch_brute_force_encode_decode():
    d, v, w, seed, tensor = 50, 3, 7, 5, 4
    x = rng(7).standard_normal(d).astype(np.float32)
    S = orc.sketch_encode(x, v, w, seed, tensor).reshape(v, w)
    want = np.zeros((v, w))
    est = np.zeros((v, d))
    for i in range(v):
        for j in range(d):
            b, s = orc.sketch_bucket(seed, tensor, i, j, w)
            want[i, b] += s * float(x[j])
    assert np.array_equal(S, want.astype(np.float32))
    for i in range(v):
        for j in range(d):
            b, s = orc.sketch_bucket(seed, tensor, i, j, w)
            est[i, j] = np.float32(s) * S[i, b]
    dec = orc.sketch_decode(S.reshape(-1), d, v, w, seed, tensor)
    assert np.array_equal(dec, np.median(est, axis=0).astype(np.float32))


def test_sketch_median_of_five_matches_numpy():
    d, v, w = 300, 5, 40
    x = rng(8).standard_normal(d).astype(np.float32)
    S = orc.sketch_encode(x, v, w, 1, 0)
    dec = orc.sketch_decode(S, d, v, w, 1, 0)
    S2 = S.reshape(v, w)
    est = np.array([[orc.sketch_bucket(1, 0, i, j, w)[1] * S2[i, orc.sketch_bucket(1, 0, i, j, w)[0]]
                     for j in range(d)] for i in range(v)], dtype=np.float32)
    assert np.array_equal(dec, np.median(est, axis=0))


def test_sketch_linearity_and_one_sparse_recovery():
    d, v, w = 1000, 5, 100
    r = rng(9)
    a = r.standard_normal(d).astype(np.float32)
    b = r.standard_normal(d).astype(np.float32)
    Sa, Sb = orc.sketch_encode(a, v, w, 3, 1), orc.sketch_encode(b, v, w, 3, 1)
    Sab = orc.sketch_encode(a + b, v, w, 3, 1)
    assert np.allclose(Sab, Sa + Sb, rtol=0, atol=1e-5)       # C(a+b) = C(a)+C(b) (Sec. 4.2.2)
    one = np.zeros(d, np.float32)
    one[123] = 2.5
    dec = orc.sketch_decode(orc.sketch_encode(one, v, w, 3, 1), d, v, w, 3, 1)
    assert dec[123] == np.float32(2.5)
    # v = 1 and no collisions: the sketch is a signed permutation, decode is exact
    dd, ww = 12, 100000
    buckets = [orc.sketch_bucket(21, 0, 0, j, ww)[0] for j in range(dd)]
    assert len(set(buckets)) == dd
    y = r.standard_normal(dd).astype(np.float32)
    assert np.array_equal(orc.sketch_decode(orc.sketch_encode(y, 1, ww, 21, 0), dd, 1, ww, 21, 0), y)


def test_sketch_row_estimates_unbiased_and_linf_bound():
    # Prop. 2: E[C(e)] = e; ||e - C(e)||_inf <= eps ||e|| w.h.p. for w = Theta(1/eps^2)
    d, w, trials = 200, 50, 1200
    x = rng(10).standard_normal(d).astype(np.float32)
    acc = np.zeros(d)
    for s in range(trials):
        acc += orc.sketch_decode(orc.sketch_encode(x, 1, w, 1000 + s, 0), d, 1, w, 1000 + s, 0)
    mean = acc / trials
    # a single-row estimate has variance <= ||x||^2 / w
    sigma = np.linalg.norm(x) / math.sqrt(w) / math.sqrt(trials)
    assert np.max(np.abs(mean - x)) < 5 * sigma
    bad = 0
    eps = 3.0 / math.sqrt(w)
    for s in range(50):
        dec = orc.sketch_decode(orc.sketch_encode(x, 5, w, 5000 + s, 0), d, 5, w, 5000 + s, 0)
        bad += np.max(np.abs(dec - x)) > eps * np.linalg.norm(x)
    assert bad <= 2


# ----------------------------------------------------------------- low-rank Q

def test_projections_match_numpy_and_are_not_transposed():
    r = rng(11)
    n, m, k = 37, 53, 4
    M = r.standard_normal((n, m)).astype(np.float32)
    Q = r.standard_normal((m, k)).astype(np.float32)
    P = orc.lowrank_project_rows(M, Q)
    assert P.shape == (n, k)
    assert np.array_equal(P, (M.astype(np.float64) @ Q.astype(np.float64)).astype(np.float32)) or \
        np.allclose(P, M.astype(np.float64) @ Q.astype(np.float64), rtol=1e-6, atol=1e-6)
    Ph = r.standard_normal((n, k)).astype(np.float32)
    Qi = orc.lowrank_project_cols(M, Ph)
    assert Qi.shape == (m, k)
    assert np.allclose(Qi, M.astype(np.float64).T @ Ph.astype(np.float64), rtol=1e-6, atol=1e-6)


def test_gram_schmidt_orthonormal_and_same_projector_as_qr():
    r = rng(12)
    A = r.standard_normal((500, 8)).astype(np.float32)
    Ph = orc.gram_schmidt(A)
    assert np.allclose(Ph.T.astype(np.float64) @ Ph, np.eye(8), atol=1e-6)
    Qn, Rn = np.linalg.qr(A.astype(np.float64))
    assert np.allclose(Ph.astype(np.float64) @ Ph.T, Qn @ Qn.T, atol=1e-5)
    # left-to-right: column c spans the same space as the first c+1 columns of A,
    # with a positive coefficient on A[:, c]
    for c in range(8):
        assert float(Ph[:, c].astype(np.float64) @ A[:, c]) > 0
        Qc, _ = np.linalg.qr(A[:, : c + 1].astype(np.float64))
        assert np.allclose(Qc @ (Qc.T @ Ph[:, c]), Ph[:, c], atol=1e-5)
    # a dependent column becomes (numerically) negligible or zero, never NaN
    B = A.copy()
    B[:, 3] = 0
    assert np.all(orc.gram_schmidt(B)[:, 3] == 0)


def test_lowrank_pythagoras_contraction_and_delta_plus_r():
    r = rng(13)
    n, m, k = 120, 96, 4
    M = r.standard_normal((n, m)).astype(np.float32)
    Q0 = r.standard_normal((m, k)).astype(np.float32)
    Ph = orc.gram_schmidt(orc.lowrank_project_rows(M, Q0))
    Qi = orc.lowrank_project_cols(M, Ph)
    res, delta = orc.lowrank_residual(M, Ph, Qi, want_delta=True)
    # Delta + r = p up to the roundings of the chain: k fused multiply-adds,
    # each within half an ulp of a partial result no larger than |p| + sum_c |P Q|
    big = np.abs(M) + np.abs(Ph) @ np.abs(Qi).T
    ulp = np.spacing(big.astype(np.float32))
    assert np.all(np.abs((delta.astype(np.float64) + res) - M) <= 0.5 * (k + 1) * ulp)
    # r = (I - P P^T) M : ||r||^2 = ||M||^2 - ||P^T M||^2 <= ||M||^2  (Assumption 4, delta <= 1)
    M64 = M.astype(np.float64)
    lhs = np.sum(res.astype(np.float64) ** 2)
    rhs = np.sum(M64 ** 2) - np.sum((Ph.astype(np.float64).T @ M64) ** 2)
    assert math.isclose(lhs, rhs, rel_tol=1e-5)
    assert lhs <= np.sum(M64 ** 2)
    assert np.allclose(res, M64 - Ph.astype(np.float64) @ (Ph.astype(np.float64).T @ M64), atol=1e-5)


def test_lowrank_exact_when_rank_fits_and_power_iteration_reaches_svd():
    r = rng(14)
    n, m, k = 80, 60, 4
    U, _ = np.linalg.qr(r.standard_normal((n, n)))
    V, _ = np.linalg.qr(r.standard_normal((m, m)))
    # rank(M) <= r: one iteration reproduces M
    low = (U[:, :k] * np.array([5.0, 3.0, 2.0, 1.0])) @ V[:, :k].T
    M = low.astype(np.float32)
    Q0 = r.standard_normal((m, k)).astype(np.float32)
    Ph = orc.gram_schmidt(orc.lowrank_project_rows(M, Q0))
    res = orc.lowrank_residual(M, Ph, orc.lowrank_project_cols(M, Ph))
    assert np.linalg.norm(res) <= 1e-5 * np.linalg.norm(M)
    # planted spectrum: repeated power iterations converge to the top-r subspace
    sig = np.concatenate([[10, 8, 6, 5], 0.5 * r.random(m - 4)])
    M = ((U[:, :m] * sig) @ V.T).astype(np.float32)
    Q = Q0
    for _ in range(40):
        Ph = orc.gram_schmidt(orc.lowrank_project_rows(M, Q))
        Q = orc.lowrank_project_cols(M, Ph)
    res = orc.lowrank_residual(M, Ph, Q)
    Us, ss, _ = np.linalg.svd(M.astype(np.float64), full_matrices=False)
    assert math.isclose(np.sum(res.astype(np.float64) ** 2), np.sum(ss[k:] ** 2), rel_tol=1e-3)
    assert np.allclose(Ph.astype(np.float64) @ Ph.T, Us[:, :k] @ Us[:, :k].T, atol=1e-3)


# ----------------------------------------------------------------- aggregate

def test_sum_workers_is_in_worker_order_fp32():
    a = np.array([1e8, 1.0], np.float32)
    b = np.array([-1e8, 1.0], np.float32)
    c = np.array([1.0, 1e-8], np.float32)
    assert orc.sum_workers([a, b, c]).tolist() == [1.0, 2.0]
    assert orc.sum_workers([c, a, b]).tolist() == [0.0, 2.0]     # (1 + 1e8) - 1e8 = 0 in fp32
    assert orc.divide(np.array([3.0], np.float32), np.float32(4)).tolist() == [0.75]
