"""Pins for the oracle's iConEF-v1 (Alg. 3): a second compressed state q = C(r - e~)."""
import numpy as np
import pytest

import oracle.conef_oracle as orc


def _one_step(c, n=8, m=64, N=2, seed=0, steps=3):
    o = orc.ConEFOracle([(n, m, 1)], N, orc.QCfg(kind="randk", k_num=1, k_den=8, seed=4), c, 0.5)
    rng = np.random.default_rng(seed)
    out = []
    for t in range(steps):
        g = [rng.standard_normal(n * m).astype(np.float32) for _ in range(N)]
        out.append((g, o.step(t, g, record=True)))
    return o, out


def test_with_identity_c_it_is_plain_error_feedback():
    a, ra = _one_step(orc.CCfg(kind="identity", iconef=1))
    b, rb = _one_step(orc.CCfg(kind="identity"))
    for (ga, resa), (gb, resb) in zip(ra, rb):
        for i in range(2):
            assert np.array_equal(resa[0].msg[i], resb[0].msg[i])
    for i in range(2):
        assert np.array_equal(a.decompress_error(i), b.decompress_error(i))
        assert not a.decode(i, 0, True).any()            # nothing is left for the second state


@pytest.mark.parametrize("kind,qmax,block", [("int8", 127, 64), ("int4", 7, 64)])
def test_second_state_shrinks_the_stored_error_quadratically(kind, qmax, block):
    """|r - e~| <= s1/2 per block with s1 = amax/qmax, and the second level quantises that remainder
    with scale <= (s1/2)/qmax: |r - e~ - q| <= amax / (4 qmax^2) (+ rounding): error feedback on top
    of error feedback (Sec. 3.2)."""
    o, out = _one_step(orc.CCfg(kind=kind, block=block, iconef=1))
    g, res = out[-1]
    for i in range(2):
        r = res[0].r[i]
        e1 = o.decode(i, 0)
        e2 = o.decode(i, 0, True)
        amax = np.abs(r).reshape(-1, block).max(axis=1)
        lvl1 = np.repeat(amax / qmax / 2, block)
        assert np.all(np.abs(r - e1) <= lvl1 * (1 + 1e-5))
        lvl2 = np.repeat(amax / (4.0 * qmax * qmax), block)
        assert np.all(np.abs(r.astype(np.float64) - e1 - e2) <= lvl2 * (1 + 1e-4) + 1e-12)
        # and it is what one level alone would leave, requantised: q = C(r - e~)
        codes, s32, _ = orc.quant_encode((r - e1).astype(np.float32), block, 8 if kind == "int8" else 4, False)
        assert np.array_equal(o.state2[i][0]["codes"], codes)
        assert np.array_equal(o.state2[i][0]["scales"], s32)


def test_p_is_eta_g_plus_both_states():
    o, out = _one_step(orc.CCfg(kind="int8", block=32, iconef=1), steps=2)
    # rerun the second step by hand from the states after the first
    o2, out2 = _one_step(orc.CCfg(kind="int8", block=32, iconef=1), steps=1)
    g2 = out[1][0]
    for i in range(2):
        e1 = o2.decode(i, 0).astype(np.float64)
        e2 = o2.decode(i, 0, True)
        first = (0.5 * g2[i].astype(np.float64) + e1).astype(np.float32)       # one fused rounding
        want = (first + e2).astype(np.float32)
        assert np.array_equal(out[1][1][0].p[i], want)


# ----------------------------------------------------------------- iConEF-v2 (Alg. 3 line 12)

@pytest.mark.parametrize("qkind", ["randk", "randblock"])
def test_v2_with_identity_c_is_plain_error_feedback(qkind):
    """e~ = Q(r) and q = r - e~ split r between them exactly, so p and the messages are those of
    Alg. 1 bit for bit."""
    def run(c):
        o = orc.ConEFOracle([(8, 64, 1)], 2, orc.QCfg(kind=qkind, k_num=1, k_den=8, seed=4), c, 0.5)
        rng = np.random.default_rng(0)
        out = []
        for t in range(4):
            g = [rng.standard_normal(512).astype(np.float32) for _ in range(2)]
            out.append(o.step(t, g, record=True))
        return o, out
    a, ra = run(orc.CCfg(kind="identity", iconef=2))
    b, rb = run(orc.CCfg(kind="identity"))
    for resa, resb in zip(ra, rb):
        assert np.array_equal(resa[0].idx, resb[0].idx)
        for i in range(2):
            assert np.array_equal(resa[0].msg[i], resb[0].msg[i])
            assert np.array_equal(resa[0].p[i], resb[0].p[i])
    for i in range(2):
        assert np.array_equal(a.decompress_error(i), b.decompress_error(i))


@pytest.mark.parametrize("qkind", ["randk", "randblock"])
def test_v2_is_alg3_written_out_with_pinned_primitives(qkind):
    """Alg. 3 with version 2, literally, from the pinned index draw and the pinned quantiser."""
    n, m, N, block, lr = 6, 128, 2, 64, np.float32(0.25)
    d, k = n * m, n * m // 16
    q = orc.QCfg(kind=qkind, k_num=1, k_den=16, seed=9)
    o = orc.ConEFOracle([(n, m, 1)], N, q, orc.CCfg(kind="int8", block=block, iconef=2), lr)
    pick = orc.randk_indices if qkind == "randk" else orc.randblock_indices
    rng = np.random.default_rng(3)
    et = [np.zeros(d, np.float32) for _ in range(N)]       # e~ (dense view)
    qq = [np.zeros(d, np.float32) for _ in range(N)]       # decoded q
    for t in range(4):
        g = [rng.standard_normal(d).astype(np.float32) for _ in range(N)]
        res = o.step(t, g, record=True)
        idx = pick(9, 0, t, d, k)
        idx2 = pick(9, 0, t + (1 << 62), d, k)
        assert np.array_equal(res[0].idx, idx) and np.array_equal(res[0].idx2, idx2)
        assert len(set(idx2.tolist())) == k and not np.array_equal(idx, idx2)
        for i in range(N):
            first = (np.float64(lr) * g[i].astype(np.float64) + et[i].astype(np.float64)).astype(np.float32)
            p = (first + qq[i]).astype(np.float32)                       # line 5
            assert np.array_equal(res[0].p[i], p)
            assert np.array_equal(res[0].msg[i], p[idx])                 # line 6
            r = p.copy()
            r[idx] = 0                                                   # p - Delta
            e_new = np.zeros(d, np.float32)
            e_new[idx2] = r[idx2]                                        # line 12: e~ = Q(p - Delta)
            rest = (r - e_new).astype(np.float32)                        # line 14: q = C(p - Delta - e~)
            codes, scales, _ = orc.quant_encode(rest, block, 8, False)
            assert np.array_equal(o.state[i][0]["codes"], codes)
            assert np.array_equal(o.state[i][0]["scales"], scales)
            assert np.array_equal(o.ev[i][0][0], idx2) and np.array_equal(o.ev[i][0][1], r[idx2])
            et[i] = e_new
            qq[i] = orc.quant_decode(codes, scales, d, block, 8)
            assert np.array_equal(o.decompress_error(i), (et[i] + qq[i]).astype(np.float32))
            # q never covers a coordinate that e~ or the message took
            assert not qq[i][idx2].any() and not qq[i][idx].any()


def test_v2_keeps_more_of_the_residual_than_alg2():
    """The k coordinates kept exactly leave C less to lose: stored error of v2 is closer to r."""
    n, m, N = 8, 256, 1
    q = orc.QCfg(kind="randk", k_num=1, k_den=4, seed=2)
    a = orc.ConEFOracle([(n, m, 1)], N, q, orc.CCfg(kind="int4", block=64), 0.5)
    b = orc.ConEFOracle([(n, m, 1)], N, q, orc.CCfg(kind="int4", block=64, iconef=2), 0.5)
    g = [np.random.default_rng(5).standard_normal(n * m).astype(np.float32)]
    ra = a.step(0, g, record=True)
    rb = b.step(0, g, record=True)
    r = ra[0].r[0]
    assert np.array_equal(r, rb[0].r[0])
    err_a = np.linalg.norm(a.decompress_error(0) - r)
    err_b = np.linalg.norm(b.decompress_error(0) - r)
    assert err_b < err_a
