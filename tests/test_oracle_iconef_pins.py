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
