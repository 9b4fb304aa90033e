"""The tuned pass-3 kernel forms a block scale amax / qmax as
    q = amax * c;  rem = fma(-qmax, q, amax);  s = fma(rem, c, q),   c = RN(1 / qmax),
instead of calling the division routine.  This must be the correctly rounded
IEEE quotient, which the oracle's `a / qmax` is.  Scaling by a power of two is
exact, so it is enough to check every fp32 significand; fp64 evaluates each of
the three steps exactly before the single rounding to fp32 (products of two
24-bit numbers, and sums whose bits span fewer than 53 positions)."""
import numpy as np
import pytest


@pytest.mark.parametrize("qmax", [7.0, 127.0])
def test_fma_sequence_equals_ieee_division_for_every_significand(qmax):
    c = np.float32(1.0) / np.float32(qmax)
    sig = np.arange(2**23, 2**24, dtype=np.int64).astype(np.float64)
    for scale in (1.0, 2.0**-60, 2.0**70):
        a = (sig * scale).astype(np.float32)
        want = a / np.float32(qmax)
        a64 = a.astype(np.float64)
        q = (a64 * np.float64(c)).astype(np.float32)
        rem = (a64 - np.float64(qmax) * q.astype(np.float64)).astype(np.float32)
        s = (rem.astype(np.float64) * np.float64(c) + q.astype(np.float64)).astype(np.float32)
        assert np.array_equal(s, want)
