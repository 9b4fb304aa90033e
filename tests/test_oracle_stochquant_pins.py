"""Pins for the oracle's unbiased stochastic s-level quantiser (Eq. 6, max-norm, block-wise) and for
the counter-based uniform generator that feeds it."""
import numpy as np
import pytest

import oracle.conef_oracle as orc


def test_grid_points_are_reproduced_whatever_the_variate():
    # values a * k / s are levels themselves: no randomness is left (Eq. 6 with u_j integer)
    s, a = 16, 4.0
    k = np.array([0, 1, -3, 16, -16, 7, 8, -9], np.float32)
    r = (k * np.float32(a / s)).astype(np.float32)
    for rnd_val in (0.0, 0.5, 0.99999994):
        codes, scales = orc.stochquant_encode(r, np.full(8, rnd_val, np.float32), 8, s)
        assert np.array_equal(codes, k.astype(np.int16))
        assert scales[0] == np.float32(a / s)
        assert np.array_equal(orc.stochquant_decode(codes, scales, 8), r)


def test_up_or_down_by_the_variate_and_levels_bounded():
    s = 8
    r = np.array([8.0, 2.5, -2.5, 0.3, -7.9], np.float32)      # a = 8, scale 1: u = |r|
    lo, _ = orc.stochquant_encode(r, np.full(5, 0.99, np.float32), 8, s)
    hi, _ = orc.stochquant_encode(r, np.zeros(5, np.float32), 8, s)
    assert np.array_equal(lo, np.array([8, 2, -2, 0, -7], np.int16))   # rnd >= frac: floor
    assert np.array_equal(hi, np.array([8, 3, -3, 1, -8], np.int16))   # rnd < frac: one level up
    # exactly at the threshold: up iff rnd < u - floor(u)
    mid, _ = orc.stochquant_encode(r, np.full(5, 0.5, np.float32), 8, s)
    assert np.array_equal(mid, np.array([8, 2, -2, 0, -8], np.int16))


@pytest.mark.parametrize("levels", [8, 16, 64, 256])
def test_unbiased_in_expectation(levels):
    """E[C(x)] = x (the property Assumption 3 needs): average the decode over many draws."""
    rng = np.random.default_rng(levels)
    d, block, trials = 512, 128, 4000
    r = rng.standard_normal(d).astype(np.float32)
    acc = np.zeros(d, np.float64)
    for t in range(trials):
        rnd = orc.uniform24(99, 0, 3, t, d)
        codes, scales = orc.stochquant_encode(r, rnd, block, levels)
        assert np.abs(codes).max() <= levels
        acc += orc.stochquant_decode(codes, scales, block)
    mean = acc / trials
    # one draw has error below one quantisation step a/s; the mean of `trials` draws is within
    # 5 standard errors of x
    step = np.repeat(np.abs(r).reshape(-1, block).max(axis=1) / levels, block)
    assert np.all(np.abs(mean - r) <= 5 * 0.5 * step / np.sqrt(trials) + 1e-7)


def test_matches_float64_restatement_on_dyadic_inputs():
    rng = np.random.default_rng(3)
    d, block, s = 256, 64, 16
    r = (rng.integers(-1024, 1024, size=d) / 64.0).astype(np.float32)
    r[::64] = 16.0                                   # block maxima a = 16: scale a/s = 1, inv = 1
    rnd = orc.uniform24(1, 2, 3, 4, d)
    codes, scales = orc.stochquant_encode(r, rnd, block, s)
    u = np.abs(r.astype(np.float64))
    want = np.floor(u) + (rnd.astype(np.float64) < (u - np.floor(u)))
    assert np.array_equal(codes, (np.sign(r) * want).astype(np.int16))
    assert np.all(scales == 1.0)


def test_zero_and_tiny_blocks_store_zeros():
    r = np.zeros(64, np.float32)
    r[32:] = 1e-44                                   # a / s underflows below the smallest normal
    codes, scales = orc.stochquant_encode(r, np.zeros(64, np.float32), 32, 16)
    assert not codes.any() and not scales.any()


def test_uniform24_is_the_top_24_bits_of_the_pinned_hash():
    d = 1000
    u = orc.uniform24(42, 3, 7, 11, d)
    seed_w = orc.mix64((42 + 3 + 1) & (2 ** 64 - 1))
    want = np.array([(orc.h64(seed_w, 7, 11, j) >> 40) / 2.0 ** 24 for j in range(d)])
    assert np.array_equal(u.astype(np.float64), want)
    assert u.min() >= 0.0 and u.max() < 1.0
    # streams of different workers, tensors and steps differ
    assert not np.array_equal(u, orc.uniform24(42, 4, 7, 11, d))
    assert not np.array_equal(u, orc.uniform24(42, 3, 8, 11, d))
    assert not np.array_equal(u, orc.uniform24(42, 3, 7, 12, d))


def test_uniform24_first_two_moments():
    u = orc.uniform24(7, 0, 0, 0, 200000).astype(np.float64)
    assert abs(u.mean() - 0.5) < 4 * np.sqrt(1 / 12 / u.size)
    assert abs(u.var() - 1 / 12) < 1e-3
