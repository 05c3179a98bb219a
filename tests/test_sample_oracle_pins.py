"""Pins of oracle/sample_oracle.py: known-answer vectors of Philox4x32-10 from its reference implementation's
test suite, the range and spacing of the uniforms, and the distribution of the draws. No GPU."""
import numpy as np

from oracle import sample_oracle as S


def test_philox_known_answers():
    """Counter / key / expected output triples published with the generator (Random123 known-answer tests)."""
    kat = [((0, 0, 0, 0), (0, 0), (0x6627e8d5, 0xe169c58d, 0xbc57ac4c, 0x9b00dbd8)),
           ((0xffffffff,) * 4, (0xffffffff, 0xffffffff), (0x408f276d, 0x41c83b0e, 0xa20bc7c6, 0x6d5451fd)),
           ((0x243f6a88, 0x85a308d3, 0x13198a2e, 0x03707344), (0xa4093822, 0x299f31d0),
            (0xd16cfe09, 0x94fdcceb, 0x5001e420, 0x24126ea1))]
    for ctr, key, want in kat:
        got = S.philox4x32_10(*(np.array([c], np.uint32) for c in ctr), key[0], key[1])
        assert tuple(int(g[0]) for g in got) == want, (ctr, [hex(int(g[0])) for g in got])


def test_counters_are_independent_streams():
    a = S.uniforms(3, 64, seed=7)
    assert len(np.unique(a)) > 180                      # no repeats to speak of among 192 draws
    assert not np.array_equal(a, S.uniforms(3, 64, seed=8))
    assert not np.array_equal(a, S.uniforms(3, 64, seed=7, offset=1))
    assert np.array_equal(a[1:], S.uniforms(2, 64, seed=7, row0=1))      # a row's stream depends on its index only


def test_uniform_range_and_grid():
    u = S.uniforms(64, 4096, seed=123)
    assert u.min() > 0 and u.max() < 1
    assert np.array_equal(u, u.astype(np.float32).astype(np.float64))     # fp32 numbers
    k = u * 2.0 ** 24
    assert np.array_equal(k, np.round(k)) and np.all(k.astype(np.int64) % 2 == 1)   # odd multiples of 2^-24
    assert abs(u.mean() - 0.5) < 3e-3 and abs(u.var() - 1 / 12) < 2e-3


def test_draws_follow_the_temperature_scaled_softmax():
    rng = np.random.default_rng(0)
    V, n, tau = 12, 40000, 0.7
    row = rng.normal(size=V) * 1.5
    tok, keys = S.sample(np.tile(row, (n, 1)), tau, seed=99)
    p = np.exp(row / tau - (row / tau).max())
    p /= p.sum()
    counts = np.bincount(tok, minlength=V)
    chi2 = ((counts - n * p) ** 2 / (n * p)).sum()
    assert chi2 < 40.0                                  # 11 degrees of freedom: P(chi2 > 40) ~ 4e-5
    assert np.array_equal(keys.argmax(axis=1), tok)


def test_ties_and_minus_infinity():
    x = np.zeros((1, 8))
    x[0, 3] = -np.inf
    tok, keys = S.sample(np.tile(x, (2000, 1)), 1.0, seed=5)
    assert 3 not in tok and len(np.unique(tok)) == 7
