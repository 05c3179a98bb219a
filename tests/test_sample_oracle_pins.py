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


def test_classes_partition_the_row_in_runs_of_eight():
    for V in (1, 8, 9, 2048, 2049, 50304):
        cls = S.class_of(V)
        assert cls.shape == (V,) and cls.min() == 0 and cls.max() == min(255, (V - 1) // 8)
        assert np.array_equal(cls[:8 * 256], (np.arange(min(V, 2048)) // 8))          # first 2048: runs of 8 in order
        assert np.array_equal(cls, S.class_of(V + 4096)[:V])                           # a prefix property
        if V > 2048:
            assert np.array_equal(cls[2048:4096], cls[:min(V, 4096) - 2048])           # dealt round-robin
    sizes = np.bincount(S.class_of(50304), minlength=256)
    assert sizes.sum() == 50304 and sizes.max() - sizes.min() <= 8
    # the two streams of uniforms never share a counter: element counters stay below 2^29, class counters start at 2^31
    assert S.CLASS_COUNTER_BASE > (2 ** 31 - 1) // 4
    assert not np.array_equal(S.class_uniforms(2, seed=7)[:, :64], S.uniforms(2, 64, seed=7))


def _chi2(counts, expected, min_expected=8.0):
    """Pearson statistic with the cells of small expectation pooled; returns (statistic, degrees of freedom)."""
    small = expected < min_expected
    c = np.append(counts[~small], counts[small].sum())
    e = np.append(expected[~small], expected[small].sum())
    keep = e > 0
    return ((c[keep] - e[keep]) ** 2 / e[keep]).sum(), int(keep.sum()) - 1


def test_draws_follow_the_temperature_scaled_softmax():
    """Both levels at work (V = 600: 75 classes of 8): the token frequencies follow softmax(logits / tau), and so do
    the two factors: the class frequencies follow the class weights and, inside a class, the element weights."""
    rng = np.random.default_rng(0)
    V, n, tau = 600, 60000, 0.7
    row = rng.normal(size=V) * 1.2
    tok, keys1, keys2, cls = S.sample(np.tile(row, (n, 1)), tau, seed=99)
    p = np.exp(row / tau - (row / tau).max())
    p /= p.sum()
    stat, dof = _chi2(np.bincount(tok, minlength=V).astype(float), n * p)
    assert dof > 200 and stat < dof + 5.0 * np.sqrt(2.0 * dof), (stat, dof)      # mean dof, sd sqrt(2 dof)
    pc = np.bincount(cls, weights=p, minlength=256)
    stat, dof = _chi2(np.bincount(cls[tok], minlength=256).astype(float), n * pc)
    assert dof >= 60 and stat < dof + 5.0 * np.sqrt(2.0 * dof), (stat, dof)
    c_big = int(pc.argmax())                                 # inside the heaviest class
    members = np.flatnonzero(cls == c_big)
    hits = tok[cls[tok] == c_big]
    stat, dof = _chi2(np.array([(hits == j).sum() for j in members], float), len(hits) * p[members] / p[members].sum())
    assert stat < dof + 5.0 * np.sqrt(2.0 * dof) + 5, (stat, dof)
    # the returned scores reproduce the decision
    assert np.array_equal(keys1.argmax(axis=1), cls[tok])
    assert np.array_equal(np.where(cls[None, :] == cls[tok][:, None], keys2, -np.inf).argmax(axis=1), tok)


def test_one_class_reduces_to_the_plain_gumbel_max():
    """V <= 8: every element is in class 0, level 1 has nothing to decide and the draw is the Gumbel-max rule over
    the element uniforms, evaluated here with library routines only."""
    rng = np.random.default_rng(2)
    x = rng.normal(size=(500, 8)) * 2
    tok, keys1, _, cls = S.sample(x, 0.7, seed=31, offset=4)
    assert not cls.any() and np.isfinite(keys1[:, 0]).all() and np.isinf(keys1[:, 1:]).all()
    u = S.uniforms(500, 8, seed=31, offset=4)
    gumbel = -np.log(-np.log(u))                              # natural-log form of the same rule
    assert np.array_equal((x / 0.7 + gumbel).argmax(axis=1), tok)


def test_level_one_is_a_race_between_class_weights():
    """Two classes with one element each (V = 16, everything else -inf): the token is decided by level 1 alone, with
    the class uniforms: class 0 wins iff -log2(v_0) / w_0 < -log2(v_1) / w_1."""
    x = np.full((3000, 16), -np.inf)
    x[:, 2], x[:, 11] = 0.3, 1.1
    tok, _, _, _ = S.sample(x, 1.0, seed=17)
    v = S.class_uniforms(3000, seed=17)
    w0, w1 = np.exp(0.3), np.exp(1.1)
    want = np.where(-np.log(v[:, 0]) / w0 < -np.log(v[:, 1]) / w1, 2, 11)
    assert np.array_equal(tok, want)
    assert abs((tok == 11).mean() - w1 / (w0 + w1)) < 0.03


def test_ties_and_minus_infinity():
    x = np.zeros((1, 8))
    x[0, 3] = -np.inf
    tok, _, _, _ = S.sample(np.tile(x, (2000, 1)), 1.0, seed=5)
    assert 3 not in tok and len(np.unique(tok)) == 7
    # a class without weight never wins; a row without any weight draws nothing
    x = np.full((400, 64), -np.inf)
    x[:, 40:48] = 0.0
    tok, keys1, _, cls = S.sample(x, 1.0, seed=6)
    assert (cls[tok] == 5).all() and np.isinf(keys1[:, :5]).all()
    tok, _, _, _ = S.sample(np.full((2, 24), -np.inf), 1.0, seed=6)
    assert (tok == -1).all()
