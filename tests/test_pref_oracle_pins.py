"""Pins of the preference-loss oracle (oracle/pref_oracle.py) to closed forms, finite differences and brute force:
section "Preliminaries" (RM loss and its alternative form, DPO loss, implicit reward). No GPU."""
import numpy as np
import pytest

from oracle import pref_oracle as R


def test_pairwise_closed_forms():
    o = R.pairwise_logistic_loss([0.3, 1.0 + np.log(3.0)], [0.3, 1.0])
    assert abs(o["per_pair"][0] - np.log(2.0)) < 1e-15                 # equal rewards: -log(1/2)
    assert abs(o["per_pair"][1] - np.log(4.0 / 3.0)) < 1e-15           # d = ln 3: sigma = 3/4
    assert abs(o["loss"] - 0.5 * (np.log(2.0) + np.log(4.0 / 3.0))) < 1e-15
    assert np.allclose(o["dr_c"], [-0.5 / 2, -0.25 / 2], atol=1e-15)   # -sigma(-d) / P
    assert np.allclose(o["dr_r"], -o["dr_c"], atol=0)
    assert o["accuracy"] == 0.5                                        # a tie is not a correct ranking


def test_pairwise_two_forms_of_the_paper_agree_and_reflection_identity():
    rng = np.random.default_rng(1)
    rc, rr = rng.normal(size=200) * 3, rng.normal(size=200) * 3
    o = R.pairwise_logistic_loss(rc, rr)
    sig = 1.0 / (1.0 + np.exp(-(rc - rr)))
    assert np.allclose(o["per_pair"], -np.log(sig), rtol=1e-12)                       # -log sigma(r_c - r_r)
    assert np.allclose(o["per_pair"], np.log(1.0 + np.exp(rr - rc)), rtol=1e-12)      # log(1 + e^(r_r - r_c))
    swapped = R.pairwise_logistic_loss(rr, rc)
    assert np.allclose(o["per_pair"] - swapped["per_pair"], -(rc - rr), atol=1e-12)   # l(d) - l(-d) = -d
    assert o["accuracy"] == np.mean(rc > rr)


def test_pairwise_extremes_do_not_overflow():
    o = R.pairwise_logistic_loss([800.0, -800.0], [0.0, 0.0])
    assert o["per_pair"][0] == 0.0 and o["per_pair"][1] == 800.0
    assert o["dr_c"][0] == 0.0 and abs(o["dr_c"][1] + 0.5) < 1e-15
    assert np.isfinite(o["loss"])


def test_pairwise_gradient_by_finite_differences():
    rng = np.random.default_rng(2)
    rc, rr = rng.normal(size=7), rng.normal(size=7)
    o = R.pairwise_logistic_loss(rc, rr)
    e = 1e-6
    for i in range(7):
        for arr, key in ((rc, "dr_c"), (rr, "dr_r")):
            a, b = arr.copy(), arr.copy()
            a[i] += e
            b[i] -= e
            up = R.pairwise_logistic_loss(a, rr)["loss"] if key == "dr_c" else R.pairwise_logistic_loss(rc, a)["loss"]
            dn = R.pairwise_logistic_loss(b, rr)["loss"] if key == "dr_c" else R.pairwise_logistic_loss(rc, b)["loss"]
            assert abs((up - dn) / (2 * e) - o[key][i]) < 1e-9


def test_dpo_policy_equal_to_reference_and_mask():
    rng = np.random.default_rng(3)
    P, T = 5, 9
    lp_c, lp_r = -rng.random((P, T)) * 4, -rng.random((P, T)) * 4
    mc = (np.arange(T)[None] >= rng.integers(0, T, (P, 1))).astype(np.uint8)
    mr = (np.arange(T)[None] >= rng.integers(0, T, (P, 1))).astype(np.uint8)
    o = R.dpo_loss(lp_c, lp_r, lp_c, lp_r, mc, mr, 0.05)
    assert np.all(o["reward_c"] == 0) and np.all(o["reward_r"] == 0)       # log(pi / pi_SFT) = 0
    assert abs(o["loss"] - np.log(2.0)) < 1e-15 and o["accuracy"] == 0.0
    assert np.allclose(o["dlp_c"], -0.05 * 0.5 / P * mc) and np.allclose(o["dlp_r"], 0.05 * 0.5 / P * mr)
    # tokens outside the mask do not matter
    lp2 = lp_c + (1 - mc) * rng.normal(size=(P, T))
    o2 = R.dpo_loss(lp2, lp_r, lp_c, lp_r, mc, mr, 0.05)
    assert o2["loss"] == o["loss"] and np.all(o2["dlp_c"] == o["dlp_c"])


def test_dpo_implicit_reward_by_brute_force_on_a_tiny_model():
    """Two-token completions over a 3-word vocabulary: pi(y|x) is a product of two table look-ups, so the
    implicit reward beta * log(pi / pi_SFT) and the loss can be written with plain probabilities."""
    rng = np.random.default_rng(4)
    beta = 0.05

    def table():
        t = rng.random((2, 3)) + 0.1
        return t / t.sum(axis=1, keepdims=True)          # step-wise distributions (context-free toy model)
    pol, ref = table(), table()
    yc, yr = [0, 2], [1, 1]
    prob = lambda tb, y: tb[0, y[0]] * tb[1, y[1]]
    h = beta * np.log(prob(pol, yc) / prob(ref, yc)) - beta * np.log(prob(pol, yr) / prob(ref, yr))
    want = -np.log(1.0 / (1.0 + np.exp(-h)))
    tok_lp = lambda tb, y: np.log([[tb[0, y[0]], tb[1, y[1]]]])
    ones = np.ones((1, 2), np.uint8)
    o = R.dpo_loss(tok_lp(pol, yc), tok_lp(pol, yr), tok_lp(ref, yc), tok_lp(ref, yr), ones, ones, beta)
    assert abs(o["loss"] - want) < 1e-14
    assert abs(o["reward_c"][0] - beta * np.log(prob(pol, yc) / prob(ref, yc))) < 1e-14
    assert o["accuracy"] == float(h > 0)


def test_dpo_gradient_by_finite_differences():
    rng = np.random.default_rng(5)
    P, T, beta = 3, 6, 0.5
    a = [-rng.random((P, T)) * 3 for _ in range(4)]
    mc = (rng.random((P, T)) < 0.7).astype(np.uint8)
    mr = (rng.random((P, T)) < 0.7).astype(np.uint8)
    o = R.dpo_loss(a[0], a[1], a[2], a[3], mc, mr, beta)
    e = 1e-6
    for which, key in ((0, "dlp_c"), (1, "dlp_r")):
        for i in range(P):
            for t in range(T):
                up = [x.copy() for x in a]
                dn = [x.copy() for x in a]
                up[which][i, t] += e
                dn[which][i, t] -= e
                fd = (R.dpo_loss(*up, mc, mr, beta)["loss"] - R.dpo_loss(*dn, mc, mr, beta)["loss"]) / (2 * e)
                assert abs(fd - o[key][i, t]) < 1e-9


def test_logprob_bwd_closed_forms_and_finite_differences(oracle):
    V, tau = 11, 0.7
    # uniform row: softmax = 1/V
    d = R.logprob_bwd(np.zeros((1, V)), [4], [2.0], tau)
    want = np.full(V, -2.0 / V / tau)
    want[4] += 2.0 / tau
    assert np.allclose(d[0], want, atol=1e-15)
    rng = np.random.default_rng(6)
    x = rng.normal(size=(3, V)).astype(np.float32)
    tok = np.array([0, 5, 10], np.int32)
    g = np.array([1.5, -0.25, 0.0])
    d = R.logprob_bwd(x.astype(np.float64), tok, g, tau)
    assert np.abs(d.sum(axis=1)).max() < 1e-15 and not d[2].any()
    # the log-prob itself comes from the C oracle (another code base); perturbations exact in fp32
    e = 2.0 ** -10
    for r in range(2):
        for j in range(V):
            up, dn = x.copy(), x.copy()
            up[r, j] += e
            dn[r, j] -= e
            lu, _, _ = oracle.logprob_entropy(up, tok, tau)
            ld, _, _ = oracle.logprob_entropy(dn, tok, tau)
            assert abs(g[r] * (lu[r] - ld[r]) / (up[r, j] - dn[r, j]).astype(np.float64) - d[r, j]) < 1e-5
