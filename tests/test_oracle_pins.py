"""Pins for the fp64 CPU oracle: closed forms, brute force, library second opinions, hand cases
and finite differences.  None of these tests touches the CUDA path; each is chosen so that a
plausible slip in the oracle (dropped term, wrong sign or index, transposed operand, wrong
normaliser) fails at least one of them."""
import itertools
import math
import os

import numpy as np
import pytest
import torch

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _kv(name):
    out = {}
    for line in open(os.path.join(GOLDEN, name)):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        k, v = line.split()
        out[k] = float(v)
    return out


def _rows(name):
    return [np.array([float(x) for x in l.split()]) for l in open(os.path.join(GOLDEN, name))
            if l.strip() and not l.startswith("#")]


# ---------------------------------------------------------------- step 1: logprob + entropy
def test_uniform_row_gives_log_V(oracle):
    g = _kv("onehot_softmax_closed_form.txt")
    for V, key in ((1000, "ln_1000"), (50304, "ln_50304")):
        x = np.full((3, V), 1.25, np.float32)
        lp, H, lse = oracle.logprob_entropy(x, [0, V // 2, V - 1], 0.7)
        assert np.allclose(lp, -g[key], atol=1e-12)
        assert np.allclose(H, g[key], atol=1e-12)
        assert np.allclose(lse, 1.25 / np.float64(0.7) + g[key], atol=1e-12)


def test_onehot_closed_form(oracle):
    g = _kv("onehot_softmax_closed_form.txt")
    V = 1000
    x = np.zeros((2, V), np.float32)
    x[:, 417] = 3.0
    lp, H, _ = oracle.logprob_entropy(x, [417, 3], 0.7)
    assert abs(lp[0] - g["lp_hot"]) < 1e-12
    assert abs(lp[1] - g["lp_other"]) < 1e-12
    assert np.allclose(H, g["entropy"], atol=1e-12)


def test_shift_and_temperature_invariance(oracle):
    rng = np.random.default_rng(1)
    x = (np.round(rng.normal(0, 2, (5, 257)) * 4096) / 4096).astype(np.float32)   # multiples of 2^-12
    tok = rng.integers(0, 257, 5)
    lp, H, lse = oracle.logprob_entropy(x, tok, 0.5)
    x2 = (x.astype(np.float64) + 8.0).astype(np.float32)      # exact for such values
    assert np.array_equal((x2.astype(np.float64) - 8.0), x.astype(np.float64))
    lp2, H2, lse2 = oracle.logprob_entropy(x2, tok, 0.5)
    assert np.allclose(lp, lp2, atol=1e-12) and np.allclose(H, H2, atol=1e-12)
    assert np.allclose(lse2 - lse, 16.0, atol=1e-12)
    # (2x, tau=1) is the same distribution as (x, tau=0.5); doubling is exact in fp32
    lp3, H3, _ = oracle.logprob_entropy((2 * x).astype(np.float32), tok, 1.0)
    assert np.allclose(lp, lp3, atol=1e-12) and np.allclose(H, H3, atol=1e-12)


def test_bruteforce_tiny_vocab(oracle):
    rng = np.random.default_rng(2)
    for V in (1, 2, 3, 8):
        x = rng.normal(0, 3, (V, V)).astype(np.float32)
        lp, H, _ = oracle.logprob_entropy(x, np.arange(V), 0.7)
        # lp[r] is the log-prob of token r in row r; rebuild all probabilities of one row
        for r in range(V):
            lps, _, _ = oracle.logprob_entropy(np.repeat(x[r:r + 1], V, 0), np.arange(V), 0.7)
            p = np.exp(lps)
            assert abs(p.sum() - 1.0) < 1e-12
            assert abs(lps[r] - lp[r]) < 1e-15
            assert abs(H[r] - (-(p * lps).sum())) < 1e-12
            assert -1e-12 <= H[r] <= math.log(V) + 1e-12
            # relative odds follow the logits
            for a, b in itertools.combinations(range(V), 2):
                assert abs((lps[a] - lps[b]) - (float(x[r, a]) - float(x[r, b])) / np.float64(0.7)) < 1e-9


def test_library_log_softmax_second_opinion(oracle):
    rng = np.random.default_rng(3)
    x = rng.normal(0, 2, (7, 1000)).astype(np.float32)
    tok = rng.integers(0, 1000, 7)
    lp, H, lse = oracle.logprob_entropy(x, tok, 1.0)
    t = torch.from_numpy(x).double()
    ls = torch.log_softmax(t, -1)
    assert np.allclose(lp, ls[torch.arange(7), torch.from_numpy(tok)].numpy(), atol=1e-12)
    assert np.allclose(H, torch.distributions.Categorical(logits=t).entropy().numpy(), atol=1e-11)
    assert np.allclose(lse, torch.logsumexp(t, -1).numpy(), atol=1e-12)
    # temperature: library result on pre-divided float64 logits
    tau = float(np.float32(0.7))
    lp7, _, _ = oracle.logprob_entropy(x, tok, tau)
    ls7 = torch.log_softmax(t / tau, -1)
    assert np.allclose(lp7, ls7[torch.arange(7), torch.from_numpy(tok)].numpy(), atol=1e-12)


def test_bf16_widening_is_exact(oracle):
    t = torch.randn(4, 300, generator=torch.Generator().manual_seed(4)).mul(2).to(torch.bfloat16)
    bits = t.view(torch.int16).numpy().view(np.uint16)
    tok = [0, 17, 299, 150]
    lp_b, H_b, _ = oracle.logprob_entropy(bits, tok, 0.7)
    lp_f, H_f, _ = oracle.logprob_entropy(t.float().numpy(), tok, 0.7)
    assert np.array_equal(lp_b, lp_f) and np.array_equal(H_b, H_f)


def test_mask_neg_inf_and_bad_token(oracle):
    x = np.zeros((3, 16), np.float32)
    x[1, 5:] = -np.inf                       # probability mass only on 5 entries
    lp, H, _ = oracle.logprob_entropy(x, [0, 2, 99], 1.0, mask=[0, 1, 1])
    assert lp[0] == 0.0 and H[0] == 0.0
    assert abs(lp[1] + math.log(5)) < 1e-12 and abs(H[1] - math.log(5)) < 1e-12
    assert math.isnan(lp[2]) and math.isnan(H[2])


def test_masked_rows_are_not_read_and_change_nothing_downstream(oracle):
    """The chained path gives step 1 the mask of the EOS trick: rows with mask 0 output exactly 0 whatever they
    hold (NaN included, and no status for a bad token there), rows with mask 1 are untouched by the option, and the
    KL rewards built from either version are identical (step 3 multiplies by the same mask)."""
    rng = np.random.default_rng(12)
    x = rng.normal(0, 2, (6, 40)).astype(np.float32)
    tok = np.array([3, 7, 1, 39, 0, 11], np.int32)
    mask = np.array([1, 1, 0, 1, 0, 0], np.uint8)
    full = oracle.logprob_entropy(x, tok, 0.7)
    y = x.copy()
    y[mask == 0] = np.nan
    tok2 = tok.copy()
    tok2[2] = 1000                                    # outside the vocabulary, but on a row with mask 0
    part = oracle.logprob_entropy(y, tok2, 0.7, mask=mask)
    for a, b in zip(full, part):
        assert np.array_equal(a[mask == 1], b[mask == 1])
        assert not b[mask == 0].any()
    ref = full[0] - 0.01
    m2, L = mask.reshape(1, 6).copy(), np.array([6], np.int32)
    kl_a, rew_a = oracle.kl_rewards(full[0].reshape(1, 6), ref.reshape(1, 6), m2, L, np.array([0.5]), 0.05)
    kl_b, rew_b = oracle.kl_rewards(part[0].reshape(1, 6), (ref * mask).reshape(1, 6), m2, L, np.array([0.5]), 0.05)
    assert np.array_equal(kl_a, kl_b) and np.array_equal(rew_a, rew_b)


# ---------------------------------------------------------------- step 2: EOS trick
def test_truncate_hand_rows(oracle):
    E, P = 0, 1
    resp = np.array([[E, 5, 6, 7, 8],          # EOS first
                     [5, 6, E, 7, 8],          # EOS in the middle
                     [5, 6, 7, 8, E],          # EOS last
                     [5, 6, 7, 8, 9],          # no EOS
                     [5, E, 6, E, 7],          # EOS twice: first one counts
                     [P, 5, E, 6, 7]], np.int32)   # a literal PAD id before EOS is an ordinary token
    scores = np.array([1.5, -2.0, 0.25, 3.0, 0.5, 0.75])
    out, e, L, m, so = oracle.truncate_and_score(resp, E, P, scores, -1.0)
    assert out.tolist() == [[E, P, P, P, P], [5, 6, E, P, P], [5, 6, 7, 8, E], [5, 6, 7, 8, 9],
                            [5, E, P, P, P], [P, 5, E, P, P]]
    assert e.tolist() == [0, 2, 4, -1, 1, 2]
    assert L.tolist() == [1, 3, 5, 5, 2, 3]
    assert m.tolist() == [[1, 0, 0, 0, 0], [1, 1, 1, 0, 0], [1, 1, 1, 1, 1], [1, 1, 1, 1, 1],
                          [1, 1, 0, 0, 0], [1, 1, 1, 0, 0]]
    assert so.tolist() == [1.5, -2.0, 0.25, -1.0, 0.5, 0.75]     # replaced, not added


def test_truncate_invariants_and_idempotence(oracle):
    rng = np.random.default_rng(5)
    resp = rng.integers(0, 6, (64, 53)).astype(np.int32)
    resp[resp == 1] = 2
    scores = rng.normal(size=64)
    out, e, L, m, so = oracle.truncate_and_score(resp, 0, 1, scores, -1.0)
    assert ((1 <= L) & (L <= 53)).all() and (m.sum(1) == L).all()
    out2, e2, L2, m2, so2 = oracle.truncate_and_score(out, 0, 1, so, -1.0)
    assert np.array_equal(out, out2) and np.array_equal(e, e2) and np.array_equal(L, L2)
    assert np.array_equal(m, m2) and np.array_equal(so, so2)
    with pytest.raises(RuntimeError):
        oracle.truncate_and_score(resp, 3, 3, scores, -1.0)    # EOS must differ from [PAD]


# ---------------------------------------------------------------- step 3: KL rewards
def test_kl_rewards_hand_case_and_sums(oracle):
    lp = np.array([[-1.0, -2.0, -0.5, -3.0]])
    lr = np.array([[-1.5, -1.0, -0.5, -9.0]])
    m = np.array([[1, 1, 1, 0]], np.uint8)
    kl, rew = oracle.kl_rewards(lp, lr, m, [3], [4.5], 0.05)
    assert np.allclose(kl, [[0.5, -1.0, 0.0, 0.0]], atol=1e-15)
    assert np.allclose(rew, [[-0.025, 0.05, 4.5, 0.0]], atol=1e-15)
    rng = np.random.default_rng(6)
    B, T = 9, 13
    L = rng.integers(1, T + 1, B).astype(np.int32)
    m = (np.arange(T)[None] < L[:, None]).astype(np.uint8)
    lp, lr, s = rng.normal(size=(B, T)), rng.normal(size=(B, T)), rng.normal(size=B)
    kl, rew = oracle.kl_rewards(lp, lr, m, L, s, 0.05)
    assert np.allclose(rew.sum(1), s - 0.05 * kl.sum(1), atol=1e-12)
    kl0, rew0 = oracle.kl_rewards(lp, lp, m, L, s, 0.05)        # ref == policy
    assert not kl0.any()
    onehot = np.zeros((B, T))
    onehot[np.arange(B), L - 1] = s
    assert np.array_equal(rew0, onehot)


# ---------------------------------------------------------------- step 4: GAE
def test_gae_hand_case(oracle):
    rew, val, adv, ret = _rows("gae_hand_case.txt")
    A, R = oracle.gae(rew[None], val[None], [3], 1.0, 0.95)
    assert np.allclose(A[0], adv, atol=1e-15) and np.allclose(R[0], ret, atol=1e-15)


def test_gae_closed_forms(oracle):
    rng = np.random.default_rng(7)
    B, T = 6, 40
    L = np.array([1, 2, 17, 39, 40, 40], np.int32)
    r, v = rng.normal(size=(B, T)), rng.normal(size=(B, T))
    # lambda = gamma = 1: reward-to-go minus value
    A, R = oracle.gae(r, v, L, 1.0, 1.0)
    for b in range(B):
        rtg = np.cumsum(r[b, :L[b]][::-1])[::-1]
        assert np.allclose(A[b, :L[b]], rtg - v[b, :L[b]], atol=1e-12)
        assert np.allclose(R[b, :L[b]], rtg, atol=1e-12)
        assert not A[b, L[b]:].any() and not R[b, L[b]:].any()
    # lambda = 0: one-step TD residual
    g = 0.9
    A, _ = oracle.gae(r, v, L, g, 0.0)
    for b in range(B):
        vn = np.append(v[b, 1:L[b]], 0.0)
        assert np.allclose(A[b, :L[b]], r[b, :L[b]] + g * vn - v[b, :L[b]], atol=1e-12)
    # general: O(T^2) discounted sum of TD residuals
    lam = 0.95
    A, R = oracle.gae(r, v, L, g, lam)
    for b in range(B):
        vn = np.append(v[b, 1:L[b]], 0.0)
        d = r[b, :L[b]] + g * vn - v[b, :L[b]]
        for t in range(L[b]):
            k = np.arange(L[b] - t)
            assert abs(A[b, t] - ((g * lam) ** k * d[t:]).sum()) < 1e-11
        assert np.allclose(R[b, :L[b]], A[b, :L[b]] + v[b, :L[b]], atol=1e-15)
    # values beyond the sequence end are ignored
    v2 = v.copy()
    v2[np.arange(T)[None] >= L[:, None]] = 1e6
    A2, _ = oracle.gae(r, v2, L, g, lam)
    assert np.array_equal(A, A2)


# ---------------------------------------------------------------- step 5: whitening
def _moments_exact(values):
    """Mean and population variance of integer-valued data from the raw power sums, in exact rational arithmetic
    (one pass, var = E[x^2] - E[x]^2): structured unlike the oracle's two passes over centred values."""
    from fractions import Fraction
    xs = [Fraction(int(v)) for v in np.asarray(values).reshape(-1)]
    n = len(xs)
    s1, s2 = sum(xs), sum(v * v for v in xs)
    mean = s1 / n
    return mean, s2 / n - mean * mean


def test_whiten_closed_forms_and_properties(oracle):
    """Listing "whiten" and detail "Advantage whitening": population (not sample) variance, 1e-8 inside the square
    root, zero mean by default and the mean added back on request."""
    # two points 0 and 2: mean 1, population variance 1 (the sample variance would be 2)
    y, st = oracle.whiten(np.array([0.0, 2.0]), None, True, 1e-8)
    assert st.tolist() == [1.0, 1.0, 2.0]
    assert np.allclose(y, np.array([-1.0, 1.0]) / np.sqrt(1.0 + 1e-8), atol=1e-15)
    y, _ = oracle.whiten(np.array([0.0, 2.0]), None, False, 1e-8)
    assert np.allclose(y, 1.0 + np.array([-1.0, 1.0]) / np.sqrt(1.0 + 1e-8), atol=1e-15)
    # a constant array: variance 0, so the 1e-8 alone keeps the division finite and the result is 0 (or the mean)
    y, st = oracle.whiten(np.full(7, 4.0), None, True, 1e-8)
    assert st[1] == 0.0 and not y.any()
    y, _ = oracle.whiten(np.full(7, 4.0), None, False, 1e-8)
    assert np.array_equal(y, np.full(7, 4.0))
    # integer-valued data against exact rational moments
    rng = np.random.default_rng(8)
    x = rng.integers(-50, 50, (16, 53)).astype(np.float64)
    mean_q, var_q = _moments_exact(x)
    for sm in (True, False):
        y, st = oracle.whiten(x, None, sm, 1e-8)
        assert abs(st[0] - float(mean_q)) < 1e-13 and abs(st[1] - float(var_q)) < 1e-11 and st[2] == x.size
        want = (x - float(mean_q)) / np.sqrt(float(var_q) + 1e-8) + (0.0 if sm else float(mean_q))
        assert np.allclose(y, want, atol=1e-12)
        # properties: mean 0 (or the input's mean), variance var / (var + 1e-8)
        assert abs(y.mean() - (0.0 if sm else float(mean_q))) < 1e-12
        assert abs(((y - y.mean()) ** 2).mean() - float(var_q) / (float(var_q) + 1e-8)) < 1e-12
    # masked: statistics over mask==1 entries only, zeros elsewhere
    m = (rng.random((16, 53)) < 0.6).astype(np.uint8)
    sel = m.astype(bool)
    y, st = oracle.whiten(x, m, True, 1e-8)
    mq, vq = _moments_exact(x[sel])
    assert abs(st[0] - float(mq)) < 1e-13 and abs(st[1] - float(vq)) < 1e-11 and st[2] == sel.sum()
    assert np.allclose(y[sel], (x[sel] - float(mq)) / np.sqrt(float(vq) + 1e-8), atol=1e-12)
    assert not y[~sel].any()
    assert abs(y[sel].mean()) < 1e-12
    assert abs((y[sel] ** 2).mean() - st[1] / (st[1] + 1e-8)) < 1e-12
    # entries behind the mask do not matter
    x2 = x.copy()
    x2[~sel] = 1e9
    y2, st2 = oracle.whiten(x2, m, True, 1e-8)
    assert np.array_equal(y2, y) and np.array_equal(st2, st)
    # an affine map a*x + b with a < 0 flips the sign and nothing else (variance far above 1e-8)
    y3, _ = oracle.whiten(-3.0 * x + 7.0, m, True, 1e-8)
    assert np.allclose(y3, -y, atol=1e-7)
    y1, _ = oracle.whiten(np.array([2.5, 9.0]), np.array([1, 0], np.uint8), True, 1e-8)   # n = 1
    assert y1.tolist() == [0.0, 0.0]


# ---------------------------------------------------------------- step 6: losses + gradients
def _tiny_loss_inputs(seed=9, B=3, T=5, V=11):
    rng = np.random.default_rng(seed)
    logits = rng.normal(0, 2, (B, T, V)).astype(np.float32)
    tok = rng.integers(0, V, (B, T)).astype(np.int32)
    L = np.array([5, 3, 1])[:B]
    m = (np.arange(T)[None] < L[:, None]).astype(np.uint8)
    adv = rng.normal(size=(B, T))
    vo = rng.normal(size=(B, T))
    vn = vo + rng.normal(0, 0.3, (B, T))
    ret = rng.normal(size=(B, T))
    return logits, tok, m, adv, vn, vo, ret


def test_loss_ratio_one_and_value_unclipped(oracle):
    logits, tok, m, adv, vn, vo, ret = _tiny_loss_inputs()
    tau = 0.7
    B, T, V = logits.shape
    lp, H, _ = oracle.logprob_entropy(logits.reshape(-1, V), tok, tau)
    lp = lp.reshape(B, T)
    sel = m.astype(bool)
    n = sel.sum()
    o = oracle.loss_fwd_bwd(logits, tok, m, lp, adv, vo, vo, ret, tau, 0.2, 0.2, 0.1)
    ls = o["losses"]
    assert abs(ls[0] + adv[sel].mean()) < 1e-12                    # ratio = 1: pg_loss = -mean(A)
    assert abs(ls[1] - 0.5 * ((vo - ret)[sel] ** 2).mean()) < 1e-12  # v = v_old: plain half-MSE
    assert abs(ls[2] - (ls[0] + 0.1 * ls[1])) < 1e-15
    assert ls[3] == 0.0 and ls[4] == 0.0 and ls[5] == 0.0 and ls[7] == n
    assert abs(ls[6] - H.reshape(B, T)[sel].mean()) < 1e-12
    assert np.allclose(o["dlogprob"][sel], -adv[sel] / n, atol=1e-15)
    assert not o["dlogprob"][~sel].any() and not o["dvalues"][~sel].any()
    assert np.allclose(o["dvalues"][sel], 0.1 * (vo - ret)[sel] / n, atol=1e-15)
    assert np.allclose(o["new_logprob"][sel], lp[sel], atol=1e-15)
    dl = o["dlogits"].reshape(B, T, V)
    assert np.abs(dl.sum(-1)).max() < 1e-15                        # softmax gradient rows sum to 0
    assert not dl[~sel].any()
    # whitened advantages: pg_loss is 0 at ratio 1
    aw, _ = oracle.whiten(adv, m, True, 1e-8)
    o2 = oracle.loss_fwd_bwd(logits, tok, m, lp, aw, vo, vo, ret, tau, 0.2, 0.2, 0.1)
    assert abs(o2["losses"][0]) < 1e-12


def test_loss_clip_branches_by_hand(oracle):
    # one token, V = 2, tau = 1: p(token 0) = sigmoid(x0 - x1)
    def run(x0, lp_old, A, v, vo, ret, eps=0.2, epsv=0.2, c1=0.1):
        logits = np.array([[[x0, 0.0]]], np.float32)
        return oracle.loss_fwd_bwd(logits, [[0]], [[1]], [[lp_old]], [[A]], [[v]], [[vo]], [[ret]],
                                   1.0, eps, epsv, c1)
    lp_new = -math.log(2.0)                     # x0 = 0
    # rho = 1.5 > 1.2 with A > 0: clipped branch wins, loss = -A*1.2, no gradient
    o = run(0.0, lp_new - math.log(1.5), 2.0, 0.0, 0.0, 1.0)
    assert abs(o["losses"][0] + 2.0 * 1.2) < 1e-12 and o["losses"][4] == 1.0
    assert o["dlogprob"][0, 0] == 0.0 and not o["dlogits"].any()
    # rho = 1.5 with A < 0: unclipped branch (pessimistic) wins, gradient flows
    o = run(0.0, lp_new - math.log(1.5), -2.0, 0.0, 0.0, 1.0)
    assert abs(o["losses"][0] - 3.0) < 1e-12 and o["losses"][4] == 0.0
    assert abs(o["dlogprob"][0, 0] - 3.0) < 1e-12
    assert np.allclose(o["dlogits"][0], [3.0 * 0.5, -3.0 * 0.5], atol=1e-12)
    # rho = 0.5 < 0.8 with A < 0: clipped branch wins (-A*0.8 > -A*0.5)
    o = run(0.0, lp_new - math.log(0.5), -2.0, 0.0, 0.0, 1.0)
    assert abs(o["losses"][0] - 1.6) < 1e-12 and o["dlogprob"][0, 0] == 0.0
    # rho = 0.5 with A > 0: unclipped wins
    o = run(0.0, lp_new - math.log(0.5), 2.0, 0.0, 0.0, 1.0)
    assert abs(o["losses"][0] + 1.0) < 1e-12 and abs(o["dlogprob"][0, 0] + 1.0) < 1e-12
    assert abs(o["losses"][3] - 0.5 * math.log(0.5) ** 2) < 1e-12
    # value: v = 1.0, v_old = 0 -> v_c = 0.2; ret = 2: (1-2)^2 = 1 < (0.2-2)^2 = 3.24: clipped, no grad
    o = run(0.0, lp_new, 0.0, 1.0, 0.0, 2.0)
    assert abs(o["losses"][1] - 0.5 * 3.24) < 1e-12 and o["losses"][5] == 1.0 and o["dvalues"][0, 0] == 0.0
    # ret = 0: (1-0)^2 = 1 > 0.04: unclipped, grad = c1 * (v - ret)
    o = run(0.0, lp_new, 0.0, 1.0, 0.0, 0.0)
    assert abs(o["losses"][1] - 0.5) < 1e-12 and abs(o["dvalues"][0, 0] - 0.1) < 1e-15
    assert abs(o["losses"][2] - 0.05) < 1e-12
    # huge clip range: never clipped
    o = run(0.0, lp_new - math.log(1.5), 2.0, 0.0, 0.0, 1.0, eps=1e9)
    assert abs(o["dlogprob"][0, 0] + 3.0) < 1e-12


def test_loss_gradients_by_finite_differences(oracle):
    logits, tok, m, adv, vn, vo, ret = _tiny_loss_inputs(seed=10)
    tau, eps, epsv, c1 = 0.7, 0.2, 0.2, 0.1
    B, T, V = logits.shape
    lp, _, _ = oracle.logprob_entropy(logits.reshape(-1, V), tok, tau)
    rng = np.random.default_rng(11)
    olp = lp.reshape(B, T) + rng.normal(0, 0.15, (B, T))          # ratios on both sides of the clip
    base = oracle.loss_fwd_bwd(logits, tok, m, olp, adv, vn, vo, ret, tau, eps, epsv, c1)
    assert 0 < base["losses"][4] < 1 and 0 < base["losses"][5] < 1   # both branches exercised

    # the oracle takes fp32 logits; perturb in a float64 copy of the *function* instead:
    # use logits scaled so that +-h is exactly representable (h = 2^-10 on values rounded to 2^-12)
    lg = np.round(logits.astype(np.float64) * 4096) / 4096
    lg32 = lg.astype(np.float32)
    assert np.array_equal(lg32.astype(np.float64), lg)
    lp, _, _ = oracle.logprob_entropy(lg32.reshape(-1, V), tok, tau)
    olp = lp.reshape(B, T) + rng.normal(0, 0.15, (B, T))
    base = oracle.loss_fwd_bwd(lg32, tok, m, olp, adv, vn, vo, ret, tau, eps, epsv, c1)
    h = 2.0 ** -10

    def total(lgx, vnx):
        return oracle.loss_fwd_bwd(lgx, tok, m, olp, adv, vnx, vo, ret, tau, eps, epsv, c1,
                                   want_dlogits=False)["losses"][2]
    dl = base["dlogits"].reshape(B, T, V)
    worst = 0.0
    for b in range(B):
        for t in range(T):
            for j in range(V):
                p, q = lg32.copy(), lg32.copy()
                p[b, t, j] += h
                q[b, t, j] -= h
                fd = (total(p, vn) - total(q, vn)) / (2 * h)
                worst = max(worst, abs(fd - dl[b, t, j]))
    assert worst < 5e-7, worst        # O(h^2) truncation of a smooth function; kinks not straddled
    hv = 1e-6
    for b in range(B):
        for t in range(T):
            p, q = vn.copy(), vn.copy()
            p[b, t] += hv
            q[b, t] -= hv
            fd = (total(lg32, p) - total(lg32, q)) / (2 * hv)
            assert abs(fd - base["dvalues"][b, t]) < 1e-8
    # dlogits is consistent with dlogprob through the softmax Jacobian
    for b in range(B):
        for t in range(T):
            assert abs(dl[b, t, tok[b, t]] - base["dlogprob"][b, t] *
                       (1 - math.exp(base["new_logprob"][b, t])) / tau) < 1e-12 or not m[b, t]


def test_loss_selected_rows_match_full(oracle):
    logits, tok, m, adv, vn, vo, ret = _tiny_loss_inputs(seed=12)
    B, T, V = logits.shape
    olp = np.random.default_rng(13).normal(-2, 0.3, (B, T))
    full = oracle.loss_fwd_bwd(logits, tok, m, olp, adv, vn, vo, ret, 0.7, 0.2, 0.2, 0.1)
    sel = [14, 0, 7, 6]
    part = oracle.loss_fwd_bwd(logits, tok, m, olp, adv, vn, vo, ret, 0.7, 0.2, 0.2, 0.1, sel_rows=sel)
    assert np.array_equal(part["dlogits"], full["dlogits"][sel])
    assert np.array_equal(part["losses"], full["losses"])


# ---------------------------------------------------------------- fused LM head
def test_lmhead_matches_library_matmul(oracle):
    g = torch.Generator().manual_seed(14)
    M, K, V = 6, 64, 96
    H = torch.randn(M, K, generator=g).to(torch.bfloat16)
    W = (0.2 * torch.randn(K, V, generator=g)).to(torch.bfloat16)
    tok = torch.randint(0, V, (M,), generator=g).int()
    bits = lambda t: t.view(torch.int16).numpy().view(np.uint16)
    sel = [5, 0, 3]
    lp, Hh, lse = oracle.lmhead_logprob_entropy(bits(H), bits(W), tok.numpy(), 0.7, sel_rows=sel)
    z = (H.double() @ W.double()) / 0.7
    ls = torch.log_softmax(z, -1)
    assert np.allclose(lp, ls[sel, tok[sel].long()].numpy(), atol=1e-11)
    assert np.allclose(Hh, torch.distributions.Categorical(logits=z[sel]).entropy().numpy(), atol=1e-10)
    assert np.allclose(lse, torch.logsumexp(z[sel], -1).numpy(), atol=1e-11)
    # and it agrees with step 1 applied to the (exactly representable) fp32 logits of a case
    # whose products are exact: H and W small integers
    Hi = torch.randint(-3, 4, (M, K), generator=g).to(torch.bfloat16)
    Wi = torch.randint(-2, 3, (K, V), generator=g).to(torch.bfloat16)
    lp2, H2, _ = oracle.lmhead_logprob_entropy(bits(Hi), bits(Wi), tok.numpy(), 0.7)
    lg = (Hi.float() @ Wi.float()).numpy()
    lp3, H3, _ = oracle.logprob_entropy(lg, tok.numpy(), 0.7)
    assert np.allclose(lp2, lp3, atol=1e-12) and np.allclose(H2, H3, atol=1e-12)


# ---------------------------------------------------------------- defaults = the paper's table
def test_default_hyperparameters_match_paper_table():
    from paper_2403_17031_b200.synthetic import CONFIGS, PPOHyper
    g = _kv("ppo_hyperparameters.txt")
    h = PPOHyper()
    for k in ("kl_coef", "gamma", "lam", "cliprange", "cliprange_value", "vf_coef", "temperature",
              "no_eos_score", "whiten_eps"):
        assert getattr(h, k) == g[k], k
    assert h.eos_id == int(g["eos_id"]) and h.pad_id != h.eos_id
    assert CONFIGS[2].B == int(g["batch_size"]) and CONFIGS[1].T == int(g["response_length"])
