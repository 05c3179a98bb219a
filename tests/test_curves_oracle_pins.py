"""Pins of the learning-curve oracle (oracle/curves_oracle.py): a hand-worked case, the identity with the per-token
rewards of step 3 (computed by the C oracle, other code), and the degenerate cases. No GPU."""
import os

import numpy as np

from oracle import curves_oracle as Q
from oracle import ppo_oracle as O

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "rollout_curves_hand_case.txt")


def _golden():
    out = {}
    for line in open(GOLDEN):
        if line.strip() and not line.startswith("#"):
            k, v = line.split()
            out[k] = float(v)
    return out


def test_hand_case():
    kl = [[0.1, -0.2, 0.3], [0.5, 9.0, 9.0]]
    mask = [[1, 1, 1], [1, 0, 0]]
    o = Q.rollout_curves(kl, mask, [1.0, -1.0], 0.05)
    g = _golden()
    for k in ("rlhf_reward", "kl", "score"):
        assert abs(o[k] - g[k]) < 1e-15, k
    assert np.allclose(o["per_response_kl"], [0.2, 0.5], atol=1e-15)
    assert np.allclose(o["per_response_reward"], [0.99, -1.025], atol=1e-15)


def test_reward_curve_is_the_mean_of_the_summed_per_token_rewards():
    """Step 3 spreads R over the tokens (KL penalty on every token, score on the last one): summing its rewards over
    a response gives R back. The rewards come from the C oracle's kl_rewards, which shares no code with this one."""
    rng = np.random.default_rng(3)
    B, T, beta = 37, 53, 0.05
    L = rng.integers(1, T + 1, size=B).astype(np.int32)
    mask = (np.arange(T)[None] < L[:, None]).astype(np.uint8)
    lp, rlp = rng.normal(size=(B, T)), rng.normal(size=(B, T))
    scores = rng.normal(size=B)
    kl, rew = O.kl_rewards(lp, rlp, mask, L, scores, beta)
    o = Q.rollout_curves(kl, mask, scores, beta)
    assert abs(o["rlhf_reward"] - rew.sum(axis=1).mean()) < 1e-13
    assert np.allclose(o["per_response_reward"], rew.sum(axis=1), atol=1e-13)
    assert abs(o["kl"] - (mask * (lp - rlp)).sum(axis=1).mean()) < 1e-13
    # the mask is optional when the k1 terms are already zero behind the responses (as step 3 writes them)
    o2 = Q.rollout_curves(kl, None, scores, beta)
    assert all(abs(o[k] - o2[k]) < 1e-13 for k in ("rlhf_reward", "kl", "score"))


def test_policy_equal_to_reference_and_masked_garbage():
    rng = np.random.default_rng(4)
    B, T = 5, 7
    scores = rng.normal(size=B)
    o = Q.rollout_curves(np.zeros((B, T)), None, scores, 0.05)
    assert o["kl"] == 0.0 and o["rlhf_reward"] == o["score"] == scores.sum() / B
    kl = rng.normal(size=(B, T))
    mask = (rng.random((B, T)) < 0.5).astype(np.uint8)
    dirty = np.where(mask == 1, kl, 1e30)
    a, b = Q.rollout_curves(kl * mask, None, scores, 0.3), Q.rollout_curves(dirty, mask, scores, 0.3)
    assert abs(a["kl"] - b["kl"]) < 1e-13 and abs(a["rlhf_reward"] - b["rlhf_reward"]) < 1e-13
    # a response with no real token contributes its score and no KL
    z = Q.rollout_curves(kl, np.zeros((B, T), np.uint8), scores, 0.3)
    assert z["kl"] == 0.0 and z["rlhf_reward"] == z["score"]


def test_means_are_over_responses_not_tokens():
    o = Q.rollout_curves(np.ones((4, 10)), None, np.zeros(4), 1.0)
    assert o["kl"] == 10.0 and o["rlhf_reward"] == -10.0
