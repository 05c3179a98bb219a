"""fp64 numpy oracle of the preference losses on sequence log-probabilities.

TEST INFRASTRUCTURE, NOT PRODUCT CODE (same rule as ppo_oracle.py: only tests/, the smoke check and
the benchmark's CPU legs import it; it imports nothing from the CUDA package).

What it defines, each as the paper's formula written out:
  pairwise_logistic_loss   section "Preliminaries", step 2: L_R = -E[log sigma(r_c - r_r)]
                           (= E[log(1 + e^(r_r - r_c))], the paper's alternative form)
  sequence_logprob         log pi(y | x) = sum over the response tokens of the token log-probs
  dpo_loss                 section "Preliminaries", "RL-free approaches": the DPO loss, and the
                           implicit reward r(x, y) = beta * log(pi(y|x) / pi_SFT(y|x))
  logprob_bwd              the chain rule from a gradient on token log-probs back to the logits:
                           d lp_tok / d logit_j = (1[j = tok] - softmax(logits / tau)_j) / tau
All means are over the pairs of the batch passed in; gradients are those of that mean.
"""
from __future__ import annotations

import numpy as np


def _f64(a):
    return np.ascontiguousarray(np.asarray(a, dtype=np.float64))


def pairwise_logistic_loss(r_c, r_r):
    """Rewards of the chosen and the rejected completion, [P] each.
    Returns dict(loss, accuracy, per_pair [P], dr_c [P], dr_r [P])."""
    r_c, r_r = _f64(r_c), _f64(r_r)
    P = r_c.size
    d = r_c - r_r
    per = np.logaddexp(0.0, -d)                     # log(1 + e^(-d)) = -log sigma(d)
    s = np.exp(-np.logaddexp(0.0, d))               # sigma(-d) = 1 / (1 + e^d)
    return {"loss": per.mean() if P else 0.0, "accuracy": float((d > 0).mean()) if P else 0.0, "per_pair": per,
            "dr_c": -s / P, "dr_r": s / P}


def sequence_logprob(logprob, mask):
    """[P,T] token log-probs and the 0/1 mask of the response tokens -> [P] sums."""
    return (_f64(logprob) * (np.asarray(mask) != 0)).sum(axis=1)


def dpo_loss(lp_c, lp_r, ref_c, ref_r, mask_c, mask_r, beta):
    """Token log-probs [P,T] of the chosen / rejected completions under the policy (lp_*) and under the
    frozen SFT reference (ref_*), masks of the response tokens, beta.
    Returns dict(loss, accuracy, reward_c [P], reward_r [P] (implicit rewards), dlp_c, dlp_r [P,T]
    (gradient of the mean loss w.r.t. the policy's token log-probs))."""
    beta = float(beta)
    reward_c = beta * (sequence_logprob(lp_c, mask_c) - sequence_logprob(ref_c, mask_c))
    reward_r = beta * (sequence_logprob(lp_r, mask_r) - sequence_logprob(ref_r, mask_r))
    o = pairwise_logistic_loss(reward_c, reward_r)
    mc, mr = (np.asarray(mask_c) != 0).astype(np.float64), (np.asarray(mask_r) != 0).astype(np.float64)
    return {"loss": o["loss"], "accuracy": o["accuracy"], "reward_c": reward_c, "reward_r": reward_r,
            "dlp_c": beta * o["dr_c"][:, None] * mc, "dlp_r": beta * o["dr_r"][:, None] * mr}


def logprob_bwd(logits, tokens, g, temperature):
    """logits [n,V] (already widened to float64), tokens [n], upstream gradient g [n] on the token
    log-probs. Returns dlogits [n,V] = g * (onehot(tok) - softmax(logits / tau)) / tau."""
    x = _f64(logits) / float(temperature)
    x = x - x.max(axis=1, keepdims=True)
    p = np.exp(x)
    p /= p.sum(axis=1, keepdims=True)
    d = -p
    d[np.arange(d.shape[0]), np.asarray(tokens, dtype=np.int64)] += 1.0
    return d * (_f64(g)[:, None] / float(temperature))
