"""fp64 numpy oracle of the three statistics the paper plots for a PPO run.

TEST INFRASTRUCTURE, NOT PRODUCT CODE (same rule as ppo_oracle.py: only tests/, the smoke check and
the benchmark's CPU legs import it; it imports nothing from the CUDA package).

The caption of the paper's figure of PPO learning curves names them:
  rlhf_reward   the RLHF reward R(x, y) of Eq. (RL), section "Preliminaries", step 3:
                R = r(x, y) - beta * KL, with the KL of one response estimated by the sum over its
                real tokens of the per-token k1 terms (log pi - log pi_SFT at the sampled token),
                averaged over the responses of the batch
  kl            per response, the per-token KL terms between the RL policy and the SFT policy are
                summed; the curve is the mean of those sums over the responses (caption of the figure
                of PPO learning curves)
  score         the scores obtained from the reward model, averaged over the responses (here the
                score array that is passed in; the PPO loop passes the scores after the EOS trick)
Plain definitions: one loop over responses, one over tokens.
"""
from __future__ import annotations

import numpy as np


def rollout_curves(kl, mask, scores, kl_coef):
    """kl [B,T] per-token k1 terms, mask [B,T] (1 = real token) or None, scores [B].
    Returns dict(rlhf_reward, kl, score, per_response_kl [B], per_response_reward [B])."""
    kl = np.asarray(kl, dtype=np.float64)
    B, T = kl.shape
    scores = np.asarray(scores, dtype=np.float64).reshape(B)
    per_kl = np.zeros(B, np.float64)
    per_R = np.zeros(B, np.float64)
    for b in range(B):
        s = 0.0
        for t in range(T):
            if mask is None or mask[b][t]:
                s += float(kl[b, t])
        per_kl[b] = s
        per_R[b] = scores[b] - float(kl_coef) * s
    return {"rlhf_reward": float(per_R.sum() / B), "kl": float(per_kl.sum() / B), "score": float(scores.sum() / B),
            "per_response_kl": per_kl, "per_response_reward": per_R}
