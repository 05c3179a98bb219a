"""fp64 numpy oracle of the LM-head backward (the step after the loss at log-prob level, config 4).

TEST INFRASTRUCTURE, NOT PRODUCT CODE (same rule as ppo_oracle.py).

With logits = H W, z = logits / tau and lp_r = z[r, tok_r] - logsumexp(z[r, :]) (the forward definition,
section "PPO Training" + Table "PPO hyperparameters": temperature), a gradient g_r on each lp_r gives
    D  = g[:, None] * (onehot(tok) - softmax(z)) / tau          (chain rule through log-softmax)
    dH = D W^T,   dW = H^T D                                     (chain rule through the product)
Everything is written out densely; use it on shapes that fit (a few thousand rows).
"""
from __future__ import annotations

import numpy as np


def bf16_to_f64(a_u16: np.ndarray) -> np.ndarray:
    """bf16 bit patterns (uint16) -> float64, exactly."""
    return (np.ascontiguousarray(a_u16).astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def lmhead_bwd(H, W, tokens, g, temperature, mask=None):
    """H [M,K], W [K,V] float64 (already widened), tokens [M], g [M] (0 where mask == 0 is enforced here).
    Returns dict(D [M,V], dH [M,K], dW [K,V], dH_abs, dW_abs) where the *_abs arrays are the same
    contractions over absolute values (the scale of the rounding error of a low-precision D)."""
    H, W = np.asarray(H, np.float64), np.asarray(W, np.float64)
    tau = float(temperature)
    g = np.asarray(g, np.float64).copy()
    if mask is not None:
        g[np.asarray(mask) == 0] = 0.0
    z = (H @ W) / tau
    z -= z.max(axis=1, keepdims=True)
    p = np.exp(z)
    p /= p.sum(axis=1, keepdims=True)
    D = -p
    D[np.arange(D.shape[0]), np.asarray(tokens, np.int64)] += 1.0
    D *= (g / tau)[:, None]
    return {"D": D, "dH": D @ W.T, "dW": H.T @ D, "dH_abs": np.abs(D) @ np.abs(W).T,
            "dW_abs": np.abs(H).T @ np.abs(D)}
