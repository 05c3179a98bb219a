"""fp64 numpy oracle of temperature sampling fused into the log-prob pass.

TEST INFRASTRUCTURE, NOT PRODUCT CODE (same rule as ppo_oracle.py).

The paper samples responses at temperature 0.7 (Table "PPO hyperparameters") and needs the log-prob of every
sampled token under the same temperature-scaled distribution. This module defines the draw so that a GPU
kernel can be compared with it token by token:

  * random numbers: Philox4x32-10 (Salmon, Moraes, Dror, Shaw: "Parallel random numbers: as easy as 1, 2, 3",
    SC'11), a counter-based generator: key = the 64-bit seed, counter = (element index / 4, row, offset low,
    offset high), output word = element index % 4;
  * uniform: u = (floor(x / 2^9) + 1/2) * 2^-23 for a 32-bit word x, so u lies strictly inside (0, 1) and is an
    fp32 number;
  * draw: the token of row r is argmax_j [ y_j - log2(-log2 u_j) ] with y_j = logit_j * log2(e) / tau (the
    Gumbel-max rule in base 2; equivalently the index that minimises the exponential variate -log2(u_j)
    divided by the unnormalised probability 2^(y_j)); exact ties go to the lowest index.
"""
from __future__ import annotations

import numpy as np

_M0, _M1 = np.uint64(0xD2511F53), np.uint64(0xCD9E8D57)
_W0, _W1 = 0x9E3779B9, 0xBB67AE85
_MASK = np.uint64(0xFFFFFFFF)


def philox4x32_10(c0, c1, c2, c3, k0: int, k1: int):
    """Ten rounds of Philox-4x32 on arrays of counters (uint32 each); returns four uint32 arrays."""
    c = [np.asarray(x, dtype=np.uint64) & _MASK for x in np.broadcast_arrays(c0, c1, c2, c3)]
    k0, k1 = int(k0) & 0xFFFFFFFF, int(k1) & 0xFFFFFFFF
    for _ in range(10):
        p0 = _M0 * c[0]                      # 64-bit products of 32-bit values
        p1 = _M1 * c[2]
        hi0, lo0 = p0 >> np.uint64(32), p0 & _MASK
        hi1, lo1 = p1 >> np.uint64(32), p1 & _MASK
        c = [hi1 ^ c[1] ^ np.uint64(k0), lo1, hi0 ^ c[3] ^ np.uint64(k1), lo0]
        k0 = (k0 + _W0) & 0xFFFFFFFF
        k1 = (k1 + _W1) & 0xFFFFFFFF
    return tuple(x.astype(np.uint32) for x in c)


def uniforms(rows: int, V: int, seed: int, offset: int = 0, row0: int = 0):
    """u [rows, V] float64 (each value is exactly an fp32 number in (0, 1))."""
    j = np.arange(V, dtype=np.uint64)
    r = (np.arange(rows, dtype=np.uint64) + np.uint64(row0))[:, None]
    words = philox4x32_10((j >> np.uint64(2))[None, :], r, np.uint64(offset & 0xFFFFFFFF),
                          np.uint64((offset >> 32) & 0xFFFFFFFF), seed & 0xFFFFFFFF, (seed >> 32) & 0xFFFFFFFF)
    sel = (j & np.uint64(3)).astype(np.int64)[None, :]
    x = np.choose(np.broadcast_to(sel, words[0].shape), words)
    return ((x >> np.uint32(9)).astype(np.float64) + 0.5) * 2.0 ** -23


def sample(logits, temperature: float, seed: int, offset: int = 0):
    """logits [rows, V] float64 (already widened). Returns (tokens int64 [rows], keys [rows, V] float64): the
    perturbed base-2 scores whose argmax is the token."""
    x = np.asarray(logits, np.float64)
    y = x * (np.log2(np.e) / float(temperature))
    u = uniforms(x.shape[0], x.shape[1], seed, offset)
    with np.errstate(divide="ignore"):
        keys = y - np.log2(-np.log2(u))
    return keys.argmax(axis=1), keys
