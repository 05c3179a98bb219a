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
  * draw, in two levels (an exponential race may be run group by group: the group whose total weight wins
    its race is the group of the overall winner with the right probability, and inside a group the members
    race with their own weights). The V elements are dealt into C = 256 classes in runs of 8:
    class(j) = floor(j / 8) mod 256.
      level 1: W_c = sum over the class of 2^(y_j), y_j = logit_j * log2(e) / tau; the class is
               argmax_c [ log2 W_c - log2(-log2 v_c) ] over the classes with W_c > 0, ties to the lowest c, with
               v_c the uniform of word c % 4 of the counter (2^31 + floor(c / 4), row, offset low, offset high);
      level 2: the token is argmax_j [ y_j - log2(-log2 u_j) ] over the elements j of that class, ties to the
               lowest j, with u_j the uniform of word j % 4 of the counter (floor(j / 4), row, offset low, offset high).
    (log2 W - log2(-log2 u) is the Gumbel-max form, in base 2, of minimising the exponential variate -log2(u)
    divided by the weight.) Every element is drawn with probability 2^(y_j) / sum_k 2^(y_k) = softmax(logits / tau)_j.
    Only 256 + V/256 uniforms per row decide the draw, so a kernel needs the generator for the winning class only.
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


N_CLASSES = 256
RUN = 8
CLASS_COUNTER_BASE = 1 << 31


def class_of(V: int):
    """class(j) for j = 0 .. V-1."""
    return (np.arange(V) // RUN) % N_CLASSES


def class_uniforms(rows: int, seed: int, offset: int = 0, row0: int = 0):
    """v [rows, 256] float64: the uniforms of level 1."""
    c = np.arange(N_CLASSES, dtype=np.uint64)
    r = (np.arange(rows, dtype=np.uint64) + np.uint64(row0))[:, None]
    words = philox4x32_10((np.uint64(CLASS_COUNTER_BASE) + (c >> np.uint64(2)))[None, :], r,
                          np.uint64(offset & 0xFFFFFFFF), np.uint64((offset >> 32) & 0xFFFFFFFF), seed & 0xFFFFFFFF,
                          (seed >> 32) & 0xFFFFFFFF)
    sel = (c & np.uint64(3)).astype(np.int64)[None, :]
    x = np.choose(np.broadcast_to(sel, words[0].shape), words)
    return ((x >> np.uint32(9)).astype(np.float64) + 0.5) * 2.0 ** -23


def sample(logits, temperature: float, seed: int, offset: int = 0):
    """logits [rows, V] float64 (already widened). Returns (tokens int64 [rows], keys1 [rows, 256], keys2 [rows, V],
    cls [V]): keys1 are the perturbed base-2 scores of the classes (-inf for a class without weight), keys2 those of the
    elements; the token is the argmax of keys2 over the class that is the argmax of keys1."""
    x = np.asarray(logits, np.float64)
    rows, V = x.shape
    y = x * (np.log2(np.e) / float(temperature))
    cls = class_of(V)
    u = uniforms(rows, V, seed, offset)
    v = class_uniforms(rows, seed, offset)
    with np.errstate(divide="ignore", invalid="ignore"):
        keys2 = y - np.log2(-np.log2(u))
        keys1 = np.full((rows, N_CLASSES), -np.inf)
        tokens = np.empty(rows, np.int64)
        for r in range(rows):
            ymax = y[r].max()
            if not np.isfinite(ymax):                      # no element with weight (or a +inf / NaN): nothing is drawn
                tokens[r] = -1
                continue
            W = np.bincount(cls, weights=np.exp2(y[r] - ymax), minlength=N_CLASSES)    # the class sums
            has = W > 0
            keys1[r, has] = (ymax + np.log2(W[has])) - np.log2(-np.log2(v[r, has]))
            c_star = int(keys1[r].argmax())
            inside = np.where(cls == c_star, keys2[r], -np.inf)
            tokens[r] = int(inside.argmax())
    return tokens, keys1, keys2, cls
