"""ctypes/numpy front end of the fp64 CPU oracle (ppo_oracle.c).

TEST INFRASTRUCTURE, NOT PRODUCT CODE: only tests/, the smoke check and the benchmark's
CPU-baseline leg import this module; the CUDA library and its Python binding never do, and
this module imports nothing from them.  All floating-point arrays are float64; logits are
passed in their storage type (float32, or bfloat16 bit patterns as uint16) and widened exactly
inside the C code.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "ppo_oracle.c")
_LIB = os.path.join(_HERE, "libppo_oracle.so")

F32, BF16 = 0, 1


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (OpenMP over rows)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11", "-Wall",
                               "-o", _LIB, _SRC, "-lm"])
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        build()
        _lib = C.CDLL(_LIB)
        _lib.oracle_num_threads.restype = C.c_int
    return _lib


def num_threads() -> int:
    return int(lib().oracle_num_threads())


def set_num_threads(n: int) -> None:
    lib().oracle_set_num_threads(C.c_int(n))


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _f64(a) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a, dtype=np.float64))


def _i32(a) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a, dtype=np.int32))


def _u8(a) -> Optional[np.ndarray]:
    return None if a is None else np.ascontiguousarray(np.asarray(a, dtype=np.uint8))


def _logits(a: np.ndarray):
    """float32 -> (array, F32); uint16 (bf16 bit patterns) -> (array, BF16)."""
    a = np.ascontiguousarray(a)
    if a.dtype == np.float32:
        return a, F32
    if a.dtype == np.uint16:
        return a, BF16
    raise TypeError("logits must be float32 or uint16 (bf16 bits), got %s" % a.dtype)


def _check(rc: int, name: str):
    if rc != 0:
        raise RuntimeError("%s failed with status %d" % (name, rc))


def logprob_entropy(logits: np.ndarray, tokens, temperature: float, mask=None):
    """logits [rows, V]; returns (logprob, entropy, lse), each float64 [rows]."""
    lg, dt = _logits(logits)
    rows, V = lg.shape
    tok = _i32(tokens).reshape(-1)
    m = _u8(mask)
    lp, H, L = (np.empty(rows, np.float64) for _ in range(3))
    rc = lib().oracle_logprob_entropy(_p(lg), C.c_int(dt), C.c_int64(rows), C.c_int64(V), C.c_int64(V),
                                      _p(tok), _p(m), C.c_double(float(temperature)), _p(lp), _p(H), _p(L))
    _check(rc, "oracle_logprob_entropy")
    return lp, H, L


def truncate_and_score(responses, eos_id: int, pad_id: int, scores, no_eos_score: float):
    r = _i32(responses)
    B, T = r.shape
    s = _f64(scores)
    out = np.empty((B, T), np.int32)
    e = np.empty(B, np.int32)
    L = np.empty(B, np.int32)
    m = np.empty((B, T), np.uint8)
    so = np.empty(B, np.float64)
    rc = lib().oracle_truncate_and_score(_p(r), C.c_int32(B), C.c_int32(T), C.c_int32(eos_id),
                                         C.c_int32(pad_id), _p(s), C.c_double(float(no_eos_score)),
                                         _p(out), _p(e), _p(L), _p(m), _p(so))
    _check(rc, "oracle_truncate_and_score")
    return out, e, L, m, so


def kl_rewards(logprob, ref_logprob, mask, seq_len, scores, kl_coef: float):
    lp, lr = _f64(logprob), _f64(ref_logprob)
    B, T = lp.shape
    m, L, s = _u8(mask), _i32(seq_len), _f64(scores)
    kl = np.empty((B, T), np.float64)
    rew = np.empty((B, T), np.float64)
    rc = lib().oracle_kl_rewards(_p(lp), _p(lr), _p(m), _p(L), _p(s), C.c_int32(B), C.c_int32(T),
                                 C.c_double(float(kl_coef)), _p(kl), _p(rew))
    _check(rc, "oracle_kl_rewards")
    return kl, rew


def gae(rewards, values, seq_len, gamma: float, lam: float):
    r, v = _f64(rewards), _f64(values)
    B, T = r.shape
    L = _i32(seq_len)
    A = np.empty((B, T), np.float64)
    R = np.empty((B, T), np.float64)
    rc = lib().oracle_gae(_p(r), _p(v), _p(L), C.c_int32(B), C.c_int32(T), C.c_double(float(gamma)),
                          C.c_double(float(lam)), _p(A), _p(R))
    _check(rc, "oracle_gae")
    return A, R


def whiten(x, mask=None, shift_mean: bool = True, eps: float = 1e-8):
    xx = _f64(x)
    m = _u8(mask)
    out = np.empty_like(xx)
    st = np.empty(3, np.float64)
    rc = lib().oracle_whiten(_p(xx), _p(m), C.c_int64(xx.size), C.c_int(1 if shift_mean else 0),
                             C.c_double(float(eps)), _p(out), _p(st))
    _check(rc, "oracle_whiten")
    return out, st


LOSS_NAMES = ("pg_loss", "vf_loss", "loss", "approx_kl", "pg_clipfrac", "vf_clipfrac", "entropy", "n")


def loss_fwd_bwd(logits: np.ndarray, tokens, mask, old_logprob, advantages, values_new, values_old,
                 returns, temperature: float, cliprange: float, cliprange_value: float, vf_coef: float,
                 want_dlogits: bool = True, sel_rows: Optional[Sequence[int]] = None):
    """logits [B,T,V]. Returns dict with losses[8], dlogits ([B*T,V] or [len(sel_rows),V] or
    None), dvalues, new_logprob, entropy, dlogprob (all float64)."""
    lg, dt = _logits(logits)
    B, T, V = lg.shape
    rows = B * T
    tok, m = _i32(tokens), _u8(mask)
    olp, adv, vn, vo, ret = (_f64(a) for a in (old_logprob, advantages, values_new, values_old, returns))
    losses = np.empty(8, np.float64)
    sel = None
    dl = None
    if want_dlogits:
        if sel_rows is not None:
            sel = np.ascontiguousarray(np.asarray(sel_rows, dtype=np.int64))
            dl = np.empty((sel.size, V), np.float64)
        else:
            dl = np.empty((rows, V), np.float64)
    dv, nlp, ent, dlp = (np.empty((B, T), np.float64) for _ in range(4))
    rc = lib().oracle_loss_fwd_bwd(_p(lg), C.c_int(dt), C.c_int32(B), C.c_int32(T), C.c_int64(V), _p(tok),
                                   _p(m), _p(olp), _p(adv), _p(vn), _p(vo), _p(ret),
                                   C.c_double(float(temperature)), C.c_double(float(cliprange)),
                                   C.c_double(float(cliprange_value)), C.c_double(float(vf_coef)),
                                   _p(losses), _p(dl), _p(sel), C.c_int64(0 if sel is None else sel.size),
                                   _p(dv), _p(nlp), _p(ent), _p(dlp))
    _check(rc, "oracle_loss_fwd_bwd")
    return {"losses": losses, "dlogits": dl, "dvalues": dv, "new_logprob": nlp, "entropy": ent,
            "dlogprob": dlp}


def lmhead_logprob_entropy(H: np.ndarray, W: np.ndarray, tokens, temperature: float,
                           sel_rows: Optional[Sequence[int]] = None):
    """H [M,K], W [K,V] as uint16 bf16 bit patterns. Returns (logprob, entropy, lse) float64 for
    the rows in sel_rows (all rows when None)."""
    Hh = np.ascontiguousarray(H)
    Ww = np.ascontiguousarray(W)
    assert Hh.dtype == np.uint16 and Ww.dtype == np.uint16
    M, K = Hh.shape
    K2, V = Ww.shape
    assert K == K2
    tok = _i32(tokens).reshape(-1)
    sel = None if sel_rows is None else np.ascontiguousarray(np.asarray(sel_rows, dtype=np.int64))
    n = M if sel is None else sel.size
    lp, H_, L = (np.empty(n, np.float64) for _ in range(3))
    rc = lib().oracle_lmhead_logprob_entropy(_p(Hh), _p(Ww), C.c_int64(M), C.c_int64(K), C.c_int64(V), _p(tok),
                                             _p(sel), C.c_int64(n), C.c_double(float(temperature)),
                                             _p(lp), _p(H_), _p(L))
    _check(rc, "oracle_lmhead_logprob_entropy")
    return lp, H_, L
