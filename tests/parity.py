"""Helpers of the GPU-vs-oracle parity tests: exact host copies of device tensors, the
tolerances, and the oracle's run of the whole chain."""
from __future__ import annotations

import numpy as np
import torch

# Tolerances (absolute unless noted). Integer outputs are compared bit-exactly.
TOL_LOGPROB = 1e-4        # log-probs, entropy, KL, losses
TOL_REL = 1e-5            # rewards, advantages, returns, whitened advantages: |d| / max(|oracle|, 1)
TOL_GRAD_F32 = 1e-4       # n * gradient, fp32 outputs
BF16_REL = 2.0 ** -8      # n * gradient, bf16 outputs: one bf16 rounding (+ BF16_ABS)
BF16_ABS = 1e-6
KINK = 1e-4               # |rho - (1 +- eps)| below this: either clip branch is accepted


def host_logits(t: torch.Tensor) -> np.ndarray:
    """Device logits -> numpy in their storage type (bf16 as uint16 bit patterns)."""
    t = t.detach().cpu().contiguous()
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view(np.uint16)
    return t.numpy()


def npy(t: torch.Tensor) -> np.ndarray:
    return t.detach().cpu().numpy()


def f32(a) -> np.ndarray:
    """Round an oracle (float64) array to the fp32 values handed to the next GPU stage."""
    return np.asarray(a, dtype=np.float64).astype(np.float32)


def dev(a: np.ndarray, device="cuda") -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(a)).to(device)


def assert_abs(got, want, tol, what):
    got, want = np.asarray(got, np.float64), np.asarray(want, np.float64)
    assert got.shape == want.shape, (what, got.shape, want.shape)
    assert np.isfinite(got).all(), what + ": non-finite output"
    err = np.abs(got - want).max() if got.size else 0.0
    assert err <= tol, "%s: max |d| = %.3e > %.1e" % (what, err, tol)
    return err


def assert_rel(got, want, tol, what):
    got, want = np.asarray(got, np.float64), np.asarray(want, np.float64)
    assert got.shape == want.shape, (what, got.shape, want.shape)
    assert np.isfinite(got).all(), what + ": non-finite output"
    err = (np.abs(got - want) / np.maximum(np.abs(want), 1.0)).max() if got.size else 0.0
    assert err <= tol, "%s: max rel d = %.3e > %.1e" % (what, err, tol)
    return err


def assert_grad(got_scaled, want_scaled, bf16: bool, what):
    """Compare n*gradient arrays."""
    got, want = np.asarray(got_scaled, np.float64), np.asarray(want_scaled, np.float64)
    assert got.shape == want.shape, (what, got.shape, want.shape)
    assert np.isfinite(got).all(), what + ": non-finite output"
    bound = (BF16_REL * np.abs(want) + BF16_ABS) if bf16 else np.full_like(want, TOL_GRAD_F32)
    bad = np.abs(got - want) > bound
    assert not bad.any(), "%s: %d entries off, worst |d| = %.3e" % (what, int(bad.sum()),
                                                                   np.abs(got - want)[bad].max())


def oracle_chain(O, batch, h, old_logprob=None, loss_logits=None, sel_rows=None, want_dlogits=True,
                 step1_mask=True):
    """The whole path on the oracle, each stage fed the previous stage's float64 results rounded
    to fp32 (the precision in which the GPU stages exchange data). step1_mask: step 1 is given the
    mask of the EOS trick (padding rows output 0, as in the chained GPU path); False computes every row
    (what the stand-alone log-prob call without a mask returns)."""
    pl = host_logits(batch["policy_logits"])
    rl = host_logits(batch["ref_logits"])
    B, T, V = pl.shape
    resp = npy(batch["responses"])
    tau = np.float32(h.temperature)
    r = {}
    r["responses_out"], r["eos_index"], r["seq_len"], r["mask"], r["scores_out"] = O.truncate_and_score(
        resp, h.eos_id, h.pad_id, npy(batch["scores"]), np.float32(h.no_eos_score))
    m1 = r["mask"].reshape(-1) if step1_mask else None
    lp, ent, _ = O.logprob_entropy(pl.reshape(-1, V), resp, tau, mask=m1)
    rlp, _, _ = O.logprob_entropy(rl.reshape(-1, V), resp, tau, mask=m1)
    r["logprob"], r["entropy"], r["ref_logprob"] = lp.reshape(B, T), ent.reshape(B, T), rlp.reshape(B, T)
    r["kl"], r["rewards"] = O.kl_rewards(f32(r["logprob"]), f32(r["ref_logprob"]), r["mask"], r["seq_len"],
                                         f32(r["scores_out"]), np.float32(h.kl_coef))
    if getattr(h, "whiten_rewards", 0):   # detail "(Optional) Reward whitening": before GAE, mean kept
        r["rewards"], _ = O.whiten(f32(r["rewards"]), r["mask"], False, np.float32(h.whiten_eps))
    r["advantages"], r["returns"] = O.gae(f32(r["rewards"]), npy(batch["values"]), r["seq_len"],
                                          np.float32(h.gamma), np.float32(h.lam))
    r["advantages_whitened"], r["whiten_stats"] = O.whiten(f32(r["advantages"]), r["mask"], True,
                                                           np.float32(h.whiten_eps))
    if old_logprob is None:
        old_logprob = f32(r["logprob"]) + npy(batch["old_logprob_noise"])
    r["old_logprob"] = np.asarray(old_logprob, np.float32)
    ll = pl if loss_logits is None else host_logits(loss_logits)
    r["loss"] = O.loss_fwd_bwd(ll, resp, r["mask"], r["old_logprob"], f32(r["advantages_whitened"]),
                               npy(batch["values_new"]), npy(batch["values"]), f32(r["returns"]), tau,
                               np.float32(h.cliprange), np.float32(h.cliprange_value), np.float32(h.vf_coef),
                               want_dlogits=want_dlogits, sel_rows=sel_rows)
    return r


def near_kink(new_logprob, old_logprob, eps):
    rho = np.exp(np.asarray(new_logprob, np.float64) - np.asarray(old_logprob, np.float64))
    e = float(np.float32(eps))
    return (np.abs(rho - (1.0 - e)) < KINK) | (np.abs(rho - (1.0 + e)) < KINK)
