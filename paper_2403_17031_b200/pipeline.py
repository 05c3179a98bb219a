"""The whole per-token path as one object: preallocated outputs + the chain of C-ABI calls in
the order a PPO iteration runs them. Pure call sequencing; every step runs in the CUDA library."""
from __future__ import annotations

from typing import Dict, Optional

import torch

from . import binding as _b


class PPOHotPath:
    """Buffers and call chain for a batch of B responses x T tokens over a vocabulary of V.

    step(...) runs: EOS trick -> log-prob/entropy of policy and reference -> KL rewards -> GAE ->
    advantage whitening -> clipped losses + gradients, all on the current CUDA stream, and
    returns the dict of output tensors (owned by this object, overwritten by the next step).
    Padding rows (after a response's first EOS) are masked out of every later step, so their logits
    are not read: log-prob and entropy are 0 there.
    """

    def __init__(self, B: int, T: int, V: int, logits_dtype: torch.dtype, params: _b.PPOParams,
                 device="cuda", want_dlogits: bool = True):
        self.B, self.T, self.V = B, T, V
        self.params = params
        self.device = torch.device(device)
        f32, i32, u8 = torch.float32, torch.int32, torch.uint8
        dev = self.device
        bt = lambda dt: torch.empty((B, T), dtype=dt, device=dev)
        self.workspace = _b.new_workspace(_b.workspace_bytes(B, T, V), dev)
        self.out: Dict[str, Optional[torch.Tensor]] = {
            "responses_out": bt(i32), "eos_index": torch.empty(B, dtype=i32, device=dev),
            "seq_len": torch.empty(B, dtype=i32, device=dev), "mask": bt(u8),
            "scores_out": torch.empty(B, dtype=f32, device=dev),
            "logprob": bt(f32), "entropy": bt(f32), "ref_logprob": bt(f32),
            "kl": bt(f32), "rewards": bt(f32), "advantages": bt(f32), "returns": bt(f32),
            "advantages_whitened": bt(f32), "whiten_stats": torch.empty(3, dtype=f32, device=dev),
            "losses": torch.empty(8, dtype=f32, device=dev),
            "dlogits": torch.empty((B, T, V), dtype=logits_dtype, device=dev) if want_dlogits else None,
            "dvalues": bt(f32), "new_logprob": bt(f32), "new_entropy": bt(f32), "dlogprob": bt(f32),
        }
        self._loss_out = {"losses": self.out["losses"], "dlogits": self.out["dlogits"],
                          "dvalues": self.out["dvalues"], "new_logprob": self.out["new_logprob"],
                          "entropy": self.out["new_entropy"], "dlogprob": self.out["dlogprob"]}

    def rollout_stats(self, policy_logits, ref_logits, responses, scores, values):
        """Steps 1-5, one C call per step: everything between sampling and the first PPO epoch."""
        o, p = self.out, self.params
        _b.truncate_and_score(responses, scores, p.eos_id, p.pad_id, p.no_eos_score,
                              out=(o["responses_out"], o["eos_index"], o["seq_len"], o["mask"], o["scores_out"]))
        m = o["mask"]
        _b.logprob_entropy(policy_logits, responses, p.temperature, mask=m, workspace=self.workspace,
                           out=(o["logprob"], o["entropy"], None))
        _b.logprob_entropy(ref_logits, responses, p.temperature, mask=m, workspace=self.workspace,
                           out=(o["ref_logprob"], None, None))
        _b.kl_rewards(o["logprob"], o["ref_logprob"], o["mask"], o["seq_len"], o["scores_out"], p.kl_coef,
                      out=(o["kl"], o["rewards"]))
        if p.whiten_rewards:   # optional reward whitening: mean kept, in place, before GAE
            _b.whiten(o["rewards"], o["mask"], False, p.whiten_eps, workspace=self.workspace, out=o["rewards"])
        _b.gae(o["rewards"], values, o["seq_len"], p.gamma, p.lam, out=(o["advantages"], o["returns"]))
        _b.whiten(o["advantages"], o["mask"], True, p.whiten_eps, workspace=self.workspace,
                  out=o["advantages_whitened"], stats=o["whiten_stats"])
        return o

    def loss(self, logits, responses, old_logprob, values_new, values_old, next_epoch: bool = False):
        """Step 6 on the loss-time logits, using the advantages/returns of rollout_stats or step.
        next_epoch: a later PPO epoch on the same batch (the call before this one on this object was loss() or
        step()): the row order left in the workspace is reused, one launch less."""
        o = self.out
        _b.loss_fwd_bwd(logits, responses, o["mask"], old_logprob, o["advantages_whitened"], values_new,
                        values_old, o["returns"], self.params, self.workspace, out=self._loss_out,
                        next_epoch=next_epoch)
        return o

    def step(self, policy_logits, ref_logits, responses, scores, values, values_new, old_logprob=None,
             loss_logits=None):
        """One pass of the whole path in one C call (ppo_step). old_logprob defaults to the rollout
        log-probs just computed (first PPO epoch: ratio = 1); loss_logits defaults to policy_logits."""
        io = self.step_io({"policy_logits": policy_logits, "ref_logits": ref_logits, "loss_logits": loss_logits,
                           "responses": responses, "scores": scores, "values": values, "values_new": values_new,
                           "old_logprob": old_logprob})
        _b.step(io, policy_logits.dtype, self.B, self.T, self.V, self.params)
        return self.out

    def capture_step(self, policy_logits, ref_logits, responses, scores, values, values_new, old_logprob=None,
                     loss_logits=None):
        """Record one step() on these (fixed) buffers into a CUDA graph; graph.replay() then runs the
        whole path with a single launch call. The caller must have run step() once before (the first
        call sets kernel attributes) and keeps the input tensors alive and in place."""
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            self.step(policy_logits, ref_logits, responses, scores, values, values_new, old_logprob=old_logprob,
                      loss_logits=loss_logits)
        return graph

    def step_io(self, inputs: dict, cuda: bool = True) -> "_b.PPOStepIO":
        """ppo_step_io for this object's output buffers plus the given input tensors."""
        o = self.out
        t = dict(inputs)
        t.update({k: o[k] for k in ("responses_out", "eos_index", "seq_len", "mask", "scores_out", "logprob", "entropy",
                                    "ref_logprob", "kl", "rewards", "advantages", "returns", "advantages_whitened",
                                    "whiten_stats", "losses", "dlogits", "dvalues", "new_logprob", "new_entropy",
                                    "dlogprob")})
        t["workspace"] = self.workspace
        return _b.PPOStepIO.from_tensors(t, cuda)

    def curves(self):
        """The three statistics the paper plots per PPO update, from the outputs of the last rollout_stats() / step():
        [mean RLHF reward, mean summed per-token KL, mean score] as a [3] f32 tensor (one small launch)."""
        o = self.out
        return _b.rollout_curves(o["kl"], o["mask"], o["scores_out"], self.params.kl_coef)

    def device_status(self) -> int:
        return _b.last_device_status(self.workspace)


class DPOStep:
    """One DPO step on materialised logits (section "Preliminaries", "RL-free approaches"), all on the
    current CUDA stream: token log-probs of the policy and of the frozen SFT reference on the response
    rows (prompt and padding rows are skipped, never read), the DPO loss with its implicit rewards, and
    the gradient back to the policy's logits. Leading axis of every tensor: 0 = chosen, 1 = rejected.
    Temperature is 1 (the loss is defined on the model's own distribution)."""

    def __init__(self, P: int, T: int, V: int, dtype: torch.dtype, beta: float, device="cuda"):
        dev = torch.device(device)
        self.P, self.T, self.V, self.beta = P, T, V, float(beta)
        f32 = torch.float32
        self.workspace = _b.new_workspace(_b.workspace_bytes(2 * P * T, 1, V), dev)
        self.out = {
            "logprob": torch.empty((2, P, T), dtype=f32, device=dev),
            "ref_logprob": torch.empty((2, P, T), dtype=f32, device=dev),
            "out4": torch.empty(4, dtype=f32, device=dev),
            "reward_c": torch.empty(P, dtype=f32, device=dev), "reward_r": torch.empty(P, dtype=f32, device=dev),
            "dlogprob": torch.empty((2, P, T), dtype=f32, device=dev),
            "dlogits": torch.empty((2, P, T, V), dtype=dtype, device=dev),
        }

    def step(self, policy_logits, ref_logits, tokens, mask):
        o = self.out
        _b.logprob_entropy_pair(policy_logits, ref_logits, tokens, 1.0, mask=mask, workspace=self.workspace,
                                out=(o["logprob"], None, o["ref_logprob"]))
        _b.dpo_loss(o["logprob"][0], o["logprob"][1], o["ref_logprob"][0], o["ref_logprob"][1], mask[0], mask[1],
                    self.beta, out={"out4": o["out4"], "reward_c": o["reward_c"], "reward_r": o["reward_r"],
                                    "dlp_c": o["dlogprob"][0], "dlp_r": o["dlogprob"][1]})
        _b.logprob_bwd(policy_logits, tokens, mask, o["dlogprob"], 1.0, self.workspace, dlogits=o["dlogits"])
        return o

    def device_status(self) -> int:
        return _b.last_device_status(self.workspace)
