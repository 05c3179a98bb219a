"""Seeded synthetic PPO batches with the shapes of the paper's TL;DR / Pythia workload.

This module only *draws data*: Gaussian logits, Gumbel-max token samples, EOS positions,
values and scores. It contains none of the hot path's arithmetic (no log-softmax, no KL, no
GAE, no whitening, no loss), so the CUDA library and the CPU oracle can both be fed from it
without sharing any of the method's code. Tensors are produced on the requested device; a
parity test copies the very same bytes to the host for the oracle.

Shapes follow the paper: responses of T = 53 tokens (Pythia tokenizer; section "Dataset
Details"), EOS id 0 (figure "actual rewards" caption), a distinct [PAD] id, batch 512 = 8 x 64
and the PPO hyper-parameters of Table "PPO hyperparameters".  The datasets themselves are not
used anywhere; nothing here reproduces an item of them.
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import Dict, Optional

import torch

BASE_SEED = 20240317


@dataclass(frozen=True)
class PPOHyper:
    """Table "PPO hyperparameters" of the paper, plus the EOS-trick constants."""
    temperature: float = 0.7
    kl_coef: float = 0.05          # beta
    gamma: float = 1.0
    lam: float = 0.95
    cliprange: float = 0.2         # epsilon
    cliprange_value: float = 0.2   # epsilon-hat
    vf_coef: float = 0.1           # c1
    no_eos_score: float = -1.0     # "EOS trick": score used when a response has no EOS
    whiten_eps: float = 1e-8       # constant inside the paper's whiten()
    eos_id: int = 0                # Pythia <|endoftext|>
    pad_id: int = 1                # a [PAD] id distinct from EOS
    whiten_rewards: int = 0        # detail "(Optional) Reward whitening": whiten(rewards, shift_mean=False) before GAE


@dataclass(frozen=True)
class WorkloadConfig:
    index: int
    name: str
    B: int
    T: int
    V: int
    dtype: str                     # "f32" | "bf16" storage type of the logits
    logit_std: float               # std of the Gaussian logits
    row_scale_lo: float = 1.0      # per-row scale ~ U[lo, hi] (flat <-> peaked rows)
    row_scale_hi: float = 1.0
    ref_mode: str = "noise"        # "noise": ref = policy + N(0, ref_noise^2); "independent"
    ref_noise: float = 0.1
    no_eos_frac: float = 0.1       # fraction of rows that never emit EOS
    n_no_eos_exact: Optional[int] = None  # tiny config: exact number of rows without EOS
    hyper: PPOHyper = PPOHyper()
    # fused LM-head shape (config 4 only)
    d_model: int = 0
    h_std: float = 1.0
    w_std: float = 0.02
    w_ref_noise: float = 0.002

    @property
    def seed(self) -> int:
        return BASE_SEED + self.index

    @property
    def rows(self) -> int:
        return self.B * self.T

    @property
    def torch_dtype(self) -> torch.dtype:
        return torch.float32 if self.dtype == "f32" else torch.bfloat16


CONFIGS: Dict[int, WorkloadConfig] = {
    0: WorkloadConfig(0, "tiny-correctness", B=4, T=16, V=1000, dtype="f32", logit_std=2.0,
                      ref_mode="independent", n_no_eos_exact=1),
    1: WorkloadConfig(1, "pythia-1b-tldr-rollout", B=64, T=53, V=50304, dtype="bf16",
                      logit_std=2.0, no_eos_frac=0.1),
    2: WorkloadConfig(2, "full-ppo-batch", B=512, T=53, V=50304, dtype="bf16", logit_std=1.0,
                      row_scale_lo=1.0, row_scale_hi=8.0, no_eos_frac=0.1),
    3: WorkloadConfig(3, "long-response-stress", B=256, T=512, V=50304, dtype="f32",
                      logit_std=3.0, no_eos_frac=0.2,
                      hyper=PPOHyper(gamma=0.99, lam=0.95)),
    4: WorkloadConfig(4, "fused-lm-head-6.9b", B=512, T=53, V=50304, dtype="bf16",
                      logit_std=0.0, no_eos_frac=0.1, d_model=4096),
}


def shard_batch(global_B: int, rank: int, world_size: int) -> range:
    """Sequences [lo, hi) of a global batch owned by `rank` (contiguous, sizes differ by <= 1).

    The paper runs data-parallel (batch 512 over 8 GPUs, section "Setup -> Tech stack"); every
    sequence is an independent unit of the per-token path, so ranks never exchange data.
    """
    if world_size <= 0 or not (0 <= rank < world_size):
        raise ValueError("bad rank/world_size")
    base, rem = divmod(global_B, world_size)
    lo = rank * base + min(rank, rem)
    hi = lo + base + (1 if rank < rem else 0)
    return range(lo, hi)


def _gen(device, seed: int) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def _gumbel_argmax(logits_f32: torch.Tensor, temperature: float, banned, g: torch.Generator):
    """Draw one token per row from softmax(logits / temperature) by the Gumbel-max trick."""
    u = torch.rand(logits_f32.shape, generator=g, device=logits_f32.device, dtype=torch.float32)
    u.clamp_(min=1e-20, max=1.0 - 1e-7)
    pert = logits_f32 / temperature - torch.log(-torch.log(u))
    for b in banned:
        pert[:, b] = float("-inf")
    return pert.argmax(dim=-1).to(torch.int32)


def _place_eos(tokens: torch.Tensor, cfg: WorkloadConfig, g: torch.Generator, rank_seed_cpu: int):
    """Write EOS into a copy of `tokens` [B,T]: first EOS uniform over positions, absent in a
    fraction of rows; a quarter of the rows with EOS get a second, later EOS (sampling goes on
    after the first EOS, so repeats occur)."""
    B, T = tokens.shape
    gc = _gen("cpu", rank_seed_cpu)
    first = torch.randint(0, T, (B,), generator=gc)
    if cfg.n_no_eos_exact is not None:
        has = torch.ones(B, dtype=torch.bool)
        has[B - cfg.n_no_eos_exact:] = False
    else:
        has = torch.rand(B, generator=gc) >= cfg.no_eos_frac
    second_gap = torch.randint(1, max(T, 2), (B,), generator=gc)
    want_second = torch.rand(B, generator=gc) < 0.25
    out = tokens.clone()
    first_d = first.to(tokens.device)
    for b in range(B):
        if bool(has[b]):
            out[b, int(first[b])] = cfg.hyper.eos_id
            s = int(first[b]) + int(second_gap[b])
            if bool(want_second[b]) and s < T:
                out[b, s] = cfg.hyper.eos_id
    return out, first_d, has


def make_batch(cfg: WorkloadConfig, device="cpu", B: Optional[int] = None, seed: Optional[int] = None,
               chunk_rows: int = 2048, with_ref: bool = True) -> Dict[str, torch.Tensor]:
    """Build one synthetic PPO batch for configs 0-3 (logits stored in HBM).

    Returns tensors (all on `device`):
      policy_logits, ref_logits  [B,T,V]  cfg dtype   (ref omitted when with_ref=False)
      responses                  [B,T]    int32   sampled tokens with EOS written in, untruncated
      scores                     [B]      float32 reward-model scores ~ N(0,1)
      values, values_new         [B,T]    float32 value-head outputs at rollout / at loss time
      old_logprob_noise          [B,T]    float32 ~ N(0,0.15^2); a harness adds it to rollout
                                                  logprobs so PPO ratios straddle the clip range
    """
    if B is not None:
        cfg = replace(cfg, B=B)
    seed = cfg.seed if seed is None else seed
    dev = torch.device(device)
    g = _gen(dev, seed)
    Bn, T, V = cfg.B, cfg.T, cfg.V
    rows = Bn * T
    dt = cfg.torch_dtype
    h = cfg.hyper
    policy = torch.empty((rows, V), dtype=dt, device=dev)
    ref = torch.empty((rows, V), dtype=dt, device=dev) if with_ref else None
    tokens = torch.empty((rows,), dtype=torch.int32, device=dev)
    for r0 in range(0, rows, chunk_rows):
        r1 = min(rows, r0 + chunk_rows)
        x = torch.randn((r1 - r0, V), generator=g, device=dev, dtype=torch.float32)
        x.mul_(cfg.logit_std)
        if cfg.row_scale_hi > cfg.row_scale_lo:
            s = torch.rand((r1 - r0, 1), generator=g, device=dev, dtype=torch.float32)
            x.mul_(cfg.row_scale_lo + (cfg.row_scale_hi - cfg.row_scale_lo) * s)
        x[:, h.pad_id] = -30.0           # [PAD] is never sampled
        p = x.to(dt)
        policy[r0:r1] = p
        tokens[r0:r1] = _gumbel_argmax(p.float(), h.temperature, (h.eos_id, h.pad_id), g)
        if with_ref:
            if cfg.ref_mode == "independent":
                y = torch.randn((r1 - r0, V), generator=g, device=dev, dtype=torch.float32)
                y.mul_(cfg.logit_std)
                y[:, h.pad_id] = -30.0
            else:
                y = p.float() + cfg.ref_noise * torch.randn((r1 - r0, V), generator=g, device=dev,
                                                            dtype=torch.float32)
            ref[r0:r1] = y.to(dt)
        del x, p
    responses, _, _ = _place_eos(tokens.view(Bn, T), cfg, g, seed + 7919)
    scores = torch.randn((Bn,), generator=g, device=dev, dtype=torch.float32)
    values = torch.randn((Bn, T), generator=g, device=dev, dtype=torch.float32)
    values_new = values + 0.1 * torch.randn((Bn, T), generator=g, device=dev, dtype=torch.float32)
    noise = 0.15 * torch.randn((Bn, T), generator=g, device=dev, dtype=torch.float32)
    out = {
        "policy_logits": policy.view(Bn, T, V),
        "responses": responses.contiguous(),
        "scores": scores,
        "values": values,
        "values_new": values_new,
        "old_logprob_noise": noise,
    }
    if with_ref:
        out["ref_logits"] = ref.view(Bn, T, V)
    return out


def make_lmhead_batch(cfg: WorkloadConfig, device="cpu", M: Optional[int] = None,
                      K: Optional[int] = None, V: Optional[int] = None, seed: Optional[int] = None,
                      chunk_rows: int = 1024) -> Dict[str, torch.Tensor]:
    """Build the fused LM-head workload (config 4): hidden states H [M,K] ~ N(0,1) bf16, the
    unembedding W [K,V] ~ N(0,0.02^2) bf16, a perturbed reference unembedding, tokens sampled
    from softmax(H W / temperature) with a library matmul (data generation only), and the
    [B,T]-shaped values/scores when M == B*T."""
    seed = cfg.seed if seed is None else seed
    dev = torch.device(device)
    g = _gen(dev, seed)
    M = cfg.rows if M is None else M
    K = cfg.d_model if K is None else K
    V = cfg.V if V is None else V
    hy = cfg.hyper
    H = (cfg.h_std * torch.randn((M, K), generator=g, device=dev, dtype=torch.float32)).to(torch.bfloat16)
    Wf = cfg.w_std * torch.randn((K, V), generator=g, device=dev, dtype=torch.float32)
    W = Wf.to(torch.bfloat16)
    W_ref = (W.float() + cfg.w_ref_noise * torch.randn((K, V), generator=g, device=dev,
                                                      dtype=torch.float32)).to(torch.bfloat16)
    del Wf
    tokens = torch.empty((M,), dtype=torch.int32, device=dev)
    for r0 in range(0, M, chunk_rows):
        r1 = min(M, r0 + chunk_rows)
        lg = (H[r0:r1].float() @ W.float()) if dev.type == "cpu" else (H[r0:r1] @ W).float()
        tokens[r0:r1] = _gumbel_argmax(lg, hy.temperature, (hy.eos_id, hy.pad_id), g)
        del lg
    out = {"H": H, "W": W, "W_ref": W_ref, "tokens": tokens}
    if M % cfg.T == 0:
        Bn = M // cfg.T
        sub = replace(cfg, B=Bn)
        responses, _, _ = _place_eos(tokens.view(Bn, cfg.T), sub, g, seed + 7919)
        out["responses"] = responses.contiguous()
        out["scores"] = torch.randn((Bn,), generator=g, device=dev, dtype=torch.float32)
        out["values"] = torch.randn((Bn, cfg.T), generator=g, device=dev, dtype=torch.float32)
        out["values_new"] = out["values"] + 0.1 * torch.randn((Bn, cfg.T), generator=g, device=dev,
                                                              dtype=torch.float32)
        out["old_logprob_noise"] = 0.15 * torch.randn((Bn, cfg.T), generator=g, device=dev,
                                                       dtype=torch.float32)
    return out


# ---------------------------------------------------------------- preference batches (RM / DPO losses)
@dataclass(frozen=True)
class PrefConfig:
    """A batch of preference pairs in the paper's pre-tokenised layout (section "Dataset": query and
    response concatenated and right-padded to 638 tokens; queries fill the first 512 positions)."""
    name: str
    P: int                 # pairs; Table "DPO hyperparameters": batch 64 over 8 GPUs = 8 pairs per GPU
    T: int = 638
    V: int = 50304
    dtype: str = "bf16"
    query_len: int = 512   # positions [0, query_len) are the prompt: not part of the loss
    resp_lo: int = 20      # response lengths ~ U[resp_lo, resp_hi]
    resp_hi: int = 126
    logit_std: float = 2.0
    ref_noise: float = 0.5
    beta: float = 0.05     # Table "DPO hyperparameters"
    seed: int = BASE_SEED + 5

    @property
    def torch_dtype(self) -> torch.dtype:
        return torch.float32 if self.dtype == "f32" else torch.bfloat16


PREF_CONFIGS: Dict[str, PrefConfig] = {
    "tiny": PrefConfig("tiny-pref", P=3, T=24, V=1000, dtype="f32", query_len=10, resp_lo=2, resp_hi=14),
    "dpo": PrefConfig("dpo-tldr-per-gpu", P=8),
}


def make_pref_batch(cfg: PrefConfig, device="cpu", seed: Optional[int] = None,
                    chunk_rows: int = 2048) -> Dict[str, torch.Tensor]:
    """Index 0 of the leading axis = chosen completions, 1 = rejected.
      policy_logits, ref_logits [2,P,T,V] cfg dtype: N(0, logit_std^2) on response rows (reference = policy
                                 + N(0, ref_noise^2)), zeros elsewhere (those rows are never read)
      tokens [2,P,T] int32       labels, uniform over the vocabulary
      mask   [2,P,T] uint8       1 on the response tokens (query_len <= t < query_len + length)
      rm_rewards [2,P] float32   stand-in reward-model outputs ~ N(0,1) (+0.5 for chosen)"""
    seed = cfg.seed if seed is None else seed
    dev = torch.device(device)
    g = _gen(dev, seed)
    gc = _gen("cpu", seed + 7919)
    P, T, V = cfg.P, cfg.T, cfg.V
    length = torch.randint(cfg.resp_lo, cfg.resp_hi + 1, (2, P), generator=gc)
    length = torch.minimum(length, torch.tensor(T - cfg.query_len))
    t = torch.arange(T)[None, None, :]
    mask = ((t >= cfg.query_len) & (t < cfg.query_len + length[:, :, None])).to(torch.uint8)
    tokens = torch.randint(2, V, (2, P, T), generator=gc, dtype=torch.int32)
    dt = cfg.torch_dtype
    policy = torch.zeros((2 * P * T, V), dtype=dt, device=dev)
    ref = torch.zeros((2 * P * T, V), dtype=dt, device=dev)
    rows = torch.nonzero(mask.reshape(-1)).reshape(-1).to(dev)
    for r0 in range(0, rows.numel(), chunk_rows):
        idx = rows[r0:r0 + chunk_rows]
        x = cfg.logit_std * torch.randn((idx.numel(), V), generator=g, device=dev, dtype=torch.float32)
        p = x.to(dt)
        policy[idx] = p
        ref[idx] = (p.float() + cfg.ref_noise * torch.randn((idx.numel(), V), generator=g, device=dev,
                                                            dtype=torch.float32)).to(dt)
        del x, p
    rm = torch.randn((2, P), generator=g, device=dev, dtype=torch.float32)
    rm[0] += 0.5
    return {"policy_logits": policy.view(2, P, T, V), "ref_logits": ref.view(2, P, T, V),
            "tokens": tokens.to(dev), "mask": mask.to(dev).contiguous(), "rm_rewards": rm}
