"""ppo_rollout_curves (the three PPO learning curves of the paper's figure) against the fp64 oracle."""
import numpy as np
import pytest
import torch

from parity import TOL_LOGPROB as TOL_ABS

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def P():
    assert torch.cuda.is_available()
    import paper_2403_17031_b200 as P
    from paper_2403_17031_b200 import build
    build.build()
    P.lib()
    return P


def _case(B, T, seed, with_mask):
    rng = np.random.default_rng(seed)
    L = rng.integers(1, T + 1, size=B)
    mask = (np.arange(T)[None] < L[:, None]).astype(np.uint8)
    kl = rng.normal(size=(B, T)).astype(np.float32) * 0.3
    if with_mask:
        kl = np.where(mask == 1, kl, np.float32(1e20))      # behind the responses: must not be read as numbers
    else:
        kl = kl * mask
    scores = rng.normal(size=B).astype(np.float32)
    return kl, mask, scores


@pytest.mark.parametrize("B,T", [(1, 1), (2, 3), (33, 31), (64, 53), (512, 53), (256, 512), (5, 1000), (1500, 7)])
@pytest.mark.parametrize("with_mask", [True, False])
def test_curves_match_the_oracle(P, B, T, with_mask):
    from oracle import curves_oracle as Q
    kl, mask, scores = _case(B, T, 100 + B + T, with_mask)
    want = Q.rollout_curves(kl, mask if with_mask else None, scores, 0.05)
    out = torch.full((3,), float("nan"), device="cuda")
    P.rollout_curves(torch.from_numpy(kl).cuda(), torch.from_numpy(mask).cuda() if with_mask else None,
                     torch.from_numpy(scores).cuda(), 0.05, out=out)
    got = out.double().cpu().numpy()
    for i, k in enumerate(("rlhf_reward", "kl", "score")):
        assert abs(got[i] - want[k]) <= TOL_ABS, (k, got[i], want[k])


def test_curves_on_the_chain_of_config1(P):
    """Fed with what steps 2 and 3 produce on a TL;DR-shaped batch: the reward curve is the mean of the summed
    per-token rewards of step 3 (oracle), and repeated calls give the same bits."""
    from oracle import curves_oracle as Q
    from oracle import ppo_oracle as O
    rng = np.random.default_rng(9)
    B, T = 64, 53
    resp = rng.integers(2, 50304, size=(B, T)).astype(np.int32)
    for b in range(0, B, 9):
        resp[b, rng.integers(0, T)] = 0
    scores = rng.normal(size=B).astype(np.float32)
    lp = (-np.abs(rng.normal(size=(B, T))) - 0.1).astype(np.float32)
    rlp = (lp + 0.2 * rng.normal(size=(B, T))).astype(np.float32)
    _, _, L, m, so = O.truncate_and_score(resp, 0, 1, scores, -1.0)
    d = lambda a, dt: torch.from_numpy(np.ascontiguousarray(a)).to(dt).cuda()
    _, _, seq_len, mask, scores_out = P.truncate_and_score(d(resp, torch.int32), d(scores, torch.float32), 0, 1, -1.0)
    kl, rew = P.kl_rewards(d(lp, torch.float32), d(rlp, torch.float32), mask, seq_len, scores_out, 0.05)
    a = P.rollout_curves(kl, mask, scores_out, 0.05).clone()
    b = P.rollout_curves(kl, None, scores_out, 0.05).clone()
    assert torch.equal(a, b) and torch.equal(a, P.rollout_curves(kl, mask, scores_out, 0.05))
    okl, orew = O.kl_rewards(lp.astype(np.float64), rlp.astype(np.float64), m, L, so, 0.05)
    want = Q.rollout_curves(okl, m, so, 0.05)
    got = a.double().cpu().numpy()
    assert abs(got[0] - orew.sum(axis=1).mean()) <= TOL_ABS
    for i, k in enumerate(("rlhf_reward", "kl", "score")):
        assert abs(got[i] - want[k]) <= TOL_ABS, k


def test_curves_argument_errors(P):
    from paper_2403_17031_b200 import binding
    kl = torch.zeros(2, 3, device="cuda")
    s = torch.zeros(2, device="cuda")
    with pytest.raises(P.PPOError) as e:
        P.rollout_curves(kl, None, s, float("nan"))
    assert e.value.code == -3
    L = binding.lib()
    assert L.ppo_rollout_curves(None, None, s.data_ptr(), 2, 3, 0.05, s.data_ptr(), None) == -1
    assert L.ppo_rollout_curves(kl.data_ptr(), None, s.data_ptr(), 0, 3, 0.05, s.data_ptr(), None) == -2


def test_curves_after_the_single_call_step(P):
    """PPOHotPath.curves() after ppo_step on a small TL;DR-shaped batch equals the oracle on the step's own outputs."""
    import dataclasses
    from oracle import curves_oracle as Q
    from paper_2403_17031_b200 import binding
    from paper_2403_17031_b200.pipeline import PPOHotPath
    from paper_2403_17031_b200.synthetic import CONFIGS, make_batch
    cfg = dataclasses.replace(CONFIGS[1], B=16, V=2048)
    batch = make_batch(cfg, "cuda")
    hp = PPOHotPath(cfg.B, cfg.T, cfg.V, cfg.torch_dtype, binding.params_from(cfg.hyper))
    o = hp.step(batch["policy_logits"], batch["ref_logits"], batch["responses"], batch["scores"], batch["values"],
                batch["values_new"])
    got = hp.curves().double().cpu().numpy()
    want = Q.rollout_curves(o["kl"].cpu().numpy(), o["mask"].cpu().numpy(), o["scores_out"].cpu().numpy(),
                            cfg.hyper.kl_coef)
    for i, k in enumerate(("rlhf_reward", "kl", "score")):
        assert abs(got[i] - want[k]) <= TOL_ABS, k
    assert abs(got[0] - float(o["rewards"].double().sum(dim=1).mean())) <= TOL_ABS
