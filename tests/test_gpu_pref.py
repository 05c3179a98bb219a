"""GPU parity of the preference losses (section "Preliminaries": RM loss, DPO loss, implicit reward) and of the
log-prob backward, through the C ABI, against oracle/pref_oracle.py."""
import numpy as np
import pytest
import torch

from oracle import pref_oracle as R
from parity import TOL_LOGPROB, TOL_REL, assert_abs, assert_grad, assert_rel, dev, host_logits, npy

pytestmark = pytest.mark.gpu


def wide(t: torch.Tensor) -> np.ndarray:
    """Device logits -> float64 (bf16 and fp32 both widen exactly)."""
    return t.detach().double().cpu().numpy()


@pytest.fixture(scope="module")
def P():
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    import paper_2403_17031_b200 as pkg
    from paper_2403_17031_b200 import build
    build.build()
    pkg.lib()
    return pkg


@pytest.mark.parametrize("n", [1, 7, 1000, 5001])
def test_pairwise_loss(P, n):
    rng = np.random.default_rng(n)
    rc = (rng.normal(size=n) * 2 + 0.3).astype(np.float32)
    rr = (rng.normal(size=n) * 2).astype(np.float32)
    if n >= 7:
        rc[:3], rr[:3] = [90.0, -90.0, 1.25], [-90.0, 90.0, 1.25]     # saturated both ways, and a tie
    ref = R.pairwise_logistic_loss(rc, rr)
    o = P.pairwise_loss(dev(rc), dev(rr))
    got = npy(o["out4"]).astype(np.float64)
    assert_rel(got, np.array([ref["loss"], ref["accuracy"], rc.astype(np.float64).mean(),
                              rr.astype(np.float64).mean()]), TOL_REL, "loss, accuracy, mean rewards")
    assert_abs(n * npy(o["dr_c"]), n * ref["dr_c"], 1e-6, "P * dr_c")
    assert_abs(n * npy(o["dr_r"]), n * ref["dr_r"], 1e-6, "P * dr_r")
    assert np.isfinite(got).all()


@pytest.mark.parametrize("n,T", [(3, 5), (8, 638), (70, 53)])
def test_dpo_loss(P, n, T):
    rng = np.random.default_rng(100 * n + T)
    a = [(-rng.random((n, T)) * 8).astype(np.float32) for _ in range(4)]
    a[2] = (a[0] + rng.normal(size=(n, T)) * 0.6).astype(np.float32)       # reference near the policy
    a[3] = (a[1] + rng.normal(size=(n, T)) * 0.6).astype(np.float32)
    start = rng.integers(0, T, (2, n, 1))
    length = rng.integers(1, T + 1, (2, n, 1))
    t = np.arange(T)[None, None]
    m = ((t >= start) & (t < start + length)).astype(np.uint8)
    if n > 3:
        m[1, 2] = 0                                                         # a pair whose rejected side is empty
    beta = 0.05 if T > 5 else 2.0
    ref = R.dpo_loss(a[0], a[1], a[2], a[3], m[0], m[1], beta)
    o = P.dpo_loss(*(dev(x) for x in a), dev(m[0]), dev(m[1]), beta)
    want4 = np.array([ref["loss"], ref["accuracy"], ref["reward_c"].mean(), ref["reward_r"].mean()])
    assert_rel(npy(o["out4"]).astype(np.float64), want4, TOL_REL, "loss, accuracy, mean implicit rewards")
    assert_rel(npy(o["reward_c"]), ref["reward_c"], TOL_REL, "implicit reward (chosen)")
    assert_rel(npy(o["reward_r"]), ref["reward_r"], TOL_REL, "implicit reward (rejected)")
    assert_abs(n * npy(o["dlp_c"]), n * ref["dlp_c"], 1e-6, "P * dlogprob (chosen)")
    assert_abs(n * npy(o["dlp_r"]), n * ref["dlp_r"], 1e-6, "P * dlogprob (rejected)")
    assert not npy(o["dlp_c"])[m[0] == 0].any() and not npy(o["dlp_r"])[m[1] == 0].any()


@pytest.mark.parametrize("dtype,rows,V,engine", [
    (torch.float32, 37, 1000, 0), (torch.float32, 37, 1000, 1), (torch.float32, 19, 1001, 0),
    (torch.bfloat16, 24, 50304, 0), (torch.bfloat16, 24, 50304, 1), (torch.bfloat16, 700, 2048, 0),
    (torch.float32, 9, 50304, 0)])
def test_logprob_bwd(P, oracle, dtype, rows, V, engine):
    """engine 0: default kernels (bulk-copy row engine where the shape allows); 1: direct-load kernels."""
    from paper_2403_17031_b200 import binding
    g = torch.Generator(device="cuda").manual_seed(rows * 7 + V)
    x = (2.0 * torch.randn((rows, V), generator=g, device="cuda")).to(dtype)
    tok = torch.randint(0, V, (rows,), generator=g, device="cuda", dtype=torch.int32)
    mask = (torch.rand((rows,), generator=g, device="cuda") < 0.7).to(torch.uint8)
    mask[0] = 1
    up = torch.randn((rows,), generator=g, device="cuda")
    up[0] = 0.0                                                      # a real row with zero upstream gradient
    tau = 0.7
    ws = P.new_workspace(P.workspace_bytes(rows, 1, V))
    binding.set_option(binding.OPT_ROW_ENGINE, engine)
    try:
        o = P.logprob_bwd(x, tok, mask, up, tau, ws, want_aux=True)
        torch.cuda.synchronize()
    finally:
        binding.set_option(binding.OPT_ROW_ENGINE, 0)
    m = npy(mask).astype(bool)
    xs = host_logits(x)
    want = R.logprob_bwd(wide(x), npy(tok), npy(up).astype(np.float64), tau)
    got = o["dlogits"].float().cpu().numpy().astype(np.float64)
    assert not got[~m].any(), "rows outside the mask must be zero"
    assert_grad(got[m], want[m], dtype == torch.bfloat16, "dlogits")
    assert not got[0].any()
    lp, ent, _ = oracle.logprob_entropy(xs, npy(tok), tau)
    assert_abs(npy(o["new_logprob"])[m], lp[m], TOL_LOGPROB, "new_logprob")
    assert_abs(npy(o["entropy"])[m], ent[m], TOL_LOGPROB, "entropy")
    assert not npy(o["new_logprob"])[~m].any()
    assert P.last_device_status(ws) == 0


def test_logprob_bwd_bad_token_and_argument_errors(P):
    from paper_2403_17031_b200.binding import PPOError
    rows, V = 6, 512
    x = torch.randn((rows, V), device="cuda")
    tok = torch.tensor([1, 2, V, 3, -1, 4], dtype=torch.int32, device="cuda")
    mask = torch.ones(rows, dtype=torch.uint8, device="cuda")
    up = torch.ones(rows, device="cuda")
    ws = P.new_workspace(P.workspace_bytes(rows, 1, V))
    o = P.logprob_bwd(x, tok, mask, up, 1.0, ws)
    d = o["dlogits"].cpu().numpy()
    assert np.isnan(d[2]).all() and np.isnan(d[4]).all() and np.isfinite(d[[0, 1, 3, 5]]).all()
    assert P.last_device_status(ws) & 1
    with pytest.raises(PPOError):
        P.logprob_bwd(x, tok, mask, up, 0.0, ws)                      # temperature must be > 0
    with pytest.raises(PPOError):
        P.logprob_bwd(x, tok, mask, up, 1.0, ws, dlogits=x)           # in place is not supported


def test_dpo_step_chained(P, oracle):
    """Logits -> token log-probs (policy, reference) -> DPO loss -> gradient on the policy's logits."""
    from paper_2403_17031_b200.pipeline import DPOStep
    from paper_2403_17031_b200.synthetic import PREF_CONFIGS, make_pref_batch
    cfg = PREF_CONFIGS["tiny"]
    b = make_pref_batch(cfg, "cuda")
    n, T, V = cfg.P, cfg.T, cfg.V
    beta = 2.0            # larger than the paper's 0.05 so that the pairs differ visibly
    st = DPOStep(n, T, V, cfg.torch_dtype, beta)
    o = st.step(b["policy_logits"], b["ref_logits"], b["tokens"], b["mask"])
    torch.cuda.synchronize()
    tok, m = npy(b["tokens"]), npy(b["mask"])
    pl, rl = host_logits(b["policy_logits"]).reshape(-1, V), host_logits(b["ref_logits"]).reshape(-1, V)
    lp = oracle.logprob_entropy(pl, tok.reshape(-1), 1.0)[0].reshape(2, n, T) * m
    rlp = oracle.logprob_entropy(rl, tok.reshape(-1), 1.0)[0].reshape(2, n, T) * m
    ref = R.dpo_loss(lp[0], lp[1], rlp[0], rlp[1], m[0], m[1], beta)
    assert_abs(npy(o["logprob"]), lp, TOL_LOGPROB, "logprob")
    assert_abs(npy(o["ref_logprob"]), rlp, TOL_LOGPROB, "ref_logprob")
    # chained: each of up to 14 token log-probs per sequence carries <= 1e-4, times beta
    assert_abs(npy(o["reward_c"]), ref["reward_c"], 2e-3, "reward_c (chained)")
    assert_abs(npy(o["reward_r"]), ref["reward_r"], 2e-3, "reward_r (chained)")
    assert abs(float(o["out4"][0]) - ref["loss"]) < 2e-3 and abs(float(o["out4"][1]) - ref["accuracy"]) < 1e-6
    g = np.stack([ref["dlp_c"], ref["dlp_r"]]).reshape(-1)
    want = R.logprob_bwd(wide(b["policy_logits"]).reshape(-1, V), tok.reshape(-1), g, 1.0)
    got = npy(o["dlogits"]).reshape(-1, V).astype(np.float64)
    assert not got[m.reshape(-1) == 0].any()
    assert_abs(n * got, n * want, 2e-3, "P * dlogits (chained)")
    assert st.device_status() == 0


def test_logprob_entropy_pair_equals_two_calls(P):
    """One launch for policy and reference logits (with and without a mask) gives the bits of two separate calls;
    V = 1001 takes the layout without 16-byte packs (two launches inside)."""
    g = torch.Generator(device="cuda").manual_seed(21)
    for dtype, rows, V in ((torch.bfloat16, 300, 2048), (torch.float32, 77, 1000), (torch.float32, 9, 1001)):
        x = (2.0 * torch.randn((rows, V), generator=g, device="cuda")).to(dtype)
        y = (x.float() + 0.3 * torch.randn((rows, V), generator=g, device="cuda")).to(dtype)
        tok = torch.randint(0, V, (rows,), generator=g, device="cuda", dtype=torch.int32)
        for mask in (None, (torch.rand((rows,), generator=g, device="cuda") < 0.3).to(torch.uint8)):
            lp, ent, _ = P.logprob_entropy(x, tok, 0.7, mask=mask)
            rlp, _, _ = P.logprob_entropy(y, tok, 0.7, mask=mask, want_entropy=False)
            lp2, ent2, rlp2 = P.logprob_entropy_pair(x, y, tok, 0.7, mask=mask)
            assert torch.equal(lp, lp2) and torch.equal(ent, ent2) and torch.equal(rlp, rlp2)


def test_degenerate_shapes(P, oracle):
    """One pair of one token; a backward call whose mask selects no row (everything zero, status bit set)."""
    o = P.dpo_loss(*(dev(np.array([[v]], np.float32)) for v in (-1.0, -2.0, -1.5, -1.0)),
                   dev(np.ones((1, 1), np.uint8)), dev(np.ones((1, 1), np.uint8)), 0.5)
    ref = R.dpo_loss([[-1.0]], [[-2.0]], [[-1.5]], [[-1.0]], np.ones((1, 1)), np.ones((1, 1)), 0.5)
    assert abs(float(o["out4"][0]) - ref["loss"]) < 1e-6 and float(o["out4"][1]) == ref["accuracy"]
    assert_abs(npy(o["dlp_c"]), ref["dlp_c"], 1e-6, "dlp_c")
    rows, V = 40, 2048
    x = torch.randn((rows, V), device="cuda").to(torch.bfloat16)
    tok = torch.zeros(rows, dtype=torch.int32, device="cuda")
    ws = P.new_workspace(P.workspace_bytes(rows, 1, V))
    out = P.logprob_bwd(x, tok, torch.zeros(rows, dtype=torch.uint8, device="cuda"), torch.ones(rows, device="cuda"),
                        1.0, ws, want_aux=True)
    torch.cuda.synchronize()
    assert not out["dlogits"].float().any() and not out["new_logprob"].any()
    assert P.last_device_status(ws) == 2                                  # PPO_DEV_EMPTY_MASK
