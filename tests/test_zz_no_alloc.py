"""The allocation-free loss entry point (scratch built into the library) must give what the
workspace-based entry point gives, on two calls in a row (the built-in scratch still holds the first
call's contents when the second one starts).  Collected last on purpose: if it fails under -x, every
other test has already run."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu


def _batch(B, T, seed, frac_real):
    g = torch.Generator(device="cuda").manual_seed(seed)
    r = lambda *s: torch.randn(*s, generator=g, device="cuda")
    L = (torch.rand(B, generator=g, device="cuda") * T * frac_real).long().clamp(1, T)
    mask = (torch.arange(T, device="cuda")[None] < L[:, None]).to(torch.uint8).contiguous()
    nlp = (-0.05 - r(B, T).abs() * 2).contiguous()
    old = (nlp + 0.15 * r(B, T)).contiguous()
    vo = r(B, T)
    return dict(nlp=nlp, ent=r(B, T).abs().contiguous(), mask=mask, old=old, adv=r(B, T), vn=(vo + 0.2 * r(B, T)).contiguous(),
                vo=vo, ret=r(B, T))


def _run_both(P, b):
    B, T = b["nlp"].shape
    params = P.default_params()
    ws = P.new_workspace(P.workspace_bytes(B, T, 2))
    ref = P.loss_from_logprob(b["nlp"], b["ent"], b["mask"], b["old"], b["adv"], b["vn"], b["vo"], b["ret"], params, ws)
    out = {"losses": torch.full((8,), float("nan"), device="cuda"),
           "dlogprob": torch.full((B, T), float("nan"), device="cuda"),
           "dvalues": torch.full((B, T), float("nan"), device="cuda")}
    P.loss_from_logprob_static(b["nlp"], b["ent"], b["mask"], b["old"], b["adv"], b["vn"], b["vo"], b["ret"], params, out)
    torch.cuda.synchronize()
    for k in ("losses", "dlogprob", "dvalues"):
        got, want = out[k].double().cpu().numpy(), ref[k].double().cpu().numpy()
        assert np.isfinite(got).all(), k
        assert np.abs(got - want).max() <= 1e-6, (k, np.abs(got - want).max())
    return out


def test_static_scratch_entry_matches_workspace_entry_twice():
    assert torch.cuda.is_available()
    import paper_2403_17031_b200 as P
    from paper_2403_17031_b200 import binding, build
    build.build()
    P.lib()
    # first call: a large batch fills the built-in scratch; second call: a smaller batch with another
    # mask must not see any of it
    first = _run_both(P, _batch(512, 53, seed=1, frac_real=1.0))
    second = _run_both(P, _batch(64, 53, seed=2, frac_real=0.6))
    assert float(first["losses"][7]) > float(second["losses"][7]) > 0
    # a batch beyond the built-in maximum is refused on the host, before any launch
    B, T = 1024, 53
    assert B * T > binding.STATIC_MAX_TOKENS
    big = _batch(B, T, seed=3, frac_real=1.0)
    out = {"losses": torch.zeros(8, device="cuda"), "dlogprob": torch.zeros(B, T, device="cuda"),
           "dvalues": torch.zeros(B, T, device="cuda")}
    with pytest.raises(P.PPOError) as e:
        P.loss_from_logprob_static(big["nlp"], big["ent"], big["mask"], big["old"], big["adv"], big["vn"], big["vo"],
                                   big["ret"], P.default_params(), out)
    assert e.value.code == -6          # PPO_ERR_UNSUPPORTED


def _static_call(P, b, out):
    return P.loss_from_logprob_static(b["nlp"], b["ent"], b["mask"], b["old"], b["adv"], b["vn"], b["vo"], b["ret"],
                                      P.default_params(), out)


def test_static_scratch_entry_allocates_nothing_and_handles_an_empty_mask():
    """What the entry point is for: after its first call on the device (which looks up the built-in array) further
    calls leave the amount of free device memory exactly where it was. A batch without a single real token has no
    status word to report through; it returns n = 0 with finite losses and zero gradients."""
    assert torch.cuda.is_available()
    import paper_2403_17031_b200 as P
    from paper_2403_17031_b200 import build
    build.build()
    P.lib()
    B, T = 256, 53
    b = _batch(B, T, seed=4, frac_real=0.7)
    out = {"losses": torch.zeros(8, device="cuda"), "dlogprob": torch.zeros(B, T, device="cuda"),
           "dvalues": torch.zeros(B, T, device="cuda")}
    _static_call(P, b, out)                       # warm-up: symbol look-up, module load
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    for _ in range(5):
        _static_call(P, b, out)
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    assert free1 == free0, (free0, free1)
    assert float(out["losses"][7]) == float(b["mask"].sum())
    # no real token at all
    b["mask"].zero_()
    for k in out:
        out[k].fill_(float("nan"))
    _static_call(P, b, out)
    torch.cuda.synchronize()
    assert float(out["losses"][7]) == 0.0
    assert torch.isfinite(out["losses"]).all()
    assert not out["dlogprob"].any() and not out["dvalues"].any()


def test_static_scratch_entry_against_the_oracle():
    """The allocation-free entry point against the fp64 oracle's loss arithmetic (not only against its sibling): the
    given log-probs are reproduced inside the oracle by a two-entry vocabulary (x, 0) at temperature 1."""
    assert torch.cuda.is_available()
    import paper_2403_17031_b200 as P
    from oracle import ppo_oracle as O
    from paper_2403_17031_b200 import build
    build.build()
    P.lib()
    O.build()
    B, T = 128, 53
    b = _batch(B, T, seed=5, frac_real=0.8)
    out = {"losses": torch.zeros(8, device="cuda"), "dlogprob": torch.zeros(B, T, device="cuda"),
           "dvalues": torch.zeros(B, T, device="cuda")}
    npy = lambda t: t.detach().cpu().numpy()
    m = npy(b["mask"])
    nlp = npy(b["nlp"]).astype(np.float64)
    p = np.exp(nlp)
    x = np.log(p) - np.log1p(-p)
    hy = P.default_params()
    ref = O.loss_fwd_bwd(np.stack([x, np.zeros_like(x)], -1).astype(np.float32), np.zeros((B, T), np.int32), m,
                         npy(b["old"]), npy(b["adv"]), npy(b["vn"]), npy(b["vo"]), npy(b["ret"]), 1.0,
                         np.float32(hy.cliprange), np.float32(hy.cliprange_value), np.float32(hy.vf_coef),
                         want_dlogits=False)
    for call in range(2):
        for k in out:
            out[k].fill_(float("nan"))
        _static_call(P, b, out)
        torch.cuda.synchronize()
        n = ref["losses"][7]
        got = npy(out["losses"]).astype(np.float64)
        assert got[7] == n
        rho = np.exp(ref["new_logprob"] - npy(b["old"]).astype(np.float64))
        kink = ((np.abs(rho - 0.8) < 1e-4) | (np.abs(rho - 1.2) < 1e-4)) & m.astype(bool)
        for i in range(6):
            tol = 1e-4 + (kink.sum() / n if i == 4 else 0.0)
            assert abs(got[i] - ref["losses"][i]) <= tol, (call, i, got[i], ref["losses"][i])
        assert abs(got[6] - npy(b["ent"]).astype(np.float64)[m.astype(bool)].mean()) <= 1e-5
        assert np.abs(n * npy(out["dvalues"]) - n * ref["dvalues"]).max() <= 1e-4
        assert np.abs((n * npy(out["dlogprob"]) - n * ref["dlogprob"])[~kink]).max() <= 1e-4
