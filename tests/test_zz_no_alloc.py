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
