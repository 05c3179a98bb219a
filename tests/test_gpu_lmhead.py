"""GPU parity of the fused LM-head call (tcgen05 GEMM + log-prob/entropy reduction) against the
fp64 oracle, which forms each logits row by explicit dot products."""
import numpy as np
import pytest
import torch

from parity import TOL_LOGPROB, assert_abs, host_logits, npy

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def P():
    assert torch.cuda.is_available()
    import paper_2403_17031_b200 as pkg
    from paper_2403_17031_b200 import build
    build.build()
    pkg.lib()
    return pkg


def _inputs(M, K, V, seed, w_std=None):
    g = torch.Generator(device="cuda").manual_seed(seed)
    H = torch.randn((M, K), generator=g, device="cuda").to(torch.bfloat16)
    w_std = 1.3 / np.sqrt(K) if w_std is None else w_std       # logits ~ N(0, 1.3^2), like 0.02 at K=4096
    W = (w_std * torch.randn((K, V), generator=g, device="cuda")).to(torch.bfloat16)
    tok = torch.randint(0, V, (M,), generator=g, device="cuda", dtype=torch.int32)
    return H, W, tok


@pytest.mark.parametrize("M,K,V", [(128, 64, 256), (256, 256, 1024), (200, 192, 1000), (384, 512, 1800),
                                   (130, 128, 4096 + 264), (1000, 64, 8)])
def test_lmhead_small_shapes_all_rows(P, oracle, M, K, V):
    H, W, tok = _inputs(M, K, V, seed=M + K + V)
    ws = P.new_workspace(P.lmhead_workspace_bytes(M, K, V))
    lp, ent, lse = P.lmhead_logprob_entropy(H, W, tok, 0.7, ws)
    torch.cuda.synchronize()
    assert P.last_device_status(ws) == 0
    rlp, rent, rlse = oracle.lmhead_logprob_entropy(host_logits(H), host_logits(W), npy(tok), np.float32(0.7))
    assert_abs(npy(lp), rlp, TOL_LOGPROB, "logprob")
    assert_abs(npy(ent), rent, TOL_LOGPROB, "entropy")
    assert_abs(npy(lse), rlse, TOL_LOGPROB, "lse")
    # same answer as the unfused path on logits rounded to bf16 is NOT expected (the fused path keeps
    # fp32 logits); but it must agree with step 1 on fp32 logits from a library matmul
    lg = (H.float() @ W.float()).contiguous()
    lp2, ent2, _ = P.logprob_entropy(lg, tok, 0.7)
    assert_abs(npy(lp), npy(lp2).astype(np.float64), 2e-4, "fused vs unfused logprob")
    assert_abs(npy(ent), npy(ent2).astype(np.float64), 2e-4, "fused vs unfused entropy")


def test_lmhead_mask_and_bad_token(P, oracle):
    M, K, V = 256, 128, 512
    H, W, tok = _inputs(M, K, V, seed=3)
    tok[5] = V
    tok[6] = -2
    mask = torch.ones(M, dtype=torch.uint8, device="cuda")
    mask[::3] = 0
    mask[5] = 1
    mask[6] = 1
    ws = P.new_workspace(P.lmhead_workspace_bytes(M, K, V))
    lp, ent, lse = P.lmhead_logprob_entropy(H, W, tok, 0.7, ws, mask=mask)
    rlp, rent, _ = oracle.lmhead_logprob_entropy(host_logits(H), host_logits(W), npy(tok).clip(0, V - 1), np.float32(0.7))
    m = npy(mask).astype(bool)
    ok = m.copy()
    ok[[5, 6]] = False
    assert_abs(npy(lp)[ok], rlp[ok], TOL_LOGPROB, "logprob")
    assert_abs(npy(ent)[ok], rent[ok], TOL_LOGPROB, "entropy")
    assert not npy(lp)[~m].any() and not npy(ent)[~m].any()
    assert torch.isnan(lp[5]) and torch.isnan(lp[6])
    assert P.last_device_status(ws) == 1


def test_lmhead_config4_full_size_sampled_rows(P, oracle):
    """[27136, 4096] x [4096, 50304] at full size; the oracle computes a sample of rows one by one."""
    from paper_2403_17031_b200.synthetic import CONFIGS, make_lmhead_batch
    cfg = CONFIGS[4]
    b = make_lmhead_batch(cfg, "cuda")
    M, K = b["H"].shape
    V = b["W"].shape[1]
    ws = P.new_workspace(P.lmhead_workspace_bytes(M, K, V))
    lp, ent, lse = P.lmhead_logprob_entropy(b["H"], b["W"], b["tokens"], cfg.hyper.temperature, ws)
    torch.cuda.synchronize()
    assert P.last_device_status(ws) == 0
    rng = np.random.default_rng(4)
    sel = np.sort(rng.choice(M, 40, replace=False)).astype(np.int64)
    sel[0], sel[-1] = 0, M - 1
    rlp, rent, rlse = oracle.lmhead_logprob_entropy(host_logits(b["H"]), host_logits(b["W"]), npy(b["tokens"]),
                                                    np.float32(cfg.hyper.temperature), sel_rows=sel)
    assert_abs(npy(lp)[sel], rlp, TOL_LOGPROB, "logprob (sampled)")
    assert_abs(npy(ent)[sel], rent, TOL_LOGPROB, "entropy (sampled)")
    assert_abs(npy(lse)[sel], rlse, TOL_LOGPROB, "lse (sampled)")
    assert torch.isfinite(lp).all() and torch.isfinite(ent).all()
    # properties that hold for every row: entropy within [0, ln V], log-prob <= 0
    assert float(ent.min()) >= 0.0 and float(ent.max()) <= np.log(V) + 1e-4 and float(lp.max()) <= 1e-5


@pytest.mark.parametrize("M,K,V,pattern", [(700, 128, 1000, "tails"), (700, 128, 1000, "random"), (300, 64, 520, "none"),
                                           (300, 64, 520, "all"), (5000, 64, 264, "one")])
def test_lmhead_mask_takes_rows_out_of_the_gemm(P, oracle, M, K, V, pattern):
    """With a mask (and more than one row tile) the call packs the rows with mask 1 and multiplies only those. Rows with
    mask 1 must carry the bits of the call without a mask (each logits row depends on its own row of H only), the
    others 0; repeated on one workspace, with a stale packed copy from a call with another mask in it."""
    H, W, tok = _inputs(M, K, V, seed=M + V)
    g = torch.Generator(device="cuda").manual_seed(7)
    if pattern == "tails":      # responses of 53 tokens, each real up to its own length: the shape of the PPO batch
        t = torch.arange(M, device="cuda") % 53
        L = torch.randint(1, 54, ((M + 52) // 53,), generator=g, device="cuda").repeat_interleave(53)[:M]
        mask = (t < L).to(torch.uint8)
    elif pattern == "random":
        mask = (torch.rand(M, generator=g, device="cuda") < 0.5).to(torch.uint8)
    elif pattern == "none":
        mask = torch.zeros(M, dtype=torch.uint8, device="cuda")
    elif pattern == "all":
        mask = torch.ones(M, dtype=torch.uint8, device="cuda")
    else:
        mask = torch.zeros(M, dtype=torch.uint8, device="cuda")
        mask[M - 3] = 1
    ws = P.new_workspace(P.lmhead_workspace_bytes(M, K, V))
    dense = [t.clone() for t in P.lmhead_logprob_entropy(H, W, tok, 0.7, ws)]
    other = (torch.rand(M, generator=g, device="cuda") < 0.8).to(torch.uint8)
    P.lmhead_logprob_entropy(H, W, tok, 0.7, ws, mask=other)      # leaves its packed rows behind
    m = mask.bool()
    for _ in range(2):
        got = P.lmhead_logprob_entropy(H, W, tok, 0.7, ws, mask=mask)
        torch.cuda.synchronize()
        for a, b, name in zip(got, dense, ("logprob", "entropy", "lse")):
            assert torch.equal(a[m], b[m]), name
            assert not a[~m].any(), name
    assert P.last_device_status(ws) == 0
    if m.any():
        sel = np.flatnonzero(npy(mask))[:64].astype(np.int64)
        rlp, rent, rlse = oracle.lmhead_logprob_entropy(host_logits(H), host_logits(W), npy(tok), np.float32(0.7),
                                                        sel_rows=sel)
        assert_abs(npy(got[0])[sel], rlp, TOL_LOGPROB, "logprob")
        assert_abs(npy(got[1])[sel], rent, TOL_LOGPROB, "entropy")
        assert_abs(npy(got[2])[sel], rlse, TOL_LOGPROB, "lse")


def test_lmhead_config4_full_size_with_the_eos_trick_mask(P, oracle):
    """Config 4 as the benchmark runs it: the call is given the mask of the EOS trick and multiplies the real rows
    only. Real rows: bits of the call without a mask, and a sample of them against the oracle; padding rows: 0."""
    from paper_2403_17031_b200.synthetic import CONFIGS, make_lmhead_batch
    cfg = CONFIGS[4]
    h = cfg.hyper
    b = make_lmhead_batch(cfg, "cuda")
    M, K = b["H"].shape
    V = b["W"].shape[1]
    _, _, _, mask, _ = P.truncate_and_score(b["responses"], b["scores"], h.eos_id, h.pad_id, h.no_eos_score)
    mask = mask.reshape(-1)
    tok = b["responses"].reshape(-1)
    ws = P.new_workspace(P.lmhead_workspace_bytes(M, K, V))
    dense = [t.clone() for t in P.lmhead_logprob_entropy(b["H"], b["W"], tok, h.temperature, ws)]
    got = P.lmhead_logprob_entropy(b["H"], b["W"], tok, h.temperature, ws, mask=mask)
    torch.cuda.synchronize()
    assert P.last_device_status(ws) == 0
    m = mask.bool()
    assert 0.3 * M < int(m.sum()) < 0.8 * M
    for a, d, name in zip(got, dense, ("logprob", "entropy", "lse")):
        assert torch.equal(a[m], d[m]), name
        assert not a[~m].any(), name
    rng = np.random.default_rng(6)
    real = np.flatnonzero(npy(mask))
    sel = np.sort(rng.choice(real, 24, replace=False)).astype(np.int64)
    sel[0], sel[-1] = real[0], real[-1]
    rlp, rent, rlse = oracle.lmhead_logprob_entropy(host_logits(b["H"]), host_logits(b["W"]), npy(tok),
                                                    np.float32(h.temperature), sel_rows=sel)
    assert_abs(npy(got[0])[sel], rlp, TOL_LOGPROB, "logprob (sampled)")
    assert_abs(npy(got[1])[sel], rent, TOL_LOGPROB, "entropy (sampled)")
    assert_abs(npy(got[2])[sel], rlse, TOL_LOGPROB, "lse (sampled)")


def test_config4_chained_path_against_the_oracle(P, oracle):
    """Config 4 as the benchmark times it, call by call: EOS trick -> fused LM head of policy and reference with the
    EOS-trick mask -> KL rewards -> GAE -> whitening -> loss at log-prob level. Log-probs and entropy on a row sample
    (the oracle forms each logits row by fp64 dot products), every [B,T] array of the later steps in full, each fed
    the GPU's own upstream fp32 values, and the loss through the oracle's own loss arithmetic."""
    from parity import TOL_REL, assert_rel, f32, near_kink
    from paper_2403_17031_b200 import binding
    from paper_2403_17031_b200.synthetic import CONFIGS, make_lmhead_batch
    cfg = CONFIGS[4]
    h = cfg.hyper
    p = binding.params_from(h)
    b = make_lmhead_batch(cfg, "cuda")
    M, K = b["H"].shape
    V = b["W"].shape[1]
    B, T = b["responses"].shape
    ws = P.new_workspace(max(P.lmhead_workspace_bytes(M, K, V), P.workspace_bytes(B, T, V)))
    tok = b["responses"].reshape(-1)
    ro, ei, sl, mask, so = P.truncate_and_score(b["responses"], b["scores"], h.eos_id, h.pad_id, h.no_eos_score)
    lp, ent, lse = P.lmhead_logprob_entropy(b["H"], b["W"], tok, h.temperature, ws, mask=mask.view(-1))
    rlp, _, _ = P.lmhead_logprob_entropy(b["H"], b["W_ref"], tok, h.temperature, ws, mask=mask.view(-1))
    lp, ent, rlp = lp.view(B, T), ent.view(B, T), rlp.view(B, T)
    kl, rew = P.kl_rewards(lp, rlp, mask, sl, so, h.kl_coef)
    adv, ret = P.gae(rew, b["values"], sl, h.gamma, h.lam)
    aw, st = P.whiten(adv, mask, True, h.whiten_eps, workspace=ws)
    old = (lp + b["old_logprob_noise"]).contiguous()
    out = P.loss_from_logprob(lp, ent, mask, old, aw, b["values_new"], b["values"], ret, p, ws)
    torch.cuda.synchronize()
    assert P.last_device_status(ws) == 0

    # EOS trick: exact
    resp = npy(b["responses"])
    o_ro, o_ei, o_sl, o_m, o_so = oracle.truncate_and_score(resp, h.eos_id, h.pad_id, npy(b["scores"]),
                                                           np.float32(h.no_eos_score))
    for got, want in ((ro, o_ro), (ei, o_ei), (sl, o_sl), (mask, o_m)):
        assert np.array_equal(npy(got), want)
    assert np.array_equal(npy(so).astype(np.float64), o_so)
    m = o_m.astype(bool)
    n = float(m.sum())
    # fused LM head on a sample of real rows, both weight matrices; padding rows are 0
    rng = np.random.default_rng(44)
    real = np.flatnonzero(m.reshape(-1)).astype(np.int64)
    sel = np.unique(np.concatenate([rng.choice(real, 96, replace=False), real[:1], real[-1:]]))
    Hh = host_logits(b["H"])
    tau = np.float32(h.temperature)
    o_lp, o_ent, _ = oracle.lmhead_logprob_entropy(Hh, host_logits(b["W"]), npy(tok), tau, sel_rows=sel)
    o_rlp, _, _ = oracle.lmhead_logprob_entropy(Hh, host_logits(b["W_ref"]), npy(tok), tau, sel_rows=sel)
    assert_abs(npy(lp).reshape(-1)[sel], o_lp, TOL_LOGPROB, "logprob (sampled)")
    assert_abs(npy(ent).reshape(-1)[sel], o_ent, TOL_LOGPROB, "entropy (sampled)")
    assert_abs(npy(rlp).reshape(-1)[sel], o_rlp, TOL_LOGPROB, "ref_logprob (sampled)")
    for t in (lp, ent, rlp):
        assert not npy(t)[~m].any()
        assert np.isfinite(npy(t)).all()
    # token-level steps in full
    o_kl, o_rew = oracle.kl_rewards(npy(lp), npy(rlp), o_m, o_sl, f32(o_so), np.float32(h.kl_coef))
    assert_abs(npy(kl), o_kl, TOL_LOGPROB, "kl")
    assert_rel(npy(rew), o_rew, TOL_REL, "rewards")
    o_adv, o_ret = oracle.gae(npy(rew), npy(b["values"]), o_sl, np.float32(h.gamma), np.float32(h.lam))
    assert_rel(npy(adv), o_adv, TOL_REL, "advantages")
    assert_rel(npy(ret), o_ret, TOL_REL, "returns")
    o_aw, o_st = oracle.whiten(npy(adv), o_m, True, np.float32(h.whiten_eps))
    assert_rel(npy(aw), o_aw, TOL_REL, "whitened advantages")
    assert_rel(npy(st), o_st, TOL_REL, "whiten stats")
    # the loss: a two-entry vocabulary (x, 0) at temperature 1 whose log-softmax at entry 0 is the given log-prob
    nlp = npy(lp).astype(np.float64)
    pt = np.exp(np.minimum(nlp, -1e-12))
    x = np.where(m, np.log(pt) - np.log1p(-pt), 0.0)
    ref = oracle.loss_fwd_bwd(np.stack([x, np.zeros_like(x)], -1).astype(np.float32), np.zeros((B, T), np.int32), o_m,
                              npy(old), npy(aw), npy(b["values_new"]), npy(b["values"]), npy(ret), 1.0,
                              np.float32(h.cliprange), np.float32(h.cliprange_value), np.float32(h.vf_coef),
                              want_dlogits=False)
    kink = near_kink(nlp, npy(old), h.cliprange) & m
    got = npy(out["losses"]).astype(np.float64)
    assert got[7] == n
    for i, name in enumerate(oracle.LOSS_NAMES[:6]):
        tol = TOL_LOGPROB + (int(kink.sum()) / n if name == "pg_clipfrac" else 0.0)
        assert abs(got[i] - ref["losses"][i]) <= tol, (name, got[i], ref["losses"][i])
    assert abs(got[6] - npy(ent).astype(np.float64)[m].sum() / n) <= 1e-5
    assert 0 < ref["losses"][4] < 1 and 0 < ref["losses"][5] < 1
    assert_abs(n * npy(out["dvalues"]), n * ref["dvalues"], 1e-4, "n*dvalues")
    assert_abs((n * npy(out["dlogprob"]).astype(np.float64))[~kink], (n * ref["dlogprob"])[~kink], 1e-4, "n*dlogprob")


def test_lmhead_step_and_host_step_match_the_separate_calls(P):
    """ppo_lmhead_step / ppo_lmhead_step_host only sequence the entry points of the fused-LM-head config: same bits as
    calling them one by one (the chained test above checks those against the oracle); the host variant copies in only the
    rows of H that the GEMMs read."""
    from paper_2403_17031_b200 import binding
    from paper_2403_17031_b200.synthetic import CONFIGS, make_lmhead_batch
    cfg = CONFIGS[4]
    h = cfg.hyper
    p = binding.params_from(h)
    B, T, K, V = 24, 53, 256, 2048
    b = make_lmhead_batch(cfg, "cuda", M=B * T, K=K, V=V)
    ws = P.new_workspace(max(P.lmhead_workspace_bytes(B * T, K, V), P.workspace_bytes(B, T, V)))
    tok = b["responses"].reshape(-1)
    ro, ei, sl, mask, so = P.truncate_and_score(b["responses"], b["scores"], h.eos_id, h.pad_id, h.no_eos_score)
    lp, ent, lse = P.lmhead_logprob_entropy(b["H"], b["W"], tok, h.temperature, ws, mask=mask.view(-1))
    rlp, _, _ = P.lmhead_logprob_entropy(b["H"], b["W_ref"], tok, h.temperature, ws, mask=mask.view(-1))
    lp, ent, lse, rlp = (t.view(B, T).clone() for t in (lp, ent, lse, rlp))
    kl, rew = P.kl_rewards(lp, rlp, mask, sl, so, h.kl_coef)
    adv, ret = P.gae(rew, b["values"], sl, h.gamma, h.lam)
    aw, st = P.whiten(adv, mask, True, h.whiten_eps, workspace=ws)
    old = (lp + b["old_logprob_noise"]).contiguous()
    want_loss = P.loss_from_logprob(lp, ent, mask, old, aw, b["values_new"], b["values"], ret, p, ws)
    want = {"responses_out": ro, "eos_index": ei, "seq_len": sl, "mask": mask, "scores_out": so, "logprob": lp, "entropy": ent,
            "lse": lse, "ref_logprob": rlp, "kl": kl, "rewards": rew, "advantages": adv, "returns": ret,
            "advantages_whitened": aw, "whiten_stats": st, "losses": want_loss["losses"], "dlogprob": want_loss["dlogprob"],
            "dvalues": want_loss["dvalues"]}
    torch.cuda.synchronize()
    inputs = {"H": b["H"], "W": b["W"], "W_ref": b["W_ref"], "responses": b["responses"], "scores": b["scores"],
              "values": b["values"], "values_new": b["values_new"], "old_logprob": old}
    out = {k: torch.full_like(v, 7) for k, v in want.items()}
    ws2 = P.new_workspace(max(P.lmhead_workspace_bytes(B * T, K, V), P.workspace_bytes(B, T, V)))
    io = binding.LMHeadStepIO.from_tensors({**inputs, **out, "workspace": ws2}, cuda=True)
    binding.lmhead_step(io, B, T, K, V, p)
    torch.cuda.synchronize()
    assert P.last_device_status(ws2) == 0
    for k in want:
        assert torch.equal(out[k], want[k]), k
    # host buffers in, host buffers out; the staging copy of H starts out as garbage behind the first EOS
    host_in = {k: v.cpu().pin_memory() for k, v in inputs.items()}
    host_out = {k: torch.empty_like(v, device="cpu").pin_memory() for k, v in want.items()}
    stage = {k: torch.empty_like(v) for k, v in inputs.items()}
    stage["H"].fill_(float("nan"))
    dev_out = {k: torch.full_like(v, 7) for k, v in want.items()}
    binding.lmhead_step_host(binding.LMHeadStepIO.from_tensors({**host_in, **host_out}, cuda=False),
                             binding.LMHeadStepIO.from_tensors({**stage, **dev_out, "workspace": ws2}, cuda=True),
                             B, T, K, V, p)
    for k in want:
        assert torch.equal(host_out[k], want[k].cpu()), k
    assert torch.isnan(stage["H"].view(B, T, K)[mask == 0]).all()       # padding rows of H were never copied
    # first-epoch default: no stored old log-probs -> ratio 1 -> nothing clipped
    io2 = binding.LMHeadStepIO.from_tensors({**{k: v for k, v in inputs.items() if k != "old_logprob"}, **out,
                                             "workspace": ws2}, cuda=True)
    binding.lmhead_step(io2, B, T, K, V, p)
    torch.cuda.synchronize()
    assert float(out["losses"][3]) == 0.0 and float(out["losses"][4]) == 0.0
