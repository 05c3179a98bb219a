"""GPU parity: every C-ABI call against the fp64 CPU oracle on the same seeded inputs.
Stage-wise (each GPU call is fed the oracle's upstream results rounded to fp32) and chained."""
import numpy as np
import pytest
import torch

from parity import (TOL_LOGPROB, TOL_REL, assert_abs, assert_grad, assert_rel, dev, f32, host_logits, near_kink,
                    npy, oracle_chain)

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def P():
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    import paper_2403_17031_b200 as pkg
    from paper_2403_17031_b200 import build
    build.build()
    pkg.lib()
    return pkg


def _params(P, h):
    from paper_2403_17031_b200 import binding
    return binding.params_from(h)


def _check_stagewise(P, O, cfg, batch, n_grad_rows=None, seed=0):
    """All six calls, each fed oracle upstream values; returns the oracle results."""
    h = cfg.hyper
    B, T, V = batch["policy_logits"].shape
    bf16 = batch["policy_logits"].dtype == torch.bfloat16
    rng = np.random.default_rng(seed)
    ref = oracle_chain(O, batch, h, want_dlogits=False, step1_mask=False)
    mask_np = ref["mask"].astype(bool)
    real_rows = np.flatnonzero(mask_np.reshape(-1))
    masked_rows = np.flatnonzero(~mask_np.reshape(-1))
    if n_grad_rows is None or n_grad_rows >= B * T:
        sel = np.arange(B * T)
    else:
        k_m = min(len(masked_rows), max(1, n_grad_rows // 8))
        sel = np.concatenate([rng.choice(real_rows, min(len(real_rows), n_grad_rows - k_m), replace=False),
                              rng.choice(masked_rows, k_m, replace=False) if k_m else np.empty(0, np.int64)])
        sel = np.sort(sel).astype(np.int64)
    ws = P.new_workspace(P.workspace_bytes(B, T, V))
    pp = _params(P, h)

    # step 2 (integers: exact)
    ro, ei, sl, m, so = P.truncate_and_score(batch["responses"], batch["scores"], h.eos_id, h.pad_id, h.no_eos_score)
    assert np.array_equal(npy(ro), ref["responses_out"]) and np.array_equal(npy(ei), ref["eos_index"])
    assert np.array_equal(npy(sl), ref["seq_len"]) and np.array_equal(npy(m), ref["mask"])
    assert np.array_equal(npy(so).astype(np.float64), ref["scores_out"])

    # step 1, policy and reference; also with the mask (rows skipped -> 0)
    lp, ent, lse = P.logprob_entropy(batch["policy_logits"], batch["responses"], h.temperature, workspace=ws,
                                     want_lse=True)
    assert_abs(npy(lp), ref["logprob"], TOL_LOGPROB, "logprob")
    assert_abs(npy(ent), ref["entropy"], TOL_LOGPROB, "entropy")
    rlp, _, _ = P.logprob_entropy(batch["ref_logits"], batch["responses"], h.temperature, workspace=ws,
                                  want_entropy=False)
    assert_abs(npy(rlp), ref["ref_logprob"], TOL_LOGPROB, "ref_logprob")
    lpm, entm, _ = P.logprob_entropy(batch["policy_logits"], batch["responses"], h.temperature, mask=m, workspace=ws)
    assert_abs(npy(lpm), ref["logprob"] * mask_np, TOL_LOGPROB, "masked logprob")
    assert not npy(lpm)[~mask_np].any() and not npy(entm)[~mask_np].any()

    # step 3
    kl, rew = P.kl_rewards(dev(f32(ref["logprob"])), dev(f32(ref["ref_logprob"])), dev(ref["mask"]),
                           dev(ref["seq_len"]), dev(f32(ref["scores_out"])), h.kl_coef)
    assert_abs(npy(kl), ref["kl"], TOL_LOGPROB, "kl")
    assert_rel(npy(rew), ref["rewards"], TOL_REL, "rewards")

    # step 4
    adv, ret = P.gae(dev(f32(ref["rewards"])), batch["values"], dev(ref["seq_len"]), h.gamma, h.lam)
    assert_rel(npy(adv), ref["advantages"], TOL_REL, "advantages")
    assert_rel(npy(ret), ref["returns"], TOL_REL, "returns")

    # step 5
    aw, st = P.whiten(dev(f32(ref["advantages"])), dev(ref["mask"]), True, h.whiten_eps, workspace=ws)
    assert_rel(npy(aw), ref["advantages_whitened"], TOL_REL, "whitened advantages")
    assert_rel(npy(st), ref["whiten_stats"], TOL_REL, "whiten stats")
    assert not npy(aw)[~mask_np].any()

    # step 6
    o_ref = O.loss_fwd_bwd(host_logits(batch["policy_logits"]), npy(batch["responses"]), ref["mask"],
                           ref["old_logprob"], f32(ref["advantages_whitened"]), npy(batch["values_new"]),
                           npy(batch["values"]), f32(ref["returns"]), np.float32(h.temperature),
                           np.float32(h.cliprange), np.float32(h.cliprange_value), np.float32(h.vf_coef),
                           want_dlogits=True, sel_rows=sel)
    out = P.loss_fwd_bwd(batch["policy_logits"], batch["responses"], dev(ref["mask"]), dev(ref["old_logprob"]),
                         dev(f32(ref["advantages_whitened"])), batch["values_new"], batch["values"],
                         dev(f32(ref["returns"])), pp, ws)
    n = o_ref["losses"][7]
    kink = near_kink(o_ref["new_logprob"], ref["old_logprob"], h.cliprange) & mask_np
    n_kink = int(kink.sum())
    got_l = npy(out["losses"]).astype(np.float64)
    assert got_l[7] == n
    for i, name in enumerate(O.LOSS_NAMES[:7]):
        tol = TOL_LOGPROB + (n_kink / n if name == "pg_clipfrac" else 0.0)
        assert abs(got_l[i] - o_ref["losses"][i]) <= tol, (name, got_l[i], o_ref["losses"][i])
    assert_abs(npy(out["new_logprob"]), o_ref["new_logprob"], TOL_LOGPROB, "new_logprob")
    assert_abs(npy(out["entropy"]), o_ref["entropy"], TOL_LOGPROB, "loss entropy")
    assert_abs(n * npy(out["dvalues"]), n * o_ref["dvalues"], 1e-4, "n*dvalues")
    g_got, g_ref = n * npy(out["dlogprob"]).astype(np.float64), n * o_ref["dlogprob"]
    assert_abs(g_got[~kink], g_ref[~kink], 1e-4, "n*dlogprob")
    dl = out["dlogits"].reshape(B * T, V)[torch.from_numpy(sel).cuda()]
    dl = n * (dl.float().cpu().numpy().astype(np.float64))
    keep = ~kink.reshape(-1)[sel]
    assert_grad(dl[keep], n * o_ref["dlogits"][keep], bf16, "n*dlogits")
    assert not dl[~mask_np.reshape(-1)[sel]].any(), "masked rows of dlogits must be zero"
    # every selected real row of dlogits sums to ~0
    assert np.abs(dl.sum(1)).max() < (2e-2 if bf16 else 1e-3)
    # both clip branches were exercised by the data
    assert 0 < o_ref["losses"][4] < 1 and 0 < o_ref["losses"][5] < 1
    assert P.last_device_status(ws) == 0
    return ref, o_ref


def test_config0_tiny_all_steps(P, oracle):
    from paper_2403_17031_b200.synthetic import CONFIGS, make_batch
    cfg = CONFIGS[0]
    batch = make_batch(cfg, "cuda")
    _check_stagewise(P, oracle, cfg, batch)


def test_config0_chained_end_to_end(P, oracle):
    from paper_2403_17031_b200.pipeline import PPOHotPath
    from paper_2403_17031_b200.synthetic import CONFIGS, make_batch
    cfg = CONFIGS[0]
    h = cfg.hyper
    batch = make_batch(cfg, "cuda")
    ref = oracle_chain(oracle, batch, h)
    hp = PPOHotPath(cfg.B, cfg.T, cfg.V, torch.float32, _params(P, h))
    o = hp.rollout_stats(batch["policy_logits"], batch["ref_logits"], batch["responses"], batch["scores"],
                         batch["values"])
    old = (o["logprob"] + batch["old_logprob_noise"]).contiguous()
    o = hp.loss(batch["policy_logits"], batch["responses"], old, batch["values_new"], batch["values"])
    torch.cuda.synchronize()
    for k in ("responses_out", "eos_index", "seq_len", "mask"):
        assert np.array_equal(npy(o[k]), ref[k]), k
    for k in ("logprob", "entropy", "ref_logprob", "kl"):
        assert_abs(npy(o[k]), ref[k], TOL_LOGPROB, k)
    # chained: upstream fp32 errors (<=1e-4 on log-probs, times kl_coef) propagate
    for k in ("rewards", "advantages", "returns"):
        assert_rel(npy(o[k]), ref[k], 2e-5, k)
    assert_rel(npy(o["advantages_whitened"]), ref["advantages_whitened"], 5e-5, "advantages_whitened")
    n = ref["loss"]["losses"][7]
    kink = near_kink(ref["loss"]["new_logprob"], ref["old_logprob"], h.cliprange).any()
    if not kink:
        assert_abs(npy(o["losses"]), ref["loss"]["losses"], 2e-4, "losses")
        assert_abs(n * npy(o["dlogits"]).reshape(-1, cfg.V), n * ref["loss"]["dlogits"], 5e-4, "n*dlogits")
        assert_abs(n * npy(o["dvalues"]), n * ref["loss"]["dvalues"], 2e-4, "n*dvalues")
    assert hp.device_status() == 0


def test_config1_pythia_rollout_shape(P, oracle):
    from paper_2403_17031_b200.synthetic import CONFIGS, make_batch
    cfg = CONFIGS[1]
    batch = make_batch(cfg, "cuda")
    _check_stagewise(P, oracle, cfg, batch, n_grad_rows=96)


def test_config2_full_ppo_batch_every_row(P, oracle):
    """B=512 at full size, through the separate calls and through the single-call step the benchmark times: integer
    steps exact; log-probs and entropy of every real row of both tensors against the oracle; every [B,T] array; the
    loss scalars and per-token gradients of every row through the oracle's own loss; every gradient row validated
    on the device; a sample of gradient rows element by element."""
    from paper_2403_17031_b200.synthetic import CONFIGS, make_batch
    cfg = CONFIGS[2]
    batch = make_batch(cfg, "cuda")
    _check_full_size(P, oracle, cfg, batch, n_grad_rows=160, seed=2)


def test_config3_long_response_stress_every_row(P, oracle):
    """B=256, T=512, fp32 logits (26 GB per tensor): the same checks as config 2 at full size."""
    from paper_2403_17031_b200.synthetic import CONFIGS, make_batch
    cfg = CONFIGS[3]
    free, _ = torch.cuda.mem_get_info()
    if free < 100e9:
        pytest.skip("needs ~90 GB of free device memory")
    batch = make_batch(cfg, "cuda", chunk_rows=4096)
    _check_full_size(P, oracle, cfg, batch, n_grad_rows=512, seed=3)


def test_config3_shape_small_batch_all_steps(P, oracle):
    """Config 3's shape (T=512, fp32, gamma=0.99) at B=4 so that every output is compared."""
    from paper_2403_17031_b200.synthetic import CONFIGS, make_batch
    cfg = CONFIGS[3]
    batch = make_batch(cfg, "cuda", B=4)
    from dataclasses import replace
    _check_stagewise(P, oracle, replace(cfg, B=4), batch, n_grad_rows=48)


_STEP_OUTPUTS = ("responses_out", "eos_index", "seq_len", "mask", "scores_out", "logprob", "entropy", "ref_logprob", "kl",
                 "rewards", "advantages", "returns", "advantages_whitened", "losses", "dvalues", "new_logprob",
                 "new_entropy", "dlogprob")


def _poison(hp):
    """Fill every output with a pattern no kernel writes: a row that a launch skipped stays visible."""
    for k, t in hp.out.items():
        if t is None or k == "whiten_stats":
            continue
        if t.is_floating_point():
            t.fill_(float("nan"))
        else:
            t.fill_(-77 if t.dtype != torch.uint8 else 201)


def _row_checksums(dl, chunk=4096):
    """One int64 per gradient row: the sum of the row's bit patterns (any changed bit changes it)."""
    rows = dl.shape[0]
    out = torch.empty(rows, dtype=torch.int64, device=dl.device)
    it = torch.int16 if dl.dtype == torch.bfloat16 else torch.int32
    for r0 in range(0, rows, chunk):
        out[r0:r0 + chunk] = dl[r0:r0 + chunk].view(it).sum(-1, dtype=torch.int64)
    return out


def _oracle_logprob_rows(O, logits2d, rows_idx, tokens, tau, chunk=4096):
    """The oracle's step 1 on the given rows of a device tensor [rows, V], copied to the host chunk by chunk."""
    lp = np.empty(len(rows_idx)); ent = np.empty(len(rows_idx))
    for i0 in range(0, len(rows_idx), chunk):
        idx = rows_idx[i0:i0 + chunk]
        x = host_logits(logits2d[torch.from_numpy(idx).to(logits2d.device)])
        lp[i0:i0 + chunk], ent[i0:i0 + chunk], _ = O.logprob_entropy(x, tokens[idx], tau)
    return lp, ent


def _check_full_size(P, O, cfg, batch, n_grad_rows, seed):
    from paper_2403_17031_b200.pipeline import PPOHotPath
    h = cfg.hyper
    B, T, V = batch["policy_logits"].shape
    rows = B * T
    bf16 = batch["policy_logits"].dtype == torch.bfloat16
    rng = np.random.default_rng(seed)
    tau = np.float32(h.temperature)
    hp = PPOHotPath(B, T, V, batch["policy_logits"].dtype, _params(P, h))
    args = (batch["policy_logits"], batch["ref_logits"], batch["responses"], batch["scores"], batch["values"])

    # ---- the separate calls
    _poison(hp)
    o = hp.rollout_stats(*args)
    old = (o["logprob"] + batch["old_logprob_noise"]).contiguous()
    o = hp.loss(batch["policy_logits"], batch["responses"], old, batch["values_new"], batch["values"])
    torch.cuda.synchronize()
    assert hp.device_status() == 0
    sep = {k: o[k].clone() for k in _STEP_OUTPUTS}
    dl2 = o["dlogits"].view(rows, V)
    sep_sums = _row_checksums(dl2)

    # ---- integer step: exact, everywhere
    resp = npy(batch["responses"])
    ro, ei, sl, m, so = O.truncate_and_score(resp, h.eos_id, h.pad_id, npy(batch["scores"]), np.float32(h.no_eos_score))
    for k, want in (("responses_out", ro), ("eos_index", ei), ("seq_len", sl), ("mask", m)):
        assert np.array_equal(npy(o[k]), want), k
    assert np.array_equal(npy(o["scores_out"]).astype(np.float64), so)
    mask_np = m.astype(bool)
    flat_mask = mask_np.reshape(-1)
    n = float(mask_np.sum())
    assert float(o["losses"][7]) == n
    real = np.flatnonzero(flat_mask).astype(np.int64)
    masked = np.flatnonzero(~flat_mask).astype(np.int64)

    # ---- step 1 on EVERY real row of both tensors (and the loss kernel's own log-prob / entropy of the policy rows)
    tok_flat = resp.reshape(-1)
    lp, ent = _oracle_logprob_rows(O, batch["policy_logits"].view(rows, V), real, tok_flat, tau)
    rlp, _ = _oracle_logprob_rows(O, batch["ref_logits"].view(rows, V), real, tok_flat, tau)
    pick = lambda name: npy(o[name]).reshape(-1)
    assert_abs(pick("logprob")[real], lp, TOL_LOGPROB, "logprob (every real row)")
    assert_abs(pick("entropy")[real], ent, TOL_LOGPROB, "entropy (every real row)")
    assert_abs(pick("ref_logprob")[real], rlp, TOL_LOGPROB, "ref_logprob (every real row)")
    assert_abs(pick("new_logprob")[real], lp, TOL_LOGPROB, "new_logprob (every real row)")
    assert_abs(pick("new_entropy")[real], ent, TOL_LOGPROB, "new_entropy (every real row)")
    for k in ("logprob", "entropy", "ref_logprob", "new_logprob", "new_entropy", "dlogprob", "dvalues"):
        assert not pick(k)[masked].any(), k + " must be 0 on padding rows"

    # ---- token-level steps: whole arrays, each fed the GPU's own upstream fp32 outputs
    kl, rew = O.kl_rewards(npy(o["logprob"]), npy(o["ref_logprob"]), m, sl, f32(so), np.float32(h.kl_coef))
    assert_abs(npy(o["kl"]), kl, TOL_LOGPROB, "kl")
    assert_rel(npy(o["rewards"]), rew, TOL_REL, "rewards")
    adv, ret = O.gae(npy(o["rewards"]), npy(batch["values"]), sl, np.float32(h.gamma), np.float32(h.lam))
    assert_rel(npy(o["advantages"]), adv, TOL_REL, "advantages")
    assert_rel(npy(o["returns"]), ret, TOL_REL, "returns")
    aw, st = O.whiten(npy(o["advantages"]), m, True, np.float32(h.whiten_eps))
    assert_rel(npy(o["advantages_whitened"]), aw, TOL_REL, "whitened advantages")

    # ---- loss scalars and per-token gradients of EVERY row through the oracle's own loss: a two-entry
    # vocabulary (x, 0) at temperature 1 whose log-softmax at entry 0 is the GPU's new_logprob (x = logit(p))
    nlp_gpu = npy(o["new_logprob"]).astype(np.float64)
    p_tok = np.exp(np.minimum(nlp_gpu, -1e-12))
    x = np.where(mask_np, np.log(p_tok) - np.log1p(-p_tok), 0.0)
    lg2 = np.stack([x, np.zeros_like(x)], -1)
    # (the oracle widens fp32 logits; x in fp32 moves new_logprob by <= 6e-8 * |x|, far inside the tolerance)
    old_np = npy(old)
    ref2 = O.loss_fwd_bwd(lg2.astype(np.float32), np.zeros((B, T), np.int32), m, old_np, npy(o["advantages_whitened"]),
                          npy(batch["values_new"]), npy(batch["values"]), npy(o["returns"]), 1.0,
                          np.float32(h.cliprange), np.float32(h.cliprange_value), np.float32(h.vf_coef),
                          want_dlogits=False)
    assert_abs(ref2["new_logprob"][mask_np], nlp_gpu[mask_np], 2e-5, "two-entry construction reproduces new_logprob")
    kink = near_kink(nlp_gpu, old_np, h.cliprange) & mask_np
    got_l = npy(o["losses"]).astype(np.float64)
    for i, name in enumerate(O.LOSS_NAMES[:6]):
        tol = TOL_LOGPROB + (int(kink.sum()) / n if name == "pg_clipfrac" else 0.0)
        assert abs(got_l[i] - ref2["losses"][i]) <= tol, (name, got_l[i], ref2["losses"][i])
    assert abs(got_l[6] - ent.sum() / n) <= TOL_LOGPROB, "mean entropy"
    assert 0 < ref2["losses"][4] < 1 and 0 < ref2["losses"][5] < 1          # both clip branches fire
    assert_abs(n * npy(o["dvalues"]), n * ref2["dvalues"], 1e-4, "n*dvalues (every row)")
    assert_abs((n * npy(o["dlogprob"]).astype(np.float64))[~kink], (n * ref2["dlogprob"])[~kink], 1e-4,
               "n*dlogprob (every row)")

    # ---- every gradient row, on the device: finite; padding rows all zero; a real row sums to ~0, its entry at
    # the sampled token is g/tau * (1 - p_tok), and its absolute values sum to 2 |g|/tau (1 - p_tok)
    tok_d = batch["responses"].reshape(-1).long()
    g_d = o["dlogprob"].reshape(-1).double() / float(tau)
    onem_p = -torch.expm1(o["new_logprob"].reshape(-1).double())
    mask_d = o["mask"].reshape(-1).bool()
    # tolerances: one rounding to the output type (2^-9 relative for bf16) on every entry, plus the fp32 evaluation
    # error of the probabilities (a few 1e-6 of |g|/tau, which matters where 1 - p_tok is tiny)
    rel = 2.0 ** -7 if bf16 else 1e-4
    for r0 in range(0, rows, 4096):
        c = dl2[r0:r0 + 4096]
        mk = mask_d[r0:r0 + 4096]
        assert bool(torch.isfinite(c).all()), "non-finite gradient rows in [%d, %d)" % (r0, r0 + 4096)
        cd = c.double()
        assert not bool(cd[~mk].any()), "padding rows of dlogits must be zero"
        want_tok = (g_d[r0:r0 + 4096] * onem_p[r0:r0 + 4096])
        got_tok = cd.gather(1, tok_d[r0:r0 + 4096, None])[:, 0]
        scale = n * want_tok.abs()
        slack = 1e-5 * n * g_d[r0:r0 + 4096].abs()
        assert bool(((n * (got_tok - want_tok)).abs() <= rel * scale + slack + 1e-6)[mk].all()), \
            "dlogits at the sampled token"
        assert bool(((n * cd.sum(1)).abs() <= rel * scale + slack + 1e-4)[mk].all()), "row sums"
        assert bool(((n * cd.abs().sum(1) - 2 * scale).abs() <= 2 * (rel * scale + slack) + 1e-4)[mk].all()), \
            "row L1 norms"
        del cd

    # ---- a sample of gradient rows element by element: the oracle runs on the sample as a [1, k, V] batch, whose
    # normaliser is k instead of n, so n*gradient of the full batch equals k*gradient of the sample
    first_last = np.array([real[0], real[-1], real[real < T][-1], real[real >= (B - 1) * T][0]], np.int64)
    sel = np.unique(np.concatenate([rng.choice(real, min(n_grad_rows, len(real)), replace=False), first_last]))
    sel_t = torch.from_numpy(sel).cuda()
    k = len(sel)
    pl = host_logits(batch["policy_logits"].view(rows, V)[sel_t])
    pk = lambda name: pick(name)[sel][None]
    sub = O.loss_fwd_bwd(pl[None], tok_flat[sel][None], np.ones((1, k), np.uint8), old_np.reshape(-1)[sel][None],
                         pk("advantages_whitened"), npy(batch["values_new"]).reshape(-1)[sel][None],
                         npy(batch["values"]).reshape(-1)[sel][None], pk("returns"), tau,
                         np.float32(h.cliprange), np.float32(h.cliprange_value), np.float32(h.vf_coef))
    kk = near_kink(sub["new_logprob"], old_np.reshape(-1)[sel][None], h.cliprange).reshape(-1)
    dl = n * dl2[sel_t].float().cpu().numpy().astype(np.float64)
    assert_grad(dl[~kk], k * sub["dlogits"][~kk], bf16, "n*dlogits (sampled rows)")

    # ---- the log-prob-level entry point on the same per-token inputs: same bits
    o2 = P.loss_from_logprob(o["new_logprob"], o["new_entropy"], o["mask"], old, o["advantages_whitened"],
                             batch["values_new"], batch["values"], o["returns"], _params(P, h), hp.workspace)
    assert torch.equal(o2["losses"], o["losses"]) and torch.equal(o2["dvalues"], o["dvalues"])
    assert torch.equal(o2["dlogprob"], o["dlogprob"])

    # ---- the single-call step (the launch configuration the benchmark times: overlapped launches, dynamic row
    # hand-out), eager and as a replayed CUDA graph, then a later epoch: every output bit equal to the separate calls
    step_args = args + (batch["values_new"],)
    for how in ("eager", "graph", "next_epoch"):
        _poison(hp)
        if how == "eager":
            hp.step(*step_args, old_logprob=old)
        elif how == "graph":
            graph = hp.capture_step(*step_args, old_logprob=old)
            _poison(hp)
            graph.replay()
        else:
            hp.step(*step_args, old_logprob=old)
            for name in ("losses", "dlogits", "dvalues", "new_logprob", "new_entropy", "dlogprob"):
                hp.out[name].fill_(float("nan"))
            hp.loss(batch["policy_logits"], batch["responses"], old, batch["values_new"], batch["values"],
                    next_epoch=True)
        torch.cuda.synchronize()
        assert hp.device_status() == 0, how
        names = _STEP_OUTPUTS if how != "next_epoch" else ("losses", "dvalues", "new_logprob", "new_entropy", "dlogprob")
        for name in names:
            assert torch.equal(hp.out[name], sep[name]), (name, how)
        assert torch.equal(_row_checksums(hp.out["dlogits"].view(rows, V)), sep_sums), ("dlogits", how)


def test_single_call_step_and_host_step_match_the_separate_calls(P):
    """ppo_step / ppo_step_host only sequence the per-step entry points: same bits as calling them one by one."""
    from paper_2403_17031_b200 import binding
    from paper_2403_17031_b200.pipeline import PPOHotPath
    from paper_2403_17031_b200.synthetic import CONFIGS, make_batch
    cfg = CONFIGS[0]
    batch = make_batch(cfg, "cuda")
    pp = _params(P, cfg.hyper)
    names = ("mask", "seq_len", "logprob", "entropy", "ref_logprob", "kl", "rewards", "advantages", "returns",
             "advantages_whitened", "losses", "dlogits", "dvalues", "new_logprob", "dlogprob")
    a = PPOHotPath(cfg.B, cfg.T, cfg.V, torch.float32, pp)
    o = a.rollout_stats(batch["policy_logits"], batch["ref_logits"], batch["responses"], batch["scores"], batch["values"])
    old = (o["logprob"] + batch["old_logprob_noise"]).contiguous()
    a.loss(batch["policy_logits"], batch["responses"], old, batch["values_new"], batch["values"])
    b = PPOHotPath(cfg.B, cfg.T, cfg.V, torch.float32, pp)
    b.step(batch["policy_logits"], batch["ref_logits"], batch["responses"], batch["scores"], batch["values"],
           batch["values_new"], old_logprob=old)
    torch.cuda.synchronize()
    for k in names:
        assert torch.equal(a.out[k], b.out[k]), k
    # host buffers in, host buffers out
    c = PPOHotPath(cfg.B, cfg.T, cfg.V, torch.float32, pp)
    inp = {"policy_logits": batch["policy_logits"], "ref_logits": batch["ref_logits"], "responses": batch["responses"],
           "scores": batch["scores"], "values": batch["values"], "values_new": batch["values_new"], "old_logprob": old}
    host_in = {k: v.cpu().pin_memory() for k, v in inp.items()}
    host_out = {k: torch.empty_like(c.out[k], device="cpu").pin_memory() for k in names}
    stage = {k: torch.empty_like(v, device="cuda") for k, v in host_in.items()}
    binding.step_host(binding.PPOStepIO.from_tensors({**host_in, **host_out}, cuda=False), c.step_io(stage),
                      torch.float32, cfg.B, cfg.T, cfg.V, pp)
    for k in names:
        assert torch.equal(host_out[k], a.out[k].cpu()), k
    # first-epoch default: no stored old log-probs -> ratio 1 -> nothing clipped
    b.step(batch["policy_logits"], batch["ref_logits"], batch["responses"], batch["scores"], batch["values"],
           batch["values_new"])
    torch.cuda.synchronize()
    assert float(b.out["losses"][3]) == 0.0 and float(b.out["losses"][4]) == 0.0


@pytest.mark.parametrize("B,T,V", [(4, 16, 1000), (70, 53, 1000)])
def test_reward_whitening_before_gae(P, oracle, B, T, V):
    """Detail "(Optional) Reward whitening": whiten(rewards, shift_mean=False) over the batch's real tokens before
    GAE. Stage-wise against the oracle, ppo_step against the separate calls (same bits) and against the oracle chain."""
    import dataclasses
    from paper_2403_17031_b200.pipeline import PPOHotPath
    from paper_2403_17031_b200.synthetic import CONFIGS, make_batch
    cfg = dataclasses.replace(CONFIGS[0], B=B, T=T, V=V,
                              hyper=dataclasses.replace(CONFIGS[0].hyper, whiten_rewards=1))
    h = cfg.hyper
    batch = make_batch(cfg, "cuda")
    ref = oracle_chain(oracle, batch, h, want_dlogits=False)
    off = oracle_chain(oracle, batch, dataclasses.replace(h, whiten_rewards=0), want_dlogits=False)
    assert np.abs(ref["rewards"] - off["rewards"]).max() > 1e-2      # the option changes the rewards ...
    m = ref["mask"].astype(bool)
    assert abs(ref["rewards"][m].mean() - off["rewards"][m].mean()) < 1e-7   # ... but not their mean (fp32 inputs)
    assert abs(ref["rewards"][m].var() - 1.0) < 1e-5                          # and the variance becomes 1
    # stage-wise: the whitening call on the oracle's raw rewards, GAE on the oracle's whitened rewards
    rw, _ = P.whiten(dev(f32(off["rewards"])), dev(ref["mask"]), False, h.whiten_eps)
    assert_rel(npy(rw), ref["rewards"], TOL_REL, "whitened rewards")
    adv, ret = P.gae(dev(f32(ref["rewards"])), batch["values"], dev(ref["seq_len"]), h.gamma, h.lam)
    assert_rel(npy(adv), ref["advantages"], TOL_REL, "advantages")
    assert_rel(npy(ret), ref["returns"], TOL_REL, "returns")
    # ppo_step == separate calls, bit for bit
    pp = _params(P, h)
    assert pp.whiten_rewards == 1
    a = PPOHotPath(B, T, V, torch.float32, pp)
    o = a.rollout_stats(batch["policy_logits"], batch["ref_logits"], batch["responses"], batch["scores"],
                        batch["values"])
    old = (o["logprob"] + batch["old_logprob_noise"]).contiguous()
    a.loss(batch["policy_logits"], batch["responses"], old, batch["values_new"], batch["values"])
    b = PPOHotPath(B, T, V, torch.float32, pp)
    b.step(batch["policy_logits"], batch["ref_logits"], batch["responses"], batch["scores"], batch["values"],
           batch["values_new"], old_logprob=old)
    torch.cuda.synchronize()
    for k in ("mask", "seq_len", "kl", "rewards", "advantages", "returns", "advantages_whitened", "losses", "dlogits",
              "dvalues"):
        assert torch.equal(a.out[k], b.out[k]), k
    # chained against the oracle: fp32 log-prob errors (<= 1e-4, times kl_coef) are divided by the rewards'
    # standard deviation and summed by GAE
    assert_rel(npy(b.out["rewards"]), ref["rewards"], 1e-4, "rewards (chained)")
    for k in ("advantages", "returns"):
        assert_rel(npy(b.out[k]), ref[k], 5e-4, k + " (chained)")
    assert_rel(npy(b.out["advantages_whitened"]), ref["advantages_whitened"], 5e-4, "advantages_whitened (chained)")
    assert b.device_status() == 0


@pytest.mark.parametrize("B,T,V,dtype", [(64, 53, 50304, "bf16"), (150, 53, 2048, "bf16"), (5, 16, 1001, "f32"),
                                         (40, 512, 1000, "f32")])
def test_step_overlapped_launches_repeatable(P, B, T, V, dtype):
    """ppo_step's launches overlap (the loss kernel starts while the token-level kernel runs, that one while the
    log-prob kernel drains) and hand results over through flags in the workspace. Repeated calls, eager and as a
    replayed CUDA graph, must give the bits of the separate calls every time; V = 1001 takes the path without
    16-byte packs (two log-prob launches, direct-load loss kernels)."""
    import dataclasses
    from paper_2403_17031_b200.pipeline import PPOHotPath
    from paper_2403_17031_b200.synthetic import CONFIGS, make_batch
    cfg = dataclasses.replace(CONFIGS[0], B=B, T=T, V=V, dtype=dtype, n_no_eos_exact=None)
    batch = make_batch(cfg, "cuda")
    pp = _params(P, cfg.hyper)
    names = ("mask", "seq_len", "logprob", "entropy", "ref_logprob", "kl", "rewards", "advantages", "returns",
             "advantages_whitened", "losses", "dlogits", "dvalues", "new_logprob", "dlogprob")
    a = PPOHotPath(B, T, V, cfg.torch_dtype, pp)
    o = a.rollout_stats(batch["policy_logits"], batch["ref_logits"], batch["responses"], batch["scores"], batch["values"])
    old = (o["logprob"] + batch["old_logprob_noise"]).contiguous()
    a.loss(batch["policy_logits"], batch["responses"], old, batch["values_new"], batch["values"])
    torch.cuda.synchronize()
    want = {k: a.out[k].clone() for k in names}
    b = PPOHotPath(B, T, V, cfg.torch_dtype, pp)
    args = (batch["policy_logits"], batch["ref_logits"], batch["responses"], batch["scores"], batch["values"],
            batch["values_new"])
    for it in range(3):
        for k in names:
            b.out[k].fill_(7)                      # stale contents must not survive
        b.step(*args, old_logprob=old)
        torch.cuda.synchronize()
        for k in names:
            assert torch.equal(b.out[k], want[k]), (k, "eager", it)
    graph = b.capture_step(*args, old_logprob=old)
    for it in range(3):
        for k in names:
            b.out[k].fill_(7)
        graph.replay()
        torch.cuda.synchronize()
        for k in names:
            assert torch.equal(b.out[k], want[k]), (k, "graph", it)
    assert b.device_status() == 0


@pytest.mark.parametrize("B,T,V,dtype", [(70, 53, 2048, "bf16"), (6, 16, 1001, "f32")])
def test_step_never_reads_padding_rows(P, B, T, V, dtype):
    """Everything after a response's first EOS is padding (EOS trick): the whole-path call must not read those rows
    of any logits tensor. NaN planted there changes no output bit and raises no status; V = 1001 takes the path
    without 16-byte packs."""
    import dataclasses
    from paper_2403_17031_b200.pipeline import PPOHotPath
    from paper_2403_17031_b200.synthetic import CONFIGS, make_batch
    cfg = dataclasses.replace(CONFIGS[0], B=B, T=T, V=V, dtype=dtype, n_no_eos_exact=None)
    batch = make_batch(cfg, "cuda")
    pp = _params(P, cfg.hyper)
    names = ("mask", "seq_len", "logprob", "entropy", "ref_logprob", "kl", "rewards", "advantages", "returns",
             "advantages_whitened", "losses", "dlogits", "dvalues", "new_logprob", "dlogprob")
    args = lambda pl, rl: (pl, rl, batch["responses"], batch["scores"], batch["values"], batch["values_new"])
    a = PPOHotPath(B, T, V, cfg.torch_dtype, pp)
    a.step(*args(batch["policy_logits"], batch["ref_logits"]))
    torch.cuda.synchronize()
    pad = a.out["mask"] == 0
    assert pad.any() and not pad.all()
    for k in ("logprob", "entropy", "ref_logprob", "kl", "rewards", "advantages", "advantages_whitened"):
        assert not a.out[k][pad].any(), k
    assert not a.out["dlogits"][pad].any()
    poisoned = []
    for k in ("policy_logits", "ref_logits"):
        t = batch[k].clone()
        t[pad] = float("nan")
        poisoned.append(t)
    b = PPOHotPath(B, T, V, cfg.torch_dtype, pp)
    b.step(*args(*poisoned))
    torch.cuda.synchronize()
    for k in names:
        assert torch.equal(a.out[k], b.out[k]), k
    assert b.device_status() == 0


@pytest.mark.parametrize("B,T,V,dtype", [(64, 53, 50304, "bf16"), (37, 53, 2048, "bf16"), (5, 16, 1001, "f32")])
def test_loss_next_epoch_reuses_the_row_order(P, B, T, V, dtype):
    """Later PPO epochs of a batch (4 per batch in the paper's table) call the loss again on new logits with the same
    mask: ppo_loss_fwd_bwd_next_epoch skips the prologue launch and must give the bits of the full call - after a
    loss call, after another next-epoch call and after ppo_step. Told to reuse an order that was built from another
    mask tensor, or that a fused LM-head call has overwritten, it must write nothing and raise PPO_DEV_BAD_REUSE."""
    import dataclasses
    from paper_2403_17031_b200 import binding
    from paper_2403_17031_b200.pipeline import PPOHotPath
    from paper_2403_17031_b200.synthetic import CONFIGS, make_batch
    cfg = dataclasses.replace(CONFIGS[0], B=B, T=T, V=V, dtype=dtype, n_no_eos_exact=None)
    batch = make_batch(cfg, "cuda")
    pp = _params(P, cfg.hyper)
    names = ("losses", "dlogits", "dvalues", "new_logprob", "new_entropy", "dlogprob")
    g = torch.Generator(device="cuda").manual_seed(5)
    epochs = []
    for e in range(3):      # logits and stored log-probs of three epochs
        lg = (batch["policy_logits"].float() + 0.05 * e * torch.randn(batch["policy_logits"].shape, generator=g,
                                                                      device="cuda")).to(batch["policy_logits"].dtype)
        epochs.append(lg)
    a = PPOHotPath(B, T, V, cfg.torch_dtype, pp)
    o = a.rollout_stats(batch["policy_logits"], batch["ref_logits"], batch["responses"], batch["scores"], batch["values"])
    old = (o["logprob"] + batch["old_logprob_noise"]).contiguous()
    want = []
    for lg in epochs:       # the full call, every epoch
        a.loss(lg, batch["responses"], old, batch["values_new"], batch["values"])
        torch.cuda.synchronize()
        want.append({k: a.out[k].clone() for k in names})
    b = PPOHotPath(B, T, V, cfg.torch_dtype, pp)
    b.rollout_stats(batch["policy_logits"], batch["ref_logits"], batch["responses"], batch["scores"], batch["values"])
    for e, lg in enumerate(epochs):
        for k in names:
            b.out[k].fill_(7)
        b.loss(lg, batch["responses"], old, batch["values_new"], batch["values"], next_epoch=e > 0)
        torch.cuda.synchronize()
        for k in names:
            assert torch.equal(b.out[k], want[e][k]), (k, "after loss", e)
    # after the single-call step
    c = PPOHotPath(B, T, V, cfg.torch_dtype, pp)
    c.step(batch["policy_logits"], batch["ref_logits"], batch["responses"], batch["scores"], batch["values"],
           batch["values_new"], old_logprob=old)
    c.loss(epochs[1], batch["responses"], old, batch["values_new"], batch["values"], next_epoch=True)
    torch.cuda.synchronize()
    for k in names:
        assert torch.equal(c.out[k], want[1][k]), (k, "after step")
    assert b.device_status() == 0 and c.device_status() == 0
    if V % 8:
        return              # (the kernels of this shape run the prologue themselves: nothing to refuse)
    # an order built from another mask tensor is refused, nothing is written
    other = c.out["mask"].clone()
    for k in names:
        c.out[k].fill_(7)
    binding.loss_fwd_bwd(epochs[2], batch["responses"], other, old, c.out["advantages_whitened"], batch["values_new"],
                         batch["values"], c.out["returns"], pp, c.workspace, out=c._loss_out, next_epoch=True)
    torch.cuda.synchronize()
    assert c.device_status() == 16
    for k in names:
        assert bool((c.out[k] == 7).all()), k
    # ... and so is one that a fused LM-head call on the same workspace has overwritten
    M, K = 256, 64
    ws = P.new_workspace(max(P.lmhead_workspace_bytes(M, K, 512), P.workspace_bytes(B, T, V)))
    d = PPOHotPath(B, T, V, cfg.torch_dtype, pp)
    d.workspace = ws
    d.step(batch["policy_logits"], batch["ref_logits"], batch["responses"], batch["scores"], batch["values"],
           batch["values_new"], old_logprob=old)
    P.lmhead_logprob_entropy(torch.randn((M, K), device="cuda").to(torch.bfloat16),
                             torch.randn((K, 512), device="cuda").to(torch.bfloat16),
                             torch.zeros(M, dtype=torch.int32, device="cuda"), 0.7, ws)
    d.loss(epochs[1], batch["responses"], old, batch["values_new"], batch["values"], next_epoch=True)
    torch.cuda.synchronize()
    assert d.device_status() == 16
