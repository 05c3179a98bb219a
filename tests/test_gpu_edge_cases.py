"""GPU edge cases: ragged / unaligned shapes, T = 1, sequences of length 1, empty masks, bad
tokens, -inf logits, both row-cache modes of the loss kernel, run-to-run bit reproducibility."""
import numpy as np
import pytest
import torch

from parity import TOL_LOGPROB, TOL_REL, assert_abs, assert_grad, assert_rel, dev, f32, host_logits, npy

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def P():
    assert torch.cuda.is_available()
    import paper_2403_17031_b200 as pkg
    from paper_2403_17031_b200 import build
    build.build()
    pkg.lib()
    return pkg


def _rand_logits(rows, V, dtype, seed, std=2.0):
    g = torch.Generator(device="cuda").manual_seed(seed)
    return (std * torch.randn((rows, V), generator=g, device="cuda")).to(dtype)


@pytest.fixture(params=[0, 2], ids=["direct", "engine"])
def lp_engine(request, P):
    """Run log-prob/entropy through the direct-load kernels (default) and through the row engine."""
    from paper_2403_17031_b200 import binding
    P.set_option(binding.OPT_ROW_ENGINE, request.param)
    yield request.param
    P.set_option(binding.OPT_ROW_ENGINE, 0)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("V", [1, 7, 1000, 1001, 4099, 50304, 65536 + 24])
def test_logprob_entropy_shapes(P, oracle, dtype, V, lp_engine):
    rows = 700 if (V == 50304 and dtype == torch.bfloat16) else 37   # more rows than blocks: several rows per block
    x = _rand_logits(rows, V, dtype, seed=V)
    tok = torch.randint(0, V, (rows,), device="cuda", dtype=torch.int32)
    lp, ent, lse = P.logprob_entropy(x, tok, 0.7, want_lse=True)
    rlp, rent, rlse = oracle.logprob_entropy(host_logits(x), npy(tok), np.float32(0.7))
    assert_abs(npy(lp), rlp, TOL_LOGPROB, "logprob")
    assert_abs(npy(ent), rent, TOL_LOGPROB, "entropy")
    assert_abs(npy(lse), rlse, TOL_LOGPROB, "lse")


def test_logprob_entropy_strided_rows_and_unaligned_base(P, oracle):
    V, pitch, rows = 1000, 1024, 9
    buf = _rand_logits(rows, pitch, torch.bfloat16, seed=5)
    x = buf[:, :V]                                   # pitch > V
    tok = torch.randint(0, V, (rows,), device="cuda", dtype=torch.int32)
    lp, ent, _ = P.logprob_entropy(x, tok, 0.7)
    rlp, rent, _ = oracle.logprob_entropy(host_logits(x.contiguous()), npy(tok), np.float32(0.7))
    assert_abs(npy(lp), rlp, TOL_LOGPROB, "logprob")
    assert_abs(npy(ent), rent, TOL_LOGPROB, "entropy")
    flat = _rand_logits(1, rows * V + 8, torch.bfloat16, seed=6).reshape(-1)
    y = flat[1:1 + rows * V].view(rows, V)            # base only 2-byte aligned -> element-wise kernel
    assert y.data_ptr() % 16 != 0
    lp, ent, _ = P.logprob_entropy(y, tok, 0.7)
    rlp, rent, _ = oracle.logprob_entropy(host_logits(y.contiguous()), npy(tok), np.float32(0.7))
    assert_abs(npy(lp), rlp, TOL_LOGPROB, "logprob")
    assert_abs(npy(ent), rent, TOL_LOGPROB, "entropy")


def test_uniform_and_peaked_rows(P, lp_engine):
    V = 50304
    x = torch.full((3, V), 1.25, device="cuda", dtype=torch.bfloat16)
    x[1, 17] = 60.0                                   # one dominant logit
    x[2, :] = -40.0
    tok = torch.tensor([5, 17, 9], device="cuda", dtype=torch.int32)
    lp, ent, _ = P.logprob_entropy(x, tok, 0.7)
    lnV = 10.825839875788878
    assert abs(float(lp[0]) + lnV) < 1e-4 and abs(float(ent[0]) - lnV) < 1e-4
    assert abs(float(lp[1])) < 1e-4 and abs(float(ent[1])) < 1e-4
    assert abs(float(lp[2]) + lnV) < 1e-4


def test_wide_range_rows_take_the_rebase_path(P, oracle, lp_engine):
    """Rows whose later elements exceed the first ones by far more than 2^127 in base-2 units."""
    V = 50304
    x = torch.full((6, V), -300.0, device="cuda", dtype=torch.float32)
    x[0, 40000] = 250.0
    x[1, 5] = 100.0; x[1, 50000] = 320.0
    x[2, ::977] = 90.0; x[2, 30011] = 400.0
    x[3] = torch.linspace(-500, 500, V, device="cuda")
    x[4] = torch.linspace(500, -500, V, device="cuda")
    x[5, 123] = float("-inf")
    for dt in (torch.float32, torch.bfloat16):
        xx = x.to(dt)
        tok = torch.tensor([40000, 5, 30011, V - 1, 3, 7], device="cuda", dtype=torch.int32)
        lp, ent, lse = P.logprob_entropy(xx, tok, 0.7, want_lse=True)
        rlp, rent, rlse = oracle.logprob_entropy(host_logits(xx), npy(tok), np.float32(0.7))
        assert_abs(npy(lp), rlp, 2e-4, "logprob")          # |lse| reaches ~700: fp32 resolution there is 6e-5
        assert_abs(npy(ent), rent, TOL_LOGPROB, "entropy")
        assert_rel(npy(lse), rlse, 1e-6, "lse")


def test_neg_inf_logits_and_bad_tokens(P, oracle, lp_engine):
    V = 4096
    x = _rand_logits(4, V, torch.float32, seed=7)
    x[0, 100:] = float("-inf")
    x[1, ::2] = float("-inf")
    tok = torch.tensor([3, 1, V, -1], device="cuda", dtype=torch.int32)
    ws = P.new_workspace(P.workspace_bytes(1, 4, V))
    lp, ent, _ = P.logprob_entropy(x, tok, 0.7, workspace=ws)
    rlp, rent, _ = oracle.logprob_entropy(host_logits(x), npy(tok), np.float32(0.7))
    assert_abs(npy(lp)[:2], rlp[:2], TOL_LOGPROB, "logprob with -inf")
    assert_abs(npy(ent)[:2], rent[:2], TOL_LOGPROB, "entropy with -inf")
    assert torch.isnan(lp[2:]).all() and torch.isnan(ent[2:]).all() and np.isnan(rlp[2:]).all()
    assert P.last_device_status(ws) == 1              # PPO_DEV_BAD_TOKEN
    assert P.last_device_status(ws) == 0              # cleared by the read
    xb = x.to(torch.bfloat16)
    lp, ent, _ = P.logprob_entropy(xb, tok, 0.7)
    rlp, rent, _ = oracle.logprob_entropy(host_logits(xb), npy(tok), np.float32(0.7))
    assert_abs(npy(lp)[:2], rlp[:2], TOL_LOGPROB, "bf16 logprob with -inf")
    assert_abs(npy(ent)[:2], rent[:2], TOL_LOGPROB, "bf16 entropy with -inf")


@pytest.mark.parametrize("B,T", [(1, 1), (3, 1), (5, 2), (7, 31), (6, 32), (5, 33), (9, 53), (3, 512), (2, 1000)])
def test_token_level_steps_shapes(P, oracle, B, T):
    rng = np.random.default_rng(B * 1000 + T)
    resp = rng.integers(2, 50, (B, T)).astype(np.int32)
    for b in range(B):
        if b % 3 != 2:
            resp[b, rng.integers(0, T)] = 0
        if b % 4 == 0:
            resp[b, 0] = 0                              # sequence of length 1
    scores = rng.normal(size=B).astype(np.float32)
    ro, ei, sl, m, so = oracle.truncate_and_score(resp, 0, 1, scores, np.float32(-1.0))
    g = P.truncate_and_score(dev(resp), dev(scores), 0, 1, -1.0)
    for got, want in zip(g[:4], (ro, ei, sl, m)):
        assert np.array_equal(npy(got), want)
    assert np.array_equal(npy(g[4]).astype(np.float64), so)
    # in place
    r2 = dev(resp)
    P.truncate_and_score(r2, dev(scores), 0, 1, -1.0, out=(r2, g[1], g[2], g[3], g[4]))
    assert np.array_equal(npy(r2), ro)
    lp = rng.normal(-3, 1, (B, T)).astype(np.float32)
    lr = rng.normal(-3, 1, (B, T)).astype(np.float32)
    kl, rew = oracle.kl_rewards(lp, lr, m, sl, f32(so), np.float32(0.05))
    gk, gr = P.kl_rewards(dev(lp), dev(lr), dev(m), dev(sl), dev(f32(so)), 0.05)
    assert_abs(npy(gk), kl, TOL_LOGPROB, "kl")
    assert_rel(npy(gr), rew, TOL_REL, "rewards")
    v = rng.normal(size=(B, T)).astype(np.float32)
    for gamma, lam in ((1.0, 0.95), (0.99, 0.95), (1.0, 1.0), (0.9, 0.0)):
        A, R = oracle.gae(f32(rew), v, sl, np.float32(gamma), np.float32(lam))
        gA, gR = P.gae(dev(f32(rew)), dev(v), dev(sl), gamma, lam)
        assert_rel(npy(gA), A, TOL_REL, "advantages")
        assert_rel(npy(gR), R, TOL_REL, "returns")
    for sm in (True, False):
        w, st = oracle.whiten(f32(A), m, sm, np.float32(1e-8))
        gw, gst = P.whiten(dev(f32(A)), dev(m), sm, 1e-8)
        assert_rel(npy(gw), w, TOL_REL, "whiten")
        assert_rel(npy(gst), st, TOL_REL, "whiten stats")
    w, st = oracle.whiten(f32(A), None, True, np.float32(1e-8))
    gw, gst = P.whiten(dev(f32(A)), None, True, 1e-8)
    assert_rel(npy(gw), w, TOL_REL, "whiten (no mask)")
    x = dev(f32(A))
    P.whiten(x, dev(m), True, 1e-8, out=x)               # in place
    w, _ = oracle.whiten(f32(A), m, True, np.float32(1e-8))
    assert_rel(npy(x), w, TOL_REL, "whiten in place")


def test_empty_mask_sets_status(P):
    B, T, V = 2, 4, 64
    ws = P.new_workspace(P.workspace_bytes(B, T, V))
    x = torch.randn(B, T, device="cuda")
    m = torch.zeros(B, T, dtype=torch.uint8, device="cuda")
    out, st = P.whiten(x, m, True, 1e-8, workspace=ws)
    assert not out.any().item() and float(st[2]) == 0
    assert P.last_device_status(ws) == 2
    lg = torch.randn(B, T, V, device="cuda")
    tok = torch.zeros(B, T, dtype=torch.int32, device="cuda")
    o = P.loss_fwd_bwd(lg, tok, m, x, x, x, x, x, P.default_params(), ws)
    assert not o["losses"].any().item() and not o["dlogits"].any().item() and not o["dvalues"].any().item()
    assert P.last_device_status(ws) == 2


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("V,mode", [(1000, 0), (1001, 0), (50304, 0), (50304, 1), (50304, 2), (70000, 0), (131072, 0)])
def test_loss_kernel_variants(P, oracle, dtype, V, mode):
    """Vector / element-wise kernels, row in shared memory / re-read from L2, rows beyond shared memory."""
    from paper_2403_17031_b200 import binding
    B, T = 3, 7
    rng = np.random.default_rng(V + mode)
    lg = _rand_logits(B * T, V, dtype, seed=V + mode).view(B, T, V)
    tok = torch.randint(0, V, (B, T), device="cuda", dtype=torch.int32)
    L = np.array([7, 4, 1])
    m = (np.arange(T)[None] < L[:, None]).astype(np.uint8)
    lp, _, _ = oracle.logprob_entropy(host_logits(lg.view(-1, V)), npy(tok), np.float32(0.7))
    old = (lp.reshape(B, T) + rng.normal(0, 0.15, (B, T))).astype(np.float32)
    adv = rng.normal(size=(B, T)).astype(np.float32)
    vo = rng.normal(size=(B, T)).astype(np.float32)
    vn = (vo + rng.normal(0, 0.2, (B, T))).astype(np.float32)
    ret = rng.normal(size=(B, T)).astype(np.float32)
    ref = oracle.loss_fwd_bwd(host_logits(lg), npy(tok), m, old, adv, vn, vo, ret, np.float32(0.7),
                              np.float32(0.2), np.float32(0.2), np.float32(0.1))
    ws = P.new_workspace(P.workspace_bytes(B, T, V))
    P.set_option(binding.OPT_LOSS_ROW_CACHE, mode)
    P.set_option(binding.OPT_ROW_ENGINE, 1 if mode else 0)     # modes 1, 2 select among the direct-load kernels
    try:
        o = P.loss_fwd_bwd(lg, tok, dev(m), dev(old), dev(adv), dev(vn), dev(vo), dev(ret), P.default_params(), ws)
        o_b = P.loss_fwd_bwd(lg, tok, dev(m), dev(old), dev(adv), dev(vn), dev(vo), dev(ret), P.default_params(), ws)
        o_n = P.loss_fwd_bwd(lg, tok, dev(m), dev(old), dev(adv), dev(vn), dev(vo), dev(ret), P.default_params(), ws,
                             want_dlogits=False)
    finally:
        P.set_option(binding.OPT_LOSS_ROW_CACHE, 0)
        P.set_option(binding.OPT_ROW_ENGINE, 0)
    n = ref["losses"][7]
    assert_abs(npy(o["losses"]), ref["losses"], TOL_LOGPROB, "losses")
    assert_abs(npy(o["new_logprob"]), ref["new_logprob"], TOL_LOGPROB, "new_logprob")
    assert_abs(n * npy(o["dvalues"]), n * ref["dvalues"], 1e-4, "n*dvalues")
    assert_abs(n * npy(o["dlogprob"]), n * ref["dlogprob"], 1e-4, "n*dlogprob")
    assert_grad(n * o["dlogits"].float().cpu().numpy().reshape(-1, V), n * ref["dlogits"],
                dtype == torch.bfloat16, "n*dlogits")
    # bit-reproducible from run to run
    for k in ("losses", "dlogits", "dvalues", "new_logprob", "entropy", "dlogprob"):
        assert torch.equal(o[k], o_b[k]), k
    # the forward-only call may run a differently shaped block (other summation order)
    for k in ("losses", "dvalues", "new_logprob", "entropy", "dlogprob"):
        assert torch.allclose(o[k], o_n[k], rtol=1e-5, atol=1e-6), k


def test_loss_from_logprob_matches_oracle(P, oracle):
    B, T = 16, 53
    rng = np.random.default_rng(21)
    L = rng.integers(1, T + 1, B)
    m = (np.arange(T)[None] < L[:, None]).astype(np.uint8)
    nlp = (-0.05 - np.abs(rng.normal(3, 1, (B, T)))).astype(np.float32)     # log-probs are negative
    old = (nlp + rng.normal(0, 0.15, (B, T))).astype(np.float32)
    adv, vo, ret = (rng.normal(size=(B, T)).astype(np.float32) for _ in range(3))
    vn = (vo + rng.normal(0, 0.2, (B, T))).astype(np.float32)
    ent = rng.random((B, T)).astype(np.float32)
    # oracle: a 2-token vocabulary whose log-softmax reproduces nlp exactly is not available, so use
    # its scalar arithmetic through V=2 logits (x, 0) with p(token 0) = exp(nlp): x = logit(p)
    p = np.exp(nlp.astype(np.float64))
    x = np.log(p) - np.log1p(-p)
    lg = np.stack([x, np.zeros_like(x)], -1).astype(np.float32)
    ref = oracle.loss_fwd_bwd(lg, np.zeros((B, T), np.int32), m, old, adv, vn, vo, ret, 1.0, np.float32(0.2),
                              np.float32(0.2), np.float32(0.1), want_dlogits=False)
    ws = P.new_workspace(P.workspace_bytes(B, T, 2))
    o = P.loss_from_logprob(dev(f32(ref["new_logprob"])), dev(ent), dev(m), dev(old), dev(adv), dev(vn), dev(vo),
                            dev(ret), P.default_params(), ws)
    n = ref["losses"][7]
    got = npy(o["losses"]).astype(np.float64)
    for i in (0, 1, 2, 3, 4, 5, 7):
        assert abs(got[i] - ref["losses"][i]) <= TOL_LOGPROB, (i, got[i], ref["losses"][i])
    assert abs(got[6] - ent[m.astype(bool)].mean()) < 1e-5
    assert_abs(n * npy(o["dlogprob"]), n * ref["dlogprob"], 1e-4, "n*dlogprob")
    assert_abs(n * npy(o["dvalues"]), n * ref["dvalues"], 1e-4, "n*dvalues")
