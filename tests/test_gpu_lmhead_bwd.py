"""GPU parity of the LM-head backward (ppo_lmhead_bwd) against oracle/lmhead_bwd_oracle.py, through the C ABI.

Tolerance (derived from the arithmetic): dlogits is stored in bf16 (relative rounding 2^-9, the logits behind it
carry fp32-accumulation error ~1e-5); dH and dW contract that bf16 dlogits with fp32 accumulation and are rounded
to bf16 once more, so |error| <= 2^-9 * sum|D||W| (worst case over the contraction) + 2^-9 |result|. The tests
allow twice that plus a small absolute term."""
import numpy as np
import pytest
import torch

from oracle import lmhead_bwd_oracle as B

pytestmark = pytest.mark.gpu

REL = 2.0 ** -8


@pytest.fixture(scope="module")
def P():
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    import paper_2403_17031_b200 as pkg
    from paper_2403_17031_b200 import build
    build.build()
    pkg.lib()
    return pkg


def _wide(t):
    return t.detach().double().cpu().numpy()


def _rows_in_place(dlogits, mask):
    """dlogits as [M, V] with every row at its own place. Given a mask (and more than one 128-row tile) the call
    leaves the gradient rows of the rows with mask 1 packed at the front of the buffer, in row order; the rest of
    the buffer is scratch."""
    if mask is None or dlogits.shape[0] <= 128:
        return dlogits
    rows = torch.nonzero(mask).flatten()
    full = torch.zeros_like(dlogits)
    full[rows] = dlogits[: rows.numel()]
    return full


def _check(P, M, K, V, seed, with_mask=True, tau=0.7):
    g = torch.Generator(device="cuda").manual_seed(seed)
    H = torch.randn((M, K), generator=g, device="cuda").to(torch.bfloat16)
    W = (torch.randn((K, V), generator=g, device="cuda") * (2.0 / K ** 0.5)).to(torch.bfloat16)
    tok = torch.randint(0, V, (M,), generator=g, device="cuda", dtype=torch.int32)
    up = torch.randn((M,), generator=g, device="cuda")
    up[0] = 0.0
    mask = (torch.rand((M,), generator=g, device="cuda") < 0.8).to(torch.uint8) if with_mask else None
    ws = P.new_workspace(P.lmhead_workspace_bytes(M, K, V))
    _, _, lse = P.lmhead_logprob_entropy(H, W, tok, tau, ws, want_lse=True)
    o = P.lmhead_bwd(H, W, tok, lse, up, tau, ws, mask=mask)
    torch.cuda.synchronize()
    assert P.last_device_status(ws) == 0
    ref = B.lmhead_bwd(_wide(H), _wide(W), tok.cpu().numpy(), up.cpu().numpy().astype(np.float64), tau,
                       mask=None if mask is None else mask.cpu().numpy())
    D, dH, dW = _wide(_rows_in_place(o["dlogits"], mask)), _wide(o["dH"]), _wide(o["dW"])
    assert np.isfinite(D).all() and np.isfinite(dH).all() and np.isfinite(dW).all()
    bad = np.abs(D - ref["D"]) > REL * np.abs(ref["D"]) + 1e-6
    assert not bad.any(), "dlogits: %d off, worst %.3e" % (bad.sum(), np.abs(D - ref["D"])[bad].max())
    if mask is not None:
        assert not D[mask.cpu().numpy() == 0].any() and not dH[mask.cpu().numpy() == 0].any()
    assert not D[0].any()
    for name, got, want, scale in (("dH", dH, ref["dH"], ref["dH_abs"]), ("dW", dW, ref["dW"], ref["dW_abs"])):
        bad = np.abs(got - want) > REL * scale + REL * np.abs(want) + 1e-6
        assert not bad.any(), "%s: %d of %d off, worst %.3e (|want| max %.3e)" % (
            name, bad.sum(), bad.size, np.abs(got - want)[bad].max(), np.abs(want).max())


@pytest.mark.parametrize("M,K,V", [(128, 64, 256), (200, 128, 1000), (300, 192, 2056), (64, 64, 520),
                                   (1000, 256, 4096)])
def test_lmhead_bwd_small_shapes(P, M, K, V):
    _check(P, M, K, V, seed=M + K + V)


def test_lmhead_bwd_without_mask_and_partial_outputs(P):
    _check(P, 256, 128, 512, seed=5, with_mask=False, tau=1.0)
    M, K, V = 128, 64, 256
    H = torch.randn((M, K), device="cuda").to(torch.bfloat16)
    W = torch.randn((K, V), device="cuda").to(torch.bfloat16)
    tok = torch.zeros(M, dtype=torch.int32, device="cuda")
    ws = P.new_workspace(P.lmhead_workspace_bytes(M, K, V))
    _, _, lse = P.lmhead_logprob_entropy(H, W, tok, 1.0, ws, want_lse=True)
    o = P.lmhead_bwd(H, W, tok, lse, torch.ones(M, device="cuda"), 1.0, ws, want_dH=False, want_dW=False)
    assert o["dH"] is None and o["dW"] is None and torch.isfinite(o["dlogits"].float()).all()


def test_lmhead_bwd_full_width_1024_rows(P):
    """Full K and V of config 4 (many vocabulary tiles, 64 contraction blocks), rows cut to what the dense oracle
    handles in seconds: every element of dlogits, dH and dW is compared."""
    _check(P, 1024, 4096, 50304, seed=11)


def test_lmhead_bwd_config4_full_size_sampled(P):
    """Config 4 in the launch configuration the benchmark times. Row-local results (dlogits and dH rows) are checked
    on sampled rows, which the oracle computes one by one; dW mixes all rows, so it is checked through properties:
    every row of dW sums to ~0 over the vocabulary (each row of dlogits does), and a random projection
    u^T dW equals (H u)^T D restricted to sampled vocabulary columns computed from the oracle-checked dlogits."""
    from paper_2403_17031_b200.synthetic import CONFIGS, make_lmhead_batch
    cfg = CONFIGS[4]
    b = make_lmhead_batch(cfg, "cuda")
    H, W, tok = b["H"], b["W"], b["tokens"]
    M, K = H.shape
    V = W.shape[1]
    tau = cfg.hyper.temperature
    g = torch.Generator(device="cuda").manual_seed(3)
    up = torch.randn((M,), generator=g, device="cuda") / M
    mask = (torch.rand((M,), generator=g, device="cuda") < 0.55).to(torch.uint8)
    ws = P.new_workspace(P.lmhead_workspace_bytes(M, K, V))
    _, _, lse = P.lmhead_logprob_entropy(H, W, tok, tau, ws, want_lse=True)
    o = P.lmhead_bwd(H, W, tok, lse, up, tau, ws, mask=mask)
    torch.cuda.synchronize()
    assert P.last_device_status(ws) == 0
    rng = np.random.default_rng(4)
    real = np.flatnonzero(mask.cpu().numpy())
    rows = np.unique(np.concatenate([[real[0], real[-1]], rng.choice(real, 10, replace=False),
                                     np.flatnonzero(mask.cpu().numpy() == 0)[:2]]))
    Wd = _wide(W)
    idx = torch.from_numpy(rows).cuda()
    ref = B.lmhead_bwd(_wide(H[idx]), Wd, tok[idx].cpu().numpy(), up[idx].cpu().numpy().astype(np.float64), tau,
                       mask=mask[idx].cpu().numpy())
    n_real = len(real)
    packed_at = torch.from_numpy(np.searchsorted(real, rows)).cuda()       # where a real row's gradient row was packed
    D = _wide(o["dlogits"][packed_at.clamp_max(n_real - 1)])
    D[mask[idx].cpu().numpy() == 0] = 0.0                                   # (rows with mask 0 have none)
    dH = _wide(o["dH"][idx])
    bad = np.abs(D - ref["D"]) > REL * np.abs(ref["D"]) + 1e-9
    assert not bad.any(), "dlogits rows: %d off, worst %.3e" % (bad.sum(), np.abs(D - ref["D"])[bad].max())
    bad = np.abs(dH - ref["dH"]) > REL * ref["dH_abs"] + REL * np.abs(ref["dH"]) + 1e-9
    assert not bad.any(), "dH rows: %d off, worst %.3e" % (bad.sum(), np.abs(dH - ref["dH"])[bad].max())
    assert not _wide(o["dH"][mask == 0][:64]).any()
    dW = o["dW"].float()
    assert torch.isfinite(dW).all()
    # rows of dW sum to zero up to the bf16 rounding of its 50304 entries
    assert float((dW.double().sum(1).abs() / dW.double().abs().sum(1).clamp_min(1e-30)).max()) < 2.0 ** -8
    # projection check against the dlogits that this call wrote (its rows were checked above): fp64 on the GPU
    cols = torch.from_numpy(np.sort(rng.choice(V, 64, replace=False))).cuda()
    u = torch.randn((K,), generator=g, device="cuda", dtype=torch.float64)
    lhs = u @ dW.double()[:, cols]
    Dc = o["dlogits"][:n_real, cols].double()                              # packed rows <-> H[real]
    Hr = H[torch.from_numpy(real).cuda()].double()
    rhs = (Hr @ u) @ Dc
    scale = (Hr.abs() @ u.abs()) @ Dc.abs()      # sum_k |u_k| (|H|^T |D|)[k, v]: the scale of dW's rounding
    assert float(((lhs - rhs).abs() / scale.clamp_min(1e-30)).max()) < 2.0 ** -8


@pytest.mark.parametrize("M", [100, 200])
def test_lmhead_bwd_all_rows_masked(P, M):
    K, V = 128, 1000
    H = torch.randn((M, K), device="cuda").to(torch.bfloat16)
    W = torch.randn((K, V), device="cuda").to(torch.bfloat16)
    tok = torch.randint(0, V, (M,), device="cuda", dtype=torch.int32)
    ws = P.new_workspace(P.lmhead_workspace_bytes(M, K, V))
    _, _, lse = P.lmhead_logprob_entropy(H, W, tok, 0.7, ws, want_lse=True)
    o = P.lmhead_bwd(H, W, tok, lse, torch.ones(M, device="cuda"), 0.7, ws,
                     mask=torch.zeros(M, dtype=torch.uint8, device="cuda"))
    torch.cuda.synchronize()
    # (M = 200 takes the packed path: no gradient row is written, dlogits is scratch)
    assert (M > 128 or not o["dlogits"].float().any()) and not o["dH"].float().any() and not o["dW"].float().any()
    assert P.last_device_status(ws) == 0


def test_lmhead_bwd_packed_rows_equal_the_dense_call(P):
    """Taking the rows with mask 0 out of the three passes must not change a bit of dH (row-local) and must give the
    dW of the dense call up to the order of the fp32 sums over rows, which does not change either: the packed rows
    keep their order and the rows left out contributed exact zeros."""
    M, K, V = 900, 128, 1032
    g = torch.Generator(device="cuda").manual_seed(11)
    H = torch.randn((M, K), generator=g, device="cuda").to(torch.bfloat16)
    W = (torch.randn((K, V), generator=g, device="cuda") * 0.2).to(torch.bfloat16)
    tok = torch.randint(0, V, (M,), generator=g, device="cuda", dtype=torch.int32)
    up = torch.randn((M,), generator=g, device="cuda")
    mask = (torch.rand((M,), generator=g, device="cuda") < 0.5).to(torch.uint8)
    ws = P.new_workspace(P.lmhead_workspace_bytes(M, K, V))
    _, _, lse = P.lmhead_logprob_entropy(H, W, tok, 0.7, ws, want_lse=True)
    dense = P.lmhead_bwd(H, W, tok, lse, up * mask, 0.7, ws)               # zero gradient on the rows left out
    packed = P.lmhead_bwd(H, W, tok, lse, up, 0.7, ws, mask=mask)
    torch.cuda.synchronize()
    assert torch.equal(_rows_in_place(packed["dlogits"], mask), dense["dlogits"])
    assert torch.equal(packed["dH"], dense["dH"])
    rel = (packed["dW"].double() - dense["dW"].double()).abs().max() / dense["dW"].double().abs().max()
    assert float(rel) < 2.0 ** -7
    assert P.last_device_status(ws) == 0
