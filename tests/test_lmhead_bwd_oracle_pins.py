"""Pins of oracle/lmhead_bwd_oracle.py: finite differences of the forward oracle (C code, another code base),
a second opinion from a library's reverse-mode differentiation, and closed forms. No GPU."""
import numpy as np
import torch

from oracle import lmhead_bwd_oracle as B


def _bf16_bits(x64):
    t = torch.from_numpy(np.asarray(x64, np.float32)).to(torch.bfloat16)
    return t.view(torch.int16).numpy().view(np.uint16)


def test_closed_forms():
    M, K, V, tau = 3, 4, 6, 0.7
    H = np.zeros((M, K))
    W = np.ones((K, V))
    tok = np.array([0, 3, 5])
    g = np.array([2.0, -1.0, 0.5])
    o = B.lmhead_bwd(H, W, tok, g, tau)
    want = -np.ones((M, V)) / V                      # zero hidden state: uniform softmax
    want[np.arange(M), tok] += 1.0
    want *= (g / tau)[:, None]
    assert np.allclose(o["D"], want, atol=1e-15)
    assert np.abs(o["D"].sum(axis=1)).max() < 1e-15  # every row of D sums to zero
    assert np.abs(o["dH"]).max() < 1e-15             # W has equal columns: D W^T = (row sums of D) * w = 0
    assert not o["dW"].any()                         # H = 0
    # masked rows carry no gradient
    o2 = B.lmhead_bwd(np.ones((M, K)), W, tok, g, tau, mask=np.array([1, 0, 1]))
    assert not o2["D"][1].any() and o2["D"][0].any()


def test_finite_differences_of_the_forward_oracle(oracle):
    """loss = sum_r g_r * lp_r with lp from the C oracle on bf16 inputs; steps are exact in bf16."""
    rng = np.random.default_rng(0)
    M, K, V, tau = 4, 8, 16, 0.7
    q = lambda a: np.round(np.clip(a, -1.9, 1.9) * 16) / 16       # multiples of 1/16 below 2: x +- 2^-6 is a bf16
    H, W = q(rng.normal(size=(M, K))), q(rng.normal(size=(K, V)) * 0.7)
    tok = rng.integers(0, V, M).astype(np.int32)
    g = rng.normal(size=M)
    o = B.lmhead_bwd(H, W, tok, g, tau)

    def loss(Hx, Wx):
        lp, _, _ = oracle.lmhead_logprob_entropy(_bf16_bits(Hx), _bf16_bits(Wx), tok, tau)
        return float((g * lp).sum())
    e = 2.0 ** -6
    for r in range(M):
        for k in range(K):
            up, dn = H.copy(), H.copy()
            up[r, k] += e
            dn[r, k] -= e
            assert abs((loss(up, W) - loss(dn, W)) / (2 * e) - o["dH"][r, k]) < 2e-3
    for k in range(K):
        for v in range(0, V, 3):
            up, dn = W.copy(), W.copy()
            up[k, v] += e
            dn[k, v] -= e
            assert abs((loss(H, up) - loss(H, dn)) / (2 * e) - o["dW"][k, v]) < 2e-3


def test_library_reverse_mode_second_opinion():
    rng = np.random.default_rng(1)
    M, K, V, tau = 37, 24, 101, 0.7
    H, W = rng.normal(size=(M, K)), rng.normal(size=(K, V)) * 0.3
    tok = rng.integers(0, V, M)
    g = rng.normal(size=M)
    mask = (rng.random(M) < 0.8).astype(np.uint8)
    o = B.lmhead_bwd(H, W, tok, g, tau, mask=mask)
    Ht = torch.tensor(H, dtype=torch.float64, requires_grad=True)
    Wt = torch.tensor(W, dtype=torch.float64, requires_grad=True)
    lp = torch.log_softmax(Ht @ Wt / tau, dim=-1)[torch.arange(M), torch.tensor(tok)]
    (lp * torch.tensor(g * mask)).sum().backward()
    assert np.allclose(o["dH"], Ht.grad.numpy(), atol=1e-12)
    assert np.allclose(o["dW"], Wt.grad.numpy(), atol=1e-12)
    assert (o["dH_abs"] >= np.abs(o["dH"]) - 1e-15).all() and (o["dW_abs"] >= np.abs(o["dW"]) - 1e-15).all()


def test_bf16_widening():
    x = np.array([1.0, -2.5, 0.0078125, 3.0e38], np.float32)
    assert np.array_equal(B.bf16_to_f64(_bf16_bits(x)), torch.from_numpy(x).to(torch.bfloat16).double().numpy())
