"""GPU parity of ppo_sample_logprob_entropy against oracle/sample_oracle.py (Philox4x32-10 + a two-level
exponential race: first between the 256 classes of the row, then inside the winning class).

The token is an integer decided by floating point. The kernel evaluates the rule in fp32 with hardware exp2 / log2
approximations (relative error ~2^-22 on scores of magnitude <= ~60), the oracle in fp64; so the comparison is, at
each level: the identical choice wherever the oracle's best and second-best scores are more than GAP apart, and
otherwise a choice whose score is within GAP of the best."""
import numpy as np
import pytest
import torch

from oracle import sample_oracle as S
from parity import TOL_LOGPROB, assert_abs, host_logits, npy

pytestmark = pytest.mark.gpu
GAP = 1e-4


@pytest.fixture(scope="module")
def P():
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    import paper_2403_17031_b200 as pkg
    from paper_2403_17031_b200 import build
    build.build()
    pkg.lib()
    return pkg


def _check_draw(x64, tau, seed, offset, tok, min_clear=0.98):
    """tok [rows]: the kernel's tokens. Level by level against the oracle's scores; returns the oracle's tokens."""
    rows = x64.shape[0]
    want, keys1, keys2, cls = S.sample(x64, tau, seed, offset)
    r = np.arange(rows)
    assert (tok >= 0).all() and (tok < x64.shape[1]).all()
    c_got = cls[tok]
    # level 1: the class
    if np.isfinite(keys1).sum(axis=1).min() >= 2:
        top2 = np.partition(keys1, -2, axis=1)[:, -2:]
        clear1 = top2[:, 1] - top2[:, 0] > GAP
    else:
        clear1 = np.ones(rows, bool)              # (a row with a single class that has weight)
    assert clear1.mean() > min_clear
    assert np.array_equal(c_got[clear1], keys1.argmax(axis=1)[clear1]), "classes of clear rows differ"
    assert (keys1.max(axis=1) - keys1[r, c_got] <= GAP).all()
    # level 2: the element inside the class the kernel took
    inside = np.where(cls[None, :] == c_got[:, None], keys2, -np.inf)
    if inside.shape[1] >= 2:
        top2 = np.partition(inside, -2, axis=1)[:, -2:]
        clear2 = ~(top2[:, 1] - top2[:, 0] <= GAP)
    else:
        clear2 = np.ones(rows, bool)
    assert clear2.mean() > min_clear
    assert np.array_equal(tok[clear2], inside.argmax(axis=1)[clear2]), "elements of clear rows differ"
    assert (inside.max(axis=1) - keys2[r, tok] <= GAP).all()
    both = clear1 & clear2
    assert np.array_equal(tok[both], want[both])
    return want


def _compare(P, oracle, x, tau, seed, offset=0):
    rows, V = x.shape
    ws = P.new_workspace(P.workspace_bytes(rows, 1, V))
    tok, lp, ent, lse = P.sample_logprob_entropy(x, tau, seed, offset, workspace=ws, want_lse=True)
    torch.cuda.synchronize()
    assert P.last_device_status(ws) == 0
    tok = npy(tok).astype(np.int64)
    want = _check_draw(x.detach().double().cpu().numpy(), tau, seed, offset, tok)
    assert (tok == want).mean() > 0.97
    # log-prob of the token that was drawn, entropy and lse: the forward oracle
    o_lp, o_ent, o_lse = oracle.logprob_entropy(host_logits(x), tok.astype(np.int32), tau)
    assert_abs(npy(lp), o_lp, TOL_LOGPROB, "logprob of the drawn token")
    assert_abs(npy(ent), o_ent, TOL_LOGPROB, "entropy")
    assert_abs(npy(lse), o_lse, TOL_LOGPROB, "lse")
    return tok


@pytest.mark.parametrize("dtype,rows,V", [(torch.float32, 64, 1000), (torch.float32, 33, 1001), (torch.bfloat16, 128, 2048),
                                          (torch.bfloat16, 40, 50304), (torch.bfloat16, 17, 1004), (torch.float32, 12, 50304),
                                          (torch.float32, 21, 4100), (torch.bfloat16, 9, 131072 + 8), (torch.float32, 7, 70004)])
def test_sample_matches_oracle(P, oracle, dtype, rows, V):
    g = torch.Generator(device="cuda").manual_seed(rows + V)
    x = (2.0 * torch.randn((rows, V), generator=g, device="cuda")).to(dtype)
    _compare(P, oracle, x, 0.7, seed=0x1234567890abcdef, offset=3)


def test_strided_rows_seed_and_offset(P, oracle):
    g = torch.Generator(device="cuda").manual_seed(1)
    big = torch.randn((50, 1536), generator=g, device="cuda")
    x = big[:, :1000]                                     # row pitch 1536 > V
    t0 = _compare(P, oracle, x, 1.0, seed=11)
    t1 = _compare(P, oracle, x, 1.0, seed=12)
    t2 = _compare(P, oracle, x, 1.0, seed=11, offset=2 ** 33 + 5)
    assert (t0 != t1).mean() > 0.5 and (t0 != t2).mean() > 0.5
    again, _, _, _ = P.sample_logprob_entropy(x, 1.0, 11)
    assert np.array_equal(npy(again), t0)                 # same seed and offset: same draw


@pytest.mark.parametrize("V,n", [(16, 20000), (304, 60000)])
def test_distribution_of_draws(P, V, n):
    """Many rows with the same logits: token frequencies follow softmax(logits / tau) (chi-square); V = 304 spreads the
    row over 38 classes, so both levels of the race decide."""
    rng = np.random.default_rng(3)
    tau = 0.7
    row = (rng.normal(size=V) * (1.5 if V == 16 else 1.0)).astype(np.float32)
    x = torch.from_numpy(np.tile(row, (n, 1))).cuda()
    tok, _, _, _ = P.sample_logprob_entropy(x, tau, seed=2024)
    p = np.exp(row.astype(np.float64) / tau)
    p /= p.sum()
    counts = np.bincount(npy(tok), minlength=V).astype(np.float64)
    small = n * p < 8.0                                             # cells of small expectation are pooled
    c = np.append(counts[~small], counts[small].sum())
    e = np.append(n * p[~small], n * p[small].sum())
    c, e = c[e > 0], e[e > 0]
    dof = len(e) - 1
    assert ((c - e) ** 2 / e).sum() < dof + 6.0 * np.sqrt(2.0 * dof)   # mean dof, sd sqrt(2 dof)


def test_minus_infinity_never_drawn_and_bad_rows(P):
    V = 512
    x = torch.randn((6, V), device="cuda")
    x[:, ::2] = float("-inf")
    x[3, 7] = float("nan")
    x[4, :] = float("-inf")
    x[5, 9] = float("inf")
    ws = P.new_workspace(P.workspace_bytes(6, 1, V))
    tok, lp, ent, _ = P.sample_logprob_entropy(x, 0.7, 5, workspace=ws)
    tok = npy(tok)
    assert (tok[:3] % 2 == 1).all() and np.isfinite(npy(lp)[:3]).all() and np.isfinite(npy(ent)[:3]).all()
    assert (tok[3:] == -1).all() and np.isnan(npy(lp)[3:]).all()
    assert P.last_device_status(ws) == 8


def test_rows_far_above_their_first_pack_take_the_exact_maximum(P, oracle):
    """The one-pass path uses the row's first pack as reference; a row whose other logits lie hundreds above it
    overflows there and must come out the same through the exact-maximum repeat."""
    g = torch.Generator(device="cuda").manual_seed(9)
    x = 2.0 * torch.randn((24, 4096), generator=g, device="cuda")
    x[::2, :8] = -300.0
    _compare(P, oracle, x, 0.7, seed=77)
    xb = x.to(torch.bfloat16)
    _compare(P, oracle, xb, 0.7, seed=78)


def test_tiny_rows_and_odd_widths(P, oracle):
    g = torch.Generator(device="cuda").manual_seed(4)
    for dtype, rows, V in ((torch.float32, 1, 8), (torch.float32, 3, 5), (torch.bfloat16, 2, 16), (torch.bfloat16, 5, 37)):
        x = torch.randn((rows, V), generator=g, device="cuda").to(dtype)
        ws = P.new_workspace(P.workspace_bytes(rows, 1, V))
        tok, lp, ent, lse = P.sample_logprob_entropy(x, 0.7, 99, workspace=ws, want_lse=True)
        t = npy(tok).astype(np.int64)
        _check_draw(x.double().cpu().numpy(), 0.7, 99, 0, t, min_clear=0.0)
        o_lp, o_ent, o_lse = oracle.logprob_entropy(host_logits(x), t.astype(np.int32), 0.7)
        assert_abs(npy(lp), o_lp, TOL_LOGPROB, "logprob")
        assert_abs(npy(ent), o_ent, TOL_LOGPROB, "entropy")
        assert P.last_device_status(ws) == 0
