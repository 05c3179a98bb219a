"""Host-side checks that need no GPU: the library builds and loads, exports every symbol the
header declares, and rejects bad arguments with the documented codes before any launch."""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def L():
    from paper_2403_17031_b200 import build, binding
    build.build()
    return binding.lib()


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "ppo_b200.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(ppo_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported_and_bound(L):
    from paper_2403_17031_b200 import binding
    names = _declared_functions()
    assert len(names) >= 15
    for n in names:
        assert hasattr(L, n), n
    assert set(names) == set(binding.exported_symbols())


def test_defaults_are_the_papers_table(L):
    from paper_2403_17031_b200 import binding
    from paper_2403_17031_b200.synthetic import PPOHyper
    import numpy as np
    p = binding.default_params()
    h = PPOHyper()
    for name, _ in binding.PPOParams._fields_:
        assert getattr(p, name) == (np.float32(getattr(h, name)) if isinstance(getattr(h, name), float)
                                     else getattr(h, name)), name
    assert L.ppo_version() >= 100


def test_workspace_sizes(L):
    from paper_2403_17031_b200 import binding
    assert binding.workspace_bytes(64, 53, 50304) == 256 + ((64 * 53 * 32 + 255) // 256) * 256 + ((64 * 53 * 4 + 255) // 256) * 256
    assert binding.workspace_bytes(0, 53, 50304) == 256
    assert binding.workspace_bytes(512, 53, 50304) % 256 == 0
    assert binding.lmhead_workspace_bytes(27136, 4096, 50304) % 256 == 0
    # header | 16 bytes per (row of a 128-row tile, chunk of 6 x 256 vocabulary columns) | row order | packed copy of H
    a256 = lambda x: (x + 255) // 256 * 256
    M, K, V = 1000, 512, 5000
    tiles, chunks = (M + 127) // 128, ((V + 255) // 256 + 5) // 6
    assert binding.lmhead_workspace_bytes(M, K, V) == 256 + a256(tiles * 128 * chunks * 16) + a256(M * 4) + a256(M * K * 2)
    import pytest
    import torch
    with pytest.raises(ValueError):     # the binding refuses a workspace that is too small before any call
        binding._need_workspace(torch.empty(1024, dtype=torch.uint8), binding.lmhead_workspace_bytes(M, K, V), "x")


FAKE = 0x10000   # a non-null, 256-byte aligned address that is never dereferenced on these paths


def test_argument_errors_are_returned_before_any_launch(L):
    from paper_2403_17031_b200 import binding as b
    P = C.c_void_p
    p = b.default_params()
    f = L.ppo_logprob_entropy
    ok = [P(FAKE), b.PPO_BF16, 4, 1000, 1000, P(FAKE), None, 0.7, P(FAKE), None, None, None, None]

    def call(fn, args, **repl):
        a = list(args)
        for k, v in repl.items():
            a[int(k[1:])] = v
        return fn(*a)
    assert call(f, ok, _1=7) == -5                       # dtype
    assert call(f, ok, _3=0) == -2                       # V
    assert call(f, ok, _4=999) == -2                     # pitch < V
    assert call(f, ok, _2=-1) == -2                      # rows
    assert call(f, ok, _7=0.0) == -3                     # temperature
    assert call(f, ok, _7=float("nan")) == -3
    assert call(f, ok, _0=None) == -1
    assert call(f, ok, _5=None) == -1
    assert call(f, ok, _8=None) == -1
    assert call(f, ok, _0=P(FAKE + 1)) == -4             # bf16 base must be 2-byte aligned
    assert call(f, ok, _2=0) == 0                        # empty batch is a no-op

    t = L.ppo_truncate_and_score
    okt = [P(FAKE), 4, 16, 0, 1, P(FAKE), -1.0, P(FAKE), P(FAKE), P(FAKE), P(FAKE), P(FAKE), None]
    assert call(t, okt, _4=0) == -3                      # EOS must differ from [PAD]
    assert call(t, okt, _2=0) == -2
    assert call(t, okt, _0=None) == -1
    assert call(t, okt, _1=0) == 0

    k = L.ppo_kl_rewards
    okk = [P(FAKE)] * 5 + [4, 16, 0.05, P(FAKE), P(FAKE), None]
    assert call(k, okk, _0=None) == -1
    assert call(k, okk, _8=None, _9=None) == -1
    assert call(k, okk, _6=0) == -2
    assert call(k, okk, _7=float("inf")) == -3

    g = L.ppo_gae
    okg = [P(FAKE)] * 3 + [4, 16, 1.0, 0.95, P(FAKE), P(FAKE), None]
    assert call(g, okg, _7=None) == -1
    assert call(g, okg, _4=-3) == -2
    assert call(g, okg, _5=float("nan")) == -3

    w = L.ppo_whiten
    okw = [P(FAKE), P(FAKE), 64, 1, 1e-8, P(FAKE), None, None, None]
    assert call(w, okw, _0=None) == -1
    assert call(w, okw, _2=-1) == -2
    assert call(w, okw, _4=-1.0) == -3
    assert call(w, okw, _2=0) == 0

    lf = L.ppo_loss_fwd_bwd
    okl = [P(FAKE), b.PPO_BF16, 4, 16, 1000] + [P(FAKE)] * 7 + [C.byref(p)] + [P(FAKE), P(2 * FAKE), P(FAKE),
                                                                                  None, None, None, P(FAKE), None]
    assert call(lf, okl, _1=3) == -5
    assert call(lf, okl, _2=0) == -2
    assert call(lf, okl, _4=0) == -2
    assert call(lf, okl, _19=None) == -1                 # workspace required
    assert call(lf, okl, _19=P(FAKE + 16)) == -4         # workspace must be 256-byte aligned
    assert call(lf, okl, _14=P(FAKE)) == -3              # dlogits must not alias logits
    bad = b.default_params(cliprange=-0.1)
    assert call(lf, okl, _12=C.byref(bad)) == -3
    bad = b.default_params(temperature=0.0)
    assert call(lf, okl, _12=C.byref(bad)) == -3

    ll = L.ppo_loss_from_logprob
    okll = [P(FAKE), None, 4, 16] + [P(FAKE)] * 6 + [C.byref(p)] + [P(FAKE), P(FAKE), P(FAKE), P(FAKE), None]
    assert call(ll, okll, _0=None) == -1
    assert call(ll, okll, _3=0) == -2

    assert L.ppo_set_option(b.OPT_LOSS_ROW_CACHE, 7) == -3
    assert L.ppo_set_option(99, 0) == -3
    assert L.ppo_set_option(b.OPT_LOSS_ROW_CACHE, 0) == 0
    assert L.ppo_workspace_init(None, 1024, None) == -1
    assert L.ppo_workspace_init(P(FAKE), 16, None) == -2
    assert L.ppo_workspace_init(P(FAKE + 8), 1024, None) == -4


def test_argument_errors_of_the_widened_entry_points(L):
    """ppo_step, the preference losses, the log-prob backward and the LM-head forward/backward validate their
    arguments on the host before anything is launched (no GPU needed to see the error codes)."""
    from paper_2403_17031_b200 import binding as b
    P = C.c_void_p
    p = b.default_params()

    def call(fn, args, **repl):
        a = list(args)
        for k, v in repl.items():
            a[int(k[1:])] = v
        return fn(*a)

    lb = L.ppo_logprob_bwd
    ok = [P(FAKE), b.PPO_BF16, 64, 1000, P(FAKE), P(FAKE), P(FAKE), 1.0, P(2 * FAKE), None, None, P(FAKE), None]
    assert call(lb, ok, _1=9) == -5
    assert call(lb, ok, _2=0) == -2 and call(lb, ok, _3=0) == -2
    assert call(lb, ok, _6=None) == -1 and call(lb, ok, _8=None) == -1 and call(lb, ok, _11=None) == -1
    assert call(lb, ok, _7=0.0) == -3
    assert call(lb, ok, _8=P(FAKE)) == -3                 # in place is not supported
    assert call(lb, ok, _11=P(FAKE + 64)) == -4

    lpp = L.ppo_logprob_entropy_pair
    okq = [P(FAKE), P(FAKE), b.PPO_BF16, 64, 1000, P(FAKE), None, 0.7, P(FAKE), None, P(FAKE), None, None]
    assert call(lpp, okq, _2=4) == -5 and call(lpp, okq, _4=0) == -2 and call(lpp, okq, _7=0.0) == -3
    assert call(lpp, okq, _1=None) == -1 and call(lpp, okq, _10=None) == -1 and call(lpp, okq, _3=0) == 0
    assert call(lpp, okq, _0=P(FAKE + 1)) == -4

    pw = L.ppo_pairwise_loss
    okp = [P(FAKE), P(FAKE), 8, P(FAKE), None, None, None]
    assert call(pw, okp, _2=0) == -2 and call(pw, okp, _0=None) == -1 and call(pw, okp, _3=None) == -1

    dp = L.ppo_dpo_loss
    okd = [P(FAKE)] * 6 + [8, 638, 0.05, P(FAKE), None, None, None, None, None]
    assert call(dp, okd, _6=0) == -2 and call(dp, okd, _7=0) == -2
    assert call(dp, okd, _3=None) == -1 and call(dp, okd, _9=None) == -1
    assert call(dp, okd, _8=float("nan")) == -3

    lm = L.ppo_lmhead_logprob_entropy
    okm = [P(FAKE), P(FAKE), 128, 4096, 50304, P(FAKE), None, 0.7, P(FAKE), None, None, P(FAKE), None]
    assert call(lm, okm, _3=4100) == -6                   # K must be a multiple of 64
    assert call(lm, okm, _4=50305) == -6                  # V must be a multiple of 8
    assert call(lm, okm, _7=-1.0) == -3 and call(lm, okm, _11=None) == -1 and call(lm, okm, _2=0) == 0
    assert call(lm, okm, _0=P(FAKE + 2)) == -4

    bw = L.ppo_lmhead_bwd
    okb = [P(FAKE), P(FAKE), 128, 4096, 50304, P(FAKE), None, P(FAKE), P(FAKE), 0.7, P(FAKE), None, None, P(FAKE),
           None]
    assert call(bw, okb, _2=0) == -2
    assert call(bw, okb, _3=4100) == -6 and call(bw, okb, _4=50306) == -6
    assert call(bw, okb, _7=None) == -1 and call(bw, okb, _10=None) == -1 and call(bw, okb, _13=None) == -1
    assert call(bw, okb, _9=0.0) == -3
    assert call(bw, okb, _10=P(FAKE + 8)) == -4

    io = b.PPOStepIO()
    st = L.ppo_step
    assert st(None, b.PPO_BF16, 4, 16, 1000, C.byref(p), None) == -1
    assert st(C.byref(io), b.PPO_BF16, 4, 16, 1000, C.byref(p), None) == -1      # every required buffer is NULL
    assert st(C.byref(io), b.PPO_BF16, 0, 16, 1000, C.byref(p), None) == -2
    sh = L.ppo_step_host
    assert sh(C.byref(io), None, b.PPO_BF16, 4, 16, 1000, C.byref(p), None) == -1
    assert sh(C.byref(io), C.byref(io), 5, 4, 16, 1000, C.byref(p), None) == -5


def test_binding_rejects_cpu_tensors():
    import torch
    from paper_2403_17031_b200 import binding as b
    with pytest.raises(TypeError):
        b.logprob_entropy(torch.zeros(2, 8), torch.zeros(2, dtype=torch.int32), 0.7)
    with pytest.raises(TypeError):
        b.gae(torch.zeros(2, 8), torch.zeros(2, 8), torch.zeros(2, dtype=torch.int32), 1.0, 0.95)


def test_product_does_not_import_the_oracle():
    pkg = os.path.join(ROOT, "paper_2403_17031_b200")
    for dirpath, _, files in os.walk(pkg):
        for fn in files:
            if fn.endswith((".py", ".cu", ".cuh", ".h")):
                src = open(os.path.join(dirpath, fn)).read()
                assert "oracle" not in src.lower() or fn == "synthetic.py", fn
