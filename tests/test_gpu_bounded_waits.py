"""The loss kernel may start before the kernel that produces its row order and advantages has finished and then polls
two flags in the workspace header. Every such wait is bounded. These tests make a wait run out the only way that is
harmless: a second copy of the library is compiled in which the producer never publishes one of the flags (and the
wait limit is short), so the consumer gives up, records PPO_DEV_TIMEOUT and returns. Nothing faults or hangs; the
context stays usable and the product library then computes the right result on the same buffers."""
import ctypes as C
import os

import pytest
import torch

pytestmark = pytest.mark.gpu

DEV_TIMEOUT = 4


def _load_variant(tmp, withhold):
    from paper_2403_17031_b200 import binding, build
    path = build.build_variant(os.path.join(str(tmp), "libppo_withhold%d.so" % withhold),
                               ["PPO_TEST_WITHHOLD_FLAGS=%d" % withhold, "PPO_WAIT_TRIES=512"])
    L = C.CDLL(path)
    for name in ("ppo_loss_fwd_bwd", "ppo_last_device_status", "ppo_step"):
        res, args = binding._SIGS[name]
        fn = getattr(L, name)
        fn.restype, fn.argtypes = res, args
    return L


@pytest.fixture(scope="module")
def P():
    assert torch.cuda.is_available()
    import paper_2403_17031_b200 as pkg
    from paper_2403_17031_b200 import build
    build.build()
    pkg.lib()
    return pkg


def _inputs(B, T, V):
    g = torch.Generator(device="cuda").manual_seed(11)
    r = lambda *s: torch.randn(*s, generator=g, device="cuda")
    lg = (2 * r(B, T, V)).to(torch.bfloat16)
    tok = torch.randint(0, V, (B, T), generator=g, device="cuda", dtype=torch.int32)
    L = torch.randint(1, T + 1, (B,), generator=g, device="cuda")
    mask = (torch.arange(T, device="cuda")[None] < L[:, None]).to(torch.uint8).contiguous()
    vo = r(B, T)
    return dict(lg=lg, tok=tok, mask=mask, old=(-3 + 0.2 * r(B, T)).contiguous(), adv=r(B, T), vn=(vo + 0.2 * r(B, T)).contiguous(),
                vo=vo, ret=r(B, T))


def _outputs(B, T, V, fill):
    f = lambda *s, dt=torch.float32: torch.full(s, fill, dtype=dt, device="cuda")
    return dict(losses=f(8), dlogits=f(B, T, V, dt=torch.bfloat16), dvalues=f(B, T), nlp=f(B, T), ent=f(B, T), dlp=f(B, T))


def _call_loss(L, x, o, params, ws):
    B, T, V = x["lg"].shape
    p = lambda t: C.c_void_p(t.data_ptr())
    st = C.c_void_p(torch.cuda.current_stream().cuda_stream)
    rc = L.ppo_loss_fwd_bwd(p(x["lg"]), 1, B, T, V, p(x["tok"]), p(x["mask"]), p(x["old"]), p(x["adv"]), p(x["vn"]), p(x["vo"]),
                            p(x["ret"]), C.byref(params), p(o["losses"]), p(o["dlogits"]), p(o["dvalues"]), p(o["nlp"]),
                            p(o["ent"]), p(o["dlp"]), p(ws), st)
    assert rc == 0
    code = C.c_int(0)
    assert L.ppo_last_device_status(p(ws), st, C.byref(code)) == 0      # synchronises the stream
    return code.value


@pytest.mark.parametrize("withhold", [1, 2], ids=["order_ready", "adv_ready"])
def test_a_wait_that_runs_out_is_reported_and_nothing_hangs(P, tmp_path_factory, withhold):
    B, T, V = 24, 16, 4096
    x = _inputs(B, T, V)
    params = P.default_params()
    ws = P.new_workspace(P.workspace_bytes(B, T, V))
    want = P.loss_fwd_bwd(x["lg"], x["tok"], x["mask"], x["old"], x["adv"], x["vn"], x["vo"], x["ret"], params, ws)
    torch.cuda.synchronize()
    assert P.last_device_status(ws) == 0
    L = _load_variant(tmp_path_factory.mktemp("variant"), withhold)
    o = _outputs(B, T, V, 7.0)
    status = _call_loss(L, x, o, params, ws)
    assert status & DEV_TIMEOUT, status
    if withhold == 1:
        # the row order was never announced: the kernel must not have indexed anything through it
        for k in ("dlogits", "dvalues", "nlp", "ent", "dlp"):
            assert bool((o[k] == 7).all()), k
        assert bool(torch.isnan(o["losses"]).all())
    # the context is alive and the same buffers give the right result through the product library
    o2 = {"losses": o["losses"], "dlogits": o["dlogits"], "dvalues": o["dvalues"], "new_logprob": o["nlp"],
          "entropy": o["ent"], "dlogprob": o["dlp"]}
    P.loss_fwd_bwd(x["lg"], x["tok"], x["mask"], x["old"], x["adv"], x["vn"], x["vo"], x["ret"], params, ws, out=o2)
    torch.cuda.synchronize()
    assert P.last_device_status(ws) == 0
    for k in ("losses", "dlogits", "dvalues", "new_logprob", "entropy", "dlogprob"):
        assert torch.equal(o2[k], want[k]), k
