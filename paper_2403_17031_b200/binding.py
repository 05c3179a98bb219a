"""ctypes binding of libppo_b200.so. Every function here only marshals arguments: it checks
that tensors are CUDA, contiguous and of the documented dtype, allocates outputs with torch,
passes raw device pointers and the current CUDA stream to the C ABI, and raises PPOError on a
non-zero status. No step of the path is computed in Python or by torch kernels."""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libppo_b200.so")

PPO_F32, PPO_BF16 = 0, 1
OPT_LOSS_ROW_CACHE = 1
OPT_ROW_ENGINE = 2
LOSS_NAMES = ("pg_loss", "vf_loss", "loss", "approx_kl", "pg_clipfrac", "vf_clipfrac", "entropy", "n")
DEV_BAD_TOKEN, DEV_EMPTY_MASK, DEV_TIMEOUT, DEV_BAD_ROW, DEV_BAD_REUSE = 1, 2, 4, 8, 16

_ERR = {-1: "PPO_ERR_NULL", -2: "PPO_ERR_SHAPE", -3: "PPO_ERR_PARAM", -4: "PPO_ERR_ALIGN", -5: "PPO_ERR_DTYPE",
        -6: "PPO_ERR_UNSUPPORTED"}


class PPOError(RuntimeError):
    def __init__(self, fn: str, code: int):
        self.code = code
        what = _ERR.get(code, "cudaError %d" % code if code > 0 else "status %d" % code)
        super().__init__("%s failed: %s" % (fn, what))


class PPOParams(C.Structure):
    _fields_ = [("temperature", C.c_float), ("kl_coef", C.c_float), ("gamma", C.c_float), ("lam", C.c_float),
                ("cliprange", C.c_float), ("cliprange_value", C.c_float), ("vf_coef", C.c_float),
                ("no_eos_score", C.c_float), ("whiten_eps", C.c_float), ("eos_id", C.c_int32),
                ("pad_id", C.c_int32), ("whiten_rewards", C.c_int32)]


class PPOStepIO(C.Structure):
    """Mirror of ppo_step_io: every buffer of one iteration (all pointers in one memory space)."""
    _in = ("policy_logits", "ref_logits", "loss_logits", "responses", "scores", "values", "values_new", "old_logprob")
    _out = ("responses_out", "eos_index", "seq_len", "mask", "scores_out", "logprob", "entropy", "ref_logprob", "kl",
            "rewards", "advantages", "returns", "advantages_whitened", "whiten_stats", "losses", "dlogits", "dvalues",
            "new_logprob", "new_entropy", "dlogprob", "workspace")
    _fields_ = [(n, C.c_void_p) for n in _in + _out]

    @classmethod
    def from_tensors(cls, tensors: dict, cuda: bool):
        """Fill from {field: tensor or None}; checks that every tensor is contiguous and on the right side."""
        io = cls()
        for name in cls._in + cls._out:
            t = tensors.get(name)
            if t is None:
                setattr(io, name, None)
                continue
            if t.is_cuda != cuda or not t.is_contiguous():
                raise TypeError("%s must be a contiguous %s tensor" % (name, "CUDA" if cuda else "CPU"))
            setattr(io, name, t.data_ptr())
        return io


class LMHeadStepIO(C.Structure):
    """Mirror of ppo_lmhead_step_io (all pointers in one memory space)."""
    _in = ("H", "W", "W_ref", "responses", "scores", "values", "values_new", "old_logprob")
    _out = ("responses_out", "eos_index", "seq_len", "mask", "scores_out", "logprob", "entropy", "lse", "ref_logprob",
            "kl", "rewards", "advantages", "returns", "advantages_whitened", "whiten_stats", "losses", "dlogprob",
            "dvalues", "workspace")
    _fields_ = [(n, C.c_void_p) for n in _in + _out]
    from_tensors = classmethod(PPOStepIO.from_tensors.__func__)


_lib = None

_SIGS = {
    "ppo_default_params": (None, [C.POINTER(PPOParams)]),
    "ppo_version": (C.c_int, []),
    "ppo_set_option": (C.c_int, [C.c_int, C.c_int]),
    "ppo_workspace_bytes": (C.c_size_t, [C.c_int32, C.c_int32, C.c_int64]),
    "ppo_lmhead_workspace_bytes": (C.c_size_t, [C.c_int64, C.c_int64, C.c_int64]),
    "ppo_workspace_init": (C.c_int, [C.c_void_p, C.c_size_t, C.c_void_p]),
    "ppo_last_device_status": (C.c_int, [C.c_void_p, C.c_void_p, C.POINTER(C.c_int)]),
    "ppo_logprob_entropy": (C.c_int, [C.c_void_p, C.c_int, C.c_int64, C.c_int64, C.c_int64, C.c_void_p, C.c_void_p,
                                      C.c_float, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]),
    "ppo_truncate_and_score": (C.c_int, [C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_void_p,
                                         C.c_float, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                                         C.c_void_p]),
    "ppo_kl_rewards": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_int32,
                                 C.c_float, C.c_void_p, C.c_void_p, C.c_void_p]),
    "ppo_rollout_curves": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_float, C.c_void_p,
                                     C.c_void_p]),
    "ppo_gae": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_float, C.c_float,
                          C.c_void_p, C.c_void_p, C.c_void_p]),
    "ppo_whiten": (C.c_int, [C.c_void_p, C.c_void_p, C.c_int64, C.c_int, C.c_float, C.c_void_p, C.c_void_p,
                             C.c_void_p, C.c_void_p]),
    "ppo_loss_fwd_bwd": (C.c_int, [C.c_void_p, C.c_int, C.c_int32, C.c_int32, C.c_int64] + [C.c_void_p] * 7 +
                         [C.POINTER(PPOParams)] + [C.c_void_p] * 8),
    "ppo_loss_fwd_bwd_next_epoch": (C.c_int, [C.c_void_p, C.c_int, C.c_int32, C.c_int32, C.c_int64] +
                                    [C.c_void_p] * 7 + [C.POINTER(PPOParams)] + [C.c_void_p] * 8),
    "ppo_loss_from_logprob": (C.c_int, [C.c_void_p, C.c_void_p, C.c_int32, C.c_int32] + [C.c_void_p] * 6 +
                              [C.POINTER(PPOParams)] + [C.c_void_p] * 5),
    "ppo_loss_from_logprob_static": (C.c_int, [C.c_void_p, C.c_void_p, C.c_int32, C.c_int32] + [C.c_void_p] * 6 +
                                     [C.POINTER(PPOParams)] + [C.c_void_p] * 4),
    "ppo_step": (C.c_int, [C.POINTER(PPOStepIO), C.c_int, C.c_int32, C.c_int32, C.c_int64, C.POINTER(PPOParams),
                           C.c_void_p]),
    "ppo_step_host": (C.c_int, [C.POINTER(PPOStepIO), C.POINTER(PPOStepIO), C.c_int, C.c_int32, C.c_int32, C.c_int64,
                                C.POINTER(PPOParams), C.c_void_p]),
    "ppo_lmhead_step": (C.c_int, [C.POINTER(LMHeadStepIO), C.c_int32, C.c_int32, C.c_int64, C.c_int64,
                                  C.POINTER(PPOParams), C.c_void_p]),
    "ppo_lmhead_step_host": (C.c_int, [C.POINTER(LMHeadStepIO), C.POINTER(LMHeadStepIO), C.c_int32, C.c_int32,
                                       C.c_int64, C.c_int64, C.POINTER(PPOParams), C.c_void_p]),
    "ppo_logprob_entropy_pair": (C.c_int, [C.c_void_p, C.c_void_p, C.c_int, C.c_int64, C.c_int64, C.c_void_p,
                                           C.c_void_p, C.c_float, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                                           C.c_void_p]),
    "ppo_sample_logprob_entropy": (C.c_int, [C.c_void_p, C.c_int, C.c_int64, C.c_int64, C.c_int64, C.c_float,
                                             C.c_uint64, C.c_uint64, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                                             C.c_void_p, C.c_void_p]),
    "ppo_lmhead_bwd": (C.c_int, [C.c_void_p, C.c_void_p, C.c_int64, C.c_int64, C.c_int64, C.c_void_p, C.c_void_p,
                                 C.c_void_p, C.c_void_p, C.c_float, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                                 C.c_void_p]),
    "ppo_logprob_bwd": (C.c_int, [C.c_void_p, C.c_int, C.c_int64, C.c_int64, C.c_void_p, C.c_void_p, C.c_void_p,
                                  C.c_float, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]),
    "ppo_pairwise_loss": (C.c_int, [C.c_void_p, C.c_void_p, C.c_int64, C.c_void_p, C.c_void_p, C.c_void_p,
                                    C.c_void_p]),
    "ppo_dpo_loss": (C.c_int, [C.c_void_p] * 6 + [C.c_int64, C.c_int32, C.c_float] + [C.c_void_p] * 6),
    "ppo_lmhead_logprob_entropy": (C.c_int, [C.c_void_p, C.c_void_p, C.c_int64, C.c_int64, C.c_int64, C.c_void_p,
                                             C.c_void_p, C.c_float, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                                             C.c_void_p]),
}


def lib():
    """Load the CUDA library (built in-tree by paper_2403_17031_b200/build.py)."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise ImportError("%s is missing: run `python -m paper_2403_17031_b200.build` (nvcc, sm_100a). "
                              "There is no fallback path." % _LIB_PATH)
        L = C.CDLL(_LIB_PATH)
        for name, (res, args) in _SIGS.items():
            fn = getattr(L, name)
            fn.restype = res
            fn.argtypes = args
        _lib = L
    return _lib


def exported_symbols():
    return tuple(_SIGS.keys())


# ---------------------------------------------------------------- helpers
def _stream() -> C.c_void_p:
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def _ptr(t: Optional[torch.Tensor], dtype=None, name="tensor"):
    if t is None:
        return None
    if not t.is_cuda:
        raise TypeError("%s must be a CUDA tensor" % name)
    if not t.is_contiguous():
        raise TypeError("%s must be contiguous" % name)
    if dtype is not None and t.dtype != dtype:
        raise TypeError("%s must have dtype %s, got %s" % (name, dtype, t.dtype))
    return C.c_void_p(t.data_ptr())


def _logits_dtype(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return PPO_F32
    if t.dtype == torch.bfloat16:
        return PPO_BF16
    raise TypeError("logits must be float32 or bfloat16, got %s" % t.dtype)


def _check(fn: str, rc: int):
    if rc != 0:
        raise PPOError(fn, rc)


def version() -> int:
    return int(lib().ppo_version())


def default_params(pad_id: Optional[int] = None, **overrides) -> PPOParams:
    p = PPOParams()
    lib().ppo_default_params(C.byref(p))
    if pad_id is not None:
        p.pad_id = pad_id
    for k, v in overrides.items():
        setattr(p, k, v)
    return p


def params_from(h) -> PPOParams:
    """PPOParams from any object with the same attribute names (e.g. synthetic.PPOHyper)."""
    p = PPOParams()
    for name, ctype in PPOParams._fields_:
        setattr(p, name, int(getattr(h, name)) if ctype is C.c_int32 else getattr(h, name))
    return p


def set_option(key: int, value: int) -> None:
    _check("ppo_set_option", lib().ppo_set_option(key, value))


def workspace_bytes(B: int, T: int, V: int) -> int:
    return int(lib().ppo_workspace_bytes(B, T, V))


def lmhead_workspace_bytes(M: int, K: int, V: int) -> int:
    return int(lib().ppo_lmhead_workspace_bytes(M, K, V))


def _need_workspace(workspace: torch.Tensor, nbytes: int, what: str) -> None:
    """The C entry points take no workspace size; refuse a buffer that is too small before the call."""
    if workspace is None or workspace.numel() * workspace.element_size() < nbytes:
        raise ValueError("%s needs a workspace of %d bytes (lmhead_workspace_bytes)" % (what, nbytes))


def new_workspace(nbytes: int, device="cuda") -> torch.Tensor:
    """Allocate (torch) and clear a workspace of at least `nbytes`."""
    ws = torch.empty(max(int(nbytes), 256), dtype=torch.uint8, device=device)
    assert ws.data_ptr() % 256 == 0
    _check("ppo_workspace_init", lib().ppo_workspace_init(_ptr(ws), ws.numel(), _stream()))
    return ws


def last_device_status(workspace: torch.Tensor) -> int:
    st = C.c_int(0)
    _check("ppo_last_device_status", lib().ppo_last_device_status(_ptr(workspace), _stream(), C.byref(st)))
    return int(st.value)


# ---------------------------------------------------------------- the path
def logprob_entropy(logits: torch.Tensor, tokens: torch.Tensor, temperature: float,
                    mask: Optional[torch.Tensor] = None, workspace: Optional[torch.Tensor] = None,
                    want_entropy: bool = True, want_lse: bool = False, out=None):
    """logits [..., V] (last dim contiguous rows), tokens [...] int32. Returns (logprob, entropy, lse)."""
    V = logits.shape[-1]
    rows = logits.numel() // V if V else 0
    lg2 = logits.reshape(rows, V) if logits.is_contiguous() else logits
    if lg2.dim() != 2 or lg2.stride(1) != 1:
        raise TypeError("logits rows must be contiguous")
    stride = lg2.stride(0) if rows > 1 else V
    shape = tokens.shape
    if out is None:
        lp = torch.empty(shape, dtype=torch.float32, device=logits.device)
        ent = torch.empty(shape, dtype=torch.float32, device=logits.device) if want_entropy else None
        lse = torch.empty(shape, dtype=torch.float32, device=logits.device) if want_lse else None
    else:
        lp, ent, lse = out
    if not lg2.is_cuda:
        raise TypeError("logits must be a CUDA tensor")
    rc = lib().ppo_logprob_entropy(C.c_void_p(lg2.data_ptr()), _logits_dtype(lg2), rows, V, stride,
                                   _ptr(tokens, torch.int32, "tokens"), _ptr(mask, torch.uint8, "mask"),
                                   float(temperature), _ptr(lp, torch.float32), _ptr(ent, torch.float32),
                                   _ptr(lse, torch.float32), _ptr(workspace), _stream())
    _check("ppo_logprob_entropy", rc)
    return lp, ent, lse


def truncate_and_score(responses: torch.Tensor, scores: torch.Tensor, eos_id: int, pad_id: int,
                       no_eos_score: float, out=None):
    """Returns (responses_out, eos_index, seq_len, mask, scores_out)."""
    B, T = responses.shape
    dev = responses.device
    if out is None:
        out = (torch.empty((B, T), dtype=torch.int32, device=dev), torch.empty((B,), dtype=torch.int32, device=dev),
               torch.empty((B,), dtype=torch.int32, device=dev), torch.empty((B, T), dtype=torch.uint8, device=dev),
               torch.empty((B,), dtype=torch.float32, device=dev))
    ro, ei, sl, m, so = out
    rc = lib().ppo_truncate_and_score(_ptr(responses, torch.int32, "responses"), B, T, eos_id, pad_id,
                                      _ptr(scores, torch.float32, "scores"), float(no_eos_score),
                                      _ptr(ro, torch.int32), _ptr(ei, torch.int32), _ptr(sl, torch.int32),
                                      _ptr(m, torch.uint8), _ptr(so, torch.float32), _stream())
    _check("ppo_truncate_and_score", rc)
    return out


def kl_rewards(logprob, ref_logprob, mask, seq_len, scores, kl_coef: float, out=None):
    B, T = logprob.shape
    if out is None:
        out = (torch.empty_like(logprob), torch.empty_like(logprob))
    kl, rew = out
    rc = lib().ppo_kl_rewards(_ptr(logprob, torch.float32), _ptr(ref_logprob, torch.float32),
                              _ptr(mask, torch.uint8), _ptr(seq_len, torch.int32), _ptr(scores, torch.float32),
                              B, T, float(kl_coef), _ptr(kl, torch.float32), _ptr(rew, torch.float32), _stream())
    _check("ppo_kl_rewards", rc)
    return out


def rollout_curves(kl, mask, scores, kl_coef: float, out=None):
    """Mean RLHF reward, mean summed per-token KL, mean score of a batch; returns a [3] f32 tensor."""
    B, T = kl.shape
    if out is None:
        out = torch.empty(3, dtype=torch.float32, device=kl.device)
    rc = lib().ppo_rollout_curves(_ptr(kl, torch.float32), None if mask is None else _ptr(mask, torch.uint8),
                                  _ptr(scores, torch.float32), B, T, float(kl_coef), _ptr(out, torch.float32), _stream())
    _check("ppo_rollout_curves", rc)
    return out


def gae(rewards, values, seq_len, gamma: float, lam: float, out=None):
    B, T = rewards.shape
    if out is None:
        out = (torch.empty_like(rewards), torch.empty_like(rewards))
    adv, ret = out
    rc = lib().ppo_gae(_ptr(rewards, torch.float32), _ptr(values, torch.float32), _ptr(seq_len, torch.int32), B, T,
                       float(gamma), float(lam), _ptr(adv, torch.float32), _ptr(ret, torch.float32), _stream())
    _check("ppo_gae", rc)
    return out


def whiten(x, mask=None, shift_mean: bool = True, eps: float = 1e-8, workspace=None, out=None, stats=None):
    if out is None:
        out = torch.empty_like(x)
    if stats is None:
        stats = torch.empty(3, dtype=torch.float32, device=x.device)
    rc = lib().ppo_whiten(_ptr(x, torch.float32), _ptr(mask, torch.uint8), x.numel(), 1 if shift_mean else 0,
                          float(eps), _ptr(out, torch.float32), _ptr(stats, torch.float32), _ptr(workspace),
                          _stream())
    _check("ppo_whiten", rc)
    return out, stats


def loss_fwd_bwd(logits, tokens, mask, old_logprob, advantages, values_new, values_old, returns,
                 params: PPOParams, workspace, want_dlogits: bool = True, want_aux: bool = True, out=None,
                 next_epoch: bool = False):
    """Returns dict(losses[8], dlogits, dvalues, new_logprob, entropy, dlogprob). next_epoch: this call follows a
    loss call (or step) on the same workspace with the same mask tensor and reuses its row order."""
    B, T, V = logits.shape
    dev = logits.device
    if out is None:
        out = {
            "losses": torch.empty(8, dtype=torch.float32, device=dev),
            "dlogits": torch.empty_like(logits) if want_dlogits else None,
            "dvalues": torch.empty((B, T), dtype=torch.float32, device=dev),
            "new_logprob": torch.empty((B, T), dtype=torch.float32, device=dev) if want_aux else None,
            "entropy": torch.empty((B, T), dtype=torch.float32, device=dev) if want_aux else None,
            "dlogprob": torch.empty((B, T), dtype=torch.float32, device=dev) if want_aux else None,
        }
    f32 = torch.float32
    fn = lib().ppo_loss_fwd_bwd_next_epoch if next_epoch else lib().ppo_loss_fwd_bwd
    rc = fn(_ptr(logits, None, "logits"), _logits_dtype(logits), B, T, V, _ptr(tokens, torch.int32, "tokens"),
            _ptr(mask, torch.uint8, "mask"), _ptr(old_logprob, f32), _ptr(advantages, f32), _ptr(values_new, f32),
            _ptr(values_old, f32), _ptr(returns, f32), C.byref(params), _ptr(out["losses"], f32),
            _ptr(out["dlogits"], logits.dtype), _ptr(out["dvalues"], f32), _ptr(out["new_logprob"], f32),
            _ptr(out["entropy"], f32), _ptr(out["dlogprob"], f32), _ptr(workspace), _stream())
    _check("ppo_loss_fwd_bwd", rc)
    return out


def loss_from_logprob(new_logprob, entropy, mask, old_logprob, advantages, values_new, values_old, returns,
                      params: PPOParams, workspace, out=None):
    B, T = new_logprob.shape
    dev = new_logprob.device
    f32 = torch.float32
    if out is None:
        out = {"losses": torch.empty(8, dtype=f32, device=dev), "dlogprob": torch.empty((B, T), dtype=f32, device=dev),
               "dvalues": torch.empty((B, T), dtype=f32, device=dev)}
    rc = lib().ppo_loss_from_logprob(_ptr(new_logprob, f32), _ptr(entropy, f32), B, T, _ptr(mask, torch.uint8),
                                     _ptr(old_logprob, f32), _ptr(advantages, f32), _ptr(values_new, f32),
                                     _ptr(values_old, f32), _ptr(returns, f32), C.byref(params),
                                     _ptr(out["losses"], f32), _ptr(out["dlogprob"], f32), _ptr(out["dvalues"], f32),
                                     _ptr(workspace), _stream())
    _check("ppo_loss_from_logprob", rc)
    return out


def step(io: PPOStepIO, dtype: torch.dtype, B: int, T: int, V: int, params: PPOParams) -> None:
    """The whole path in one C call on device buffers (asynchronous on the current stream)."""
    code = PPO_F32 if dtype == torch.float32 else PPO_BF16
    _check("ppo_step", lib().ppo_step(C.byref(io), code, B, T, V, C.byref(params), _stream()))


def step_host(host: PPOStepIO, dev: PPOStepIO, dtype: torch.dtype, B: int, T: int, V: int, params: PPOParams) -> None:
    """Host buffers in, host buffers out: copies, the whole path, copies back, stream synchronised."""
    code = PPO_F32 if dtype == torch.float32 else PPO_BF16
    _check("ppo_step_host", lib().ppo_step_host(C.byref(host), C.byref(dev), code, B, T, V, C.byref(params), _stream()))


def lmhead_step(io: LMHeadStepIO, B: int, T: int, K: int, V: int, params: PPOParams) -> None:
    """The fused-LM-head config in one C call on device buffers (asynchronous on the current stream)."""
    _check("ppo_lmhead_step", lib().ppo_lmhead_step(C.byref(io), B, T, K, V, C.byref(params), _stream()))


def lmhead_step_host(host: LMHeadStepIO, dev: LMHeadStepIO, B: int, T: int, K: int, V: int, params: PPOParams) -> None:
    """Host buffers in, host buffers out: copies, the fused-LM-head path, copies back, stream synchronised."""
    _check("ppo_lmhead_step_host", lib().ppo_lmhead_step_host(C.byref(host), C.byref(dev), B, T, K, V, C.byref(params),
                                                               _stream()))


STATIC_MAX_TOKENS = 32768


def loss_from_logprob_static(new_logprob, entropy, mask, old_logprob, advantages, values_new, values_old, returns,
                             params: PPOParams, out):
    """Allocation-free variant of loss_from_logprob: scratch is built into the library, and `out`
    (dict with preallocated losses[8], dlogprob, dvalues) is mandatory so that nothing here allocates."""
    B, T = new_logprob.shape
    f32 = torch.float32
    rc = lib().ppo_loss_from_logprob_static(_ptr(new_logprob, f32), _ptr(entropy, f32), B, T, _ptr(mask, torch.uint8),
                                            _ptr(old_logprob, f32), _ptr(advantages, f32), _ptr(values_new, f32),
                                            _ptr(values_old, f32), _ptr(returns, f32), C.byref(params),
                                            _ptr(out["losses"], f32), _ptr(out["dlogprob"], f32),
                                            _ptr(out["dvalues"], f32), _stream())
    _check("ppo_loss_from_logprob_static", rc)
    return out


def lmhead_logprob_entropy(H, W, tokens, temperature: float, workspace, mask=None, want_lse: bool = True,
                           out=None):
    M, K = H.shape
    K2, V = W.shape
    if K != K2:
        raise ValueError("H [M,K] and W [K,V] disagree on K")
    dev = H.device
    if out is None:
        out = (torch.empty(M, dtype=torch.float32, device=dev), torch.empty(M, dtype=torch.float32, device=dev),
               torch.empty(M, dtype=torch.float32, device=dev) if want_lse else None)
    lp, ent, lse = out
    _need_workspace(workspace, lmhead_workspace_bytes(M, K, V), "lmhead_logprob_entropy")
    rc = lib().ppo_lmhead_logprob_entropy(_ptr(H, torch.bfloat16, "H"), _ptr(W, torch.bfloat16, "W"), M, K, V,
                                          _ptr(tokens, torch.int32, "tokens"), _ptr(mask, torch.uint8),
                                          float(temperature), _ptr(lp, torch.float32), _ptr(ent, torch.float32),
                                          _ptr(lse, torch.float32), _ptr(workspace), _stream())
    _check("ppo_lmhead_logprob_entropy", rc)
    return out


def logprob_bwd(logits, tokens, mask, dlogprob, temperature: float, workspace, dlogits=None, want_aux: bool = False):
    """Gradient on token log-probs -> gradient on the logits [..., V] (rows with mask 0: zeros, never read).
    Returns dict(dlogits[, new_logprob, entropy])."""
    V = logits.shape[-1]
    rows = logits.numel() // V
    if dlogits is None:
        dlogits = torch.empty_like(logits)
    out = {"dlogits": dlogits}
    if want_aux:
        out["new_logprob"] = torch.empty(tokens.shape, dtype=torch.float32, device=logits.device)
        out["entropy"] = torch.empty(tokens.shape, dtype=torch.float32, device=logits.device)
    rc = lib().ppo_logprob_bwd(_ptr(logits), _logits_dtype(logits), rows, V, _ptr(tokens, torch.int32),
                               _ptr(mask, torch.uint8), _ptr(dlogprob, torch.float32), float(temperature),
                               _ptr(dlogits, logits.dtype), _ptr(out.get("new_logprob")), _ptr(out.get("entropy")),
                               _ptr(workspace), _stream())
    _check("ppo_logprob_bwd", rc)
    return out


def pairwise_loss(reward_chosen, reward_rejected, want_grad: bool = True):
    """Reward-model loss of a batch of pairs. Returns dict(out4 = [loss, accuracy, mean r_c, mean r_r][, dr_c, dr_r])."""
    P = reward_chosen.numel()
    o = {"out4": torch.empty(4, dtype=torch.float32, device=reward_chosen.device)}
    if want_grad:
        o["dr_c"], o["dr_r"] = torch.empty_like(reward_chosen), torch.empty_like(reward_rejected)
    rc = lib().ppo_pairwise_loss(_ptr(reward_chosen, torch.float32), _ptr(reward_rejected, torch.float32), P,
                                 _ptr(o["out4"]), _ptr(o.get("dr_c")), _ptr(o.get("dr_r")), _stream())
    _check("ppo_pairwise_loss", rc)
    return o


def dpo_loss(lp_c, lp_r, ref_c, ref_r, mask_c, mask_r, beta: float, out=None):
    """DPO loss of P pairs from token log-probs [P,T]. Returns dict(out4 = [loss, accuracy, mean implicit reward
    chosen, rejected], reward_c, reward_r [P], dlp_c, dlp_r [P,T])."""
    P, T = lp_c.shape
    if out is None:
        dev = lp_c.device
        out = {"out4": torch.empty(4, dtype=torch.float32, device=dev),
               "reward_c": torch.empty(P, dtype=torch.float32, device=dev),
               "reward_r": torch.empty(P, dtype=torch.float32, device=dev),
               "dlp_c": torch.empty_like(lp_c), "dlp_r": torch.empty_like(lp_r)}
    rc = lib().ppo_dpo_loss(_ptr(lp_c, torch.float32), _ptr(lp_r, torch.float32), _ptr(ref_c, torch.float32),
                            _ptr(ref_r, torch.float32), _ptr(mask_c, torch.uint8), _ptr(mask_r, torch.uint8), P, T,
                            float(beta), _ptr(out["out4"]), _ptr(out["reward_c"]), _ptr(out["reward_r"]),
                            _ptr(out["dlp_c"]), _ptr(out["dlp_r"]), _stream())
    _check("ppo_dpo_loss", rc)
    return out


def lmhead_bwd(H, W, tokens, lse, dlogprob, temperature: float, workspace, mask=None, dlogits=None,
               want_dH: bool = True, want_dW: bool = True, out=None):
    """Backward of the fused LM head. Returns dict(dlogits [M,V], dH [M,K] | None, dW [K,V] | None), all bf16."""
    M, K = H.shape
    V = W.shape[1]
    if out is None:
        out = {"dlogits": dlogits if dlogits is not None else torch.empty((M, V), dtype=torch.bfloat16, device=H.device),
               "dH": torch.empty_like(H) if want_dH else None, "dW": torch.empty_like(W) if want_dW else None}
    _need_workspace(workspace, lmhead_workspace_bytes(M, K, V), "lmhead_bwd")
    rc = lib().ppo_lmhead_bwd(_ptr(H, torch.bfloat16), _ptr(W, torch.bfloat16), M, K, V, _ptr(tokens, torch.int32),
                              _ptr(mask, torch.uint8), _ptr(lse, torch.float32), _ptr(dlogprob, torch.float32),
                              float(temperature), _ptr(out["dlogits"], torch.bfloat16), _ptr(out["dH"]),
                              _ptr(out["dW"]), _ptr(workspace), _stream())
    _check("ppo_lmhead_bwd", rc)
    return out


def sample_logprob_entropy(logits: torch.Tensor, temperature: float, seed: int, offset: int = 0, workspace=None,
                           want_entropy: bool = True, want_lse: bool = False, out=None):
    """Draw one token per row of logits [..., V] at the given temperature; returns (tokens, logprob, entropy, lse)."""
    V = logits.shape[-1]
    rows = logits.numel() // V
    lg2 = logits.reshape(rows, V) if logits.is_contiguous() else logits
    if lg2.dim() != 2 or lg2.stride(1) != 1:
        raise TypeError("logits rows must be contiguous")
    stride = lg2.stride(0) if rows > 1 else V
    shape = logits.shape[:-1]
    if out is None:
        dev = logits.device
        out = (torch.empty(shape, dtype=torch.int32, device=dev), torch.empty(shape, dtype=torch.float32, device=dev),
               torch.empty(shape, dtype=torch.float32, device=dev) if want_entropy else None,
               torch.empty(shape, dtype=torch.float32, device=dev) if want_lse else None)
    tok, lp, ent, lse = out
    if not lg2.is_cuda:
        raise TypeError("logits must be a CUDA tensor")
    rc = lib().ppo_sample_logprob_entropy(C.c_void_p(lg2.data_ptr()), _logits_dtype(lg2), rows, V, stride,
                                          float(temperature), int(seed) & (2 ** 64 - 1), int(offset) & (2 ** 64 - 1),
                                          _ptr(tok, torch.int32), _ptr(lp, torch.float32), _ptr(ent, torch.float32),
                                          _ptr(lse, torch.float32), _ptr(workspace), _stream())
    _check("ppo_sample_logprob_entropy", rc)
    return tok, lp, ent, lse


def logprob_entropy_pair(policy_logits, ref_logits, tokens, temperature: float, mask=None, workspace=None,
                         want_entropy: bool = True, out=None):
    """Step 1 for policy and reference logits [..., V] (contiguous) in one launch. Returns (logprob, entropy, ref_logprob)."""
    V = policy_logits.shape[-1]
    rows = policy_logits.numel() // V
    if ref_logits.shape != policy_logits.shape or ref_logits.dtype != policy_logits.dtype:
        raise TypeError("policy and reference logits must have the same shape and dtype")
    if out is None:
        dev = policy_logits.device
        out = (torch.empty(tokens.shape, dtype=torch.float32, device=dev),
               torch.empty(tokens.shape, dtype=torch.float32, device=dev) if want_entropy else None,
               torch.empty(tokens.shape, dtype=torch.float32, device=dev))
    lp, ent, rlp = out
    rc = lib().ppo_logprob_entropy_pair(_ptr(policy_logits), _ptr(ref_logits), _logits_dtype(policy_logits), rows, V,
                                        _ptr(tokens, torch.int32), _ptr(mask, torch.uint8), float(temperature),
                                        _ptr(lp, torch.float32), _ptr(ent, torch.float32), _ptr(rlp, torch.float32),
                                        _ptr(workspace), _stream())
    _check("ppo_logprob_entropy_pair", rc)
    return lp, ent, rlp
