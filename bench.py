#!/usr/bin/env python
"""Benchmark of the per-token PPO hot path (arXiv 2403.17031) on B200.

One "step" = one pass of the whole path over one synthetic batch: EOS trick, log-prob/entropy of
policy and reference logits, KL rewards, GAE, advantage whitening, clipped losses + gradients
(ppo_step: 3 kernel launches). Prints ONE JSON line (rank 0).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--config 1|2|3|4|5|6] [--impl ours|reference|plumbing]

Headline workload: config 2, the full PPO batch (B=512, T=53, V=50304, bf16). After its timed region the
same process runs configs 1, 3 and 4 for a bounded number of steps and reports them under config.others.
The K-step block is repeated until the timed region is long enough for the clocks to be sampled; the
reported time per step is that of the median block.

--gpus N > 1 without a launcher: this script starts N ranks itself (torch.distributed.run, one rank per GPU,
NCCL); under a launcher (WORLD_SIZE set) it is one of the ranks. Every rank runs the same per-GPU batch shape on
its own seeded batch (weak scaling, no data-path collective); only the time is reduced (max over ranks).

--impl reference times the fp64 CPU oracle (the only "reference" this work has) on the host cores, on a bounded
sample of the same workload per step. --impl plumbing checks the multi-rank launch and the time reduction alone
(gloo on CPU when there is no GPU; no kernel runs).
"""
from __future__ import annotations

import argparse
import hashlib
import json
import math
import os
import socket
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import torch  # noqa: E402

LAUNCHES_PER_STEP = 3   # ppo_step: logprob pair (policy + reference), rollout (token-level steps + loss prologue), row_engine (loss)
TIMED_REGION_TARGET_S = 0.6   # the K-step block is repeated until the timed region is about this long

# DRAM bytes of one launch of the loss kernel come from a stored ncu capture; they are only reported while the
# kernel's sources are the ones that were captured
_TRAFFIC_FILE = os.path.join(ROOT, "profiles", "loss_kernel_dram_traffic.json")
_LOSS_KERNEL_SOURCES = ("ppo_rows_bulk.cu", "ppo_rows.cuh", "ppo_common.cuh")


def _loss_kernel_hash():
    """Hash of the loss kernel's sources with comments and white space taken out (a comment edit changes no kernel)."""
    import re
    h = hashlib.sha256()
    for name in _LOSS_KERNEL_SOURCES:
        with open(os.path.join(ROOT, "paper_2403_17031_b200", "csrc", name), "r") as f:
            text = f.read()
        text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
        text = re.sub(r"//[^\n]*", "", text)
        h.update("".join(text.split()).encode())
    return h.hexdigest()


def _ncu_traffic(key: str, read_bytes: float, write_bytes: float):
    """DRAM bytes (read + write) of one launch with the given algorithmic read / write bytes, from the stored capture
    of workload `key` (taken on a cut of the batch): reads scale with the rows read, writes with the rows written, and
    the tail of the write stream that was still in L2 when the captured launch ended is the same at any size. None
    without a capture of the current kernel."""
    try:
        d = json.load(open(_TRAFFIC_FILE))
        e = d["captures"][key]
        if d["sources_sha256"] != _loss_kernel_hash():
            return None
        in_l2 = e["algorithmic_bytes_write"] - e["dram_bytes_write"]
        return e["dram_bytes_read"] * read_bytes / e["algorithmic_bytes_read"] + max(write_bytes - in_l2, 0.0)
    except Exception:
        return None


def _peaks(key="hbm_gbs", fallback=6650.0):
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        try:
            d = json.load(open(path))
            return float(d[key]), "measured"
        except Exception:
            pass
    return fallback, "fallback"


class ClockSampler:
    """Samples SM clock and throttle reasons of one GPU through NVML while the timed region runs."""

    def __init__(self, device_index: int, period_s: float = 0.01):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        self._period = period_s
        self._h = None
        try:
            import pynvml
            self._nv = pynvml
            pynvml.nvmlInit()
            uuid = str(torch.cuda.get_device_properties(device_index).uuid)
            h = None
            for cand in ("GPU-" + uuid, uuid):
                try:
                    h = pynvml.nvmlDeviceGetHandleByUUID(cand.encode() if isinstance(cand, str) else cand)
                    break
                except Exception:
                    try:
                        h = pynvml.nvmlDeviceGetHandleByUUID(cand)
                        break
                    except Exception:
                        h = None
            if h is None:
                h = pynvml.nvmlDeviceGetHandleByIndex(device_index)
            self._h = h
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self._h = None

    def _reason_names(self, bits: int):
        nv = self._nv
        table = {
            "sw_power_cap": getattr(nv, "nvmlClocksThrottleReasonSwPowerCap", 0x4),
            "hw_slowdown": getattr(nv, "nvmlClocksThrottleReasonHwSlowdown", 0x8),
            "sw_thermal_slowdown": getattr(nv, "nvmlClocksThrottleReasonSwThermalSlowdown", 0x20),
            "hw_thermal_slowdown": getattr(nv, "nvmlClocksThrottleReasonHwThermalSlowdown", 0x40),
            "hw_power_brake_slowdown": getattr(nv, "nvmlClocksThrottleReasonHwPowerBrakeSlowdown", 0x80),
        }
        return [k for k, v in table.items() if bits & v]

    def _run(self):
        nv = self._nv
        while not self._stop.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM)))
                try:
                    bits = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self._h))
                except Exception:
                    bits = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self._h))
                self.reasons.update(self._reason_names(bits))
            except Exception:
                pass
            self._stop.wait(self._period)

    def __enter__(self):
        if self._h is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *exc):
        self._stop.set()
        if self._thread is not None:
            self._thread.join(timeout=2)

    def summary(self):
        return {"sm_mhz": statistics.median(self.samples) if self.samples else None,
                "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(self.samples)}


def _dist_env():
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    return rank, world, local


def _oracle_inputs(cfg, B_sample: int, seed: int):
    """Host copies of a B_sample-sequence batch of cfg's shape, in the oracle's input types."""
    import numpy as np
    from paper_2403_17031_b200.synthetic import make_batch
    batch = make_batch(cfg, "cpu", B=B_sample, seed=seed)

    def host(t):
        t = t.contiguous()
        return t.view(torch.int16).numpy().view(np.uint16) if t.dtype == torch.bfloat16 else t.numpy()
    return {k: host(v) for k, v in batch.items()}


def _oracle_chain_time(cfg, inp):
    """One pass of the whole path on the oracle; returns (seconds, real tokens)."""
    import numpy as np
    from oracle import ppo_oracle as O
    h = cfg.hyper
    V = cfg.V
    pl, rl, resp = inp["policy_logits"], inp["ref_logits"], inp["responses"]
    tau = np.float32(h.temperature)
    f32 = lambda a: np.asarray(a, np.float64).astype(np.float32)
    t0 = time.perf_counter()
    _, _, L, m, so = O.truncate_and_score(resp, h.eos_id, h.pad_id, inp["scores"], np.float32(h.no_eos_score))
    lp, _, _ = O.logprob_entropy(pl.reshape(-1, V), resp, tau, mask=m.reshape(-1))    # padding rows: not read, 0
    rlp, _, _ = O.logprob_entropy(rl.reshape(-1, V), resp, tau, mask=m.reshape(-1))
    lp, rlp = lp.reshape(resp.shape), rlp.reshape(resp.shape)
    _, rew = O.kl_rewards(f32(lp), f32(rlp), m, L, f32(so), np.float32(h.kl_coef))
    adv, ret = O.gae(f32(rew), inp["values"], L, np.float32(h.gamma), np.float32(h.lam))
    aw, _ = O.whiten(f32(adv), m, True, np.float32(h.whiten_eps))
    old = f32(lp) + inp["old_logprob_noise"]
    O.loss_fwd_bwd(pl, resp, m, old, f32(aw), inp["values_new"], inp["values"], f32(ret), tau,
                   np.float32(h.cliprange), np.float32(h.cliprange_value), np.float32(h.vf_coef), want_dlogits=True)
    return time.perf_counter() - t0, int(m.sum())


def _workload_name(cfg):
    return "config%d %s (B=%d, T=%d, V=%d, %s logits)" % (cfg.index, cfg.name, cfg.B, cfg.T, cfg.V, cfg.dtype)


def run_reference(args, cfg):
    """The reference arm: the fp64 CPU oracle, as it stands, on the host cores."""
    rank, world, _ = _dist_env()
    if rank != 0:
        return
    from oracle import ppo_oracle as O
    O.build()
    cores = O.num_threads()
    # size the per-step sample so that the whole run stays within a few minutes
    probe_s, _ = _oracle_chain_time(cfg, _oracle_inputs(cfg, 1, cfg.seed + 99))
    budget = args.ref_seconds / max(args.steps + args.warmup, 1)
    B_s = int(max(1, min(cfg.B, args.ref_sample, budget / max(probe_s, 1e-6))))
    inp = _oracle_inputs(cfg, B_s, cfg.seed + 100)
    for i in range(args.warmup):
        _oracle_chain_time(cfg, inp)
    total_s, total_tok = 0.0, 0
    for i in range(args.steps):
        s, tok = _oracle_chain_time(cfg, inp)
        total_s += s
        total_tok += tok
    value = total_tok / total_s
    sample = ("%d of %d sequences per step (%d response positions, %d of them real tokens, V=%d), oracle chain incl. "
              "dlogits" % (B_s, cfg.B, B_s * cfg.T, total_tok // max(args.steps, 1), cfg.V))
    line = {
        "impl": "reference", "metric": "response tokens/s", "value": value, "unit": "tokens/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total_s / max(args.steps, 1),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": _workload_name(cfg), "B": cfg.B, "T": cfg.T, "V": cfg.V,
                   "logits_dtype": cfg.dtype, "sample": sample,
                   "tokens": "real tokens (positions up to and including a response's first EOS) per second"},
        "cpu_baseline": {"value": value, "unit": "tokens/s", "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


class _Dist:
    """The process group of a multi-rank run (None-safe helpers for the single-rank run)."""

    def __init__(self, dev):
        self.rank, self.world, self.local = _dist_env()
        self.dev = dev
        self.on = self.world > 1
        if self.on:
            import torch.distributed as dist
            self.dist = dist
            if not dist.is_initialized():
                dist.init_process_group("nccl", device_id=dev)

    def barrier(self):
        if self.on:
            self.dist.barrier()

    def max_float(self, x: float) -> float:
        if not self.on:
            return x
        t = torch.tensor([x], dtype=torch.float64, device=self.dev)
        self.dist.all_reduce(t, op=self.dist.ReduceOp.MAX)
        return float(t.item())

    def close(self):
        if self.on:
            self.dist.destroy_process_group()


def _timed_blocks(run_step, K, est_ms_per_step, D, target_s, max_blocks=400):
    """Run R blocks of K steps between CUDA events (barrier + synchronize on both sides of the whole region);
    returns (list of block times in ms, total ms). R is chosen so that the region lasts about target_s."""
    R = int(min(max_blocks, max(1, math.ceil(target_s * 1e3 / max(K * est_ms_per_step, 1e-3)))))
    R = int(D.max_float(float(R)))
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(R + 1)]
    D.barrier()
    torch.cuda.synchronize()
    ev[0].record()
    for r in range(R):
        for _ in range(K):
            run_step()
        ev[r + 1].record()
    torch.cuda.synchronize()
    D.barrier()
    blocks = [ev[r].elapsed_time(ev[r + 1]) for r in range(R)]
    return blocks, ev[0].elapsed_time(ev[R])


def _back_to_back_ms(fn, n=20):
    """Average duration of one call of fn when n of them run back to back on the stream."""
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    fn()
    a.record()
    for _ in range(n):
        fn()
    b.record()
    torch.cuda.synchronize()
    return a.elapsed_time(b) / n


def measure_ppo(cfg, args, D, K, warmup, target_s, full: bool):
    """The whole path on stored logits (configs 1-3) at cfg's shape on this rank's GPU. full: also the end-to-end
    and the CPU-baseline legs. Returns the pieces of the JSON line."""
    from paper_2403_17031_b200 import binding
    from paper_2403_17031_b200.pipeline import PPOHotPath
    from paper_2403_17031_b200.synthetic import make_batch
    dev = D.dev
    h = cfg.hyper
    if args.whiten_rewards:   # optional reward whitening before GAE: one more token-level launch per step
        import dataclasses
        h = dataclasses.replace(h, whiten_rewards=1)
    launches_per_step = LAUNCHES_PER_STEP + (1 if args.whiten_rewards else 0)
    B, T, V = cfg.B, cfg.T, cfg.V
    batch = make_batch(cfg, dev, seed=cfg.seed + 1000 * D.rank, chunk_rows=4096)
    hp = PPOHotPath(B, T, V, cfg.torch_dtype, binding.params_from(h), device=dev)
    # stored rollout log-probs + noise: PPO ratios straddle the clip range (data, prepared untimed)
    o = hp.rollout_stats(batch["policy_logits"], batch["ref_logits"], batch["responses"], batch["scores"],
                         batch["values"])
    old_logprob = (o["logprob"] + batch["old_logprob_noise"]).contiguous()
    n_real = int(o["mask"].sum().item())
    torch.cuda.synchronize()
    esize = 2 if cfg.dtype == "bf16" else 4
    R_bytes = B * T * V * esize
    step_args = (batch["policy_logits"], batch["ref_logits"], batch["responses"], batch["scores"], batch["values"],
                 batch["values_new"])

    def step():
        hp.step(*step_args, old_logprob=old_logprob)

    for _ in range(max(warmup, 3)):
        step()
    torch.cuda.synchronize()
    # the step is recorded once into a CUDA graph and replayed; --eager launches it call by call instead
    graph = None
    if not args.eager:
        graph = hp.capture_step(*step_args, old_logprob=old_logprob)
    run_step = graph.replay if graph is not None else step
    t0 = torch.cuda.Event(enable_timing=True)
    t1 = torch.cuda.Event(enable_timing=True)
    t0.record()
    for _ in range(3):
        run_step()
    t1.record()
    torch.cuda.synchronize()
    est = t0.elapsed_time(t1) / 3

    with ClockSampler(D.local) as clk:
        blocks, total_ms = _timed_blocks(run_step, K, est, D, target_s)
        # ---- same workload, same clocks: the logits-bound kernels alone, 20 launches back to back each; the
        # dominant kernel first, right behind the timed region (the step's own loss launch has left the row order
        # in the workspace, so the later-epoch call is valid here)
        p = hp.params
        m = hp.out["mask"]
        loss_args = (batch["policy_logits"], batch["responses"], old_logprob, batch["values_new"], batch["values"])
        next_ms = _back_to_back_ms(lambda: hp.loss(*loss_args, next_epoch=True))    # later epoch: the kernel alone
        loss_ms = _back_to_back_ms(lambda: hp.loss(*loss_args))                     # first epoch: prologue + kernel
        lp_all_ms = _back_to_back_ms(lambda: binding.logprob_entropy(
            batch["policy_logits"], batch["responses"], p.temperature, workspace=hp.workspace,
            out=(o["logprob"], o["entropy"], None)))
        lp_real_ms = _back_to_back_ms(lambda: binding.logprob_entropy(
            batch["policy_logits"], batch["responses"], p.temperature, mask=m, workspace=hp.workspace,
            out=(o["logprob"], o["entropy"], None)))
    ms_per_step = D.max_float(statistics.median(blocks) / K)
    mean_ms = D.max_float(total_ms / (len(blocks) * K))
    status = hp.device_status()
    world = D.world
    # all ranks run the same shape; rank 0's count of real tokens stands for each (seeds differ, counts within 1%)
    tokens_real = n_real * world
    value = tokens_real / (ms_per_step * 1e-3)

    # ---- roofline of the dominant kernel (loss forward+backward): algorithmic bytes per launch =
    # V*s read per real token + V*s written per token (zeros on masked rows)
    peak, peak_kind = _peaks()
    loss_bytes = n_real * V * esize + B * T * V * esize
    loss_gbs = loss_bytes / (next_ms * 1e-3) / 1e9
    # the step reads the logits of the real rows only (policy, reference, loss) and writes every gradient row
    path_bytes = 2 * n_real * V * esize + loss_bytes
    traffic = _ncu_traffic("config%d" % cfg.index, n_real * V * esize, B * T * V * esize)
    roofline = {"bound": "hbm", "kernel": "row_engine_kernel (ppo_loss_fwd_bwd)", "achieved": loss_gbs,
                "peak": peak, "peak_kind": peak_kind, "unit": "GB/s", "frac": loss_gbs / peak,
                "frac_of_8tbs": loss_gbs / 8000.0, "traffic": traffic,
                "frac_on_traffic": None if traffic is None else traffic / (next_ms * 1e-3) / 1e9 / peak,
                "algorithmic_bytes": loss_bytes,
                "timing": "CUDA events around 20 back-to-back launches of the kernel (ppo_loss_fwd_bwd_next_epoch: a "
                          "later PPO epoch of the batch, which is exactly this launch), same workload, right after "
                          "the timed region and inside the same clock record"}
    config = {"workload": _workload_name(cfg), "B_per_gpu": B, "T": T, "V": V, "logits_dtype": cfg.dtype,
              "real_tokens": n_real, "response_positions": B * T,
              "tokens": "value counts real tokens (positions up to and including a response's first EOS); "
                        "response_positions_per_s counts all B*T positions, padding included",
              "response_positions_per_s": B * T * world / (ms_per_step * 1e-3),
              "blocks": len(blocks), "steps_timed": len(blocks) * K, "timed_region_ms": total_ms,
              "ms_per_step_mean": mean_ms,
              "ms_per_step_min_block": min(blocks) / K, "ms_per_step_max_block": max(blocks) / K,
              "l2": "inputs larger than L2 (%.0f MB of logits read on the %d real rows, 3 tensors, + %.0f MB "
                    "of gradient written per step; padding rows are not read)" %
                    (3 * n_real * V * esize / 1e6, n_real, R_bytes / 1e6),
              "path_hbm_gbs": path_bytes / (ms_per_step * 1e-3) / 1e9,
              "path_hbm_frac_of_8tbs": path_bytes / (ms_per_step * 1e-3) / 8e12,
              "logprob_entropy_ms": lp_all_ms, "logprob_entropy_gbs": R_bytes / (lp_all_ms * 1e-3) / 1e9,
              "logprob_entropy_frac_of_peak": R_bytes / (lp_all_ms * 1e-3) / 1e9 / peak,
              "logprob_entropy_frac_of_8tbs": R_bytes / (lp_all_ms * 1e-3) / 8e12,
              "logprob_entropy_real_rows_ms": lp_real_ms,
              "logprob_entropy_real_rows_gbs": n_real * V * esize / (lp_real_ms * 1e-3) / 1e9,
              "loss_fwd_bwd_ms": loss_ms, "loss_fwd_bwd_next_epoch_ms": next_ms,
              "launch": "cuda graph replay of ppo_step" if graph is not None else "eager ppo_step",
              "whiten_rewards": bool(args.whiten_rewards), "device_status": status}
    res = {"value": value, "ms_per_step": ms_per_step, "config": config, "roofline": roofline, "clocks": clk.summary(),
           "gpu_launches": launches_per_step * K * len(blocks), "e2e": None, "cpu_baseline": None,
           "cpu_baseline_1thread": None}
    del graph

    # ---- end to end: inputs start in pinned host memory, results are read back to the host
    if full and not args.no_e2e:
        names = ["policy_logits", "ref_logits", "responses", "scores", "values", "values_new"]
        host = {k: batch[k].cpu().pin_memory() for k in names}
        host["old_logprob"] = old_logprob.cpu().pin_memory()
        devbuf = {k: (batch[k] if k in batch else old_logprob) for k in host}      # staging = the resident tensors
        res_names = ["losses", "dvalues", "advantages_whitened", "returns", "logprob", "ref_logprob"]
        host_res = {k: torch.empty_like(hp.out[k], device="cpu").pin_memory() for k in res_names}
        # the call copies, of the two logits tensors, the real rows only (padding rows are never read)
        h2d = sum(v.numel() * v.element_size() for k, v in host.items() if not k.endswith("logits"))
        h2d += 2 * n_real * V * esize
        d2h = sum(v.numel() * v.element_size() for v in host_res.values())
        host_io = binding.PPOStepIO.from_tensors({**host, **host_res}, cuda=False)
        dev_io = hp.step_io(devbuf)

        def e2e_step():
            # one C-ABI call: host->device copies, the whole path, device->host copies, stream sync
            binding.step_host(host_io, dev_io, cfg.torch_dtype, B, T, V, hp.params)
        Ke = max(3, min(K, args.e2e_steps))
        for _ in range(2):
            e2e_step()
        torch.cuda.synchronize()
        D.barrier()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(Ke):
            e2e_step()
        b.record()
        torch.cuda.synchronize()
        e_ms = D.max_float(a.elapsed_time(b))
        res["e2e"] = {"value": tokens_real / (e_ms / Ke * 1e-3), "unit": "tokens/s", "h2d_bytes_per_step": h2d,
                      "d2h_bytes_per_step": d2h, "steps": Ke, "ms_per_step": e_ms / Ke,
                      "call": "ppo_step_host (pinned host buffers in; losses and the [B,T] results out; the "
                              "gradient on the logits, %.0f MB, is left on the device for the backward pass "
                              "that consumes it)" % (R_bytes / 1e6)}
        del host, devbuf, host_res

    # ---- CPU baseline: the oracle on a bounded sample, rank 0, N = 1 only; all cores, then one thread
    if full and D.rank == 0 and world == 1 and not args.no_cpu_baseline:
        from oracle import ppo_oracle as O
        O.build()
        cores = O.num_threads()

        def timed(seconds, threads):
            O.set_num_threads(threads)
            try:
                per_seq, _ = _oracle_chain_time(cfg, _oracle_inputs(cfg, 1, cfg.seed + 300))   # size probe
                B_s = int(max(1, min(cfg.B, 0.5 * seconds / max(per_seq, 1e-6))))
                inp = _oracle_inputs(cfg, B_s, cfg.seed + 301)
                tot_s, tot_tok, passes = 0.0, 0, 0
                while tot_s < seconds and passes < 64:
                    s_, tok_ = _oracle_chain_time(cfg, inp)
                    tot_s += s_
                    tot_tok += tok_
                    passes += 1
            finally:
                O.set_num_threads(cores)
            return {"value": tot_tok / tot_s, "unit": "tokens/s", "cores": threads, "kind": "oracle",
                    "sample": "%d of %d sequences (%d positions, V=%d) x %d passes, whole chain incl. dlogits, %.1f s; "
                              "real tokens per second" % (B_s, cfg.B, B_s * cfg.T, V, passes, tot_s)}
        res["cpu_baseline"] = timed(args.cpu_seconds, cores)
        res["cpu_baseline_1thread"] = timed(min(args.cpu_seconds, 8.0), 1)
    del hp, batch
    torch.cuda.empty_cache()
    return res


def _lmhead_oracle_baseline(cfg, b, seconds=10.0):
    """The oracle's fused-LM-head rows (fp64 dot products) on a few rows: rows per second on all host cores."""
    import numpy as np
    from oracle import ppo_oracle as O
    O.build()
    to_np = lambda t: t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)
    H, W = to_np(b["H"]), to_np(b["W"])
    tok = b["responses"].reshape(-1).cpu().numpy()
    def timed(n):
        sel = np.arange(0, H.shape[0], max(1, H.shape[0] // n))[:n].astype(np.int64)
        t0 = time.perf_counter()
        O.lmhead_logprob_entropy(H, W, tok, np.float32(cfg.hyper.temperature), sel_rows=sel)
        return sel, time.perf_counter() - t0
    sel, dt = timed(max(O.num_threads(), 8))                       # size probe
    n = int(min(H.shape[0], max(len(sel), len(sel) * seconds / max(dt, 1e-3))))
    sel, dt = timed(n)
    # one step of the config needs two such passes per real row (policy and reference unembedding)
    return {"value": len(sel) / dt / 2.0, "unit": "tokens/s", "cores": O.num_threads(), "kind": "oracle",
            "sample": "%d rows of H x W [%d, %d] in fp64 for one unembedding, %.1f s; halved for the two unembeddings of a "
                      "step; the [B,T] steps are not included (they are < 0.1%% of this)" % (len(sel), W.shape[0], W.shape[1], dt)}


def measure_lmhead(cfg, args, D, K, warmup, target_s, full: bool):
    """Config 4: fused LM head (policy and reference) + token-level steps + loss at log-prob level."""
    from paper_2403_17031_b200 import binding
    from paper_2403_17031_b200.synthetic import make_lmhead_batch
    dev = D.dev
    h = cfg.hyper
    p = binding.params_from(h)
    b = make_lmhead_batch(cfg, dev, M=args.lm_rows, seed=cfg.seed + 1000 * D.rank)
    M, Kd = b["H"].shape
    V = b["W"].shape[1]
    B, T = b["responses"].shape
    f32 = torch.float32
    ws = binding.new_workspace(max(binding.lmhead_workspace_bytes(M, Kd, V), binding.workspace_bytes(B, T, V)), dev)
    bt = lambda dt=f32: torch.empty((B, T), dtype=dt, device=dev)
    o = {"ro": bt(torch.int32), "ei": torch.empty(B, dtype=torch.int32, device=dev),
         "sl": torch.empty(B, dtype=torch.int32, device=dev), "mask": bt(torch.uint8),
         "so": torch.empty(B, dtype=f32, device=dev), "lp": bt(), "ent": bt(), "lse": bt(), "rlp": bt(), "rent": bt(),
         "kl": bt(), "rew": bt(), "adv": bt(), "ret": bt(), "aw": bt(), "st": torch.empty(3, dtype=f32, device=dev)}
    loss_out = {"losses": torch.empty(8, dtype=f32, device=dev), "dlogprob": bt(), "dvalues": bt()}
    tok = b["responses"].reshape(-1)
    bwd_out = None
    if args.lm_backward:   # the step after the loss: gradient on the log-probs back to H and W
        bwd_out = {"dlogits": torch.empty((M, V), dtype=torch.bfloat16, device=dev),
                   "dH": torch.empty_like(b["H"]), "dW": torch.empty_like(b["W"])}

    def backward():
        binding.lmhead_bwd(b["H"], b["W"], tok, o["lse"].view(-1), loss_out["dlogprob"].view(-1), p.temperature, ws,
                           mask=o["mask"].view(-1), out=bwd_out)

    def lm_policy():
        binding.lmhead_logprob_entropy(b["H"], b["W"], tok, p.temperature, ws, mask=o["mask"].view(-1),
                                       out=(o["lp"].view(-1), o["ent"].view(-1), o["lse"].view(-1)))

    def step(old):
        binding.truncate_and_score(b["responses"], b["scores"], p.eos_id, p.pad_id, p.no_eos_score,
                                   out=(o["ro"], o["ei"], o["sl"], o["mask"], o["so"]))
        # (with the mask of the EOS trick: padding rows are taken out of the GEMM and get 0)
        lm_policy()
        binding.lmhead_logprob_entropy(b["H"], b["W_ref"], tok, p.temperature, ws, mask=o["mask"].view(-1),
                                       out=(o["rlp"].view(-1), o["rent"].view(-1), None))
        binding.kl_rewards(o["lp"], o["rlp"], o["mask"], o["sl"], o["so"], p.kl_coef, out=(o["kl"], o["rew"]))
        binding.gae(o["rew"], b["values"], o["sl"], p.gamma, p.lam, out=(o["adv"], o["ret"]))
        binding.whiten(o["adv"], o["mask"], True, p.whiten_eps, workspace=ws, out=o["aw"], stats=o["st"])
        binding.loss_from_logprob(o["lp"], o["ent"], o["mask"], o["lp"] if old is None else old, o["aw"],
                                  b["values_new"], b["values"], o["ret"], p, ws, out=loss_out)
        if bwd_out is not None:
            backward()
    step(None)
    old = (o["lp"] + b["old_logprob_noise"]).contiguous()
    for _ in range(max(warmup, 3)):
        step(old)
    torch.cuda.synchronize()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record()
    step(old)
    t1.record()
    torch.cuda.synchronize()
    est = t0.elapsed_time(t1)
    with ClockSampler(D.local) as clk:
        blocks, total_ms = _timed_blocks(lambda: step(old), K, est, D, target_s)
        lm_ms = _back_to_back_ms(lm_policy, n=10)
        bwd_ms = _back_to_back_ms(backward, n=5) if bwd_out is not None else None
        if bwd_out is None and full:
            # the step after the loss (gradient on the log-probs back to dlogits, dH, dW), timed on its own
            bwd_out = {"dlogits": torch.empty((M, V), dtype=torch.bfloat16, device=dev),
                       "dH": torch.empty_like(b["H"]), "dW": torch.empty_like(b["W"])}
            bwd_ms = _back_to_back_ms(backward, n=3)
            bwd_out = None
    ms_per_step = D.max_float(statistics.median(blocks) / K)
    status = binding.last_device_status(ws)
    n_real = int(o["mask"].sum().item())
    flops = 2.0 * n_real * Kd * V      # the forward call multiplies the real rows only
    tf = flops / (lm_ms * 1e-3) / 1e12
    # the kernel runs back to back for the whole timed region: compare with the sustained figure
    peak, kind = _peaks("bf16_tflops_sustained", 1400.0)
    burst, _ = _peaks("bf16_tflops", 1590.0)
    world = D.world
    res = {"value": n_real * world / (ms_per_step * 1e-3), "ms_per_step": ms_per_step,
           "config": {"workload": "config4 %s (M=%d, K=%d, V=%d, bf16)" % (cfg.name, M, Kd, V), "M_per_gpu": M, "K": Kd,
                      "V": V, "l2": "inputs larger than L2 (H %.0f MB + 2 x W %.0f MB per step)" %
                      (M * Kd * 2 / 1e6, Kd * V * 2 / 1e6),
                      "blocks": len(blocks), "steps_timed": len(blocks) * K, "timed_region_ms": total_ms,
                      "lmhead_ms": lm_ms, "lmhead_bwd_ms": bwd_ms, "real_tokens": n_real, "response_positions": M,
                      "response_positions_per_s": M * world / (ms_per_step * 1e-3),
                      "lmhead_bwd_tflops": None if bwd_ms is None else 3.0 * flops / (bwd_ms * 1e-3) / 1e12,
                      "device_status": status},
           "roofline": {"bound": "tensor", "kernel": "lmhead_kernel (ppo_lmhead_logprob_entropy)", "achieved": tf,
                        "peak": peak, "peak_kind": kind + " (sustained)", "unit": "TFLOP/s", "frac": tf / peak,
                        "frac_of_burst": tf / burst, "traffic": None,
                        "timing": "CUDA events around 10 back-to-back C-ABI calls (row order, packing of the real rows, "
                                  "GEMM kernel, finalize kernel); flops = 2 x real rows x K x V"},
           "clocks": clk.summary(), "e2e": None, "cpu_baseline": None, "cpu_baseline_1thread": None,
           "gpu_launches": (13 + (6 if bwd_out is not None else 0)) * K * len(blocks)}
    if full and not args.no_e2e:
        # end to end through ppo_lmhead_step_host: H (its real rows), both unembeddings, tokens, scores and values
        # start in pinned host memory and are copied in every step; the loss scalars and the [B,T] results come back
        names = ["H", "W", "W_ref", "responses", "scores", "values", "values_new"]
        host = {k: b[k].cpu().pin_memory() for k in names}
        host["old_logprob"] = old.cpu().pin_memory()
        dev_out = {"responses_out": o["ro"], "eos_index": o["ei"], "seq_len": o["sl"], "mask": o["mask"], "scores_out": o["so"],
                   "logprob": o["lp"], "entropy": o["ent"], "lse": o["lse"], "ref_logprob": o["rlp"], "kl": o["kl"],
                   "rewards": o["rew"], "advantages": o["adv"], "returns": o["ret"], "advantages_whitened": o["aw"],
                   "whiten_stats": o["st"], "losses": loss_out["losses"], "dlogprob": loss_out["dlogprob"],
                   "dvalues": loss_out["dvalues"]}
        res_names = ["losses", "dlogprob", "dvalues", "advantages_whitened", "returns", "logprob", "ref_logprob"]
        host_res = {k: torch.empty_like(dev_out[k], device="cpu").pin_memory() for k in res_names}
        h2d = sum(v.numel() * v.element_size() for k, v in host.items() if k != "H") + n_real * Kd * 2
        d2h = sum(v.numel() * v.element_size() for v in host_res.values())
        host_io = binding.LMHeadStepIO.from_tensors({**host, **host_res}, cuda=False)
        dev_io = binding.LMHeadStepIO.from_tensors({**{k: b[k] for k in names}, "old_logprob": old, **dev_out,
                                                    "workspace": ws}, cuda=True)

        def e2e_step():
            binding.lmhead_step_host(host_io, dev_io, B, T, Kd, V, p)
        Ke = max(3, min(K, args.e2e_steps))
        e2e_step()
        D.barrier()
        a, c = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(Ke):
            e2e_step()
        c.record()
        torch.cuda.synchronize()
        e_ms = D.max_float(a.elapsed_time(c))
        res["e2e"] = {"value": n_real * world / (e_ms / Ke * 1e-3), "unit": "tokens/s", "h2d_bytes_per_step": h2d,
                      "d2h_bytes_per_step": d2h, "steps": Ke, "ms_per_step": e_ms / Ke,
                      "call": "ppo_lmhead_step_host (pinned host buffers in: the real rows of H, both unembeddings, the "
                              "[B,T] inputs; losses and the [B,T] results out)"}
    if full and D.rank == 0 and world == 1 and not args.no_cpu_baseline:
        res["cpu_baseline"] = _lmhead_oracle_baseline(cfg, b)
    del b, ws
    torch.cuda.empty_cache()
    return res


def _summary_of(res):
    """The short form of a measurement that goes into config.others."""
    keep = ("achieved", "peak", "unit", "frac", "frac_of_8tbs", "frac_of_burst", "kernel", "traffic")
    c = res["config"]
    out = {"workload": c["workload"], "ms_per_step": res["ms_per_step"], "tokens_per_s": res["value"],
           "real_tokens": c.get("real_tokens"), "response_positions": c.get("response_positions"),
           "blocks": c.get("blocks"), "steps_timed": c.get("steps_timed"), "timed_region_ms": c.get("timed_region_ms"),
           "roofline": {k: res["roofline"].get(k) for k in keep if k in res["roofline"]},
           "clocks": res["clocks"], "device_status": c.get("device_status")}
    for k in ("path_hbm_frac_of_8tbs", "logprob_entropy_ms", "logprob_entropy_frac_of_8tbs", "loss_fwd_bwd_next_epoch_ms",
              "lmhead_ms", "lmhead_bwd_ms", "lmhead_bwd_tflops"):
        if k in c:
            out[k] = c[k]
    return out


def _extra_dpo(args, D, K, target_s):
    """The DPO step on preference pairs (the paper's (B, 638) layout, 8 pairs per GPU), short form for config.others."""
    from paper_2403_17031_b200 import binding
    from paper_2403_17031_b200.pipeline import DPOStep
    from paper_2403_17031_b200.synthetic import PREF_CONFIGS, make_pref_batch
    cfg = PREF_CONFIGS["dpo"]
    b = make_pref_batch(cfg, D.dev, seed=cfg.seed + 1000 * D.rank)
    P, T, V = cfg.P, cfg.T, cfg.V
    st = DPOStep(P, T, V, cfg.torch_dtype, cfg.beta, device=D.dev)
    run = lambda: st.step(b["policy_logits"], b["ref_logits"], b["tokens"], b["mask"])
    for _ in range(3):
        run()
    torch.cuda.synchronize()
    n_real, rows, es = int(b["mask"].sum().item()), 2 * P * T, 2 if cfg.dtype == "bf16" else 4
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record(); run(); t1.record(); torch.cuda.synchronize()
    with ClockSampler(D.local) as clk:
        blocks, total_ms = _timed_blocks(run, K, t0.elapsed_time(t1), D, target_s)
        bwd_ms = _back_to_back_ms(lambda: binding.logprob_bwd(b["policy_logits"], b["tokens"], b["mask"], st.out["dlogprob"],
                                                              1.0, st.workspace, dlogits=st.out["dlogits"]))
    ms = D.max_float(statistics.median(blocks) / K)
    peak, _ = _peaks("hbm_gbs", 6650.0)
    bwd_bytes = (n_real + rows) * V * es
    gbs = bwd_bytes / (bwd_ms * 1e-3) / 1e9
    return {"workload": "config5 %s (DPO step, %d pairs x (2, %d) positions, V=%d, %s)" % (cfg.name, P, T, V, cfg.dtype),
            "ms_per_step": ms, "tokens_per_s": n_real * D.world / (ms * 1e-3), "real_tokens": n_real,
            "response_positions": rows, "blocks": len(blocks), "steps_timed": len(blocks) * K, "timed_region_ms": total_ms,
            "roofline": {"kernel": "row_engine_kernel (ppo_logprob_bwd)", "achieved": gbs, "peak": peak, "unit": "GB/s",
                         "frac": gbs / peak, "frac_of_8tbs": gbs / 8000.0, "algorithmic_bytes": bwd_bytes},
            "clocks": clk.summary(), "device_status": st.device_status()}


def _extra_sample(args, D, K, target_s):
    """Temperature sampling fused with the log-prob pass on config-1 logits, short form for config.others."""
    from paper_2403_17031_b200 import binding
    from paper_2403_17031_b200.synthetic import CONFIGS, make_batch
    cfg = CONFIGS[1]
    x = make_batch(cfg, D.dev, seed=cfg.seed + 1000 * D.rank, with_ref=False)["policy_logits"]
    B, T, V = x.shape
    ws = binding.new_workspace(binding.workspace_bytes(B, T, V), D.dev)
    out = binding.sample_logprob_entropy(x, cfg.hyper.temperature, 20240317, 0, workspace=ws)
    ctr = [0]

    def run():
        ctr[0] += 1
        binding.sample_logprob_entropy(x, cfg.hyper.temperature, 20240317, ctr[0], workspace=ws, out=out)
    for _ in range(3):
        run()
    torch.cuda.synchronize()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record(); run(); t1.record(); torch.cuda.synchronize()
    with ClockSampler(D.local) as clk:
        blocks, total_ms = _timed_blocks(run, K, t0.elapsed_time(t1), D, target_s)
    ms = D.max_float(statistics.median(blocks) / K)
    peak, _ = _peaks("hbm_gbs", 6650.0)
    gbs = B * T * V * 2 / (ms * 1e-3) / 1e9
    return {"workload": "config6 fused sampling + log-prob on config1 logits (%d rows x %d, bf16)" % (B * T, V),
            "ms_per_step": ms, "tokens_per_s": B * T * D.world / (ms * 1e-3), "response_positions": B * T,
            "blocks": len(blocks), "steps_timed": len(blocks) * K, "timed_region_ms": total_ms,
            "roofline": {"kernel": "sample_kernel (ppo_sample_logprob_entropy)", "achieved": gbs, "peak": peak, "unit": "GB/s",
                         "frac": gbs / peak, "frac_of_8tbs": gbs / 8000.0, "algorithmic_bytes": B * T * V * 2},
            "clocks": clk.summary(), "device_status": binding.last_device_status(ws)}


def run_ours(args, cfgs):
    """Headline workload (args.config) in full, then the other PPO configs in short form under config.others."""
    rank, world, local = _dist_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    if local >= torch.cuda.device_count():
        raise SystemExit("rank %d has no GPU: %d visible, %d ranks" % (rank, torch.cuda.device_count(), world))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    D = _Dist(dev)
    from paper_2403_17031_b200 import binding, build
    if rank == 0:
        build.build()
    D.barrier()
    binding.lib()
    K, W = args.steps, max(args.warmup, 3)
    measure = lambda c, full, k, tgt: (measure_lmhead if c.index == 4 else measure_ppo)(c, args, D, k, W, tgt, full)
    head_cfg = cfgs[args.config]
    head = measure(head_cfg, True, K, args.target_seconds)
    others = []
    if not args.no_others:
        for idx in (1, 2, 3, 4):
            if idx == args.config:
                continue
            c = cfgs[idx]
            free, _ = torch.cuda.mem_get_info()
            need = (3.3 * c.B * c.T * c.V * (2 if c.dtype == "bf16" else 4)) if idx != 4 else 8e9
            ok = torch.tensor([1.0 if free > need else 0.0], device=dev)
            if D.on:
                D.dist.all_reduce(ok, op=D.dist.ReduceOp.MIN)
            if float(ok.item()) < 1.0:
                others.append({"workload": _workload_name(c), "skipped": "needs %.0f GB of free device memory, %.0f GB free"
                               % (need / 1e9, free / 1e9)})
                continue
            # bounded: at most K steps per block and a shorter timed region than the headline's
            # (the fused-LM-head config also gets its end-to-end and oracle legs here: it has no line of its own)
            res = measure(c, idx == 4, min(K, 20), min(0.3, args.target_seconds))
            summary = _summary_of(res)
            if idx == 4:
                summary["e2e"], summary["cpu_baseline"] = res["e2e"], res["cpu_baseline"]
            others.append(summary)
        # the widened workloads, so that they too are measured by whoever runs the default command
        others.append(_extra_dpo(args, D, min(K, 20), min(0.2, args.target_seconds)))
        torch.cuda.empty_cache()
        others.append(_extra_sample(args, D, min(K, 20), min(0.2, args.target_seconds)))
        torch.cuda.empty_cache()
    if rank == 0:
        line = {
            "metric": "response tokens/s", "value": head["value"], "unit": "tokens/s", "n_gpus": world, "steps": K,
            "warmup": W, "ms_per_step": head["ms_per_step"], "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16" if head_cfg.index == 4 else "f32", "data": "synthetic",
            "config": head["config"], "roofline": head["roofline"], "clocks": head["clocks"], "e2e": head["e2e"],
            "cpu_baseline": head["cpu_baseline"], "cpu_baseline_1thread": head["cpu_baseline_1thread"],
            "gpu_launches": head["gpu_launches"],
        }
        line["config"]["others"] = others
        print(json.dumps(line), flush=True)
    D.close()


def run_dpo(args):
    """Config 5: one DPO step on a batch of preference pairs in the paper's (B, 638) layout: token log-probs of
    policy and reference on the response rows, DPO loss + implicit rewards, gradient back to the policy's logits."""
    rank, world, local = _dist_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    distributed = world > 1
    if distributed:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    from paper_2403_17031_b200 import binding, build
    from paper_2403_17031_b200.pipeline import DPOStep
    from paper_2403_17031_b200.synthetic import PREF_CONFIGS, make_pref_batch
    if rank == 0:
        build.build()
    if distributed:
        dist.barrier()
    binding.lib()
    cfg = PREF_CONFIGS["dpo"]
    b = make_pref_batch(cfg, dev, seed=cfg.seed + 1000 * rank)
    P, T, V = cfg.P, cfg.T, cfg.V
    st = DPOStep(P, T, V, cfg.torch_dtype, cfg.beta, device=dev)
    run = lambda: st.step(b["policy_logits"], b["ref_logits"], b["tokens"], b["mask"])
    for _ in range(max(args.warmup, 3)):
        run()
    torch.cuda.synchronize()
    K = args.steps
    n_real = int(b["mask"].sum().item())
    rows = 2 * P * T
    es = 2 if cfg.dtype == "bf16" else 4
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    if distributed:
        dist.barrier()
    torch.cuda.synchronize()
    with ClockSampler(local) as clk:
        ev0.record()
        for _ in range(K):
            run()
        ev1.record()
        torch.cuda.synchronize()
        # the dominant call alone, same workload, right after the timed region
        bw = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(20)]
        for e0, e1 in bw:
            e0.record()
            binding.logprob_bwd(b["policy_logits"], b["tokens"], b["mask"], st.out["dlogprob"], 1.0, st.workspace,
                                dlogits=st.out["dlogits"])
            e1.record()
        torch.cuda.synchronize()
    total_ms = ev0.elapsed_time(ev1)
    if distributed:
        t = torch.tensor([total_ms], dtype=torch.float64, device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        total_ms = float(t.item())
    ms_per_step = total_ms / K
    bwd_ms = statistics.mean(a.elapsed_time(c) for a, c in bw)
    bwd_bytes = (n_real + rows) * V * es
    bwd_gbs = bwd_bytes / (bwd_ms * 1e-3) / 1e9
    path_bytes = (3 * n_real + rows) * V * es     # two log-prob passes + backward read, backward write of all rows
    peak, kind = _peaks("hbm_gbs", 6650.0)
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        import numpy as np
        from oracle import ppo_oracle as O, pref_oracle as R
        O.build()
        m = b["mask"].cpu().numpy()
        idx = np.flatnonzero(m.reshape(-1))
        tok = b["tokens"].cpu().numpy().reshape(-1)
        pl = b["policy_logits"].reshape(-1, V)[torch.from_numpy(idx).to(dev)].cpu()
        rl = b["ref_logits"].reshape(-1, V)[torch.from_numpy(idx).to(dev)].cpu()
        to_np = lambda t: t.view(torch.int16).numpy().view(np.uint16) if t.dtype == torch.bfloat16 else t.numpy()
        t0 = time.perf_counter()
        lp = np.zeros(rows)
        rlp = np.zeros(rows)
        lp[idx] = O.logprob_entropy(to_np(pl), tok[idx], 1.0)[0]
        rlp[idx] = O.logprob_entropy(to_np(rl), tok[idx], 1.0)[0]
        lp, rlp = lp.reshape(2, P, T), rlp.reshape(2, P, T)
        d = R.dpo_loss(lp[0], lp[1], rlp[0], rlp[1], m[0], m[1], cfg.beta)
        g = np.stack([d["dlp_c"], d["dlp_r"]]).reshape(-1)[idx]
        R.logprob_bwd(pl.double().numpy(), tok[idx], g, 1.0)
        dt_s = time.perf_counter() - t0
        cpu = {"value": n_real / dt_s, "unit": "tokens/s", "cores": O.num_threads(), "kind": "oracle",
               "sample": "the whole batch once: %d response rows of V=%d (log-probs x2 in C/OpenMP, loss and "
                         "backward in numpy), %.1f s" % (n_real, V, dt_s)}
    if rank == 0:
        line = {
            "metric": "response tokens/s", "value": n_real * world / (ms_per_step * 1e-3), "unit": "tokens/s",
            "n_gpus": world, "steps": K, "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": "config5 %s (DPO step)" % cfg.name, "pairs_per_gpu": P, "T": T, "V": V,
                       "logits_dtype": cfg.dtype, "response_tokens": n_real, "rows": rows,
                       "l2": "inputs larger than L2 (%.0f MB of logits read, %.0f MB of gradient written per step)" %
                             (3 * n_real * V * es / 1e6, rows * V * es / 1e6),
                       "path_hbm_gbs": path_bytes / (ms_per_step * 1e-3) / 1e9, "logprob_bwd_ms": bwd_ms,
                       "launch": "eager: ppo_logprob_entropy_pair, ppo_dpo_loss, ppo_logprob_bwd (4 kernel launches)",
                       "device_status": st.device_status()},
            "roofline": {"bound": "hbm", "kernel": "row_engine_kernel (ppo_logprob_bwd)", "achieved": bwd_gbs,
                         "peak": peak, "peak_kind": kind, "unit": "GB/s", "frac": bwd_gbs / peak,
                         "frac_of_8tbs": bwd_gbs / 8000.0, "traffic": _ncu_traffic("config5", n_real * V * es, rows * V * es),
                         "algorithmic_bytes": bwd_bytes,
                         "timing": "CUDA events around the ppo_logprob_bwd call (prologue + row engine launches), "
                                   "right after the timed region"},
            "clocks": clk.summary(), "e2e": None, "cpu_baseline": cpu, "gpu_launches": 4 * K,
        }
        print(json.dumps(line), flush=True)
    if distributed:
        dist.destroy_process_group()


def run_sample(args):
    """Config 6: temperature sampling fused with the log-prob / entropy pass on the config-1 logits."""
    rank, world, local = _dist_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    distributed = world > 1
    if distributed:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    from paper_2403_17031_b200 import binding, build
    from paper_2403_17031_b200.synthetic import CONFIGS, make_batch
    if rank == 0:
        build.build()
    if distributed:
        dist.barrier()
    binding.lib()
    cfg = CONFIGS[1]
    x = make_batch(cfg, dev, seed=cfg.seed + 1000 * rank, with_ref=False)["policy_logits"]
    B, T, V = x.shape
    ws = binding.new_workspace(binding.workspace_bytes(B, T, V), dev)
    out = binding.sample_logprob_entropy(x, cfg.hyper.temperature, 20240317, 0, workspace=ws)
    for i in range(max(args.warmup, 3)):
        binding.sample_logprob_entropy(x, cfg.hyper.temperature, 20240317, i + 1, workspace=ws, out=out)
    torch.cuda.synchronize()
    K = args.steps
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    if distributed:
        dist.barrier()
    torch.cuda.synchronize()
    with ClockSampler(local) as clk:
        ev0.record()
        for i in range(K):
            binding.sample_logprob_entropy(x, cfg.hyper.temperature, 20240317, 100 + i, workspace=ws, out=out)
        ev1.record()
        torch.cuda.synchronize()
    total_ms = ev0.elapsed_time(ev1)
    if distributed:
        t = torch.tensor([total_ms], dtype=torch.float64, device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        total_ms = float(t.item())
    ms = total_ms / K
    logits = B * T * V
    # one read of the logits: HBM bound like the plain log-prob pass (the generator runs for 256 classes and the
    # members of one class per row)
    clocks = clk.summary()
    peak, peak_kind = _peaks("hbm_gbs", 6650.0)
    achieved = logits * 2 / (ms * 1e-3) / 1e9
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        from oracle import sample_oracle as S
        n = 48
        xs = x.reshape(-1, V)[:n].double().cpu().numpy()
        t0 = time.perf_counter()
        S.sample(xs, cfg.hyper.temperature, 20240317, 0)
        dt_s = time.perf_counter() - t0
        cpu = {"value": n / dt_s, "unit": "tokens/s", "cores": 1, "kind": "oracle",
               "sample": "%d rows of V=%d (numpy Philox + two-level race, draw only), %.1f s" % (n, V, dt_s)}
    if rank == 0:
        line = {
            "metric": "response tokens/s", "value": B * T * world / (ms * 1e-3), "unit": "tokens/s", "n_gpus": world,
            "steps": K, "warmup": max(args.warmup, 3), "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": "config6 fused sampling + log-prob on config1 logits", "B_per_gpu": B, "T": T, "V": V,
                       "logits_dtype": cfg.dtype, "l2": "inputs larger than L2 (%.0f MB of logits per step)" %
                       (logits * 2 / 1e6), "hbm_gbs": logits * 2 / (ms * 1e-3) / 1e9,
                       "device_status": binding.last_device_status(ws)},
            "roofline": {"bound": "hbm", "kernel": "sample_kernel (ppo_sample_logprob_entropy)", "achieved": achieved,
                         "peak": peak, "peak_kind": peak_kind, "unit": "GB/s", "frac": achieved / peak,
                         "frac_of_8tbs": achieved / 8000.0, "traffic": None, "algorithmic_bytes": logits * 2},
            "clocks": clocks, "e2e": None, "cpu_baseline": cpu, "gpu_launches": K,
        }
        print(json.dumps(line), flush=True)
    if distributed:
        dist.destroy_process_group()


def run_plumbing(args):
    """The multi-rank launch and the reduction of the timing, without any kernel: every rank joins the process group
    (NCCL on GPUs, gloo on a machine without one), times a short sleep, the maximum over ranks is taken and rank 0
    prints one JSON line with the number of ranks that took part."""
    rank, world, local = _dist_env()
    import torch.distributed as dist
    use_cuda = torch.cuda.is_available() and torch.cuda.device_count() >= world
    if world > 1:
        if use_cuda:
            torch.cuda.set_device(local)
            dist.init_process_group("nccl", device_id=torch.device("cuda", local))
        else:
            dist.init_process_group("gloo")
    dev = torch.device("cuda", local) if use_cuda else torch.device("cpu")
    from paper_2403_17031_b200.synthetic import CONFIGS, shard_batch
    mine = shard_batch(CONFIGS[2].B, rank, world)          # the sequences this rank would own of the paper's batch of 512
    if world > 1:
        dist.barrier()
    t0 = time.perf_counter()
    time.sleep(0.01 * (1 + rank))
    ms = (time.perf_counter() - t0) * 1e3
    t = torch.tensor([ms, float(len(mine)), 1.0], dtype=torch.float64, device=dev)
    mx = t.clone()
    if world > 1:
        dist.all_reduce(mx, op=dist.ReduceOp.MAX)
        dist.all_reduce(t, op=dist.ReduceOp.SUM)
        dist.barrier()
    if rank == 0:
        print(json.dumps({"impl": "plumbing", "n_gpus": world, "ranks_seen": int(t[2].item()),
                          "sequences_owned_total": int(t[1].item()), "max_ms": float(mx[0].item()),
                          "backend": "nccl" if use_cuda else "gloo", "scaling": "weak"}), flush=True)
    if world > 1:
        dist.destroy_process_group()


def _free_port() -> int:
    with socket.socket(socket.AF_INET, socket.SOCK_STREAM) as sk:
        sk.bind(("127.0.0.1", 0))
        return sk.getsockname()[1]


def _spawn_ranks(n: int):
    """--gpus N without a launcher: become `torch.distributed.run` with one rank per GPU on this node."""
    env = dict(os.environ)
    env.setdefault("NCCL_DEBUG", "INFO")            # the communicator's own record of its ranks reaches stderr
    env.setdefault("NCCL_DEBUG_SUBSYS", "INIT")
    env.setdefault("OMP_NUM_THREADS", "1")
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", str(n),
           "--master-addr", "127.0.0.1", "--master-port", str(_free_port()), os.path.abspath(__file__), *sys.argv[1:]]
    sys.stdout.flush()
    os.execve(sys.executable, cmd, env)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--config", type=int, default=2, choices=[1, 2, 3, 4, 5, 6],
                    help="1-3: PPO path on stored logits (2 = the full PPO batch, the headline); 4: fused LM head; "
                         "5: DPO step on preference pairs; 6: fused sampling + log-prob")
    ap.add_argument("--batch", type=int, default=None, help="configs 1-3: sequences per GPU instead of the config's B "
                    "(for profiler captures on a cut of the batch)")
    ap.add_argument("--no-others", action="store_true", help="only the headline workload, no config.others")
    ap.add_argument("--target-seconds", type=float, default=TIMED_REGION_TARGET_S,
                    help="the K-step block is repeated until the timed region is about this long (0: one block)")
    ap.add_argument("--lm-rows", type=int, default=None, help="config 4: rows of H (default 512*53)")
    ap.add_argument("--lm-backward", action="store_true",
                    help="config 4: the step also runs the LM-head backward (dlogits, dH, dW)")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference", "plumbing"])
    ap.add_argument("--eager", action="store_true", help="launch every step call by call instead of replaying a CUDA graph")
    ap.add_argument("--whiten-rewards", action="store_true",
                    help="detail '(Optional) Reward whitening': whiten the rewards (mean kept) before GAE")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--e2e-steps", type=int, default=10)
    ap.add_argument("--cpu-seconds", type=float, default=15.0)
    ap.add_argument("--ref-sample", type=int, default=16, help="max sequences per step of the reference arm")
    ap.add_argument("--ref-seconds", type=float, default=150.0, help="time budget of the reference arm")
    args = ap.parse_args()
    if args.gpus < 1:
        raise SystemExit("--gpus must be >= 1")
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and args.impl != "reference":
        _spawn_ranks(args.gpus)
    _, world, _ = _dist_env()
    if args.impl != "reference" and world != args.gpus:
        raise SystemExit("--gpus %d but the launcher started %d ranks" % (args.gpus, world))
    import dataclasses
    from paper_2403_17031_b200.synthetic import CONFIGS
    cfgs = dict(CONFIGS)
    if args.batch is not None and args.config in (1, 2, 3):
        cfgs[args.config] = dataclasses.replace(cfgs[args.config], B=args.batch)
    if args.impl == "plumbing":
        run_plumbing(args)
    elif args.impl == "reference":
        # (configs 4-6 have no whole-chain oracle of their own shape here: the reference arm times config 2's chain)
        run_reference(args, cfgs[args.config] if args.config in (1, 2, 3) else cfgs[2])
    elif args.config == 5:
        run_dpo(args)
    elif args.config == 6:
        run_sample(args)
    else:
        run_ours(args, cfgs)


if __name__ == "__main__":
    main()
