#!/usr/bin/env python
"""Benchmark of the per-token PPO hot path (arXiv 2403.17031) on B200.

One "step" = one pass of the whole path over one synthetic batch: EOS trick, log-prob/entropy of
policy and reference logits, KL rewards, GAE, advantage whitening, clipped losses + gradients
(9 kernel launches). Prints ONE JSON line (rank 0).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--config 1|2|3] [--impl ours|reference]

N > 1: launch with torch.distributed.run (one rank per GPU, NCCL); every rank runs the same
per-GPU batch shape on its own seeded batch (weak scaling, no data-path collective); the time is
the max over ranks of the device-timed region.

--impl reference times the fp64 CPU oracle (the only "reference" this work has) on the host
cores, on a bounded sample of the same workload per step.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import torch  # noqa: E402

# DRAM bytes (read + write) of one launch of the dominant kernel, from the committed ncu capture of the same
# configuration (profiles/loss_fwd_bwd_row_engine_config1.md, profiles/dpo_step_config5.md); None where no capture
# of the current kernel exists.
NCU_TRAFFIC_BYTES = {1: 160.007e6 + 283.877e6, 5: 109.9e6 + 965.3e6}
LAUNCHES_PER_STEP = 3   # ppo_step: logprob pair (policy + reference), rollout (token-level steps + loss prologue), row_engine (loss)


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
    """One pass of the whole path on the oracle; returns (seconds, tokens)."""
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
    return time.perf_counter() - t0, resp.size


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
    sample = "%d of %d sequences per step (%d tokens, V=%d), oracle chain incl. dlogits" % (B_s, cfg.B, B_s * cfg.T, cfg.V)
    line = {
        "impl": "reference", "metric": "response tokens/s", "value": value, "unit": "tokens/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total_s / max(args.steps, 1),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": "config%d %s" % (cfg.index, cfg.name), "B": cfg.B, "T": cfg.T, "V": cfg.V,
                   "logits_dtype": cfg.dtype, "sample": sample},
        "cpu_baseline": {"value": value, "unit": "tokens/s", "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def run_ours(args, cfg):
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
    from paper_2403_17031_b200.pipeline import PPOHotPath
    from paper_2403_17031_b200.synthetic import make_batch
    if rank == 0:
        build.build()
    if distributed:
        dist.barrier()
    binding.lib()

    h = cfg.hyper
    if args.whiten_rewards:   # optional reward whitening before GAE: one more token-level launch per step
        import dataclasses
        h = dataclasses.replace(h, whiten_rewards=1)
    launches_per_step = LAUNCHES_PER_STEP + (1 if args.whiten_rewards else 0)
    B, T, V = cfg.B, cfg.T, cfg.V
    batch = make_batch(cfg, dev, seed=cfg.seed + 1000 * rank)
    hp = PPOHotPath(B, T, V, cfg.torch_dtype, binding.params_from(h), device=dev)
    # stored rollout log-probs + noise: PPO ratios straddle the clip range (data, prepared untimed)
    o = hp.rollout_stats(batch["policy_logits"], batch["ref_logits"], batch["responses"], batch["scores"],
                         batch["values"])
    old_logprob = (o["logprob"] + batch["old_logprob_noise"]).contiguous()
    n_real = int(o["mask"].sum().item())
    torch.cuda.synchronize()
    esize = 2 if cfg.dtype == "bf16" else 4
    R = B * T * V * esize

    def step():
        hp.step(batch["policy_logits"], batch["ref_logits"], batch["responses"], batch["scores"], batch["values"],
                batch["values_new"], old_logprob=old_logprob)

    for _ in range(max(args.warmup, 3)):
        step()
    torch.cuda.synchronize()

    # ---- timed region: K steps of the whole path (ppo_step: 3 launches per step), device-timed.
    # Default: the step is recorded once into a CUDA graph and replayed K times; --eager launches it
    # call by call instead.
    K = args.steps
    graph = None
    if not args.eager:
        graph = hp.capture_step(batch["policy_logits"], batch["ref_logits"], batch["responses"], batch["scores"],
                                batch["values"], batch["values_new"], old_logprob=old_logprob)
        for _ in range(3):
            graph.replay()
    run_step = graph.replay if graph is not None else step
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    if distributed:
        dist.barrier()
    torch.cuda.synchronize()
    with ClockSampler(local) as clk:
        ev0.record()
        for i in range(K):
            run_step()
        ev1.record()
        torch.cuda.synchronize()
        # ---- same workload, same clocks: the six entry points called one by one with CUDA events around
        # the two logits-bound calls (durations of the dominant kernels for the roofline)
        Kk = min(K, 200)
        loss_ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(Kk)]
        lp_ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(Kk)]
        next_ev = [torch.cuda.Event(enable_timing=True) for _ in range(Kk)]
        for i in range(Kk):
            o = hp.out
            p = hp.params
            binding.truncate_and_score(batch["responses"], batch["scores"], p.eos_id, p.pad_id, p.no_eos_score,
                                       out=(o["responses_out"], o["eos_index"], o["seq_len"], o["mask"], o["scores_out"]))
            lp_ev[i][0].record()
            binding.logprob_entropy(batch["policy_logits"], batch["responses"], p.temperature, workspace=hp.workspace,
                                    out=(o["logprob"], o["entropy"], None))
            lp_ev[i][1].record()
            binding.logprob_entropy(batch["ref_logits"], batch["responses"], p.temperature, workspace=hp.workspace,
                                    out=(o["ref_logprob"], None, None))
            binding.kl_rewards(o["logprob"], o["ref_logprob"], o["mask"], o["seq_len"], o["scores_out"], p.kl_coef,
                               out=(o["kl"], o["rewards"]))
            binding.gae(o["rewards"], batch["values"], o["seq_len"], p.gamma, p.lam, out=(o["advantages"], o["returns"]))
            binding.whiten(o["advantages"], o["mask"], True, p.whiten_eps, workspace=hp.workspace,
                           out=o["advantages_whitened"], stats=o["whiten_stats"])
            loss_ev[i][0].record()
            hp.loss(batch["policy_logits"], batch["responses"], old_logprob, batch["values_new"], batch["values"])
            loss_ev[i][1].record()
            # a later PPO epoch of the same batch: the same kernel, launched alone (row order reused)
            hp.loss(batch["policy_logits"], batch["responses"], old_logprob, batch["values_new"], batch["values"],
                    next_epoch=True)
            next_ev[i].record()
        torch.cuda.synchronize()
    total_ms = ev0.elapsed_time(ev1)
    if distributed:
        t = torch.tensor([total_ms], dtype=torch.float64, device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        total_ms = float(t.item())
        dist.barrier()
    ms_per_step = total_ms / K
    tokens_per_step = B * T * world
    value = tokens_per_step / (ms_per_step * 1e-3)
    loss_ms = statistics.mean(a.elapsed_time(b) for a, b in loss_ev)
    next_ms = statistics.mean(ab[1].elapsed_time(c) for ab, c in zip(loss_ev, next_ev))
    lp_ms = statistics.mean(a.elapsed_time(b) for a, b in lp_ev)
    status = hp.device_status()

    # ---- roofline of the dominant kernel (loss forward+backward): algorithmic bytes per launch =
    # V*s read per real token + V*s written per token (zeros on masked rows)
    peak, peak_kind = _peaks()
    loss_bytes = n_real * V * esize + B * T * V * esize
    loss_gbs = loss_bytes / (next_ms * 1e-3) / 1e9
    lp_gbs = R / (lp_ms * 1e-3) / 1e9
    # the step reads the logits of the real rows only (policy, reference, loss) and writes every gradient row
    path_bytes = 2 * n_real * V * esize + loss_bytes

    # ---- end to end: inputs start in pinned host memory, results are read back to the host
    e2e = None
    if not args.no_e2e:
        names = ["policy_logits", "ref_logits", "responses", "scores", "values", "values_new"]
        host = {k: batch[k].cpu().pin_memory() for k in names}
        host["old_logprob"] = old_logprob.cpu().pin_memory()
        devbuf = {k: torch.empty_like(v, device=dev) for k, v in host.items()}
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
        if distributed:
            dist.barrier()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(Ke):
            e2e_step()
        b.record()
        torch.cuda.synchronize()
        e_ms = a.elapsed_time(b)
        if distributed:
            t = torch.tensor([e_ms], dtype=torch.float64, device=dev)
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
            e_ms = float(t.item())
        e2e = {"value": tokens_per_step / (e_ms / Ke * 1e-3), "unit": "tokens/s", "h2d_bytes_per_step": h2d,
               "d2h_bytes_per_step": d2h, "steps": Ke, "call": "ppo_step_host (pinned host buffers)"}
        del host, devbuf

    # ---- CPU baseline: the oracle on a bounded sample, rank 0, N = 1 only
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        from oracle import ppo_oracle as O
        O.build()
        per_seq, _ = _oracle_chain_time(cfg, _oracle_inputs(cfg, 1, cfg.seed + 300))   # size probe
        B_s = int(max(1, min(cfg.B, args.cpu_seconds / max(per_seq, 1e-6))))
        inp = _oracle_inputs(cfg, B_s, cfg.seed + 301)
        # repeat the sample until about cpu_seconds of oracle work have been timed (at most the whole batch per pass)
        tot_s, tot_tok, passes = 0.0, 0, 0
        while tot_s < args.cpu_seconds and passes < 64:
            s_, tok_ = _oracle_chain_time(cfg, inp)
            tot_s += s_
            tot_tok += tok_
            passes += 1
        cpu = {"value": tot_tok / tot_s, "unit": "tokens/s", "cores": O.num_threads(), "kind": "oracle",
               "sample": "%d of %d sequences (%d tokens, V=%d) x %d passes, whole chain incl. dlogits, %.1f s" %
                         (B_s, cfg.B, B_s * cfg.T, V, passes, tot_s)}

    if rank == 0:
        line = {
            "metric": "response tokens/s", "value": value, "unit": "tokens/s", "n_gpus": world, "steps": K,
            "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": "config%d %s" % (cfg.index, cfg.name), "B_per_gpu": B, "T": T, "V": V,
                       "logits_dtype": cfg.dtype, "real_tokens": n_real,
                       # `value` counts all B*T response positions of the batch (padding after the first EOS
                       # included, as the workload is stated); this one counts the positions before it only
                       "real_tokens_per_s": n_real * world / (ms_per_step * 1e-3),
                       "l2": "inputs larger than L2 (%.0f MB of logits read on the %d real rows, 3 tensors, + %.0f MB "
                             "of gradient written per step; padding rows are not read)" %
                             (3 * n_real * V * esize / 1e6, n_real, R / 1e6),
                       "path_hbm_gbs": path_bytes / (ms_per_step * 1e-3) / 1e9,
                       "path_hbm_frac_of_8tbs": path_bytes / (ms_per_step * 1e-3) / 8e12,
                       "logprob_entropy_ms": lp_ms, "logprob_entropy_gbs": lp_gbs,
                       "logprob_entropy_frac_of_peak": lp_gbs / peak, "loss_fwd_bwd_ms": loss_ms,
                       "loss_fwd_bwd_next_epoch_ms": next_ms,
                       "launch": "cuda graph replay of ppo_step" if graph is not None else "eager ppo_step",
                       "whiten_rewards": bool(args.whiten_rewards),
                       "device_status": status},
            "roofline": {"bound": "hbm", "kernel": "row_engine_kernel (ppo_loss_fwd_bwd)", "achieved": loss_gbs,
                         "peak": peak, "peak_kind": peak_kind, "unit": "GB/s", "frac": loss_gbs / peak,
                         "frac_of_8tbs": loss_gbs / 8000.0, "traffic": NCU_TRAFFIC_BYTES.get(cfg.index),
                         "algorithmic_bytes": loss_bytes,
                         "timing": "CUDA events around one launch of the kernel (ppo_loss_fwd_bwd_next_epoch: a later "
                                   "PPO epoch of the batch, no prologue launch), in a second pass over the same workload "
                                   "right after the timed region; config.loss_fwd_bwd_ms is the first-epoch call "
                                   "(prologue + kernel)"},
            "clocks": clk.summary(),
            "e2e": e2e,
            "cpu_baseline": cpu,
            "gpu_launches": launches_per_step * K,
        }
        print(json.dumps(line), flush=True)
    if distributed:
        dist.destroy_process_group()


def run_lmhead(args, cfg):
    """Config 4: fused LM head (policy and reference) + token-level steps + loss at log-prob level."""
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
    from paper_2403_17031_b200.synthetic import make_lmhead_batch
    if rank == 0:
        build.build()
    if distributed:
        dist.barrier()
    binding.lib()
    h = cfg.hyper
    p = binding.params_from(h)
    b = make_lmhead_batch(cfg, dev, M=args.lm_rows, seed=cfg.seed + 1000 * rank)
    M, K = b["H"].shape
    V = b["W"].shape[1]
    B, T = b["responses"].shape
    f32 = torch.float32
    ws = binding.new_workspace(max(binding.lmhead_workspace_bytes(M, K, V), binding.workspace_bytes(B, T, V)), dev)
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

    def step(old):
        binding.truncate_and_score(b["responses"], b["scores"], p.eos_id, p.pad_id, p.no_eos_score,
                                   out=(o["ro"], o["ei"], o["sl"], o["mask"], o["so"]))
        # (with the mask of the EOS trick: padding rows are taken out of the GEMM and get 0)
        binding.lmhead_logprob_entropy(b["H"], b["W"], tok, p.temperature, ws, mask=o["mask"].view(-1),
                                       out=(o["lp"].view(-1), o["ent"].view(-1), o["lse"].view(-1)))
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
    for _ in range(max(args.warmup, 3)):
        step(old)
    torch.cuda.synchronize()
    K_steps = args.steps
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    lm_ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(K_steps)]
    bw_ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(K_steps)]
    if distributed:
        dist.barrier()
    torch.cuda.synchronize()
    with ClockSampler(local) as clk:
        ev0.record()
        for i in range(K_steps):
            binding.truncate_and_score(b["responses"], b["scores"], p.eos_id, p.pad_id, p.no_eos_score,
                                       out=(o["ro"], o["ei"], o["sl"], o["mask"], o["so"]))
            lm_ev[i][0].record()
            binding.lmhead_logprob_entropy(b["H"], b["W"], tok, p.temperature, ws, mask=o["mask"].view(-1),
                                           out=(o["lp"].view(-1), o["ent"].view(-1), o["lse"].view(-1)))
            lm_ev[i][1].record()
            binding.lmhead_logprob_entropy(b["H"], b["W_ref"], tok, p.temperature, ws, mask=o["mask"].view(-1),
                                           out=(o["rlp"].view(-1), o["rent"].view(-1), None))
            binding.kl_rewards(o["lp"], o["rlp"], o["mask"], o["sl"], o["so"], p.kl_coef, out=(o["kl"], o["rew"]))
            binding.gae(o["rew"], b["values"], o["sl"], p.gamma, p.lam, out=(o["adv"], o["ret"]))
            binding.whiten(o["adv"], o["mask"], True, p.whiten_eps, workspace=ws, out=o["aw"], stats=o["st"])
            binding.loss_from_logprob(o["lp"], o["ent"], o["mask"], old, o["aw"], b["values_new"], b["values"],
                                      o["ret"], p, ws, out=loss_out)
            if bwd_out is not None:
                bw_ev[i][0].record()
                backward()
                bw_ev[i][1].record()
        ev1.record()
        torch.cuda.synchronize()
    total_ms = ev0.elapsed_time(ev1)
    if distributed:
        t = torch.tensor([total_ms], dtype=torch.float64, device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        total_ms = float(t.item())
    ms_per_step = total_ms / K_steps
    lm_ms = statistics.mean(a.elapsed_time(c) for a, c in lm_ev)
    status = binding.last_device_status(ws)
    bwd_ms = statistics.mean(a.elapsed_time(c) for a, c in bw_ev) if bwd_out is not None else None
    n_real = int(o["mask"].sum().item())
    flops = 2.0 * n_real * K * V      # the forward call multiplies the real rows only
    tf = flops / (lm_ms * 1e-3) / 1e12
    # the kernel runs back to back for the whole timed region: compare with the sustained figure
    peak, kind = _peaks("bf16_tflops_sustained", 1400.0)
    burst, _ = _peaks("bf16_tflops", 1590.0)
    if rank == 0:
        line = {
            "metric": "response tokens/s", "value": M * world / (ms_per_step * 1e-3), "unit": "tokens/s",
            "n_gpus": world, "steps": K_steps, "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": "config4 %s" % cfg.name, "M_per_gpu": M, "K": K, "V": V,
                       "l2": "inputs larger than L2 (H %.0f MB + 2 x W %.0f MB per step)" %
                             (M * K * 2 / 1e6, K * V * 2 / 1e6),
                       "lmhead_ms": lm_ms, "lmhead_bwd_ms": bwd_ms,
                       "real_tokens": n_real,
                       "lmhead_bwd_tflops": None if bwd_ms is None else 3.0 * flops / (bwd_ms * 1e-3) / 1e12,
                       "device_status": status},
            "roofline": {"bound": "tensor", "kernel": "lmhead_kernel (ppo_lmhead_logprob_entropy)", "achieved": tf,
                         "peak": peak, "peak_kind": kind + " (sustained)", "unit": "TFLOP/s", "frac": tf / peak,
                         "frac_of_burst": tf / burst, "traffic": None,
                         "timing": "CUDA events around the C-ABI call (row order, packing of the real rows, GEMM kernel, "
                                   "finalize kernel); flops = 2 x real rows x K x V"},
            "clocks": clk.summary(), "e2e": None, "cpu_baseline": None,
            "gpu_launches": (13 + (6 if bwd_out is not None else 0)) * K_steps,
        }
        print(json.dumps(line), flush=True)
    if distributed:
        dist.destroy_process_group()


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
                         "frac_of_8tbs": bwd_gbs / 8000.0, "traffic": NCU_TRAFFIC_BYTES.get(5),
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
    # instructions the method needs per logit: Philox4x32-10 10, uniform 2, log2 1, widen 1,
    # scale 1, exp2 1, two sums 2, race 3
    ops_per_logit = 21
    clocks = clk.summary()
    sm_ghz = (clocks.get("sm_max_mhz") or 1965) / 1e3
    peak = 148 * 4 * 32 * sm_ghz          # Ginstr/s: one warp instruction per scheduler and clock
    achieved = ops_per_logit * logits / (ms * 1e-3) / 1e9
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        from oracle import sample_oracle as S
        n = 48
        xs = x.reshape(-1, V)[:n].double().cpu().numpy()
        t0 = time.perf_counter()
        S.sample(xs, cfg.hyper.temperature, 20240317, 0)
        dt_s = time.perf_counter() - t0
        cpu = {"value": n / dt_s, "unit": "tokens/s", "cores": 1, "kind": "oracle",
               "sample": "%d rows of V=%d (numpy Philox + Gumbel-max, draw only), %.1f s" % (n, V, dt_s)}
    if rank == 0:
        line = {
            "metric": "response tokens/s", "value": B * T * world / (ms * 1e-3), "unit": "tokens/s", "n_gpus": world,
            "steps": K, "warmup": max(args.warmup, 3), "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": "config6 fused sampling + log-prob on config1 logits", "B_per_gpu": B, "T": T, "V": V,
                       "logits_dtype": cfg.dtype, "l2": "inputs larger than L2 (%.0f MB of logits per step)" %
                       (logits * 2 / 1e6), "hbm_gbs": logits * 2 / (ms * 1e-3) / 1e9,
                       "device_status": binding.last_device_status(ws)},
            "roofline": {"bound": "alu", "kernel": "sample_kernel (ppo_sample_logprob_entropy)", "achieved": achieved,
                         "peak": peak, "peak_kind": "derived: 148 SMs x 4 schedulers x 32 lanes x max SM clock",
                         "unit": "Ginstr/s", "frac": achieved / peak, "traffic": None,
                         "ops_per_logit": ops_per_logit},
            "clocks": clocks, "e2e": None, "cpu_baseline": cpu, "gpu_launches": K,
        }
        print(json.dumps(line), flush=True)
    if distributed:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--config", type=int, default=1, choices=[1, 2, 3, 4, 5, 6],
                    help="1-3: PPO path on stored logits; 4: fused LM head; 5: DPO step on preference pairs; "
                         "6: fused sampling + log-prob")
    ap.add_argument("--lm-rows", type=int, default=None, help="config 4: rows of H (default 512*53)")
    ap.add_argument("--lm-backward", action="store_true",
                    help="config 4: the step also runs the LM-head backward (dlogits, dH, dW)")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
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
    from paper_2403_17031_b200.synthetic import CONFIGS
    if args.config == 5 and args.impl != "reference":
        run_dpo(args)
        return
    if args.config == 6 and args.impl != "reference":
        run_sample(args)
        return
    cfg = CONFIGS[1 if args.config in (5, 6) else args.config]
    if args.impl == "reference":
        run_reference(args, CONFIGS[1] if args.config == 4 else cfg)
    elif args.config == 4:
        run_lmhead(args, cfg)
    else:
        run_ours(args, cfg)


if __name__ == "__main__":
    main()
