"""Multi-process CPU tests (gloo, world_size 2) of the data-parallel layer: the path shards by
sequence with no data-path collective; only timing is reduced across ranks."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2403_17031_b200.synthetic import CONFIGS, make_batch, shard_batch


def test_shard_batch_partitions_every_sequence_once():
    for B in (1, 7, 64, 512):
        for W in (1, 2, 3, 8):
            seen = []
            for r in range(W):
                seen += list(shard_batch(B, r, W))
            assert seen == list(range(B))
            sizes = [len(shard_batch(B, r, W)) for r in range(W)]
            assert max(sizes) - min(sizes) <= 1
    with pytest.raises(ValueError):
        shard_batch(8, 2, 2)


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        from oracle import ppo_oracle as O
        cfg = CONFIGS[0]
        batch = make_batch(cfg, "cpu", B=6)          # same seed on every rank: the global batch
        mine = shard_batch(6, rank, world)
        sl = slice(mine.start, mine.stop)
        h = cfg.hyper
        V = cfg.V
        resp = batch["responses"][sl].numpy()
        lp, ent, _ = O.logprob_entropy(batch["policy_logits"][sl].reshape(-1, V).numpy(), resp, np.float32(h.temperature))
        _, _, L, m, so = O.truncate_and_score(resp, h.eos_id, h.pad_id, batch["scores"][sl].numpy(), h.no_eos_score)
        # per-rank timing reduced with MAX, as bench.py does
        t = torch.tensor([1.0 + rank], dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        units = torch.tensor([float(len(mine) * cfg.T)], dtype=torch.float64)
        dist.all_reduce(units, op=dist.ReduceOp.SUM)
        q.put((rank, mine.start, mine.stop, lp.tolist(), L.tolist(), float(t), float(units)))
    finally:
        dist.destroy_process_group()


def test_two_rank_sharded_rows_equal_unsharded(oracle):
    world = 2
    port = _free_port()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    cfg = CONFIGS[0]
    batch = make_batch(cfg, "cpu", B=6)
    h = cfg.hyper
    lp_full, _, _ = oracle.logprob_entropy(batch["policy_logits"].reshape(-1, cfg.V).numpy(),
                                           batch["responses"].numpy(), np.float32(h.temperature))
    _, _, L_full, _, _ = oracle.truncate_and_score(batch["responses"].numpy(), h.eos_id, h.pad_id,
                                                   batch["scores"].numpy(), h.no_eos_score)
    lp_cat, L_cat = [], []
    for rank, lo, hi, lp, L, tmax, units in got:
        lp_cat += lp
        L_cat += L
        assert tmax == 2.0 and units == 6 * cfg.T
    assert lp_cat == lp_full.tolist() and L_cat == L_full.tolist()


def test_bench_starts_its_own_ranks_and_prints_one_line():
    """`bench.py --gpus 2` without a launcher starts two ranks itself; the plumbing arm runs the launch, the process
    group and the reduction of the timing without any kernel (gloo here), and rank 0 alone prints the JSON line."""
    import json
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    env["CUDA_VISIBLE_DEVICES"] = ""
    out = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--gpus", "2", "--impl", "plumbing"],
                         capture_output=True, text=True, timeout=240, env=env)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [ln for ln in out.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1, out.stdout
    d = json.loads(lines[0])
    assert d["n_gpus"] == 2 and d["ranks_seen"] == 2 and d["sequences_owned_total"] == 512
    assert d["max_ms"] >= 19.0          # the slower rank's time (rank 1 sleeps 20 ms), not rank 0's
    # a rank count that contradicts the launcher is refused
    env2 = dict(env, RANK="0", WORLD_SIZE="1", LOCAL_RANK="0")
    bad = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--gpus", "2", "--impl", "plumbing"],
                         capture_output=True, text=True, timeout=120, env=env2)
    assert bad.returncode != 0 and "ranks" in bad.stderr
