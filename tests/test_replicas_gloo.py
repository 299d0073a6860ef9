"""The multi-GPU mode is replicas only; its cross-rank bookkeeping runs here on two gloo ranks on CPU."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_2607_26475_b200 import replicas
    ms_local = 40.0 + 5.0 * rank            # rank 1 is the slower replica
    tokens_local = 8 * 16                   # batch 8, 16 steps on every replica (weak scaling)
    dist.barrier()
    ms, n = replicas.aggregate(ms_local, tokens_local)
    tps = replicas.throughput(ms_local, tokens_local)
    out[rank] = (ms, n, tps)
    dist.barrier()
    dist.destroy_process_group()


def test_two_replicas_report_the_slowest_time_and_the_total_tokens():
    world, port = 2, _free_port()
    with mp.get_context("spawn").Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert res[0] == res[1]
    ms, n, tps = res[0]
    assert ms == 45.0 and n == 256
    assert abs(tps - 256 / 0.045) < 1e-6


def test_single_process_needs_no_process_group():
    from paper_2607_26475_b200 import replicas
    assert replicas.aggregate(12.5, 64) == (12.5, 64)
    assert replicas.host_budget_per_rank(100 << 30, 8) == int((100 << 30) * 0.6 / 8)


def test_bench_starts_its_own_ranks_when_no_launcher_did():
    """`python bench.py --gpus 2` without torchrun: the script launches two ranks itself; with the CPU stub they
    rendezvous over gloo, and rank 0 prints one line for the whole job (slowest rank's time, all ranks' tokens)."""
    import json
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    r = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--gpus", "2", "--cpu-stub", "--steps", "3",
                        "--warmup", "1"], capture_output=True, text=True, env=env, timeout=300)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["n_gpus"] == 2 and d["steps"] == 3 and len(d["per_rank"]["tok_s"]) == 2
    assert abs(d["ms_per_step"] - 11.0) < 1e-9                       # the slower rank sets the time
    assert abs(d["value"] - 2 * 8 * 3 / 0.033) < 1e-6                # tokens of both replicas
    assert d["per_rank"]["tok_s"][0] > d["per_rank"]["tok_s"][1]


def test_per_rank_values_without_a_process_group():
    from paper_2607_26475_b200 import replicas
    assert replicas.gather_per_rank(3.5) == [3.5]
