"""The multi-GPU plumbing on CPU: two gloo ranks, no GPU.

Replicas share nothing but the measurement: a barrier and the maximum of the per-rank times.
"""
import json
import os
import socket
import subprocess
import sys

import torch
import torch.multiprocessing as mp

from paper_2506_15969_b200 import replicas, traces

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank: int, world: int, port: int, out_dir: str):
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    assert replicas.rank_env() == (rank, rank, world)
    dist = replicas.init("gloo")
    assert dist is not None and dist.get_world_size() == world
    replicas.barrier(dist)
    ms = 10.0 + 5.0 * rank                                   # rank 1 is the slow replica
    ms_max = replicas.max_over_ranks(ms, dist)
    cfg = traces.tiny_config()
    gen = traces.TraceGen(cfg, replicas.replica_seed(7, rank), device="cpu", units=[0])
    q, _, _ = gen.steps(1)
    gathered = [torch.zeros_like(q, dtype=torch.float32) for _ in range(world)]
    dist.all_gather(gathered, q.float())                     # test-only exchange: the traces must differ
    replicas.barrier(dist)
    with open(os.path.join(out_dir, f"rank{rank}.json"), "w") as f:
        json.dump({"ms_max": ms_max, "value": replicas.job_tokens_per_second(32, 8, world, ms_max),
                   "same_trace": bool(torch.equal(gathered[0], gathered[1]))}, f)
    dist.destroy_process_group()


def test_two_ranks_agree_on_the_slowest_time_and_the_job_throughput(tmp_path):
    port = _free_port()
    mp.spawn(_worker, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    res = [json.load(open(tmp_path / f"rank{r}.json")) for r in range(2)]
    for r in res:
        assert r["ms_max"] == 15.0                           # max over ranks, on every rank
        assert r["value"] == 2 * 32 * 8 / 15e-3              # both replicas' tokens over the slowest time
        assert not r["same_trace"]                           # each replica has its own data


def test_single_process_needs_no_group():
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "LOCAL_RANK", "WORLD_SIZE")}
    code = ("from paper_2506_15969_b200 import replicas as r; assert r.rank_env() == (0, 0, 1); "
            "assert r.init('gloo') is None; r.barrier(None); assert r.max_over_ranks(3.5, None) == 3.5; print('ok')")
    out = subprocess.run([sys.executable, "-c", code], cwd=ROOT, env=env, capture_output=True, text=True, timeout=120)
    assert out.returncode == 0 and out.stdout.strip() == "ok", out.stderr


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", LOCAL_RANK="1", WORLD_SIZE="2")
    out = subprocess.run([sys.executable, "bench.py", "--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup", "0"],
                         cwd=ROOT, env=env, capture_output=True, text=True, timeout=120)
    assert out.returncode == 0 and out.stdout.strip() == ""
