"""Step latency against generated length for three cache policies on the same kernels.

    python -m paper_2506_15969_b200.latency_table [--config 4] [--positions 2048,4096,...] [--batch B]

Reproduces the SHAPE of the paper's latency table (Appendix "Efficiency analysis": per-step
latency at 2 K .. 16 K generated tokens for FullKV, LazyEviction and per-step eviction), for
the attention / tracking / eviction path only, on synthetic traces:

* fullkv   -- budget above the whole sequence: nothing is ever evicted, the cache grows;
* lazy     -- the configuration's budget and window W (lagged eviction every W steps);
* perstep  -- the same budget with W = 1: an eviction decision at every step.

Each cell starts from a prompt of min(position, budget) tokens (position for fullkv) and
times one observation window of decode steps with CUDA events, evictions included.
Prints one JSON line per cell and a markdown table.
"""
from __future__ import annotations

import argparse
import dataclasses
import json


def measure(cfg, steps: int, seed: int = 0):
    import torch
    from . import binding, traces
    gen = traces.TraceGen(cfg, seed, device="cuda")
    eng = binding.Engine(cfg.layers, cfg.q_heads, cfg.kv_heads, cfg.head_dim, cfg.budget, cfg.window,
                         cfg.threshold, batch=cfg.batch, n_recent=cfg.n_recent, n_initial=cfg.n_initial,
                         max_prefill=cfg.prefill)
    shape = (cfg.layers, cfg.batch, cfg.kv_heads, cfg.prefill, cfg.head_dim)
    k, v = gen.prefill()
    eng.prefill(k.view(shape), v.view(shape))
    del k, v
    out = torch.empty(cfg.layers, cfg.batch, cfg.q_heads, cfg.head_dim, dtype=torch.bfloat16, device="cuda")
    stream = torch.cuda.current_stream()
    ms, done = 0.0, 0
    for phase, count in (("warm", 4), ("timed", steps)):
        left = count
        while left > 0:
            c = min(traces.TraceGen.CHUNK, left)
            q, kn, vn = gen.steps(c)
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            for s in range(c):
                eng.decode_step(q[s], kn[s], vn[s], out)
            e1.record(stream)
            torch.cuda.synchronize()
            if phase == "timed":
                ms += e0.elapsed_time(e1)
                done += c
            left -= c
    eng.synchronize()
    inf = eng.info()
    eng.close()
    return ms / done, inf


def main():
    from . import traces
    ap = argparse.ArgumentParser()
    ap.add_argument("--config", type=int, default=4)
    ap.add_argument("--positions", default="2048,4096,8192,12288,16384")
    ap.add_argument("--batch", type=int, default=0)
    ap.add_argument("--modes", default="fullkv,lazy,perstep")
    args = ap.parse_args()
    base = traces.CONFIGS[args.config]
    if args.batch:
        base = dataclasses.replace(base, batch=args.batch)
    positions = [int(x) for x in args.positions.split(",")]
    rows = {}
    for mode in args.modes.split(","):
        for pos in positions:
            steps = base.window
            if mode == "fullkv":
                cfg = dataclasses.replace(base, prefill=pos, budget=pos + 2 * base.window + 8, name=f"{base.name}-fullkv")
            elif mode == "lazy":
                cfg = dataclasses.replace(base, prefill=min(pos, base.budget), name=f"{base.name}-lazy")
            elif mode == "perstep":
                cfg = dataclasses.replace(base, prefill=min(pos, base.budget), window=1, n_recent=1,
                                          alpha=base.threshold, name=f"{base.name}-perstep")
            else:
                raise SystemExit(f"unknown mode {mode}")
            ms, inf = measure(cfg, steps)
            rows[(mode, pos)] = ms
            print(json.dumps({"mode": mode, "position": pos, "ms_per_step": round(ms, 4), "tokens_per_s": round(cfg.batch / ms * 1e3, 1),
                              "cached_tokens_at_end": inf.n, "evictions": inf.evictions, "units": inf.units,
                              "decode_launch": {"splits": inf.splits, "stages": inf.stages, "groups": inf.groups}}), flush=True)
    print("\n| policy | " + " | ".join(f"{p} tokens" for p in positions) + " |")
    print("|---|" + "---|" * len(positions))
    for mode in args.modes.split(","):
        print(f"| {mode} | " + " | ".join(f"{rows[(mode, p)]:.3f} ms" for p in positions) + " |")


if __name__ == "__main__":
    main()
