"""Time of the prompt pass with tracking (lazyev_prefill_observed), tiled kernel against replay.

    python -m paper_2506_15969_b200.prompt_table [--cases 5:512,4:256,5:2048:4] [--no-replay]

A case is `config:prompt_length[:layers]`: the benchmark configuration's heads and batch, a prompt of
that length and (optionally) fewer layers, so that long prompts fit in memory.  For each case the
prompt is loaded with tracking once per implementation -- the tiled tensor-core kernel (one launch)
and the replay through the decode kernel (one launch per prompt row) -- and timed with CUDA events,
after one untimed pass of each.  Flops are the algorithmic ones of causal attention,
4 * G * D * P (P + 1) / 2 per unit (Q K^T and P V once each); the tiled kernel executes Q K^T twice
and P V as two bf16 products.  Prints one JSON line per case and a markdown table.
"""
from __future__ import annotations

import argparse
import dataclasses
import json


def time_case(cfg, mode: int, repeats: int = 2):
    import torch
    from . import binding
    P = cfg.prefill
    eng = binding.Engine(cfg.layers, cfg.q_heads, cfg.kv_heads, cfg.head_dim, cfg.budget, cfg.window,
                         cfg.threshold, batch=cfg.batch, n_recent=cfg.n_recent, n_initial=cfg.n_initial,
                         max_prefill=P)
    eng.set_prompt_mode(mode)
    g = torch.Generator(device="cuda").manual_seed(1)
    k = torch.randn(cfg.layers, cfg.batch, cfg.kv_heads, P, cfg.head_dim, generator=g, device="cuda").to(torch.bfloat16)
    v = torch.randn(k.shape, generator=g, device="cuda").to(torch.bfloat16)
    q = torch.randn(P, cfg.layers, cfg.batch, cfg.q_heads, cfg.head_dim, generator=g, device="cuda").to(torch.bfloat16)
    out = torch.empty_like(q)
    stream = torch.cuda.current_stream()
    best = None
    for r in range(repeats + 1):                       # the first pass is a warm-up
        eng.reset()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        eng.prefill_observed(q, k, v, out)
        e1.record(stream)
        torch.cuda.synchronize()
        eng.synchronize()
        if r > 0:
            ms = e0.elapsed_time(e1)
            best = ms if best is None else min(best, ms)
    launches = eng.info().launches
    eng.close()
    return best, launches


def main():
    import torch
    from . import binding, traces
    ap = argparse.ArgumentParser()
    ap.add_argument("--cases", default="4:256,5:512,2:512,5:2048:4,4:4096:2")
    ap.add_argument("--no-replay", action="store_true")
    args = ap.parse_args()
    rows = []
    for case in args.cases.split(","):
        parts = [int(x) for x in case.split(":")]
        base = traces.CONFIGS[parts[0]]
        cfg = dataclasses.replace(base, prefill=parts[1], budget=max(base.budget, parts[1] + base.window),
                                  layers=parts[2] if len(parts) > 2 else base.layers, budget_frac_tenths=0)
        P, G = cfg.prefill, cfg.group
        flops = cfg.units * 4.0 * G * cfg.head_dim * P * (P + 1) / 2
        tiled_ms, _ = time_case(cfg, binding.PROMPT_TILED)
        replay_ms = None if args.no_replay else time_case(cfg, binding.PROMPT_REPLAY, repeats=1)[0]
        row = {"config": parts[0], "units": cfg.units, "group": G, "prompt": P, "tiled_ms": round(tiled_ms, 3),
               "tiled_TFLOPs": round(flops / tiled_ms / 1e9, 1),
               "replay_ms": None if replay_ms is None else round(replay_ms, 3),
               "speedup": None if replay_ms is None else round(replay_ms / tiled_ms, 1),
               "device": torch.cuda.get_device_name(0)}
        print(json.dumps(row), flush=True)
        rows.append(row)
    print("\n| config | units | G | prompt | tiled ms | algorithmic TFLOP/s | replay ms | replay / tiled |")
    print("|---|---|---|---|---|---|---|---|")
    for r in rows:
        print(f"| {r['config']} | {r['units']} | {r['group']} | {r['prompt']} | {r['tiled_ms']} | {r['tiled_TFLOPs']} | "
              f"{r['replay_ms']} | {r['speedup']} |")


if __name__ == "__main__":
    main()
