"""Host-side logic of bench.py that needs no GPU: which steps are replayed untimed, how a workload is
shaped from the flags, and when the stored ncu traffic figure is still valid."""
import argparse
import dataclasses
import hashlib
import os

import bench
from paper_2506_15969_b200 import traces


def _args(**kw):
    base = dict(config=4, batch=0, layers=0, fast_start=False, alpha=0.0)
    base.update(kw)
    return argparse.Namespace(**base)


def test_first_eviction_step_matches_the_configurations():
    # the first decision step at which the cache exceeds the budget (Section 4: t = kW and n > B)
    want = {1: 384, 2: 1664, 4: 8064, 5: 4608}
    for c, t in want.items():
        cfg = traces.CONFIGS[c]
        assert bench.first_eviction_step(cfg) == t
        assert cfg.prefill + t > cfg.budget_at(t) and cfg.prefill + t - cfg.window <= cfg.budget_at(t - cfg.window)
    cfg3 = traces.CONFIGS[3]                       # budget = 30 % of the length: 1024 + 256 > 384
    assert bench.first_eviction_step(cfg3) == 256


def test_steady_state_start():
    assert bench.steady_state_start(traces.CONFIGS[4], 256) == 8064
    cfg3 = traces.CONFIGS[3]
    start = bench.steady_state_start(cfg3, 256)    # a growing budget is timed near the end of the trace
    assert start % cfg3.window == 0 and cfg3.steps - 2 * cfg3.window - 256 < start <= cfg3.steps - 256 - cfg3.window


def test_pick_config_shapes_the_workload_from_the_flags():
    cfg = bench.pick_config(_args(batch=4, layers=37, fast_start=True, alpha=1e-4))
    base = traces.CONFIGS[4]
    assert (cfg.batch, cfg.layers, cfg.prefill, cfg.threshold) == (4, 37, base.budget, 1e-4)
    assert cfg.units == 4 * 37 * 4 and "alpha" in cfg.name and "faststart" in cfg.name
    assert bench.pick_config(_args()) == base and base.threshold == 8.0 / (base.budget + base.window)


def test_ncu_traffic_is_dropped_when_the_kernel_sources_change(tmp_path, monkeypatch):
    csrc = os.path.join(bench.ROOT, "paper_2506_15969_b200", "csrc")
    current = {name: hashlib.sha256(open(os.path.join(csrc, name), "rb").read()).hexdigest()
               for name in bench.NCU_DECODE_CAPTURE["sha256"]}
    monkeypatch.setitem(bench.NCU_DECODE_CAPTURE, "sha256", current)
    got = bench.ncu_traffic(1e9)
    assert got == bench.NCU_DECODE_CAPTURE["traffic_per_algorithmic_byte"] * 1e9
    stale = dict(current, **{"decode.cu": "0" * 64})
    monkeypatch.setitem(bench.NCU_DECODE_CAPTURE, "sha256", stale)
    assert bench.ncu_traffic(1e9) is None
