"""Parity at the benchmark configurations' full sizes, in the launch shapes bench.py times.

The oracle cannot follow thousands of units for thousands of steps, so each case starts in
the configuration's steady state -- a prompt as long as the budget (or, for the
length-proportional budget of configuration 3, far longer than it) -- and runs a little
more than two observation windows: every decode step of the sampled units is compared with
the oracle (outputs, probabilities, then TS / MRI / positions bit for bit), the evictions at
the end of each window are compared row by row, and a pure-oracle run of the same steps
gives the kept-set Jaccard index.  Sampled units include the first and last of the main
launch and units of the second launch that takes the partly filled last round.
"""
import dataclasses

import pytest
import torch

from paper_2506_15969_b200 import traces

pytestmark = pytest.mark.gpu


def _steady(cfg, prefill):
    return dataclasses.replace(cfg, prefill=prefill, name=cfg.name + "-steady")


def _run(cfg, sample, steps, check_every, evictions):
    from tests.harness import Lockstep
    need = cfg.units * (max(cfg.budget, cfg.prefill) + cfg.window) * 512 * 1.1 + cfg.units * cfg.prefill * 512 + (8 << 30)
    free, _ = torch.cuda.mem_get_info()
    if free < need:
        pytest.skip(f"needs {need / 2**30:.0f} GiB of device memory, {free / 2**30:.0f} GiB free")
    ls = Lockstep(cfg, seed=0, sample_units=sample)
    rep = ls.run(steps, check_every=check_every)
    ls.assert_ok()
    assert rep.evictions == evictions and rep.near_tie_events == 0
    assert rep.activations > 0
    return ls


def test_config2_full_batch():
    cfg = _steady(traces.CONFIGS[2], traces.CONFIGS[2].budget)          # 64 units, 2048 + 1..128 tokens
    ls = _run(cfg, [0, 17, 31, 63], 2 * cfg.window + 4, 1, 2)
    assert ls.eng.info().n == cfg.budget + 4


def test_config3_full_batch_long_prompt_and_proportional_budget():
    cfg = _steady(traces.CONFIGS[3], 8000)                              # 4096 units, prompt far above the budget
    ls = _run(cfg, [0, 2047, 4095], 2 * cfg.window + 2, 1, 2)
    inf = ls.eng.info()
    assert inf.n == cfg.budget_at(2 * cfg.window) + 2 == (3 * (8000 + 512)) // 10 + 2


def test_config4_bench_launch_shape():
    cfg = _steady(traces.CONFIGS[4], traces.CONFIGS[4].budget)          # 3584 units, 8192 + 1..128 tokens
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    ls = _run(cfg, [0, 1, sms - 1, sms, 2000, cfg.units - 32, cfg.units - 1], 2 * cfg.window + 2, 1, 2)
    inf = ls.eng.info()
    assert (inf.splits, inf.groups, inf.grid) == (1, 2, sms)
    if sms == 148:
        assert (inf.stages, inf.tail_units, inf.tail_splits) == (5, 32, 4)


def test_config5_full_batch():
    cfg = _steady(traces.CONFIGS[5], traces.CONFIGS[5].budget)          # 12288 units, 4915 + 1..256 tokens
    ls = _run(cfg, [0, 147, 6000, cfg.units - 4, cfg.units - 1], 2 * cfg.window + 2, 1, 2)
    assert ls.eng.info().n == cfg.budget + 2


def test_config2_whole_trace_end_to_end():
    """Configuration 2 from its 512-token prompt through all 4096 decode steps (20 evictions): every step
    of two units in lock step with the oracle, and the kept sets of a pure-oracle run at the end."""
    from tests.harness import Lockstep
    cfg = traces.CONFIGS[2]
    ls = Lockstep(cfg, seed=0, sample_units=[5, 42])
    rep = ls.run(cfg.steps, check_every=4)
    ls.assert_ok()
    assert rep.evictions == (cfg.steps - 1664) // cfg.window + 1 and ls.eng.info().n == cfg.budget
    assert rep.near_tie_events == 0 and rep.min_jaccard >= 0.999
