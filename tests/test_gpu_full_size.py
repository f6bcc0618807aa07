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


def _whole_trace(cfg, sample, pure_units, check_every):
    """A configuration from its own prompt through all of its decode steps, on fewer layers / a
    smaller batch than the benchmark but with more units than SMs plus a partly filled round, so the
    launch shape (persistent grid + second launch) is the benchmark's.  The sampled units run in lock
    step with the oracle: TS / MRI / positions bit for bit at every step (the bookkeeping consumes the
    GPU's probabilities), attention outputs and probabilities every `check_every` steps and at every
    window end, every eviction row by row; `pure_units` also get a pure-oracle run for the Jaccard bar."""
    from tests.harness import Lockstep
    ls = Lockstep(cfg, seed=0, sample_units=sample, pure_units=pure_units)
    rep = ls.run(cfg.steps, check_every=check_every)
    ls.assert_ok()
    assert rep.near_tie_events == 0 and rep.min_jaccard >= 0.999
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


def test_config4_whole_trace_on_two_layers():
    """Configuration 4 (28 query / 4 KV heads, budget 8192, window 128, 10 % recurring tokens with
    log-uniform periods, one-shot spikes) from its 256-token prompt through all 16384 steps: 65
    evictions over 8192 candidates each, on 184 units (148 + 36: the second launch takes the rest)."""
    cfg = dataclasses.replace(traces.CONFIGS[4], batch=23, layers=2, name="cfg4-b23-l2")
    assert cfg.units == 184
    ls = _whole_trace(cfg, [3, 150], [150], check_every=97)
    inf, cnt = ls.eng.info(), ls.eng.counters()
    assert ls.rep.evictions == (cfg.steps - 8064) // cfg.window + 1 and inf.n == cfg.budget
    assert inf.tail_units == 36 or torch.cuda.get_device_properties(0).multi_processor_count != 148
    # which route the selection took, per unit and event (at the default threshold few tokens are
    # re-activated, so the k-th score is 0 and the tie rule decides)
    assert cnt.select_radix_units + cnt.select_zero_cut_units == ls.rep.evictions * cfg.units
    assert cnt.device_status == 0


def test_config5_whole_trace_on_one_layer():
    """Configuration 5 (40 query / 8 KV heads, budget 4915, window 256, 32 protected recent tokens)
    from its 512-token prompt through all 16384 steps on 200 units."""
    cfg = dataclasses.replace(traces.CONFIGS[5], batch=25, layers=1, name="cfg5-b25-l1")
    assert cfg.units == 200
    ls = _whole_trace(cfg, [0, 199], [199], check_every=131)
    cnt = ls.eng.counters()
    assert ls.rep.evictions == (cfg.steps - 4608) // cfg.window + 1 and ls.eng.info().n == cfg.budget
    assert cnt.select_radix_units + cnt.select_zero_cut_units == ls.rep.evictions * cfg.units


@pytest.mark.parametrize("config", [4, 5])
def test_dense_activation_takes_the_radix_route_at_full_candidate_counts(config):
    """The paper's own thresholds (1e-4 .. 5e-4, Appendix C) on these traces re-activate a large share
    of all tokens at every step: nearly every score is non-zero, the selection has to find the k-th of
    8192 (5139) distinct fp64 keys with the radix passes, and the fused epilogue updates TS / MRI for
    thousands of tokens per unit and step.  Full batch, the benchmark's launch shape, a little more than
    two windows from a prompt as long as the budget."""
    base = traces.CONFIGS[config]
    cfg = dataclasses.replace(base, prefill=base.budget, alpha=1e-4, name=base.name + "-dense")
    sample = [0, 147, 148, cfg.units - 1]
    ls = _run(cfg, sample, 2 * cfg.window + 2, 1, 2)
    cnt = ls.eng.counters()
    assert cnt.select_radix_units == 2 * cfg.units and cnt.select_zero_cut_units == 0
    assert ls.rep.activations > 0.2 * ls.rep.tokens_seen       # a dense regime indeed
