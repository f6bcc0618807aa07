"""The synthetic trace generator: reproducibility (subset = slice of the whole,
chunking does not matter, CPU bits = CUDA bits) and the advertised statistics."""
import dataclasses
import math
import random

import pytest
import torch

from paper_2506_15969_b200 import traces as tr


def test_mix_matches_python_integers():
    rnd = random.Random(1)
    vals = [rnd.getrandbits(64) for _ in range(200)] + [0, 1, (1 << 64) - 1, 1 << 63]
    x = torch.tensor([tr._s64(v) for v in vals], dtype=torch.int64)
    got = tr._mix(x).tolist()
    assert got == [tr._s64(tr.mix_python(v)) for v in vals]


def test_configs_match_the_benchmark_table():
    c = tr.CONFIGS
    assert [c[i].units for i in range(1, 6)] == [2, 64, 4096, 3584, 12288]
    assert [c[i].group for i in range(1, 6)] == [4, 7, 4, 7, 5]
    assert c[3].budget_at(256) == 384 and c[3].budget_at(8192) == 2764 and c[3].budget_at(10 ** 6) == 4096
    assert c[4].budget_at(5) == 8192 and c[5].capacity() == 4915 + 256
    assert c[4].threshold == pytest.approx(8 / 8320)


def test_subset_of_units_equals_slice_and_chunking_is_irrelevant():
    cfg = tr.tiny_config()
    full = tr.TraceGen(cfg, seed=3)
    sub = tr.TraceGen(cfg, seed=3, units=[1, 6])
    kf, vf = full.prefill(); ks, vs = sub.prefill()
    assert torch.equal(kf[[1, 6]], ks) and torch.equal(vf[[1, 6]], vs)
    qa, ka, va = full.steps(32)
    q1, k1, v1 = sub.steps(7); q2, k2, v2 = sub.steps(25)
    assert torch.equal(qa[:, [1, 6]], torch.cat([q1, q2]))
    assert torch.equal(ka[:, [1, 6]], torch.cat([k1, k2]))
    assert torch.equal(va[:, [1, 6]], torch.cat([v1, v2]))
    # skipping ahead lands on the same walk
    late = tr.TraceGen(cfg, seed=3, units=[6]); late.skip_to(32)
    qb, _, _ = full.steps(5); ql, _, _ = late.steps(5)
    assert torch.equal(qb[:, [6]], ql)
    other = tr.TraceGen(cfg, seed=4, units=[1, 6])
    assert not torch.equal(other.prefill()[0], ks)


def test_value_statistics():
    cfg = tr.tiny_config(batch=4, layers=4, prefill=256)
    g = tr.TraceGen(cfg, seed=0)
    k, v = g.prefill()
    for x in (k.float(), v.float()):
        assert abs(x.mean().item()) < 0.01 and abs(x.var().item() - 1.0) < 0.02
        assert x.abs().max().item() < 6.01
    plain = dataclasses.replace(cfg, plant_prob_1024=0, spike_prob_1024=0)
    g = tr.TraceGen(plain, seed=0)
    qs = torch.cat([g.steps(32)[0] for _ in range(12)]).float()[64:]      # past the warm-up
    assert abs(qs.var().item() - 1.0) < 0.05
    lag1 = (qs[1:] * qs[:-1]).mean().item() / qs.var().item()
    assert abs(lag1 - 0.95) < 0.02
    iid = tr.TraceGen(dataclasses.replace(plain, query="iid"), seed=0)
    qi = torch.cat([iid.steps(32)[0] for _ in range(4)]).float()
    assert abs((qi[1:] * qi[:-1]).mean().item()) < 0.02


def test_firing_adds_four_to_the_scaled_logit():
    cfg = tr.tiny_config()
    g = tr.TraceGen(cfg, seed=5)
    g0 = tr.TraceGen(dataclasses.replace(cfg, plant_prob_1024=0, spike_prob_1024=0), seed=5)
    seen = 0
    for chunk in range(6):
        t0 = g.t_done + 1
        es, eu, ep = g.firing_events(t0, 32)
        q, _, _ = g.steps(32); qn, _, _ = g0.steps(32)
        assert es.numel() > 0
        k = g._to_bf16(g.key_int(eu, ep)).double()                    # [E, D]
        # steps where exactly one token of the unit fires
        key = (es * g.U + eu).tolist()
        for e in range(es.numel()):
            if key.count(key[e]) != 1:
                continue
            dq = (q[es[e], eu[e]].double() - qn[es[e], eu[e]].double())      # [G, D]
            logit = dq @ k[e] / math.sqrt(cfg.head_dim)
            assert torch.all((logit - 4.0).abs() < 0.15), logit
            assert ep[e] < cfg.prefill + t0 + es[e] - 1                      # the token already exists
            seen += 1
    assert seen > 50


def test_planted_tokens_fire_periodically():
    cfg = tr.tiny_config(spike_prob_1024=0)
    g = tr.TraceGen(cfg, seed=9, units=[2])
    fires = {}
    for c in range(12):
        t0 = 1 + 32 * c
        es, eu, ep = g.firing_events(t0, 32)
        for s, p in zip(es.tolist(), ep.tolist()):
            fires.setdefault(p, []).append(t0 + s)
    multi = [v for v in fires.values() if len(v) >= 3]
    assert len(multi) > 5
    for v in multi:
        gaps = {b - a for a, b in zip(v, v[1:])}
        assert len(gaps) == 1 and cfg.period_lo <= gaps.pop() <= cfg.period_hi
    frac = len([p for p in fires if p < cfg.prefill]) / cfg.prefill
    assert 0.03 < frac < 0.2                                          # about 10 % are planted


def test_config1_plants_exactly_32_prefill_tokens():
    g = tr.TraceGen(tr.CONFIGS[1], seed=0)
    assert g._prefill_planted.sum(dim=1).tolist() == [32, 32]
    pos = set()
    for c in range(20):
        es, eu, ep = g.firing_events(1 + 32 * c, 32)
        pos |= {(u, p) for u, p in zip(eu.tolist(), ep.tolist())}
    assert all(p < 256 for _, p in pos) and len(pos) == 64


def test_octave_periods_cover_the_range():
    g = tr.TraceGen(tr.CONFIGS[4], seed=0, units=[0])
    period, phase = g._period_phase(g.units[:, None], torch.arange(20000)[None, :])
    assert period.min().item() >= 64 and period.max().item() < 4096
    assert (phase < period).all() and (phase >= 0).all()
    logs = torch.log2(period.double())
    assert abs(logs.mean().item() - 9.0) < 0.1                        # log-uniform on [64, 4096)


@pytest.mark.gpu
def test_cpu_and_cuda_bits_agree():
    cfg = tr.tiny_config()
    a = tr.TraceGen(cfg, seed=2, device="cpu")
    b = tr.TraceGen(cfg, seed=2, device="cuda")
    for x, y in zip(a.prefill(), b.prefill()):
        assert torch.equal(x, y.cpu())
    for _ in range(3):
        for x, y in zip(a.steps(32), b.steps(32)):
            assert torch.equal(x, y.cpu())
