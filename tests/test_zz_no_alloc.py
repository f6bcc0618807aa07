"""lazyev_evict_static -- the eviction entry point that takes its work lists from an array
built into the library, for callers that cannot allocate device memory (a plug-in living in a
fixed arena, a process whose pool is already full of KV cache).

It must leave the cache in exactly the state lazyev_evict leaves it in.  The check runs two
engines on the same seeded trace, one evicting through each entry point, and compares
everything an eviction touches -- positions, TS, MRI and the moved K / V rows, bit for bit --
after each of two consecutive evictions.  This file sorts last on purpose, so that a run that
stops at the first failure has already been through every other test; it does not depend on
any of them and passes in a fresh process as well.
"""
import numpy as np
import pytest
import torch

from paper_2506_15969_b200 import binding, traces

pytestmark = pytest.mark.gpu


def _engine(cfg):
    eng = binding.Engine(cfg.layers, cfg.q_heads, cfg.kv_heads, cfg.head_dim, cfg.budget, cfg.window,
                         cfg.threshold, batch=cfg.batch, n_recent=cfg.n_recent, n_initial=cfg.n_initial,
                         max_prefill=cfg.prefill)
    eng.set_auto_evict(False)
    return eng


def test_static_scratch_eviction_matches_the_regular_entry_point():
    cfg = traces.tiny_config(n_recent=8, n_initial=2)
    gen = traces.TraceGen(cfg, seed=12, device="cuda")
    ref, stat = _engine(cfg), _engine(cfg)
    k, v = gen.prefill()
    shape = (cfg.layers, cfg.batch, cfg.kv_heads, cfg.prefill, cfg.head_dim)
    for e in (ref, stat):
        e.prefill(k.view(shape), v.view(shape))
    out = torch.empty(cfg.layers, cfg.batch, cfg.q_heads, cfg.head_dim, dtype=torch.bfloat16, device="cuda")
    events = 0
    for chunk in range(4):                                   # 128 steps: evictions are due at t = 96 and t = 128
        q, kn, vn = gen.steps(32)
        for s in range(32):
            for e in (ref, stat):
                e.decode_step(q[s], kn[s], vn[s], out)
            assert stat.evict_static() == ref.evict()        # also exercises the "not due" early return
        if ref.info().evictions > events:
            events = ref.info().evictions
            a, b = ref.dump_state(kv=True), stat.dump_state(kv=True)
            assert a["n"] == b["n"] == cfg.budget and a["device_status"] == b["device_status"] == 0
            for key in ("pos", "ts", "mri", "k", "v"):
                assert np.array_equal(a[key], b[key]), f"{key} differs after eviction {events}"
    assert events == 2 and stat.info().evictions == 2


def test_static_scratch_rejects_handles_beyond_its_limit():
    # 4097 units exceed the 4096-unit limit of the built-in array; the call must say so and do nothing.
    eng = binding.Engine(4097, 1, 1, 128, 65, 64, 0.01, max_prefill=1)
    z = torch.zeros(4097, 1, 1, 1, 128, dtype=torch.bfloat16, device="cuda")
    eng.prefill(z, z)
    with pytest.raises(binding.LazyEvError) as err:
        eng.evict_static()
    assert err.value.code == binding.ECAPACITY and "4096" in str(err.value)
    assert eng.evict() == 0                                  # the regular entry point is unaffected
    eng.synchronize()
