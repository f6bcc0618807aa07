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


def _run_pair(cfg, seed, chunks, want_events):
    """Two engines on the same trace, one evicting through each entry point; everything an eviction
    touches is compared after every event.  Device memory in use must not move across the calls."""
    gen = traces.TraceGen(cfg, seed=seed, device="cuda")
    ref, stat = _engine(cfg), _engine(cfg)
    k, v = gen.prefill()
    shape = (cfg.layers, cfg.batch, cfg.kv_heads, cfg.prefill, cfg.head_dim)
    for e in (ref, stat):
        e.prefill(k.view(shape), v.view(shape))
    out = torch.empty(cfg.layers, cfg.batch, cfg.q_heads, cfg.head_dim, dtype=torch.bfloat16, device="cuda")
    events = 0
    # The first call on a device resolves the built-in array's address; with CUDA's lazy module loading
    # that is also the moment the runtime materialises the library's static data, once per process.
    # No eviction is due yet, so this call does nothing else.
    assert stat.evict_static() == 0
    for chunk in range(chunks):
        q, kn, vn = gen.steps(32)
        for s in range(32):
            for e in (ref, stat):
                e.decode_step(q[s], kn[s], vn[s], out)
            want = ref.evict()
            torch.cuda.synchronize()
            free_before = torch.cuda.mem_get_info()[0]
            got = stat.evict_static()                        # also exercises the "not due" early return
            torch.cuda.synchronize()
            assert torch.cuda.mem_get_info()[0] == free_before, "evict_static changed the device memory in use"
            assert got == want
        if ref.info().evictions > events:
            events = ref.info().evictions
            a, b = ref.dump_state(kv=True), stat.dump_state(kv=True)
            assert a["n"] == b["n"] == cfg.budget and a["device_status"] == b["device_status"] == 0
            for key in ("pos", "ts", "mri", "k", "v"):
                assert np.array_equal(a[key], b[key]), f"{key} differs after eviction {events}"
    assert events == want_events and stat.info().evictions == want_events


def test_static_scratch_eviction_matches_the_regular_entry_point():
    # 128 steps: evictions are due at t = 96 and t = 128
    _run_pair(traces.tiny_config(n_recent=8, n_initial=2), seed=12, chunks=4, want_events=2)
    # A second pair with another unit count, budget and protection: its source lists have another
    # stride, so they land on top of whatever the first pair left in the shared array.
    _run_pair(traces.tiny_config(batch=3, layers=1, q_heads=6, kv_heads=3, prefill=70, budget=111, window=16,
                                 n_recent=5, n_initial=0), seed=13, chunks=3, want_events=4)


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
    eng.close()
    # The other half of the limit: few enough units, but units * budget above 2^20 source indices.
    eng = binding.Engine(129, 1, 1, 128, 8192, 64, 0.01, max_prefill=1)
    z = torch.zeros(129, 1, 1, 1, 128, dtype=torch.bfloat16, device="cuda")
    eng.prefill(z, z)
    with pytest.raises(binding.LazyEvError) as err:
        eng.evict_static()
    assert err.value.code == binding.ECAPACITY and str(129 * 8192) in str(err.value)
    eng.synchronize()
