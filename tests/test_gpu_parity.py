"""Parity of the CUDA library with the fp64 oracle, through the C ABI.

Tolerances (see tests/harness.py): attention output within 2e-3 absolute plus
1e-2 relative; probabilities within 1e-4 absolute; TS, MRI, positions, evict
sets and moved K/V rows bit-exact when the oracle's bookkeeping consumes the
GPU's probabilities; kept-set Jaccard with the pure oracle >= 0.999.
"""
import dataclasses

import numpy as np
import pytest
import torch

from paper_2506_15969_b200 import binding, traces

pytestmark = pytest.mark.gpu


def lockstep(*a, **kw):
    from tests.harness import Lockstep
    return Lockstep(*a, **kw)


@pytest.mark.parametrize("splits", [1, 2, 3, 4, 5, 8])
def test_attention_and_tracking_without_eviction(splits):
    """Budget >= prompt + steps: the GPU output is full attention at every step;
    n sweeps across page boundaries and ragged tails (97 .. 296 tokens)."""
    cfg = traces.tiny_config(budget=512, window=32, prefill=96, steps=200)
    ls = lockstep(cfg, seed=1, sample_units=range(cfg.units), splits=splits)
    rep = ls.run(200)
    ls.assert_ok()
    assert rep.evictions == 0 and rep.steps == 200
    assert rep.activations > 200                      # the tracking path was exercised
    assert ls.eng.info().splits == splits


def test_partly_filled_last_round_goes_to_a_second_launch():
    """158 units on 148 SMs: 148 in the main launch, the other 10 in a launch with larger clusters."""
    cfg = traces.tiny_config(batch=2, layers=79, q_heads=7, kv_heads=1, budget=1520, window=32, prefill=1500)
    ls = lockstep(cfg, seed=14, sample_units=[0, 1, 147, 148, 149, 156, 157], pure=False)
    ls.run(40)
    ls.assert_ok()
    inf = ls.eng.info()
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    assert inf.splits == 1 and inf.grid == sms
    assert inf.tail_units == cfg.units - sms and inf.tail_splits > 1
    assert ls.rep.evictions == 1


def test_softmax_reference_is_raised_late():
    """Logits that grow by far more than the 2^8 margin inside one unit, and a dominant token:
    the lazily raised softmax reference must give the same sums as an exact running maximum."""
    eng = binding.Engine(1, 4, 1, 128, 400, 32, 0.05, max_prefill=200)
    from oracle import lazyev_oracle as orc
    gen = torch.Generator().manual_seed(5)
    k = torch.randn(200, 128, generator=gen)
    k *= torch.linspace(0.05, 6.0, 200)[:, None]            # later keys are much longer
    v = torch.randn(200, 128, generator=gen)
    q = (torch.randn(4, 128, generator=gen) + 0.8 * k[150] / k[150].norm() * 11.3).to(torch.bfloat16)
    kb, vb = k.to(torch.bfloat16), v.to(torch.bfloat16)
    eng.prefill(kb.view(1, 1, 1, 200, 128).cuda(), vb.view(1, 1, 1, 200, 128).cuda())
    out = torch.empty(1, 1, 4, 128, dtype=torch.bfloat16, device="cuda")
    kn, vn = torch.randn(1, 128, generator=gen).to(torch.bfloat16), torch.randn(1, 128, generator=gen).to(torch.bfloat16)
    eng.decode_step(q.view(1, 1, 4, 128).cuda(), kn.view(1, 1, 1, 128).cuda(), vn.view(1, 1, 1, 128).cuda(), out)
    o = orc.OracleUnit(4, 128, 400, 32, 0.05)
    o.prefill(kb.double().numpy(), vb.double().numpy())
    ref_out, ref_pbar = o.attend(q.double().numpy(), kn[0].double().numpy(), vn[0].double().numpy())
    d = eng.dump_state()
    assert np.abs(d["pbar"][0] - ref_pbar).max() <= 1e-4
    assert ref_pbar.max() > 0.05                            # some token really dominates
    got = out.view(4, 128).double().cpu().numpy()
    assert (np.abs(got - ref_out) <= 2e-3 + 1e-2 * np.abs(ref_out)).all()


@pytest.mark.parametrize("groups", [1, 2])
@pytest.mark.parametrize("splits,stages", [(1, 2), (1, 3), (2, 3), (1, 5), (4, 2), (3, 4), (6, 5)])
def test_ring_depths_and_warp_groups(splits, stages, groups):
    """Shallow and odd ring depths with one and two groups of consumer warps: with two groups a
    stage's consecutive uses go to different groups, and a block's page count may be odd, so
    the group that owns a logit tile changes from unit to unit."""
    cfg = traces.tiny_config(budget=900, window=32, prefill=500, steps=200, batch=1, layers=2)
    ls = lockstep(cfg, seed=11, sample_units=range(cfg.units), splits=splits, stages=stages, groups=groups,
                  pure=False)
    ls.run(150)
    ls.assert_ok()
    inf = ls.eng.info()
    assert (inf.splits, inf.stages, inf.groups) == (splits, stages, groups)


@pytest.mark.parametrize("groups", [1, 2])
def test_many_units_per_block(groups):
    """More units than blocks: every block walks several units, so the probabilities of one unit are
    produced while the next one streams, and the last one is flushed at the end."""
    cfg = traces.tiny_config(batch=40, layers=8, q_heads=14, kv_heads=2, budget=300, window=32, prefill=280)
    assert cfg.units == 640
    ls = lockstep(cfg, seed=13, sample_units=[0, 1, 147, 148, 149, 295, 296, 500, 638, 639], groups=groups, pure=False)
    ls.run(70)
    ls.assert_ok()
    assert ls.rep.evictions == 2


@pytest.mark.parametrize("groups", [1, 2])
def test_many_units_with_fewer_pages_than_warp_groups(groups):
    """Thousands of units with one or two pages each: every block walks two dozen units, a group of
    consumer warps owns no page in every other unit, and the page ring is reused many times (the
    order in which warps look at the ring's barriers must hold across unit boundaries)."""
    cfg = traces.tiny_config(batch=32, layers=28, q_heads=8, kv_heads=4, budget=200, window=32, prefill=10)
    assert cfg.units == 3584
    ls = lockstep(cfg, seed=19, sample_units=[0, 147, 148, 2000, 3551, 3552, 3583], groups=groups, pure=False)
    ls.run(70)                                                # 11 .. 80 cached tokens: crosses the one-page boundary
    ls.assert_ok()
    assert ls.eng.counters().device_status == 0


@pytest.mark.parametrize("q_heads,kv_heads", [(7, 1), (10, 2), (8, 1), (2, 2), (6, 2)])
def test_group_sizes(q_heads, kv_heads):
    cfg = traces.tiny_config(q_heads=q_heads, kv_heads=kv_heads, batch=3, layers=1, budget=400, prefill=70)
    ls = lockstep(cfg, seed=2, sample_units=range(cfg.units))
    ls.run(100)
    ls.assert_ok()


@pytest.mark.parametrize("splits", [0, 1, 4])
def test_lockstep_with_evictions(splits):
    """Tracking, lagged eviction, selection and in-place compaction over 12 windows."""
    cfg = traces.tiny_config()
    ls = lockstep(cfg, seed=3, sample_units=range(cfg.units), splits=splits)
    rep = ls.run(400)
    ls.assert_ok()
    assert rep.evictions == (400 - 96) // 32 + 1       # first at t = 96 (n = 192 > 160)
    assert rep.near_tie_events == 0


def test_protected_tokens_and_score_variants():
    cfg = traces.tiny_config(n_recent=8, n_initial=4, budget=130, window=16, prefill=100)
    for mode in (binding.SCORE_H1_PLUS_H2, binding.SCORE_H1_ONLY, binding.SCORE_H2_ONLY,
                 binding.SCORE_H1_PLUS_H2_DECREASING):
        ls = lockstep(cfg, seed=4, sample_units=[0, 3, 7], score_mode=mode)
        rep = ls.run(160)
        ls.assert_ok()
        assert rep.evictions >= 8
        d = ls.eng.dump_state(0, 1)
        assert d["pos"][0][:4].tolist() == [0, 1, 2, 3]                 # initial tokens survive
        assert d["pos"][0][-8:].tolist() == list(range(100 + 160 - 8, 100 + 160))


def test_dynamic_budget_and_long_prompt():
    """Budget follows 30 % of the length (config 3's rule) and the prompt is longer than it."""
    cfg = traces.tiny_config(budget=200, window=32, n_recent=32, prefill=150, budget_frac_tenths=3)
    ls = lockstep(cfg, seed=5, sample_units=[1, 4])
    rep = ls.run(320)
    ls.assert_ok()
    assert rep.evictions == 10
    assert ls.eng.info().n == cfg.budget_at(320)


def test_shuffled_page_table_gives_identical_results():
    cfg = traces.tiny_config()
    eng = binding.Engine(cfg.layers, cfg.q_heads, cfg.kv_heads, 128, cfg.budget, cfg.window, cfg.threshold,
                         batch=cfg.batch, n_recent=cfg.n_recent, max_prefill=cfg.prefill)
    total = eng.info().units * eng.info().pages_per_unit
    perm = np.random.default_rng(0).permutation(total).astype(np.int32)
    eng.close()
    a = lockstep(cfg, seed=6, sample_units=[0, 5], pure=False)
    b = lockstep(cfg, seed=6, sample_units=[0, 5], pure=False, page_table=perm)
    a.run(200); b.run(200)
    a.assert_ok(); b.assert_ok()
    da, db = a.eng.dump_state(kv=True), b.eng.dump_state(kv=True)
    for key in ("pos", "ts", "mri", "pbar", "k", "v"):
        assert np.array_equal(da[key], db[key]), key
    assert torch.equal(a.out, b.out)
    with pytest.raises(binding.LazyEvError):
        b.eng.set_page_table(perm)                       # only before prefill


def test_threshold_extremes_reduce_to_a_sliding_window():
    """alpha > 1: nothing activates, every score ties at 0; alpha = 0: everything
    activates, every score ties at 1.  Either way the B most recent tokens stay."""
    for alpha in (1.5, 1e-30):
        cfg = traces.tiny_config(alpha=alpha, batch=1, layers=1)
        ls = lockstep(cfg, seed=7, sample_units=[0, 1])
        ls.run(128)
        ls.assert_ok()
        d = ls.eng.dump_state()
        n_total = cfg.prefill + 128
        for u in range(cfg.units):
            assert d["pos"][u].tolist() == list(range(n_total - cfg.budget, n_total))
            if alpha > 1:
                assert not d["mri"][u].any()
            else:
                assert (d["ts"][u] == 128).all() and (d["mri"][u][:-1] == 1).all()


def test_config1_full_trace():
    """Benchmark configuration 1 end to end: 256-token prompt, 1024 steps, 6 evictions."""
    cfg = traces.CONFIGS[1]
    ls = lockstep(cfg, seed=0, sample_units=[0, 1])
    rep = ls.run(cfg.steps, check_every=1)
    ls.assert_ok()
    assert rep.evictions == 6 and ls.eng.info().n == 512
    # planted recurring tokens must survive: the point of the method
    planted = ls.gen_cpu._prefill_planted.numpy()
    for i in range(2):
        kept = set(ls.shadow[i].pos.tolist())
        alive = sum(1 for p in np.nonzero(planted[i])[0] if int(p) in kept)
        assert alive >= 30, alive


@pytest.mark.parametrize("prefill,splits", [(8150, 1), (9000, 1), (16900, 2), (16900, 0)])
def test_full_cache_long_contexts(prefill, splits):
    """No eviction (budget above prompt + steps, the FullKV setting) at lengths where a unit's logits
    fill tensor memory and spill to shared memory (8193..9040 tokens, one block per unit) and where
    a unit needs a cluster (16.9 k tokens)."""
    cfg = traces.tiny_config(batch=1, layers=2, q_heads=14, kv_heads=2, budget=prefill + 200, window=64,
                             prefill=prefill, n_recent=64)
    ls = lockstep(cfg, seed=15, sample_units=[0, 3], pure=False, splits=splits)
    ls.run(48, check_every=1)
    ls.assert_ok()
    inf = ls.eng.info()
    assert ls.rep.evictions == 0 and inf.n == prefill + 48
    assert splits == 0 or inf.splits == splits


def test_per_step_eviction_window_of_one():
    """W = 1: an eviction decision at every step (the greedy setting the paper contrasts with)."""
    cfg = traces.tiny_config(budget=120, window=1, n_recent=1, prefill=100)
    ls = lockstep(cfg, seed=16, sample_units=[0, 2, 7])
    ls.run(90)
    ls.assert_ok()
    assert ls.rep.evictions == 90 - 20 and ls.eng.info().n == 120


@pytest.mark.parametrize("case", range(24))
def test_random_shapes_and_launch_shapes(case):
    """Seeded random combinations of group size, unit count, cache length, window, protection and
    forced launch shapes (cluster size, ring depth, warp groups), a few windows each."""
    rng = np.random.default_rng(1000 + case)
    kv_heads = int(rng.integers(1, 4))
    group = int(rng.integers(1, 9))
    batch, layers = int(rng.integers(1, 4)), int(rng.integers(1, 4))
    window = int(rng.choice([8, 16, 32, 48]))
    n_recent = int(rng.integers(1, window + 1))
    n_initial = int(rng.integers(0, 5))
    prefill = int(rng.integers(1, 700))
    budget = max(n_recent + n_initial + 2, window + 1, int(prefill * rng.uniform(0.5, 1.3)))
    splits = int(rng.choice([0, 0, 1, 2, 3, 5, 8]))
    groups = int(rng.choice([0, 1, 2]))
    stages = int(rng.choice([0, 0, 2, 3, 4, 5]))
    cfg = traces.tiny_config(batch=batch, layers=layers, q_heads=group * kv_heads, kv_heads=kv_heads, prefill=prefill,
                             budget=budget, window=window, n_recent=n_recent, n_initial=n_initial,
                             alpha=float(rng.choice([0.0, 0.003, 0.02])), period_lo=40, period_hi=120)
    units = sorted(set(int(x) for x in rng.integers(0, cfg.units, size=3)))
    ls = lockstep(cfg, seed=case, sample_units=units, splits=splits, stages=stages, groups=groups, pure=False)
    rep = ls.run(3 * window + 5)
    ls.assert_ok()
    assert rep.steps == 3 * window + 5 and ls.eng.dump_state(0, 1)["device_status"] == 0


def test_mri_histogram_and_quantile_match_the_oracle():
    """The live distribution of MRI (the paper's offline rule for choosing W): bit-exact counts."""
    from oracle import lazyev_oracle as orc
    cfg = traces.tiny_config(budget=400, window=32, prefill=200, alpha=0.004)
    ls = lockstep(cfg, seed=9, sample_units=range(cfg.units), pure=False)
    ls.run(230)
    ls.assert_ok()
    mri = [sh.MRI for sh in ls.shadow]
    assert sum(int((m > 0).sum()) for m in mri) > 200              # plenty of re-activated tokens
    for bins in (2, 17, 64, 9000, 65536):
        assert np.array_equal(ls.eng.mri_histogram(bins), orc.mri_histogram(mri, bins)), bins
    assert np.array_equal(ls.eng.mri_histogram(64, 3, 2), orc.mri_histogram(mri[3:5], 64))
    for frac in (0.1, 0.5, 0.8, 1.0):
        assert ls.eng.mri_quantile(frac) == orc.mri_quantile(mri, frac)
        assert ls.eng.mri_quantile(frac, 5, 1) == orc.mri_quantile(mri[5:6], frac)
    with pytest.raises(binding.LazyEvError):
        ls.eng.mri_histogram(1)
    with pytest.raises(binding.LazyEvError):
        ls.eng.mri_histogram(16, 7, 2)


@pytest.mark.parametrize("mode", [binding.PROMPT_TILED, binding.PROMPT_REPLAY])
@pytest.mark.parametrize("prefill,q_heads,kv_heads", [(150, 8, 2), (333, 8, 2), (512, 10, 2), (700, 7, 1), (2048, 6, 2),
                                                     (97, 2, 2), (260, 16, 2), (17, 8, 2)])
def test_observed_prompt_then_decode(prefill, q_heads, kv_heads, mode):
    """lazyev_prefill_observed: causal prompt attention with tracking from the first token, by the tiled
    tensor-core kernel and by the row-by-row replay through the decode kernel, each against the oracle
    (outputs and probabilities within the tolerances; TS / MRI bit for bit, the oracle's tracking
    consuming the probabilities the library dumped for every prompt row); then decoding with evictions
    continues in lock step."""
    if mode == binding.PROMPT_REPLAY and prefill > 600:
        pytest.skip("the replay is covered at the shorter prompts")
    cfg = traces.tiny_config(prefill=prefill, budget=prefill + 40, window=32, alpha=0.02, q_heads=q_heads,
                             kv_heads=kv_heads, batch=2, layers=2 if prefill < 1000 else 1)
    sample = [0, cfg.units // 2, cfg.units - 1]
    ls = lockstep(cfg, seed=17, sample_units=sample, observed=True, prompt_mode=mode)
    d = ls.eng.dump_state(0, 1)
    assert (d["ts"][0] >= np.arange(prefill) - (prefill - 1)).all() and d["ts"][0].max() == 0
    assert (d["mri"][0] > 0).sum() >= min(5, prefill // 8)    # prompt tokens were re-activated
    rep = ls.run(100, check_every=1 if prefill < 1000 else 8)
    ls.assert_ok()
    assert rep.evictions == 2


@pytest.mark.parametrize("batch,layers,prefill", [(3, 2, 400), (40, 4, 300)])
def test_tiled_prompt_kernel_agrees_with_the_replay(batch, layers, prefill):
    """The two implementations of the prompt pass on the same prompt: attention outputs equal to within
    bf16 rounding, probabilities to float32 rounding; the statistics they produce may differ only for
    tokens whose probability came within that rounding of the threshold.  The second case has 320 units:
    every block of the tiled kernel walks two or three units, so its rings, Q slots and output stores run
    across unit boundaries."""
    from tests.harness import make_engine
    cfg = traces.tiny_config(prefill=prefill, budget=prefill + 100, window=32, alpha=0.02, batch=batch, layers=layers)
    gen = traces.TraceGen(cfg, 23, device="cuda")
    k, v = gen.prefill()
    shape = (cfg.layers, cfg.batch, cfg.kv_heads, cfg.prefill, 128)
    g = torch.Generator().manual_seed(5)
    q = torch.randn(cfg.prefill, cfg.units, cfg.group, 128, generator=g).to(torch.bfloat16).cuda()
    dumped = min(cfg.units, 24)                               # per-row probabilities of the last units only
    res = {}
    for mode in (binding.PROMPT_TILED, binding.PROMPT_REPLAY):
        eng = make_engine(cfg)
        eng.set_prompt_mode(mode)
        rows = torch.zeros(dumped, cfg.prefill, cfg.prefill, dtype=torch.float32, device="cuda")
        out = torch.zeros(cfg.prefill, cfg.units, cfg.group, 128, dtype=torch.bfloat16, device="cuda")
        eng.set_prompt_dump(rows, cfg.units - dumped, dumped)
        eng.prefill_observed(q, k.view(shape), v.view(shape), out)
        eng.synchronize()
        res[mode] = (out.float().cpu(), rows.cpu(), eng.dump_state())
        if cfg.units <= 148:
            assert eng.info().launches == (3 if mode == binding.PROMPT_TILED else 2 + cfg.prefill)
    (o_t, r_t, d_t), (o_r, r_r, d_r) = res[binding.PROMPT_TILED], res[binding.PROMPT_REPLAY]
    assert ((o_t - o_r).abs() <= 4e-3 + 2e-2 * o_r.abs()).all()            # two implementations, each within the oracle's bar
    assert (r_t - r_r).abs().max() <= 2e-6
    assert np.abs(d_t["pbar"] - d_r["pbar"]).max() <= 2e-6
    near = ((r_r - cfg.threshold).abs() <= 2e-6).any(dim=1).numpy()            # [dumped units, tokens]: ever close to alpha
    same = (d_t["ts"] == d_r["ts"]) & (d_t["mri"] == d_r["mri"])
    assert (same[cfg.units - dumped:] | near).all() and same.mean() > 0.99
    assert d_t["device_status"] == 0 and d_r["device_status"] == 0


def test_reset_then_a_new_sequence_gives_the_same_results_as_a_fresh_handle():
    """A handle that served one batch of sequences is reset and serves another: outputs, statistics
    and cache are those of a freshly created handle (nothing of the first batch leaks through)."""
    from tests.harness import make_engine
    cfg = traces.tiny_config()
    shape = (cfg.layers, cfg.batch, cfg.kv_heads, cfg.prefill, 128)
    used, fresh = make_engine(cfg), make_engine(cfg)
    out_u = torch.empty(cfg.layers, cfg.batch, cfg.q_heads, 128, dtype=torch.bfloat16, device="cuda")
    out_f = torch.empty_like(out_u)
    first = traces.TraceGen(cfg, 30, device="cuda")
    k, v = first.prefill()
    used.prefill(k.view(shape), v.view(shape))
    for _ in range(5):
        q, kn, vn = first.steps(32)
        for s in range(32):
            used.decode_step(q[s], kn[s], vn[s], out_u)
    assert used.info().evictions == 3
    used.reset()
    assert (used.info().t, used.info().n) == (0, 0)
    second = traces.TraceGen(cfg, 31, device="cuda")
    k, v = second.prefill()
    used.prefill(k.view(shape), v.view(shape)); fresh.prefill(k.view(shape), v.view(shape))
    for _ in range(4):
        q, kn, vn = second.steps(32)
        for s in range(32):
            used.decode_step(q[s], kn[s], vn[s], out_u)
            fresh.decode_step(q[s], kn[s], vn[s], out_f)
            assert torch.equal(out_u, out_f)
    du, df = used.dump_state(kv=True), fresh.dump_state(kv=True)
    for key in ("pos", "ts", "mri", "pbar", "k", "v"):
        assert np.array_equal(du[key], df[key]), key
    assert du["n"] == df["n"] == cfg.budget + 0 and du["device_status"] == 0


def test_resume_from_a_snapshot_continues_bit_for_bit():
    """dump_state -> load_state into a fresh handle (with a larger capacity): the resumed run must
    produce the same outputs, statistics, evictions and cache as the run that was never stopped."""
    from tests.harness import make_engine
    cfg = traces.tiny_config()
    gen = traces.TraceGen(cfg, 21, device="cuda")
    a = make_engine(cfg)
    k, v = gen.prefill()
    shape = (cfg.layers, cfg.batch, cfg.kv_heads, cfg.prefill, 128)
    a.prefill(k.view(shape), v.view(shape))
    out_a = torch.empty(cfg.layers, cfg.batch, cfg.q_heads, 128, dtype=torch.bfloat16, device="cuda")
    out_b = torch.empty_like(out_a)
    for _ in range(5):                                       # 160 steps: three evictions, t not on a window edge + 0
        q, kn, vn = gen.steps(32)
        for s in range(32):
            a.decode_step(q[s], kn[s], vn[s], out_a)
    q, kn, vn = gen.steps(13)
    for s in range(13):
        a.decode_step(q[s], kn[s], vn[s], out_a)
    snap = a.dump_state(kv=True)
    big = dataclasses.replace(cfg, prefill=cfg.prefill + 200)          # another capacity than the original
    b = make_engine(big)
    with pytest.raises(binding.LazyEvError):
        b.load_state({k2: (v2[:3] if hasattr(v2, "shape") else v2) for k2, v2 in snap.items()}, cfg.prefill)   # partial
    b.load_state(snap, cfg.prefill)
    assert (b.info().t, b.info().n) == (173, snap["n"])
    with pytest.raises(binding.LazyEvError):
        b.load_state(snap, cfg.prefill)                                  # already holds a cache
    for _ in range(3):
        q, kn, vn = gen.steps(32)
        for s in range(32):
            a.decode_step(q[s], kn[s], vn[s], out_a)
            b.decode_step(q[s], kn[s], vn[s], out_b)
            assert torch.equal(out_a, out_b)
    da, db = a.dump_state(kv=True), b.dump_state(kv=True)
    assert a.info().evictions == b.info().evictions + 3 and da["n"] == db["n"]
    for key in ("pos", "ts", "mri", "pbar", "k", "v"):
        assert np.array_equal(da[key], db[key]), key


def test_call_order_errors_and_capacity():
    cfg = traces.tiny_config(batch=1, layers=1)
    eng = binding.Engine(1, 8, 2, 128, 160, 32, 0.01, max_prefill=96)
    x = torch.zeros(1, 1, 8, 128, dtype=torch.bfloat16, device="cuda")
    kv = torch.zeros(1, 1, 2, 128, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(binding.LazyEvError) as e:
        eng.decode_step(x, kv, kv, x)
    assert e.value.code == binding.ESTATE
    with pytest.raises(binding.LazyEvError) as e:
        eng.prefill(torch.zeros(1, 1, 2, 97, 128, dtype=torch.bfloat16, device="cuda"),
                    torch.zeros(1, 1, 2, 97, 128, dtype=torch.bfloat16, device="cuda"))
    assert e.value.code == binding.ECAPACITY
    p = torch.zeros(1, 1, 2, 96, 128, dtype=torch.bfloat16, device="cuda")
    eng.prefill(p, p)
    with pytest.raises(binding.LazyEvError) as e:
        eng.prefill(p, p)
    assert e.value.code == binding.ESTATE
    eng.set_auto_evict(False)
    cap = eng.info().capacity
    for _ in range(cap - 96):
        eng.decode_step(x, kv, kv, x)
    with pytest.raises(binding.LazyEvError) as e:
        eng.decode_step(x, kv, kv, x)                    # eviction disabled and never called
    assert e.value.code == binding.ECAPACITY
    eng.synchronize()
    assert eng.dump_state()["device_status"] == 0


def test_eviction_over_too_many_candidates_is_refused():
    """More than 25 600 unprotected tokens per unit: lazyev_evict says so and leaves the cache alone."""
    eng = binding.Engine(1, 2, 1, 128, 25700, 64, 0.5, max_prefill=25700)
    z = torch.zeros(1, 1, 1, 25700, 128, dtype=torch.bfloat16, device="cuda")
    eng.prefill(z, z)
    eng.set_auto_evict(False)
    x = torch.zeros(1, 1, 2, 128, dtype=torch.bfloat16, device="cuda")
    kv = torch.zeros(1, 1, 1, 128, dtype=torch.bfloat16, device="cuda")
    for _ in range(64):
        eng.decode_step(x, kv, kv, x)
    with pytest.raises(binding.LazyEvError) as e:
        eng.evict()
    assert e.value.code == binding.EINVAL and "candidates" in str(e.value)
    eng.synchronize()
    assert eng.info().n == 25764 and eng.dump_state()["device_status"] == 0


def test_step_whose_automatic_eviction_cannot_run_is_refused_up_front():
    """Automatic eviction on (the default) and a prompt beyond the selection's candidate limit: the decode
    step at the first decision point returns EINVAL before anything is queued -- t and n do not move,
    so the caller can retry -- instead of completing the step and then failing in the eviction."""
    eng = binding.Engine(1, 2, 1, 128, 25700, 64, 0.5, max_prefill=25800)
    z = torch.zeros(1, 1, 1, 25800, 128, dtype=torch.bfloat16, device="cuda")
    eng.prefill(z, z)                                        # 25800 > budget: the step at t = 64 must evict
    x = torch.zeros(1, 1, 2, 128, dtype=torch.bfloat16, device="cuda")
    kv = torch.zeros(1, 1, 1, 128, dtype=torch.bfloat16, device="cuda")
    for _ in range(63):
        eng.decode_step(x, kv, kv, x)
    for _ in range(2):                                       # refused twice: nothing changed in between
        with pytest.raises(binding.LazyEvError) as e:
            eng.decode_step(x, kv, kv, x)
        assert e.value.code == binding.EINVAL and "candidates" in str(e.value)
        assert (eng.info().t, eng.info().n) == (63, 25863)
    eng.set_auto_evict(False)                                # the caller's way out: step without evicting
    eng.decode_step(x, kv, kv, x)
    assert (eng.info().t, eng.info().n) == (64, 25864)
    eng.synchronize()
    assert eng.counters().device_status == 0


def test_a_bounded_wait_that_runs_out_is_reported_and_the_handle_recovers():
    """The decode kernel's waits are bounded: a block whose page ring is starved (a diagnostic switch
    makes the producer warp stop after two pages) gives up after the wait limit, the kernel ends by
    itself, the status word says so, and after lazyev_reset the handle serves a new sequence with the
    results of a fresh handle.  Nothing faults and the CUDA context stays usable throughout."""
    from tests.harness import make_engine
    cfg = traces.tiny_config(batch=1, layers=1, prefill=300, budget=400)          # 2 units, 5 pages each
    shape = (cfg.layers, cfg.batch, cfg.kv_heads, cfg.prefill, 128)
    used, fresh = make_engine(cfg), make_engine(cfg)
    used.set_splits(1); fresh.set_splits(1)
    used.set_wait_limit(0.004)
    out_u = torch.empty(cfg.layers, cfg.batch, cfg.q_heads, 128, dtype=torch.bfloat16, device="cuda")
    out_f = torch.empty_like(out_u)
    gen = traces.TraceGen(cfg, 40, device="cuda")
    k, v = gen.prefill()
    used.prefill(k.view(shape), v.view(shape))
    q, kn, vn = gen.steps(4)
    used.decode_step(q[0], kn[0], vn[0], out_u)
    used.synchronize()                                        # a healthy step first
    used.debug_starve_page_ring(2)
    used.decode_step(q[1], kn[1], vn[1], out_u)               # queued; the kernel gives up after ~4 ms
    with pytest.raises(binding.LazyEvError) as e:
        used.synchronize()
    assert e.value.code == binding.EDEVICE
    assert used.counters().device_status & 1                  # "a bounded wait gave up"
    torch.cuda.synchronize()                                  # the context is alive
    used.debug_starve_page_ring(-1)
    used.reset()
    assert used.counters().device_status == 0
    gen2 = traces.TraceGen(cfg, 41, device="cuda")
    k, v = gen2.prefill()
    used.prefill(k.view(shape), v.view(shape)); fresh.prefill(k.view(shape), v.view(shape))
    for _ in range(4):                                        # 128 steps with evictions
        q, kn, vn = gen2.steps(32)
        for s in range(32):
            used.decode_step(q[s], kn[s], vn[s], out_u)
            fresh.decode_step(q[s], kn[s], vn[s], out_f)
            assert torch.equal(out_u, out_f)
    du, df = used.dump_state(kv=True), fresh.dump_state(kv=True)
    for key in ("pos", "ts", "mri", "pbar", "k", "v"):
        assert np.array_equal(du[key], df[key]), key
    assert du["device_status"] == 0 and used.info().evictions == fresh.info().evictions + 0


def test_a_bounded_wait_that_runs_out_in_the_prompt_kernel_is_reported_and_the_handle_recovers():
    """The same for the tiled prompt kernel: its producer thread stops after two key tiles (the
    diagnostic switch), the thread that issues the tensor-core products and the softmax warps wait for
    a tile that never comes, give up after the wait limit, and the kernel ends by itself with the
    status word set.  After lazyev_reset the handle observes a prompt with the results of a fresh one."""
    from tests.harness import make_engine
    cfg = traces.tiny_config(batch=1, layers=1, prefill=300, budget=400)          # 2 units, 19 query tiles each
    shape = (cfg.layers, cfg.batch, cfg.kv_heads, cfg.prefill, 128)
    used, fresh = make_engine(cfg), make_engine(cfg)
    used.set_wait_limit(0.004)
    gen = traces.TraceGen(cfg, 42, device="cuda")
    k, v = gen.prefill()
    g = torch.Generator().manual_seed(6)
    q = torch.randn(cfg.prefill, cfg.units, cfg.group, 128, generator=g).to(torch.bfloat16).cuda()
    out_u = torch.zeros(cfg.prefill, cfg.units, cfg.group, 128, dtype=torch.bfloat16, device="cuda")
    out_f = torch.zeros_like(out_u)
    used.debug_starve_page_ring(2)
    used.prefill_observed(q, k.view(shape), v.view(shape), out_u)      # queued; the kernel gives up after ~4 ms
    with pytest.raises(binding.LazyEvError) as e:
        used.synchronize()
    assert e.value.code == binding.EDEVICE
    assert used.counters().device_status & 1                  # "a bounded wait gave up"
    torch.cuda.synchronize()                                  # the context is alive
    used.debug_starve_page_ring(-1)
    used.reset()
    assert used.counters().device_status == 0
    used.prefill_observed(q, k.view(shape), v.view(shape), out_u)
    fresh.prefill_observed(q, k.view(shape), v.view(shape), out_f)
    used.synchronize(); fresh.synchronize()
    assert torch.equal(out_u, out_f)
    du, df = used.dump_state(kv=True), fresh.dump_state(kv=True)
    for key in ("pos", "ts", "mri", "pbar", "k", "v"):
        assert np.array_equal(du[key], df[key]), key
    assert du["device_status"] == 0


@pytest.mark.parametrize("splits", [0, 1, 3])
def test_append_inside_the_decode_launch_matches_the_separate_launch(splits):
    """Small problems write the new token inside the decode launch (one launch less per step); with the
    switch off the append is a launch of its own.  Same outputs, state and cache, bit for bit, across a
    page boundary and two evictions; and one launch per step less."""
    from tests.harness import make_engine
    cfg = traces.tiny_config(prefill=100)
    gen = traces.TraceGen(cfg, 27, device="cuda")
    fused, plain = make_engine(cfg), make_engine(cfg)
    plain.set_fused_append(False)
    for e in (fused, plain):
        e.set_splits(splits)
    k, v = gen.prefill()
    shape = (cfg.layers, cfg.batch, cfg.kv_heads, cfg.prefill, 128)
    fused.prefill(k.view(shape), v.view(shape)); plain.prefill(k.view(shape), v.view(shape))
    out_f = torch.empty(cfg.layers, cfg.batch, cfg.q_heads, 128, dtype=torch.bfloat16, device="cuda")
    out_p = torch.empty_like(out_f)
    l0 = (fused.info().launches, plain.info().launches)
    for _ in range(4):
        q, kn, vn = gen.steps(32)
        for s in range(32):
            fused.decode_step(q[s], kn[s], vn[s], out_f)
            plain.decode_step(q[s], kn[s], vn[s], out_p)
            assert torch.equal(out_f, out_p)
    df, dp = fused.dump_state(kv=True), plain.dump_state(kv=True)
    for key in ("pos", "ts", "mri", "pbar", "k", "v"):
        assert np.array_equal(df[key], dp[key]), key
    assert df["device_status"] == 0 and fused.info().evictions == plain.info().evictions == 3
    assert (plain.info().launches - l0[1]) - (fused.info().launches - l0[0]) == 128


def test_library_flavour_is_the_one_the_environment_asks_for():
    assert bool(binding.lib().lazyev_build_flags() & 1) == binding.debug_bounds_requested()


def test_range_checked_build_runs_the_lockstep_tests_clean():
    """The sanitizer substitute: the same sources compiled with every slot, page-table and work-list
    index range-checked (a failed check flags the device status word).  The lock-step tests, the
    random-shape sweep and the prompt tests run again through that build in a child process; they
    assert a clean status word themselves."""
    import os, subprocess, sys
    if binding.debug_bounds_requested():
        pytest.skip("already inside the range-checked run")
    env = dict(os.environ, LAZYEV_DEBUG_BOUNDS="1")
    here = os.path.dirname(os.path.abspath(__file__))
    sel = ("lockstep_with_evictions or random_shapes or many_units or group_sizes or observed_prompt or append_inside or "
           "partly_filled or protected_tokens or dynamic_budget or window_of_one or library_flavour or "
           "long_contexts or histogram")
    res = subprocess.run([sys.executable, "-m", "pytest", os.path.join(here, "test_gpu_parity.py"),
                          os.path.join(here, "test_zz_no_alloc.py"), "-q", "-x", "-m", "gpu", "-k",
                          sel + " or static_scratch"], env=env, capture_output=True, text=True, cwd=os.path.dirname(here))
    assert res.returncode == 0, res.stdout[-3000:] + res.stderr[-2000:]
    assert " passed" in res.stdout and "failed" not in res.stdout


def test_host_buffer_entry_point_matches_device_entry_point():
    cfg = traces.tiny_config()
    gen = traces.TraceGen(cfg, 8, device="cuda")
    from tests.harness import make_engine
    a, b = make_engine(cfg), make_engine(cfg)
    k, v = gen.prefill()
    shape = (cfg.layers, cfg.batch, cfg.kv_heads, cfg.prefill, 128)
    a.prefill(k.view(shape), v.view(shape)); b.prefill(k.view(shape), v.view(shape))
    out_a = torch.empty(cfg.layers, cfg.batch, cfg.q_heads, 128, dtype=torch.bfloat16, device="cuda")
    out_b = torch.empty(out_a.shape, dtype=torch.bfloat16).pin_memory()
    for _ in range(4):
        q, kn, vn = gen.steps(32)
        qh, kh, vh = q.cpu().pin_memory(), kn.cpu().pin_memory(), vn.cpu().pin_memory()
        for s in range(32):
            a.decode_step(q[s], kn[s], vn[s], out_a)
            b.decode_step_host(qh[s], kh[s], vh[s], out_b)
            assert torch.equal(out_a.cpu(), out_b)
    da, db = a.dump_state(), b.dump_state()
    assert a.info().evictions == 2 and b.info().evictions == 2          # automatic eviction ran
    for key in ("pos", "ts", "mri", "pbar"):
        assert np.array_equal(da[key], db[key])


def test_host_buffer_pipeline_of_unit_ranges_matches_the_resident_step():
    """1792 units: 12 full rounds of the persistent grid (split by the host-buffer entry point into
    three unit ranges with overlapped copies) and a partly filled last round that goes to the second
    launch.  The synchronous host call, the asynchronous host call and the resident call run side by
    side through four evictions; outputs and all state must be identical bit for bit."""
    from tests.harness import make_engine
    cfg = traces.tiny_config(batch=32, layers=14, q_heads=28, kv_heads=4, prefill=1500, budget=1520, window=32,
                             n_recent=32)
    assert cfg.units == 1792                                 # 24 pages per unit: long enough for the second launch to pay
    gen = traces.TraceGen(cfg, 18, device="cuda")
    res, host, asy = make_engine(cfg), make_engine(cfg), make_engine(cfg)
    k, v = gen.prefill()
    shape = (cfg.layers, cfg.batch, cfg.kv_heads, cfg.prefill, 128)
    res.prefill(k.view(shape), v.view(shape))
    host.copy_state_from(res)                                # the fork entry point, checked by what follows
    asy.copy_state_from(res)
    oshape = (cfg.layers, cfg.batch, cfg.q_heads, 128)
    out_r = torch.empty(oshape, dtype=torch.bfloat16, device="cuda")
    out_h = torch.empty(oshape, dtype=torch.bfloat16).pin_memory()
    out_a = [torch.empty(oshape, dtype=torch.bfloat16).pin_memory() for _ in range(2)]
    expect = [None, None]
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    for chunk in range(4):                                   # 128 steps: an eviction every 32
        q, kn, vn = gen.steps(32)
        qh, kh, vh = q.cpu().pin_memory(), kn.cpu().pin_memory(), vn.cpu().pin_memory()
        for s in range(32):
            res.decode_step(q[s], kn[s], vn[s], out_r)
            host.decode_step_host(qh[s], kh[s], vh[s], out_h)
            ref = out_r.cpu()
            assert torch.equal(ref, out_h), f"synchronous host step differs at chunk {chunk} step {s}"
            i = (chunk * 32 + s) & 1
            asy.decode_step_host_async(qh[s], kh[s], vh[s], out_a[i])
            asy.host_wait(1)                                 # everything but the step just queued is complete
            if expect[i ^ 1] is not None:
                assert torch.equal(expect[i ^ 1], out_a[i ^ 1]), f"asynchronous host step differs before chunk {chunk} step {s}"
            expect[i] = ref
        asy.host_wait(0)
        assert torch.equal(expect[1], out_a[1])
        inf = host.info()
        if sms == 148:
            assert inf.host_ranges == 4 and inf.tail_units == 16      # three ranges of whole rounds + the last round's units
        else:
            assert inf.host_ranges >= 2
    dr = res.dump_state(kv=True)
    assert res.info().evictions == 4 and dr["n"] == cfg.budget
    for other in (host, asy):
        assert other.info().evictions == 4
        do = other.dump_state(kv=True)
        for key in ("pos", "ts", "mri", "pbar", "k", "v"):
            assert np.array_equal(dr[key], do[key]), key
        assert do["device_status"] == 0
