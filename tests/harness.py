"""Lock-step comparison of the CUDA library with the fp64 oracle on one trace.

For every sampled unit two oracles run beside the GPU engine:
* the SHADOW oracle attends with its own arithmetic (its outputs and
  probabilities are compared with the GPU's within the floating-point
  tolerances), but its bookkeeping consumes the probabilities the GPU wrote;
  from there on TS, MRI, positions and evict sets must match bit for bit, so
  its cache always holds exactly what the GPU kept;
* the PURE oracle never sees anything from the GPU; at the end the kept sets
  are compared by Jaccard index.
"""
from __future__ import annotations

import dataclasses

import numpy as np
import torch

from oracle import lazyev_oracle as orc
from paper_2506_15969_b200 import binding, traces

OUT_RTOL, OUT_ATOL = 1e-2, 2e-3      # attention output: |gpu - ref| <= atol + rtol * |ref|
PBAR_ATOL = 1e-4                     # probabilities
SCORE_ATOL = 1e-13                   # fp64 scores (exp() may differ in the last place)
TIE_GAP = 1e-12                      # below this gap the evict boundary is not unique


@dataclasses.dataclass
class Report:
    steps: int = 0
    evictions: int = 0
    max_out_err: float = 0.0         # max of |gpu - ref| / (atol + rtol |ref|), must stay <= 1
    max_pbar_err: float = 0.0
    max_score_err: float = 0.0
    near_tie_events: int = 0
    min_jaccard: float = 1.0
    activations: int = 0
    tokens_seen: int = 0
    threshold_flips: int = 0         # (step, token) pairs where fp64 and GPU probabilities fall on different sides of alpha
    max_kept_diff: int = 0           # most positions by which a unit's kept set differs from the pure oracle's


def f64(x: torch.Tensor) -> np.ndarray:
    return x.detach().to("cpu", torch.float64).numpy()


def make_engine(cfg: traces.TraceConfig, **kw) -> binding.Engine:
    return binding.Engine(cfg.layers, cfg.q_heads, cfg.kv_heads, cfg.head_dim, cfg.budget, cfg.window,
                          cfg.threshold, batch=cfg.batch, n_recent=cfg.n_recent, n_initial=cfg.n_initial,
                          max_prefill=cfg.prefill, **kw)


def make_oracle(cfg: traces.TraceConfig, score_mode="h1+h2") -> orc.OracleUnit:
    return orc.OracleUnit(cfg.group, cfg.head_dim, cfg.budget, cfg.window, cfg.threshold,
                          n_recent=cfg.n_recent, n_initial=cfg.n_initial, score_mode=score_mode)


class Lockstep:
    def __init__(self, cfg: traces.TraceConfig, seed: int, sample_units, splits: int = 0, stages: int = 0,
                 score_mode: int = 0, page_table=None, pure: bool = True, check_inputs: bool = True,
                 groups: int = 0, observed: bool = False, gen_device: str = "cuda", pure_units=None,
                 prompt_mode: int = 0):
        """`gen_device`: where the trace of all units is generated ("cpu": generated on the host and
        uploaded, so that the library's kernels are the only ones launched).  `pure_units`: the sampled
        units that also get a pure-oracle run (default: all of them, when `pure`)."""
        self.cfg, self.sample = cfg, list(sample_units)
        self.eng = make_engine(cfg)
        self.eng.set_auto_evict(False)
        if splits:
            self.eng.set_splits(splits)
        if stages:
            self.eng.set_stages(stages)
        if groups:
            self.eng.set_groups(groups)
        if score_mode:
            self.eng.set_score_mode(score_mode)
        if page_table is not None:
            self.eng.set_page_table(page_table)
        if prompt_mode:
            self.eng.set_prompt_mode(prompt_mode)
        mode = orc.SCORE_MODES[score_mode]
        self.gen_gpu = traces.TraceGen(cfg, seed, device=gen_device)
        self.gen_cpu = traces.TraceGen(cfg, seed, device="cpu", units=self.sample)
        self.check_inputs = check_inputs
        self.shadow = [make_oracle(cfg, mode) for _ in self.sample]
        self.pure = None
        if pure:
            on = set(self.sample if pure_units is None else pure_units)
            self.pure = [make_oracle(cfg, mode) if u in on else None for u in self.sample]
        self.rep = Report()
        L, Bt = cfg.layers, cfg.batch
        self.out = torch.empty(L, Bt, cfg.q_heads, cfg.head_dim, dtype=torch.bfloat16, device="cuda")
        k, v = (x.cuda() for x in self.gen_gpu.prefill())
        kc, vc = self.gen_cpu.prefill()
        if check_inputs:
            assert torch.equal(k[self.sample].cpu(), kc) and torch.equal(v[self.sample].cpu(), vc)
        kk = k.view(L, Bt, cfg.kv_heads, cfg.prefill, cfg.head_dim)
        vv = v.view(L, Bt, cfg.kv_heads, cfg.prefill, cfg.head_dim)
        if not observed:
            self.eng.prefill(kk, vv)
            for i in range(len(self.sample)):
                self.shadow[i].prefill(f64(kc[i]), f64(vc[i]))
                if self.pure and self.pure[i]:
                    self.pure[i].prefill(f64(kc[i]), f64(vc[i]))
        else:
            self._observed_prefill(kk, vv, kc, vc, seed)
        self.t = 0

    def _observed_prefill(self, kk, vv, kc, vc, seed):
        """Prompt load with tracking: seeded prompt queries, some rows re-aligned with earlier keys so
        that prompt tokens are re-activated.  The library also dumps the probabilities of every prompt
        row for the sampled units; the shadow oracle's tracking consumes them (as it does in the decode
        steps), so TS and MRI of every prompt token must match bit for bit, while outputs and
        probabilities are compared with the oracle's own within the tolerances."""
        cfg, P = self.cfg, self.cfg.prefill
        g = torch.Generator().manual_seed(1000 + seed)
        q = torch.randn(P, cfg.units, cfg.group, cfg.head_dim, generator=g)
        kf = kk.reshape(cfg.units, P, cfg.head_dim).float().cpu()
        rows = torch.randint(1, P, (cfg.units, P // 6), generator=g)
        for u in range(cfg.units):
            for j in rows[u].tolist():
                i = int(torch.randint(0, j, (1,), generator=g))
                q[j, u] += 4.0 * (cfg.head_dim ** 0.5) * kf[u, i] / kf[u, i].pow(2).sum()
        q = q.to(torch.bfloat16)
        out = torch.empty(P, cfg.units, cfg.group, cfg.head_dim, dtype=torch.bfloat16, device="cuda")
        u0, u1 = min(self.sample), max(self.sample) + 1
        rows_gpu = torch.zeros(u1 - u0, P, P, dtype=torch.float32, device="cuda")
        self.eng.set_prompt_dump(rows_gpu, u0, u1 - u0)
        self.eng.prefill_observed(q.cuda(), kk, vv, out)
        self.eng.set_prompt_dump(None)
        rows_gpu = rows_gpu.cpu().numpy()
        rep = self.rep
        a32 = np.float32(cfg.threshold)
        for i, u in enumerate(self.sample):
            sh = self.shadow[i]
            ref = sh.prefill_observed(f64(q[:, u]), f64(kc[i]), f64(vc[i]), pbar_rows=rows_gpu[u - u0])
            if self.pure and self.pure[i]:
                self.pure[i].prefill_observed(f64(q[:, u]), f64(kc[i]), f64(vc[i]))
            got = f64(out[:, u])
            rep.max_out_err = max(rep.max_out_err, float((np.abs(got - ref) / (OUT_ATOL + OUT_RTOL * np.abs(ref))).max()))
            for j in range(P):
                mine, theirs = sh.prompt_pbar[j], rows_gpu[u - u0, j, : j + 1]
                rep.max_pbar_err = max(rep.max_pbar_err, float(np.abs(theirs - mine).max()))
                rep.threshold_flips += int(((mine.astype(np.float32) >= a32) != (theirs >= a32)).sum())
            d = self._dump(u)
            assert d["n"] == P and d["t"] == 0
            assert np.array_equal(d["pbar"][0], rows_gpu[u - u0, P - 1]), "stored probabilities are not the last row's"
            assert np.array_equal(d["ts"][0], sh.TS), f"prompt TS mismatch unit {u}"
            assert np.array_equal(d["mri"][0], sh.MRI), f"prompt MRI mismatch unit {u}"
            assert np.array_equal(d["pos"][0], sh.pos)
            rep.activations += int((sh.MRI > 0).sum())

    def _dump(self, u, **kw):
        return self.eng.dump_state(u, 1, **kw)

    def run(self, steps: int, check_every: int = 1) -> Report:
        cfg, rep = self.cfg, self.rep
        done = 0
        while done < steps:
            cnt = min(traces.TraceGen.CHUNK, steps - done)
            q, kn, vn = (x.cuda() for x in self.gen_gpu.steps(cnt))
            qc, knc, vnc = self.gen_cpu.steps(cnt)
            if self.check_inputs:
                assert torch.equal(q[:, self.sample].cpu(), qc)
            for s in range(cnt):
                self.t += 1
                t = self.t
                self.eng.decode_step(q[s], kn[s], vn[s], self.out)
                # Attention is compared on the check steps; on the others the shadow oracle only appends
                # the token.  Tracking consumes the GPU's probabilities at every step either way.
                check = (t % check_every == 0) or (t % cfg.window == 0)
                out_gpu = f64(self.out.cpu().view(cfg.units, cfg.group, cfg.head_dim)[self.sample]) if check else None
                if cfg.budget_frac_tenths and t % cfg.window == 0:
                    self.eng.set_budget(cfg.budget_at(t))
                for i, u in enumerate(self.sample):
                    sh = self.shadow[i]
                    qi, ki, vi = f64(qc[s, i]), f64(knc[s, i]), f64(vnc[s, i])
                    d = self._dump(u)
                    if check:
                        ref_out, ref_pbar = sh.attend(qi, ki, vi)
                    else:
                        sh.append(ki, vi)
                    assert d["n"] == sh.n and d["t"] == t
                    if check:
                        err = np.abs(out_gpu[i] - ref_out) / (OUT_ATOL + OUT_RTOL * np.abs(ref_out))
                        rep.max_out_err = max(rep.max_out_err, float(err.max()))
                        rep.max_pbar_err = max(rep.max_pbar_err, float(np.abs(d["pbar"][0] - ref_pbar).max()))
                        a32 = np.float32(cfg.threshold)
                        rep.threshold_flips += int(((ref_pbar.astype(np.float32) >= a32) != (d["pbar"][0] >= a32)).sum())
                    act = sh.track(d["pbar"][0])
                    rep.activations += int(act.sum()); rep.tokens_seen += sh.n
                    assert np.array_equal(d["ts"][0], sh.TS), f"TS mismatch unit {u} step {t}"
                    assert np.array_equal(d["mri"][0], sh.MRI), f"MRI mismatch unit {u} step {t}"
                    assert np.array_equal(d["pos"][0], sh.pos), f"pos mismatch unit {u} step {t}"
                    if cfg.budget_frac_tenths and t % cfg.window == 0:
                        sh.set_budget(cfg.budget_at(t))
                        if self.pure and self.pure[i]:
                            self.pure[i].set_budget(cfg.budget_at(t))
                    if sh.evict_due():
                        ds = self._dump(u, score=True)
                        rep.max_score_err = max(rep.max_score_err,
                                                float(np.abs(ds["score"][0] - sh.scores()).max()))
                    if self.pure and self.pure[i]:
                        self.pure[i].step(qi, ki, vi)
                removed = self.eng.evict()
                if removed:
                    rep.evictions += 1
                for i, u in enumerate(self.sample):
                    sh = self.shadow[i]
                    assert sh.evict_due() == (removed > 0)
                    if not removed:
                        continue
                    kept, info = sh.select_keep()
                    assert info["n_before"] - len(kept) == removed
                    d = self._dump(u, kv=True)
                    if np.array_equal(d["pos"][0], sh.pos[kept]):
                        sh.apply_keep(kept)
                    else:
                        # only acceptable when the k-th and (k+1)-th scores are equal up to exp() rounding
                        assert info["kept_min"] - info["evicted_max"] < TIE_GAP, \
                            f"evict set mismatch unit {u} step {t}"
                        rep.near_tie_events += 1
                        sh.force_keep_positions(d["pos"][0])
                    assert np.array_equal(d["ts"][0], sh.TS) and np.array_equal(d["mri"][0], sh.MRI)
                    assert np.array_equal(orc.bf16_bits_to_f64(d["k"][0]), sh.K), "K rows moved wrongly"
                    assert np.array_equal(orc.bf16_bits_to_f64(d["v"][0]), sh.V), "V rows moved wrongly"
                rep.steps += 1
            done += cnt
        self.eng.synchronize()
        if self.pure:
            for i, u in enumerate(self.sample):
                if self.pure[i] is None:
                    continue
                a, b = set(self.shadow[i].pos.tolist()), set(self.pure[i].pos.tolist())
                rep.min_jaccard = min(rep.min_jaccard, len(a & b) / len(a | b))
                rep.max_kept_diff = max(rep.max_kept_diff, len(a - b))
        return rep

    def assert_ok(self, jaccard: float = 0.999):
        """The bars of the three comparison modes.  The kept-set bar against the pure oracle is a
        Jaccard index of 0.999.  In a cache of a few hundred tokens a single differing token already
        costs more than that, and a single token can legitimately differ: when a probability lies
        within float32 rounding of the threshold, the GPU's value and the oracle's fall on different
        sides of it, the token's TS / MRI then differ, and so may its rank.  Such cases are counted
        (threshold_flips, on the steps where attention is compared); below the Jaccard bar the test
        passes only if the kept sets differ by no more positions than there were such flips."""
        rep = self.rep
        assert rep.max_out_err <= 1.0, f"attention output outside tolerance ({rep.max_out_err:.3f} x)"
        assert rep.max_pbar_err <= PBAR_ATOL, f"probability error {rep.max_pbar_err:.2e}"
        assert rep.max_score_err <= SCORE_ATOL, f"score error {rep.max_score_err:.2e}"
        if self.pure and rep.min_jaccard < jaccard:
            assert rep.max_kept_diff <= rep.threshold_flips, \
                f"kept-set Jaccard {rep.min_jaccard:.5f}: {rep.max_kept_diff} positions differ, {rep.threshold_flips} threshold flips"
