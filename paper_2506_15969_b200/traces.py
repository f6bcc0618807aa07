"""Seeded synthetic decode traces (inputs only; none of the method's arithmetic).

The paper measures on reasoning benchmarks with real models; neither is
available offline, so these traces stand in for them: bf16 Q/K/V with the
shapes of the five benchmark configurations, queries with temporal locality,
and "planted" recurring tokens -- cached keys that the queries re-align with
periodically -- so that attention shows the token-importance-recurrence
pattern the method tracks (Section 3 of the paper).

Everything is a pure function of (seed, unit, position / step, dimension)
computed with 64-bit integer arithmetic in torch, so the same code gives the
same bits on a CPU tensor and on a CUDA tensor, for all units or for any
subset of them.  The trace is open loop: inputs never depend on what any
implementation keeps in its cache.

Recipe, per unit u = (layer, batch, kv_head):
* keys / values of the token at position p: Irwin-Hall(12) sums of 16-bit
  hash fields, scaled by 2^-16 (zero mean, unit variance), rounded to bf16.
* queries: "iid" -- fresh draws every step; "ar1" -- per query head and
  dimension an integer AR(1) walk s_t = floor(973 s_{t-1} / 1024) +
  floor(319 z_t / 1024) (rho = 0.95, stationary variance 1).
* planted recurring tokens: a token with period T and phase phi born at step b
  "fires" at steps b + 1 + phi + m T.  When token j fires, every query head of
  its group gets q += beta_j k_j with beta_j = 4 sqrt(D) / |k_j|^2, i.e. +4 on
  that token's scaled logit.
* one-shot spikes (configs 4, 5): each step, with probability 1/2 per unit,
  one uniformly drawn earlier position gets the same +4 once.
"""
from __future__ import annotations

import dataclasses
import math
from typing import Optional, Tuple

import torch

_M64 = (1 << 64) - 1


def _s64(x: int) -> int:
    x &= _M64
    return x - (1 << 64) if x >= (1 << 63) else x


_C_ADD = _s64(0x9E3779B97F4A7C15)
_C_M1 = _s64(0xBF58476D1CE4E5B9)
_C_M2 = _s64(0x94D049BB133111EB)
_C_D = _s64(0xD6E8FEB86659FD93)
_C_J = _s64(0xA0761D6478BD642F)

# hash streams
_ST_K, _ST_V, _ST_Q, _ST_PLANT, _ST_PERIOD, _ST_PHASE, _ST_SPIKE, _ST_SPIKEPOS = range(1, 9)


def _lsr(x: torch.Tensor, s: int) -> torch.Tensor:
    """Logical right shift of an int64 tensor."""
    return (x >> s) & ((1 << (64 - s)) - 1)


def _mix(x: torch.Tensor) -> torch.Tensor:
    """A 64-bit finaliser (xor-shift / multiply rounds), wrapping arithmetic."""
    x = x + _C_ADD
    x = (x ^ _lsr(x, 30)) * _C_M1
    x = (x ^ _lsr(x, 27)) * _C_M2
    return x ^ _lsr(x, 31)


def mix_python(x: int) -> int:
    """The same finaliser on Python integers (used by the tests)."""
    x = (x + 0x9E3779B97F4A7C15) & _M64
    x = ((x ^ (x >> 30)) * 0xBF58476D1CE4E5B9) & _M64
    x = ((x ^ (x >> 27)) * 0x94D049BB133111EB) & _M64
    return x ^ (x >> 31)


@dataclasses.dataclass(frozen=True)
class TraceConfig:
    name: str
    batch: int
    layers: int
    q_heads: int
    kv_heads: int
    prefill: int
    steps: int
    budget: int
    window: int
    n_recent: int
    head_dim: int = 128
    n_initial: int = 0
    budget_frac_tenths: int = 0          # > 0: budget_t = min(budget, tenths*(P+t)//10)
    query: str = "ar1"                   # "iid" | "ar1"
    plant_mode: str = "prob"             # "prob" | "count_prefill"
    plant_count: int = 0
    plant_prob_1024: int = 0             # planted with probability x/1024
    period_mode: str = "uniform"         # "uniform" | "octave" (piecewise log-uniform)
    period_lo: int = 100
    period_hi: int = 1000
    spike_prob_1024: int = 0
    alpha: float = 0.0                   # 0: use the default 8 / (budget + window)

    @property
    def group(self) -> int:
        return self.q_heads // self.kv_heads

    @property
    def units(self) -> int:
        return self.batch * self.layers * self.kv_heads

    @property
    def threshold(self) -> float:
        return self.alpha if self.alpha > 0 else 8.0 / (self.budget + self.window)

    def budget_at(self, t: int) -> int:
        """Budget in force at decode step t (fixed, or a fraction of the length)."""
        if self.budget_frac_tenths <= 0:
            return self.budget
        return max(self.n_recent + self.n_initial + 1,
                   min(self.budget, (self.budget_frac_tenths * (self.prefill + t)) // 10))

    def capacity(self) -> int:
        return max(self.budget, self.prefill) + self.window


CONFIGS = {
    1: TraceConfig("cfg1-b1-l1-8q2kv", batch=1, layers=1, q_heads=8, kv_heads=2, prefill=256, steps=1024,
                   budget=512, window=128, n_recent=16, query="iid", plant_mode="count_prefill",
                   plant_count=32, period_mode="uniform", period_lo=50, period_hi=300),
    2: TraceConfig("cfg2-b4-l4-28q4kv", batch=4, layers=4, q_heads=28, kv_heads=4, prefill=512, steps=4096,
                   budget=2048, window=128, n_recent=128, plant_prob_1024=51,
                   period_mode="uniform", period_lo=100, period_hi=1000),
    3: TraceConfig("cfg3-b16-l32-32q8kv", batch=16, layers=32, q_heads=32, kv_heads=8, prefill=1024, steps=8192,
                   budget=4096, window=256, n_recent=256, budget_frac_tenths=3, plant_prob_1024=51,
                   period_mode="uniform", period_lo=100, period_hi=1000),
    4: TraceConfig("cfg4-b32-l28-28q4kv", batch=32, layers=28, q_heads=28, kv_heads=4, prefill=256, steps=16384,
                   budget=8192, window=128, n_recent=128, plant_prob_1024=102,
                   period_mode="octave", period_lo=64, period_hi=4096, spike_prob_1024=512),
    5: TraceConfig("cfg5-b32-l48-40q8kv", batch=32, layers=48, q_heads=40, kv_heads=8, prefill=512, steps=16384,
                   budget=4915, window=256, n_recent=32, plant_prob_1024=102,
                   period_mode="octave", period_lo=64, period_hi=4096, spike_prob_1024=512),
}


def tiny_config(**kw) -> TraceConfig:
    """A small configuration for tests; keyword arguments override the defaults."""
    base = dict(name="tiny", batch=2, layers=2, q_heads=8, kv_heads=2, prefill=96, steps=400, budget=160,
                window=32, n_recent=32, plant_prob_1024=102, period_mode="uniform", period_lo=40,
                period_hi=160, spike_prob_1024=256)
    base.update(kw)
    return TraceConfig(**base)


class TraceGen:
    """Generator of one configuration's inputs for all units or a subset.

    `units`: 1-D sequence of unit ids (default: all).  Tensors are returned in
    unit-major layout: prefill K/V [U, P, D]; steps q [n, U, G, D] and
    k_new / v_new [n, U, D], all bf16.  With all units selected, [U, ...]
    reshapes to the library's [layers, batch, kv_heads, ...] layout, and
    [U, G, D] to [layers, batch, q_heads, D].
    """

    CHUNK = 32      # steps per firing scan; must not exceed the shortest period

    def __init__(self, cfg: TraceConfig, seed: int = 0, device="cpu", units=None):
        assert cfg.period_lo >= self.CHUNK
        self.cfg, self.seed, self.device = cfg, int(seed), torch.device(device)
        ids = torch.arange(cfg.units) if units is None else torch.as_tensor(list(units))
        self.units = ids.to(device=self.device, dtype=torch.int64)
        self.U, self.G, self.D = int(self.units.numel()), cfg.group, cfg.head_dim
        self._d = torch.arange(self.D, device=self.device, dtype=torch.int64)
        self._heads = (self.units[:, None] * self.G
                       + torch.arange(self.G, device=self.device, dtype=torch.int64)[None, :])   # [U, G]
        self._beta_num = 4.0 * math.sqrt(self.D) * float(1 << 32)
        self._state: Optional[torch.Tensor] = None      # AR(1) state after step t_done
        self.t_done = 0
        if cfg.plant_mode == "count_prefill":
            h = self._hash(_ST_PLANT, self.units[:, None],
                           torch.arange(cfg.prefill, device=self.device)[None, :])
            order = torch.sort(_lsr(h, 1), dim=1, stable=True).indices
            rank = torch.empty_like(order)
            rank.scatter_(1, order, torch.arange(cfg.prefill, device=self.device).expand_as(order).contiguous())
            self._prefill_planted = rank < cfg.plant_count              # [U, P]

    # -- hashing ----------------------------------------------------------------
    def _hash(self, stream: int, *coords: torch.Tensor) -> torch.Tensor:
        x = torch.tensor(_s64(self.seed * 0x100000001B3 + stream * 0x51ED27), device=self.device,
                         dtype=torch.int64)
        x = _mix(x)
        for c in coords:
            x = _mix(x ^ c.to(torch.int64))
        return x

    def _normal_int(self, stream: int, a: torch.Tensor, b: torch.Tensor) -> torch.Tensor:
        """Irwin-Hall(12) integers in units of 2^-16 for coordinates (a, b, d);
        a and b broadcast against each other, a trailing D axis is added."""
        base = self._hash(stream, a, b)[..., None] + self._d * _C_D
        acc = None
        for j in range(3):
            h = _mix(base + _s64(j * _C_J))
            f = (h & 0xFFFF) + (_lsr(h, 16) & 0xFFFF) + (_lsr(h, 32) & 0xFFFF) + _lsr(h, 48)
            acc = f if acc is None else acc + f
        return acc - 6 * 65535

    @staticmethod
    def _to_bf16(z: torch.Tensor) -> torch.Tensor:
        return (z.to(torch.float32) * (1.0 / 65536.0)).to(torch.bfloat16)

    # -- keys and values ----------------------------------------------------------
    def key_int(self, unit_idx: torch.Tensor, pos: torch.Tensor) -> torch.Tensor:
        return self._normal_int(_ST_K, self.units[unit_idx], pos)

    def kv_at(self, pos: torch.Tensor) -> Tuple[torch.Tensor, torch.Tensor]:
        """bf16 K and V [U, len(pos), D] of the tokens at the given positions."""
        pos = pos.to(self.device, torch.int64)
        npos = int(pos.numel())
        rows = max(1, (1 << 25) // max(1, npos * self.D))       # units per slice: bounds the int64 temporaries
        if rows >= self.U:
            k = self._normal_int(_ST_K, self.units[:, None], pos[None, :])
            v = self._normal_int(_ST_V, self.units[:, None], pos[None, :])
            return self._to_bf16(k), self._to_bf16(v)
        k = torch.empty(self.U, npos, self.D, dtype=torch.bfloat16, device=self.device)
        v = torch.empty_like(k)
        for a in range(0, self.U, rows):
            u = self.units[a:a + rows, None]
            k[a:a + rows] = self._to_bf16(self._normal_int(_ST_K, u, pos[None, :]))
            v[a:a + rows] = self._to_bf16(self._normal_int(_ST_V, u, pos[None, :]))
        return k, v

    def prefill(self) -> Tuple[torch.Tensor, torch.Tensor]:
        return self.kv_at(torch.arange(self.cfg.prefill, device=self.device))

    # -- recurrence structure -------------------------------------------------------
    def _period_phase(self, u: torch.Tensor, pos: torch.Tensor):
        cfg = self.cfg
        hp = _lsr(self._hash(_ST_PERIOD, u, pos), 1)
        if cfg.period_mode == "uniform":
            period = cfg.period_lo + hp % (cfg.period_hi - cfg.period_lo + 1)
        else:   # one octave drawn uniformly, then uniform inside it
            octaves = int(round(math.log2(cfg.period_hi / cfg.period_lo)))
            lo = cfg.period_lo << (hp % octaves)
            period = lo + (_lsr(hp, 8) % lo)
        phase = _lsr(self._hash(_ST_PHASE, u, pos), 1) % period
        return period, phase

    def _planted(self, u_idx: torch.Tensor, u: torch.Tensor, pos: torch.Tensor) -> torch.Tensor:
        cfg = self.cfg
        if cfg.plant_mode == "count_prefill":
            inside = pos < cfg.prefill
            return inside & self._prefill_planted[u_idx, pos.clamp(max=cfg.prefill - 1)]
        return (self._hash(_ST_PLANT, u, pos) & 1023) < cfg.plant_prob_1024

    def firing_events(self, t0: int, count: int):
        """Planted-token firings and one-shot spikes in steps [t0, t0 + count).

        Returns int64 tensors (step_offset, unit_index, position), unsorted.
        """
        cfg = self.cfg
        assert count <= self.CHUNK
        P = cfg.prefill
        npos = P + t0 + count - 1                       # positions that exist by the last step
        ev_s, ev_u, ev_p = [], [], []
        rows = max(1, (1 << 24) // max(npos, 1))        # bound the scan's temporaries
        pos = torch.arange(npos, device=self.device, dtype=torch.int64)[None, :]
        birth = (pos - P + 1).clamp(min=0)              # step at which the token was appended
        for a in range(0, self.U, rows):
            u_idx = torch.arange(a, min(a + rows, self.U), device=self.device)[:, None]
            u = self.units[u_idx]
            period, phase = self._period_phase(u, pos)
            first = birth + 1 + phase                   # first firing step
            m = ((t0 - first).clamp(min=0) + period - 1) // period
            fire = first + m * period                   # first firing step >= t0
            hit = (fire < t0 + count) & self._planted(u_idx.expand_as(fire), u, pos.expand_as(fire))
            iu, ip = hit.nonzero(as_tuple=True)
            ev_s.append(fire[iu, ip] - t0); ev_u.append(iu + a); ev_p.append(ip)
        if cfg.spike_prob_1024 > 0:
            steps = torch.arange(t0, t0 + count, device=self.device, dtype=torch.int64)[None, :]
            u = self.units[:, None]
            on = (self._hash(_ST_SPIKE, u, steps) & 1023) < cfg.spike_prob_1024
            target = _lsr(self._hash(_ST_SPIKEPOS, u, steps), 1) % (P + steps - 1).clamp(min=1)
            iu, it = on.nonzero(as_tuple=True)
            ev_s.append(it); ev_u.append(iu); ev_p.append(target[iu, it])
        return torch.cat(ev_s), torch.cat(ev_u), torch.cat(ev_p)

    # -- queries -----------------------------------------------------------------
    def _query_noise(self, t: int) -> torch.Tensor:
        return self._normal_int(_ST_Q, self._heads, torch.tensor(t, device=self.device))      # [U, G, D]

    def _advance(self, t: int) -> torch.Tensor:
        """Integer query (before boosts) of step t; keeps the AR(1) state."""
        z = self._query_noise(t)
        if self.cfg.query == "iid":
            self._state = z
        elif self._state is None:
            self._state = self._query_noise(0)
            self._state = ((self._state * 973) >> 10) + ((z * 319) >> 10)
        else:
            self._state = ((self._state * 973) >> 10) + ((z * 319) >> 10)
        return self._state

    def skip_to(self, t_done: int) -> None:
        """Advance the query walk so that the next generated step is t_done + 1."""
        assert t_done >= self.t_done
        for t in range(self.t_done + 1, t_done + 1):
            self._advance(t)
        self.t_done = t_done

    def steps(self, count: int):
        """Inputs of the next `count` decode steps (t_done + 1 ...).

        Returns (q [count, U, G, D], k_new [count, U, D], v_new [count, U, D]) in bf16.
        """
        cfg = self.cfg
        t0 = self.t_done + 1
        assert 1 <= count <= self.CHUNK
        q = torch.stack([self._advance(t) for t in range(t0, t0 + count)])       # [count, U, G, D] int64
        es, eu, ep = self.firing_events(t0, count)
        if es.numel():
            z = self.key_int(eu, ep)                                             # [E, D]
            norm2 = (z * z).sum(dim=1)                                           # exact integers
            beta = self._beta_num / norm2.to(torch.float64)
            boost = torch.round(beta[:, None] * z.to(torch.float64)).to(torch.int64)
            flat = q.view(count * self.U, self.G, self.D)
            flat.index_add_(0, es * self.U + eu, boost[:, None, :].expand(-1, self.G, -1).contiguous())
        newpos = torch.arange(cfg.prefill + t0 - 1, cfg.prefill + t0 - 1 + count, device=self.device)
        k, v = self.kv_at(newpos)                                                # [U, count, D]
        self.t_done += count
        return self._to_bf16(q), k.transpose(0, 1).contiguous(), v.transpose(0, 1).contiguous()
