"""fp64 CPU oracle for the LazyEviction decode / track / evict path.

THIS FILE IS TEST INFRASTRUCTURE.  It is a slow, plain restatement of the
method in numpy fp64, one independent cache "unit" (one KV head of one layer
of one sequence) at a time.  Only the tests, the smoke check and the bench's
CPU-baseline leg may import it; the CUDA library never does, and this file
imports nothing from the CUDA package.

What it follows (paper sections / equations):

* decode attention ............ Appendix A, Eq. (attn): softmax(q K^T / sqrt(d_h)) V
  over every cached token including the one appended at this step.
* recurrence tracking ......... Section 4 "Recurrence Interval Tracking",
  Eq. (1), Algorithm 1 (the per-token loop and the MRI update).
* importance score ............ Section 4 "MRI-Centric Eviction": H1, H2, Eq. (2).
* lagged eviction ............. Section 4 first paragraph, Appendix A Eq. (evic),
  Algorithm 1 (the `t == kW` branch).
* MRI distribution ............ Section 4 "Discussion about the choice of W and alpha"
  (histogram of MRI and the value below which a given share of the tokens falls).

Readings taken where the paper is silent or inconsistent (each is listed with
its reason in the design notes of the repository):

* A_t[i] of a GQA group is the mean over the group's query heads of their
  softmax rows (the paper does not say how heads are aggregated).
* prefill tokens start with TS = 0, MRI = 0; decode steps count t = 1, 2, ...;
  a token appended at step t starts with TS = t, MRI = 0.
* the test against the threshold is `>=` (Algorithm 1) in float32, because the
  probabilities the tracking consumes are float32 values.
* H2 is the printed formula 2*sigmoid(-1/(MRI-1)); MRI = 1 takes its one-sided
  limit 0 and MRI = 0 is forced to 0 as the text says.
* H1 with MRI = 0: elapsed time > 0 gives 0 (ratio = +inf), elapsed time 0 gives 1.
* eviction fires when t is a multiple of W and the cache holds MORE than B
  tokens (the text; Algorithm 1 prints the comparison the other way round).
* Top_{B-W} is taken over the non-protected tokens only, so that exactly B
  remain; ties are broken towards the more recent token (larger position).
* protected tokens generalise to `n_recent` (paper: W) and `n_initial`
  (paper: 0); the budget may be lowered between windows.

Pinned by tests/test_oracle_pins.py against closed forms, invariants, an
independent library attention routine and brute force on tiny inputs.
PARITY UNPINNED (the paper prints no worked example for them): the H2 reading,
the head aggregation, the initial TS, the tie-break direction.
"""
from __future__ import annotations

import math

import numpy as np

SCORE_MODES = ("h1+h2", "h1", "h2", "h1+h2dec")


def bf16_bits_to_f64(bits) -> np.ndarray:
    """Decode an array of bfloat16 bit patterns (uint16) to float64 exactly."""
    b = np.ascontiguousarray(bits).astype(np.uint32) << np.uint32(16)
    return b.view(np.float32).astype(np.float64)


def sigmoid(x):
    """sigma(x) = 1 / (1 + exp(-x))  (Section 4, H1 definition)."""
    with np.errstate(over="ignore"):
        return 1.0 / (1.0 + np.exp(-np.asarray(x, dtype=np.float64)))


def h1_score(t, ts, mri) -> np.ndarray:
    """H1[i] = 2*sigma(-(t - TS[i]) / MRI[i])  (Section 4, H1-score).

    MRI = 0 (never re-activated): the ratio is +inf for an elapsed time > 0,
    giving 0; an elapsed time of 0 is read as 2*sigma(0) = 1.
    """
    ts = np.asarray(ts, dtype=np.int64)
    mri = np.asarray(mri, dtype=np.int64)
    d = (np.int64(t) - ts).astype(np.float64)
    out = np.empty(d.shape, dtype=np.float64)
    zero = mri == 0
    out[zero] = np.where(d[zero] == 0.0, 1.0, 0.0)
    nz = ~zero
    out[nz] = 2.0 * sigmoid(-(d[nz] / mri[nz].astype(np.float64)))
    return out


def h2_score(mri) -> np.ndarray:
    """H2[i] = 2*sigma(-1 / (MRI[i] - 1)), 0 when MRI[i] = 0  (Section 4, H2-score).

    MRI = 1 makes the argument -1/0 = -inf, whose sigmoid is 0.
    """
    mri = np.asarray(mri, dtype=np.int64)
    out = np.zeros(mri.shape, dtype=np.float64)
    big = mri > 1
    out[big] = 2.0 * sigmoid(-1.0 / (mri[big].astype(np.float64) - 1.0))
    return out


def h2_decreasing(mri) -> np.ndarray:
    """A variant of H2 that does what the paper's prose asks of it: 2*sigma(-(MRI[i] - 1)).

    Section 4 says that a smaller MRI must score higher, and the appendix on the score's
    formulation requires a monotonically decreasing function with values in [0, 1]; the
    printed H2 increases with MRI.  Dropping the reciprocal from the printed argument gives
    the same 2*sigma(-x) form as H1 with x = MRI - 1 >= 0: 1 at MRI = 1, falling to 0.
    MRI = 0 stays 0 as in the text.  This is a reading offered as a switch, not the default.
    """
    mri = np.asarray(mri, dtype=np.int64)
    out = np.zeros(mri.shape, dtype=np.float64)
    on = mri >= 1
    out[on] = 2.0 * sigmoid(-(mri[on].astype(np.float64) - 1.0))
    return out


def importance(t, ts, mri, mode: str = "h1+h2") -> np.ndarray:
    """I_t[i] of Eq. (2): H1 + H2 when MRI != 0, H1 alone when MRI = 0.

    `mode` selects the paper's ablations: "h1" (without H2), "h2" (without H1), and
    "h1+h2dec", Eq. (2) with the decreasing variant of H2.
    """
    if mode not in SCORE_MODES:
        raise ValueError(f"unknown score mode {mode!r}")
    mri = np.asarray(mri, dtype=np.int64)
    h1 = h1_score(t, ts, mri)
    h2 = np.where(mri != 0, h2_score(mri), 0.0)
    if mode == "h1":
        return h1
    if mode == "h2":
        return h2
    if mode == "h1+h2dec":
        return h1 + np.where(mri != 0, h2_decreasing(mri), 0.0)
    return h1 + h2


def mri_histogram(mri_arrays, bins: int) -> np.ndarray:
    """Counts of MRI values over the cached tokens of several units: out[b] = tokens with
    MRI = b for b < bins - 1, out[bins - 1] = tokens with MRI >= bins - 1."""
    out = np.zeros(bins, dtype=np.int64)
    for arr in mri_arrays:
        for v in np.asarray(arr, dtype=np.int64):
            out[min(int(v), bins - 1)] += 1
    return out


def mri_quantile(mri_arrays, fraction: float):
    """The paper's rule for the observation window (Section 4, "Discussion about the choice
    of W and alpha": W = the MRI value below which 80 % of the tokens fall), over the
    re-activated tokens (MRI >= 1): the smallest v with #(MRI <= v) >= fraction * #(MRI >= 1).
    Returns (v, number of re-activated tokens); v = 0 when there are none."""
    vals = np.sort(np.concatenate([np.asarray(a, dtype=np.int64) for a in mri_arrays]))
    vals = vals[vals >= 1]
    if vals.size == 0:
        return 0, 0
    need = fraction * vals.size
    for rank, v in enumerate(vals, start=1):
        if rank >= need:
            return int(v), int(vals.size)
    return int(vals[-1]), int(vals.size)


def attention(q, K, V):
    """Eq. (attn) for the G query heads that share one KV head.

    q [G, D], K [n, D], V [n, D] (float64).  Returns (out [G, D], p [G, n])
    where p[g] is the softmax row of head g over the n cached tokens.
    """
    q = np.asarray(q, dtype=np.float64)
    K = np.asarray(K, dtype=np.float64)
    V = np.asarray(V, dtype=np.float64)
    d_h = K.shape[1]
    s = (q @ K.T) / math.sqrt(d_h)                      # [G, n]
    e = np.exp(s - s.max(axis=1, keepdims=True))
    p = e / e.sum(axis=1, keepdims=True)
    return p @ V, p


class OracleUnit:
    """One independent cache unit stepped through Algorithm 1.

    State per cached token (slot order = generation order, always):
    `pos` original position, `K`, `V`, `TS` last activation step, `MRI`.
    """

    def __init__(self, group: int, head_dim: int, budget: int, window: int,
                 alpha: float, n_recent: int | None = None, n_initial: int = 0,
                 score_mode: str = "h1+h2"):
        if score_mode not in SCORE_MODES:
            raise ValueError(f"unknown score mode {score_mode!r}")
        self.G, self.D = int(group), int(head_dim)
        self.budget = int(budget)          # B: the create-time (maximum) budget
        self.budget_now = int(budget)      # B_t: may be lowered between windows
        self.W = int(window)
        self.alpha32 = np.float32(alpha)
        self.R = self.W if n_recent is None else int(n_recent)
        self.S = int(n_initial)
        self.score_mode = score_mode
        if self.budget <= self.R + self.S:
            raise ValueError("budget must exceed the protected token count")
        self.t = 0
        self.P = 0
        self.pos = np.zeros(0, dtype=np.int64)
        self._set_rows(np.zeros((0, self.D)), np.zeros((0, self.D)))
        self.TS = np.zeros(0, dtype=np.int64)
        self.MRI = np.zeros(0, dtype=np.int64)
        self.last_pbar = np.zeros(0)
        self.last_evict = None             # dict describing the latest eviction

    # -- storage of the cached rows ------------------------------------------------
    # K and V are the first n rows of two buffers that grow by doubling, so that appending one
    # token per step does not copy the whole cache (storage only; no arithmetic lives here).
    def _set_rows(self, K, V) -> None:
        self._K = np.array(K, dtype=np.float64)
        self._V = np.array(V, dtype=np.float64)
        self._rows = self._K.shape[0]

    def _append_row(self, k_new, v_new) -> None:
        if self._rows == self._K.shape[0]:
            grow = max(64, self._rows)
            self._K = np.vstack([self._K, np.zeros((grow, self.D))])
            self._V = np.vstack([self._V, np.zeros((grow, self.D))])
        self._K[self._rows] = np.asarray(k_new, dtype=np.float64)
        self._V[self._rows] = np.asarray(v_new, dtype=np.float64)
        self._rows += 1

    @property
    def K(self) -> np.ndarray:
        return self._K[: self._rows]

    @K.setter
    def K(self, rows) -> None:
        self._K = np.array(rows, dtype=np.float64)
        self._rows = self._K.shape[0]

    @property
    def V(self) -> np.ndarray:
        return self._V[: self._rows]

    @V.setter
    def V(self, rows) -> None:
        self._V = np.array(rows, dtype=np.float64)

    # -- set-up ---------------------------------------------------------------
    @property
    def n(self) -> int:
        return int(self.pos.shape[0])

    def set_budget(self, budget_now: int) -> None:
        budget_now = int(budget_now)
        if not (self.R + self.S < budget_now <= self.budget):
            raise ValueError("budget_now out of range")
        self.budget_now = budget_now

    def prefill(self, K, V) -> None:
        """Load P prompt tokens: TS = 0, MRI = 0, positions 0..P-1, t = 0."""
        K = np.asarray(K, dtype=np.float64)
        V = np.asarray(V, dtype=np.float64)
        self.P = K.shape[0]
        self.pos = np.arange(self.P, dtype=np.int64)
        self._set_rows(K, V)
        self.TS = np.zeros(self.P, dtype=np.int64)
        self.MRI = np.zeros(self.P, dtype=np.int64)
        self.t = 0

    def prefill_observed(self, Q, K, V, pbar_rows=None) -> np.ndarray:
        """Prompt load with tracking from the first prompt token (the paper does not say how
        TS / MRI of prompt tokens start; this is the reading in which Algorithm 1's per-token
        loop already runs over the prompt).  Row j of the prompt attends causally over rows
        0..j at time j - (P - 1), so the last row is time 0 and decode steps go on at t = 1.
        Q [P, G, D], K, V [P, D].  Returns the attention outputs [P, G, D]; the probabilities
        of every row are kept in `prompt_pbar` (list of arrays, row j has j + 1 entries).
        `pbar_rows` [P, P] replaces the oracle's own probabilities in the tracking (bookkeeping
        fed another implementation's float32 values, row j uses its first j + 1 entries)."""
        Q = np.asarray(Q, dtype=np.float64)
        K = np.asarray(K, dtype=np.float64)
        V = np.asarray(V, dtype=np.float64)
        P = K.shape[0]
        self.P = P
        self.pos = np.zeros(0, dtype=np.int64)
        self._set_rows(np.zeros((0, self.D)), np.zeros((0, self.D)))
        self.TS, self.MRI = np.zeros(0, dtype=np.int64), np.zeros(0, dtype=np.int64)
        self.t = -P                       # attend() advances t before it appends: row j runs at j - (P - 1)
        outs = np.zeros((P, self.G, self.D))
        self.prompt_pbar = []
        for j in range(P):
            outs[j], pbar = self.attend(Q[j], K[j], V[j])
            self.prompt_pbar.append(pbar)
            self.track(pbar if pbar_rows is None else np.asarray(pbar_rows)[j, : j + 1])
        assert self.t == 0 and self.n == P
        return outs

    # -- one decode step --------------------------------------------------------
    def append(self, k_new, v_new) -> None:
        """t += 1 and the new token joins the cache with TS = t, MRI = 0 (Section 4)."""
        self.t += 1
        self.pos = np.append(self.pos, self.P + self.t - 1)
        self._append_row(k_new, v_new)
        self.TS = np.append(self.TS, self.t)       # a new token starts at TS = t
        self.MRI = np.append(self.MRI, 0)          # and MRI = 0 (Section 4)

    def attend(self, q, k_new, v_new):
        """t += 1, append the new token, evaluate Eq. (attn).

        Returns (out [G, D], pbar [n]) with pbar[i] the group-mean probability.
        """
        self.append(k_new, v_new)
        out, p = attention(q, self.K, self.V)
        pbar = p.mean(axis=0)
        self.last_pbar = pbar
        return out, pbar

    def track(self, pbar) -> np.ndarray:
        """Algorithm 1's per-token loop and Eq. (1).

        For every token whose weight reaches alpha: MRI = max(MRI, t - TS_old)
        and TS = t.  Tokens below alpha keep TS, so their TS_t - TS_{t-1} = 0
        and their MRI is unchanged.  Returns the boolean activation mask.
        """
        act = np.asarray(pbar, dtype=np.float32) >= self.alpha32
        gap = self.t - self.TS[act]
        self.MRI[act] = np.maximum(self.MRI[act], gap)
        self.TS[act] = self.t
        return act

    def evict_due(self) -> bool:
        """Decision steps are t = kW, and only when the cache exceeds the budget."""
        return self.t > 0 and self.t % self.W == 0 and self.n > self.budget_now

    def scores(self) -> np.ndarray:
        """I_t for every cached token (Eq. 2), protected ones included."""
        return importance(self.t, self.TS, self.MRI, self.score_mode)

    def select_keep(self):
        """Eq. (evic) generalised: initial S + Top_{B-R-S}(I_t) + recent R.

        Returns (kept slot indices ascending, info dict).  The top-k is over the
        unprotected slots [S, n-R) ordered by (I, position) descending.
        """
        n, B, S, R = self.n, self.budget_now, self.S, self.R
        cand = np.arange(S, n - R)
        k = B - R - S
        I = importance(self.t, self.TS[cand], self.MRI[cand], self.score_mode)
        order = np.lexsort((self.pos[cand], I))     # ascending by I, then by pos
        top = order[len(order) - k:]
        rest = order[:len(order) - k]
        kept = np.concatenate([np.arange(S), np.sort(cand[top]), np.arange(n - R, n)])
        info = {
            "t": self.t, "n_before": n, "budget": B, "k": k,
            "kept_pos": self.pos[kept].copy(),
            "evicted_pos": np.sort(self.pos[cand[rest]]),
            # smallest kept score and largest evicted score: when they are
            # closer than rounding noise of exp() the split is not unique
            "kept_min": float(I[top].min()) if k > 0 else math.inf,
            "evicted_max": float(I[rest].max()) if len(rest) else -math.inf,
        }
        return kept, info

    def apply_keep(self, kept) -> None:
        kept = np.asarray(kept, dtype=np.int64)
        self._set_rows(self.K[kept], self.V[kept])
        self.pos = self.pos[kept]
        self.TS, self.MRI = self.TS[kept], self.MRI[kept]

    def evict_if_due(self):
        if not self.evict_due():
            return None
        kept, info = self.select_keep()
        self.apply_keep(kept)
        self.last_evict = info
        return info

    def force_keep_positions(self, positions) -> None:
        """Make the cache hold exactly the given original positions (used when a
        test pins the oracle's cache to another implementation's kept set)."""
        want = np.asarray(positions, dtype=np.int64)
        idx = np.searchsorted(self.pos, want)
        if idx.max(initial=-1) >= self.n or not np.array_equal(self.pos[idx], want):
            raise ValueError("positions not all present in the oracle cache")
        self.apply_keep(idx)

    def step(self, q, k_new, v_new, pbar_override=None):
        """One full decode step in Algorithm 1's order.

        `pbar_override` replaces the oracle's own probabilities in the tracking
        (bookkeeping fed another implementation's float32 probabilities).
        Returns (out, pbar, eviction-info-or-None).
        """
        out, pbar = self.attend(q, k_new, v_new)
        self.track(pbar if pbar_override is None else pbar_override)
        info = self.evict_if_due()
        return out, pbar, info
