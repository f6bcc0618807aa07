"""Pins for the fp64 oracle: each test checks it against something other than
itself -- a closed form, an invariant the paper states, a library routine, a
hand-worked trace or brute force -- so that a dropped term, a wrong sign or
index, or a transposed operand fails at least one of them."""
import itertools
import math
import os

import numpy as np
import pytest
import torch

from oracle import lazyev_oracle as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def two_sigma_neg(x):
    """2*sigma(-x) through the identity 2*sigma(-x) = 1 - tanh(x/2)."""
    return 1.0 - math.tanh(x / 2.0)


def make_unit(G=2, D=8, budget=64, window=4, alpha=0.1, **kw):
    return orc.OracleUnit(G, D, budget, window, alpha, **kw)


# ---------------------------------------------------------------- Eq. (attn)
def test_full_attention_matches_library_sdpa():
    """Budget >= prompt + generated tokens: nothing is ever evicted, so every
    step's output is plain softmax attention over all tokens (Eq. attn)."""
    rng = np.random.default_rng(7)
    G, D, P, T = 4, 16, 9, 37
    u = orc.OracleUnit(G, D, budget=P + T + 8, window=5, alpha=0.02)
    K0, V0 = rng.normal(size=(P, D)), rng.normal(size=(P, D))
    u.prefill(K0, V0)
    allK, allV = [K0], [V0]
    for t in range(1, T + 1):
        q, k, v = rng.normal(size=(G, D)) * 1.7, rng.normal(size=D), rng.normal(size=D)
        out, pbar, info = u.step(q, k, v)
        allK.append(k[None]); allV.append(v[None])
        Kf, Vf = np.concatenate(allK), np.concatenate(allV)
        ref = torch.nn.functional.scaled_dot_product_attention(
            torch.from_numpy(q)[None, :, None, :],                      # [1, G, 1, D]
            torch.from_numpy(Kf)[None, None].expand(1, G, -1, -1),
            torch.from_numpy(Vf)[None, None].expand(1, G, -1, -1))
        np.testing.assert_allclose(out, ref[0, :, 0].numpy(), rtol=1e-12, atol=1e-13)
        assert info is None and u.n == P + t
        assert abs(pbar.sum() - 1.0) < 1e-12 and pbar.shape == (P + t,)
    assert np.array_equal(u.pos, np.arange(P + T))


def test_attention_rows_are_softmax_and_scale_is_sqrt_d():
    rng = np.random.default_rng(3)
    G, D, n = 3, 32, 11
    q, K, V = rng.normal(size=(G, D)), rng.normal(size=(n, D)), rng.normal(size=(n, D))
    out, p = orc.attention(q, K, V)
    assert p.shape == (G, n)
    np.testing.assert_allclose(p.sum(axis=1), 1.0, atol=1e-14)
    # explicit double loop, no vectorisation
    for g in range(G):
        s = [sum(q[g, d] * K[i, d] for d in range(D)) / math.sqrt(D) for i in range(n)]
        z = sum(math.exp(x) for x in s)
        for i in range(n):
            assert abs(p[g, i] - math.exp(s[i]) / z) < 1e-14
        for d in range(D):
            assert abs(out[g, d] - sum(math.exp(s[i]) / z * V[i, d] for i in range(n))) < 1e-13


def test_single_token_and_uniform_keys():
    """One cached token gets weight 1; identical keys get weight 1/n each and
    the output is the mean of V."""
    q = np.ones((2, 4))
    out, p = orc.attention(q, np.ones((1, 4)), np.array([[1.0, 2.0, 3.0, 4.0]]))
    assert np.allclose(p, 1.0) and np.allclose(out, [[1, 2, 3, 4]] * 2)
    V = np.arange(20.0).reshape(5, 4)
    out, p = orc.attention(q, np.ones((5, 4)) * 0.3, V)
    assert np.allclose(p, 0.2) and np.allclose(out, V.mean(axis=0))


def test_group_mean_is_over_query_heads():
    """pbar is the arithmetic mean of the G softmax rows (reading of A_t[i])."""
    rng = np.random.default_rng(11)
    u = make_unit(G=3, D=8, budget=100)
    u.prefill(rng.normal(size=(6, 8)), rng.normal(size=(6, 8)))
    q = rng.normal(size=(3, 8)) * 3
    out, pbar = u.attend(q, rng.normal(size=8), rng.normal(size=8))
    rows = [orc.attention(q[g:g + 1], u.K, u.V)[1][0] for g in range(3)]
    np.testing.assert_allclose(pbar, (rows[0] + rows[1] + rows[2]) / 3.0, atol=1e-15)


# -------------------------------------------------------- Eq. (1), Algorithm 1
def read_traces():
    rows = []
    with open(os.path.join(GOLDEN, "recurrence_traces.txt")) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if not line:
                continue
            name, ts0, hits, last, ts, mri = [c.strip() for c in line.split("|")]
            rows.append((name, int(ts0), [int(x) for x in hits.split()], int(last), int(ts), int(mri)))
    return rows


@pytest.mark.parametrize("row", read_traces(), ids=lambda r: r[0])
def test_track_reproduces_hand_worked_traces(row):
    name, ts0, hits, last, ts_want, mri_want = row
    u = make_unit(alpha=0.25)
    u.pos = np.arange(2); u.K = np.zeros((2, 8)); u.V = np.zeros((2, 8))
    u.TS = np.array([ts0, 0]); u.MRI = np.array([0, 0])
    for t in range(max(ts0, 1), last + 1):
        u.t = t
        pbar = np.array([0.6 if t in hits else 0.1, 0.05])
        u.track(pbar)
    assert (u.TS[0], u.MRI[0]) == (ts_want, mri_want)
    assert (u.TS[1], u.MRI[1]) == (0, 0)            # the bystander never moves


def test_recurring_key_through_full_steps():
    """A planted key direction that the query re-aligns with at chosen steps:
    attention + tracking together must give TS = last hit, MRI = longest gap."""
    D, P = 8, 3
    c = 8.0
    eye = np.eye(D)
    u = orc.OracleUnit(2, D, budget=200, window=50, alpha=0.1)
    u.prefill(np.stack([c * eye[0], c * eye[1], c * eye[2]]), np.zeros((P, D)))
    hits = {1: [5, 8, 15, 20], 2: [12]}             # prefill token -> steps
    born = {4: (3, [9, 11, 25]), 7: (4, [])}        # birth step -> (direction, later hits)
    for t in range(1, 31):
        target = 0                                  # the sink direction by default
        for tok, steps in hits.items():
            if t in steps:
                target = tok
        for b, (direc, steps) in born.items():
            if t in steps:
                target = direc
        q = np.tile(6.0 * eye[target], (2, 1))
        k_new = c * eye[born[t][0]] if t in born else np.zeros(D)
        u.step(q, k_new, np.zeros(D))
    slot = {p: i for i, p in enumerate(u.pos)}
    assert (u.TS[slot[1]], u.MRI[slot[1]]) == (20, 7)
    assert (u.TS[slot[2]], u.MRI[slot[2]]) == (12, 12)
    assert (u.TS[slot[P + 4 - 1]], u.MRI[slot[P + 4 - 1]]) == (25, 14)   # born at 4: hits 9, 11, 25
    assert (u.TS[slot[P + 7 - 1]], u.MRI[slot[P + 7 - 1]]) == (7, 0)     # never re-activated
    # zero-key tokens never reach alpha after their own step
    z = slot[P + 10 - 1]
    assert (u.TS[z], u.MRI[z]) == (10, 0)


def test_threshold_is_inclusive_and_float32():
    u = make_unit(alpha=0.3)
    u.pos = np.arange(3); u.K = np.zeros((3, 8)); u.V = np.zeros((3, 8))
    u.TS = np.zeros(3, dtype=np.int64); u.MRI = np.zeros(3, dtype=np.int64)
    u.t = 5
    a32 = np.float32(0.3)
    below = np.nextafter(a32, np.float32(0), dtype=np.float32)
    act = u.track(np.array([a32, below, 0.9], dtype=np.float32))
    assert act.tolist() == [True, False, True]
    assert u.TS.tolist() == [5, 0, 5] and u.MRI.tolist() == [5, 0, 5]


def test_alpha_zero_activates_everything():
    """alpha = 0: every token is active at every step, so every token older
    than the newest has MRI = 1, TS = t; all scores tie at 1 and eviction
    degenerates to a sliding window."""
    rng = np.random.default_rng(5)
    P, W, B = 6, 4, 10
    u = orc.OracleUnit(2, 8, budget=B, window=W, alpha=0.0)
    u.prefill(rng.normal(size=(P, 8)), rng.normal(size=(P, 8)))
    for t in range(1, 41):
        u.step(rng.normal(size=(2, 8)), rng.normal(size=8), rng.normal(size=8))
        assert np.all(u.TS == t)
        assert np.all(u.MRI[u.pos < P + t - 1] == 1) and u.MRI[-1] == 0
        assert np.allclose(u.scores()[:-1], 1.0)
        if t % W == 0 and P + t > B:
            assert np.array_equal(u.pos, np.arange(P + t - B, P + t))


def test_alpha_above_one_gives_sliding_window():
    """alpha > 1: nothing ever activates; every unprotected score is 0, and the
    tie-break keeps the most recent tokens: exactly the B latest positions."""
    rng = np.random.default_rng(6)
    P, W, B, R = 7, 5, 13, 3
    u = orc.OracleUnit(3, 8, budget=B, window=W, alpha=1.5, n_recent=R)
    u.prefill(rng.normal(size=(P, 8)), rng.normal(size=(P, 8)))
    for t in range(1, 61):
        _, _, info = u.step(rng.normal(size=(3, 8)), rng.normal(size=8), rng.normal(size=8))
        assert np.all(u.MRI == 0)
        if info is not None:
            assert np.array_equal(u.pos, np.arange(P + t - B, P + t))
            assert np.all(u.scores()[: u.n - R][u.TS[: u.n - R] < t] == 0.0)


# ------------------------------------------------------------ H1, H2, Eq. (2)
def test_score_closed_forms():
    e = math.e
    I = lambda d, mri, mode="h1+h2": float(orc.importance(100, 100 - d, mri, mode))
    assert I(0, 2) == pytest.approx(1.0 + 2.0 / (1.0 + e), abs=1e-15)             # 1.5378828...
    assert I(2, 2) == pytest.approx(4.0 / (1.0 + e), abs=1e-15)                   # 1.0757656...
    assert I(1, 1) == pytest.approx(2.0 / (1.0 + e), abs=1e-15)                   # H2(MRI=1) = 0
    assert I(0, 1) == 1.0
    assert I(0, 0) == 1.0
    assert I(1, 0) == 0.0 and I(5000, 0) == 0.0
    assert I(3, 3) == pytest.approx(2.0 / (1.0 + e) + 2.0 / (1.0 + math.sqrt(e)), abs=1e-15)
    assert I(10, 5) == pytest.approx(2.0 / (1.0 + e * e) + 2.0 / (1.0 + e ** 0.25), abs=1e-15)
    assert I(10, 5, "h1") == pytest.approx(2.0 / (1.0 + e * e), abs=1e-15)
    assert I(10, 5, "h2") == pytest.approx(2.0 / (1.0 + e ** 0.25), abs=1e-15)
    assert I(10 ** 6, 1) == 0.0                                                    # exp overflow -> 0
    # H2 tends to 2*sigma(0) = 1 for very long intervals
    assert float(orc.h2_score(10 ** 9)) == pytest.approx(1.0, abs=1e-8)


def test_score_against_tanh_identity_and_properties():
    """2*sigma(-x) = 1 - tanh(x/2): an independent evaluation of both terms on a
    grid; H1 strictly decreases with the elapsed time; both terms lie in [0, 1]."""
    t = 5000
    for mri in [1, 2, 3, 7, 50, 175, 1000, 4096]:
        prev = None
        for d in [0, 1, 2, 5, 17, 100, 999, 4999]:
            h1 = float(orc.h1_score(t, t - d, mri))
            h2 = float(orc.h2_score(mri))
            assert h1 == pytest.approx(two_sigma_neg(d / mri), abs=2e-15)
            want_h2 = 0.0 if mri == 1 else two_sigma_neg(1.0 / (mri - 1))
            assert h2 == pytest.approx(want_h2, abs=2e-15)
            assert 0.0 <= h1 <= 1.0 and 0.0 <= h2 <= 1.0
            assert float(orc.importance(t, t - d, mri)) == pytest.approx(h1 + h2, abs=1e-15)
            if prev is not None and h1 > 0:
                assert h1 < prev
            prev = h1
    # vectorised call equals element-wise calls
    ts = np.array([10, 20, 4990, 5000]); mri = np.array([0, 3, 9, 0])
    vec = orc.importance(t, ts, mri)
    for i in range(4):
        assert vec[i] == float(orc.importance(t, ts[i], mri[i]))


def test_decreasing_h2_variant_has_the_properties_the_appendix_requires():
    """The appendix on the score's formulation asks for a monotonically decreasing function
    with values in [0, 1], and Section 4 for "smaller MRI, higher score": the variant
    2*sigma(-(MRI - 1)) has them, the printed H2 does not (it increases with MRI)."""
    e = math.e
    assert float(orc.h2_decreasing(0)) == 0.0                       # never re-activated: stays 0 as in the text
    assert float(orc.h2_decreasing(1)) == 1.0                       # 2*sigma(0)
    assert float(orc.h2_decreasing(2)) == pytest.approx(2.0 / (1.0 + e), abs=1e-15)
    assert float(orc.h2_decreasing(4)) == pytest.approx(1.0 - math.tanh(1.5), abs=1e-15)
    grid = np.arange(1, 60)
    dec, printed = orc.h2_decreasing(grid), orc.h2_score(grid)
    assert (np.diff(dec) < 0).all() and (dec >= 0).all() and (dec <= 1).all()
    assert (np.diff(printed) > 0).all()                             # the printed formula goes the other way
    assert float(orc.h2_decreasing(10 ** 6)) == 0.0
    # inside Eq. (2): H1 + variant when MRI != 0, H1 alone when MRI = 0
    I = lambda d, mri: float(orc.importance(100, 100 - d, mri, "h1+h2dec"))
    assert I(2, 2) == pytest.approx(2.0 / (1.0 + e) + 2.0 / (1.0 + e), abs=1e-15)
    assert I(0, 0) == 1.0 and I(7, 0) == 0.0
    # two tokens, equally overdue relative to their intervals: the frequent one now ranks higher
    assert I(3, 3) > I(30, 30) and float(orc.importance(100, 97, 3)) < float(orc.importance(100, 70, 30))


def test_observed_prompt_is_causal_attention_with_tracking_from_the_first_token():
    """Outputs equal the library's causal SDPA; with alpha > 1 nothing is re-activated and every
    token keeps TS = its own time j - (P - 1); a planted key re-activated at known rows gets
    the hand-computed TS and MRI; decode steps continue at t = 1."""
    rng = np.random.default_rng(11)
    P, G, D = 37, 3, 16
    Q, K, V = rng.standard_normal((P, G, D)), rng.standard_normal((P, D)), rng.standard_normal((P, D))
    o = orc.OracleUnit(G, D, 100, 8, 1.5)
    outs = o.prefill_observed(Q, K, V)
    ref = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(Q).permute(1, 0, 2)[None], torch.from_numpy(K)[None, None].expand(1, G, P, D),
        torch.from_numpy(V)[None, None].expand(1, G, P, D), is_causal=True)[0].permute(1, 0, 2).numpy()
    assert np.abs(outs - ref).max() < 1e-12
    assert o.TS.tolist() == [j - (P - 1) for j in range(P)] and not o.MRI.any()
    assert o.pos.tolist() == list(range(P)) and o.t == 0
    # token 2 is made to dominate rows 5, 9 and 20 (and is active at its own row 2): gaps 3, 4, 11
    K2, Q2 = 0.01 * rng.standard_normal((P, D)), 0.01 * rng.standard_normal((P, G, D))
    K2[2] = 0.0; K2[2, 0] = 8.0
    for j in (5, 9, 20):
        Q2[j, :, 0] = 8.0
    o2 = orc.OracleUnit(G, D, 100, 8, 0.6)
    o2.prefill_observed(Q2, K2, V)
    assert o2.TS[2] == 20 - (P - 1) and o2.MRI[2] == 11
    # every token is active at its own row only when it takes >= 0.6 of the weight: row 0 always does
    assert o2.TS[0] == 0 - (P - 1) and o2.MRI[0] == 0
    _, pbar = o2.attend(Q2[5], K2[3], V[3])                  # first decode step: t = 1, position P
    o2.track(pbar)
    assert o2.t == 1 and o2.pos[-1] == P and o2.TS[2] == 1 and o2.MRI[2] == 1 - (20 - (P - 1))


def test_mri_histogram_and_quantile_closed_forms_and_library_routine():
    """One token per MRI value 1..100 (plus never re-activated ones): the 80 % value is 80;
    on random data the rule equals numpy's inverted-CDF percentile of the re-activated tokens."""
    a = [np.arange(0, 51), np.concatenate([np.arange(51, 101), np.zeros(500, dtype=np.int64)])]
    assert orc.mri_quantile(a, 0.8) == (80, 100)
    assert orc.mri_quantile(a, 1.0) == (100, 100) and orc.mri_quantile(a, 0.005) == (1, 100)
    assert orc.mri_quantile([np.zeros(7)], 0.8) == (0, 0)
    h = orc.mri_histogram(a, 64)
    assert h[0] == 501 and (h[1:63] == 1).all() and h[63] == 100 - 62 and h.sum() == 601
    rng = np.random.default_rng(3)
    for _ in range(20):
        arrs = [rng.integers(0, 300, size=rng.integers(1, 400)) * (rng.random(1) < 0.9) for _ in range(3)]
        pooled = np.concatenate(arrs)
        pooled = pooled[pooled >= 1]
        frac = float(rng.uniform(0.05, 1.0))
        if pooled.size:
            want = int(np.percentile(pooled, 100 * frac, method="inverted_cdf"))
            assert orc.mri_quantile(arrs, frac) == (want, pooled.size)
        hist = orc.mri_histogram(arrs, 128)
        assert hist.sum() == sum(len(x) for x in arrs)
        assert np.array_equal(hist[:127], np.bincount(np.concatenate(arrs), minlength=300)[:127])


def test_elapsed_beyond_mri_is_evicted_first():
    """Two tokens with the same MRI = 10: the one last seen 50 steps ago goes
    before the one last seen 5 steps ago (Introduction: evict when the elapsed
    time exceeds the MRI)."""
    u = orc.OracleUnit(1, 4, budget=4, window=2, alpha=0.5, n_recent=2)
    u.pos = np.arange(5); u.K = np.zeros((5, 4)); u.V = np.arange(20.0).reshape(5, 4)
    u.t = 100
    u.TS = np.array([95, 50, 100, 99, 100]); u.MRI = np.array([10, 10, 0, 0, 0])
    assert u.evict_due()
    info = u.evict_if_due()
    assert info["evicted_pos"].tolist() == [1]
    assert u.pos.tolist() == [0, 2, 3, 4]
    assert u.V[:, 0].tolist() == [0.0, 8.0, 12.0, 16.0]          # rows moved with their tokens
    assert u.TS.tolist() == [95, 100, 99, 100] and u.MRI.tolist() == [10, 0, 0, 0]


# -------------------------------------------------------------- Eq. (evic)
def brute_force_keep(pos, ts, mri, t, B, R, S):
    """Enumerate every subset of the candidates of the right size and take the
    one that is lexicographically best: the k largest (score, position) pairs."""
    n = len(pos)
    cand = list(range(S, n - R))
    k = B - R - S

    def score(i):
        d = t - ts[i]
        if mri[i] == 0:
            return 1.0 if d == 0 else 0.0
        h1 = two_sigma_neg(d / mri[i])
        h2 = 0.0 if mri[i] == 1 else two_sigma_neg(1.0 / (mri[i] - 1))
        return h1 + h2

    best, best_key = None, None
    for sub in itertools.combinations(cand, k):
        key = sorted(((round(score(i), 13), pos[i]) for i in sub), reverse=True)
        if best_key is None or key > best_key:
            best, best_key = sub, key
    return sorted(list(range(S)) + list(best) + list(range(n - R, n)))


@pytest.mark.parametrize("seed", range(12))
def test_select_matches_brute_force(seed):
    rng = np.random.default_rng(100 + seed)
    n = int(rng.integers(7, 13))
    R = int(rng.integers(1, 3)); S = int(rng.integers(0, 2))
    B = int(rng.integers(R + S + 1, n))
    t = 60
    u = orc.OracleUnit(1, 4, budget=B, window=1, alpha=0.5, n_recent=R, n_initial=S)
    u.pos = np.sort(rng.choice(80, size=n, replace=False)).astype(np.int64)
    u.K = np.zeros((n, 4)); u.V = np.zeros((n, 4)); u.t = t
    u.TS = rng.integers(0, t + 1, size=n)
    u.MRI = rng.choice([0, 0, 1, 2, 3, 5, 20], size=n)          # many exact ties
    kept, info = u.select_keep()
    assert kept.tolist() == brute_force_keep(u.pos, u.TS, u.MRI, t, B, R, S)
    assert len(kept) == B and info["kept_min"] >= info["evicted_max"]


def test_sawtooth_budget_and_protection_invariants():
    """After every eviction exactly B tokens remain; the cache never exceeds
    B + W; it grows by one per step in between; the recent R tokens and the
    initial S tokens always survive; slot order stays generation order."""
    rng = np.random.default_rng(21)
    G, D, P, W, B, R, S = 2, 8, 20, 8, 32, 5, 2
    u = orc.OracleUnit(G, D, budget=B, window=W, alpha=0.03, n_recent=R, n_initial=S)
    u.prefill(rng.normal(size=(P, D)), rng.normal(size=(P, D)))
    prev_n, events = P, 0
    for t in range(1, 161):
        before = u.pos.copy()
        _, _, info = u.step(rng.normal(size=(G, D)) * 2, rng.normal(size=D), rng.normal(size=D))
        assert np.all(np.diff(u.pos) > 0)
        assert u.n <= B + W
        if info is None:
            assert u.n == prev_n + 1
            assert not (t % W == 0 and u.n > B)
        else:
            events += 1
            assert t % W == 0 and info["n_before"] == prev_n + 1 > B and u.n == B
            assert np.array_equal(u.pos[-R:], np.arange(P + t - R, P + t))
            assert np.array_equal(u.pos[:S], np.arange(S))
            assert set(info["kept_pos"]) | set(info["evicted_pos"]) == set(before) | {P + t - 1}
            assert info["kept_min"] >= info["evicted_max"]
        prev_n = u.n
    assert events == (160 - 16) // W + 1            # first at t = 16 (n = 36 > 32), then every W


def test_dynamic_budget_and_prompt_longer_than_budget():
    rng = np.random.default_rng(22)
    u = orc.OracleUnit(1, 8, budget=40, window=4, alpha=0.05)
    u.prefill(rng.normal(size=(50, 8)), rng.normal(size=(50, 8)))      # P > B
    sizes = []
    for t in range(1, 25):
        if t == 9:
            u.set_budget(20)
        u.step(rng.normal(size=(1, 8)), rng.normal(size=8), rng.normal(size=8))
        sizes.append(u.n)
    assert sizes[:4] == [51, 52, 53, 40]            # first decision step cuts P + W to B
    assert sizes[11] == 20 and max(sizes[12:]) <= 24
    with pytest.raises(ValueError):
        u.set_budget(41)
    with pytest.raises(ValueError):
        u.set_budget(4)


def test_override_probabilities_drive_bookkeeping():
    rng = np.random.default_rng(23)
    u = orc.OracleUnit(1, 8, budget=30, window=5, alpha=0.2)
    u.prefill(rng.normal(size=(4, 8)), rng.normal(size=(4, 8)))
    fake = np.array([0.0, 0.5, 0.0, 0.0, 0.0], dtype=np.float32)
    u.step(rng.normal(size=(1, 8)), rng.normal(size=8), rng.normal(size=8), pbar_override=fake)
    assert u.TS.tolist() == [0, 1, 0, 0, 1] and u.MRI.tolist() == [0, 1, 0, 0, 0]


def test_force_keep_positions():
    rng = np.random.default_rng(24)
    u = orc.OracleUnit(1, 4, budget=30, window=5, alpha=0.2)
    u.prefill(rng.normal(size=(6, 4)), rng.normal(size=(6, 4)))
    k3 = u.K[3].copy()
    u.force_keep_positions([0, 3, 5])
    assert u.pos.tolist() == [0, 3, 5] and np.array_equal(u.K[1], k3)
    with pytest.raises(ValueError):
        u.force_keep_positions([1])


def test_bf16_decoding():
    bits = np.array([0x3F80, 0xBF80, 0x4000, 0x0000, 0x3DCD], dtype=np.uint16)
    want = torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16).double().numpy()
    got = orc.bf16_bits_to_f64(bits)
    assert np.array_equal(got, want) and got[:3].tolist() == [1.0, -1.0, 2.0]


def test_append_without_attention_keeps_the_same_cache():
    """append() is attend() without the arithmetic: after any mix of the two, and across the storage's
    growth steps and an eviction, both units hold the same tokens and give the same attention."""
    rng = np.random.default_rng(31)
    a = orc.OracleUnit(2, 8, budget=150, window=50, alpha=0.01, n_recent=10)
    b = orc.OracleUnit(2, 8, budget=150, window=50, alpha=0.01, n_recent=10)
    K0, V0 = rng.normal(size=(3, 8)), rng.normal(size=(3, 8))
    a.prefill(K0, V0); b.prefill(K0, V0)
    for t in range(1, 301):
        q, k, v = rng.normal(size=(2, 8)), rng.normal(size=8), rng.normal(size=8)
        out_a, pbar = a.attend(q, k, v)
        if t % 7 == 0:
            out_b, pbar_b = b.attend(q, k, v)
            assert np.array_equal(out_a, out_b) and np.array_equal(pbar, pbar_b)
        else:
            b.append(k, v)
        a.track(pbar); b.track(pbar)                 # the same probabilities drive both bookkeepings
        assert (a.evict_if_due() is None) == (b.evict_if_due() is None)
        assert a.n == b.n and a.t == b.t == t
    assert a.n == 150 + 0 and np.array_equal(a.K, b.K) and np.array_equal(a.V, b.V)
    assert np.array_equal(a.pos, b.pos) and np.array_equal(a.TS, b.TS) and np.array_equal(a.MRI, b.MRI)


def test_observed_prompt_tracking_can_consume_supplied_probabilities():
    """prefill_observed(pbar_rows=...): Eq. (1) over the prompt rows driven by given float32 rows.
    Hand-worked: alpha = 0.3, rows (times -2, -1, 0) [0.9], [0.05, 0.95], [0.5, 0.1, 0.4]:
    token 0 is active at -2 and again at 0 (MRI 2, TS 0); token 1 only at its own row; token 2 at its own."""
    rng = np.random.default_rng(32)
    Q, K, V = rng.normal(size=(3, 1, 4)), rng.normal(size=(3, 4)), rng.normal(size=(3, 4))
    rows = np.zeros((3, 3), dtype=np.float32)
    rows[0, :1], rows[1, :2], rows[2, :3] = [0.9], [0.05, 0.95], [0.5, 0.1, 0.4]
    o = orc.OracleUnit(1, 4, budget=10, window=4, alpha=0.3)
    outs = o.prefill_observed(Q, K, V, pbar_rows=rows)
    assert o.TS.tolist() == [0, -1, 0] and o.MRI.tolist() == [2, 0, 0] and o.t == 0
    # the attention itself is untouched by the override, and its own rows are kept for comparison
    ref = orc.OracleUnit(1, 4, budget=10, window=4, alpha=0.3)
    assert np.array_equal(outs, ref.prefill_observed(Q, K, V))
    assert len(o.prompt_pbar) == 3 and np.allclose([r.sum() for r in o.prompt_pbar], 1.0)
    # feeding a unit its own rows back changes nothing
    own = np.zeros((3, 3)); [own.__setitem__((j, slice(0, j + 1)), ref.prompt_pbar[j]) for j in range(3)]
    again = orc.OracleUnit(1, 4, budget=10, window=4, alpha=0.3)
    again.prefill_observed(Q, K, V, pbar_rows=own)
    assert np.array_equal(again.TS, ref.TS) and np.array_equal(again.MRI, ref.MRI)


# ---- property-based pins (hypothesis): the bookkeeping against a per-token restatement of Eq. (1) ----
from hypothesis import given, settings, strategies as st_


@settings(max_examples=60, deadline=None)
@given(st_.integers(1, 6), st_.integers(1, 40), st_.integers(0, 2 ** 32 - 1))
def test_track_equals_a_per_token_state_machine(n_tokens, steps, seed):
    """Eq. (1) token by token: a token's MRI is the largest gap between consecutive activations
    (its birth counts as one), its TS the last of them.  Random activation patterns through track()
    against that restatement computed from the whole history at once."""
    rng = np.random.default_rng(seed)
    alpha = 0.5
    u = orc.OracleUnit(1, 4, budget=1000, window=500, alpha=alpha)
    u.prefill(np.zeros((n_tokens, 4)), np.zeros((n_tokens, 4)))
    history = []                                     # per step: activation mask over the tokens alive then
    for t in range(1, steps + 1):
        u.append(np.zeros(4), np.zeros(4))
        act = rng.random(u.n) < 0.3
        pbar = np.where(act, 0.9, 0.1).astype(np.float32)
        got = u.track(pbar)
        assert np.array_equal(got, act)
        history.append(act)
    for i in range(u.n):
        birth = 0 if i < n_tokens else i - n_tokens + 1          # prompt tokens start at TS = 0
        times = [birth] + [t for t in range(max(birth, 1), steps + 1) if history[t - 1][i]]
        gaps = [b - a for a, b in zip(times, times[1:])]
        assert u.TS[i] == times[-1] and u.MRI[i] == max(gaps + [0])


@settings(max_examples=40, deadline=None)
@given(st_.integers(0, 2 ** 32 - 1))
def test_eviction_invariants_on_random_runs(seed):
    """Whatever the probabilities: the cache holds exactly B_t tokens after an eviction and never more than
    B + W, positions stay strictly increasing, the R newest and S oldest tokens always survive, and what is
    kept scores at least as high as what goes (Eq. (evic) generalised)."""
    rng = np.random.default_rng(seed)
    W = int(rng.integers(1, 9)); R = int(rng.integers(1, W + 1)); S = int(rng.integers(0, 3))
    B = int(rng.integers(max(W, R + S) + 1, 40)); P = int(rng.integers(1, 30))
    u = orc.OracleUnit(2, 4, budget=B, window=W, alpha=float(rng.choice([0.0, 0.02, 0.2, 2.0])), n_recent=R, n_initial=S)
    u.prefill(rng.normal(size=(P, 4)), rng.normal(size=(P, 4)))
    for t in range(1, 5 * W + 7):
        n_before = u.n
        _, _, info = u.step(rng.normal(size=(2, 4)) * 3, rng.normal(size=4), rng.normal(size=4))
        assert (t % W == 0 and n_before + 1 > B) == (info is not None)
        if info is not None:
            assert u.n == B and info["kept_min"] >= info["evicted_max"]
            assert u.pos[-R:].tolist() == list(range(P + t - R, P + t))
            assert u.pos[:S].tolist() == list(range(S))         # the oldest S tokens are never evicted
        assert u.n <= max(B, P) + W and np.all(np.diff(u.pos) > 0) and u.t == t
