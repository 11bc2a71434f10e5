"""Pins for the CPU oracle: everything here checks the oracle against something
other than itself — numpy's full attention, identities from the proof of
Theorem 4.1, closed forms, a from-the-definition brute force with exhaustive
subset search, hand-worked fixtures, and an independent int4 quantiser."""
import itertools
import math
import os

import numpy as np
import pytest

import oracle
from bruteforce import BruteForceUnit, full_attention

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _stream(T, U, d, seed, peaked=0.0):
    rng = np.random.default_rng(seed)
    q = rng.standard_normal((T, U, d))
    k = rng.standard_normal((T, U, d))
    v = rng.standard_normal((T, U, d))
    if peaked:
        u = rng.standard_normal((U, d))
        u /= np.linalg.norm(u, axis=1, keepdims=True)
        hit = rng.random((T, U, 1)) < 0.15
        q = q + peaked * u
        k = k + hit * peaked * math.sqrt(d) * u
    return q, k, v


# --- attention: B >= T never compresses and equals full causal attention --------
# (Theorem 4.1 discussion: the error is zero when B = T_max; Algorithm 1 only
# compresses once the budget is reached.)
def test_budget_at_least_stream_length_is_full_attention():
    T, U, d = 40, 3, 16
    q, k, v = _stream(T, U, d, 1, peaked=2.0)
    o = oracle.Oracle(U, B=T + 1, r=2, w=8, m=4, head_dim=d)
    for t in range(T):
        out, dropped = o.step(q[t], k[t], v[t])
        assert dropped is None
        for u in range(U):
            ref, _ = full_attention(q[t, u], k[: t + 1, u], v[: t + 1, u], 1 / math.sqrt(d))
            np.testing.assert_allclose(out[u], ref, rtol=0, atol=1e-13)
    assert o.n == T and o.t == T
    assert (o.positions() == np.arange(1, T + 1)).all()


def test_scale_argument_is_applied_to_logits():
    T, U, d = 12, 1, 8
    q, k, v = _stream(T, U, d, 2)
    o = oracle.Oracle(U, B=T + 1, r=1, w=4, m=1, head_dim=d, scale=0.37)
    for t in range(T):
        out, _ = o.step(q[t], k[t], v[t])
    ref, _ = full_attention(q[T - 1, 0], k[:, 0], v[:, 0], 0.37)
    np.testing.assert_allclose(out[0], ref, atol=1e-13)


# --- closed forms ---------------------------------------------------------------
def test_equal_keys_give_uniform_scores_zero_record_and_fifo_eviction():
    # All keys equal => alpha_j = 1/n exactly-ish.  With n < t that is above 1/t,
    # so no token is ever low once the first compression has happened, every
    # counter stays 0 and eviction is oldest-first.
    T, U, d, B, r, w, m = 60, 2, 8, 10, 3, 5, 4
    rng = np.random.default_rng(3)
    kk = rng.standard_normal(d)
    q = rng.standard_normal((T, U, d))
    v = rng.standard_normal((T, U, d))
    o = oracle.Oracle(U, B, r, w, m, d)
    live = []
    for t in range(1, T + 1):
        live.append(t)
        out, alpha, low, amb = o.attend(q[t - 1], np.tile(kk, (U, 1)), v[t - 1])
        n = len(live)
        np.testing.assert_allclose(alpha, 1.0 / n, atol=1e-15)
        for u in range(U):
            np.testing.assert_allclose(out[u], v[np.array(live) - 1, u].mean(0), atol=1e-13)
        if n < t:
            assert not low.any()
        o.record(low)
        if t > B + w:  # the window no longer reaches back to steps where n == t (alpha == 1/t ties)
            assert (o.counters() == 0).all()
            dropped = o.compress()
            if dropped is not None:
                assert (dropped == np.array(live[:m])).all()
                live = live[m:]
        else:
            dropped = o.compress()
            if dropped is not None:
                live = [p for p in live if p not in set(dropped[0].tolist())]
        assert (o.positions() == np.array(live)).all()


def test_dominant_key_takes_all_the_mass():
    T, d = 9, 8
    rng = np.random.default_rng(4)
    q = rng.standard_normal((T, 1, d))
    k = 0.01 * rng.standard_normal((T, 1, d))
    v = rng.standard_normal((T, 1, d))
    k[3, 0] = 200.0 * q[T - 1, 0] / np.linalg.norm(q[T - 1, 0])
    o = oracle.Oracle(1, 32, 1, 4, 1, d, scale=1.0)
    for t in range(T):
        out, alpha, low, amb = o.attend(q[t], k[t], v[t])
        o.record(low)
    np.testing.assert_allclose(out[0], v[3, 0], atol=1e-12)
    assert low[0].sum() == T - 1 and not low[0, 3]


# --- identities from the proof of Theorem 4.1 -----------------------------------
def test_renormalisation_identity_and_output_bound():
    # With S the kept set and beta the full-cache softmax of the same query,
    # alpha_j = beta_j / (1 - sum_{i not in S} beta_i), and
    # ||a_hat - b|| <= 2 max||v|| * sum_{i not in S} beta_i.
    T, U, d, B, r, w, m = 80, 2, 16, 12, 3, 6, 4
    q, k, v = _stream(T, U, d, 5, peaked=2.5)
    o = oracle.Oracle(U, B, r, w, m, d)
    scale = 1 / math.sqrt(d)
    for t in range(1, T + 1):
        out, alpha, low, amb = o.attend(q[t - 1], k[t - 1], v[t - 1])
        pos = o.positions()
        for u in range(U):
            b_out, beta = full_attention(q[t - 1, u], k[:t, u], v[:t, u], scale)
            kept = pos[u] - 1
            lost = 1.0 - beta[kept].sum()
            np.testing.assert_allclose(alpha[u], beta[kept] / (1.0 - lost), rtol=1e-11, atol=1e-15)
            vmax = np.linalg.norm(v[:t, u], axis=1).max()
            assert np.linalg.norm(out[u] - b_out) <= 2 * vmax * lost + 1e-12
        # the threshold is 1/t with t the stream position of the query, not 1/n
        assert (low == (alpha < 1.0 / t)).all()
        o.record(low)
        o.compress()
    assert o.n < t  # the run did compress


# --- the whole method against the brute force -----------------------------------
@pytest.mark.parametrize("B,r,w,m", [(8, 2, 4, 3), (10, 0, 3, 5), (9, 3, 20, 1), (7, 1, 1, 6), (12, 4, 7, 2)])
@pytest.mark.parametrize("seed", [0, 1])
def test_matches_bruteforce_on_tiny_streams(B, r, w, m, seed):
    T, U, d = 45, 2, 4
    q, k, v = _stream(T, U, d, 100 + seed, peaked=3.0)
    o = oracle.Oracle(U, B, r, w, m, d)
    bf = [BruteForceUnit(B, r, w, m, d, 1 / math.sqrt(d)) for _ in range(U)]
    n_compress = 0
    for t in range(T):
        out, alpha, low, amb = o.attend(q[t], k[t], v[t])
        o.record(low)
        I_before = o.counters()
        pos_before = o.positions()
        dropped = o.compress()
        for u in range(U):
            bout, balpha, bdropped = bf[u].step(q[t, u], k[t, u], v[t, u])
            np.testing.assert_allclose(out[u], bout, atol=1e-13)
            np.testing.assert_allclose(alpha[u], [balpha[p] for p in pos_before[u]], atol=1e-14)
            if bdropped is None:
                assert dropped is None
            else:
                assert dropped[u].tolist() == bdropped
            assert o.positions()[u].tolist() == sorted(bf[u].live)
        if dropped is not None:
            n_compress += 1
        # record by definition, evaluated after the step (and after any drop)
        I_now, pos_now = o.counters(), o.positions()
        for u in range(U):
            bI = bf[u].counters()
            assert I_now[u].tolist() == [bI[p] for p in pos_now[u]]
        assert o.n <= B and o.n < B  # never above budget; below it between steps (Definition 4.1)
    assert n_compress >= 5


def test_history_window_is_the_last_w_steps_and_w1_is_current_bit():
    T, U, d, B, r, m = 30, 1, 4, 64, 1, 1
    q, k, v = _stream(T, U, d, 7, peaked=3.0)
    lows = []
    o1 = oracle.Oracle(U, B, r, 1, m, d)
    o5 = oracle.Oracle(U, B, r, 5, m, d)
    for t in range(T):
        for o in (o1, o5):
            out, alpha, low, amb = o.attend(q[t], k[t], v[t])
            o.record(low)
        lows.append(low[0])
        assert (o1.counters()[0] == low[0].astype(int)).all()
        want = np.zeros(t + 1, dtype=int)
        for i in range(max(0, t - 4), t + 1):  # last 5 steps
            want[: i + 1] += lows[i].astype(int)
        assert (o5.counters()[0] == want).all()


# --- budget invariants -----------------------------------------------------------
@pytest.mark.parametrize("B,r,m", [(16, 4, 5), (16, 0, 16), (16, 15, 1), (5, 2, 3)])
def test_budget_sawtooth_and_recent_window_survives(B, r, m):
    T, U, d, w = 90, 2, 4, 6
    q, k, v = _stream(T, U, d, 8, peaked=2.0)
    o = oracle.Oracle(U, B, r, w, m, d)
    n_expect = 0
    for t in range(1, T + 1):
        n_expect += 1
        out, alpha, low, amb = o.attend(q[t - 1], k[t - 1], v[t - 1])
        assert o.n == n_expect <= B
        o.record(low)
        dropped = o.compress()
        if n_expect == B:
            assert dropped is not None and dropped.shape == (U, m)
            n_expect -= m
            # nothing from the r newest positions was dropped
            assert (dropped <= t - r).all()
        else:
            assert dropped is None
        pos = o.positions()
        assert pos.shape == (U, n_expect)
        assert (np.diff(pos, axis=1) > 0).all()           # order kept
        if r:
            assert (pos[:, -min(r, n_expect):] == np.arange(t - min(r, n_expect) + 1, t + 1)).all()
        assert o.n < B
    # m = 1 keeps exactly B-1 .. B tokens (the paper: "the cache will always maintain B tokens")
    if m == 1:
        assert o.n == B - 1


def test_step_on_full_cache_is_refused():
    o = oracle.Oracle(1, 4, 1, 2, 2, 4)
    z = np.zeros((1, 4))
    for _ in range(4):
        out, a, low, amb = o.attend(z, z, z)
        o.record(low)
    assert o.full
    with pytest.raises(RuntimeError):
        o.attend(z, z, z)
    assert o.compress() is not None and o.n == 2


def test_invalid_parameters():
    with pytest.raises(ValueError):
        oracle.Oracle(1, 8, 4, 2, 5, 4)     # m > B - r
    with pytest.raises(ValueError):
        oracle.Oracle(1, 8, 4, 0, 2, 4)     # w < 1
    with pytest.raises(ValueError):
        oracle.Oracle(1, 8, 1, 2, 2, 32, quant=True)


# --- selection -------------------------------------------------------------------
def _parse_golden(path):
    cases, cur = [], {}
    for line in open(path):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        key, val = [s.strip() for s in line.split("=")]
        if key == "I" and cur:
            cases.append(cur)
            cur = {}
        cur[key] = [int(x) for x in val.split()]
    cases.append(cur)
    return cases


def test_selection_hand_worked_examples():
    cases = _parse_golden(os.path.join(GOLDEN, "select_micro_example.txt"))
    assert len(cases) == 3 and sum("tie" in c for c in cases) == 1
    for c in cases:
        ev = oracle.select(c["I"], c["r"][0], c["m"][0], newest_first=bool(c.get("tie", [0])[0]))
        assert (ev + 1).tolist() == c["dropped_positions"]
        kept = [p for p in range(1, len(c["I"]) + 1) if p not in set((ev + 1).tolist())]
        assert kept == c["kept_positions"]


@pytest.mark.parametrize("seed", range(6))
def test_selection_is_the_unique_maximiser_over_all_subsets(seed):
    rng = np.random.default_rng(seed)
    n = int(rng.integers(5, 12))
    r = int(rng.integers(0, 4))
    m = int(rng.integers(1, n - r + 1))
    I = rng.integers(0, 4, size=n)  # few distinct values: many ties
    ev = oracle.select(I, r, m)
    key = [int(I[j]) * (n + 1) + (n - j) for j in range(n - r)]
    best = max(itertools.combinations(range(n - r), m), key=lambda s: sum(key[j] for j in s))
    assert ev.tolist() == sorted(best)
    kept_cand = [j for j in range(n - r) if j not in set(ev.tolist())]
    if kept_cand:
        assert I[ev].min() >= I[kept_cand].max()


# --- int4 group-64 store -----------------------------------------------------------
def _quant_ref(x):
    """Independent scalar float32 implementation of the store's rounding rule."""
    x = np.asarray(x, dtype=np.float32)
    rows, d = x.shape
    out = np.zeros((rows, d), dtype=np.float64)
    codes = np.zeros((rows, d), dtype=np.int8)
    scales = np.zeros((rows, d // 64), dtype=np.float32)
    seven = np.float32(7.0)
    for i in range(rows):
        for g in range(d // 64):
            grp = x[i, g * 64:(g + 1) * 64]
            a = np.float32(np.abs(grp).max())
            sc = np.float32(np.float16(a / seven))
            scales[i, g] = sc
            for e in range(64):
                c = 0
                if sc != 0:
                    c = int(np.clip(np.rint(np.float32(grp[e] / sc)), -7, 7))
                codes[i, g * 64 + e] = c
                out[i, g * 64 + e] = float(c) * float(sc)
    return out, codes, scales


def test_int4_quantiser_matches_independent_implementation_and_error_bound():
    rng = np.random.default_rng(11)
    x = rng.standard_normal((37, 128)).astype(np.float16).astype(np.float64)
    x[3] = 0.0
    x[4, :64] *= 1e-6      # tiny group: fp16 subnormal scale
    x[5, 7] = 60000.0      # near the top of fp16
    x = x.astype(np.float16).astype(np.float64)
    stored, codes, scales = oracle.quantize_int4_g64(x)
    rs, rc, rsc = _quant_ref(x)
    assert (codes == rc).all() and (scales == rsc).all() and (stored == rs).all()
    assert np.abs(codes).max() <= 7
    sc_full = np.repeat(scales.astype(np.float64), 64, axis=1)
    assert (np.abs(x - stored) <= sc_full / 2 + 1e-12 + np.abs(x) * 2e-3).all()
    assert (stored[3] == 0).all()


def test_int4_store_attends_over_dequantised_rows():
    T, U, d = 20, 2, 64
    rng = np.random.default_rng(12)
    q, k, v = (rng.standard_normal((T, U, d)).astype(np.float16).astype(np.float64) for _ in range(3))
    o = oracle.Oracle(U, 64, 2, 4, 2, d, quant=True)
    for t in range(T):
        out, _ = o.step(q[t], k[t], v[t])
    for u in range(U):
        Kq, _, _ = _quant_ref(k[:, u])
        Vq, _, _ = _quant_ref(v[:, u])
        K, V = o.cache(u)
        assert (K == Kq).all() and (V == Vq).all()
        ref, _ = full_attention(q[T - 1, u], Kq, Vq, 1 / math.sqrt(d))
        np.testing.assert_allclose(out[u], ref, atol=1e-13)


def test_ambiguity_flag_marks_scores_near_the_threshold():
    # two equal keys at t = 2: alpha = 1/2 = 1/t exactly -> not low (strict <), flagged ambiguous
    o = oracle.Oracle(1, 8, 1, 4, 1, 4)
    kk = np.ones((1, 4))
    out, alpha, low, amb = o.attend(kk, kk, kk)
    o.record(low)
    out, alpha, low, amb = o.attend(kk, kk, kk)
    assert not low.any() and amb.all()


def _stream_with_scores(p):
    """A stream of t = len(p) tokens whose last query sees exactly the scores p (sum 1): key j is
    log(p_j) times the j-th unit vector, the last query is all ones, scale 1.  Returns (q, k, v)
    as [t, 1, t] arrays."""
    t = len(p)
    k = np.zeros((t, 1, t))
    k[np.arange(t), 0, np.arange(t)] = np.log(p)
    q = np.zeros((t, 1, t))
    q[t - 1] = 1.0
    return q, k, np.zeros((t, 1, t))


@pytest.mark.parametrize("t", [2, 5, 37])
@pytest.mark.parametrize("delta,flagged", [(0.0, True), (5e-7, True), (-5e-7, True), (0.99e-6, True), (-0.99e-6, True),
                                           (1.01e-6, False), (-1.01e-6, False), (2e-6, False), (-2e-6, False),
                                           (1e-3, False)])
def test_ambiguity_window_is_one_millionth_wide(t, delta, flagged):
    # The benchmark definition lets an fp32 implementation disagree with the fp64 comparison
    # alpha < 1/t only where alpha lies within 1e-6 of 1/t.  Scores are planted exactly: slot 0 gets
    # 1/t + delta, slot 1 gets 1/t + 3e-3 (well outside), the rest share what is left.
    assert oracle._load().sho_amb_window() == 1e-6 == oracle.AMB_WINDOW
    p = np.full(t, 0.0)
    p[0] = 1.0 / t + delta
    if t > 2:
        p[1] = 1.0 / t + 3e-3
        p[2:] = (1.0 - p[0] - p[1]) / (t - 2)
    else:
        p[1] = 1.0 - p[0]
    q, k, v = _stream_with_scores(p)
    o = oracle.Oracle(1, t + 1, 0, 4, 1, t, scale=1.0)
    for s in range(t):
        out, alpha, low, amb = o.attend(q[s], k[s], v[s])
        o.record(low)
    np.testing.assert_allclose(alpha[0], p, rtol=0, atol=1e-15)
    assert bool(amb[0, 0]) == flagged
    if delta != 0.0:
        assert bool(low[0, 0]) == (delta < 0)                  # strict comparison, in fp64
    if t > 2:
        assert not amb[0, 1] and not low[0, 1]
        assert bool(amb[0, 2]) == (abs(p[2] - 1.0 / t) <= 1e-6)
    # the same query scored again by the recompute-at-compression variant carries the same flag
    a2, low2, amb2, steps = o.recount()
    row = t % 4
    assert steps[row] == t
    np.testing.assert_allclose(a2[0, row], p, rtol=0, atol=1e-15)
    assert bool(amb2[0, row, 0]) == flagged and (delta == 0.0 or bool(low2[0, row, 0]) == (delta < 0))
    if t > 2:
        assert not amb2[0, row, 1]


# --- the record recomputed at compression time -------------------------------------------
def test_recount_matches_causal_attention_of_stored_queries_over_the_kept_set():
    # From the definition: each of the last w queries against the tokens still cached that
    # existed at its step, softmax over those, compared with 1/step.
    T, U, d, B, r, w, m = 70, 2, 8, 14, 3, 9, 5
    q, k, v = _stream(T, U, d, 21, peaked=2.5)
    o = oracle.Oracle(U, B, r, w, m, d)
    scale = 1 / math.sqrt(d)
    n_compress = 0
    for t in range(1, T + 1):
        out, alpha, low, amb = o.attend(q[t - 1], k[t - 1], v[t - 1])
        if o.full:
            a, lo, am, steps = o.recount()
            pos = o.positions()
            window = [s for s in range(max(1, t - w + 1), t + 1)]
            assert sorted(int(x) for x in steps if x) == window
            for u in range(U):
                for s in window:
                    row = s % w
                    vis = pos[u] <= s
                    _, beta = full_attention(q[s - 1, u], k[pos[u][vis] - 1, u], v[pos[u][vis] - 1, u], scale)
                    np.testing.assert_allclose(a[u, row][vis], beta, rtol=1e-11, atol=1e-15)
                    assert (a[u, row][~vis] == 0).all() and not lo[u, row][~vis].any()
                    assert (lo[u, row][vis] == (beta < 1.0 / s)).all()
            o.set_record(lo, steps)
            # counters now count the recomputed flags, by definition
            I = o.counters()
            for u in range(U):
                want = sum(lo[u, s % w].astype(int) for s in window)
                assert (I[u] == want).all()
            dropped = o.compress()
            assert dropped is not None and (dropped <= t - r).all()
            n_compress += 1
    assert n_compress >= 10


def test_step_recompute_keeps_the_budget_and_full_attention_when_it_never_fills():
    T, U, d = 30, 2, 8
    q, k, v = _stream(T, U, d, 22, peaked=2.0)
    o = oracle.Oracle(U, T + 1, 2, 6, 3, d)
    for t in range(T):
        out, dropped = o.step_recompute(q[t], k[t], v[t])
        assert dropped is None
    ref, _ = full_attention(q[T - 1, 0], k[:, 0], v[:, 0], 1 / math.sqrt(d))
    np.testing.assert_allclose(out[0], ref, atol=1e-13)
    o2 = oracle.Oracle(U, 10, 2, 6, 3, d)
    for t in range(T):
        o2.step_recompute(q[t], k[t], v[t])
        assert o2.n < 10


# --- alternative readings of the paper (oracle only) ------------------------------------------------
@pytest.mark.parametrize("reading", [dict(threshold=1), dict(threshold=2), dict(window_plus1=True), dict(tie_newest=True),
                                     dict(trigger_literal=True),
                                     dict(threshold=1, window_plus1=True, tie_newest=True, trigger_literal=True)])
@pytest.mark.parametrize("B,r,w,m", [(8, 2, 4, 3), (9, 3, 20, 1), (7, 1, 1, 6), (12, 4, 7, 2)])
def test_alternative_readings_match_bruteforce(reading, B, r, w, m):
    # Algorithm 2's fixed threshold 1/t of the compression step, the 1/n threshold, the w+1-step window,
    # newest-first ties and Algorithm 1's literal "n > B" trigger, each against the brute force that
    # evaluates the same reading from the full table of scores.
    T, U, d = 45, 2, 4
    q, k, v = _stream(T, U, d, 300 + B, peaked=3.0)
    o = oracle.Oracle(U, B, r, w, m, d, **reading)
    bf = [BruteForceUnit(B, r, w, m, d, 1 / math.sqrt(d), **reading) for _ in range(U)]
    cap = B + (1 if reading.get("trigger_literal") else 0)
    n_compress = 0
    for t in range(T):
        out, alpha, low, amb = o.attend(q[t], k[t], v[t])
        o.record(low)
        pos_before = o.positions()
        assert o.n <= cap
        dropped = o.compress()
        for u in range(U):
            bout, balpha, bdropped = bf[u].step(q[t, u], k[t, u], v[t, u])
            np.testing.assert_allclose(out[u], bout, atol=1e-13)
            np.testing.assert_allclose(alpha[u], [balpha[p] for p in pos_before[u]], atol=1e-14)
            assert (dropped is None) == (bdropped is None)
            if bdropped is not None:
                assert dropped[u].tolist() == bdropped
            assert o.positions()[u].tolist() == sorted(bf[u].live)
            bI = bf[u].counters()
            assert o.counters()[u].tolist() == [bI[p] for p in o.positions()[u]]
        n_compress += dropped is not None
        assert o.n < cap
    assert n_compress >= 5


@pytest.mark.parametrize("reading", [dict(), dict(tie_newest=True), dict(trigger_literal=True)])
@pytest.mark.parametrize("p,B,r,w,m", [(30, 8, 2, 5, 3), (23, 12, 4, 40, 2), (9, 9, 3, 4, 1), (7, 9, 3, 4, 1)])
def test_bulk_prompt_reading_matches_bruteforce(reading, p, B, r, w, m):
    # Prompt cached in full (Section 2), record from its last w steps, then Algorithm 2 in rounds until the
    # cache is under budget; generation continues from there.  Brute force: full attention over the
    # prompt, one sort for the rounds, then its usual steps.
    T, U, d = p + 25, 2, 4
    q, k, v = _stream(T, U, d, 400 + p, peaked=3.0)
    src = oracle.Oracle(U, p + 1, 0, w, 1, d, **{kk: vv for kk, vv in reading.items() if kk != "trigger_literal"})
    bf = [BruteForceUnit(10 ** 6, r, w, m, d, 1 / math.sqrt(d), **reading) for _ in range(U)]
    for t in range(p):
        out, dropped = src.step(q[t], k[t], v[t])
        assert dropped is None
        for u in range(U):
            bout, _, _ = bf[u].step(q[t, u], k[t, u], v[t, u])
            np.testing.assert_allclose(out[u], bout, atol=1e-13)       # full causal attention over the prompt
    dst = oracle.Oracle(U, B, r, w, m, d, **reading)
    rounds = dst.import_compressed(src)
    cap = B + (1 if reading.get("trigger_literal") else 0)
    want_rounds = 0 if p < cap else (p - cap) // m + 1
    assert rounds == want_rounds and dst.n == p - rounds * m < cap and dst.t == p
    for u in range(U):
        brounds, _gone = bf[u].shrink_below(B, m, r)
        bf[u].B = B
        assert brounds == rounds
        assert dst.positions()[u].tolist() == sorted(bf[u].live)
        bI = bf[u].counters()
        assert dst.counters()[u].tolist() == [bI[pp] for pp in dst.positions()[u]]
        if r:
            assert set(range(p - min(r, dst.n) + 1, p + 1)) <= set(dst.positions()[u].tolist())
    for t in range(p, T):                                               # generation goes on as usual
        out, dropped = dst.step(q[t], k[t], v[t])
        for u in range(U):
            bout, _, bdropped = bf[u].step(q[t, u], k[t, u], v[t, u])
            np.testing.assert_allclose(out[u], bout, atol=1e-13)
            assert (dropped is None) == (bdropped is None)
            assert dst.positions()[u].tolist() == sorted(bf[u].live)
