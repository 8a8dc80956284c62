"""Pins for the CPU oracle: each test fixes the oracle to something other than itself
(hand arithmetic, brute force, a lemma, a closed form, the paper's printed table)."""
import dataclasses
import math
import os

import numpy as np
import pytest

from oracle import routerelay_oracle as O
from paper_2609_07306_b200 import workload as W


def _params(w, **kw):
    base = dict(n_q=w.n_q, n_k=w.n_k, k=w.k, m=w.m, r=w.r, gamma=w.gamma, causal=w.causal,
                causal_offset=0, seed=w.seed)
    base.update(kw)
    return O.OracleParams(**base)


def _load_rows(path):
    rows = []
    with open(path) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                rows.append(line.split())
    return rows


# ------------------------------------------------------------------ Eq. 1
def test_scores_hand_computed():
    # Eq. 1 on a 2x3 problem with d=2, worked by hand:
    q = np.array([[1.0, 2.0], [-1.0, 0.5]])
    k = np.array([[3.0, 4.0], [0.0, -1.0], [2.0, 2.0]])
    p = O.OracleParams(n_q=2, n_k=3, k=1, m=1, r=0)
    s = O.scores(q, k, p)
    expect = np.array([[11.0, -2.0, 6.0], [-1.0, -0.5, -1.0]])
    assert np.array_equal(s, expect)
    # transposed operands or a 1/sqrt(d) factor would give different numbers
    assert s[0, 0] == 1 * 3 + 2 * 4


def test_scores_causal_mask_and_offset():
    q = np.ones((4, 2))
    k = np.ones((4, 2))
    s = O.scores(q, k, O.OracleParams(n_q=4, n_k=4, k=1, m=0, r=0, causal=True))
    for i in range(4):
        assert np.all(s[i, : i + 1] == 2.0) and np.all(np.isneginf(s[i, i + 1:]))
    s = O.scores(q[:2], k, O.OracleParams(n_q=2, n_k=4, k=1, m=0, r=0, causal=True,
                                           causal_offset=2))
    assert np.isfinite(s[0]).sum() == 3 and np.isfinite(s[1]).sum() == 4


# ------------------------------------------------------------------ Eq. 2 + Sec 3.1 near-miss
def _brute_rank(s_row, v):
    return [j for _, j in sorted((-float(s_row[j]), j) for j in range(v))]


@pytest.mark.parametrize("seed", range(6))
def test_topk_nearmiss_bruteforce(seed):
    rng = np.random.default_rng(seed)
    n_k = int(rng.integers(3, 17))
    # coarse values force many exact ties
    s_row = rng.integers(-3, 4, size=n_k).astype(np.float64) / 4.0
    for v in range(1, n_k + 1):
        brute = _brute_rank(s_row, v)
        assert list(O.rank_order(s_row, v)) == brute
        for k in range(1, n_k + 1):
            for m in (0, 1, 3):
                p = O.OracleParams(n_q=1, n_k=n_k, k=k, m=m, r=0)
                route, sent, kth, margin = O.route_row(s_row, v, p, g=0, layer=0)
                kk = min(k, v)
                assert [j for j in route if j >= 0] == brute[:kk]
                assert [j for j in sent if j >= 0] == brute[kk:kk + m]
                assert kth == s_row[brute[kk - 1]]
                if v > kk:
                    assert margin == s_row[brute[kk - 1]] - s_row[brute[kk]]
                    # Sec 3.3: min selected - max unselected
                    assert margin == min(s_row[j] for j in brute[:kk]) - \
                        max(s_row[j] for j in brute[kk:v])
                else:
                    assert margin == float("inf")


def test_topk_matches_library_when_no_ties():
    rng = np.random.default_rng(7)
    s = rng.standard_normal((32, 200))
    for i in range(32):
        lib = set(np.argpartition(-s[i], 12)[:12].tolist())
        assert set(O.full_route(s[i], 200, 12).tolist()) == lib


def test_negative_zero_ties_with_positive_zero():
    q = np.array([[0.0, 1.0]])
    k = np.array([[-1.0, 0.0], [1.0, 0.0], [0.0, -1.0]])     # scores: -0.0, +0.0, -1
    p = O.OracleParams(n_q=1, n_k=3, k=1, m=1, r=0)
    s = O.scores(q, k, p)
    assert list(O.rank_order(s[0], 3)) == [0, 1, 2]           # tie -> smaller index first


# ------------------------------------------------------------------ Lemma 1
@pytest.mark.parametrize("seed", range(5))
def test_lemma1_margin_stability(seed):
    rng = np.random.default_rng(100 + seed)
    n_k, k, m, r = 96, 8, 4, 4
    p = O.OracleParams(n_q=1, n_k=n_k, k=k, m=m, r=r, seed=seed)
    s_row = rng.standard_normal(n_k)
    route, sent, kth, margin = O.route_row(s_row, n_k, p, g=3, layer=0)
    assert margin > 0
    # any perturbation with sup-norm < margin/2 keeps the route and does not trigger
    for _ in range(20):
        e = rng.uniform(-1, 1, n_k)
        e *= 0.49 * margin / np.abs(e).max()
        s2 = s_row + e
        assert set(O.full_route(s2, n_k, k)) == set(route)
        led = O.Ledger.empty(1, p)
        led.routes[0], led.sentinels[0], led.ages[0] = route, sent, 0
        _, a, b, _ = O.candidate_scores(s2[None, :], led.routes, led.sentinels)
        assert a[0] > b[0]
    # adversarial perturbation just above margin/2 on the k-th / (k+1)-th pair flips the set
    order = O.rank_order(s_row, n_k)
    e = np.zeros(n_k)
    e[order[k - 1]] = -0.51 * margin
    e[order[k]] = +0.51 * margin
    s3 = s_row + e
    assert set(O.full_route(s3, n_k, k)) != set(route)
    _, a, b, _ = O.candidate_scores(s3[None, :], route[None, :], sent[None, :])
    assert not (a[0] > b[0])          # and the near-miss sentinel catches it


def test_lemma1_query_level_perturbation():
    rng = np.random.default_rng(5)
    d, n_k, k = 16, 64, 6
    kk = rng.standard_normal((n_k, d))
    q = rng.standard_normal((1, d))
    p = O.OracleParams(n_q=1, n_k=n_k, k=k, m=3, r=0)
    s = O.scores(q, kk, p)
    route, _, _, margin = O.route_row(s[0], n_k, p, 0, 0)
    dq = rng.standard_normal((1, d))
    # |dq . k_j| <= ||dq|| max||k_j|| = eps < margin/2
    dq *= 0.49 * margin / (np.linalg.norm(dq) * np.linalg.norm(kk, axis=1).max())
    s2 = O.scores(q + dq, kk, p)
    assert np.abs(s2 - s).max() <= 0.5 * margin
    assert set(O.full_route(s2[0], n_k, k)) == set(route)


# ------------------------------------------------------------------ trigger invariants
def _run(w, problems, **over):
    q, k = W.generate(w, problems=problems)
    p = _params(w, **over)
    res, summ = O.run_layers(W.as_float32(q), W.as_float32(k), p, w.anchor_every,
                             problem_ids=problems, keep_scores=True)
    return p, res, summ


@pytest.mark.parametrize("wl,problems", [(W.tiny(), [0]), (W.moderate(), [0, 5])])
def test_trigger_invariants(wl, problems):
    p, res, summ = _run(wl, problems)
    v = np.tile(p.valid_counts(), len(problems))
    lost_on_flagged = 0
    for l in range(1, len(res)):
        cur, prev = res[l], res[l - 1]
        if cur.is_anchor:
            assert np.all(cur.flags == 1) and np.all(cur.ledger.ages == 0)
            assert len(cur.refresh_rows) == len(v)
            continue
        stable = cur.flags == 0
        # (i) unflagged: route and sentinels relayed bit-identically, age advances
        assert np.array_equal(cur.ledger.routes[stable], prev.ledger.routes[stable])
        assert np.array_equal(cur.ledger.sentinels[stable], prev.ledger.sentinels[stable])
        assert np.array_equal(cur.ledger.ages[stable], prev.ledger.ages[stable] + 1)
        # (ii) flagged: route = exact TopK of this layer, age 0
        fl = ~stable
        assert np.array_equal(cur.ledger.routes[fl], cur.full_routes[fl])
        assert np.all(cur.ledger.ages[fl] == 0)
        # compaction order: ascending ids of the flagged rows, nothing else
        assert np.array_equal(cur.refresh_rows, np.nonzero(cur.flags)[0])
        # (iii) gamma = 0: a flagged row's exact TopK differs from the stale route unless an
        # exact tie sits on the boundary (no false positives of the trigger)
        for gr in np.nonzero(fl)[0]:
            if cur.alpha[gr] == cur.beta[gr]:
                continue
            old = set(int(j) for j in prev.ledger.routes[gr] if j >= 0)
            new = set(int(j) for j in cur.full_routes[gr] if j >= 0)
            assert old != new
        # rows that can select everything they see carry no sentinels and never flag
        assert not np.any(cur.flags[v <= p.k])
        # (iv) recall is lost on unflagged rows only
        h, t = O.recall_counts(cur.ledger.routes[fl], cur.full_routes[fl])
        lost_on_flagged += t - h
    assert lost_on_flagged == 0
    assert 0.0 < summ.flagged_relay_fraction < 1.0
    assert summ.recall_all >= summ.recall_relay * (1 - 1e-12) or summ.recall_relay == 1.0


def test_no_sentinels_is_fixed_stride_reuse():
    # m = r = 0: nothing can challenge -> pure reuse between anchors ("fixed stride")
    w = W.tiny().replace(m=0, r=0)
    p, res, summ = _run(w, [0])
    assert summ.flagged_relay_fraction == 0.0
    for l in range(1, len(res)):
        assert np.array_equal(res[l].ledger.routes, res[0].ledger.routes)
        assert np.all(res[l].ledger.ages == l)


def test_infinite_guard_margin_is_route_every_layer():
    w = W.tiny()
    p, res, summ = _run(w, [0], gamma=float("inf"))
    assert summ.recall_all == 1.0
    for l in range(1, len(res)):
        assert np.all(res[l].flags == 1)
        assert np.array_equal(res[l].ledger.routes, res[l].full_routes)


def test_zero_drift_never_flags():
    w = W.tiny().replace(rho=0.0)
    p, res, summ = _run(w, [0])
    assert summ.flagged_relay_fraction == 0.0 and summ.recall_all == 1.0
    for l in range(1, len(res)):
        assert np.array_equal(res[l].ledger.routes, res[0].ledger.routes)


def test_flagged_fraction_grows_with_drift():
    fr = []
    for rho in (0.01, 0.05, 0.2):
        _, _, summ = _run(W.tiny().replace(rho=rho), [0])
        fr.append(summ.flagged_relay_fraction)
    assert fr[0] <= fr[1] <= fr[2] and fr[0] < fr[2]


# ------------------------------------------------------------------ random sentinels
def test_finaliser_published_vectors(golden_dir):
    vec = [int(r[0]) for r in _load_rows(os.path.join(golden_dir, "splitmix64_vectors.txt"))]
    state = 1234567
    for expect in vec:
        state = (state + 0x9E3779B97F4A7C15) & ((1 << 64) - 1)
        assert O.fmix64(state) == expect


def test_sampler_invariants_and_small_pools():
    for v in range(1, 40):
        for n_ex in range(0, min(v, 20) + 1):
            excluded = list(range(0, 2 * n_ex, 2))[:n_ex]
            excluded = [j for j in excluded if j < v]
            pool = [j for j in range(v) if j not in excluded]
            for r in (0, 1, 4, 9):
                out = O.draw_random_sentinels(excluded, v, r, seed=3, g=v * 131 + n_ex, layer=2)
                assert len(out) == min(r, len(pool))
                assert len(set(out)) == len(out)
                assert all(0 <= j < v and j not in excluded for j in out)
                if len(pool) <= r:
                    assert out == pool          # whole pool, ascending, no RNG involved


def test_sampler_depends_on_seed_row_layer():
    ex = list(range(12))
    a = O.draw_random_sentinels(ex, 512, 8, 1, 10, 3)
    assert a != O.draw_random_sentinels(ex, 512, 8, 2, 10, 3)
    assert a != O.draw_random_sentinels(ex, 512, 8, 1, 11, 3)
    assert a != O.draw_random_sentinels(ex, 512, 8, 1, 10, 4)
    assert a == O.draw_random_sentinels(ex, 512, 8, 1, 10, 3)


def test_sampler_uniform_and_miss_probability():
    """Eq. 6: P(miss) = C(N-u, r) / C(N, r) for r draws without replacement from a pool of N
    that hides u challengers; plus chi-square uniformity over the pool."""
    from scipy import stats
    v, r, u = 64, 8, 5
    excluded = list(range(0, 32, 2))                 # 16 excluded -> N = 48
    pool = [j for j in range(v) if j not in excluded]
    N = len(pool)
    challengers = set(pool[3::10][:u])
    assert len(challengers) == u
    rows = 30000
    counts = dict.fromkeys(pool, 0)
    miss = 0
    for g in range(rows):
        out = O.draw_random_sentinels(excluded, v, r, seed=11, g=g, layer=1)
        for j in out:
            counts[j] += 1
        miss += not challengers.intersection(out)
    p_exact = math.comb(N - u, r) / math.comb(N, r)
    assert p_exact <= (1 - u / N) ** r                # the paper's upper bound
    sigma = math.sqrt(p_exact * (1 - p_exact) / rows)
    assert abs(miss / rows - p_exact) < 4 * sigma
    chi2 = stats.chisquare(list(counts.values()))
    assert chi2.pvalue > 1e-4
    # a sampler that drew WITH replacement would have a visibly different miss rate
    assert abs((1 - u / N) ** r - p_exact) > 8 * sigma


# ------------------------------------------------------------------ work accounting
def test_score_pair_definition_matches_paper_table(golden_dir):
    """The paper's sentinel-ablation table fixes what 'score pairs' and 'rerouted rows'
    count: given its rerouted-row column, the accounting must reproduce its score-pair
    column (values printed to 0.1 %)."""
    L, n, k = 24, 256, 12
    for m, r, rer_pct, pairs_pct in _load_rows(os.path.join(golden_dir,
                                                            "sentinel_ablation_table.txt")):
        m, r, rer_pct, pairs_pct = int(m), int(r), float(rer_pct), float(pairs_pct)
        p = O.OracleParams(n_q=n, n_k=n, k=k, m=m, r=r)
        flagged_total = int(round(rer_pct / 100 * L * n - n))
        kinds = [True] + [False] * (L - 1)
        flags = [np.ones(n, np.uint8)]
        left = flagged_total
        for l in range(1, L):
            f = np.zeros(n, np.uint8)
            take = min(n, -(-left // (L - l)))
            f[:take] = 1
            left -= take
            flags.append(f)
        cc = [None] + [np.full(n, p.c)] * (L - 1)
        c = O.work_counters(p, 1, kinds, flags, cc)
        rerouted, flagged, pairs = O.fractions_from_counters(c)
        assert abs(100 * rerouted - rer_pct) < 0.06
        assert abs(100 * pairs - pairs_pct) < 0.06, (m, r, 100 * pairs)


def test_ledger_size(golden_dir):
    (n_q, c, nbytes), = _load_rows(os.path.join(golden_dir, "ledger_size.txt"))
    p = O.OracleParams(n_q=int(n_q), n_k=4096, k=32, m=16, r=16)
    assert p.c == int(c)
    assert O.Ledger.empty(int(n_q), p).index_bytes() == int(nbytes)


def test_counters_consistent_with_run():
    w = W.moderate()
    p, res, summ = _run(w, [1])
    c = summ.counters
    v = p.valid_counts()
    n_anchor = sum(r.is_anchor for r in res)
    assert c["anchor_rows"] == n_anchor * w.n_q
    assert c["dense_pairs"] == len(res) * int(v.sum())
    assert c["flagged_rows"] == sum(int(r.flags.sum()) for r in res if not r.is_anchor)
    # causal rows with v_i <= k have v_i candidates, later rows up to c
    first_relay = res[1]
    assert first_relay.cand_scores.shape == (w.n_q, w.c)
    assert np.isfinite(first_relay.cand_scores[0]).sum() == 1
    assert np.isfinite(first_relay.cand_scores[-1]).sum() == w.c


def test_token_ranges():
    routes = np.array([[5, 2, -1], [0, 7, 3]], np.int32)
    tr = O.token_ranges(routes, 64)
    assert tr[0].tolist() == [[128, 192], [320, 384], [-1, -1]]
    assert tr[1].tolist() == [[0, 64], [192, 256], [448, 512]]
    # coalesced: runs of consecutive chunks merge (hand-worked: {3,4,5}, {9}, {11,12}, T = 10)
    routes = np.array([[12, 3, 9, 5, 4, 11, -1]], np.int32)
    tr = O.token_ranges(routes, 10, coalesce=True)
    assert tr[0].tolist() == [[30, 60], [90, 100], [110, 130], [-1, -1], [-1, -1], [-1, -1], [-1, -1]]
    assert O.token_ranges(routes, 10)[0, :6].tolist() == [[30, 40], [40, 50], [50, 60], [90, 100],
                                                         [110, 120], [120, 130]]


def test_relay_requires_anchor():
    p = O.OracleParams(n_q=4, n_k=4, k=1, m=1, r=0)
    with pytest.raises(ValueError):
        O.relay_layer(O.Ledger.empty(4, p), np.ones((1, 4, 2)), np.ones((1, 4, 2)), p, 1)


# ---------------------------------------------------------------- optional policies
def test_global_sentinels_hand_case():
    """Sink (chunk 0) and most recent chunk (v - 1) are sentinels unless already in the route
    or among the near-miss ones; the random draw avoids them (Section 3.1, item 3)."""
    # one row, 8 chunks, scores descending in the order 3,4,0,7,1,2,5,6
    s = np.full(8, -np.inf)
    for rank, j in enumerate([3, 4, 0, 7, 1, 2, 5, 6]):
        s[j] = 10.0 - rank
    p = O.OracleParams(n_q=1, n_k=8, k=2, m=1, r=2, global_sentinels=3)
    route, sent, kth, margin = O.route_row(s, 8, p, g=0, layer=0)
    assert set(route) == {3, 4}
    assert sent[0] == 0                       # near-miss: rank 3 is chunk 0 ...
    assert sent[3] == -1 and sent[4] == 7     # ... so the sink slot stays empty; recent = 7
    rnd = [int(x) for x in sent[1:3]]
    assert len(set(rnd)) == 2 and not (set(rnd) & {3, 4, 0, 7}) and all(0 <= x < 8 for x in rnd)
    # sink not in route or near-miss: it takes its slot
    p2 = O.OracleParams(n_q=1, n_k=8, k=2, m=0, r=0, global_sentinels=3)
    _, sent2, _, _ = O.route_row(s, 8, p2, g=0, layer=0)
    assert list(sent2) == [0, 7]
    # a row that sees one chunk: it is the route, nothing is left
    _, sent3, _, _ = O.route_row(s, 1, p2, g=0, layer=0)
    assert list(sent3) == [-1, -1]
    # sink and recent coincide (v = 1 is covered above; v = 3 with route {0,...}): no duplicate
    p4 = O.OracleParams(n_q=1, n_k=8, k=1, m=0, r=0, global_sentinels=3)
    s4 = np.array([1.0, 5.0, -np.inf, -np.inf, -np.inf, -np.inf, -np.inf, -np.inf])
    _, sent4, _, _ = O.route_row(s4, 2, p4, g=0, layer=0)
    assert list(sent4) == [0, -1]             # route {1}; sink 0; recent = 1 is in the route


def _one_row_ledger(p, route, sent, age, margin):
    led = O.Ledger.empty(1, p)
    led.routes[0, :len(route)] = route
    led.sentinels[0, :len(sent)] = sent
    led.ages[0] = age
    led.margin[0] = margin
    return led


def test_hysteresis_and_forced_rerouting_hand_case():
    """d = 1, q = 1: scores are the key values.  alpha - beta = 0.5."""
    q = np.ones((1, 1, 1)); k = np.array([[[3.0], [2.5], [1.0]]])
    base = dict(n_q=1, n_k=3, k=1, m=1, r=0)
    # plain Eq. 5 with gamma = 0: reuse
    p = O.OracleParams(**base)
    led = _one_row_ledger(p, [0], [1], age=2, margin=0.1)
    assert O.relay_layer(led, q, k, p, 1).flags[0] == 0
    # larger guard margin while the recorded margin is below the recovery level
    p = O.OracleParams(**base, gamma_boost=1.0, margin_recover=0.2)
    assert O.relay_layer(led, q, k, p, 1).flags[0] == 1
    led_ok = _one_row_ledger(p, [0], [1], age=2, margin=0.3)
    assert O.relay_layer(led_ok, q, k, p, 1).flags[0] == 0
    # minimum reuse horizon: a row routed at the previous layer (age 0) is not tested
    p = O.OracleParams(**base, gamma=1.0, min_reuse=1)
    fresh = _one_row_ledger(p, [0], [1], age=0, margin=0.1)
    res = O.relay_layer(fresh, q, k, p, 1)
    assert res.flags[0] == 0 and res.ledger.ages[0] == 1
    assert O.relay_layer(res.ledger, q, k, p, 2).flags[0] == 1      # tested one layer later
    # forced re-routing: the route is h_max layers old
    p = O.OracleParams(**base, h_max=3)
    assert O.relay_layer(_one_row_ledger(p, [0], [1], age=2, margin=9.0), q, k, p, 1).flags[0] == 0
    res = O.relay_layer(_one_row_ledger(p, [0], [1], age=3, margin=9.0), q, k, p, 1)
    assert res.flags[0] == 1 and res.ledger.ages[0] == 0


def test_forced_rerouting_period_closed_form():
    """With nothing to challenge a route (m = r = 0) and h_max = 2, one anchor at layer 0:
    every row is re-routed exactly at layers 3, 6, 9, ... and nowhere else."""
    w = W.tiny().replace(m=0, r=0, layers=10, anchor_every=100, h_max=2)
    q, k = W.generate(w)
    p = O.OracleParams(n_q=w.n_q, n_k=w.n_k, k=w.k, m=0, r=0, h_max=2)
    res, _ = O.run_layers(W.as_float32(q).astype(np.float64), W.as_float32(k).astype(np.float64),
                          p, w.anchor_every)
    for l in range(1, w.layers):
        assert res[l].flags.all() == (l % 3 == 0) and res[l].flags.any() == (l % 3 == 0)
        if l % 3 == 0:
            assert np.array_equal(res[l].ledger.routes, res[l].full_routes)
    assert max(int(r_.ledger.ages.max()) for r_ in res) == 2


def test_minimum_reuse_horizon_invariant():
    """A row re-routed at layer l is never flagged at layer l + 1 when min_reuse = 1."""
    w = W.moderate().replace(heads=2, layers=8, anchor_every=100, rho=0.3, min_reuse=1)
    q, k = W.generate(w)
    p = O.OracleParams(n_q=w.n_q, n_k=w.n_k, k=w.k, m=w.m, r=w.r, causal=True, min_reuse=1)
    res, _ = O.run_layers(W.as_float32(q).astype(np.float64), W.as_float32(k).astype(np.float64),
                          p, w.anchor_every)
    assert res[1].flags.sum() == 0                       # the layer after the anchor
    seen = 0
    for l in range(2, w.layers):
        both = (res[l - 1].flags != 0) & (res[l].flags != 0)
        assert not both.any()
        seen += int(res[l].flags.sum())
    assert seen > 0


# ------------------------------------------------------------------ recall and run-level accounting
def test_recall_counts_partial_overlap_hand_case():
    """Section 5: recall compares the reused chunk ids with the exact per-layer top-k.
    Hand-worked rows with partial overlap, -1 padding on either side and different valid widths."""
    routes = np.array([[3, 5, -1], [0, 1, 2], [4, -1, -1], [7, 8, 9]], np.int32)
    full = np.array([[5, 7, -1], [2, 1, 0], [4, -1, -1], [1, 2, -1]], np.int32)
    # row 0: {3,5} vs {5,7} -> 1 of 2; row 1: 3 of 3; row 2: 1 of 1; row 3: {7,8,9} vs {1,2} -> 0 of 2
    assert O.recall_counts(routes, full) == (5, 8)
    # the denominator is the size of the exact set, not of the reused one
    assert O.recall_counts(np.array([[1, 2, 3]], np.int32), np.array([[3, -1, -1]], np.int32)) == (1, 1)
    assert O.recall_counts(np.array([[3, -1, -1]], np.int32), np.array([[1, 2, 3]], np.int32)) == (1, 3)
    # a -1 on both sides is padding, never a hit
    assert O.recall_counts(np.array([[-1, -1]], np.int32), np.array([[-1, -1]], np.int32)) == (0, 0)


def test_run_recall_hand_worked():
    """Whole run whose recall is known by hand: d = 1, 4 key chunks, k = 2, no sentinels (so the
    relay layer can only reuse), one anchor.  Keys (4,3,2,1) then (4,2,3,1); query rows +1, 0, -1.
    Layer 0 routes {0,1}, {0,1} (all ties -> smallest ids), {3,2}; exact top-2 at layer 1:
    {0,2}, {0,1}, {3,1} -> hits 1 + 2 + 1 of 6 on the relay layer, 10 of 12 over the run."""
    p = O.OracleParams(n_q=3, n_k=4, k=2, m=0, r=0)
    q = np.array([[[1.0], [0.0], [-1.0]]])
    k0 = np.array([[[4.0], [3.0], [2.0], [1.0]]])
    k1 = np.array([[[4.0], [2.0], [3.0], [1.0]]])
    res, summ = O.run_layers(np.stack([q, q]), np.stack([k0, k1]), p, anchor_every=8)
    assert [sorted(r) for r in res[0].ledger.routes.tolist()] == [[0, 1], [0, 1], [2, 3]]
    assert [sorted(r) for r in res[1].full_routes.tolist()] == [[0, 2], [0, 1], [1, 3]]
    assert not res[1].flags.any()                       # nothing can challenge a route
    assert summ.recall_relay == pytest.approx(4 / 6, abs=1e-15)
    assert summ.recall_all == pytest.approx(10 / 12, abs=1e-15)
    assert summ.rerouted_fraction == pytest.approx(0.5) and summ.flagged_relay_fraction == 0.0
    # score pairs: anchor 3 rows x 4, relay 3 rows x 2 candidates, over 2 x 12
    assert summ.score_pair_fraction == pytest.approx((12 + 6) / 24)


@pytest.mark.parametrize("L,n_k,k", [(4, 32, 3), (6, 64, 12), (3, 16, 16)])
def test_run_accounting_fixed_stride_closed_form(L, n_k, k):
    """Run-level score pairs of the ORACLE's own run with m = r = 0 and a single anchor, no
    mask: 1/L + (L-1)/L * k/n_k (the arithmetic of the sentinel-ablation table, Section 5.2)."""
    rng = np.random.default_rng(L * 1000 + n_k)
    q = rng.standard_normal((L, 2, 9, 8))
    kk = rng.standard_normal((L, 2, n_k, 8))
    p = O.OracleParams(n_q=9, n_k=n_k, k=k, m=0, r=0)
    res, summ = O.run_layers(q, kk, p, anchor_every=10 ** 6)
    assert summ.score_pair_fraction == pytest.approx(1 / L + (L - 1) / L * k / n_k, abs=1e-15)
    assert summ.rerouted_fraction == pytest.approx(1 / L, abs=1e-15)
    c = summ.counters
    assert c["cand_pairs"] == (L - 1) * 2 * 9 * k and c["full_pairs"] == 2 * 9 * n_k
    assert c["anchor_rows"] == 18 and c["relay_rows"] == (L - 1) * 18 and c["flagged_rows"] == 0


def test_run_accounting_causal_candidate_pairs():
    """Under the causal mask every relay layer charges every row min(v_i, c) candidate pairs
    (route, near-miss and random slots that exist), every flagged row v_i more; anchors charge
    v_i per row.  Asserted on the oracle's run-level counters against the flags it reports."""
    w = W.moderate().replace(heads=2, layers=5, anchor_every=3)
    p, res, summ = _run(w, [0, 1])
    v = np.tile(p.valid_counts(), 2)
    c = summ.counters
    n_relay = sum(not r.is_anchor for r in res)
    n_anchor = len(res) - n_relay
    assert n_relay == 3 and n_anchor == 2
    assert c["cand_pairs"] == n_relay * int(np.minimum(v, p.c).sum())
    flagged_v = sum(int(v[r.flags != 0].sum()) for r in res if not r.is_anchor)
    assert flagged_v > 0
    assert c["full_pairs"] == n_anchor * int(v.sum()) + flagged_v
    assert c["dense_pairs"] == len(res) * int(v.sum())
    assert summ.score_pair_fraction == pytest.approx(
        (c["cand_pairs"] + c["full_pairs"]) / (len(res) * v.sum()), abs=1e-15)
    # the per-row candidate count the run used equals the closed form slot by slot
    led = res[0].ledger
    assert np.array_equal(O.valid_candidate_counts(led), np.minimum(v, p.c))


# ---- forced anchors before layers of low route persistence (Section 3.2) ---------------------
def test_anchor_forcer_back_off_sequence_by_hand():
    """Threshold 100 of 1000 rows, runs up to 4: T(high) F T(high) F F T(high) F F F F T(low) T(high) F."""
    p = O.OracleParams(n_q=1000, n_k=8, k=1, m=1, r=0, force_permille=100, force_max_run=4)
    f = O.AnchorForcer(p, 1000)
    assert f.threshold == 100
    trace = []
    flagged = iter([100, 500, 999, 99, 100])          # what the tested layers see, in order
    for _ in range(14):
        if f.forced_now():
            trace.append("F"); f.after_forced()
        else:
            trace.append("T"); f.after_tested(next(flagged, 0))
    assert "".join(trace) == "TFTFFTFFFFTTFT"


def test_anchor_forcer_threshold_rounds_up_and_scheduled_anchor_clears():
    p = O.OracleParams(n_q=7, n_k=8, k=1, m=1, r=0, force_permille=500, force_max_run=2)
    f = O.AnchorForcer(p, 7)
    assert f.threshold == 4                            # ceil(3.5)
    f.after_tested(3); assert not f.forced_now()
    f.after_tested(4); assert f.forced_now() and f.left == 1
    f.after_anchor(); assert not f.forced_now() and f.run == 1
    f.after_tested(7); assert f.left == 2              # back-off memory survived the anchor
    off = O.AnchorForcer(O.OracleParams(n_q=7, n_k=8, k=1, m=1, r=0), 7)
    off.after_tested(7); assert not off.forced_now()


def test_run_with_forced_anchors_routes_every_row_on_forced_layers():
    """permille = 1 (any flagged row triggers), max run 1, strong drift: relay calls alternate
    tested / forced; a forced layer equals full routing of that layer and resets every age."""
    w = W.tiny().replace(rho=0.5, layers=6, anchor_every=6)
    q, k = W.generate(w)
    qf, kf = W.as_float32(q).astype(np.float64), W.as_float32(k).astype(np.float64)
    p = O.OracleParams(n_q=w.n_q, n_k=w.n_k, k=w.k, m=w.m, r=w.r, seed=w.seed,
                       force_permille=1, force_max_run=1)
    res, summ = O.run_layers(qf, kf, p, w.anchor_every)
    assert [r.forced for r in res] == [False, False, True, False, True, False]
    assert [r.is_anchor for r in res] == [True, False, True, False, True, False]
    for l in (2, 4):
        assert np.array_equal(res[l].ledger.routes, res[l].full_routes)
        assert not res[l].ledger.ages.any() and res[l].flags.all()
    # forced layers are charged as anchors
    assert summ.counters["anchor_rows"] == 3 * w.n_q and summ.counters["relay_rows"] == 3 * w.n_q
    plain, _ = O.run_layers(qf, kf, dataclasses.replace(p, force_permille=0), w.anchor_every)
    assert not any(r.forced for r in plain)
