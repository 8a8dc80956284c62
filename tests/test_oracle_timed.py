"""The vectorised fp32 timed mode of the oracle, held to the float64 checker: same routes,
sentinels, ages and refresh decisions wherever fp32 rounding cannot change a ranking."""
import numpy as np

from oracle import routerelay_oracle as O
from oracle import routerelay_timed as T
from paper_2609_07306_b200 import workload as W


def test_vectorised_sampler_equals_sequential_definition():
    rng = np.random.default_rng(5)
    n_k, r = 40, 6
    v = np.array([40, 40, 9, 7, 25, 12, 6, 1], np.int64)
    g = np.arange(100, 108)
    taken = np.zeros((len(v), n_k), bool)
    excluded = []
    for i, vi in enumerate(v):
        e = rng.choice(vi, size=min(vi, [5, 30, 3, 3, 20, 11, 2, 1][i]), replace=False)
        taken[i, e] = True
        excluded.append([int(x) for x in e])
    got = T.random_sentinels(taken.copy(), v, r, 77, g, 3)
    for i in range(len(v)):
        want = O.draw_random_sentinels(excluded[i], int(v[i]), r, 77, int(g[i]), 3)
        assert [int(x) for x in got[i] if x >= 0] == want, i


def _both(w, layers, problems):
    q, k = W.generate(w, problems=problems, layers=layers)
    qf, kf = W.as_float32(q), W.as_float32(k)
    p = O.OracleParams(n_q=w.n_q, n_k=w.n_k, k=w.k, m=w.m, r=w.r, gamma=w.gamma, causal=w.causal,
                       seed=w.seed)
    res, _ = O.run_layers(qf.astype(np.float64), kf.astype(np.float64), p, w.anchor_every, problems)
    led, flagged = T.run_layers(qf, kf, w.n_q, w.n_k, w.k, w.m, w.r, w.gamma, w.causal, w.seed,
                                w.anchor_every, problems)
    return res, led, flagged


def test_timed_mode_matches_checker_on_tiny_f32():
    w = W.tiny()
    res, led, flagged = _both(w, 4, [0])
    ref = res[-1].ledger
    same = (led.routes == ref.routes).all(axis=1) & (led.sentinels == ref.sentinels).all(axis=1)
    assert same.mean() > 0.98                 # fp32 vs float64 near-ties only
    assert np.array_equal(led.ages[same], ref.ages[same])
    assert flagged[0] == w.n_q
    for l in range(1, 4):
        assert abs(flagged[l] - int(res[l].flags.sum())) <= 2


def test_timed_mode_matches_checker_causal_bf16():
    w = W.moderate()
    res, led, flagged = _both(w, 3, [1, 4])
    ref = res[-1].ledger
    same = (led.routes == ref.routes).all(axis=1) & (led.sentinels == ref.sentinels).all(axis=1)
    assert same.mean() > 0.98
    np.testing.assert_allclose(led.kth[same], ref.kth[same], rtol=1e-4, atol=1e-4)
    fin = same & np.isfinite(ref.margin)
    np.testing.assert_allclose(led.margin[fin], ref.margin[fin], rtol=1e-3, atol=1e-3)
    assert np.array_equal(np.isfinite(led.margin[same]), np.isfinite(ref.margin[same]))
