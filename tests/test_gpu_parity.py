"""CUDA path vs CPU oracle (through the C ABI), teacher-forced layer by layer."""
import numpy as np
import pytest
import torch

import parity
from oracle import routerelay_oracle as O
from paper_2609_07306_b200 import binding as B
from paper_2609_07306_b200 import workload as W
from paper_2609_07306_b200.ledger import RouteLedger, config_from_workload, device_tensor

pytestmark = pytest.mark.gpu


def _report(rep, record_property=None, name="parity"):
    """Prints the counts of ambiguous / soft-mismatching rows and, when the test passes pytest's
    record_property fixture, stores them with the test's result (junit / report plugins)."""
    line = parity.summary_line(rep)
    print(line)
    if record_property is not None:
        record_property(name, line)


def test_tiny_fp32_all_layers():
    rep = parity.run_teacher_forced(W.tiny())
    _report(rep)
    parity.assert_clean(rep)


@pytest.mark.parametrize("two_pass,gathered", [(False, False), (False, True), (True, True)],
                         ids=["fused+strip", "fused+gathered", "two_pass+gathered"])
def test_moderate_bf16_causal_all_layers(two_pass, gathered):
    rep = parity.run_teacher_forced(W.moderate(), two_pass=two_pass, gathered=gathered)
    _report(rep)
    parity.assert_clean(rep)


@pytest.mark.parametrize("two_pass,gathered", [(False, False), (False, True), (True, True)],
                         ids=["fused+strip", "fused+gathered", "two_pass+gathered"])
@pytest.mark.parametrize("n", [128, 512])
def test_sweep_shapes(n, two_pass, gathered):
    w = W.sweep(n, 0.15).replace(heads=4, layers=4, anchor_every=3)
    rep = parity.run_teacher_forced(w, two_pass=two_pass, gathered=gathered)
    _report(rep)
    parity.assert_clean(rep)


@pytest.mark.parametrize("variant", ["slow_rows", "streaming", "inplace", "inplace+slow_rows"])
@pytest.mark.parametrize("wl", ["moderate", "sweep512", "sweep1024"])
def test_routing_kernel_variants(wl, variant):
    """The other ways a bf16 row can be routed in one kernel (and "inplace": the relay whose
    challenge test runs inside the routing kernel, Section 3.2 and 4.2 in one pass): the two-sweep kernel with every
    fifth row handed to its exact slow path (complete score row in shared memory + warp-level
    radix select), and the streaming kernel that serves the shapes the two-sweep kernel does
    not hold."""
    w = {"moderate": W.moderate(),
         "sweep512": W.sweep(512, 0.15).replace(heads=4, layers=4, anchor_every=3),
         "sweep1024": W.sweep(1024, 0.30).replace(heads=3, layers=3, anchor_every=2)}[wl]
    rep = parity.run_teacher_forced(w, force_slow_rows="slow_rows" in variant,
                                    streaming=variant == "streaming", inplace="inplace" in variant)
    _report(rep)
    parity.assert_clean(rep)


@pytest.mark.parametrize("two_sweep", [True, False])
def test_degenerate_all_equal_scores_bf16(two_sweep):
    """All-zero bf16 inputs through the fused routing kernels (every score ties; in the two-sweep
    kernel every list is one run of equal keys, so all rows take its slow path; a grid this small
    uses the streaming kernel unless the two-sweep kernel is asked for): TopK must take the
    smallest ids under the causal mask, margin 0."""
    w = W.moderate().replace(heads=2)
    led = RouteLedger(config_from_workload(w, two_sweep=two_sweep))
    z = torch.zeros(1, w.problems, w.n_q, w.d, device="cuda", dtype=torch.bfloat16)
    led.route_anchor(z, z, 0)
    torch.cuda.synchronize()
    assert led.status() == 0
    r = led.routes.cpu().numpy().reshape(w.problems, w.n_q, w.k)
    s = led.sentinels.cpu().numpy().reshape(w.problems, w.n_q, w.sw)
    for i in (0, 5, w.k - 1, w.k, w.k + 3, w.k + w.m, 100, w.n_q - 1):
        v = i + 1
        kk, nn = min(w.k, v), min(w.m, max(0, v - w.k))
        assert (np.sort(r[:, i, :kk], axis=1) == np.arange(kk)).all(), i
        assert (r[:, i, kk:] == -1).all()
        assert (np.sort(s[:, i, :nn], axis=1) == np.arange(kk, kk + nn)).all(), i
        rnd = s[:, i, w.m:w.m + w.r]
        n_rnd = min(w.r, max(0, v - kk - nn))
        assert ((rnd >= 0).sum(axis=1) == n_rnd).all(), i
        assert all(len(set(x[x >= 0])) == n_rnd and (x[x >= 0] >= kk + nn).all() and
                   (x[x >= 0] < v).all() for x in rnd), i
    mg = led.margin.cpu().numpy().reshape(w.problems, w.n_q)
    assert (mg[:, w.k:] == 0).all() and np.isinf(mg[:, :w.k]).all()
    assert (led.kth_score.cpu().numpy() == 0).all()
    led.close()


def test_ragged_shapes_and_wide_ledger():
    # n_q not a multiple of any tile, n_q != n_k, non-causal, d=64 bf16, wide candidate set
    w = W.RouteWorkload("ragged", 1, 3, 200, 333, 64, 12, 24, 12, layers=3, anchor_every=3,
                        dtype=W.DTYPE_BF16, centroids=16, rho=0.05, causal=False, seed=3)
    for two_pass, gathered in ((False, False), (False, True), (True, True)):
        rep = parity.run_teacher_forced(w, two_pass=two_pass, gathered=gathered)
        _report(rep)
        parity.assert_clean(rep)
    w = W.RouteWorkload("ragged32", 2, 1, 130, 130, 128, 5, 0, 7, layers=3, anchor_every=2,
                        dtype=W.DTYPE_F32, centroids=8, rho=0.1, causal=True, seed=4)
    rep = parity.run_teacher_forced(w)
    _report(rep)
    parity.assert_clean(rep)


def test_long_context_shape_small():
    # n_k = 2048, k = 64, 32 + 32 sentinels (c = 128), token ranges; 2 heads, 3 layers
    w = W.long_ctx().replace(batch=1, heads=2, layers=3, anchor_every=2)
    for two_pass, gathered in ((False, False), (True, True)):
        rep = parity.run_teacher_forced(w, two_pass=two_pass, gathered=gathered)
        _report(rep)
        parity.assert_clean(rep)
        assert rep.token_range_rows == 3 * w.rows
    # the same with runs of adjacent chunks merged (k = 64: the multi-block coalescing path)
    rep = parity.run_teacher_forced(w.replace(coalesce_ranges=True))
    _report(rep)
    parity.assert_clean(rep)
    assert rep.token_range_rows == 3 * w.rows


def test_high_drift_full_size_sampled_problems(record_property):
    """The high-drift configuration at full size (batch 8 x 32 heads = 256 problems of 1024 x
    1024 chunks, k/m/r = 32/16/16: the launch the benchmark times), layers 0-9: the first
    anchor, relays before and after the centroid re-draws at layers 4 and 8, the second anchor
    at layer 8 and the relay after it.  Eight problems are checked row by row against the oracle,
    the integer work (compaction, ages, stable rows) on all 262144 rows."""
    w = W.high_drift()
    rep = parity.run_teacher_forced(w, check_problems=[0, 37, 74, 101, 128, 190, 233, 255],
                                    layers=10, gen_threads=16)
    _report(rep, record_property, "high_drift_full_size")
    parity.assert_clean(rep)


def test_long_context_full_size_sampled_problems(record_property):
    """The long-context configuration at full size (64 problems x 2048 chunks, k/m/r =
    64/32/32, 64-token chunks expanded to token ranges), 3 layers, eight problems checked
    against the oracle, token ranges included."""
    w = W.long_ctx()
    rep = parity.run_teacher_forced(w, check_problems=[0, 3, 17, 26, 35, 44, 53, 63], layers=3,
                                    gen_threads=16)
    _report(rep, record_property, "long_ctx_full_size")
    parity.assert_clean(rep)
    assert rep.token_range_rows == 3 * 8 * w.n_q


def test_degenerate_all_equal_scores():
    """All-zero inputs: every score ties; TopK must take the smallest ids, margin 0, and the
    challenge test (tie => flagged) must flag every row that has a sentinel."""
    w = W.tiny()
    led = RouteLedger(config_from_workload(w))
    z = torch.zeros(1, 1, w.n_q, w.d, device="cuda")
    led.route_anchor(z, z, 0)
    torch.cuda.synchronize()
    r = led.routes.cpu().numpy()
    s = led.sentinels.cpu().numpy()
    assert (np.sort(r, axis=1) == np.arange(w.k)).all()
    assert (np.sort(s[:, :w.m], axis=1) == np.arange(w.k, w.k + w.m)).all()
    assert (led.margin.cpu().numpy() == 0).all() and (led.kth_score.cpu().numpy() == 0).all()
    rnd = s[:, w.m:]
    assert (rnd >= w.k + w.m).all() and (rnd < w.n_k).all()
    assert all(len(set(row)) == w.r for row in rnd)
    led.route_relay(z, z, 1)
    torch.cuda.synchronize()
    assert led.flags.cpu().numpy().all()
    assert int(led.refresh_count.item()) == w.n_q
    led.close()


def test_relay_before_anchor_and_reset():
    w = W.tiny()
    led = RouteLedger(config_from_workload(w))
    z = torch.zeros(1, 1, w.n_q, w.d, device="cuda")
    with pytest.raises(B.RouteRelayError) as ei:
        led.route_relay(z, z, 1)
    assert ei.value.code == B.RR_ERR_STATE
    led.route_anchor(z, z, 0)
    led.reset()
    torch.cuda.synchronize()
    assert (led.routes.cpu().numpy() == -1).all() and (led.ages.cpu().numpy() == -1).all()
    assert led.counters.cpu().numpy().sum() == 0
    with pytest.raises(B.RouteRelayError):
        led.route_relay(z, z, 1)
    led.close()


def test_export_import_roundtrip_and_counters():
    w = W.moderate().replace(heads=2)
    q, k = W.generate(w, layers=3)
    led = RouteLedger(config_from_workload(w))
    led.route_anchor(device_tensor(q[0]), device_tensor(k[0]), 0)
    blob = led.export_blob()
    led.route_relay(device_tensor(q[1]), device_tensor(k[1]), 1)
    torch.cuda.synchronize()
    after1 = led.routes.clone()
    flags1 = led.flags.cpu().numpy().copy()
    led.import_blob(blob)                       # rewind to the anchor state
    led.route_relay(device_tensor(q[1]), device_tensor(k[1]), 1)
    torch.cuda.synchronize()
    assert torch.equal(led.routes, after1)
    c = led.counters_dict()
    v = np.tile(parity.oracle_params(w).valid_counts(), w.problems)
    assert c["layer_calls"] == 3 and c["anchor_rows"] == w.rows and c["relay_rows"] == 2 * w.rows
    assert c["dense_pairs"] == 3 * v.sum()
    assert c["flagged_rows"] == 2 * flags1.sum()
    assert c["full_pairs"] == v.sum() + 2 * v[flags1 != 0].sum()
    assert c["cand_pairs"] == 2 * np.minimum(v, w.c).sum()
    led.close()


def test_host_buffer_entry_point():
    w = W.moderate().replace(heads=2)
    q, k = W.generate(w, layers=2)
    led = RouteLedger(config_from_workload(w))
    ref = RouteLedger(config_from_workload(w))
    hq = [torch.from_numpy(q[l].view(np.int16)).pin_memory() for l in range(2)]
    hk = [torch.from_numpy(k[l].view(np.int16)).pin_memory() for l in range(2)]
    dq, dk = torch.empty_like(hq[0], device="cuda"), torch.empty_like(hk[0], device="cuda")
    out = torch.empty(w.rows, w.k, dtype=torch.int32).pin_memory()
    for l in range(2):
        led.route_layer_host(hq[l], hk[l], dq, dk, l, l == 0, out)
        (ref.route_anchor if l == 0 else ref.route_relay)(device_tensor(q[l]), device_tensor(k[l]), l)
        torch.cuda.synchronize()
        assert torch.equal(out, ref.routes.cpu())
    led.close(); ref.close()


def test_pipelined_host_layers_entry_point():
    """rr_route_layers_host (copies overlapped on a second stream) returns, for every layer,
    exactly the routes of the device-buffer calls."""
    w = W.moderate().replace(heads=2)
    L = 6
    q, k = W.generate(w, layers=L)
    led = RouteLedger(config_from_workload(w))
    ref = RouteLedger(config_from_workload(w))
    hq = [torch.from_numpy(q[l].view(np.int16)).pin_memory() for l in range(L)]
    hk = [torch.from_numpy(k[l].view(np.int16)).pin_memory() for l in range(L)]
    dq = [torch.empty_like(hq[0], device="cuda") for _ in range(2)]
    dk = [torch.empty_like(hk[0], device="cuda") for _ in range(2)]
    dr = [torch.empty(w.rows, w.k, dtype=torch.int32, device="cuda") for _ in range(2)]
    outs = [torch.empty(w.rows, w.k, dtype=torch.int32).pin_memory() for _ in range(L)]
    cs = torch.cuda.Stream()
    anchors = [l % 3 == 0 for l in range(L)]
    led.route_layers_host(hq, hk, anchors, 0, dq, dk, dr, outs, cs, torch.cuda.Stream())
    torch.cuda.synchronize()
    for l in range(L):
        (ref.route_anchor if anchors[l] else ref.route_relay)(device_tensor(q[l]), device_tensor(k[l]), l)
        torch.cuda.synchronize()
        assert torch.equal(outs[l], ref.routes.cpu()), f"layer {l}"
    assert led.counters_dict() == ref.counters_dict()
    led.close(); ref.close()


def test_pipelined_host_layers_back_to_back_calls():
    """Two rr_route_layers_host calls on the same ledger and staging buffers with NO
    synchronisation between them (what a serving loop does): the second call's uploads must
    wait for the first call's last readers of each staging set.  The first call routes other
    inputs, so a staging set overwritten too early (or too late) shows in the routes."""
    w = W.sweep(512, 0.15).replace(heads=8, layers=5, anchor_every=3)
    L = w.layers
    q, k = W.generate(w)
    q2, k2 = W.generate(w.replace(seed=9))
    led = RouteLedger(config_from_workload(w))
    ref = RouteLedger(config_from_workload(w))
    pin = lambda x: torch.from_numpy(x.view(np.int16)).pin_memory()
    hq, hk = [pin(q[l]) for l in range(L)], [pin(k[l]) for l in range(L)]
    hq2, hk2 = [pin(q2[l]) for l in range(L)], [pin(k2[l]) for l in range(L)]
    dq = [torch.empty_like(hq[0], device="cuda") for _ in range(2)]
    dk = [torch.empty_like(hk[0], device="cuda") for _ in range(2)]
    dr = [torch.empty(w.rows, w.k, dtype=torch.int32, device="cuda") for _ in range(2)]
    outs1 = [torch.empty(w.rows, w.k, dtype=torch.int32).pin_memory() for _ in range(L)]
    outs2 = [torch.empty(w.rows, w.k, dtype=torch.int32).pin_memory() for _ in range(L)]
    cs, ds = torch.cuda.Stream(), torch.cuda.Stream()
    anchors = [w.is_anchor(l) for l in range(L)]
    for rep_ in range(3):                        # a few rounds: a race need not show at once
        led.reset()
        led.route_layers_host(hq2, hk2, anchors, 0, dq, dk, dr, outs1, cs, ds)
        led.route_layers_host(hq, hk, anchors, 0, dq, dk, dr, outs2, cs, ds)   # no sync before
        torch.cuda.synchronize()
        ref.reset()
        for l in range(L):
            (ref.route_anchor if anchors[l] else ref.route_relay)(device_tensor(q[l]), device_tensor(k[l]), l)
            torch.cuda.synchronize()
            assert torch.equal(outs2[l], ref.routes.cpu()), f"round {rep_} layer {l}"
    led.close(); ref.close()


@pytest.mark.parametrize("coalesce", [False, True], ids=["per_chunk", "coalesced"])
@pytest.mark.parametrize("two_pass", [False, True], ids=["fused", "two_pass"])
def test_token_ranges(two_pass, coalesce):
    """Token ranges of the routes (per chunk, or runs of adjacent chunks merged), from rows in
    ascending chunk id (fused kernel) and in rank order (two-pass path, imported ledgers)."""
    w = W.moderate().replace(heads=2, chunk_tokens=64, coalesce_ranges=coalesce)
    q, k = W.generate(w, layers=2)
    led = RouteLedger(config_from_workload(w, two_pass=two_pass))
    led.route_anchor(device_tensor(q[0]), device_tensor(k[0]), 0)
    led.route_relay(device_tensor(q[1]), device_tensor(k[1]), 1)
    torch.cuda.synchronize()
    routes = led.routes.cpu().numpy()
    expect = O.token_ranges(routes, 64, coalesce=coalesce)
    assert np.array_equal(led.token_ranges.cpu().numpy(), expect)
    if coalesce:      # the causal rows select runs of neighbours: something must have merged
        per_chunk = O.token_ranges(routes, 64)
        assert (expect[:, :, 0] >= 0).sum() < (per_chunk[:, :, 0] >= 0).sum()
    led.close()


@pytest.mark.parametrize("two_sweep", [False, True], ids=["streaming", "two_sweep"])
@pytest.mark.parametrize("wl", ["moderate", "sweep_1024_rho0.30_4heads"])
def test_free_running_summary_matches_oracle(wl, two_sweep):
    """All layers without teacher forcing: recall / refreshed-row / score-pair fractions of
    the device run agree with the oracle's run up to the ambiguous rows.  Second case: the
    routing-scale sweep at 1024 chunks and the highest drift (4 of its 32 heads, 16 layers)."""
    w = W.moderate() if wl == "moderate" else W.sweep(1024, 0.30).replace(heads=4)
    q, k = W.generate(w)
    p = parity.oracle_params(w)
    res, summ = O.run_layers(W.as_float32(q).astype(np.float64), W.as_float32(k).astype(np.float64),
                             p, w.anchor_every)
    led = RouteLedger(config_from_workload(w, two_sweep=two_sweep))
    hit = tot = 0
    for l in range(w.layers):
        fn = led.route_anchor if w.is_anchor(l) else led.route_relay
        fn(device_tensor(q[l]), device_tensor(k[l]), l)
        torch.cuda.synchronize()
        h, t = O.recall_counts(led.routes.cpu().numpy(), res[l].full_routes)
        hit += h; tot += t
    c = led.counters_dict()
    rer, flg, pairs = O.fractions_from_counters(c)
    print(f"device: recall {hit / tot:.6f} rerouted {rer:.4f} flagged {flg:.4f} pairs {pairs:.4f}"
          f" | oracle: {summ.recall_all:.6f} {summ.rerouted_fraction:.4f} "
          f"{summ.flagged_relay_fraction:.4f} {summ.score_pair_fraction:.4f}")
    assert abs(hit / tot - summ.recall_all) < 2e-4
    assert abs(rer - summ.rerouted_fraction) < 2e-3
    assert abs(pairs - summ.score_pair_fraction) < 2e-3
    led.close()


@pytest.mark.parametrize("m,r", [(0, 12), (12, 12), (48, 12), (12, 0), (0, 0)])
def test_sentinel_ablation_shapes(m, r):
    """The (m, r) grid of the sentinel-ablation table (Section 5.2), including random-only,
    near-miss-only and the fixed-stride baseline m = r = 0 (nothing can challenge a route)."""
    w = W.ablation(m, r).replace(batch=1, heads=3, layers=5)
    for two_pass, gathered in ((False, False), (False, True), (True, True)):
        rep = parity.run_teacher_forced(w, two_pass=two_pass, gathered=gathered)
        _report(rep)
        parity.assert_clean(rep)


def test_fixed_stride_never_flags_and_low_drift_flags_few():
    """Free-running: with m = r = 0 only the anchor layer routes (rerouted fraction 1/L; the
    pairs are the anchor's plus k per relay row); at low drift the flagged fraction stays far below the high-drift regime's."""
    def run(w):
        q, k = W.generate(w)
        led = RouteLedger(config_from_workload(w))
        for l in range(w.layers):
            fn = led.route_anchor if w.is_anchor(l) else led.route_relay
            fn(device_tensor(q[l]), device_tensor(k[l]), l)
        torch.cuda.synchronize()
        c = led.counters_dict()
        led.close()
        return O.fractions_from_counters(c)
    w = W.ablation(0, 0).replace(batch=1, heads=4, layers=6)
    rer, flg, pairs = run(w)
    assert flg == 0.0 and abs(rer - 1 / 6) < 1e-12
    assert abs(pairs - (1 / 6 + (5 / 6) * 12 / 256)) < 1e-12
    w = W.low_drift().replace(batch=1, heads=2, layers=4)
    rer, flg, pairs = run(w)
    w_hi = W.high_drift().replace(batch=1, heads=2, layers=4, redraw_every=0)
    _, flg_hi, _ = run(w_hi)
    print(f"flagged fraction: low drift {flg:.3f}, high drift {flg_hi:.3f}")
    assert flg < 0.5 * flg_hi


_POLICIES = {
    "global_sentinels": dict(global_sentinels=3),
    "sink_only": dict(global_sentinels=1, m=0),
    "min_reuse": dict(min_reuse=1),
    "gamma_boost": dict(gamma_boost=0.05, margin_recover=0.02),
    "h_max": dict(h_max=2),
    "all": dict(global_sentinels=3, min_reuse=1, gamma_boost=0.05, margin_recover=0.02, h_max=3),
}


@pytest.mark.parametrize("policy", sorted(_POLICIES))
def test_policies_either_side_of_the_trigger(policy):
    """Mandatory global sentinels (Section 3.1 item 3), hysteresis and per-row forced
    re-routing (Section 3.2) against the oracle, on every kernel variant."""
    base = W.moderate().replace(heads=3, layers=7, anchor_every=100, rho=0.2)
    w = base.replace(**_POLICIES[policy])
    for two_pass, gathered in ((False, False), (False, True), (True, True)):
        rep = parity.run_teacher_forced(w, two_pass=two_pass, gathered=gathered)
        _report(rep)
        parity.assert_clean(rep)
    # non-causal, ragged shape, d = 64
    w2 = W.RouteWorkload("ragged_policy", 1, 2, 200, 333, 64, 12, 8, 6, layers=5, anchor_every=100,
                         dtype=W.DTYPE_BF16, centroids=16, rho=0.1, causal=False, seed=5,
                         **{k_: v_ for k_, v_ in _POLICIES[policy].items() if k_ != "m"})
    rep = parity.run_teacher_forced(w2)
    _report(rep)
    parity.assert_clean(rep)


def test_forced_rerouting_bounds_every_age():
    """Free-running with h_max = 3 and a single anchor: no age ever exceeds 3."""
    w = W.moderate().replace(heads=2, layers=9, anchor_every=100, rho=0.01, h_max=3)
    q, k = W.generate(w)
    led = RouteLedger(config_from_workload(w))
    worst = 0
    for l in range(w.layers):
        fn = led.route_anchor if w.is_anchor(l) else led.route_relay
        fn(device_tensor(q[l]), device_tensor(k[l]), l)
        torch.cuda.synchronize()
        worst = max(worst, int(led.ages.max().item()))
    led.close()
    assert worst == 3


def test_maximum_sizes():
    """The limits of the interface: n_k = 4096 key chunks and k + m + r = 256 candidates per row
    (the fused kernel cannot hold such a candidate set, so this also covers the automatic
    fall-back to the two-pass path), and n_k = 4096 with a ledger the fused kernel does hold."""
    w = W.RouteWorkload("max_c", 1, 1, 96, 4096, 128, 128, 64, 64, layers=3, anchor_every=100,
                        dtype=W.DTYPE_BF16, centroids=64, rho=0.2, causal=False, seed=7)
    rep = parity.run_teacher_forced(w)
    _report(rep)
    parity.assert_clean(rep)
    w = W.RouteWorkload("max_nk", 1, 2, 160, 4096, 128, 32, 16, 16, layers=3, anchor_every=100,
                        dtype=W.DTYPE_BF16, centroids=64, rho=0.2, causal=False, seed=8)
    for two_pass, gathered in ((False, False), (True, True)):
        rep = parity.run_teacher_forced(w, two_pass=two_pass, gathered=gathered)
        _report(rep)
        parity.assert_clean(rep)
    # one key chunk more than the interface allows is refused, not truncated
    with pytest.raises(B.RouteRelayError):
        B.rr_workspace_bytes(config_from_workload(w.replace(n_k=4097)))


@pytest.mark.parametrize("n_q,n_k", [(384, 192), (192, 1024)])
def test_rectangular_shapes_of_the_paper(n_q, n_k):
    """Query and key chunk counts differ (the paper's 384 x 192 and 192 x 1024 problems),
    without and with a causal offset that lets the last query row see every key chunk."""
    for causal in (False, True):
        w = W.RouteWorkload(f"rect_{n_q}x{n_k}", 1, 2, n_q, n_k, 128, 16, 8, 8, layers=4,
                            anchor_every=100, dtype=W.DTYPE_BF16, centroids=32, rho=0.1,
                            causal=causal, seed=11, causal_offset=max(0, n_k - n_q))
        rep = parity.run_teacher_forced(w)
        _report(rep)
        parity.assert_clean(rep)


@pytest.mark.parametrize("variant", ["default", "two_pass", "gathered"])
def test_forced_anchors_after_low_persistence_follow_the_oracle(variant):
    """Forced anchors before layers of low route persistence (Section 3.2), decided on the
    device from the flagged count of the last tested relay: the sequence of tested / forced
    calls, the work counters and the routes follow the oracle's run of the same policy."""
    w = W.moderate().replace(force_permille=500, force_max_run=2, layers=12, anchor_every=6)
    q, k = W.generate(w)
    p = parity.oracle_params(w)
    res, summ = O.run_layers(W.as_float32(q).astype(np.float64), W.as_float32(k).astype(np.float64),
                             p, w.anchor_every)
    want = [r.forced for r in res]
    assert any(want) and not all(want[1:6])            # the policy fires and also probes
    led = RouteLedger(config_from_workload(w, two_pass=(variant == "two_pass"),
                                           gathered=(variant == "gathered")))
    got = []
    for l in range(w.layers):
        fn = led.route_anchor if w.is_anchor(l) else led.route_relay
        fn(device_tensor(q[l]), device_tensor(k[l]), l)
        torch.cuda.synchronize()
        st = led.force_state.cpu().numpy()
        got.append(bool(st[5]))
        if got[-1]:                                     # a forced call is an anchor in all but name
            assert led.flags.all() and not led.ages.any()
            assert int(led.refresh_count.item()) == w.rows
            assert torch.equal(led.refresh_rows, torch.arange(w.rows, dtype=torch.int32, device="cuda"))
        same = np.array([set(a) == set(b) for a, b in zip(led.routes.cpu().numpy(), res[l].ledger.routes)])
        assert same.mean() > 0.99, (l, same.mean())
    assert got == want
    c = led.counters_dict()
    assert c["anchor_rows"] == summ.counters["anchor_rows"]
    assert c["relay_rows"] == summ.counters["relay_rows"]
    assert abs(c["flagged_rows"] - summ.counters["flagged_rows"]) <= 0.01 * c["relay_rows"]
    assert int(led.force_state[4].item()) == sum(want)
    assert led.status() == 0
    # reset clears the policy's state
    led.reset()
    torch.cuda.synchronize()
    assert not led.force_state.any()
    led.close()


def test_forced_anchor_policy_is_refused_with_the_in_place_relay():
    w = W.moderate().replace(force_permille=500)
    with pytest.raises(B.RouteRelayError) as ei:
        RouteLedger(config_from_workload(w, inplace=True))
    assert ei.value.code == B.RR_ERR_UNSUPPORTED
