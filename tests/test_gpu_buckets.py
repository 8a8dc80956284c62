"""Route-width buckets (Section 4.4) and the reference consumer of token ranges (Eq. 3).

Buckets: problems grouped by requested route width, one ledger per bucket, one call per layer.
Checked (a) against stand-alone ledgers on the same inputs, bit for bit (the front end adds no
arithmetic), and (b) against the oracle run per bucket with rows numbered inside the bucket."""
import numpy as np
import pytest
import torch

import parity
from oracle import routerelay_oracle as O
from paper_2609_07306_b200 import workload as W
from paper_2609_07306_b200.ledger import (BucketSet, RouteLedger, attend_token_ranges,
                                          config_from_workload, device_tensor)

pytestmark = pytest.mark.gpu

WIDTHS = [16, 8, 16, 12, 8, 16, 12, 16]


def _bucket_major(w, widths, layers):
    cfg = config_from_workload(w)
    bs = BucketSet(cfg, widths)
    q, k = W.generate(w, layers=layers)                       # [L, P, n, d], input order
    qb, kb = q[:, bs.order], k[:, bs.order]                   # bucket-major
    return bs, np.ascontiguousarray(qb), np.ascontiguousarray(kb)


def test_plan_groups_problems_by_width():
    w = W.moderate()
    bs = BucketSet(config_from_workload(w), WIDTHS)
    assert [i.k for i in bs.info] == [8, 12, 16]
    assert [i.problems for i in bs.info] == [2, 2, 4]
    assert [i.first_slot for i in bs.info] == [0, 2, 4]
    assert bs.order == [1, 4, 3, 6, 0, 2, 5, 7]
    assert bs.status() == 0
    bs.close()


def test_buckets_equal_standalone_ledgers_bit_for_bit():
    w = W.moderate()
    L = 4
    bs, qb, kb = _bucket_major(w, WIDTHS, L)
    dq, dk = [device_tensor(x) for x in qb], [device_tensor(x) for x in kb]
    for l in range(L):
        bs.route_layer(dq[l], dk[l], l, is_anchor=(l == 0))
    torch.cuda.synchronize()
    assert bs.status() == 0
    for inf, bl in zip(bs.info, bs.buckets):
        wb = w.replace(batch=1, heads=inf.problems, k=inf.k)
        ref = RouteLedger(config_from_workload(wb))
        sl = slice(inf.first_slot, inf.first_slot + inf.problems)
        for l in range(L):
            fn = ref.route_anchor if l == 0 else ref.route_relay
            fn(device_tensor(qb[l][sl]), device_tensor(kb[l][sl]), l)
        torch.cuda.synchronize()
        assert bl.routes.shape == (inf.problems * w.n_q, inf.k)
        for name in ("routes", "sentinels", "ages", "flags", "kth_score", "margin", "refresh_rows",
                     "problem_offsets"):
            assert torch.equal(getattr(bl, name), getattr(ref, name)), (inf.k, name)
        assert bl.counters_dict() == ref.counters_dict()
        ref.close()
    bs.close()


def test_buckets_match_per_bucket_oracle():
    w = W.moderate()
    L = 3
    bs, qb, kb = _bucket_major(w, WIDTHS, L)
    for l in range(L):
        bs.route_layer(device_tensor(qb[l]), device_tensor(kb[l]), l, is_anchor=(l == 0))
    torch.cuda.synchronize()
    for inf, bl in zip(bs.info, bs.buckets):
        sl = slice(inf.first_slot, inf.first_slot + inf.problems)
        p = parity.oracle_params(w.replace(k=inf.k))
        qf = W.as_float32(qb[:, sl]).astype(np.float64)
        kf = W.as_float32(kb[:, sl]).astype(np.float64)
        res, _ = O.run_layers(qf, kf, p, L, list(range(inf.problems)))   # one anchor, then relays
        led = res[-1].ledger
        routes, sent = bl.routes.cpu().numpy(), bl.sentinels.cpu().numpy()
        same_route = np.array([set(a) == set(b) for a, b in zip(routes, led.routes)])
        # free-running fp32 device vs float64 oracle: only near-ties may differ
        assert same_route.mean() > 0.995, (inf.k, same_route.mean())
        same_near = np.array([set(a) == set(b) for a, b in zip(sent[:, :w.m], led.sentinels[:, :w.m])])
        both = same_route & same_near & (bl.ages.cpu().numpy() == led.ages)
        assert both.mean() > 0.98
        # rows whose route and near-miss sets agree and that were last routed at the same layer
        # drew the same random sentinels (sampler keyed by the row id inside the bucket)
        assert np.array_equal(sent[both][:, w.m:], led.sentinels[both][:, w.m:])
        flags = bl.flags.cpu().numpy()
        assert abs(int(flags.sum()) - int(res[-1].flags.sum())) <= max(2, 0.01 * len(flags))
    bs.close()


@pytest.mark.parametrize("k", [8, 12])
def test_teacher_forced_parity_at_bucket_widths(k):
    rep = parity.run_teacher_forced(W.moderate().replace(k=k, heads=2, layers=3))
    print(parity.summary_line(rep))
    parity.assert_clean(rep)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_reference_consumer_matches_eq3_and_ignores_coalescing(dtype):
    T, dh = 4, 64
    w = W.moderate().replace(heads=2, chunk_tokens=T)
    q, k = W.generate(w, layers=1)
    outs, routes = [], None
    rng = np.random.default_rng(11)
    tokens = w.n_k * T
    qt = torch.from_numpy(rng.standard_normal((w.rows, dh)).astype(np.float32)).cuda().to(dtype)
    kt = torch.from_numpy(rng.standard_normal((w.problems, tokens, dh)).astype(np.float32)).cuda().to(dtype)
    vt = torch.from_numpy(rng.standard_normal((w.problems, tokens, dh)).astype(np.float32)).cuda().to(dtype)
    scale = dh ** -0.5
    for coalesce in (False, True):
        led = RouteLedger(config_from_workload(w.replace(coalesce_ranges=coalesce)))
        led.route_anchor(device_tensor(q[0]), device_tensor(k[0]), 0)
        rg = led.token_ranges
        if coalesce:                                   # some rows really have merged ranges
            assert int((rg[:, :, 0] >= 0).sum()) < int((led.routes >= 0).sum())
        outs.append(attend_token_ranges(rg.contiguous(), w.n_q, qt, kt, vt, scale))
        routes = led.routes.cpu().numpy()
        torch.cuda.synchronize()
        led.close()
    assert torch.equal(outs[0], outs[1])               # same tokens, same order: same bits
    got = outs[0].cpu().numpy()
    for prob in range(w.problems):
        sl = slice(prob * w.n_q, (prob + 1) * w.n_q)
        want = O.routed_attention(qt[sl].float().cpu().numpy(), kt[prob].float().cpu().numpy(),
                                  vt[prob].float().cpu().numpy(), routes[sl], T, scale)
        # FP32 dot products of width 64 and sums over <= 64 tokens against float64
        np.testing.assert_allclose(got[sl], want, rtol=2e-4, atol=2e-5)
