"""Vectorised fp32 "timed mode" of the CPU oracle.  TEST INFRASTRUCTURE ONLY.

The same route-maintenance algorithm as routerelay_oracle.py (Eq. 1, Eq. 2, Sec 3.1-3.2,
Sec 4.1-4.2), arranged the way a reasonable unfused CPU implementation would run it: fp32
BLAS `matmul` for the score GEMMs, `argpartition` for the TopK, fancy-index gathers for the
candidate rescoring, whole-array NumPy for the rest.  It exists so that the benchmark can put
a CPU number that is not a pure-Python loop beside the GPU number.  It is not the checker: the
plain float64 oracle is, and tests/test_oracle_timed.py holds this file to it.

Differences from the checker, all deliberate: scores are fp32 (a pair of scores closer than
fp32 rounding may rank the other way round, and ties at the TopK boundary are broken by
`argpartition`, not by index); the optional policies (global sentinels, hysteresis, forced
re-routing) are not implemented.  Only tests and the benchmark's CPU legs may import this
file; it shares no code with the CUDA library.
"""
from __future__ import annotations

import numpy as np

_GOLDEN = np.uint64(0x9E3779B97F4A7C15)
_MUL_A = np.uint64(0xBF58476D1CE4E5B9)
_MUL_B = np.uint64(0x94D049BB133111EB)
DRAW_LIMIT_PER_SLOT = 64


def _fmix64(x: np.ndarray) -> np.ndarray:
    """SplitMix64's output function on uint64 arrays (wrap-around arithmetic)."""
    x = x ^ (x >> np.uint64(30))
    x = x * _MUL_A
    x = x ^ (x >> np.uint64(27))
    x = x * _MUL_B
    return x ^ (x >> np.uint64(31))


def random_sentinels(taken: np.ndarray, v: np.ndarray, r: int, seed: int, g: np.ndarray,
                     layer: int) -> np.ndarray:
    """Sec 3.1 item 2 for many rows at once: the sequential accept/reject definition of the
    checker's draw_random_sentinels, one draw index t per sweep over the rows still short.

    taken: [R, n_k] bool, True for excluded chunks (modified); v, g: [R].  -> [R, r] int32."""
    R = len(v)
    out = np.full((R, r), -1, np.int32)
    if r <= 0 or R == 0:
        return out
    cols = np.arange(taken.shape[1])
    taken |= cols[None, :] >= v[:, None]               # chunks a row cannot see never qualify
    pool = taken.shape[1] - taken.sum(axis=1)
    small = pool <= r                                   # the whole pool, ascending
    for i in np.nonzero(small)[0]:
        free = np.nonzero(~taken[i])[0]
        out[i, : len(free)] = free
    with np.errstate(over="ignore"):
        key = _fmix64(np.uint64(seed) ^ (g.astype(np.uint64) * _GOLDEN))
        count = np.zeros(R, np.int64)
        active = np.nonzero(~small)[0]
        hi = np.uint64((layer & 0xFFFFFFFF) << 32)
        for t in range(DRAW_LIMIT_PER_SLOT * r):
            if len(active) == 0:
                break
            u = _fmix64(key[active] ^ (hi | np.uint64(t))) >> np.uint64(32)
            j = ((u * v[active].astype(np.uint64)) >> np.uint64(32)).astype(np.int64)
            ok = ~taken[active, j]
            rows = active[ok]
            taken[rows, j[ok]] = True
            out[rows, count[rows]] = j[ok]
            count[rows] += 1
            active = active[count[active] < r]
    for i in active:                                    # draw limit reached: fill in index order
        free = np.nonzero(~taken[i])[0][: r - count[i]]
        out[i, count[i]: count[i] + len(free)] = free
    return out


class TimedLedger:
    def __init__(self, rows: int, k: int, m: int, r: int):
        self.routes = np.full((rows, k), -1, np.int32)
        self.sentinels = np.full((rows, m + r), -1, np.int32)
        self.ages = np.full(rows, -1, np.int32)
        self.kth = np.zeros(rows, np.float32)
        self.margin = np.zeros(rows, np.float32)


def route_rows(s: np.ndarray, v: np.ndarray, k: int, m: int, r: int, seed: int, g: np.ndarray,
               layer: int):
    """Eq. 2 + Sec 3.1 + Sec 3.3 for the rows of `s` ([R, n_k] fp32, -inf beyond v):
    argpartition to the k + max(m, 1) best, sort those by (score desc, index asc), then the
    near-miss and random sentinels.  -> routes [R,k], sentinels [R,m+r], kth [R], margin [R]."""
    R, n_k = s.shape
    keep = min(n_k, k + max(m, 1))
    part = np.argpartition(-s, keep - 1, axis=1)[:, :keep] if keep < n_k else \
        np.broadcast_to(np.arange(n_k), (R, n_k)).copy()
    ps = np.take_along_axis(s, part, axis=1)
    order = np.lexsort((part, -ps), axis=1)
    top = np.take_along_axis(part, order, axis=1).astype(np.int32)
    ts = np.take_along_axis(ps, order, axis=1)
    top = np.where(np.arange(keep)[None, :] < v[:, None], top, -1)
    routes = np.full((R, k), -1, np.int32)
    routes[:, : min(k, keep)] = top[:, :k]
    sent = np.full((R, m + r), -1, np.int32)
    if m:
        sent[:, : max(0, min(m, keep - k))] = top[:, k:k + m]
    rows = np.arange(R)
    kk = np.minimum(k, v)
    kth = ts[rows, np.maximum(kk, 1) - 1]
    nxt = ts[rows, np.minimum(kk, keep - 1)]
    margin = np.where(v > kk, kth - nxt, np.float32(np.inf)).astype(np.float32)
    if r:
        taken = np.zeros((R, n_k), bool)
        listed = top[:, : k + m]
        rr, cc = np.nonzero(listed >= 0)
        taken[rr, listed[rr, cc]] = True
        sent[:, m:] = random_sentinels(taken, v, r, seed, g, layer)
    return routes, sent, kth.astype(np.float32), margin


def _scores(q: np.ndarray, k: np.ndarray, v: np.ndarray) -> np.ndarray:
    s = np.matmul(q, k.T)                                # Eq. 1, fp32 BLAS
    s[np.arange(k.shape[0])[None, :] >= v[:, None]] = -np.inf
    return s


def run_layers(q_layers: np.ndarray, k_layers: np.ndarray, n_q: int, n_k: int, k: int, m: int,
               r: int, gamma: float, causal: bool, seed: int, anchor_every: int, problem_ids):
    """The layer schedule on [L, P, n, d] fp32 inputs.  Anchor layers route every row from the
    full score matrix; relay layers gather the candidates' key chunks and rescore them
    (c * d multiply-adds per row), test alpha > beta + gamma (Eq. 5), compact the flagged row
    ids and route only those from a score GEMM over the compacted rows.
    -> (ledger, per-layer flagged counts)."""
    L, P = q_layers.shape[:2]
    led = TimedLedger(P * n_q, k, m, r)
    i = np.arange(n_q)
    v = np.clip(i + 1, 0, n_k) if causal else np.full(n_q, n_k)
    flagged_per_layer = []
    for layer in range(L):
        anchor = layer % anchor_every == 0
        n_flagged = 0
        for slot in range(P):
            q, kc = q_layers[layer, slot], k_layers[layer, slot]
            sl = slice(slot * n_q, (slot + 1) * n_q)
            g0 = int(problem_ids[slot]) * n_q
            if anchor:
                rows = i
            else:
                cand = np.concatenate([led.routes[sl], led.sentinels[sl]], axis=1)
                kg = kc[np.maximum(cand, 0)]                         # [n_q, c, d] gather
                cs = np.einsum("icd,id->ic", kg, q, optimize=True)
                a = np.where(cand[:, :k] >= 0, cs[:, :k], np.inf).min(axis=1)
                b = np.where(cand[:, k:] >= 0, cs[:, k:], -np.inf).max(axis=1) if m + r else \
                    np.full(n_q, -np.inf, np.float32)
                has_sent = (cand[:, k:] >= 0).any(axis=1)
                rows = np.nonzero(has_sent & ~(a > b + np.float32(gamma)))[0]   # compaction
            if len(rows):
                s = _scores(q[rows], kc, v[rows])
                ro, se, kth, mg = route_rows(s, v[rows], k, m, r, seed, g0 + rows, layer)
                gr = slot * n_q + rows
                led.routes[gr], led.sentinels[gr], led.kth[gr], led.margin[gr] = ro, se, kth, mg
            led.ages[sl] += 1
            led.ages[slot * n_q + rows] = 0
            n_flagged += len(rows)
        flagged_per_layer.append(n_flagged)
    return led, flagged_per_layer
