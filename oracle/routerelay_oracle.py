"""CPU oracle for RouteRelay's route-maintenance path.  TEST INFRASTRUCTURE ONLY.

Only the test-suite, the smoke check and the benchmark's CPU-baseline leg may
import this file.  It shares no code with the CUDA library and the library never
calls it.  Everything is NumPy float64 (scores are exact dot products of the
bf16/fp32 input values up to float64 rounding) or plain Python integers.

The method is a heuristic (a relayed route need not equal the exact TopK of the
current layer), so the oracle follows the algorithm step by step:

* Eq. 1   scores S = Qc Kc^T (no 1/sqrt(d)), masked to the valid key chunks of a row;
* Eq. 2   route = TopK over the row under the total order (score desc, index asc);
* Sec 3.1 ledger = route + m near-miss (ranks k+1..k+m) + r random sentinels drawn
          without replacement from the valid chunks outside route and near-miss;
* Sec 3.2 relay: alpha = min route score, beta = max sentinel score, the route is reused
          iff alpha > beta + gamma (Eq. 5); otherwise the row is fully re-routed and its
          sentinels rebuilt;
* Sec 4.1 unstable row ids are compacted in ascending order; stable rows keep route and
          sentinels and their age advances; rebuilt rows get age 0;
* Sec 3.3 anchor margin Delta = min selected - max unselected;
* Sec 3.1 item 3 / Sec 3.2 (optional policies, off by default): mandatory global sentinels
          (sink chunk, most recent chunk), a minimum reuse horizon and a larger guard margin
          for rows whose recorded margin is small (hysteresis), forced re-routing of rows
          whose route is h_max layers old (forced anchors, per row).

Readings of points the paper leaves open are listed in the design notes of the
repository; the ones that matter here: ties break towards the smaller chunk index;
-0.0 equals +0.0; a row with no valid sentinel is never flagged; slots a row cannot
fill (fewer valid chunks than k, m or r) hold -1; under the causal chunk mask row i of
a problem sees chunks j <= i + causal_offset.

Pins (tests/test_oracle_*.py): hand-computed scores, brute-force sorting of tuples,
Lemma 1, the trigger's logical consequences, special cases that reduce to "route
every layer" and "fixed stride", the hypergeometric miss probability (Eq. 6), the
arithmetic of the paper's sentinel-ablation table, the 256 KB ledger size, and
published output values of the 64-bit finaliser used by the sentinel sampler.
The paper's printed recall / reroute / latency numbers are NOT reproducible (its
generator is unspecified): for those, parity unpinned.
"""
from __future__ import annotations

import dataclasses
from typing import Dict, List, Optional, Sequence

import numpy as np

_M64 = (1 << 64) - 1
_GOLDEN = 0x9E3779B97F4A7C15
_MUL_A = 0xBF58476D1CE4E5B9
_MUL_B = 0x94D049BB133111EB
SAMPLER_DRAW_LIMIT_PER_SLOT = 64   # after 64*r draws the rest is filled in index order


# --------------------------------------------------------------------------- sampler RNG
def fmix64(x: int) -> int:
    """64-bit avalanche finaliser (the output function of the SplitMix64 generator)."""
    x &= _M64
    x ^= x >> 30
    x = (x * _MUL_A) & _M64
    x ^= x >> 27
    x = (x * _MUL_B) & _M64
    x ^= x >> 31
    return x


def row_key(seed: int, g: int) -> int:
    """Per-row 64-bit key: finalise(seed xor g*golden)."""
    return fmix64((seed & _M64) ^ ((g * _GOLDEN) & _M64))


def draw_u32(seed: int, g: int, layer: int, t: int) -> int:
    """The t-th 32-bit draw of global row g when its sentinels are rebuilt at `layer`."""
    ctr = ((layer & 0xFFFFFFFF) << 32) | (t & 0xFFFFFFFF)
    return fmix64(row_key(seed, g) ^ ctr) >> 32


def draw_random_sentinels(excluded: Sequence[int], v: int, r: int, seed: int, g: int,
                          layer: int) -> List[int]:
    """r distinct chunks, uniform over {0..v-1} minus `excluded` (Sec 3.1 item 2, Sec 3.4).

    Sequential definition: if the pool has at most r members take all of it in ascending
    order.  Otherwise for t = 0,1,2,...: j = floor(u_t * v / 2^32); accept j iff it is not
    excluded and not yet drawn; stop after r accepts.  After 64*r draws the remaining slots
    are filled with the smallest pool members not yet taken (bounded work).
    """
    taken = set(int(j) for j in excluded if j >= 0)
    pool = v - len(taken)
    if r <= 0 or pool <= 0:
        return []
    if pool <= r:
        return [j for j in range(v) if j not in taken]
    out: List[int] = []
    limit = SAMPLER_DRAW_LIMIT_PER_SLOT * r
    t = 0
    while len(out) < r and t < limit:
        j = (draw_u32(seed, g, layer, t) * v) >> 32
        t += 1
        if j not in taken:
            taken.add(j)
            out.append(j)
    j = 0
    while len(out) < r:
        if j not in taken:
            taken.add(j)
            out.append(j)
        j += 1
    return out


# --------------------------------------------------------------------------- parameters
@dataclasses.dataclass(frozen=True)
class OracleParams:
    n_q: int
    n_k: int
    k: int
    m: int
    r: int
    gamma: float = 0.0
    causal: bool = False
    causal_offset: int = 0
    seed: int = 0
    # policies either side of the trigger (Sec 3.1 item 3, Sec 3.2 "Hysteresis", "Forced anchors")
    global_sentinels: int = 0     # bit 0: sink chunk 0, bit 1: most recent valid chunk
    min_reuse: int = 0            # a row routed fewer than this many layers ago is not tested
    gamma_boost: float = 0.0      # added to gamma while the row's recorded margin < margin_recover
    margin_recover: float = 0.0
    h_max: int = 0                # >0: a row last routed h_max or more layers ago is re-routed
    # forced anchors before layers of low route persistence (Sec 3.2), decided from the flagged
    # count of the last tested relay layer; 0 = off
    force_permille: int = 0       # a tested relay that flags >= this many per mille of the rows ...
    force_max_run: int = 1        # ... forces the next relay calls to route every row (see AnchorForcer)

    @property
    def n_global(self) -> int:
        return (self.global_sentinels & 1) + ((self.global_sentinels >> 1) & 1)

    @property
    def sw(self) -> int:
        """Width of a sentinel row: near-miss, random, then mandatory global slots."""
        return self.m + self.r + self.n_global

    @property
    def c(self) -> int:
        return self.k + self.sw

    def valid_counts(self) -> np.ndarray:
        """v_i: how many key chunks query row i may select."""
        if not self.causal:
            return np.full(self.n_q, self.n_k, dtype=np.int64)
        i = np.arange(self.n_q, dtype=np.int64)
        return np.clip(i + 1 + self.causal_offset, 0, self.n_k)


@dataclasses.dataclass
class Ledger:
    """Route-maintenance state (Sec 4.1): routes, sentinels (near-miss then random), ages,
    plus the k-th score and margin recorded when each row was last routed."""
    routes: np.ndarray      # [rows, k] int32, -1 = empty slot
    sentinels: np.ndarray   # [rows, m+r+globals] int32
    ages: np.ndarray        # [rows] int32, -1 = never routed
    kth: np.ndarray         # [rows] float64
    margin: np.ndarray      # [rows] float64

    @staticmethod
    def empty(rows: int, p: OracleParams) -> "Ledger":
        return Ledger(np.full((rows, p.k), -1, np.int32),
                      np.full((rows, p.sw), -1, np.int32),
                      np.full(rows, -1, np.int32),
                      np.zeros(rows, np.float64), np.zeros(rows, np.float64))

    def copy(self) -> "Ledger":
        return Ledger(self.routes.copy(), self.sentinels.copy(), self.ages.copy(),
                      self.kth.copy(), self.margin.copy())

    def index_bytes(self) -> int:
        """Bytes of 32-bit index storage (Sec 4.4): rows * c * 4."""
        return 4 * (self.routes.size + self.sentinels.size)


# --------------------------------------------------------------------------- Eq. 1 / Eq. 2
def scores(q: np.ndarray, k: np.ndarray, p: OracleParams) -> np.ndarray:
    """Eq. 1 in float64 with the chunks a row may not select set to -inf."""
    s = np.matmul(np.asarray(q, np.float64), np.asarray(k, np.float64).T)
    s = s + 0.0                      # -0.0 -> +0.0
    if not np.all(np.isfinite(s)):
        raise ValueError("routing scores must be finite")
    v = p.valid_counts()
    col = np.arange(p.n_k)[None, :]
    return np.where(col < v[:, None], s, -np.inf)


def rank_order(s_row: np.ndarray, v: int) -> np.ndarray:
    """Valid chunk ids of one row sorted by (score descending, index ascending)."""
    order = np.argsort(-s_row[:v], kind="stable")
    return order.astype(np.int64)


def full_route(s_row: np.ndarray, v: int, k: int) -> np.ndarray:
    """Eq. 2: the exact TopK set of the row (first min(k,v) ranks)."""
    return rank_order(s_row, v)[: min(k, v)]


def route_row(s_row: np.ndarray, v: int, p: OracleParams, g: int, layer: int):
    """Full routing of one row plus sentinel construction (Sec 3.1) and margin (Sec 3.3).

    Sentinel row: m near-miss slots, r random slots, then one slot per mandatory global
    candidate (sink = chunk 0, recent = the last chunk the row may select).  A global
    candidate that is already in the route or among the near-miss sentinels (or equals an
    earlier global one) leaves its slot empty; the random sentinels are drawn from what is
    left after route, near-miss and global candidates.

    Returns (route[k], sentinels[sw], kth_score, margin) with -1 padding."""
    order = rank_order(s_row, v)
    kk = min(p.k, v)
    mm = min(p.m, max(0, v - p.k))
    route = np.full(p.k, -1, np.int32)
    route[:kk] = order[:kk]
    sent = np.full(p.sw, -1, np.int32)
    sent[:mm] = order[kk:kk + mm]
    excluded = [int(j) for j in order[:kk + mm]]
    wanted = ([0] if p.global_sentinels & 1 else []) + ([v - 1] if p.global_sentinels & 2 else [])
    for slot, j in enumerate(wanted):
        if v > 0 and j not in excluded:
            sent[p.m + p.r + slot] = j
            excluded.append(j)
    rand = draw_random_sentinels(excluded, v, p.r, p.seed, g, layer)
    sent[p.m:p.m + len(rand)] = rand
    kth = float(s_row[order[kk - 1]])
    margin = float(kth - s_row[order[kk]]) if v > kk else float("inf")
    return route, sent, kth, margin


# --------------------------------------------------------------------------- layer steps
@dataclasses.dataclass
class LayerResult:
    ledger: Ledger
    flags: np.ndarray          # [rows] uint8 (anchor: all 1)
    alpha: np.ndarray          # [rows] float64 (anchor: nan)
    beta: np.ndarray           # [rows] float64
    refresh_rows: np.ndarray   # ascending global-within-call row ids with flag set
    cand_scores: Optional[np.ndarray]  # [rows, c] float64, nan for empty slots (relay only)
    full_routes: np.ndarray    # [rows, k] exact TopK of this layer (recall reference)
    scores: List[np.ndarray]   # per problem S (float64, masked)
    is_anchor: bool
    forced: bool = False       # a relay call that the adaptive policy ran as an anchor


def _problem_rows(p: OracleParams, slot: int) -> slice:
    return slice(slot * p.n_q, (slot + 1) * p.n_q)


def _exact_routes(s: np.ndarray, p: OracleParams) -> np.ndarray:
    v = p.valid_counts()
    out = np.full((p.n_q, p.k), -1, np.int32)
    for i in range(p.n_q):
        fr = full_route(s[i], int(v[i]), p.k)
        out[i, : len(fr)] = fr
    return out


def anchor_layer(q: np.ndarray, k: np.ndarray, p: OracleParams, layer: int,
                 problem_ids: Optional[Sequence[int]] = None) -> LayerResult:
    """Anchor: full routing of every row, ledger rebuilt from a complete score matrix
    (Sec 4.1).  q, k: [P, n, d]."""
    P = q.shape[0]
    problem_ids = list(range(P)) if problem_ids is None else list(problem_ids)
    rows = P * p.n_q
    led = Ledger.empty(rows, p)
    v = p.valid_counts()
    full = np.full((rows, p.k), -1, np.int32)
    all_s = []
    for slot in range(P):
        s = scores(q[slot], k[slot], p)
        all_s.append(s)
        base = slot * p.n_q
        for i in range(p.n_q):
            g = problem_ids[slot] * p.n_q + i
            route, sent, kth, margin = route_row(s[i], int(v[i]), p, g, layer)
            led.routes[base + i] = route
            led.sentinels[base + i] = sent
            led.kth[base + i] = kth
            led.margin[base + i] = margin
        led.ages[base:base + p.n_q] = 0
        full[base:base + p.n_q] = led.routes[base:base + p.n_q]
    nan = np.full(rows, np.nan)
    return LayerResult(led, np.ones(rows, np.uint8), nan, nan.copy(),
                       np.arange(rows, dtype=np.int64), None, full, all_s, True)


def candidate_scores(s: np.ndarray, routes: np.ndarray, sentinels: np.ndarray):
    """Sec 3.2: current scores of the candidate set A_i = route U sentinels.

    Returns (cand[rows_of_problem, c] with nan in empty slots, alpha, beta, has_sentinel)."""
    cand_idx = np.concatenate([routes, sentinels], axis=1)
    safe = np.where(cand_idx >= 0, cand_idx, 0)
    cand = np.take_along_axis(s, safe, axis=1)
    cand = np.where(cand_idx >= 0, cand, np.nan)
    kw = routes.shape[1]
    r_sc = np.where(routes >= 0, cand[:, :kw], np.inf)
    s_sc = np.where(sentinels >= 0, cand[:, kw:], -np.inf)
    alpha = r_sc.min(axis=1)
    beta = s_sc.max(axis=1) if sentinels.shape[1] else np.full(len(routes), -np.inf)
    has_sent = (sentinels >= 0).any(axis=1) if sentinels.shape[1] else np.zeros(len(routes), bool)
    return cand, alpha, beta, has_sent


def relay_layer(prev: Ledger, q: np.ndarray, k: np.ndarray, p: OracleParams, layer: int,
                problem_ids: Optional[Sequence[int]] = None) -> LayerResult:
    """Relay step (Sec 3.2, 4.1, 4.2): rescore candidates, challenge test (Eq. 5),
    compaction, full re-route of the flagged rows, ledger update."""
    P = q.shape[0]
    problem_ids = list(range(P)) if problem_ids is None else list(problem_ids)
    rows = P * p.n_q
    if np.any(prev.ages < 0):
        raise ValueError("relay on a ledger that was never anchored")
    led = prev.copy()
    v = p.valid_counts()
    flags = np.zeros(rows, np.uint8)
    alpha = np.empty(rows)
    beta = np.empty(rows)
    cand_all = np.empty((rows, p.c))
    full = np.full((rows, p.k), -1, np.int32)
    all_s = []
    for slot in range(P):
        sl = _problem_rows(p, slot)
        s = scores(q[slot], k[slot], p)
        all_s.append(s)
        full[sl] = _exact_routes(s, p)
        cand, a, b, has_sent = candidate_scores(s, prev.routes[sl], prev.sentinels[sl])
        cand_all[sl] = cand
        alpha[sl] = a
        beta[sl] = b
        reuse = np.zeros(p.n_q, bool)
        for i in range(p.n_q):
            age = int(prev.ages[sl][i])
            # guard margin of the row: larger while the margin recorded at its last routing is
            # below the recovery level (decided in float32, the precision the ledger stores)
            weak = bool(np.float32(prev.margin[sl][i]) < np.float32(p.margin_recover))
            gamma_i = p.gamma + (p.gamma_boost if weak else 0.0)
            # Eq. 5: reuse iff alpha > beta + gamma_i; a row without sentinels is never flagged
            reuse[i] = (not has_sent[i]) or bool(a[i] > b[i] + gamma_i)
            if age < p.min_reuse:              # minimum reuse horizon: not tested yet
                reuse[i] = True
            if p.h_max > 0 and age >= p.h_max:  # forced re-routing of an old route
                reuse[i] = False
        flags[sl] = (~reuse).astype(np.uint8)
    refresh_rows = np.nonzero(flags)[0].astype(np.int64)       # ascending = prefix-sum order
    for gr in refresh_rows:
        slot, i = divmod(int(gr), p.n_q)
        g = problem_ids[slot] * p.n_q + i
        route, sent, kth, margin = route_row(all_s[slot][i], int(v[i]), p, g, layer)
        led.routes[gr] = route
        led.sentinels[gr] = sent
        led.kth[gr] = kth
        led.margin[gr] = margin
    stable = flags == 0
    led.ages[stable] += 1
    led.ages[~stable] = 0
    return LayerResult(led, flags, alpha, beta, refresh_rows, cand_all, full, all_s, False)


class AnchorForcer:
    """Forced anchors "before layers known to have low route persistence" (Sec 3.2), with the
    persistence read off the last tested relay layer.  State: `left` = relay calls still to be
    run as forced anchors, `run` = length of the last forced run (back-off memory).

    * a tested relay layer that flags F >= ceil(rows * force_permille / 1000) rows forces the next
      `run` relay calls, run = min(max(1, 2 * previous run), force_max_run): while the flagged
      count stays high the forced runs double, up to force_max_run, and one tested layer probes
      between two runs; a tested layer below the threshold resets the back-off (run = 0);
    * a forced relay call routes every row exactly like an anchor (flags all 1, ages 0, sentinels
      redrawn at that layer) and decrements `left`;
    * a scheduled anchor clears `left` and leaves `run`."""

    def __init__(self, p: "OracleParams", rows: int):
        self.on = p.force_permille > 0
        self.threshold = (rows * p.force_permille + 999) // 1000
        self.max_run = max(1, p.force_max_run)
        self.left = 0
        self.run = 0

    def forced_now(self) -> bool:
        return self.on and self.left > 0

    def after_forced(self) -> None:
        self.left -= 1

    def after_anchor(self) -> None:
        self.left = 0

    def after_tested(self, flagged: int) -> None:
        if not self.on:
            return
        if flagged >= self.threshold:
            self.run = min(max(1, 2 * self.run), self.max_run)
            self.left = self.run
        else:
            self.run = 0


# --------------------------------------------------------------------------- metrics
def recall_counts(routes: np.ndarray, full: np.ndarray):
    """(|route ∩ full| summed over rows, |full| summed over rows)."""
    hit = 0
    tot = 0
    for a, b in zip(routes, full):
        fb = set(int(x) for x in b if x >= 0)
        hit += len(fb.intersection(int(x) for x in a if x >= 0))
        tot += len(fb)
    return hit, tot


def valid_candidate_counts(led: Ledger) -> np.ndarray:
    return (led.routes >= 0).sum(axis=1) + (led.sentinels >= 0).sum(axis=1)


@dataclasses.dataclass
class RunSummary:
    recall_all: float
    recall_relay: float
    rerouted_fraction: float       # (anchor rows + flagged relay rows) / (L * rows)
    flagged_relay_fraction: float  # flagged relay rows / relay rows
    score_pair_fraction: float
    counters: Dict[str, int]


def work_counters(p: OracleParams, P: int, layer_kinds: Sequence[bool],
                  flags_per_layer: Sequence[np.ndarray],
                  cand_counts_per_layer: Sequence[Optional[np.ndarray]]) -> Dict[str, int]:
    """Work accounting as recovered from the paper's sentinel-ablation table:
    every anchor row is charged its full row (v_i pairs); every relay row is charged its
    candidate count; every flagged relay row is additionally charged its full row.  The
    denominator is full routing on every layer."""
    v = np.tile(p.valid_counts(), P)
    c = dict(anchor_rows=0, relay_rows=0, flagged_rows=0, cand_pairs=0, full_pairs=0,
             dense_pairs=0)
    for is_anchor, flags, cc in zip(layer_kinds, flags_per_layer, cand_counts_per_layer):
        c["dense_pairs"] += int(v.sum())
        if is_anchor:
            c["anchor_rows"] += len(v)
            c["full_pairs"] += int(v.sum())
        else:
            c["relay_rows"] += len(v)
            c["flagged_rows"] += int(flags.sum())
            c["cand_pairs"] += int(cc.sum())
            c["full_pairs"] += int(v[flags != 0].sum())
    return c


def fractions_from_counters(c: Dict[str, int]):
    total_rows = c["anchor_rows"] + c["relay_rows"]
    rerouted = (c["anchor_rows"] + c["flagged_rows"]) / total_rows
    pairs = (c["cand_pairs"] + c["full_pairs"]) / c["dense_pairs"]
    flagged = c["flagged_rows"] / c["relay_rows"] if c["relay_rows"] else 0.0
    return rerouted, flagged, pairs


def run_layers(q_layers: np.ndarray, k_layers: np.ndarray, p: OracleParams,
               anchor_every: int, problem_ids: Optional[Sequence[int]] = None,
               keep_scores: bool = False):
    """Free-running pass over all layers.  q_layers/k_layers: [L, P, n, d].
    Layer l is an anchor iff l % anchor_every == 0 (forced anchors, Sec 3.2).
    Returns (list of LayerResult, RunSummary)."""
    L, P = q_layers.shape[0], q_layers.shape[1]
    results: List[LayerResult] = []
    led: Optional[Ledger] = None
    kinds, flags_l, cc_l = [], [], []
    hit_all = tot_all = hit_rel = tot_rel = 0
    forcer = AnchorForcer(p, P * p.n_q)
    for l in range(L):
        is_anchor = (l % anchor_every == 0)
        if is_anchor:
            res = anchor_layer(q_layers[l], k_layers[l], p, l, problem_ids)
            cc = None
            forcer.after_anchor()
        elif forcer.forced_now():                  # a relay call run as a forced anchor
            res = anchor_layer(q_layers[l], k_layers[l], p, l, problem_ids)
            res.forced = True
            cc = None
            is_anchor = True
            forcer.after_forced()
        else:
            cc = valid_candidate_counts(led)
            res = relay_layer(led, q_layers[l], k_layers[l], p, l, problem_ids)
            forcer.after_tested(int(res.flags.sum()))
        led = res.ledger
        h, t = recall_counts(led.routes, res.full_routes)
        hit_all += h
        tot_all += t
        if not is_anchor:
            hit_rel += h
            tot_rel += t
        kinds.append(is_anchor)
        flags_l.append(res.flags)
        cc_l.append(cc)
        if not keep_scores:
            res.scores = []
        results.append(res)
    counters = work_counters(p, P, kinds, flags_l, cc_l)
    rerouted, flagged, pairs = fractions_from_counters(counters)
    summary = RunSummary(hit_all / tot_all, (hit_rel / tot_rel) if tot_rel else 1.0,
                         rerouted, flagged, pairs, counters)
    return results, summary


def token_ranges(routes: np.ndarray, chunk_tokens: int, coalesce: bool = False) -> np.ndarray:
    """Expansion of selected chunks into token index ranges (Sec 2.1): each row's chunk ids
    in ascending order, chunk j -> [j*T, (j+1)*T); empty slots (-1,-1) at the end.
    With `coalesce`, runs of consecutive chunk ids become one range."""
    rows, k = routes.shape
    out = np.full((rows, k, 2), -1, np.int32)
    for i in range(rows):
        ids = sorted(int(j) for j in routes[i] if j >= 0)
        s = 0
        for pos, j in enumerate(ids):
            if coalesce and pos > 0 and ids[pos - 1] == j - 1:
                out[i, s - 1, 1] = (j + 1) * chunk_tokens       # extends the current run
                continue
            out[i, s, 0] = j * chunk_tokens
            out[i, s, 1] = (j + 1) * chunk_tokens
            s += 1
    return out


def routed_attention(q: np.ndarray, keys: np.ndarray, values: np.ndarray, routes: np.ndarray,
                     chunk_tokens: int, scale: float) -> np.ndarray:
    """Eq. 3: o_i = softmax(q_i K_R^T * scale) V_R, R = the tokens of the chunks in row i's route
    (chunk j = tokens [j*T, (j+1)*T), clipped to the sequence).  One problem: q [n_q, dh],
    keys / values [tokens, dh], routes [n_q, k] with -1 for empty slots.  float64; a row with an
    empty route gets zeros."""
    q = np.asarray(q, np.float64)
    keys = np.asarray(keys, np.float64)
    values = np.asarray(values, np.float64)
    out = np.zeros((q.shape[0], values.shape[1]))
    for i in range(q.shape[0]):
        tok: List[int] = []
        for j in sorted(set(int(c) for c in routes[i] if c >= 0)):
            tok.extend(range(j * chunk_tokens, min((j + 1) * chunk_tokens, keys.shape[0])))
        if not tok:
            continue
        logits = keys[tok] @ q[i] * scale
        w = np.exp(logits - logits.max())
        out[i] = (w / w.sum()) @ values[tok]
    return out
