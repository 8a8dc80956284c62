"""Seeded synthetic chunk-embedding workloads (inputs only).

This module draws the per-layer chunk representations Qc, Kc that feed both the
CUDA path and the CPU checker.  It holds none of the routing method's
arithmetic: no scores, no selection, no sentinels.

The paper's evaluation (Section 5, "Cross-Layer Route Stability" setup) uses
synthetic rows with "persistent preferred chunks" and "layer-local Gaussian
drift" without specifying the generator.  The stand-in used here:

* per problem (one batch x head pair) C centroids mu_c ~ N(0, I/d), shared by
  the query chunks and the key chunks of that problem;
* every row draws one centroid uniformly at random and starts at
  X_0 = mu + (0.5/sqrt(d)) * N(0, I);
* every later layer applies X <- sqrt(1-rho^2) * X + rho * G, G ~ N(0, I/d),
  independently for Qc and Kc, on an fp32 master copy;
* optionally (the "high drift at scale" configuration) every `redraw_every`-th
  layer re-draws round(redraw_frac * C) centroids and re-samples the rows that
  belong to them around the new centroid (abrupt route shifts);
* for bf16 configurations each layer's master is rounded once to bf16
  (round-to-nearest-even); that exact tensor is what every consumer sees.

Streams are per problem: problem p of a configuration is a function of
(seed, p) alone, so any subset of problems can be regenerated bit-identically.
"""
from __future__ import annotations

import dataclasses
from concurrent.futures import ThreadPoolExecutor
from typing import Iterable, List, Optional, Sequence, Tuple

import numpy as np

DTYPE_BF16 = 0
DTYPE_F32 = 1


@dataclasses.dataclass(frozen=True)
class RouteWorkload:
    """One routing configuration: shapes, ledger widths, drift recipe, schedule."""

    name: str
    batch: int
    heads: int
    n_q: int
    n_k: int
    d: int
    k: int            # route width (Eq. 2)
    m: int            # near-miss sentinels per row (Section 3.1)
    r: int            # random sentinels per row (Section 3.1)
    layers: int
    anchor_every: int  # layer l is an anchor iff l % anchor_every == 0
    dtype: int         # DTYPE_BF16 or DTYPE_F32
    centroids: int
    rho: float
    causal: bool
    gamma: float = 0.0
    seed: int = 0
    redraw_every: int = 0     # 0 = never
    redraw_frac: float = 0.0
    chunk_tokens: int = 0     # >0: routes are also expanded to token ranges
    coalesce_ranges: bool = False   # token ranges of adjacent chunks merged
    causal_offset: int = 0    # causal: row i sees chunks j < min(n_k, i + 1 + causal_offset)
    # optional policies (Section 3.1 item 3, Section 3.2 "Hysteresis" / "Forced anchors")
    global_sentinels: int = 0   # bit 0: sink chunk, bit 1: most recent chunk
    min_reuse: int = 0
    gamma_boost: float = 0.0
    margin_recover: float = 0.0
    h_max: int = 0
    force_permille: int = 0     # forced anchors after a relay that flags this many per mille of the rows
    force_max_run: int = 1

    @property
    def problems(self) -> int:
        return self.batch * self.heads

    @property
    def rows(self) -> int:
        return self.problems * self.n_q

    @property
    def sw(self) -> int:
        return self.m + self.r + (self.global_sentinels & 1) + ((self.global_sentinels >> 1) & 1)

    @property
    def c(self) -> int:
        return self.k + self.sw

    def is_anchor(self, layer: int) -> bool:
        return layer % self.anchor_every == 0

    def replace(self, **kw) -> "RouteWorkload":
        return dataclasses.replace(self, **kw)


def tiny() -> RouteWorkload:
    return RouteWorkload("tiny", 1, 1, 128, 128, 64, 8, 4, 4, layers=4, anchor_every=4,
                         dtype=DTYPE_F32, centroids=16, rho=0.05, causal=False)


def moderate() -> RouteWorkload:
    return RouteWorkload("moderate", 1, 8, 256, 256, 128, 16, 8, 8, layers=12, anchor_every=6,
                         dtype=DTYPE_BF16, centroids=32, rho=0.15, causal=True)


def sweep(n: int = 1024, rho: float = 0.30) -> RouteWorkload:
    return RouteWorkload(f"sweep_n{n}_rho{rho:g}", 1, 32, n, n, 128, 32, 16, 16, layers=16,
                         anchor_every=8, dtype=DTYPE_BF16, centroids=64, rho=rho, causal=True)


def high_drift() -> RouteWorkload:
    return RouteWorkload("high_drift", 8, 32, 1024, 1024, 128, 32, 16, 16, layers=32,
                         anchor_every=8, dtype=DTYPE_BF16, centroids=64, rho=0.30, causal=True,
                         redraw_every=4, redraw_frac=0.10)


def long_ctx() -> RouteWorkload:
    return RouteWorkload("long_ctx", 2, 32, 2048, 2048, 128, 64, 32, 32, layers=32,
                         anchor_every=16, dtype=DTYPE_BF16, centroids=128, rho=0.15, causal=True,
                         chunk_tokens=64)


def low_drift() -> RouteWorkload:
    """The headline shape in the regime the method is built for: slow drift, few flagged rows."""
    return RouteWorkload("low_drift", 8, 32, 1024, 1024, 128, 32, 16, 16, layers=32,
                         anchor_every=8, dtype=DTYPE_BF16, centroids=64, rho=0.005, causal=True)


def ablation(m: int = 12, r: int = 12) -> RouteWorkload:
    """Shape of the sentinel-ablation table (Section 5.2): 256 x 256 chunks, top-12 routes,
    24 layers with a single anchor at layer 0; (m, r) = (0, 0) is the fixed-stride baseline."""
    return RouteWorkload(f"ablation_m{m}_r{r}", 8, 32, 256, 256, 128, 12, m, r, layers=24,
                         anchor_every=24, dtype=DTYPE_BF16, centroids=32, rho=0.003, causal=False)


PRESETS = {
    "tiny": tiny,
    "moderate": moderate,
    "sweep": sweep,
    "high_drift": high_drift,
    "long_ctx": long_ctx,
    "low_drift": low_drift,
    "ablation_m0_r12": lambda: ablation(0, 12),
    "ablation_m12_r12": lambda: ablation(12, 12),
    "ablation_m24_r12": lambda: ablation(24, 12),
    "ablation_m48_r12": lambda: ablation(48, 12),
    "ablation_m12_r0": lambda: ablation(12, 0),
    "fixed_stride": lambda: ablation(0, 0),
}


# ----------------------------------------------------------------------------- bf16 helpers
def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round fp32 to bf16 (nearest, ties to even); returns the uint16 bit patterns."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32)
    bias = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + bias) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """Exact fp32 value of bf16 bit patterns."""
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


# ----------------------------------------------------------------------------- generator
class ProblemStream:
    """Layer-by-layer generator for one problem (one batch x head pair)."""

    def __init__(self, w: RouteWorkload, problem: int):
        self.w = w
        self.problem = problem
        self.rng = np.random.default_rng([int(w.seed), int(problem), 0x52525F77])
        d = w.d
        self.inv_sqrt_d = np.float32(1.0 / np.sqrt(d))
        self.mu = self.rng.standard_normal((w.centroids, d), dtype=np.float32) * self.inv_sqrt_d
        self.assign_q = self.rng.integers(0, w.centroids, size=w.n_q)
        self.assign_k = self.rng.integers(0, w.centroids, size=w.n_k)
        self.q = self._around(self.mu[self.assign_q])
        self.k = self._around(self.mu[self.assign_k])
        self.layer = 0

    def _around(self, centre: np.ndarray) -> np.ndarray:
        noise = self.rng.standard_normal(centre.shape, dtype=np.float32)
        return (centre + np.float32(0.5) * self.inv_sqrt_d * noise).astype(np.float32)

    def _drift(self, x: np.ndarray) -> np.ndarray:
        w = self.w
        g = self.rng.standard_normal(x.shape, dtype=np.float32) * self.inv_sqrt_d
        keep = np.float32(np.sqrt(1.0 - w.rho * w.rho))
        return (keep * x + np.float32(w.rho) * g).astype(np.float32)

    def _redraw(self) -> None:
        w = self.w
        n_new = int(round(w.redraw_frac * w.centroids))
        if n_new <= 0:
            return
        which = self.rng.choice(w.centroids, size=n_new, replace=False)
        self.mu[which] = self.rng.standard_normal((n_new, w.d), dtype=np.float32) * self.inv_sqrt_d
        hit_q = np.isin(self.assign_q, which)
        hit_k = np.isin(self.assign_k, which)
        self.q[hit_q] = self._around(self.mu[self.assign_q[hit_q]])
        self.k[hit_k] = self._around(self.mu[self.assign_k[hit_k]])

    def next_layer(self) -> Tuple[np.ndarray, np.ndarray]:
        """fp32 masters (n_q,d), (n_k,d) of the next layer (layer 0 first)."""
        w = self.w
        if self.layer > 0:
            self.q = self._drift(self.q)
            self.k = self._drift(self.k)
            if w.redraw_every and self.layer % w.redraw_every == 0:
                self._redraw()
        self.layer += 1
        return self.q, self.k


def _problem_layers(w: RouteWorkload, problem: int, layers: int):
    s = ProblemStream(w, problem)
    if w.dtype == DTYPE_BF16:
        q = np.empty((layers, w.n_q, w.d), np.uint16)
        k = np.empty((layers, w.n_k, w.d), np.uint16)
        for l in range(layers):
            mq, mk = s.next_layer()
            q[l] = f32_to_bf16_bits(mq)
            k[l] = f32_to_bf16_bits(mk)
    else:
        q = np.empty((layers, w.n_q, w.d), np.float32)
        k = np.empty((layers, w.n_k, w.d), np.float32)
        for l in range(layers):
            mq, mk = s.next_layer()
            q[l] = mq
            k[l] = mk
    return q, k


def generate(w: RouteWorkload, problems: Optional[Sequence[int]] = None,
             layers: Optional[int] = None, threads: int = 0,
             out_q: Optional[np.ndarray] = None, out_k: Optional[np.ndarray] = None):
    """Generate all layers for the listed problems (default: all).

    Returns (Qc, Kc) with shape [layers, len(problems), n, d]; dtype uint16 (bf16 bit
    patterns) for bf16 configurations, float32 otherwise.  `out_q`/`out_k` may be
    preallocated arrays of that shape (e.g. views of pinned host memory).
    """
    if problems is None:
        problems = range(w.problems)
    problems = list(problems)
    layers = w.layers if layers is None else int(layers)
    np_dtype = np.uint16 if w.dtype == DTYPE_BF16 else np.float32
    if out_q is None:
        out_q = np.empty((layers, len(problems), w.n_q, w.d), np_dtype)
    if out_k is None:
        out_k = np.empty((layers, len(problems), w.n_k, w.d), np_dtype)

    def work(slot_problem):
        slot, p = slot_problem
        q, k = _problem_layers(w, p, layers)
        out_q[:, slot] = q
        out_k[:, slot] = k

    jobs = list(enumerate(problems))
    if threads and threads > 1 and len(jobs) > 1:
        with ThreadPoolExecutor(max_workers=threads) as ex:
            list(ex.map(work, jobs))
    else:
        for j in jobs:
            work(j)
    return out_q, out_k


def as_float32(x: np.ndarray) -> np.ndarray:
    """Exact fp32 values of a generated tensor (bf16 bit patterns or fp32)."""
    if x.dtype == np.uint16:
        return bf16_bits_to_f32(x)
    return np.asarray(x, dtype=np.float32)
