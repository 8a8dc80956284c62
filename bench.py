#!/usr/bin/env python
"""Benchmark of the route-maintenance hot path (one JSON line on stdout).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload high_drift]
    python bench.py --impl reference ...        # the CPU oracle on the host cores

A step is one pass of the whole hot path over one batch of synthetic input: every layer
of the workload's schedule (anchor layers: score GEMM + TopK + sentinel build; relay layers:
candidate rescoring, challenge test, compaction, row-selective refresh, ledger update).
`value` = query rows routed per second per layer = rows * layers * n_gpus / time.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2609_07306_b200 import workload as W  # noqa: E402

METRIC = "layer-route rows/sec per layer (n_k=1024) vs full GEMM+TopK routing"
UNIT = "rows/s"


def _peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return dict(hbm_gbs=float(d["hbm_gbs"]), bf16_tflops=float(d["bf16_tflops"]),
                    bf16_tflops_sustained=float(d.get("bf16_tflops_sustained", d["bf16_tflops"])),
                    source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0,
                source="fallback")


L2_BYTES = 126 << 20


def _workload(name: str) -> W.RouteWorkload:
    if name == "sweep1024":
        return W.sweep(1024, 0.30)
    if name.startswith("sweep_"):                     # sweep_<n>_<rho>, e.g. sweep_256_0.15
        _, n, rho = name.split("_")
        return W.sweep(int(n), float(rho))
    return W.PRESETS[name]()


# ----------------------------------------------------------------------------- reference arm
def _oracle_sample(w: W.RouteWorkload, n_problems: int, n_layers: int):
    """Times the CPU oracle, as it stands, on a bounded sample of the workload."""
    from oracle import routerelay_oracle as O
    problems = list(range(min(n_problems, w.problems)))
    n_layers = min(n_layers, w.layers)
    q, k = W.generate(w, problems=problems, layers=n_layers)
    qf = W.as_float32(q).astype(np.float64)
    kf = W.as_float32(k).astype(np.float64)
    p = O.OracleParams(n_q=w.n_q, n_k=w.n_k, k=w.k, m=w.m, r=w.r, gamma=w.gamma, causal=w.causal,
                       causal_offset=0, seed=w.seed)
    t0 = time.perf_counter()
    _, summ = O.run_layers(qf, kf, p, w.anchor_every, problems)
    dt = time.perf_counter() - t0
    rows = len(problems) * w.n_q * n_layers
    return rows / dt, dt, summ, f"{len(problems)} of {w.problems} problems x first {n_layers} of " \
                                f"{w.layers} layers ({rows} row-layers, {dt:.1f} s)"


def _timed_sample(w: W.RouteWorkload, n_problems: int, n_layers: int, repeats: int = 5):
    """Times the oracle's vectorised fp32 mode (BLAS matmul + argpartition) on a sample of the
    workload; median of `repeats` runs."""
    from oracle import routerelay_timed as T
    problems = list(range(min(n_problems, w.problems)))
    n_layers = min(n_layers, w.layers)
    q, k = W.generate(w, problems=problems, layers=n_layers)
    qf, kf = W.as_float32(q), W.as_float32(k)
    times = []
    for _ in range(repeats):
        t0 = time.perf_counter()
        T.run_layers(qf, kf, w.n_q, w.n_k, w.k, w.m, w.r, w.gamma, w.causal, w.seed,
                     w.anchor_every, problems)
        times.append(time.perf_counter() - t0)
    dt = statistics.median(times)
    rows = len(problems) * w.n_q * n_layers
    return rows / dt, dt, f"{len(problems)} of {w.problems} problems x first {n_layers} of " \
                          f"{w.layers} layers ({rows} row-layers, median of {repeats} runs, " \
                          f"{dt:.2f} s each)"


def _blas_threads() -> int:
    try:
        from threadpoolctl import threadpool_info
        return max([int(i.get("num_threads", 1)) for i in threadpool_info()] or [1])
    except Exception:
        return 1


def run_reference(args) -> None:
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    w = _workload(args.workload)
    vals = []
    sample = ""
    for s in range(args.warmup + args.steps):
        v, dt, summ, sample = _oracle_sample(w, 2, 5)
        if s >= args.warmup:
            vals.append((v, dt))
    ms = 1e3 * statistics.median(dt for _, dt in vals)
    value = statistics.median(v for v, _ in vals)
    cores = _blas_threads()
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": w.name, "sample_per_step": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores,
                         "os_cpu_count": os.cpu_count(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# ----------------------------------------------------------------------------- clocks
class ClockSampler:
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.proc = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                 "-lms", "50", "-i", str(gpu_index)],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except Exception:
            self.proc.kill()
            out = ""
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.strip().splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); mx.append(float(f[2]))
            except ValueError:
                continue
            for nm, val in zip(names, f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(nm)
        return {"sm_mhz": statistics.median(sm) if sm else None,
                "sm_max_mhz": max(mx) if mx else None, "samples": len(sm),
                "reasons": sorted(reasons)}


# DRAM traffic per launch (dram__bytes_read.sum + dram__bytes_write.sum) of the kernels that
# dominate a high_drift step, from the ncu captures summarised in profiles/
# (route_sweep_high_drift.md: 199.1 MB anchor / 198.6 MB refresh; rescore_dense_high_drift.md;
# sentinels_high_drift.md), and the algorithmic bytes per launch of the same launches.  Other
# workloads report the capture's traffic-to-algorithmic ratio times their own algorithmic bytes
# and say so.
NCU_TRAFFIC_BYTES = {"route_fused": ((4 * 199.1e6 + 28 * 198.6e6) / 32, (4 * 203.4e6 + 28 * 196.7e6) / 32),
                     "rescore_dense": (241.3e6, 203.7e6),
                     "sentinels": (66.5e6, 0.971 * 262144 * 64 * 4)}


def _traffic(kind, workload_name, alg_bytes_per_launch, truncated):
    if kind not in NCU_TRAFFIC_BYTES or alg_bytes_per_launch is None:
        return None, None
    measured, alg = NCU_TRAFFIC_BYTES[kind]
    if workload_name == "high_drift" and not truncated:
        return measured, "ncu capture (profiles/)"
    return measured / alg * alg_bytes_per_launch, "scaled from the high_drift capture by algorithmic bytes"


# ----------------------------------------------------------------------------- roofline
def _kernel_roofline(kind, ms, launches, w, cnt, peaks, sm_mhz):
    """Algorithmic work of one kernel kind over one step, its bound and measured peak.

    cnt: work counters of one step (anchor_rows, relay_rows, flagged_rows, cand_pairs,
    full_pairs).  Per unit: a routed row = 2*d*v_i FLOP of scores and (c+2)*4 bytes of ledger
    row; a layer call reads its inputs once, P*(n_q+n_k)*d*element bytes; a relay row reads c*4
    bytes of ledger ids and writes 13 bytes (flag, alpha, beta, tau)."""
    esz = 2 if w.dtype == W.DTYPE_BF16 else 4
    routed = cnt["anchor_rows"] + cnt["flagged_rows"]
    layer_calls = cnt["layer_calls"]
    n_anchor = cnt["anchor_rows"] // w.rows
    in_bytes = w.problems * (w.n_q + w.n_k) * w.d * esz
    ledger_row = (w.c + 2) * 4
    sec = ms * 1e-3
    if kind == "topk_rows":        # reads score rows, writes ledger rows
        alg = cnt["full_pairs"] * 4 + routed * ledger_row
        return dict(bound="hbm", achieved=alg / sec / 1e9, peak=peaks["hbm_gbs"], unit="GB/s",
                    alg_per_launch=alg / launches, alg_bytes_per_launch=alg / launches)
    if kind in ("rescore", "rescore_dense"):   # unique bytes: inputs + ledger ids + flags/alpha/beta
        alg = (layer_calls - n_anchor) * (in_bytes + w.rows * (w.c * 4 + 9))
        return dict(bound="hbm", achieved=alg / sec / 1e9, peak=peaks["hbm_gbs"], unit="GB/s",
                    alg_per_launch=alg / launches, alg_bytes_per_launch=alg / launches)
    if kind == "score_simt":       # fp32 FMA: 2*d flop per score pair
        alg = 2.0 * w.d * cnt["full_pairs"]
        mhz = sm_mhz or 1965.0
        peak = 148 * 128 * 2 * mhz * 1e6 / 1e12
        return dict(bound="alu", achieved=alg / sec / 1e12, peak=peak, unit="TFLOP/s",
                    alg_per_launch=alg / launches)
    if kind in ("score_tc", "route_fused"):
        alg = 2.0 * w.d * cnt["full_pairs"]
        out = dict(bound="tensor", achieved=alg / sec / 1e12,
                   peak=peaks["bf16_tflops_sustained"], unit="TFLOP/s",
                   alg_per_launch=alg / launches)
        if kind == "route_fused":   # also against HBM: inputs of every routed tile + ledger rows
            calls = layer_calls
            alg_b = calls * in_bytes * (routed / (calls * w.rows)) + routed * ledger_row
            out["hbm_achieved_gbs"] = alg_b / sec / 1e9
            out["hbm_frac"] = out["hbm_achieved_gbs"] / peaks["hbm_gbs"]
            out["alg_bytes_per_launch"] = alg_b / launches
        return out
    if kind == "sentinels":        # reads a routed row's route + near-miss ids, writes the rest
        alg = routed * w.c * 4
        return dict(bound="hbm", achieved=alg / sec / 1e9, peak=peaks["hbm_gbs"], unit="GB/s",
                    alg_per_launch=alg / launches, alg_bytes_per_launch=alg / launches)
    if kind == "compact":
        alg = (layer_calls - n_anchor) * w.rows + cnt["flagged_rows"] * 4
        return dict(bound="hbm", achieved=alg / sec / 1e9, peak=peaks["hbm_gbs"], unit="GB/s",
                    alg_per_launch=alg / launches, alg_bytes_per_launch=alg / launches)
    alg = layer_calls * w.rows * 9
    return dict(bound="hbm", achieved=alg / sec / 1e9, peak=peaks["hbm_gbs"], unit="GB/s",
                alg_per_launch=alg / launches, alg_bytes_per_launch=alg / launches)


# ----------------------------------------------------------------------------- multi-GPU plumbing
def shard_workload(w: W.RouteWorkload, rank: int) -> W.RouteWorkload:
    """Routing problems are independent (the ledger, the scores and the refresh decisions of a
    row never cross its batch x head pair), so N GPUs need no exchange on the data path: every
    rank routes its own batch of problems (weak scaling).  Rank r's batch is the workload with
    seed r, i.e. different problems on every rank."""
    return w.replace(seed=int(w.seed) + int(rank))


def max_over_ranks(x: float, world: int, device=None) -> float:
    """Step time of the job = the slowest rank's device time."""
    if world == 1:
        return float(x)
    import torch
    import torch.distributed as dist
    t = torch.tensor([x], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_rows_per_s(rows_per_rank: int, layers: int, world: int, ms_per_step: float) -> float:
    """Whole-job throughput: all ranks' rows x layers over the slowest rank's step time."""
    return rows_per_rank * layers * world / (ms_per_step * 1e-3)


# ----------------------------------------------------------------------------- our arm
def run_ours(args) -> None:
    import torch
    import torch.distributed as dist

    from paper_2609_07306_b200 import binding as B
    from paper_2609_07306_b200.ledger import RouteLedger, config_from_workload

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU path "
                         "(use --impl reference for the CPU oracle)")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=dev)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    w = shard_workload(_workload(args.workload), rank)   # weak scaling: own problems per rank
    if args.layers:
        w = w.replace(layers=min(args.layers, w.layers))
    L = w.layers
    peaks = _peaks()
    esz = 2 if w.dtype == W.DTYPE_BF16 else 4
    tdt = torch.int16 if w.dtype == W.DTYPE_BF16 else torch.float32
    ndt = np.uint16 if w.dtype == W.DTYPE_BF16 else np.float32

    # ---- inputs: generated on the host into pinned memory, then staged to the device -----
    t_gen = time.perf_counter()
    hq = torch.empty((L, w.problems, w.n_q, w.d), dtype=tdt).pin_memory()
    hk = torch.empty((L, w.problems, w.n_k, w.d), dtype=tdt).pin_memory()
    W.generate(w, threads=max(1, (os.cpu_count() or 8) // max(1, world)),
               out_q=hq.numpy().view(ndt), out_k=hk.numpy().view(ndt))
    t_gen = time.perf_counter() - t_gen
    dq, dk = hq.to(dev), hk.to(dev)
    if w.dtype == W.DTYPE_BF16:
        dq, dk = dq.view(torch.bfloat16), dk.view(torch.bfloat16)

    cfg = config_from_workload(w, two_pass=args.two_pass, gathered=args.gathered,
                               streaming=args.streaming, inplace=args.inplace)
    led = RouteLedger(cfg, device=str(dev))
    stream = torch.cuda.current_stream(dev)

    def step():
        for l in range(L):
            if w.is_anchor(l):
                led.route_anchor(dq[l], dk[l], l)
            else:
                led.route_relay(dq[l], dk[l], l)

    # ---- timed region: device-resident inputs ----------------------------------------------
    for _ in range(args.warmup):
        step()
    timed_step, launches_per_replay = step, None
    if args.graph:                       # one capture of the whole step, replayed K times
        torch.cuda.synchronize(dev)
        graph, side = torch.cuda.CUDAGraph(), torch.cuda.Stream(dev)
        n0 = B.rr_kernel_launch_count()
        with torch.cuda.graph(graph, stream=side):
            step()
        launches_per_replay = B.rr_kernel_launch_count() - n0    # kernels recorded in the graph
        timed_step = graph.replay
        for _ in range(args.warmup):
            timed_step()
    barrier()
    clocks = ClockSampler(local)
    launches0 = B.rr_kernel_launch_count()
    # Every step is timed with its own pair of events on the launching stream; the reported
    # step time is the median over the K steps (the paper's statistic), the mean is kept beside
    # it.  L2: a step reads every layer's inputs once.  Where one step's inputs exceed L2
    # several times over nothing survives from step to step; smaller workloads get L2 flushed
    # (a 256 MB buffer written) before each step, outside its event pair.
    step_input_bytes = L * w.problems * (w.n_q + w.n_k) * w.d * esz
    flush_l2 = step_input_bytes < 2 * L2_BYTES
    scratch = torch.empty(256 << 20, dtype=torch.uint8, device=dev) if flush_l2 else None
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
           for _ in range(args.steps)]
    for a_ev, b_ev in evs:
        if flush_l2:
            scratch.zero_()
        a_ev.record(stream)
        timed_step()
        b_ev.record(stream)
    barrier()
    step_ms = [a_ev.elapsed_time(b_ev) for a_ev, b_ev in evs]
    del scratch
    local_ms = statistics.median(step_ms)
    mean_ms = max_over_ranks(sum(step_ms) / len(step_ms), world, dev)
    ms_per_step = max_over_ranks(local_ms, world, dev)
    launches = B.rr_kernel_launch_count() - launches0
    if launches_per_replay is not None:
        launches = launches_per_replay * args.steps
    clock_info = clocks.stop()
    value = aggregate_rows_per_s(w.rows, L, world, ms_per_step)
    if args.profile_only:            # short run for profiler captures: no extra passes
        if rank == 0:
            print(json.dumps({"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world,
                              "steps": args.steps, "warmup": args.warmup,
                              "ms_per_step": ms_per_step, "gpu_launches": int(launches),
                              "config": {"workload": w.name, "layers": L},
                              "note": "profile-only run"}))
        led.close()
        if world > 1:
            dist.destroy_process_group()
        return

    # ---- per-kernel device times (same steps, events around every launch) ---------------
    led.reset()
    B.rr_profile_begin(led.handle)
    for _ in range(args.steps):
        step()
    prof = B.rr_profile_end(led.handle, stream.cuda_stream)
    cnt = {k: v // args.steps for k, v in led.counters_dict().items()}
    tot_ms = sum(ms for ms, _ in prof.values())
    kernels = {}
    for kind, (ms, n) in sorted(prof.items(), key=lambda kv: -kv[1][0]):
        r = _kernel_roofline(kind, ms / args.steps, n / args.steps, w, cnt, peaks,
                             clock_info.get("sm_mhz"))
        kernels[kind] = {"launches_per_step": n // args.steps, "avg_us": 1e3 * ms / n,
                         "share": ms / tot_ms, "bound": r["bound"], "achieved": r["achieved"],
                         "peak": r["peak"], "unit": r["unit"], "frac": r["achieved"] / r["peak"]}
        if "hbm_frac" in r:
            kernels[kind]["hbm_achieved_gbs"] = r["hbm_achieved_gbs"]
            kernels[kind]["hbm_frac"] = r["hbm_frac"]
        kernels[kind]["alg_bytes_per_launch"] = r.get("alg_bytes_per_launch")
        tr, src = _traffic(kind, w.name, r.get("alg_bytes_per_launch"), bool(args.layers))
        if tr is not None:
            kernels[kind]["traffic"] = tr
            kernels[kind]["traffic_source"] = src
    top = next(iter(kernels))
    tk = kernels[top]
    roofline = {"kernel": top, "bound": tk["bound"], "achieved": tk["achieved"],
                "peak": tk["peak"], "unit": tk["unit"], "frac": tk["frac"],
                "peak_source": (peaks["source"] + " (sustained bf16)" if tk["bound"] == "tensor"
                                else peaks["source"]) if tk["bound"] != "alu" else
                "148 SMs x 128 FMA/clk x 2 x sampled SM clock",
                "traffic": tk.get("traffic"), "traffic_source": tk.get("traffic_source"),
                "alg_bytes_per_launch": tk.get("alg_bytes_per_launch")}
    if "hbm_frac" in tk:
        roofline["hbm_achieved_gbs"] = tk["hbm_achieved_gbs"]
        roofline["hbm_frac"] = tk["hbm_frac"]

    # ---- per-layer times: anchor layers, relay layers, and full routing on every layer ---
    def per_layer_ms(fn_of_layer):
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(L + 1)]
        ev[0].record(stream)
        for l in range(L):
            fn_of_layer(l)
            ev[l + 1].record(stream)
        torch.cuda.synchronize()
        return [ev[l].elapsed_time(ev[l + 1]) for l in range(L)]

    def sched(l):
        (led.route_anchor if w.is_anchor(l) else led.route_relay)(dq[l], dk[l], l)

    reps = [per_layer_ms(sched) for _ in range(3)]
    layer_ms = [statistics.median(r[l] for r in reps) for l in range(L)]
    anchor_ms = statistics.median(layer_ms[l] for l in range(L) if w.is_anchor(l))
    relay_ms = statistics.median(layer_ms[l] for l in range(L) if not w.is_anchor(l))
    full_led = RouteLedger(cfg, device=str(dev))
    freps = [per_layer_ms(lambda l: full_led.route_anchor(dq[l], dk[l], l)) for _ in range(3)]
    full_ms = statistics.median(statistics.median(r[l] for r in freps) for l in range(L))

    # ---- quality: recall vs full routing, refreshed-row and score-pair fractions -----------
    led.reset()
    hit = tot = 0
    for l in range(L):
        sched(l)
        full_led.route_anchor(dq[l], dk[l], l)
        a, b = led.routes, full_led.routes
        for lo in range(0, w.rows, 65536):
            aa, bb = a[lo:lo + 65536], b[lo:lo + 65536]
            inter = ((aa.unsqueeze(2) == bb.unsqueeze(1)) & (bb.unsqueeze(1) >= 0)).any(2)
            hit += int(inter.sum().item())
            tot += int((bb >= 0).sum().item())
    c1 = led.counters_dict()
    rerouted = (c1["anchor_rows"] + c1["flagged_rows"]) / (c1["anchor_rows"] + c1["relay_rows"])
    flagged = c1["flagged_rows"] / max(1, c1["relay_rows"])
    pairs = (c1["cand_pairs"] + c1["full_pairs"]) / c1["dense_pairs"]
    status = led.status()

    # ---- the forced-anchor policy (Section 3.2) on the same inputs -----------------------------
    # Relay calls that follow a tested relay with at least 90 % of the rows flagged route every
    # row like an anchor (decided on the device; runs double up to 8 calls).  Not the headline:
    # it shows what the schedule costs when the method itself notices that routes do not persist.
    adaptive = None
    if not args.inplace:
        wa = w.replace(force_permille=args.force_permille, force_max_run=args.force_max_run)
        aled = RouteLedger(config_from_workload(wa, two_pass=args.two_pass, gathered=args.gathered,
                                                streaming=args.streaming), device=str(dev))

        def astep():
            for l in range(L):
                (aled.route_anchor if w.is_anchor(l) else aled.route_relay)(dq[l], dk[l], l)

        astep()
        torch.cuda.synchronize()
        forced0 = int(aled.force_state[4].item())
        aev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
               for _ in range(5)]
        for a_ev, b_ev in aev:
            a_ev.record(stream)
            astep()
            b_ev.record(stream)
        torch.cuda.synchronize()
        a_ms = max_over_ranks(statistics.median(a.elapsed_time(b) for a, b in aev), world, dev)
        forced = (int(aled.force_state[4].item()) - forced0) / 5
        n_anchor_l = sum(1 for l in range(L) if w.is_anchor(l))
        relay_call_ms = (a_ms - n_anchor_l * anchor_ms) / max(1, L - n_anchor_l)
        adaptive = {"force_permille": args.force_permille, "force_max_run": args.force_max_run,
                    "ms_per_step": a_ms, "value": aggregate_rows_per_s(w.rows, L, world, a_ms),
                    "forced_relay_calls_per_step": forced, "relay_calls_per_step": L - n_anchor_l,
                    "mean_relay_call_ms": relay_call_ms,
                    "relay_call_speedup_vs_full": full_ms / relay_call_ms}
        aled.close()

    # ---- end to end: host buffers through rr_route_layers_host ------------------------------
    # (pinned host inputs copied in, every layer's routes copied back, copies overlapped with
    # the routing on a second stream -- all inside the library call)
    sq = [torch.empty_like(dq[0]) for _ in range(2)]
    sk = [torch.empty_like(dk[0]) for _ in range(2)]
    sr = [torch.empty((w.rows, w.k), dtype=torch.int32, device=dev) for _ in range(2)]
    host_routes = [torch.empty((w.rows, w.k), dtype=torch.int32).pin_memory() for _ in range(2)]
    copy_stream = torch.cuda.Stream(dev)
    d2h_stream = torch.cuda.Stream(dev)
    anchors = [w.is_anchor(l) for l in range(L)]

    def step_e2e():
        led.route_layers_host([hq[l] for l in range(L)], [hk[l] for l in range(L)], anchors, 0,
                              sq, sk, sr, [host_routes[l & 1] for l in range(L)], copy_stream,
                              d2h_stream)

    step_e2e()
    barrier()
    e2e_evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
               for _ in range(args.steps)]
    for a_ev, b_ev in e2e_evs:
        a_ev.record(stream)
        step_e2e()
        stream.wait_stream(copy_stream)        # the step ends when its last routes are on the host
        stream.wait_stream(d2h_stream)
        b_ev.record(stream)
    barrier()
    ms_e2e = max_over_ranks(statistics.median(a.elapsed_time(b) for a, b in e2e_evs), world, dev)
    h2d = L * w.problems * (w.n_q + w.n_k) * w.d * esz
    d2h = L * w.rows * w.k * 4
    e2e = {"value": aggregate_rows_per_s(w.rows, L, world, ms_e2e), "unit": UNIT,
           "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "ms_per_step": ms_e2e,
           "api": "rr_route_layers_host (copies overlapped on a second stream)"}

    # ---- CPU oracle beside it (rank 0, N = 1 only) -----------------------------------------
    cpu = cpu_timed = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        v, dt, summ, sample = _oracle_sample(w, 12, 9)
        cpu = {"value": v, "unit": UNIT, "cores": _blas_threads(), "os_cpu_count": os.cpu_count(),
               "kind": "oracle", "sample": sample, "oracle_recall": summ.recall_all,
               "oracle_flagged_fraction": summ.flagged_relay_fraction}
        tp = min(w.problems, 4)
        tv, tdt, tsample = _timed_sample(w, tp, w.layers)
        cpu_timed = {"value": tv, "unit": UNIT, "cores": _blas_threads(),
                     "os_cpu_count": os.cpu_count(), "kind": "oracle, vectorised fp32 timed mode "
                     "(BLAS matmul + argpartition, gathered rescoring)", "sample": tsample}

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_per_step, "ms_per_step_mean": mean_ms,
            "ms_per_step_min": min(step_ms), "ms_per_step_max": max(step_ms),
            "timing": "one CUDA-event pair per step; ms_per_step = median over steps, max "
                      "over ranks", "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16" if w.dtype == W.DTYPE_BF16 else "f32", "data": "synthetic",
            "config": {"workload": w.name, "problems": w.problems, "n_q": w.n_q, "n_k": w.n_k,
                       "d": w.d, "k": w.k, "m": w.m, "r": w.r, "layers": L,
                       "anchor_every": w.anchor_every, "rho": w.rho, "causal": w.causal,
                       "l2": ("L2 flushed between steps (256 MB written); a step's inputs are "
                              f"{step_input_bytes / 1e6:.0f} MB" if flush_l2 else
                              "inputs of consecutive layers differ and exceed L2 "
                              f"({w.problems * (w.n_q + w.n_k) * w.d * esz / 1e6:.0f} MB/layer)"),
                       "graph": bool(args.graph),
                       "host_generation_s": round(t_gen, 1)},
            "clocks": clock_info, "e2e": e2e, "gpu_launches": int(launches),
            "roofline": roofline, "cpu_baseline": cpu, "cpu_baseline_vectorised": cpu_timed,
            "layers": {"anchor_ms": anchor_ms, "relay_ms": relay_ms, "full_routing_ms": full_ms,
                       "anchor_rows_per_s": w.rows / anchor_ms * 1e3,
                       "relay_rows_per_s": w.rows / relay_ms * 1e3,
                       "full_routing_rows_per_s": w.rows / full_ms * 1e3,
                       "relay_speedup_vs_full": full_ms / relay_ms},
            "adaptive_forced_anchors": adaptive,
            "quality": {"recall_vs_full_routing": hit / tot, "rerouted_row_fraction": rerouted,
                        "flagged_relay_row_fraction": flagged, "score_pair_fraction": pairs,
                        "status_word": status},
            "kernels": kernels,
        }
        print(json.dumps(line))
    led.close(); full_led.close()
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="high_drift",
                    help="one of %s, or sweep_<n>_<rho> (the routing-scale sweep: 32 heads, n "
                         "chunks, drift rho; e.g. sweep_256_0.15)"
                         % ", ".join(sorted(W.PRESETS) + ["sweep1024"]))
    ap.add_argument("--graph", action="store_true",
                    help="time the device-resident step as replays of one CUDA graph of it "
                         "(for the launch-bound small shapes)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--layers", type=int, default=0, help="truncate the layer schedule")
    ap.add_argument("--profile-only", action="store_true",
                    help="warm-up + timed steps only (for profiler captures)")
    ap.add_argument("--two-pass", action="store_true",
                    help="route through score rows in scratch + warp-level TopK")
    ap.add_argument("--streaming", action="store_true",
                    help="route with the streaming fused kernel instead of the two-sweep kernel")
    ap.add_argument("--inplace", action="store_true",
                    help="relay layers: challenge test inside the routing kernel (one pass over "
                         "the score strip, no compacted second GEMM)")
    ap.add_argument("--force-permille", type=int, default=900,
                    help="forced-anchor policy of the extra 'adaptive_forced_anchors' pass: a tested "
                         "relay that flags this many per mille of the rows forces the next ones")
    ap.add_argument("--force-max-run", type=int, default=8)
    ap.add_argument("--gathered", action="store_true",
                    help="rescore candidates with the gathered FP32 kernel")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
