"""RouteLedger: device buffers (torch) + the C handle.  PyTorch is used for device memory
and streams only; every step of the routing path runs in the library's kernels."""
from __future__ import annotations

import numpy as np
import torch

from . import binding as B
from .workload import DTYPE_BF16, RouteWorkload

_TORCH_DT = {"i32": torch.int32, "f32": torch.float32, "u8": torch.uint8, "i64": torch.int64}


def config_from_workload(w: RouteWorkload, debug_outputs: bool = False,
                         two_pass: bool = False, gathered: bool = False,
                         force_slow_rows: bool = False, streaming: bool = False,
                         inplace: bool = False, forced_timeouts: int = 0,
                         two_sweep: bool = False) -> B.rr_config:
    return B.rr_config(batch=w.batch, heads=w.heads, n_q=w.n_q, n_k=w.n_k, d=w.d, k=w.k, m=w.m,
                       r=w.r, dtype=B.RR_BF16 if w.dtype == DTYPE_BF16 else B.RR_F32,
                       causal=1 if w.causal else 0, causal_offset=int(w.causal_offset),
                       gamma=float(w.gamma),
                       seed=int(w.seed), chunk_tokens=int(w.chunk_tokens),
                       debug_outputs=(1 if debug_outputs else 0) | (2 if two_pass else 0) |
                       (4 if gathered else 0) | (8 if force_slow_rows else 0) |
                       (16 if streaming else 0) | (32 if inplace else 0) |
                       ((forced_timeouts & 3) << 6) | (256 if two_sweep else 0),
                       global_sentinels=int(w.global_sentinels), min_reuse=int(w.min_reuse),
                       h_max=int(w.h_max), gamma_boost=float(w.gamma_boost),
                       margin_recover=float(w.margin_recover),
                       coalesce_ranges=1 if w.coalesce_ranges else 0,
                       force_permille=int(w.force_permille), force_max_run=int(w.force_max_run))


class RouteLedger:
    """Owns the two device buffers of one ledger and exposes the C calls as methods."""

    def __init__(self, cfg: B.rr_config, device: str = "cuda:0"):
        if not torch.cuda.is_available():
            raise RuntimeError("RouteLedger needs a CUDA device (there is no CPU path)")
        self.cfg = cfg
        self.device = torch.device(device)
        lb, sb = B.rr_workspace_bytes(cfg)
        with torch.cuda.device(self.device):
            self.ledger_buf = torch.empty(lb + 256, dtype=torch.uint8, device=self.device)
            self.scratch_buf = torch.empty(sb + 256, dtype=torch.uint8, device=self.device)
            self._lo = (-self.ledger_buf.data_ptr()) % 256
            self._so = (-self.scratch_buf.data_ptr()) % 256
            self.handle = B.rr_ledger_init(cfg, self.ledger_buf.data_ptr() + self._lo, lb,
                                           self.scratch_buf.data_ptr() + self._so, sb)
        self.P = cfg.batch * cfg.heads
        self.rows = self.P * cfg.n_q
        self.sw = cfg.m + cfg.r + (cfg.global_sentinels & 1) + ((cfg.global_sentinels >> 1) & 1)
        self.c = cfg.k + self.sw
        self._views = B.rr_ledger_views(self.handle)
        self.reset()

    # -- lifetime ------------------------------------------------------------------------
    def close(self):
        if getattr(self, "handle", None):
            torch.cuda.synchronize(self.device)
            B.rr_ledger_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _stream(self) -> int:
        return torch.cuda.current_stream(self.device).cuda_stream

    # -- calls -----------------------------------------------------------------------------
    def reset(self):
        B.rr_ledger_reset(self.handle, self._stream())

    def route_anchor(self, qc: torch.Tensor, kc: torch.Tensor, layer: int):
        B.rr_route_anchor(self.handle, qc.data_ptr(), kc.data_ptr(), layer, self._stream())

    def route_relay(self, qc: torch.Tensor, kc: torch.Tensor, layer: int):
        B.rr_route_relay(self.handle, qc.data_ptr(), kc.data_ptr(), layer, self._stream())

    def route_layer_host(self, host_qc: torch.Tensor, host_kc: torch.Tensor,
                         dev_qc: torch.Tensor, dev_kc: torch.Tensor, layer: int,
                         is_anchor: bool, host_routes: torch.Tensor | None):
        B.rr_route_layer_host(self.handle, host_qc.data_ptr(), host_kc.data_ptr(),
                              dev_qc.data_ptr(), dev_kc.data_ptr(), layer, is_anchor,
                              host_routes.data_ptr() if host_routes is not None else None,
                              self._stream())

    def route_layers_host(self, host_qc, host_kc, is_anchor, first_layer, dev_qc, dev_kc,
                          dev_routes, host_routes, copy_stream: "torch.cuda.Stream",
                          d2h_stream: "torch.cuda.Stream | None" = None):
        """Lists of tensors (host: one per layer; device: two staging buffers each)."""
        B.rr_route_layers_host(
            self.handle, [t.data_ptr() for t in host_qc], [t.data_ptr() for t in host_kc],
            list(is_anchor), first_layer, [t.data_ptr() for t in dev_qc],
            [t.data_ptr() for t in dev_kc],
            [t.data_ptr() for t in dev_routes] if dev_routes is not None else None,
            [t.data_ptr() for t in host_routes] if host_routes is not None else None,
            self._stream(), copy_stream.cuda_stream,
            d2h_stream.cuda_stream if d2h_stream is not None else 0)

    def status(self) -> int:
        return B.rr_ledger_status(self.handle, self._stream())

    # -- views (zero-copy torch tensors over the library's device pointers) ---------------
    def _view(self, name: str, kind: str, shape):
        ptr = getattr(self._views, name)
        if not ptr:
            return None
        n = int(np.prod(shape))
        dt = _TORCH_DT[kind]
        nbytes = n * torch.empty((), dtype=dt).element_size()
        for buf in (self.ledger_buf, self.scratch_buf):
            off = ptr - buf.data_ptr()
            if 0 <= off and off + nbytes <= buf.numel():
                return buf[off:off + nbytes].view(dt).view(*shape)
        raise RuntimeError(f"view {name} lies outside the ledger buffers")

    @property
    def routes(self): return self._view("routes", "i32", (self.rows, self.cfg.k))
    @property
    def sentinels(self): return self._view("sentinels", "i32", (self.rows, self.sw))
    @property
    def ages(self): return self._view("ages", "i32", (self.rows,))
    @property
    def kth_score(self): return self._view("kth_score", "f32", (self.rows,))
    @property
    def margin(self): return self._view("margin", "f32", (self.rows,))
    @property
    def flags(self): return self._view("flags", "u8", (self.rows,))
    @property
    def alpha(self): return self._view("alpha", "f32", (self.rows,))
    @property
    def beta(self): return self._view("beta", "f32", (self.rows,))
    @property
    def refresh_rows(self): return self._view("refresh_rows", "i32", (self.rows,))
    @property
    def refresh_count(self): return self._view("refresh_count", "i32", (1,))
    @property
    def problem_offsets(self): return self._view("problem_offsets", "i32", (self.P + 1,))
    @property
    def token_ranges(self): return self._view("token_ranges", "i32", (self.rows, self.cfg.k, 2))
    @property
    def cand_scores(self): return self._view("cand_scores", "f32", (self.rows, self.c))
    @property
    def force_state(self): return self._view("force_state", "i32", (8,))

    @property
    def counters(self): return self._view("counters", "i64", (B.RR_NUM_COUNTERS,))

    def counters_dict(self):
        vals = self.counters.cpu().tolist()
        return dict(zip(B.COUNTER_NAMES, vals))

    # -- checkpoint ---------------------------------------------------------------------------
    def export_blob(self) -> np.ndarray:
        n = B.rr_export_bytes(self.cfg)
        blob = np.empty(n, np.uint8)
        B.rr_ledger_export(self.handle, blob.ctypes.data, n, self._stream())
        return blob

    def import_blob(self, blob: np.ndarray):
        blob = np.ascontiguousarray(blob, np.uint8)
        B.rr_ledger_import(self.handle, blob.ctypes.data, blob.size, self._stream())

    def pack_blob(self, routes, sentinels, ages, kth, margin) -> np.ndarray:
        """Host arrays -> checkpoint blob layout (routes, sentinels, ages, kth, margin)."""
        parts = [np.ascontiguousarray(routes, np.int32), np.ascontiguousarray(sentinels, np.int32),
                 np.ascontiguousarray(ages, np.int32), np.ascontiguousarray(kth, np.float32),
                 np.ascontiguousarray(margin, np.float32)]
        return np.concatenate([p.reshape(-1).view(np.uint8) for p in parts])


def device_tensor(x: np.ndarray, device="cuda:0") -> torch.Tensor:
    """Generated inputs (bf16 bit patterns as uint16, or float32) -> device tensor."""
    if x.dtype == np.uint16:
        return torch.from_numpy(x.view(np.int16)).to(device).view(torch.bfloat16)
    return torch.from_numpy(np.ascontiguousarray(x, np.float32)).to(device)


class _BucketLedger(RouteLedger):
    """A bucket's ledger inside a BucketSet: same views and status calls as RouteLedger, but the
    handle and the device buffers belong to the set."""

    def __init__(self, handle: int, cfg: B.rr_config, ledger_buf, scratch_buf, device):
        self.cfg, self.handle, self.device = cfg, handle, device
        self.ledger_buf, self.scratch_buf = ledger_buf, scratch_buf
        self.P = cfg.batch * cfg.heads
        self.rows = self.P * cfg.n_q
        self.sw = cfg.m + cfg.r + (cfg.global_sentinels & 1) + ((cfg.global_sentinels >> 1) & 1)
        self.c = cfg.k + self.sw
        self._views = B.rr_ledger_views(handle)

    def close(self):
        self.handle = None


class BucketSet:
    """Route-width buckets (Section 4.4): problems grouped by requested route width, one ledger
    per bucket, one call per layer.  Inputs are bucket-major: use `order` to lay them out."""

    def __init__(self, cfg: B.rr_config, widths, device: str = "cuda:0"):
        if not torch.cuda.is_available():
            raise RuntimeError("BucketSet needs a CUDA device (there is no CPU path)")
        self.cfg, self.device = cfg, torch.device(device)
        self.order, n_buckets, lb, sb = B.rr_bucket_plan(cfg, widths)
        with torch.cuda.device(self.device):
            self.ledger_buf = torch.empty(lb + 256, dtype=torch.uint8, device=self.device)
            self.scratch_buf = torch.empty(sb + 256, dtype=torch.uint8, device=self.device)
            lo = (-self.ledger_buf.data_ptr()) % 256
            so = (-self.scratch_buf.data_ptr()) % 256
            self.handle = B.rr_bucket_set_init(cfg, widths, self.ledger_buf.data_ptr() + lo, lb,
                                               self.scratch_buf.data_ptr() + so, sb)
        assert B.rr_bucket_set_count(self.handle) == n_buckets
        self.info = [B.rr_bucket_set_info(self.handle, b) for b in range(n_buckets)]
        self.buckets = []
        for b, inf in enumerate(self.info):
            bc = B.rr_config()
            C_fields = [f[0] for f in B.rr_config._fields_]
            for f in C_fields:
                setattr(bc, f, getattr(cfg, f))
            bc.batch, bc.heads, bc.k = 1, inf.problems, inf.k
            self.buckets.append(_BucketLedger(B.rr_bucket_set_ledger(self.handle, b), bc,
                                              self.ledger_buf, self.scratch_buf, self.device))
        self.reset()

    def _stream(self) -> int:
        return torch.cuda.current_stream(self.device).cuda_stream

    def reset(self):
        B.rr_bucket_set_reset(self.handle, self._stream())

    def route_layer(self, qc: torch.Tensor, kc: torch.Tensor, layer: int, is_anchor: bool):
        B.rr_bucket_route_layer(self.handle, qc.data_ptr(), kc.data_ptr(), layer, is_anchor,
                                self._stream())

    def status(self) -> int:
        return B.rr_bucket_set_status(self.handle, self._stream())

    def close(self):
        if getattr(self, "handle", None):
            torch.cuda.synchronize(self.device)
            B.rr_bucket_set_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def attend_token_ranges(ranges: torch.Tensor, n_q: int, q: torch.Tensor, keys: torch.Tensor,
                        values: torch.Tensor, scale: float) -> torch.Tensor:
    """Eq. 3 over the tokens the ranges cover (the library's reference consumer).
    ranges [rows, slots, 2] int32; q [rows, dh]; keys / values [P, tokens, dh] (bf16 or fp32)."""
    rows, slots = ranges.shape[0], ranges.shape[1]
    dtype = {torch.bfloat16: B.RR_BF16, torch.float32: B.RR_F32}[q.dtype]
    assert keys.dtype == q.dtype and values.dtype == q.dtype
    assert ranges.is_contiguous() and q.is_contiguous() and keys.is_contiguous() and values.is_contiguous()
    out = torch.empty((rows, q.shape[1]), dtype=torch.float32, device=q.device)
    B.rr_attend_token_ranges(ranges.data_ptr(), rows, slots, n_q, q.data_ptr(), keys.data_ptr(),
                             values.data_ptr(), keys.shape[1], q.shape[1], dtype, float(scale),
                             out.data_ptr(), torch.cuda.current_stream(q.device).cuda_stream)
    return out
