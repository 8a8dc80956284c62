"""ctypes binding of librouterelay.so -- argument marshalling only.

Every function here has the name of the C entry point it wraps (include/routerelay.h).
Nothing is computed in Python, and there is no fallback: if the shared library is missing
or fails to load, importing the symbols raises.
"""
from __future__ import annotations

import ctypes as C
import os

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "librouterelay.so")

RR_OK = 0
RR_ERR_INVALID_ARG = -1
RR_ERR_UNSUPPORTED = -2
RR_ERR_STATE = -3
RR_ERR_CUDA = -4
RR_ERR_TIMEOUT = -5
RR_ERR_TOO_SMALL = -6
RR_ERR_TOO_LARGE = -7
RR_NOALLOC_MAX_TILES = 65536
RR_BF16 = 0
RR_F32 = 1
RR_STATUS_TIMEOUT = 1
RR_STATUS_BAD_INDEX = 2
RR_NUM_COUNTERS = 8
RR_NUM_KINDS = 12
COUNTER_NAMES = ("layer_calls", "anchor_rows", "relay_rows", "flagged_rows", "cand_pairs",
                 "full_pairs", "dense_pairs")


class rr_config(C.Structure):
    _fields_ = [("batch", C.c_int32), ("heads", C.c_int32), ("n_q", C.c_int32),
                ("n_k", C.c_int32), ("d", C.c_int32), ("k", C.c_int32), ("m", C.c_int32),
                ("r", C.c_int32), ("dtype", C.c_int32), ("causal", C.c_int32),
                ("causal_offset", C.c_int32), ("gamma", C.c_float), ("seed", C.c_uint64),
                ("chunk_tokens", C.c_int32), ("debug_outputs", C.c_int32),
                ("global_sentinels", C.c_int32), ("min_reuse", C.c_int32), ("h_max", C.c_int32),
                ("gamma_boost", C.c_float), ("margin_recover", C.c_float),
                ("coalesce_ranges", C.c_int32), ("force_permille", C.c_int32),
                ("force_max_run", C.c_int32)]


class rr_views(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in (
        "routes", "sentinels", "ages", "kth_score", "margin", "flags", "alpha", "beta",
        "refresh_rows", "refresh_count", "problem_offsets", "token_ranges", "cand_scores",
        "counters", "status", "force_state")]


class rr_bucket_info(C.Structure):
    _fields_ = [("k", C.c_int32), ("problems", C.c_int32), ("first_slot", C.c_int32),
                ("ledger_offset", C.c_size_t), ("scratch_offset", C.c_size_t),
                ("ledger_bytes", C.c_size_t), ("scratch_bytes", C.c_size_t)]


class RouteRelayError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        msg = f"{where}: {strerror(code)} ({code})"
        if code == RR_ERR_CUDA:
            msg += ": " + last_cuda_error()
        super().__init__(msg)


_lib = None


def lib() -> C.CDLL:
    """The loaded shared library; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2609_07306_b200.build` "
                "(there is no CPU fallback)")
        L = C.CDLL(LIB_PATH)
        vp, i32, sz = C.c_void_p, C.c_int32, C.c_size_t
        cfgp = C.POINTER(rr_config)
        L.rr_workspace_bytes.argtypes = [cfgp, C.POINTER(sz), C.POINTER(sz)]
        L.rr_export_bytes.argtypes = [cfgp, C.POINTER(sz)]
        L.rr_ledger_init.argtypes = [cfgp, vp, sz, vp, sz, C.POINTER(vp)]
        L.rr_ledger_reset.argtypes = [vp, vp]
        L.rr_ledger_destroy.argtypes = [vp]
        L.rr_route_anchor.argtypes = [vp, vp, vp, i32, vp]
        L.rr_route_relay.argtypes = [vp, vp, vp, i32, vp]
        L.rr_route_layer_host.argtypes = [vp, vp, vp, vp, vp, i32, i32, vp, vp]
        L.rr_route_layers_host.argtypes = [vp, i32, C.POINTER(vp), C.POINTER(vp), C.POINTER(i32), i32,
                                           C.POINTER(vp), C.POINTER(vp), C.POINTER(vp),
                                           C.POINTER(vp), vp, vp, vp]
        L.rr_ledger_views.argtypes = [vp, C.POINTER(rr_views)]
        L.rr_ledger_export.argtypes = [vp, vp, sz, vp]
        L.rr_ledger_import.argtypes = [vp, vp, sz, vp]
        L.rr_ledger_status.argtypes = [vp, vp, C.POINTER(C.c_uint32)]
        L.rr_sampler_draw_u32.argtypes = [C.c_uint64, C.c_uint32, C.c_uint32, C.c_uint32]
        L.rr_sampler_draw_u32.restype = C.c_uint32
        L.rr_compact_flags_noalloc.argtypes = [vp, i32, i32, vp, vp, vp, vp]
        L.rr_compact_flags_noalloc.restype = C.c_int
        L.rr_bucket_plan.argtypes = [C.POINTER(rr_config), vp, i32, vp, C.POINTER(C.c_int32),
                                     C.POINTER(C.c_size_t), C.POINTER(C.c_size_t)]
        L.rr_bucket_set_init.argtypes = [C.POINTER(rr_config), vp, i32, vp, C.c_size_t, vp, C.c_size_t,
                                         C.POINTER(vp)]
        L.rr_bucket_set_destroy.argtypes = [vp]
        L.rr_bucket_set_count.argtypes = [vp]
        L.rr_bucket_set_info.argtypes = [vp, i32, C.POINTER(rr_bucket_info)]
        L.rr_bucket_set_ledger.argtypes = [vp, i32]
        L.rr_bucket_set_ledger.restype = vp
        L.rr_bucket_set_reset.argtypes = [vp, vp]
        L.rr_bucket_route_layer.argtypes = [vp, vp, vp, i32, i32, vp]
        L.rr_bucket_set_status.argtypes = [vp, vp, C.POINTER(C.c_uint32)]
        L.rr_attend_token_ranges.argtypes = [vp, i32, i32, i32, vp, vp, vp, i32, i32, i32, C.c_float,
                                             vp, vp]
        for name in ("rr_bucket_plan", "rr_bucket_set_init", "rr_bucket_set_destroy",
                     "rr_bucket_set_count", "rr_bucket_set_info", "rr_bucket_set_reset",
                     "rr_bucket_route_layer", "rr_bucket_set_status", "rr_attend_token_ranges"):
            getattr(L, name).restype = C.c_int
        L.rr_profile_begin.argtypes = [vp]
        L.rr_profile_begin.restype = C.c_int
        L.rr_profile_end.argtypes = [vp, vp, C.POINTER(C.c_float), C.POINTER(C.c_int64)]
        L.rr_profile_end.restype = C.c_int
        L.rr_kind_name.argtypes = [C.c_int]
        L.rr_kind_name.restype = C.c_char_p
        L.rr_kernel_launch_count.argtypes = []
        L.rr_kernel_launch_count.restype = C.c_uint64
        L.rr_strerror.argtypes = [C.c_int]
        L.rr_strerror.restype = C.c_char_p
        L.rr_last_cuda_error.argtypes = []
        L.rr_last_cuda_error.restype = C.c_char_p
        for name in ("rr_workspace_bytes", "rr_export_bytes", "rr_ledger_init", "rr_ledger_reset",
                     "rr_ledger_destroy", "rr_route_anchor", "rr_route_relay",
                     "rr_route_layer_host", "rr_route_layers_host", "rr_ledger_views", "rr_ledger_export",
                     "rr_ledger_import", "rr_ledger_status"):
            getattr(L, name).restype = C.c_int
        _lib = L
    return _lib


def _check(code: int, where: str) -> None:
    if code != RR_OK:
        raise RouteRelayError(code, where)


def strerror(code: int) -> str:
    return lib().rr_strerror(code).decode()


def last_cuda_error() -> str:
    return lib().rr_last_cuda_error().decode()


def rr_workspace_bytes(cfg: rr_config):
    a, b = C.c_size_t(), C.c_size_t()
    _check(lib().rr_workspace_bytes(C.byref(cfg), C.byref(a), C.byref(b)), "rr_workspace_bytes")
    return a.value, b.value


def rr_export_bytes(cfg: rr_config) -> int:
    a = C.c_size_t()
    _check(lib().rr_export_bytes(C.byref(cfg), C.byref(a)), "rr_export_bytes")
    return a.value


def rr_ledger_init(cfg: rr_config, dev_ledger: int, ledger_bytes: int, dev_scratch: int,
                   scratch_bytes: int) -> int:
    h = C.c_void_p()
    _check(lib().rr_ledger_init(C.byref(cfg), dev_ledger, ledger_bytes, dev_scratch,
                                scratch_bytes, C.byref(h)), "rr_ledger_init")
    return h.value


def rr_ledger_reset(h: int, stream: int) -> None:
    _check(lib().rr_ledger_reset(h, stream), "rr_ledger_reset")


def rr_ledger_destroy(h: int) -> None:
    _check(lib().rr_ledger_destroy(h), "rr_ledger_destroy")


def rr_route_anchor(h: int, qc: int, kc: int, layer: int, stream: int) -> None:
    _check(lib().rr_route_anchor(h, qc, kc, layer, stream), "rr_route_anchor")


def rr_route_relay(h: int, qc: int, kc: int, layer: int, stream: int) -> None:
    _check(lib().rr_route_relay(h, qc, kc, layer, stream), "rr_route_relay")


def rr_route_layer_host(h: int, host_qc: int, host_kc: int, dev_qc: int, dev_kc: int,
                        layer: int, is_anchor: bool, host_routes: int, stream: int) -> None:
    _check(lib().rr_route_layer_host(h, host_qc, host_kc, dev_qc, dev_kc, layer,
                                     1 if is_anchor else 0, host_routes, stream),
           "rr_route_layer_host")


def rr_route_layers_host(h: int, host_qc, host_kc, is_anchor, first_layer: int, dev_qc, dev_kc,
                         dev_routes, host_routes, stream: int, copy_stream: int,
                         d2h_stream: int = 0) -> None:
    """host_qc/host_kc/host_routes: sequences of host addresses (one per layer; host_routes may be
    None); dev_qc/dev_kc/dev_routes: two device addresses each (dev_routes may be None)."""
    n = len(host_qc)
    arr = lambda xs: (C.c_void_p * len(xs))(*xs)
    _check(lib().rr_route_layers_host(
        h, n, arr(host_qc), arr(host_kc), (C.c_int32 * n)(*[1 if a else 0 for a in is_anchor]),
        first_layer, arr(dev_qc), arr(dev_kc), arr(dev_routes) if dev_routes else None,
        arr(host_routes) if host_routes else None, stream, copy_stream, d2h_stream or None),
           "rr_route_layers_host")


def rr_ledger_views(h: int) -> rr_views:
    v = rr_views()
    _check(lib().rr_ledger_views(h, C.byref(v)), "rr_ledger_views")
    return v


def rr_ledger_export(h: int, host_blob: int, nbytes: int, stream: int) -> None:
    _check(lib().rr_ledger_export(h, host_blob, nbytes, stream), "rr_ledger_export")


def rr_ledger_import(h: int, host_blob: int, nbytes: int, stream: int) -> None:
    _check(lib().rr_ledger_import(h, host_blob, nbytes, stream), "rr_ledger_import")


def rr_ledger_status(h: int, stream: int) -> int:
    s = C.c_uint32()
    _check(lib().rr_ledger_status(h, stream, C.byref(s)), "rr_ledger_status")
    return s.value


def rr_sampler_draw_u32(seed: int, g: int, layer: int, t: int) -> int:
    return int(lib().rr_sampler_draw_u32(seed, g, layer, t))


def rr_compact_flags_noalloc(dev_flags: int, n_problems: int, n_q: int, dev_rows_out: int,
                             dev_count_out: int, dev_problem_offsets_out: int,
                             stream: int) -> None:
    """Compaction without any allocation: the scratch is a fixed array inside the library
    (for callers that may not call cudaMalloc).  Arguments are raw device addresses."""
    _check(lib().rr_compact_flags_noalloc(dev_flags, n_problems, n_q, dev_rows_out,
                                          dev_count_out, dev_problem_offsets_out, stream),
           "rr_compact_flags_noalloc")


def rr_bucket_plan(cfg: rr_config, widths):
    """(order, n_buckets, ledger_bytes, scratch_bytes) for the per-problem route widths."""
    w = (C.c_int32 * len(widths))(*[int(x) for x in widths])
    order = (C.c_int32 * len(widths))()
    nb, a, b = C.c_int32(), C.c_size_t(), C.c_size_t()
    _check(lib().rr_bucket_plan(C.byref(cfg), w, len(widths), order, C.byref(nb), C.byref(a),
                                C.byref(b)), "rr_bucket_plan")
    return list(order), nb.value, a.value, b.value


def rr_bucket_set_init(cfg: rr_config, widths, dev_ledger: int, ledger_bytes: int,
                       dev_scratch: int, scratch_bytes: int) -> int:
    w = (C.c_int32 * len(widths))(*[int(x) for x in widths])
    h = C.c_void_p()
    _check(lib().rr_bucket_set_init(C.byref(cfg), w, len(widths), dev_ledger, ledger_bytes,
                                    dev_scratch, scratch_bytes, C.byref(h)), "rr_bucket_set_init")
    return h.value


def rr_bucket_set_destroy(h: int) -> None:
    _check(lib().rr_bucket_set_destroy(h), "rr_bucket_set_destroy")


def rr_bucket_set_count(h: int) -> int:
    n = lib().rr_bucket_set_count(h)
    if n < 0:
        _check(n, "rr_bucket_set_count")
    return n


def rr_bucket_set_info(h: int, b: int) -> rr_bucket_info:
    info = rr_bucket_info()
    _check(lib().rr_bucket_set_info(h, b, C.byref(info)), "rr_bucket_set_info")
    return info


def rr_bucket_set_ledger(h: int, b: int) -> int:
    return lib().rr_bucket_set_ledger(h, b)


def rr_bucket_set_reset(h: int, stream: int) -> None:
    _check(lib().rr_bucket_set_reset(h, stream), "rr_bucket_set_reset")


def rr_bucket_route_layer(h: int, qc: int, kc: int, layer: int, is_anchor: bool, stream: int) -> None:
    _check(lib().rr_bucket_route_layer(h, qc, kc, layer, 1 if is_anchor else 0, stream),
           "rr_bucket_route_layer")


def rr_bucket_set_status(h: int, stream: int) -> int:
    st = C.c_uint32()
    _check(lib().rr_bucket_set_status(h, stream, C.byref(st)), "rr_bucket_set_status")
    return st.value


def rr_attend_token_ranges(ranges: int, rows: int, slots: int, n_q: int, q: int, keys: int,
                           values: int, tokens: int, dh: int, dtype: int, scale: float, out: int,
                           stream: int) -> None:
    _check(lib().rr_attend_token_ranges(ranges, rows, slots, n_q, q, keys, values, tokens, dh,
                                        dtype, scale, out, stream), "rr_attend_token_ranges")


def rr_profile_begin(h: int) -> None:
    _check(lib().rr_profile_begin(h), "rr_profile_begin")


def rr_profile_end(h: int, stream: int):
    """{kind name: (total ms, launches)} for the kinds that ran."""
    ms = (C.c_float * RR_NUM_KINDS)()
    n = (C.c_int64 * RR_NUM_KINDS)()
    _check(lib().rr_profile_end(h, stream, ms, n), "rr_profile_end")
    out = {}
    for i in range(RR_NUM_KINDS):
        if n[i]:
            out[lib().rr_kind_name(i).decode()] = (float(ms[i]), int(n[i]))
    return out


def rr_kernel_launch_count() -> int:
    return int(lib().rr_kernel_launch_count())
