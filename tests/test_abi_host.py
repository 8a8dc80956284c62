"""Host-side checks of the C ABI: the library builds, loads and exports every symbol the
header declares; argument validation; buffer sizing; the sampler's generator.  No GPU."""
import ctypes as C
import os
import re

import numpy as np
import pytest

import __graft_entry__ as entry
from paper_2609_07306_b200 import binding as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def built():
    entry.build()


def _cfg(**kw):
    base = dict(batch=1, heads=2, n_q=256, n_k=256, d=128, k=16, m=8, r=8, dtype=B.RR_BF16,
                causal=1, causal_offset=0, gamma=0.0, seed=1, chunk_tokens=0, debug_outputs=0)
    base.update(kw)
    return B.rr_config(**base)


def test_every_declared_symbol_is_exported():
    hdr = open(os.path.join(ROOT, "include", "routerelay.h")).read()
    names = set(re.findall(r"\b(rr_[a-z0-9_]+)\s*\(", hdr))
    assert {"rr_route_anchor", "rr_route_relay", "rr_ledger_init", "rr_ledger_reset"} <= names
    lib = B.lib()
    for n in names:
        assert hasattr(lib, n), f"{n} declared in routerelay.h but not exported"


def test_config_struct_matches_header_order():
    hdr = open(os.path.join(ROOT, "include", "routerelay.h")).read()
    body = hdr[hdr.index("typedef struct rr_config {"):hdr.index("} rr_config;")]
    body = re.sub(r"/\*.*?\*/", "", body, flags=re.S)
    fields = []
    for decl in body.split("{", 1)[1].split(";"):
        toks = decl.replace(",", " ").split()
        fields += toks[1:]
    assert fields == [f[0] for f in B.rr_config._fields_]
    vbody = hdr[hdr.index("typedef struct rr_views {"):hdr.index("} rr_views;")]
    vbody = re.sub(r"/\*.*?\*/", "", vbody, flags=re.S)
    vfields = re.findall(r"\*\s*([a-z_]+)\s*;", vbody)
    assert vfields == [f[0] for f in B.rr_views._fields_]


def test_workspace_sizes():
    cfg = _cfg()
    lb, sb = B.rr_workspace_bytes(cfg)
    rows = 2 * 256
    assert lb >= rows * (16 + 16 + 3) * 4
    assert sb < rows * 256 * 4                       # fused path: no score rows in scratch
    _, sb2 = B.rr_workspace_bytes(_cfg(debug_outputs=2))
    assert sb2 >= rows * 256 * 4                     # two-pass path: score rows
    assert B.rr_export_bytes(cfg) == rows * (16 + 16 + 3) * 4
    # paper, Section 4.4: int32 index ledger, n_q = 1024, c = 64 -> 256 KB
    cfg = _cfg(heads=1, n_q=1024, n_k=1024, k=32, m=16, r=16)
    assert B.rr_export_bytes(cfg) - 1024 * 3 * 4 == 256 * 1024


@pytest.mark.parametrize("kw,code", [
    (dict(d=96), B.RR_ERR_UNSUPPORTED),
    (dict(dtype=7), B.RR_ERR_UNSUPPORTED),
    (dict(n_k=8192, n_q=8192), B.RR_ERR_UNSUPPORTED),
    (dict(k=0), B.RR_ERR_INVALID_ARG),
    (dict(k=300), B.RR_ERR_INVALID_ARG),
    (dict(m=-1), B.RR_ERR_INVALID_ARG),
    (dict(gamma=-1.0), B.RR_ERR_INVALID_ARG),
    (dict(gamma=float("nan")), B.RR_ERR_INVALID_ARG),
    (dict(causal=2), B.RR_ERR_INVALID_ARG),
    (dict(causal_offset=-1), B.RR_ERR_INVALID_ARG),
    (dict(k=128, m=100, r=100), B.RR_ERR_UNSUPPORTED),
])
def test_invalid_configs_are_rejected(kw, code):
    with pytest.raises(B.RouteRelayError) as ei:
        B.rr_workspace_bytes(_cfg(**kw))
    assert ei.value.code == code


def test_init_validates_buffers_without_a_gpu():
    cfg = _cfg()
    lb, sb = B.rr_workspace_bytes(cfg)
    lib = B.lib()
    h = C.c_void_p()
    assert lib.rr_ledger_init(C.byref(cfg), None, lb, 0x1000, sb, C.byref(h)) == B.RR_ERR_INVALID_ARG
    assert lib.rr_ledger_init(C.byref(cfg), 0x1010, lb, 0x100000, sb, C.byref(h)) == B.RR_ERR_INVALID_ARG
    assert lib.rr_ledger_init(C.byref(cfg), 0x1000, lb - 1, 0x100000, sb, C.byref(h)) == B.RR_ERR_TOO_SMALL
    # fake (never dereferenced) device addresses: handle creation is host-only
    assert lib.rr_ledger_init(C.byref(cfg), 0x10000, lb, 0x7000000, sb, C.byref(h)) == B.RR_OK
    # relay before any anchor is a state error, reported before anything is enqueued
    assert lib.rr_route_relay(h, 0x100, 0x200, 1, None) == B.RR_ERR_STATE
    assert lib.rr_route_anchor(h, None, 0x200, 0, None) == B.RR_ERR_INVALID_ARG
    assert lib.rr_route_anchor(h, 0x104, 0x200, 0, None) == B.RR_ERR_INVALID_ARG   # misaligned
    assert lib.rr_ledger_destroy(h) == B.RR_OK
    assert lib.rr_ledger_destroy(None) == B.RR_ERR_INVALID_ARG
    assert "relay before anchor" in B.strerror(B.RR_ERR_STATE)


def test_sampler_generator_matches_known_answers(golden_dir):
    """The library's host-callable copy of the kernels' generator against vectors written
    by the oracle (tests/golden/make_sampler_vectors.py)."""
    n = 0
    for line in open(os.path.join(golden_dir, "sampler_vectors.txt")):
        if line.startswith("U "):
            _, seed, g, layer, t, u = line.split()
            assert B.rr_sampler_draw_u32(int(seed), int(g), int(layer), int(t)) == int(u)
            n += 1
    assert n >= 100
