"""rr_compact_flags_noalloc against the compaction done inside rr_route_relay.

The entry point exists for embedders that may not allocate device memory (frozen memory
pools, plugins that only receive input/output buffers): its scratch is a fixed array in the
library image instead of a caller-provided buffer.  The test calls it through the C ABI on
the flags of two consecutive relay layers and requires the list, the count and the
per-problem offsets to equal, bit for bit, what the relay call itself produced -- the same
bar the other compaction checks use.  Collected last on purpose (file name)."""
import numpy as np
import pytest
import torch

from paper_2609_07306_b200 import binding as B
from paper_2609_07306_b200 import workload as W
from paper_2609_07306_b200.ledger import RouteLedger, config_from_workload, device_tensor

pytestmark = pytest.mark.gpu


def test_noalloc_compaction_matches_relay_twice_in_a_row():
    w = W.sweep(512, 0.15).replace(heads=3, layers=3, anchor_every=8)
    q, k = W.generate(w)
    led = RouteLedger(config_from_workload(w))
    rows_out = torch.full((w.rows,), -7, dtype=torch.int32, device="cuda")
    count_out = torch.full((1,), -7, dtype=torch.int32, device="cuda")
    offs_out = torch.full((w.problems + 1,), -7, dtype=torch.int32, device="cuda")
    stream = torch.cuda.current_stream().cuda_stream
    led.route_anchor(device_tensor(q[0]), device_tensor(k[0]), 0)
    seen = []
    for l in (1, 2):                         # two calls in a row, different flag patterns
        led.route_relay(device_tensor(q[l]), device_tensor(k[l]), l)
        rows_out.fill_(-7)
        B.rr_compact_flags_noalloc(led.flags.data_ptr(), w.problems, w.n_q, rows_out.data_ptr(),
                                   count_out.data_ptr(), offs_out.data_ptr(), stream)
        torch.cuda.synchronize()
        n = int(led.refresh_count.item())
        assert 0 < n < w.rows
        assert int(count_out.item()) == n
        assert torch.equal(rows_out[:n], led.refresh_rows[:n])
        assert (rows_out[n:] == -7).all()                 # nothing written past the count
        assert torch.equal(offs_out, led.problem_offsets)
        assert np.array_equal(rows_out[:n].cpu().numpy(), np.nonzero(led.flags.cpu().numpy())[0])
        seen.append(n)
    assert seen[0] != seen[1]
    led.close()


def test_noalloc_ragged_tiles_against_nonzero():
    """Problems whose row count is not a multiple of the 128-row tile (200 rows, 3 problems: a
    full tile and a ragged one per problem), twice in a row with different flag patterns:
    list, count and per-problem offsets against numpy.nonzero of the flags."""
    n_problems, n_q = 3, 200
    rng = np.random.default_rng(5)
    rows_out = torch.empty(n_problems * n_q, dtype=torch.int32, device="cuda")
    count_out = torch.empty(1, dtype=torch.int32, device="cuda")
    offs_out = torch.empty(n_problems + 1, dtype=torch.int32, device="cuda")
    stream = torch.cuda.current_stream().cuda_stream
    for density in (0.3, 0.9):
        flags = (rng.random(n_problems * n_q) < density).astype(np.uint8) * 3   # any non-zero counts
        dflags = torch.from_numpy(flags).cuda()
        rows_out.fill_(-7)
        B.rr_compact_flags_noalloc(dflags.data_ptr(), n_problems, n_q, rows_out.data_ptr(),
                                   count_out.data_ptr(), offs_out.data_ptr(), stream)
        torch.cuda.synchronize()
        nz = np.nonzero(flags)[0]
        assert int(count_out.item()) == len(nz)
        assert np.array_equal(rows_out[:len(nz)].cpu().numpy(), nz)
        assert (rows_out[len(nz):] == -7).all()
        per_problem = (flags != 0).reshape(n_problems, n_q).sum(axis=1)
        assert np.array_equal(offs_out.cpu().numpy(), np.concatenate([[0], np.cumsum(per_problem)]))


def test_noalloc_rejects_oversize_and_bad_arguments():
    flags = torch.zeros(256, dtype=torch.uint8, device="cuda")
    out = torch.zeros(256, dtype=torch.int32, device="cuda")
    lib = B.lib()
    args = (out.data_ptr(), out.data_ptr(), out.data_ptr(), None)
    too_many = B.RR_NOALLOC_MAX_TILES + 1
    assert lib.rr_compact_flags_noalloc(flags.data_ptr(), too_many, 128, *args) == B.RR_ERR_TOO_LARGE
    assert lib.rr_compact_flags_noalloc(None, 1, 128, *args) == B.RR_ERR_INVALID_ARG
    assert lib.rr_compact_flags_noalloc(flags.data_ptr(), 0, 128, *args) == B.RR_ERR_INVALID_ARG
    assert "capacity" in B.strerror(B.RR_ERR_TOO_LARGE)
