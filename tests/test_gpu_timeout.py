"""A bounded device-side wait that runs out: the kernel must give up cleanly (abort flag, every
role leaves its loop, TMEM freed only after the issued MMAs have finished), the status word must
carry RR_STATUS_TIMEOUT, rr_ledger_status must return RR_ERR_TIMEOUT, and after a reset the
same ledger must route correctly again.  Nothing hangs and nothing faults: a test hook makes
the first wait of one CTA count as expired."""
import numpy as np
import pytest
import torch

from paper_2609_07306_b200 import binding as B
from paper_2609_07306_b200 import workload as W
from paper_2609_07306_b200.ledger import RouteLedger, config_from_workload, device_tensor

pytestmark = pytest.mark.gpu


def _expect_timeout(led):
    with pytest.raises(B.RouteRelayError) as ei:
        led.status()
    assert ei.value.code == B.RR_ERR_TIMEOUT
    status = led._view("status", "i32", (1,)).item()
    assert status & B.RR_STATUS_TIMEOUT


@pytest.mark.parametrize("which", ["routing", "rescoring"])
def test_forced_timeout_is_reported_and_recoverable(which):
    w = W.moderate().replace(heads=2)
    q, k = W.generate(w, layers=2)
    led = RouteLedger(config_from_workload(w, forced_timeouts=1 if which == "routing" else 2,
                                          two_sweep=True))
    ref = RouteLedger(config_from_workload(w, two_sweep=True))
    dq, dk = [device_tensor(x) for x in q], [device_tensor(x) for x in k]
    led.route_anchor(dq[0], dk[0], 0)
    ref.route_anchor(dq[0], dk[0], 0)
    torch.cuda.synchronize()
    if which == "routing":
        _expect_timeout(led)            # the anchor's routing kernel gave up in one CTA
        # ... which left that CTA's 128 rows as the reset had them; all other rows are routed
        untouched = (led.routes.cpu().numpy() == -1).all(axis=1)
        assert untouched.sum() == 128
        assert torch.equal(led.routes[~torch.from_numpy(untouched).cuda()],
                           ref.routes[~torch.from_numpy(untouched).cuda()])
    else:
        assert led.status() == 0
        assert torch.equal(led.routes, ref.routes)
        led.route_relay(dq[1], dk[1], 1)
        torch.cuda.synchronize()
        _expect_timeout(led)            # the relay's strip rescoring kernel gave up in one CTA
    # the hook fires once per ledger: after a reset the same ledger is as good as new
    led.reset()
    led.route_anchor(dq[0], dk[0], 0)
    led.route_relay(dq[1], dk[1], 1)
    ref.reset()
    ref.route_anchor(dq[0], dk[0], 0)
    ref.route_relay(dq[1], dk[1], 1)
    torch.cuda.synchronize()
    assert led.status() == 0
    assert torch.equal(led.routes, ref.routes) and torch.equal(led.sentinels, ref.sentinels)
    assert torch.equal(led.flags, ref.flags) and torch.equal(led.ages, ref.ages)
    led.close(); ref.close()
