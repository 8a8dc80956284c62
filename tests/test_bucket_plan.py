"""Host logic of the route-width bucket front end (no GPU): grouping, order, sizes, errors."""
import pytest

from paper_2609_07306_b200 import binding as B
from paper_2609_07306_b200 import workload as W
from paper_2609_07306_b200.ledger import config_from_workload


def _cfg(**kw):
    return config_from_workload(W.moderate().replace(**kw))


def test_plan_orders_buckets_by_width_and_keeps_input_order_inside():
    order, n, lb, sb = B.rr_bucket_plan(_cfg(), [16, 8, 16, 12, 8, 16, 12, 16])
    assert n == 3
    assert order == [1, 4, 3, 6, 0, 2, 5, 7]
    # the set's buffers hold every bucket's stand-alone buffers, each rounded up to 256 bytes
    total_l = total_s = 0
    for k, heads in ((8, 2), (12, 2), (16, 4)):
        l, s = B.rr_workspace_bytes(_cfg(batch=1, heads=heads, k=k))
        total_l += -(-l // 256) * 256
        total_s += -(-s // 256) * 256
    assert (lb, sb) == (total_l, total_s)


def test_one_width_is_one_bucket_with_the_plain_ledger_size():
    cfg = _cfg()
    order, n, lb, sb = B.rr_bucket_plan(cfg, [16] * 8)
    assert n == 1 and order == list(range(8))
    l, s = B.rr_workspace_bytes(cfg)
    assert lb == -(-l // 256) * 256 and sb == -(-s // 256) * 256


@pytest.mark.parametrize("widths", [[16] * 7, [16] * 7 + [0], [16] * 7 + [257]])
def test_bad_widths_are_rejected(widths):
    with pytest.raises(B.RouteRelayError) as ei:
        B.rr_bucket_plan(_cfg(), widths)
    assert ei.value.code == B.RR_ERR_INVALID_ARG
