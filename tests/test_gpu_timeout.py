"""The path a kernel takes when one of its bounded waits runs out.

Every wait inside the tensor-core kernels gives up after a clock budget, sets the device status word and lets the CTA
wind down: in-flight copies and products are awaited, tensor memory is released, nothing further is written, and the
CTAs that start afterwards return at once.  cosa_options.wait_cycles sets that budget per call; a budget of one cycle
makes every wait that is not satisfied on the spot run out, so the path is reached without any kernel ever waiting
for something that does not come.  After such a call cosa_device_status() reports COSA_ERR_DEVICE_TIMEOUT once, and
the same call with the default budget then gives the regular result.
"""
import numpy as np
import pytest
import torch

import paper_2607_25291_b200 as cosa
from synth.configs import WORKLOADS
from tests.helpers import alloc_lists, alloc_outputs, to_dev

pytestmark = pytest.mark.gpu

TIMEOUT = -5


@pytest.fixture(scope="module")
def cfg1():
    w = WORKLOADS["gqa4_4k"]
    qb, kb, vb, _ = w.make()
    return dict(w=w, dev=tuple(to_dev(x) for x in (qb, kb, vb)))


def test_kap_wait_budget_of_one_cycle_reports_a_timeout_and_the_next_call_is_clean(cfg1):
    w, (q, k, _) = cfg1["w"], cfg1["dev"]
    nqb = w.n // 128
    ref_order, ref_count = alloc_lists(w.hq, nqb)
    cosa.cosa_kap_select(q, k, w.kap_budget, ref_order, ref_count, opt=cosa.default_options(stride=w.stride))
    assert cosa.cosa_device_status() == 0
    order, count = alloc_lists(w.hq, nqb)
    cosa.cosa_kap_select(q, k, w.kap_budget, order, count, opt=cosa.default_options(stride=w.stride, wait_cycles=1))
    assert cosa.cosa_device_status() == TIMEOUT        # reported once ...
    assert cosa.cosa_device_status() == 0              # ... then cleared
    assert int((count == -7).sum()) == count.numel()   # the later kernels of the call wrote nothing
    cosa.cosa_kap_select(q, k, w.kap_budget, order, count, opt=cosa.default_options(stride=w.stride))
    assert cosa.cosa_device_status() == 0
    assert torch.equal(order, ref_order) and torch.equal(count, ref_count)


@pytest.mark.parametrize("impl", [0, 4, 5])     # one work item per CTA, two work items per CTA, the two row tiles of a 256-row block per CTA
def test_osk_wait_budget_of_one_cycle_reports_a_timeout_and_the_next_call_is_clean(cfg1, impl):
    w, (q, k, v) = cfg1["w"], cfg1["dev"]
    nqb = w.n // 128
    order, count = alloc_lists(w.hq, nqb)
    cosa.cosa_kap_select(q, k, w.kap_budget, order, count, opt=cosa.default_options(stride=w.stride),
                         block_q=256 if impl == 5 else 128)
    ref = alloc_outputs(q, nqb)
    cosa.cosa_osk_attention(q, k, v, order, count, w.osk_budget, ref["out"], ref["lse"], ref["visited"],
                            opt=cosa.default_options(skip_scale=w.skip_scale, impl=impl))
    assert cosa.cosa_device_status() == 0
    for _ in range(2):                                  # twice: a timed-out call leaves nothing behind that trips the next
        bufs = alloc_outputs(q, nqb)
        bufs["visited"].fill_(-7)
        cosa.cosa_osk_attention(q, k, v, order, count, w.osk_budget, bufs["out"], bufs["lse"], bufs["visited"],
                                opt=cosa.default_options(skip_scale=w.skip_scale, wait_cycles=1, impl=impl))
        assert cosa.cosa_device_status() == TIMEOUT
        assert cosa.cosa_device_status() == 0
        assert int((bufs["visited"] == -7).sum()) > 0   # the CTAs that started after the first timeout returned at once
    bufs = alloc_outputs(q, nqb)
    cosa.cosa_osk_attention(q, k, v, order, count, w.osk_budget, bufs["out"], bufs["lse"], bufs["visited"],
                            opt=cosa.default_options(skip_scale=w.skip_scale, impl=impl))
    assert cosa.cosa_device_status() == 0
    assert torch.equal(bufs["out"], ref["out"]) and torch.equal(bufs["visited"], ref["visited"])
    assert torch.equal(bufs["lse"], ref["lse"])


def test_status_word_set_by_hand_makes_both_stages_return_at_once(cfg1):
    """The same early return, reached without any wait: with the status word already set when the kernels start, they
    leave their outputs untouched; reading the status clears it."""
    w, (q, k, v) = cfg1["w"], cfg1["dev"]
    nqb = w.n // 128
    good_order, good_count = alloc_lists(w.hq, nqb)
    cosa.cosa_kap_select(q, k, w.kap_budget, good_order, good_count, opt=cosa.default_options(stride=w.stride))
    assert cosa.cosa_device_status() == 0
    cosa.cosa_debug_set_device_status(TIMEOUT)
    order, count = alloc_lists(w.hq, nqb)
    cosa.cosa_kap_select(q, k, w.kap_budget, order, count, opt=cosa.default_options(stride=w.stride))
    bufs = alloc_outputs(q, nqb)
    bufs["visited"].fill_(-7)
    bufs["out"].fill_(3.0)
    cosa.cosa_osk_attention(q, k, v, good_order, good_count, w.osk_budget, bufs["out"], bufs["lse"], bufs["visited"],
                            opt=cosa.default_options(skip_scale=w.skip_scale))
    assert cosa.cosa_device_status() == TIMEOUT
    assert cosa.cosa_device_status() == 0
    assert int((count == -7).sum()) == count.numel() and int((order == -7).sum()) == order.numel()
    assert int((bufs["visited"] == -7).sum()) == bufs["visited"].numel()
    assert bool((bufs["out"] == 3.0).all())
