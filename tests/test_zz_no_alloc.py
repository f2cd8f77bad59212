"""cosa_kap_select_static: the allocation-free Stage-1 entry point must give exactly the lists of the regular one.

It serves hosts that cannot allocate device memory at call time (a server whose pool owns the whole GPU, a
request loop that must not synchronise the device), so its scratch is a fixed array inside the library.
The test calls it twice in a row through the C ABI -- the second call finds the array as the first left
it -- and compares both results with cosa_kap_select_ex; it also checks the size limit is enforced.
"""
import numpy as np
import pytest
import torch

import paper_2607_25291_b200 as cosa
from synth.configs import tiny
from tests.helpers import alloc_lists, to_dev

pytestmark = pytest.mark.gpu


def test_static_scratch_entry_point_matches_regular_one_twice():
    results = []
    for seed, hq, hkv, n, budget in ((31, 4, 2, 2048, 0.3), (32, 8, 2, 4096, 0.2)):
        qb, kb, _, _ = tiny(seed=seed, hq=hq, hkv=hkv, n=n, needles=3).make()
        q, k = to_dev(qb), to_dev(kb)
        nqb = n // 128
        ref_order, ref_count = alloc_lists(hq, nqb)
        cosa.cosa_kap_select(q, k, budget, ref_order, ref_count, opt=cosa.default_options())
        order, count = alloc_lists(hq, nqb)
        cosa.cosa_kap_select_static(q, k, budget, order, count, opt=cosa.default_options())
        assert cosa.cosa_device_status() == 0
        assert torch.equal(order, ref_order) and torch.equal(count, ref_count)
        assert int(count.min()) >= 1
        results.append((order, count))
    assert len(results) == 2


def test_static_scratch_rejects_problems_beyond_its_size():
    n, hq = 32768, 32
    assert cosa.cosa_workspace_bytes(0, cosa.CosaShape(1, hq, 8, n, 128, 128, 128, 1)) > cosa.cosa_kap_select_static_max_bytes()
    q = torch.zeros(1, hq, n, 128, dtype=torch.bfloat16, device="cuda")
    k = torch.zeros(1, 8, n, 128, dtype=torch.bfloat16, device="cuda")
    order, count = alloc_lists(hq, n // 128)
    with pytest.raises(cosa.CosaError) as e:
        cosa.cosa_kap_select_static(q, k, 0.1, order, count)
    assert e.value.status == -3
    assert int(count[0, 0, 0]) == -7                      # nothing was enqueued
