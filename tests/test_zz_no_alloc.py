"""cosa_kap_select_static: the allocation-free Stage-1 entry point must give exactly the lists of the regular one.

It serves hosts that cannot allocate device memory at call time (a server whose pool owns the whole GPU, a
request loop that must not synchronise the device), so its scratch is a fixed array inside the library.
The test calls it twice in a row through the C ABI -- the second call finds the array as the first left
it -- and compares both results with cosa_kap_select_ex and one of them with the fp64 oracle; it checks that
the free device memory does not move across the calls, and that the size limit is enforced at the sizes the
header names.
"""
import numpy as np
import pytest
import torch

import paper_2607_25291_b200 as cosa
from oracle import cosa_oracle as O
from synth.configs import tiny
from tests.helpers import alloc_lists, to_dev, widen

pytestmark = pytest.mark.gpu


def test_static_scratch_entry_point_matches_regular_one_twice():
    results = []
    cases = ((31, 4, 2, 2048, 0.3), (32, 8, 2, 4096, 0.2))
    inputs = []
    for seed, hq, hkv, n, budget in cases:
        qb, kb, _, _ = tiny(seed=seed, hq=hq, hkv=hkv, n=n, needles=3).make()
        inputs.append((qb, kb, to_dev(qb), to_dev(kb)))
    # every buffer of the loop below exists before the first call, and one warm-up call has looked up the array's
    # address: from here on the free memory of the device must not move
    bufs = [(alloc_lists(hq, n // 128), alloc_lists(hq, n // 128)) for _, hq, _, n, _ in cases]
    cosa.cosa_kap_select_static(inputs[0][2], inputs[0][3], cases[0][4], *bufs[0][1], opt=cosa.default_options())
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    for (seed, hq, hkv, n, budget), (qb, kb, q, k), ((ref_order, ref_count), (order, count)) in zip(cases, inputs, bufs):
        order.fill_(-7); count.fill_(-7)
        cosa.cosa_kap_select_static(q, k, budget, order, count, opt=cosa.default_options())
        assert cosa.cosa_device_status() == 0
        results.append((order, count))
    assert torch.cuda.mem_get_info()[0] == free_before     # nothing was allocated (or freed) by the two calls
    for (seed, hq, hkv, n, budget), (qb, kb, q, k), ((ref_order, ref_count), (order, count)) in zip(cases, inputs, bufs):
        cosa.cosa_kap_select(q, k, budget, ref_order, ref_count, opt=cosa.default_options())
        assert cosa.cosa_device_status() == 0
        assert torch.equal(order, ref_order) and torch.equal(count, ref_count)
        assert int(count.min()) >= 1
    # the first case against the oracle as well
    (seed, hq, hkv, n, budget), (qb, kb, _, _) = cases[0], inputs[0][:4]
    qf, kf = widen(qb, kb)
    o_order, o_count = O.kap_select(qf, kf, s=8, budget=budget, order_stride=n // 128)
    assert np.array_equal(results[0][0][0].cpu().numpy(), o_order)
    assert np.array_equal(results[0][1][0].cpu().numpy(), o_count)


def test_static_scratch_size_limit_at_the_sizes_the_header_names():
    limit = cosa.cosa_kap_select_static_max_bytes()
    fits = cosa.CosaShape(1, 32, 8, 4096, 128, 128, 128, 1)
    assert cosa.cosa_workspace_bytes(0, fits) <= limit
    for hq, hkv, n in ((32, 8, 8192), (8, 2, 16384), (32, 8, 32768)):
        assert cosa.cosa_workspace_bytes(0, cosa.CosaShape(1, hq, hkv, n, 128, 128, 128, 1)) > limit
    # accepted at the limit's near side ...
    q = torch.randn(1, 32, 4096, 128, device="cuda").to(torch.bfloat16)
    k = torch.randn(1, 8, 4096, 128, device="cuda").to(torch.bfloat16)
    order, count = alloc_lists(32, 32)
    ref_order, ref_count = alloc_lists(32, 32)
    cosa.cosa_kap_select_static(q, k, 0.25, order, count)
    cosa.cosa_kap_select(q, k, 0.25, ref_order, ref_count)
    assert cosa.cosa_device_status() == 0
    assert torch.equal(order, ref_order) and torch.equal(count, ref_count)
    # ... and refused beyond it, with nothing enqueued
    n, hq, hkv = 16384, 8, 2
    q = torch.zeros(1, hq, n, 128, dtype=torch.bfloat16, device="cuda")
    k = torch.zeros(1, hkv, n, 128, dtype=torch.bfloat16, device="cuda")
    order, count = alloc_lists(hq, n // 128)
    with pytest.raises(cosa.CosaError) as e:
        cosa.cosa_kap_select_static(q, k, 0.1, order, count)
    assert e.value.status == -3
    torch.cuda.synchronize()
    assert int(count[0, 0, 0]) == -7 and int((order == -7).sum()) == order.numel()


def test_static_scratch_entry_point_in_a_fresh_process_touches_no_allocator():
    """In a process of its own, before any other entry point of the library has run: were the call to fall back on
    the library's cudaMalloc'ed scratch, the free memory of the device would drop across it."""
    import subprocess
    import sys
    code = r'''
import sys, torch
sys.path.insert(0, ".")
import paper_2607_25291_b200 as cosa
from synth.configs import tiny
from tests.helpers import alloc_lists, to_dev
qb, kb, _, _ = tiny(seed=31, hq=4, hkv=2, n=2048, needles=3).make()
q, k = to_dev(qb), to_dev(kb)
order, count = alloc_lists(4, 16)
torch.cuda.synchronize()
before = torch.cuda.mem_get_info()[0]
cosa.cosa_kap_select_static(q, k, 0.3, order, count, opt=cosa.default_options())
torch.cuda.synchronize()
mid = torch.cuda.mem_get_info()[0]          # (the first launch loads the kernels' code: allowed to cost memory once)
cosa.cosa_kap_select_static(q, k, 0.3, order, count, opt=cosa.default_options())
torch.cuda.synchronize()
after = torch.cuda.mem_get_info()[0]
assert cosa.cosa_device_status() == 0 and int(count.min()) >= 1
assert after == mid, (before, mid, after)
assert before - mid < (64 << 20), (before, mid)   # (code loading only)
print("ok", before - mid)
'''
    import os
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    res = subprocess.run([sys.executable, "-c", code], cwd=root, capture_output=True, text=True, timeout=300)
    assert res.returncode == 0 and "ok" in res.stdout, res.stdout + res.stderr
