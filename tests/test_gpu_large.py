"""Parity at the benchmark's full sizes, in the launch configuration bench.py times: the CUDA path runs the
whole workload, the fp64 oracle re-derives a sample of (head, query block) pairs one by one -- all heads x
query blocks {0, 1, 2, every 37th, last 3} -- plus properties that hold at any size."""
import numpy as np
import pytest
import torch

import paper_2607_25291_b200 as cosa
from oracle import cosa_oracle as O
from synth.configs import SWEEP_STAGE1, SWEEP_STAGE2_MULT, WORKLOADS
from synth.generator import bf16_bits_to_f64, scatter_to_pages
from tests.helpers import to_dev
from tests.test_gpu_parity import TOPP_MARGIN, _np, check_osk_against_oracle, check_topp_lists

pytestmark = pytest.mark.gpu


def sample_blocks(nqb):
    return sorted(set([0, 1, 2] + list(range(37, nqb, 37)) + [nqb - 3, nqb - 2, nqb - 1]))


class HeadView:
    """Presents one query head (and its KV head) of the bf16 bit tensors as the fp64 arrays the oracle takes."""
    def __init__(self, qb, kb, vb):
        self.qb, self.kb, self.vb = qb, kb, vb
        self.G = qb.shape[0] // kb.shape[0]
        self.cache = {}

    def get(self, h):
        g = h // self.G
        if ("q", h) not in self.cache:
            self.cache = {k: v for k, v in self.cache.items() if k[0] != "q"}
            self.cache[("q", h)] = bf16_bits_to_f64(self.qb[h])[None]
        if ("kv", g) not in self.cache:
            self.cache = {k: v for k, v in self.cache.items() if k[0] != "kv"}
            self.cache[("kv", g)] = (bf16_bits_to_f64(self.kb[g])[None], bf16_bits_to_f64(self.vb[g])[None])
        return (self.cache[("q", h)],) + self.cache[("kv", g)]


def run_and_check(w, qb, kb, vb, kap_budget, osk_budget, skip_scale, kap_heads, blocks, check_all_kap=False, top_p=0.0):
    q, k, v = (to_dev(x) for x in (qb, kb, vb))
    nqb = w.n_blocks
    pitch = (cosa.cosa_budget_count(kap_budget, nqb) + 7) // 8 * 8
    order = torch.empty(1, w.hq, nqb, pitch, dtype=torch.int32, device="cuda")
    count = torch.empty(1, w.hq, nqb, dtype=torch.int32, device="cuda")
    bufs = dict(out=torch.empty_like(q), lse=torch.empty(1, w.hq, w.n, dtype=torch.float32, device="cuda"),
                visited=torch.empty(1, w.hq, nqb, dtype=torch.int32, device="cuda"),
                scored=torch.empty(1, w.hq, nqb, dtype=torch.int32, device="cuda"),
                decisions=torch.zeros(1, w.hq, nqb, (pitch + 31) // 32, dtype=torch.int32, device="cuda"))
    ex = {}
    if top_p > 0:      # the float32 scores the Top-p count is decided on
        ex = dict(kap_scores=torch.zeros(1, w.hq, nqb, nqb, dtype=torch.float32, device="cuda"),
                  kap_flags=torch.zeros(1, w.hq, nqb, nqb, dtype=torch.uint8, device="cuda"))
    opt = cosa.default_options(stride=w.stride, skip_scale=skip_scale, order_stride=pitch, top_p=top_p,
                               out_scored=bufs["scored"], out_decisions=bufs["decisions"], **ex)
    cosa.cosa_kap_select(q, k, kap_budget, order, count, opt=opt)
    cosa.cosa_osk_attention(q, k, v, order, count, osk_budget, bufs["out"], bufs["lse"], bufs["visited"], opt=opt)
    assert cosa.cosa_device_status() == 0
    # properties at full size
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    cosa.cosa_validate_order(order, count, cosa.make_shape(q, k, True), status)
    assert int(status.item()) == 0
    order_np, count_np = _np(order), _np(count)
    J = np.arange(1, nqb + 1)
    want_count = np.array([O.budget_count(kap_budget, int(j)) for j in J])
    if top_p > 0:
        assert (count_np >= 1).all() and (count_np <= want_count[None, :]).all()
    else:
        assert (count_np == want_count[None, :]).all()
    vis, sco = _np(bufs["visited"]), _np(bufs["scored"])
    if osk_budget < 1.0:
        cap = np.minimum(want_count, np.array([O.budget_count(osk_budget, int(j)) for j in J]))
        assert (vis <= np.minimum(cap[None, :], count_np)).all()
    else:
        assert (vis == count_np).all()
    assert (sco <= count_np).all() and (vis >= 1).all() and (vis <= sco).all()
    assert torch.isfinite(bufs["out"].float()).all() and torch.isfinite(bufs["lse"]).all()
    for h in range(w.hq):                                   # every list holds distinct ids
        rows = np.sort(np.where(order_np[h] < 0, np.arange(order_np.shape[-1])[None, :] + 10 ** 6, order_np[h]), axis=1)
        assert (np.diff(rows, axis=1) != 0).all()
    # sampled parity against the oracle
    hv = HeadView(qb, kb, vb)
    stats = []
    s32, f8 = (_np(ex["kap_scores"]), _np(ex["kap_flags"])) if ex else (None, None)
    for h in kap_heads:
        qf, kf, vf = hv.get(h)
        sel = range(nqb) if check_all_kap else blocks
        if top_p > 0:
            ref_order, ref_count, audit = O.kap_select(qf, kf, s=w.stride, budget=kap_budget, order_stride=pitch,
                                                       query_blocks=(None if check_all_kap else blocks), top_p=top_p,
                                                       audit=True)
            check_topp_lists(order_np, count_np, ref_order, ref_count, audit["topp_margin"], TOPP_MARGIN[0],
                             [(h, 0, i) for i in sel], scores32=s32, flags=f8,
                             top_p=top_p, budget=kap_budget)
        else:
            ref_order, ref_count = O.kap_select(qf, kf, s=w.stride, budget=kap_budget, order_stride=pitch,
                                                query_blocks=(None if check_all_kap else blocks))
            for i in sel:
                assert ref_count[0, i] == count_np[h, i], (h, i)
                assert np.array_equal(ref_order[0, i], order_np[h, i]), (h, i)
        one = {k_: t[:, h:h + 1] for k_, t in bufs.items()}
        stats.append(check_osk_against_oracle(qf, kf, vf, order_np[h:h + 1], count_np[h:h + 1], one, osk_budget,
                                              skip_scale, [0], blocks))
    return dict(max_abs=max(s["max_abs"] for s in stats), mean_abs=float(np.mean([s["mean_abs"] for s in stats])),
                lse=max(s["lse"] for s in stats), near_margin=sum(s["near_margin"] for s in stats),
                scored=int(sco.sum()), computed=int(vis.sum()), listed=int(count_np.sum()))


def test_qwen3_32k_full_kap_and_sampled_osk():
    w = WORKLOADS["qwen3_32k"]
    qb, kb, vb, _ = w.make()
    stats = run_and_check(w, qb, kb, vb, w.kap_budget, w.osk_budget, w.skip_scale, range(w.hq),
                          sample_blocks(w.n_blocks), check_all_kap=True)
    assert stats["computed"] < stats["scored"] < stats["listed"]        # both Stage-2 mechanisms are at work
    print("32k", stats)


def test_qwen3_32k_sort_routes_agree():
    """The sort stage has three routes to the same list: head by pivot selection (taken here by nearly every list),
    head by radix selection, everything sorted.  All 8192 lists must come out identical on each (the first one is
    checked against the oracle, list by list, by the test above)."""
    w = WORKLOADS["qwen3_32k"]
    qb, kb, _, _ = w.make()
    q, k = to_dev(qb), to_dev(kb)
    nqb = w.n_blocks
    pitch = (cosa.cosa_budget_count(w.kap_budget, nqb) + 7) // 8 * 8
    lists = []
    for impl in (0, 2, 3):
        order = torch.empty(1, w.hq, nqb, pitch, dtype=torch.int32, device="cuda")
        count = torch.empty(1, w.hq, nqb, dtype=torch.int32, device="cuda")
        cosa.cosa_kap_select(q, k, w.kap_budget, order, count, opt=cosa.default_options(stride=w.stride, order_stride=pitch, impl=impl))
        assert cosa.cosa_device_status() == 0
        lists.append((order, count))
    for order, count in lists[1:]:
        assert torch.equal(count, lists[0][1]) and torch.equal(order, lists[0][0])


def test_qwen3_128k_sampled():
    w = WORKLOADS["qwen3_128k"]
    qb, kb, vb, _ = w.make()
    stats = run_and_check(w, qb, kb, vb, w.kap_budget, w.osk_budget, w.skip_scale, range(w.hq),
                          sample_blocks(w.n_blocks))
    assert stats["computed"] < stats["scored"]
    print("128k", stats)


def test_qwen3_32k_and_128k_topp_sampled():
    """Stage 1 by Top-p (p = 0.95, no budget cap), Stage 2 as configured: lists of data-dependent length."""
    for name, heads in (("qwen3_32k", range(0, 32, 5)), ("qwen3_128k", [3, 17, 30])):
        w = WORKLOADS[name]
        qb, kb, vb, _ = w.make()
        stats = run_and_check(w, qb, kb, vb, 1.0, w.osk_budget, w.skip_scale, heads, sample_blocks(w.n_blocks), top_p=0.95)
        pairs = w.hq * w.n_blocks * (w.n_blocks + 1) // 2
        assert stats["listed"] < pairs
        print(name, "top-p 0.95", stats, "listed fraction", stats["listed"] / pairs)


def test_qwen3_32k_paged_equals_dense():
    """Page pools of 16-, 64- and 256-token pages (Sec. C.1) against the dense tensors they hold, whole workload."""
    w = WORKLOADS["qwen3_32k"]
    qb, kb, vb, _ = w.make()
    q, k, v = (to_dev(x) for x in (qb, kb, vb))
    nqb = w.n_blocks
    pitch = (cosa.cosa_budget_count(w.kap_budget, nqb) + 7) // 8 * 8

    def run(kk, vv, **paging):
        order = torch.empty(1, w.hq, nqb, pitch, dtype=torch.int32, device="cuda")
        count = torch.empty(1, w.hq, nqb, dtype=torch.int32, device="cuda")
        out = torch.empty_like(q)
        vis = torch.empty(1, w.hq, nqb, dtype=torch.int32, device="cuda")
        opt = cosa.default_options(stride=w.stride, skip_scale=w.skip_scale, order_stride=pitch, **paging)
        cosa.cosa_kap_select(q, kk, w.kap_budget, order, count, opt=opt)
        cosa.cosa_osk_attention(q, kk, vv, order, count, w.osk_budget, out, None, vis, opt=opt)
        assert cosa.cosa_device_status() == 0
        return order, count, out, vis

    dense = run(k, v)
    for page_size in (16, 64, 256):
        kpool, table = scatter_to_pages(kb, page_size, seed=12)
        vpool, _ = scatter_to_pages(vb, page_size, seed=12)
        dev = lambda a: torch.from_numpy(a.view(np.int16)).view(torch.bfloat16).cuda().contiguous()
        paged = run(dev(kpool), dev(vpool), kv_page_table=torch.from_numpy(table).cuda()[None].contiguous(),
                    kv_page_size=page_size, kv_num_pages=kpool.shape[0])
        for a, b in zip(dense, paged):
            assert torch.equal(a, b)


def test_qwen3_32k_wide_query_blocks_sampled():
    """block_q = 256 lists at 32K against the oracle on sampled blocks, and OSK on them."""
    w = WORKLOADS["qwen3_32k"]
    qb, kb, vb, _ = w.make()
    q, k, v = (to_dev(x) for x in (qb, kb, vb))
    nqb = w.n_blocks
    pitch = (cosa.cosa_budget_count(w.kap_budget, nqb) + 7) // 8 * 8
    order = torch.empty(1, w.hq, nqb, pitch, dtype=torch.int32, device="cuda")
    count = torch.empty(1, w.hq, nqb, dtype=torch.int32, device="cuda")
    bufs = dict(out=torch.empty_like(q), lse=torch.empty(1, w.hq, w.n, dtype=torch.float32, device="cuda"),
                visited=torch.empty(1, w.hq, nqb, dtype=torch.int32, device="cuda"),
                scored=torch.empty(1, w.hq, nqb, dtype=torch.int32, device="cuda"),
                decisions=torch.zeros(1, w.hq, nqb, (pitch + 31) // 32, dtype=torch.int32, device="cuda"))
    opt = cosa.default_options(stride=w.stride, skip_scale=w.skip_scale, order_stride=pitch,
                               out_scored=bufs["scored"], out_decisions=bufs["decisions"])
    cosa.cosa_kap_select(q, k, w.kap_budget, order, count, opt=opt, block_q=256)
    cosa.cosa_osk_attention(q, k, v, order, count, w.osk_budget, bufs["out"], bufs["lse"], bufs["visited"], opt=opt)
    assert cosa.cosa_device_status() == 0
    order_np, count_np = _np(order), _np(count)
    wide = sorted(set(b // 2 for b in sample_blocks(nqb)))
    hv = HeadView(qb, kb, vb)
    for h in range(0, w.hq, 3):
        qf, kf, vf = hv.get(h)
        ref_order, ref_count = O.kap_select_wide(qf, kf, s=w.stride, budget=w.kap_budget, order_stride=pitch, wide_blocks=wide)
        tiles = [2 * b + t for b in wide for t in (0, 1)]
        for i in tiles:
            assert ref_count[0, i] == count_np[h, i] and np.array_equal(ref_order[0, i], order_np[h, i]), (h, i)
        one = {k_: t[:, h:h + 1] for k_, t in bufs.items()}
        check_osk_against_oracle(qf, kf, vf, order_np[h:h + 1], count_np[h:h + 1], one, w.osk_budget, w.skip_scale, [0], tiles[::3])
    # the same lists walked by one CTA per 256-row block, every fetched K/V tile serving both row tiles (impl = 5): every
    # decision and counter of the layer as above, outputs within rounding of them
    shared = {k_: torch.zeros_like(t) for k_, t in bufs.items()}
    opt5 = cosa.default_options(stride=w.stride, skip_scale=w.skip_scale, order_stride=pitch, impl=5,
                                out_scored=shared["scored"], out_decisions=shared["decisions"])
    cosa.cosa_osk_attention(q, k, v, order, count, w.osk_budget, shared["out"], shared["lse"], shared["visited"], opt=opt5)
    assert cosa.cosa_device_status() == 0
    for key in ("visited", "scored", "decisions"):
        assert torch.equal(shared[key], bufs[key]), key
    assert float((shared["out"].float() - bufs["out"].float()).abs().max()) < 2e-2
    assert float((shared["lse"] - bufs["lse"]).abs().max()) < 1e-3


def test_llama31_64k_budget_sweep_sampled():
    w = WORKLOADS["llama31_64k_sweep"]
    qb, kb, vb, _ = w.make()
    blocks = sample_blocks(w.n_blocks)[::2]
    for b1 in SWEEP_STAGE1:
        for mult in SWEEP_STAGE2_MULT:
            tb = 1.0 if mult == 1.0 else b1 * mult            # the 1.0x column runs with Stage 2 off
            stats = run_and_check(w, qb, kb, vb, b1, tb, w.skip_scale, [0, 13, 31], blocks)
            print("64k sweep", b1, mult, stats)


def test_qwen3_128k_stack_layers_sampled():
    w = WORKLOADS["qwen3_128k_x36"]
    for layer in (0, 4):                                       # 8 and 128 needle blocks per head
        qb, kb, vb, _ = w.make(layer=layer)
        stats = run_and_check(w, qb, kb, vb, w.kap_budget, w.osk_budget, w.skip_scale, [1, 18], sample_blocks(w.n_blocks)[::3])
        print("128k stack layer", layer, stats)


def test_dense_path_long_lists_sampled():
    """The library's dense path (full causal lists of up to 1024 blocks, Stage 2 off) at 128K: sampled query
    blocks against the oracle's dense attention, every block counted as visited."""
    w = WORKLOADS["qwen3_128k"]
    qb, kb, vb, _ = w.make()
    q, k, v = (to_dev(x) for x in (qb, kb, vb))
    nqb = w.n_blocks
    tri = torch.arange(nqb, device="cuda", dtype=torch.int32)
    full = torch.where(tri[None, :] <= tri[:, None], tri[None, :].expand(nqb, nqb),
                       torch.full((), -1, dtype=torch.int32, device="cuda")).expand(1, w.hq, nqb, nqb).contiguous()
    fcount = (tri + 1).expand(1, w.hq, nqb).contiguous()
    out = torch.empty_like(q)
    lse = torch.empty(1, w.hq, w.n, dtype=torch.float32, device="cuda")
    vis = torch.empty(1, w.hq, nqb, dtype=torch.int32, device="cuda")
    cosa.cosa_osk_attention(q, k, v, full, fcount, 1.0, out, lse, vis, opt=cosa.default_options(order_stride=nqb))
    assert cosa.cosa_device_status() == 0
    assert torch.equal(vis, fcount)
    hv = HeadView(qb, kb, vb)
    for h, blocks in ((0, [0, 1, 300, 1023]), (17, [511, 1022]), (31, [2, 777])):
        qf, kf, vf = hv.get(h)
        ref_o, ref_l = O.dense_attention(qf, kf, vf, query_blocks=blocks)
        for a, i in enumerate(blocks):
            got = out[0, h, i * 128:(i + 1) * 128].float().cpu().numpy().astype(np.float64)
            err = np.abs(got - ref_o[0, a * 128:(a + 1) * 128])
            assert err.max() < 2e-2 and err.mean() < 2e-3, (h, i, err.max(), err.mean())
            assert np.abs(lse[0, h, i * 128:(i + 1) * 128].cpu().numpy() - ref_l[0, a * 128:(a + 1) * 128]).max() < 1e-3
