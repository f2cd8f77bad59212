"""CUDA path vs the fp64 oracle, element by element, through the C ABI (via the thin binding).

Bars: KAP order/count lists bit-exact; OSK visited/scored counts and decisions exact except at
list positions whose oracle skip margin |gap - theta| / |theta| is below 1e-4 (either decision
is then accepted and the comparison follows the GPU's choice there); OSK outputs (bf16 inputs,
fp32 accumulation) within max-abs 2e-2 and mean-abs 2e-3 of the oracle, LSE within 1e-3.
"""
import ctypes
import math

import numpy as np
import pytest
import torch

import paper_2607_25291_b200 as cosa
from oracle import cosa_oracle as O
from synth.configs import WORKLOADS, tiny
from synth.generator import bf16_bits_to_f64, scatter_to_pages
from tests.helpers import alloc_lists, alloc_outputs, to_dev, widen

pytestmark = pytest.mark.gpu

OUT_MAX, OUT_MEAN, LSE_TOL, MARGIN = 2e-2, 2e-3, 1e-3, 1e-4
IMPLS = (0, 1)
OSK_IMPLS = (0, 1, 4)     # tensor-core kernel, CUDA-core check kernel, tensor-core kernel with two work items per CTA


def _np(t):
    return t[0].cpu().numpy()


def run_kap(q, k, budget, stride=8, causal=True, order_stride=None, scores=False, impl=0, top_p=0.0):
    _, hq, n, _ = q.shape
    nqb = n // 128
    order, count = alloc_lists(hq, nqb, order_stride)
    kw = {}
    if scores:
        kw["kap_scores"] = torch.zeros(1, hq, nqb, nqb, dtype=torch.float32, device="cuda")
        kw["kap_flags"] = torch.zeros(1, hq, nqb, nqb, dtype=torch.uint8, device="cuda")
    opt = cosa.default_options(stride=stride, impl=impl, top_p=top_p, **kw)
    cosa.cosa_kap_select(q, k, budget, order, count, causal=causal, opt=opt)
    assert cosa.cosa_device_status() == 0
    return (order, count, kw) if scores else (order, count)


# Top-p counts: an integer decided by floating point, which both sides take in the same precision.  On the fast path
# that is the kernel's: float32 scores (relative error < 2^-17 against exact arithmetic, asserted on the full-size
# workloads), cumulated in double precision -- the count must be exactly the one those float32 scores give
# (check_topp_lists, `scores32`).  Against the all-double oracle it may then differ by one, and only where the
# oracle's own prefix sum lies within 2^-16 of the threshold; the exact kernel (impl = 1) agrees with the oracle to a
# few ulp of double precision.
TOPP_MARGIN = {0: 2.0 ** -16, 1: 1e-12}


def topp_count_in_kernel_precision(s32, flags, top_p, cap):
    """The Top-p count decided on the float32 scores the fast path sorts (the precision the kernel takes this
    decision in): candidates in the order (flag descending, float32 score descending, id ascending), prefix sums in
    double precision.  Returns (K, relative margin of the deciding prefix sums)."""
    J = len(s32)
    ids = np.lexsort((np.arange(J), -s32.astype(np.float64), -flags.astype(np.int64)))
    c = np.cumsum(s32[ids].astype(np.float64))
    thr = float(top_p) * c[-1]
    K = min(J, int(np.searchsorted(c, thr, side="left")) + 1)
    gaps = [abs(c[K - 1] - thr)] + ([abs(c[K - 2] - thr)] if K >= 2 else [])
    return min(K, cap), min(gaps) / c[-1]


def check_topp_lists(order_np, count_np, ref_order, ref_count, margin, tol, pairs, scores32=None, flags=None, top_p=None,
                     budget=1.0):
    """GPU lists against the oracle's Top-p lists for the (h_gpu, h_ref, i) triples in `pairs`.  With the fast path's
    exported float32 scores the count is also held to the decision taken in that precision, exactly."""
    off = 0
    for hg, hr, i in pairs:
        kept, want = int(count_np[hg, i]), int(ref_count[hr, i])
        if scores32 is not None:
            k32, m32 = topp_count_in_kernel_precision(scores32[hg, i, :i + 1], flags[hg, i, :i + 1], top_p,
                                                      O.budget_count(budget, i + 1))
            # (a query block the fast path hands to the double-precision kernel is counted there)
            assert kept == k32 or kept == want or m32 <= 1e-12, (hg, i, kept, k32, want, m32)
        if margin[hr, i] > tol:
            assert kept == want, (hg, i, kept, want, margin[hr, i])
        else:
            assert abs(kept - want) <= 1, (hg, i, kept, want)
            off += kept != want
        both = min(kept, want)
        assert np.array_equal(order_np[hg, i, :both], ref_order[hr, i, :both]), (hg, i)
        assert (order_np[hg, i, kept:] == -1).all()
        if kept > want:                                     # one more entry than the oracle: a fresh candidate id
            extra = int(order_np[hg, i, want])
            assert 0 <= extra <= i and extra not in set(ref_order[hr, i, :want].tolist())
    return off


def run_osk(q, k, v, order, count, tb, skip_scale, impl=0, causal=True):
    bufs = alloc_outputs(q, order.shape[-1])
    opt = cosa.default_options(skip_scale=skip_scale, impl=impl, out_scored=bufs["scored"],
                               out_decisions=bufs["decisions"])
    cosa.cosa_osk_attention(q, k, v, order, count, tb, bufs["out"], bufs["lse"], bufs["visited"], causal=causal,
                            opt=opt)
    assert cosa.cosa_device_status() == 0
    return bufs


def check_osk_against_oracle(qf, kf, vf, order_np, count_np, bufs, tb, skip_scale, heads, query_blocks, causal=True):
    """Decisions, counters and outputs of the listed (head, query block) pairs."""
    n = qf.shape[1]
    nkb = n // 128
    out = _np(bufs["out"].float()).astype(np.float64)
    lse = _np(bufs["lse"]).astype(np.float64)
    visited, scored = _np(bufs["visited"]), _np(bufs["scored"])
    dec_words = _np(bufs["decisions"]).view(np.uint32)
    stage2 = tb < 1.0
    use_rule = stage2 and skip_scale > 0
    theta = math.log(skip_scale / n) if use_rule else None
    worst_max, sum_abs, n_el, worst_lse, free = 0.0, 0.0, 0, 0.0, 0
    for h in heads:
        for i in query_blocks:
            cnt = int(count_np[h, i])
            J = i + 1 if causal else nkb
            cap = min(cnt, O.budget_count(tb, J)) if stage2 else cnt
            gaps = O.osk_gaps_offline(qf, kf, order_np, count_np, h, i, causal=causal)
            gpu_dec = [(int(dec_words[h, i, kk >> 5]) >> (kk & 31)) & 1 == 1 for kk in range(cnt)]
            want, computed = [], 0
            for kk in range(cnt):
                if computed == cap:
                    break
                if use_rule and abs(gaps[kk] - theta) < MARGIN * abs(theta):
                    d = gpu_dec[kk]                       # near the margin: either decision is accepted
                    free += 1
                else:
                    d = not (use_rule and gaps[kk] < theta)
                want.append(d)
                computed += d
            assert gpu_dec[:len(want)] == want and not any(gpu_dec[len(want):]), (h, i)
            assert scored[h, i] == len(want) and visited[h, i] == sum(want), (h, i)
            ids = [int(order_np[h, i, kk]) for kk, d in enumerate(want) if d]
            ref_o, ref_l = _masked_one(qf, kf, vf, h, i, ids, causal)
            rows = slice(i * 128, (i + 1) * 128)
            err = np.abs(out[h, rows] - ref_o)
            worst_max = max(worst_max, err.max())
            sum_abs += err.sum()
            n_el += err.size
            worst_lse = max(worst_lse, np.abs(lse[h, rows] - ref_l).max())
    assert worst_max < OUT_MAX, worst_max
    assert sum_abs / n_el < OUT_MEAN, sum_abs / n_el
    assert worst_lse < LSE_TOL, worst_lse
    return dict(max_abs=worst_max, mean_abs=sum_abs / n_el, lse=worst_lse, near_margin=free)


def _masked_one(qf, kf, vf, h, i, ids, causal):
    """Oracle masked attention of one (head, query block) over key blocks `ids`."""
    G = qf.shape[0] // kf.shape[0]
    o, l = O.masked_attention(qf[h:h + 1], kf[h // G:h // G + 1], vf[h // G:h // G + 1], [[ids]], causal=causal,
                              query_blocks=[i])
    return o[0], l[0]


# ---------------------------------------------------------------------------------- fixtures
@pytest.fixture(scope="module")
def small():
    w = tiny(seed=21, hq=4, hkv=2, n=1024, needles=2)
    qb, kb, vb, _ = w.make()
    return dict(w=w, dev=tuple(to_dev(x) for x in (qb, kb, vb)), f64=widen(qb, kb, vb))


@pytest.fixture(scope="module")
def cfg1():
    w = WORKLOADS["gqa4_4k"]
    qb, kb, vb, _ = w.make()
    return dict(w=w, dev=tuple(to_dev(x) for x in (qb, kb, vb)), f64=widen(qb, kb, vb))


# ---------------------------------------------------------------------------------- KAP
@pytest.mark.parametrize("impl", IMPLS)
@pytest.mark.parametrize("stride", [4, 8, 16, 32, 128])
@pytest.mark.parametrize("budget", [0.1, 0.5, 1.0])
def test_kap_lists_bit_exact_small(small, stride, budget, impl):
    q, k, _ = small["dev"]
    qf, kf, _ = small["f64"]
    order, count = run_kap(q, k, budget, stride, impl=impl)
    ref_order, ref_count = O.kap_select(qf, kf, s=stride, budget=budget, order_stride=order.shape[-1])
    assert np.array_equal(_np(count), ref_count)
    assert np.array_equal(_np(order), ref_order)


@pytest.mark.parametrize("impl", IMPLS)
@pytest.mark.parametrize("top_p,budget", [(0.5, 1.0), (0.9, 1.0), (0.95, 1.0), (1.0, 1.0), (0.95, 0.3)])
def test_kap_topp_small(small, impl, top_p, budget):
    q, k, _ = small["dev"]
    qf, kf, _ = small["f64"]
    for stride in (8, 32):
        order, count, ex = run_kap(q, k, budget, stride, impl=impl, top_p=top_p, scores=True)
        ref_order, ref_count, audit = O.kap_select(qf, kf, s=stride, budget=budget, order_stride=order.shape[-1],
                                                   top_p=top_p, audit=True)
        pairs = [(h, h, i) for h in range(qf.shape[0]) for i in range(qf.shape[1] // 128)]
        strict = dict(scores32=_np(ex["kap_scores"]), flags=_np(ex["kap_flags"]), top_p=top_p, budget=budget) if impl == 0 else {}
        check_topp_lists(_np(order), _np(count), ref_order, ref_count, audit["topp_margin"], TOPP_MARGIN[impl], pairs, **strict)
        if top_p == 1.0:
            assert np.array_equal(_np(count), ref_count)


@pytest.mark.parametrize("impl", IMPLS)
def test_kap_topp_4k(cfg1, impl):
    q, k, _ = cfg1["dev"]
    qf, kf, _ = cfg1["f64"]
    w = cfg1["w"]
    order, count, ex = run_kap(q, k, 1.0, w.stride, impl=impl, top_p=0.95, scores=True)
    ref_order, ref_count, audit = O.kap_select(qf, kf, s=w.stride, budget=1.0, order_stride=order.shape[-1],
                                               top_p=0.95, audit=True)
    pairs = [(h, h, i) for h in range(w.hq) for i in range(w.n_blocks)]
    strict = dict(scores32=_np(ex["kap_scores"]), flags=_np(ex["kap_flags"]), top_p=0.95) if impl == 0 else {}
    off = check_topp_lists(_np(order), _np(count), ref_order, ref_count, audit["topp_margin"], TOPP_MARGIN[impl], pairs, **strict)
    assert off <= 2
    assert (ref_count < np.arange(1, w.n_blocks + 1)[None, :]).any()      # Top-p does drop blocks on this workload


def test_kap_topp_rejects_bad_p(small):
    q, k, _ = small["dev"]
    order, count = alloc_lists(q.shape[1], q.shape[2] // 128, None)
    for bad in (-0.1, 1.5, float("nan")):
        with pytest.raises(cosa.CosaError):
            cosa.cosa_kap_select(q, k, 1.0, order, count, opt=cosa.default_options(top_p=bad))


@pytest.mark.parametrize("impl", IMPLS)
def test_kap_noncausal_and_narrow_pitch(small, impl):
    q, k, _ = small["dev"]
    qf, kf, _ = small["f64"]
    order, count = run_kap(q, k, 0.4, 8, causal=False, order_stride=5, impl=impl)
    ref_order, ref_count = O.kap_select(qf, kf, s=8, budget=0.4, causal=False, order_stride=5)
    assert np.array_equal(_np(count), ref_count) and np.array_equal(_np(order), ref_order)
    # a pitch that cannot hold the longest list is refused before anything is launched
    order, count = alloc_lists(4, 8, 3)
    with pytest.raises(cosa.CosaError) as e:
        cosa.cosa_kap_select(q, k, 0.5, order, count, opt=cosa.default_options())
    assert e.value.status == -1


@pytest.mark.parametrize("impl", IMPLS)
def test_kap_exported_scores_and_flags(cfg1, impl):
    """The float32 screen must stay well inside the near-tie threshold (2^-13 relative) that decides
    what the double-precision recount looks at: its error is asserted below a quarter of it."""
    q, k, _ = cfg1["dev"]
    qf, kf, _ = cfg1["f64"]
    order, count, ex = run_kap(q, k, 0.5, 8, scores=True, impl=impl)
    sc, fl = _np(ex["kap_scores"]), _np(ex["kap_flags"])
    worst = 0.0
    for h in range(4):
        for i in range(32):
            s_ref, f_ref, _ = O.kap_scores(qf, kf, h, i, 8)
            worst = max(worst, float(np.abs(sc[h, i, :i + 1] / s_ref - 1).max()))
            assert np.array_equal(fl[h, i, :i + 1].astype(bool), f_ref)
    assert worst < (2.0 ** -13) / 4, worst


def test_kap_duplicate_key_blocks_tie_break(small):
    """Two identical key blocks give exactly equal scores: the float32 screen sees a tie chain (and rows whose
    two best blocks coincide), the recount must still deliver the ascending-id tie-break of the oracle."""
    q, k, _ = small["dev"]
    qf, kf, _ = small["f64"]
    k2, kf2 = k.clone(), kf.copy()
    for src, dst in ((0, 2), (3, 5)):                     # block 0 is the sink: rows tie at their maximum
        k2[0, :, dst * 128:(dst + 1) * 128] = k2[0, :, src * 128:(src + 1) * 128]
        kf2[:, dst * 128:(dst + 1) * 128] = kf2[:, src * 128:(src + 1) * 128]
    for impl in IMPLS:
        order, count = run_kap(q, k2, 0.6, 8, impl=impl)
        ref_order, ref_count = O.kap_select(qf, kf2, s=8, budget=0.6, order_stride=8)
        assert np.array_equal(_np(count), ref_count) and np.array_equal(_np(order), ref_order)


@pytest.mark.parametrize("impl", IMPLS)
def test_kap_lists_bit_exact_4k(cfg1, impl):
    w = cfg1["w"]
    q, k, _ = cfg1["dev"]
    qf, kf, _ = cfg1["f64"]
    order, count = run_kap(q, k, w.kap_budget, w.stride, impl=impl)
    ref_order, ref_count, audit = O.kap_select(qf, kf, s=w.stride, budget=w.kap_budget, order_stride=w.n_blocks,
                                               audit=True)
    assert audit["min_rel_score_gap"] > 1e-9 and audit["min_row_top2_gap"] > 1e-9   # inputs are well conditioned
    assert np.array_equal(_np(count), ref_count) and np.array_equal(_np(order), ref_order)


@pytest.fixture(scope="module")
def mid():
    w = tiny(seed=33, hq=4, hkv=2, n=16384, needles=6)
    qb, kb, vb, _ = w.make()
    return dict(w=w, dev=tuple(to_dev(x) for x in (qb, kb, vb)), f64=widen(qb, kb, vb))


MID_BLOCKS = [0, 1, 63, 64, 71, 72, 89, 90, 100, 117, 126, 127]


@pytest.mark.parametrize("impl", [0, 2, 3])
@pytest.mark.parametrize("budget", [0.05, 0.1, 0.25, 0.6])
def test_kap_16k_head_of_the_order(mid, budget, impl):
    """At 128 key blocks and a small budget the fast path selects and sorts only the head of the order (kept prefix
    plus a margin); larger budgets and short candidate lists sort everything.  Both must give the oracle's lists."""
    q, k, _ = mid["dev"]
    qf, kf, _ = mid["f64"]
    order, count = run_kap(q, k, budget, 8, impl=impl)   # 2, 3: the sort stage's fall-back routes, forced
    ref_order, ref_count = O.kap_select(qf, kf, s=8, budget=budget, order_stride=order.shape[-1], query_blocks=MID_BLOCKS)
    for i in MID_BLOCKS:
        assert np.array_equal(_np(count)[:, i], ref_count[:, i]), i
        assert np.array_equal(_np(order)[:, i], ref_order[:, i]), i


def test_kap_16k_tie_chain_longer_than_the_margin(mid):
    """Forty identical key blocks score exactly alike: a chain of near ties far longer than the margin kept beyond the
    prefix, which the head selection must hand over to the full sort, and whose members the double-precision
    recount must put in ascending-id order."""
    q, k, _ = mid["dev"]
    qf, kf, _ = mid["f64"]
    k2, kf2 = k.clone(), kf.copy()
    for dst in range(21, 61):
        k2[0, :, dst * 128:(dst + 1) * 128] = k2[0, :, 20 * 128:21 * 128]
        kf2[:, dst * 128:(dst + 1) * 128] = kf2[:, 20 * 128:21 * 128]
    blocks = [64, 90, 110, 127]
    for budget, impl in ((0.1, 0), (0.3, 0), (0.1, 2), (0.3, 3)):
        order, count = run_kap(q, k2, budget, 8, impl=impl)
        ref_order, ref_count = O.kap_select(qf, kf2, s=8, budget=budget, order_stride=order.shape[-1], query_blocks=blocks)
        for i in blocks:
            assert np.array_equal(_np(count)[:, i], ref_count[:, i]), (budget, i)
            assert np.array_equal(_np(order)[:, i], ref_order[:, i]), (budget, i)


def _scaled_bits(bits, factor, outliers=(), outlier_factor=1.0):
    """bf16 bit patterns times a power of two, a few channels times another one: exact in bf16."""
    x = bf16_bits_to_f64(bits) * factor
    for c in outliers:
        x[..., c] *= outlier_factor
    u = x.astype(np.float32).view(np.uint32)
    assert ((u & 0xffff) == 0).all()                      # still exactly representable
    return (u >> 16).astype(np.uint16)


@pytest.mark.parametrize("factor,outlier_factor", [(4.0, 1.0), (4.0, 8.0), (16.0, 4.0)])
def test_kap_inputs_of_large_magnitude(factor, outlier_factor):
    """Activations far larger than the benchmark's, with a few outlier channels (Sec. 4.2 is silent on magnitudes): the
    rounding error of the float32 screen grows with |q| |k|, and the thresholds below which its verdicts are
    re-examined in double precision grow with it, so the lists stay those of exact arithmetic."""
    w = tiny(seed=77, hq=4, hkv=2, n=2048, needles=3)
    qb, kb, _, _ = w.make()
    qs = _scaled_bits(qb, factor, outliers=(3, 64, 101), outlier_factor=outlier_factor)
    ks = _scaled_bits(kb, factor, outliers=(3, 64, 101), outlier_factor=outlier_factor)
    q, k = to_dev(qs), to_dev(ks)
    qf, kf = widen(qs, ks)
    nqb = w.n // 128
    ref_order, ref_count = O.kap_select(qf, kf, s=8, budget=0.4, order_stride=nqb)
    for impl in (0, 1):
        order, count = run_kap(q, k, 0.4, impl=impl)
        assert np.array_equal(_np(count), ref_count), impl
        assert np.array_equal(_np(order), ref_order), impl


@pytest.mark.parametrize("stride", [4, 8, 16])
@pytest.mark.parametrize("hq,hkv", [(8, 1), (16, 2), (2, 2)])
def test_kap_query_group_sizes(hq, hkv, stride):
    """Query groups of 8 and 1 heads per KV head (the screen's CTA holds 256 sampled rows however they split
    into heads and query blocks); combinations the screen does not take fall to the double-precision kernel."""
    w = tiny(seed=41, hq=hq, hkv=hkv, n=2048, needles=2)
    qb, kb, vb, _ = w.make()
    q, k = to_dev(qb), to_dev(kb)
    qf, kf, _ = widen(qb, kb, vb)
    order, count = run_kap(q, k, 0.4, stride)
    ref_order, ref_count = O.kap_select(qf, kf, s=stride, budget=0.4, order_stride=order.shape[-1])
    assert np.array_equal(_np(count), ref_count)
    assert np.array_equal(_np(order), ref_order)


# ---------------------------------------------------------------------------------- OSK
@pytest.mark.parametrize("impl", OSK_IMPLS)
def test_osk_dense_path_matches_dense_attention(small, impl):
    """Full lists, Stage 2 off: the library's dense path (Property 2, Eq. 4)."""
    q, k, v = small["dev"]
    qf, kf, vf = small["f64"]
    rng = np.random.default_rng(0)
    ref_o, ref_l = O.dense_attention(qf, kf, vf)
    for permute in (False, True):
        order_np = np.full((4, 8, 8), -1, np.int32)
        count_np = np.zeros((4, 8), np.int32)
        for h in range(4):
            for i in range(8):
                ids = rng.permutation(i + 1) if permute else np.arange(i + 1)
                order_np[h, i, :i + 1], count_np[h, i] = ids, i + 1
        order = torch.from_numpy(order_np).cuda()[None].contiguous()
        count = torch.from_numpy(count_np).cuda()[None].contiguous()
        bufs = run_osk(q, k, v, order, count, 1.0, 2000.0, impl)
        err = np.abs(_np(bufs["out"].float()) - ref_o)
        assert err.max() < OUT_MAX and err.mean() < OUT_MEAN
        assert np.abs(_np(bufs["lse"]) - ref_l).max() < LSE_TOL
        assert np.array_equal(_np(bufs["visited"]), count_np) and np.array_equal(_np(bufs["scored"]), count_np)


@pytest.mark.parametrize("impl", OSK_IMPLS)
@pytest.mark.parametrize("tb,skip_scale", [(0.3, 200.0), (0.999, 100.0), (0.2, -1.0), (1.0, 200.0), (0.05, 500.0)])
def test_osk_skip_rule_and_cap_small(small, impl, tb, skip_scale):
    q, k, v = small["dev"]
    qf, kf, vf = small["f64"]
    order_np, count_np = O.kap_select(qf, kf, s=8, budget=0.75)
    order = torch.from_numpy(order_np).cuda()[None].contiguous()
    count = torch.from_numpy(count_np).cuda()[None].contiguous()
    bufs = run_osk(q, k, v, order, count, tb, skip_scale, impl)
    check_osk_against_oracle(qf, kf, vf, order_np, count_np, bufs, tb, skip_scale, range(4), range(8))


@pytest.mark.parametrize("impl", OSK_IMPLS)
def test_osk_4k_workload(cfg1, impl):
    w = cfg1["w"]
    q, k, v = cfg1["dev"]
    qf, kf, vf = cfg1["f64"]
    order, count = run_kap(q, k, w.kap_budget, w.stride)
    bufs = run_osk(q, k, v, order, count, w.osk_budget, w.skip_scale, impl)
    stats = check_osk_against_oracle(qf, kf, vf, _np(order), _np(count), bufs, w.osk_budget, w.skip_scale,
                                     range(w.hq), range(w.n_blocks))
    assert int(_np(bufs["visited"]).sum()) < int(_np(count).sum())        # Stage 2 removed something
    print("4k", stats)


@pytest.mark.parametrize("impl", OSK_IMPLS)
def test_osk_noncausal(small, impl):
    q, k, v = small["dev"]
    qf, kf, vf = small["f64"]
    order_np, count_np = O.kap_select(qf, kf, s=8, budget=0.6, causal=False)
    order = torch.from_numpy(order_np).cuda()[None].contiguous()
    count = torch.from_numpy(count_np).cuda()[None].contiguous()
    bufs = run_osk(q, k, v, order, count, 0.5, 300.0, impl, causal=False)
    check_osk_against_oracle(qf, kf, vf, order_np, count_np, bufs, 0.5, 300.0, range(4), range(8), causal=False)


# ---------------------------------------------------------------------------------- list tools, logical-mask walk
def test_list_tools_bit_exact(small, cfg1):
    for fx, budget in ((small, 0.6), (cfg1, 0.45)):
        q, k, _ = fx["dev"]
        order, count = run_kap(q, k, budget)
        order_np, count_np = _np(order), _np(count)
        shape = cosa.make_shape(q, k, True)
        nqb = q.shape[2] // 128
        mask = torch.full((1, q.shape[1], nqb, (nqb + 31) // 32), -1, dtype=torch.int32, device="cuda")
        cosa.cosa_lists_to_mask(order, count, shape, mask)
        assert np.array_equal(_np(mask).view(np.uint32), O.lists_to_mask(order_np, count_np, nqb))
        for desc in (False, True):
            o2 = order.clone()
            cosa.cosa_reorder_lists(o2, count, shape, descending=desc)
            assert np.array_equal(_np(o2), O.lists_reordered(order_np, count_np, descending=desc))
    # a list of one, and lists longer than one sorting pass of a warp
    o3 = torch.tensor([[[[5, -1, -1, -1], [3, 1, 2, 0]]]], dtype=torch.int32, device="cuda").expand(1, 1, 2, 4).contiguous()
    c3 = torch.tensor([[[1, 4]]], dtype=torch.int32, device="cuda")
    sh = cosa.CosaShape(1, 1, 1, 256, 128, 128, 128, 0)
    cosa.cosa_reorder_lists(o3, c3, sh)
    assert _np(o3).tolist() == [[[5, -1, -1, -1], [0, 1, 2, 3]]]


@pytest.mark.parametrize("impl", OSK_IMPLS)
@pytest.mark.parametrize("tb,skip_scale", [(1.0, 200.0), (0.4, 150.0)])
def test_osk_logical_mask_walk(small, cfg1, impl, tb, skip_scale):
    """Walking the binary mask visits the kept blocks in ascending order: same decisions and outputs as the
    ascending lists (bit for bit on the GPU, within tolerance against the oracle)."""
    for fx, budget in ((small, 0.6), (cfg1, 0.45)):
        q, k, v = fx["dev"]
        qf, kf, vf = fx["f64"]
        nqb = q.shape[2] // 128
        order, count = run_kap(q, k, budget)
        shape = cosa.make_shape(q, k, True)
        mask = torch.zeros(1, q.shape[1], nqb, (nqb + 31) // 32, dtype=torch.int32, device="cuda")
        cosa.cosa_lists_to_mask(order, count, shape, mask)
        mask[0, :, 0, -1] |= 1 << 30                                      # a non-candidate bit must be ignored
        bufs = alloc_outputs(q, nqb)
        opt = cosa.default_options(skip_scale=skip_scale, impl=impl, out_scored=bufs["scored"],
                                   out_decisions=bufs["decisions"], logical_mask=mask, order_stride=nqb)
        cosa.cosa_osk_attention(q, k, v, None, None, tb, bufs["out"], bufs["lse"], bufs["visited"], opt=opt)
        assert cosa.cosa_device_status() == 0
        ref_order, ref_count = O.mask_to_lists(_np(mask).view(np.uint32), nqb, order_stride=nqb)
        heads = range(q.shape[1]) if fx is small else [0, q.shape[1] - 1]
        blocks = range(nqb) if fx is small else [0, 1, 7, 30, 31]
        check_osk_against_oracle(qf, kf, vf, ref_order, ref_count, bufs, tb, skip_scale, heads, blocks)
        asc = torch.from_numpy(ref_order).cuda()[None].contiguous()
        cnt = torch.from_numpy(ref_count).cuda()[None].contiguous()
        ref = run_osk(q, k, v, asc, cnt, tb, skip_scale, impl)
        assert torch.equal(ref["out"], bufs["out"]) and torch.equal(ref["visited"], bufs["visited"])
        assert torch.equal(ref["scored"], bufs["scored"]) and torch.equal(ref["lse"], bufs["lse"])


def test_ablation_tables_run_and_show_the_effect_of_order():
    from paper_2607_25291_b200 import ablation
    w = WORKLOADS["gqa4_4k"]
    rows = ablation.remap_table(w, budgets=(1.0, 0.5), deltas=(200.0, 800.0, 3000.0))
    assert len(rows) == 6
    for r in rows:
        assert 0.0 <= r["skip_natural"] <= 1.0 and 0.0 <= r["skip_remap"] <= 1.0
        assert np.isfinite(r["err_remap"]) and np.isfinite(r["err_natural"])
    # visiting the HRM blocks first lets more of the rest fall below the threshold (Sec. 5.3)
    assert sum(r["skip_remap"] for r in rows) > sum(r["skip_natural"] for r in rows)
    # a larger Delta skips more, in either order
    for b in (1.0, 0.5):
        sel = [r for r in rows if r["stage1"] == b]
        assert sel[0]["skip_remap"] <= sel[1]["skip_remap"] <= sel[2]["skip_remap"]
        assert sel[0]["skip_natural"] <= sel[1]["skip_natural"] <= sel[2]["skip_natural"]
    micro = ablation.micro_table([w], budgets=(0.5,), with_sdpa=False)
    assert len(micro) == 1 and micro[0]["jump_ms"] > 0 and micro[0]["logical_ms"] > 0 and micro[0]["dense_ms"] > 0


# ---------------------------------------------------------------------------------- block_q = 256 variant
@pytest.mark.parametrize("impl", IMPLS)
@pytest.mark.parametrize("budget", [0.3, 0.6, 1.0])
def test_kap_wide_query_blocks_small(small, impl, budget):
    q, k, v = small["dev"]
    qf, kf, vf = small["f64"]
    nqb = q.shape[2] // 128
    for stride in (8, 16):
        order, count = alloc_lists(q.shape[1], nqb)
        cosa.cosa_kap_select(q, k, budget, order, count, opt=cosa.default_options(stride=stride, impl=impl), block_q=256)
        assert cosa.cosa_device_status() == 0
        ref_order, ref_count = O.kap_select_wide(qf, kf, s=stride, budget=budget, order_stride=nqb)
        assert np.array_equal(_np(count), ref_count) and np.array_equal(_np(order), ref_order)
    # the per-tile lists are ordinary lists: OSK runs on them unchanged
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    cosa.cosa_validate_order(order, count, cosa.make_shape(q, k, True), status)
    assert int(status.item()) == 0
    bufs = run_osk(q, k, v, order, count, 0.4, 150.0, impl)
    check_osk_against_oracle(qf, kf, vf, ref_order, ref_count, bufs, 0.4, 150.0, range(q.shape[1]), range(nqb))


@pytest.mark.parametrize("impl", IMPLS)
def test_kap_wide_query_blocks_noncausal_and_top_p(small, impl):
    q, k, _ = small["dev"]
    qf, kf, _ = small["f64"]
    nqb = q.shape[2] // 128
    order, count = alloc_lists(q.shape[1], nqb)
    cosa.cosa_kap_select(q, k, 0.5, order, count, causal=False, opt=cosa.default_options(impl=impl), block_q=256)
    ref_order, ref_count = O.kap_select_wide(qf, kf, s=8, budget=0.5, causal=False, order_stride=nqb)
    assert np.array_equal(_np(count), ref_count) and np.array_equal(_np(order), ref_order)
    assert (ref_count[:, 0::2] == ref_count[:, 1::2]).all()          # nothing lies after a tile: both lists are the ranking
    # Top-p on the summed scores: p = 1 keeps every candidate, a vanishing p the first entry
    cosa.cosa_kap_select(q, k, 1.0, order, count, opt=cosa.default_options(impl=impl, top_p=1.0), block_q=256)
    ref_order, ref_count = O.kap_select_wide(qf, kf, s=8, budget=1.0, order_stride=nqb, top_p=1.0)
    assert np.array_equal(_np(count), ref_count) and np.array_equal(_np(order), ref_order)
    cosa.cosa_kap_select(q, k, 1.0, order, count, opt=cosa.default_options(impl=impl, top_p=1e-9), block_q=256)
    c = _np(count)
    assert (c[:, 1::2] == 1).all() and (c[:, 0::2] <= 1).all()
    # shapes the variant cannot take
    with pytest.raises(cosa.CosaError):
        cosa.cosa_kap_select(q[:, :, :896].contiguous(), k[:, :, :896].contiguous(), 0.5, order, count, block_q=256,
                             opt=cosa.default_options())


@pytest.mark.parametrize("impl", IMPLS)
def test_kap_wide_query_blocks_4k(cfg1, impl):
    w = cfg1["w"]
    q, k, _ = cfg1["dev"]
    qf, kf, _ = cfg1["f64"]
    order, count = alloc_lists(w.hq, w.n_blocks)
    cosa.cosa_kap_select(q, k, w.kap_budget, order, count, opt=cosa.default_options(stride=w.stride, impl=impl, top_p=0.0),
                         block_q=256)
    ref_order, ref_count = O.kap_select_wide(qf, kf, s=w.stride, budget=w.kap_budget, order_stride=w.n_blocks)
    assert np.array_equal(_np(count), ref_count) and np.array_equal(_np(order), ref_order)
    # both tiles of a block share the ranking: the first tile's list is the second's minus the last key block
    o, c = _np(order), _np(count)
    for h in range(w.hq):
        for big in range(w.n_blocks // 2):
            hi = o[h, 2 * big + 1, :c[h, 2 * big + 1]].tolist()
            assert o[h, 2 * big, :c[h, 2 * big]].tolist() == [j for j in hi if j != 2 * big + 1]


def _wide_lists(q, k, budget, causal=True, stride=8):
    order, count = alloc_lists(q.shape[1], q.shape[2] // 128)
    cosa.cosa_kap_select(q, k, budget, order, count, causal=causal, opt=cosa.default_options(stride=stride), block_q=256)
    assert cosa.cosa_device_status() == 0
    return order, count


@pytest.mark.parametrize("budget,tb,skip_scale", [(0.3, 0.4, 150.0), (0.6, 0.5, 400.0), (1.0, 0.3, 150.0), (0.6, 0.5, -1.0),
                                                  (0.6, 1.0, -1.0), (1.0, 1.0, -1.0)])
def test_osk_two_row_tiles_of_a_wide_block_share_each_fetched_tile(small, budget, tb, skip_scale):
    """impl = 5: one CTA walks the ranking of a 256-row query block once for both of its 128-row tiles (Sec. C.1: the
    skip test stays per 128 rows).  Each tile must come out as if it had walked its own list alone: decisions,
    counters, outputs and LSE against the oracle on every tile, and the same decisions and counters as the
    one-item kernel on the same lists."""
    q, k, v = small["dev"]
    qf, kf, vf = small["f64"]
    nqb = q.shape[2] // 128
    order, count = _wide_lists(q, k, budget)
    bufs = run_osk(q, k, v, order, count, tb, skip_scale, impl=5)
    check_osk_against_oracle(qf, kf, vf, _np(order), _np(count), bufs, tb, skip_scale, range(q.shape[1]), range(nqb))
    one = run_osk(q, k, v, order, count, tb, skip_scale, impl=0)
    for key in ("visited", "scored", "decisions"):
        assert torch.equal(bufs[key], one[key]), key
    assert (bufs["out"].float() - one["out"].float()).abs().max() < OUT_MAX


def test_osk_wide_blocks_noncausal_and_4k(small, cfg1):
    q, k, v = small["dev"]
    qf, kf, vf = small["f64"]
    nqb = q.shape[2] // 128
    order, count = _wide_lists(q, k, 0.5, causal=False)
    bufs = run_osk(q, k, v, order, count, 0.5, 150.0, impl=5, causal=False)
    check_osk_against_oracle(qf, kf, vf, _np(order), _np(count), bufs, 0.5, 150.0, range(q.shape[1]), range(nqb), causal=False)
    w = cfg1["w"]
    q, k, v = cfg1["dev"]
    qf, kf, vf = cfg1["f64"]
    order, count = _wide_lists(q, k, w.kap_budget, stride=w.stride)
    bufs = run_osk(q, k, v, order, count, w.osk_budget, w.skip_scale, impl=5)
    check_osk_against_oracle(qf, kf, vf, _np(order), _np(count), bufs, w.osk_budget, w.skip_scale, range(w.hq),
                             [0, 1, 2, 3, 14, 15, 30, 31])


def test_osk_wide_blocks_refuse_lists_that_are_not_nested(small):
    """The first tile's list must be a subsequence of the second's (what block_q = 256 selection writes); ordinary
    per-tile lists are not, in general, and the kernel reports that instead of walking something else."""
    q, k, v = small["dev"]
    nqb = q.shape[2] // 128
    order, count = alloc_lists(q.shape[1], nqb)
    order.fill_(-1)
    order[..., 0] = 0
    count.fill_(1)
    order[:, :, 1::2, 0] = 1          # second tiles list block 1 only, first tiles block 0 only
    bufs = alloc_outputs(q, nqb)
    cosa.cosa_osk_attention(q, k, v, order, count, 0.5, bufs["out"], bufs["lse"], bufs["visited"],
                            opt=cosa.default_options(skip_scale=150.0, impl=5))
    assert cosa.cosa_device_status() == -6
    assert cosa.cosa_device_status() == 0
    # the same lists nested by hand (block 0 for both) are fine, and masks, lengths and odd block counts are refused up front
    order[..., 0] = 0
    cosa.cosa_osk_attention(q, k, v, order, count, 0.5, bufs["out"], bufs["lse"], bufs["visited"],
                            opt=cosa.default_options(skip_scale=150.0, impl=5))
    assert cosa.cosa_device_status() == 0
    assert int(bufs["visited"].min()) == 1 and int(bufs["visited"].max()) == 1
    with pytest.raises((cosa.CosaError, ValueError)):
        cosa.cosa_osk_attention(q[:, :, :896].contiguous(), k[:, :, :896].contiguous(), v[:, :, :896].contiguous(),
                                order[:, :, :7].contiguous(), count[:, :, :7].contiguous(), 0.5, bufs["out"][:, :, :896].contiguous(),
                                bufs["lse"][:, :, :896].contiguous(), bufs["visited"][:, :, :7].contiguous(),
                                opt=cosa.default_options(skip_scale=150.0, impl=5, order_stride=nqb))


# ---------------------------------------------------------------------------------- paged K/V
def _pools(w, page_size):
    """K and V of the workload as page pools that share one seeded page table."""
    _, kb, vb, _ = w.make()
    kpool, table = scatter_to_pages(kb, page_size, seed=9)
    vpool, table_v = scatter_to_pages(vb, page_size, seed=9)
    assert np.array_equal(table, table_v)
    dev = lambda a: torch.from_numpy(a.view(np.int16)).view(torch.bfloat16).cuda().contiguous()
    return dev(kpool), dev(vpool), torch.from_numpy(table).cuda()[None].contiguous(), kpool.shape[0]


@pytest.mark.parametrize("impl", OSK_IMPLS)
@pytest.mark.parametrize("page_size", [8, 16, 32, 64, 128, 256])
def test_paged_kv_small(small, impl, page_size):
    """Pools + page table give the lists and outputs of the dense tensors behind them (Sec. C.1)."""
    q, k, v = small["dev"]
    qf, kf, vf = small["f64"]
    nqb = q.shape[2] // 128
    kpool, vpool, table, n_pages = _pools(small["w"], page_size)
    for stride in (8, 16):
        paging = dict(kv_page_table=table, kv_page_size=page_size, kv_num_pages=n_pages)
        order, count = alloc_lists(q.shape[1], nqb)
        cosa.cosa_kap_select(q, kpool, 0.6, order, count, opt=cosa.default_options(stride=stride, impl=impl, **paging))
        assert cosa.cosa_device_status() == 0
        ref_order, ref_count = O.kap_select(qf, kf, s=stride, budget=0.6, order_stride=nqb)
        assert np.array_equal(_np(count), ref_count) and np.array_equal(_np(order), ref_order)
    # pages smaller than a block: staged as dense tensors (default), or read in place, tile by tile (no scratch)
    for in_place in ((0, 1) if (impl == 0 and page_size < 128) else (0,)):
        for tb, skip_scale in ((1.0, 200.0), (0.4, 150.0)):
            bufs = alloc_outputs(q, nqb)
            opt = cosa.default_options(skip_scale=skip_scale, impl=impl, out_scored=bufs["scored"],
                                       out_decisions=bufs["decisions"], kv_pages_in_place=in_place, **paging)
            if in_place:
                assert cosa.cosa_workspace_bytes(1, cosa.make_shape(q, k), opt) == 0
            cosa.cosa_osk_attention(q, kpool, vpool, order, count, tb, bufs["out"], bufs["lse"], bufs["visited"], opt=opt)
            assert cosa.cosa_device_status() == 0
            check_osk_against_oracle(qf, kf, vf, ref_order, ref_count, bufs, tb, skip_scale, range(q.shape[1]), range(nqb))
            dense = run_osk(q, k, v, order, count, tb, skip_scale, impl)
            assert torch.equal(dense["out"], bufs["out"]) and torch.equal(dense["visited"], bufs["visited"])
            assert torch.equal(dense["lse"], bufs["lse"])


def test_paged_kv_4k(cfg1):
    w = cfg1["w"]
    q, k, v = cfg1["dev"]
    for page_size in (16, 64, 512):
        kpool, vpool, table, n_pages = _pools(w, page_size)
        paging = dict(kv_page_table=table, kv_page_size=page_size, kv_num_pages=n_pages)
        order, count = alloc_lists(w.hq, w.n_blocks)
        cosa.cosa_kap_select(q, kpool, w.kap_budget, order, count, opt=cosa.default_options(stride=w.stride, **paging))
        d_order, d_count = run_kap(q, k, w.kap_budget, w.stride)
        assert torch.equal(order, d_order) and torch.equal(count, d_count)
        bufs = alloc_outputs(q, w.n_blocks)
        opt = cosa.default_options(skip_scale=w.skip_scale, out_scored=bufs["scored"], out_decisions=bufs["decisions"], **paging)
        cosa.cosa_osk_attention(q, kpool, vpool, order, count, w.osk_budget, bufs["out"], bufs["lse"], bufs["visited"], opt=opt)
        assert cosa.cosa_device_status() == 0
        dense = run_osk(q, k, v, order, count, w.osk_budget, w.skip_scale)
        assert torch.equal(dense["out"], bufs["out"]) and torch.equal(dense["visited"], bufs["visited"])


def test_paged_kv_rejects_bad_arguments(small):
    q, _, _ = small["dev"]
    kpool, vpool, table, n_pages = _pools(small["w"], 64)
    order, count = alloc_lists(q.shape[1], q.shape[2] // 128)
    for bad in (dict(kv_page_size=48), dict(kv_page_size=4), dict(kv_num_pages=3), dict(kv_page_size=4096)):
        args = dict(kv_page_table=table, kv_page_size=64, kv_num_pages=n_pages)
        args.update(bad)
        with pytest.raises(cosa.CosaError):
            cosa.cosa_kap_select(q, kpool, 0.5, order, count, opt=cosa.default_options(**args))



def test_paged_kv_small_pages_with_caller_workspace(small):
    """Pages smaller than a key block are staged as dense tensors in the scratch: a caller-owned workspace of the size
    the library asks for gives the dense results, a smaller one is refused; with kv_pages_in_place OSK needs none."""
    q, k, v = small["dev"]
    nqb = q.shape[2] // 128
    kpool, vpool, table, n_pages = _pools(small["w"], 16)
    paging = dict(kv_page_table=table, kv_page_size=16, kv_num_pages=n_pages)
    shape = cosa.make_shape(q, k)
    kv_bytes = k.numel() * 2
    need = cosa.cosa_workspace_bytes(2, shape, cosa.default_options(**paging))
    assert need >= 2 * kv_bytes
    assert cosa.cosa_workspace_bytes(1, shape, cosa.default_options(**paging)) >= 2 * kv_bytes
    assert cosa.cosa_workspace_bytes(1, shape, cosa.default_options(kv_pages_in_place=1, **paging)) == 0
    assert cosa.cosa_workspace_bytes(1, shape, cosa.default_options()) == 0
    ws = torch.empty(need, dtype=torch.uint8, device="cuda")
    order, count = alloc_lists(q.shape[1], nqb)
    opt = cosa.default_options(workspace=ws, workspace_bytes=need, **paging)
    cosa.cosa_kap_select(q, kpool, 0.6, order, count, opt=opt)
    d_order, d_count = run_kap(q, k, 0.6)
    assert torch.equal(order, d_order) and torch.equal(count, d_count)
    dense = run_osk(q, k, v, order, count, 0.4, 150.0)
    for extra in (dict(workspace=ws, workspace_bytes=need), dict(kv_pages_in_place=1)):
        bufs = alloc_outputs(q, nqb)
        cosa.cosa_osk_attention(q, kpool, vpool, order, count, 0.4, bufs["out"], bufs["lse"], bufs["visited"],
                                opt=cosa.default_options(skip_scale=150.0, **extra, **paging))
        assert cosa.cosa_device_status() == 0
        assert torch.equal(dense["out"], bufs["out"]) and torch.equal(dense["visited"], bufs["visited"])
    small_opt = cosa.default_options(workspace=ws, workspace_bytes=kv_bytes, **paging)
    with pytest.raises(cosa.CosaError):
        cosa.cosa_kap_select(q, kpool, 0.6, order, count, opt=small_opt)
    with pytest.raises(cosa.CosaError):
        cosa.cosa_osk_attention(q, kpool, vpool, order, count, 0.4, bufs["out"], bufs["lse"], bufs["visited"], opt=small_opt)


@pytest.mark.parametrize("impl", OSK_IMPLS)
def test_batch_of_two_equals_single_items(impl):
    """Two different sequences in one call give exactly the results of two calls (dense and paged)."""
    items = []
    for seed in (31, 32):
        w = tiny(seed=seed, hq=4, hkv=2, n=1024, needles=2)
        qb, kb, vb, _ = w.make()
        items.append((w, qb, kb, vb))
    stack = lambda idx: torch.cat([to_dev(it[idx]) for it in items], dim=0).contiguous()
    q2, k2, v2 = stack(1), stack(2), stack(3)
    nqb = 8

    def run(q, k, v, batch, **paging):
        order = torch.full((batch, 4, nqb, nqb), -7, dtype=torch.int32, device="cuda")
        count = torch.full((batch, 4, nqb), -7, dtype=torch.int32, device="cuda")
        out = torch.empty_like(q)
        lse = torch.empty(batch, 4, 1024, dtype=torch.float32, device="cuda")
        vis = torch.empty(batch, 4, nqb, dtype=torch.int32, device="cuda")
        opt = cosa.default_options(impl=impl, skip_scale=200.0, **paging)
        cosa.cosa_kap_select(q, k, 0.6, order, count, opt=opt)
        cosa.cosa_osk_attention(q, k, v, order, count, 0.4, out, lse, vis, opt=opt)
        assert cosa.cosa_device_status() == 0
        return order, count, out, lse, vis

    both = run(q2, k2, v2, 2)
    for b in range(2):
        one = run(q2[b:b + 1].contiguous(), k2[b:b + 1].contiguous(), v2[b:b + 1].contiguous(), 1)
        for x, y in zip(both, one):
            assert torch.equal(x[b:b + 1], y)
    # the same through page pools: both sequences share one pool, each with its own row of the page table
    page_size = 64
    pools, tables = [], []
    for _, _, kb, vb in items:
        kp, tab = scatter_to_pages(kb, page_size, seed=4)
        vp, _ = scatter_to_pages(vb, page_size, seed=4)
        tables.append(tab + sum(p_[0].shape[0] for p_ in pools))
        pools.append((kp, vp))
    dev = lambda a: torch.from_numpy(a.view(np.int16)).view(torch.bfloat16).cuda().contiguous()
    kpool = dev(np.concatenate([p_[0] for p_ in pools])); vpool = dev(np.concatenate([p_[1] for p_ in pools]))
    table = torch.from_numpy(np.stack(tables).astype(np.int32)).cuda().contiguous()
    paged = run(q2, kpool, vpool, 2, kv_page_table=table, kv_page_size=page_size, kv_num_pages=kpool.shape[0])
    for x, y in zip(both, paged):
        assert torch.equal(x, y)


@pytest.mark.parametrize("impl", OSK_IMPLS)
@pytest.mark.parametrize("causal", [True, False])
@pytest.mark.parametrize("n,lens", [(1024, [1024, 640]), (4096, [1536, 4096])])
def test_batch_with_different_lengths(impl, causal, n, lens):
    """Prompts of 1024 and 640 tokens in one call, padded to 1024 (cosa_options.seq_lens): every item gives exactly
    what a call on its unpadded tensors gives -- lists also checked against the oracle -- and the padding gets empty
    lists, zero output, lse = -inf.  The same through page pools whose table rows point at a wrong (but valid) page
    past the length: nothing there may be read.  (At 4096 tokens whole CTAs of the screen kernel lie in the padding.)"""
    items = []
    for seed in (51, 52):
        w = tiny(seed=seed, hq=4, hkv=2, n=n, needles=2)
        qb, kb, vb, _ = w.make()
        items.append((qb, kb, vb))
    stack = lambda idx: torch.cat([to_dev(it[idx]) for it in items], dim=0).contiguous()
    q2, k2, v2 = stack(0), stack(1), stack(2)
    seq_lens = torch.tensor(lens, dtype=torch.int32, device="cuda")

    def run(q, k, v, batch, n_tok, **extra):
        nqb = n_tok // 128
        order = torch.full((batch, 4, nqb, nqb), -7, dtype=torch.int32, device="cuda")
        count = torch.full((batch, 4, nqb), -7, dtype=torch.int32, device="cuda")
        out = torch.full_like(q, 3.0)
        lse = torch.full((batch, 4, n_tok), 3.0, dtype=torch.float32, device="cuda")
        vis = torch.full((batch, 4, nqb), -7, dtype=torch.int32, device="cuda")
        opt = cosa.default_options(impl=impl, skip_scale=200.0, **extra)
        cosa.cosa_kap_select(q, k, 0.6, order, count, causal=causal, opt=opt)
        cosa.cosa_osk_attention(q, k, v, order, count, 0.4, out, lse, vis, causal=causal, opt=opt)
        assert cosa.cosa_device_status() == 0
        return order, count, out, lse, vis

    def check(both):
        order, count, out, lse, vis = both
        for b, ln in enumerate(lens):
            nb = ln // 128
            cut = lambda t: t[b:b + 1, :, :ln].contiguous()
            o1, c1, out1, lse1, vis1 = run(cut(q2), cut(k2), cut(v2), 1, ln)
            assert torch.equal(count[b:b + 1, :, :nb], c1) and torch.equal(vis[b:b + 1, :, :nb], vis1)
            assert torch.equal(order[b:b + 1, :, :nb, :nb], o1) and bool((order[b, :, :nb, nb:] == -1).all())
            assert torch.equal(out[b:b + 1, :, :ln], out1) and torch.equal(lse[b:b + 1, :, :ln], lse1)
            assert bool((count[b, :, nb:] == 0).all()) and bool((order[b, :, nb:] == -1).all())
            assert bool((vis[b, :, nb:] == 0).all()) and bool((out[b, :, ln:] == 0).all())
            assert bool(torch.isinf(lse[b, :, ln:]).all()) and bool((lse[b, :, ln:] < 0).all())
            qf, kf, _ = widen(items[b][0][:, :ln], items[b][1][:, :ln], items[b][2][:, :ln])
            ref_order, ref_count = O.kap_select(qf, kf, s=8, budget=0.6, causal=causal, order_stride=nb)
            assert np.array_equal(count.cpu().numpy()[b, :, :nb], ref_count)
            assert np.array_equal(order.cpu().numpy()[b, :, :nb, :nb], ref_order)

    check(run(q2, k2, v2, 2, n, seq_lens=seq_lens))
    page_size = 64
    pools, tables = [], []
    for (_, kb, vb), ln in zip(items, lens):
        kp, tab = scatter_to_pages(kb, page_size, seed=6)
        vp, _ = scatter_to_pages(vb, page_size, seed=6)
        tab = tab + sum(p_[0].shape[0] for p_ in pools)
        tab[ln // page_size:] = 0                       # past the length: some other sequence's page
        tables.append(tab)
        pools.append((kp, vp))
    dev = lambda a: torch.from_numpy(a.view(np.int16)).view(torch.bfloat16).cuda().contiguous()
    kpool = dev(np.concatenate([p_[0] for p_ in pools])); vpool = dev(np.concatenate([p_[1] for p_ in pools]))
    table = torch.from_numpy(np.stack(tables).astype(np.int32)).cuda().contiguous()
    paged = run(q2, kpool, vpool, 2, n, seq_lens=seq_lens, kv_page_table=table, kv_page_size=page_size,
                kv_num_pages=kpool.shape[0])
    check(paged)


@pytest.mark.parametrize("impl", OSK_IMPLS)
def test_token_major_and_fused_qkv_layouts(cfg1, impl):
    """q, k, v as three views into one token-major buffer [B, N, Hq + 2 Hkv, d] (what a fused QKV projection writes) and
    out as a view of a token-major [B, N, Hq, d] tensor: passed by their strides, no transpose copy, and every
    result equals the dense call's bit for bit."""
    w = cfg1["w"]
    q, k, v = cfg1["dev"]
    nqb = w.n // 128
    dense_order, dense_count = run_kap(q, k, w.kap_budget, w.stride, impl=impl)
    dense = run_osk(q, k, v, dense_order, dense_count, w.osk_budget, w.skip_scale, impl=impl)
    fused = torch.empty(1, w.n, w.hq + 2 * w.hkv, 128, dtype=torch.bfloat16, device="cuda")
    fused[:, :, :w.hq] = q.transpose(1, 2)
    fused[:, :, w.hq:w.hq + w.hkv] = k.transpose(1, 2)
    fused[:, :, w.hq + w.hkv:] = v.transpose(1, 2)
    qv = fused[:, :, :w.hq].transpose(1, 2)                   # [B, Hq, N, d] views with token-major strides
    kv_ = fused[:, :, w.hq:w.hq + w.hkv].transpose(1, 2)
    vv = fused[:, :, w.hq + w.hkv:].transpose(1, 2)
    assert not qv.is_contiguous() and qv.stride(2) == (w.hq + 2 * w.hkv) * 128 and qv.stride(1) == 128
    order, count = alloc_lists(w.hq, nqb)
    cosa.cosa_kap_select(qv, kv_, w.kap_budget, order, count, opt=cosa.default_options(stride=w.stride, impl=impl))
    assert cosa.cosa_device_status() == 0
    assert torch.equal(order, dense_order) and torch.equal(count, dense_count)
    out_tm = torch.zeros(1, w.n, w.hq, 128, dtype=torch.bfloat16, device="cuda")
    bufs = alloc_outputs(q, nqb)
    opt = cosa.default_options(skip_scale=w.skip_scale, impl=impl, out_scored=bufs["scored"], out_decisions=bufs["decisions"])
    cosa.cosa_osk_attention(qv, kv_, vv, order, count, w.osk_budget, out_tm.transpose(1, 2), bufs["lse"], bufs["visited"], opt=opt)
    assert cosa.cosa_device_status() == 0
    assert torch.equal(out_tm.transpose(1, 2), dense["out"])
    for key in ("lse", "visited", "scored", "decisions"):
        assert torch.equal(bufs[key], dense[key]), key
    # strides that cannot be mapped are refused, and so are strides together with page pools
    bad = cosa.default_options()
    bad.q_strides = (ctypes.c_int64 * 3)(w.hq * w.n * 128, w.n * 128, 100)
    with pytest.raises(cosa.CosaError) as e:      # (the binding sets strides itself: this goes through the raw call)
        shape = cosa.make_shape(q, k, True)
        rc = cosa.library().cosa_kap_select_ex(q.data_ptr(), k.data_ptr(), ctypes.byref(shape), ctypes.c_float(0.25),
                                               order.data_ptr(), count.data_ptr(), None, ctypes.byref(bad))
        if rc != 0:
            raise cosa.CosaError(rc, "cosa_kap_select_ex")
    assert e.value.status == -1


def test_kv_head_shards_concatenate_to_the_unsharded_result(small):
    """One layer split by KV-head group (what bench.py --shard kv_head gives each rank): every shard runs KAP + OSK on
    its heads alone, here one after the other on one GPU, and the concatenated lists and outputs are those of the
    unsharded call, bit for bit (work items of different KV heads share nothing)."""
    from paper_2607_25291_b200.shard import shard_tensors
    w = small["w"]
    q, k, v = small["dev"]
    whole_order, whole_count = run_kap(q, k, 0.5)
    whole = run_osk(q, k, v, whole_order, whole_count, 0.3, 200.0)
    for world in (2,):
        parts = []
        for rank in range(world):
            qs, ks, vs = (t.contiguous() for t in shard_tensors(q, k, v, world, rank))
            order, count = run_kap(qs, ks, 0.5)
            parts.append((order, count, run_osk(qs, ks, vs, order, count, 0.3, 200.0)))
        assert torch.equal(torch.cat([p[0] for p in parts], 1), whole_order)
        assert torch.equal(torch.cat([p[1] for p in parts], 1), whole_count)
        for key in ("out", "lse", "visited", "scored"):
            assert torch.equal(torch.cat([p[2][key] for p in parts], 1), whole[key]), key


def test_reserved_scratch_makes_plain_calls_allocation_free(cfg1):
    """cosa_reserve_scratch sizes the library's own scratch ahead of time: the plain calls that follow allocate
    nothing (the free memory of the device does not move)."""
    w = cfg1["w"]
    q, k, v = cfg1["dev"]
    nqb = w.n // 128
    cosa.cosa_reserve_scratch(cosa.cosa_workspace_bytes(2, cosa.make_shape(q, k)))
    order, count = alloc_lists(w.hq, nqb)
    bufs = alloc_outputs(q, nqb)
    def both():
        cosa.cosa_kap_select(q, k, w.kap_budget, order, count)
        cosa.cosa_osk_attention(q, k, v, order, count, w.osk_budget, bufs["out"], bufs["lse"], bufs["visited"])
        torch.cuda.synchronize()
    both()                                               # (first use loads the kernels' code)
    free = torch.cuda.mem_get_info()[0]
    both()
    assert torch.cuda.mem_get_info()[0] == free
    assert cosa.cosa_device_status() == 0


def test_osk_is_deterministic(cfg1):
    w = cfg1["w"]
    q, k, v = cfg1["dev"]
    order, count = run_kap(q, k, w.kap_budget, w.stride)
    a = run_osk(q, k, v, order, count, w.osk_budget, w.skip_scale)
    b = run_osk(q, k, v, order, count, w.osk_budget, w.skip_scale)
    assert torch.equal(a["out"], b["out"]) and torch.equal(a["lse"], b["lse"]) and torch.equal(a["visited"], b["visited"])


# ---------------------------------------------------------------------------------- boundary
def test_validator_flags_bad_lists(small):
    q, k, _ = small["dev"]
    shape = cosa.make_shape(q, k, True)
    order, count = run_kap(q, k, 0.5, 8)
    status = torch.full((1,), 5, dtype=torch.int32, device="cuda")
    cosa.cosa_validate_order(order, count, shape, status)
    assert int(status.item()) == 0
    bad = order.clone()
    bad[0, 1, 3, 0] = 4                               # key block 4 > query block 3 under a causal mask
    cosa.cosa_validate_order(bad, count, shape, status)
    assert int(status.item()) == -6
    badc = count.clone()
    badc[0, 0, 0] = 0
    cosa.cosa_validate_order(order, badc, shape, status)
    assert int(status.item()) == -6


def test_host_call_equals_device_calls(small):
    w = small["w"]
    q, k, v = small["dev"]
    order, count = run_kap(q, k, 0.5, 8)
    ref = run_osk(q, k, v, order, count, 0.3, 200.0)
    shape = cosa.make_shape(q, k, True)
    opt = cosa.default_options(skip_scale=200.0)
    ws = torch.empty(cosa.cosa_host_call_workspace_bytes(shape, opt), dtype=torch.uint8, device="cuda")
    qh, kh, vh = (t.cpu().pin_memory() for t in (q, k, v))
    out_h = torch.empty(q.shape, dtype=torch.bfloat16).pin_memory()
    lse_h = torch.empty(ref["lse"].shape, dtype=torch.float32).pin_memory()
    vis_h = torch.empty(ref["visited"].shape, dtype=torch.int32).pin_memory()
    cosa.cosa_prefill_host(qh, kh, vh, shape, 0.5, 0.3, out_h, lse_h, vis_h, ws, opt=opt)
    assert cosa.cosa_device_status() == 0
    assert torch.equal(out_h, ref["out"].cpu()) and torch.equal(lse_h, ref["lse"].cpu())
    assert torch.equal(vis_h, ref["visited"].cpu())
    small_ws = torch.empty(1024, dtype=torch.uint8, device="cuda")
    with pytest.raises(cosa.CosaError) as e:
        cosa.cosa_prefill_host(qh, kh, vh, shape, 0.5, 0.3, out_h, lse_h, vis_h, small_ws, opt=opt)
    assert e.value.status == -3


def test_host_call_with_different_lengths():
    """cosa_prefill_host on a padded batch with per-item lengths gives the device calls' results."""
    n, lens, hq, hkv = 1024, [640, 1024], 4, 2
    items = [tiny(seed=71 + b, hq=hq, hkv=hkv, n=n, needles=2).make() for b in range(2)]
    q = torch.stack([to_dev(it[0])[0] for it in items]).contiguous()
    k = torch.stack([to_dev(it[1])[0] for it in items]).contiguous()
    v = torch.stack([to_dev(it[2])[0] for it in items]).contiguous()
    nqb = n // 128
    seq_lens = torch.tensor(lens, dtype=torch.int32, device="cuda")
    order = torch.empty(2, hq, nqb, nqb, dtype=torch.int32, device="cuda")
    count = torch.empty(2, hq, nqb, dtype=torch.int32, device="cuda")
    out = torch.empty_like(q)
    lse = torch.empty(2, hq, n, dtype=torch.float32, device="cuda")
    vis = torch.empty(2, hq, nqb, dtype=torch.int32, device="cuda")
    opt = cosa.default_options(skip_scale=100.0, seq_lens=seq_lens)
    cosa.cosa_kap_select(q, k, 0.5, order, count, opt=opt)
    cosa.cosa_osk_attention(q, k, v, order, count, 0.3, out, lse, vis, opt=opt)
    assert cosa.cosa_device_status() == 0
    shape = cosa.make_shape(q, k, True)
    ws = torch.empty(cosa.cosa_host_call_workspace_bytes(shape, opt), dtype=torch.uint8, device="cuda")
    qh, kh, vh = (t.cpu().pin_memory() for t in (q, k, v))
    out_h = torch.empty(q.shape, dtype=torch.bfloat16).pin_memory()
    lse_h = torch.empty(lse.shape, dtype=torch.float32).pin_memory()
    vis_h = torch.empty(vis.shape, dtype=torch.int32).pin_memory()
    cosa.cosa_prefill_host(qh, kh, vh, shape, 0.5, 0.3, out_h, lse_h, vis_h, ws, opt=opt)
    assert cosa.cosa_device_status() == 0
    assert torch.equal(vis_h, vis.cpu()) and torch.equal(out_h, out.cpu())
    assert torch.equal(lse_h[0, :, :lens[0]], lse.cpu()[0, :, :lens[0]]) and torch.equal(lse_h[1], lse.cpu()[1])
    assert bool((out_h[0, :, lens[0]:] == 0).all()) and bool((vis_h[0, :, lens[0] // 128:] == 0).all())
