"""Pins of the fp64 oracle against things other than itself: library routines,
closed forms, brute force on tiny inputs, and the invariants the paper states
(order invariance, Eq. 4; the skip rule, Eq. 5; the HRM-first ordering, Eq. 13)."""
import math
from fractions import Fraction

import numpy as np
import pytest
import torch

from oracle import cosa_oracle as O
from synth.configs import tiny
from synth.generator import bf16_bits_to_f64


def _inputs(seed=7, hq=2, hkv=1, n=1024, needles=2):
    q, k, v, planted = tiny(seed, hq, hkv, n, needles).make()
    return bf16_bits_to_f64(q), bf16_bits_to_f64(k), bf16_bits_to_f64(v), planted


@pytest.fixture(scope="module")
def small():
    return _inputs()


# ---------------------------------------------------------------- dense / masked
def test_dense_matches_library_sdpa(small):
    q, k, v, _ = small
    out, lse = O.dense_attention(q, k, v, causal=True)
    tq, tk, tv = (torch.from_numpy(x) for x in (q, k, v))
    ref = torch.nn.functional.scaled_dot_product_attention(
        tq[None], tk[None].repeat_interleave(2, dim=1), tv[None].repeat_interleave(2, dim=1), is_causal=True)[0]
    assert np.abs(out - ref.numpy()).max() < 1e-12
    # lse against a library logsumexp
    logits = torch.einsum("hqd,hkd->hqk", tq, tk.repeat_interleave(2, dim=0)) / math.sqrt(q.shape[2])
    mask = torch.ones(q.shape[1], q.shape[1], dtype=torch.bool).tril()
    ref_lse = torch.logsumexp(logits.masked_fill(~mask, -float("inf")), dim=-1)
    assert np.abs(lse - ref_lse.numpy()).max() < 1e-12


def test_dense_noncausal_matches_library(small):
    q, k, v, _ = small
    out, _ = O.dense_attention(q, k, v, causal=False, query_blocks=[0, 3])
    tq, tk, tv = (torch.from_numpy(x) for x in (q, k, v))
    ref = torch.nn.functional.scaled_dot_product_attention(tq[:1, None][:, 0][None], tk[None], tv[None])[0, 0]
    rows = np.r_[0:128, 384:512]
    assert np.abs(out[0] - ref.numpy()[rows]).max() < 1e-12


def test_dense_closed_forms(small):
    q, k, v, _ = small
    out, lse, probs = O.dense_attention(q, k, v, query_blocks=[0, 5], return_probs=True)
    for p in probs:                                      # rows of probabilities sum to one
        assert np.abs(p.sum(axis=1) - 1).max() < 1e-12
    assert np.allclose(out[:, 0], v[0, 0], atol=0, rtol=0)   # the first token sees only key 0
    vc = np.broadcast_to(np.linspace(-1, 1, v.shape[2]), v.shape).copy()
    outc, _ = O.dense_attention(q, k, vc, query_blocks=[2])
    assert np.abs(outc - vc[0, :128]).max() < 1e-12      # constant V rows come back unchanged


def test_masked_reduces_to_dense(small):
    q, k, v, _ = small
    qbs = [0, 3, 7]
    sets = [[list(range(i + 1)) for i in qbs] for _ in range(q.shape[0])]
    mo, ml = O.masked_attention(q, k, v, sets, query_blocks=qbs)
    do, dl = O.dense_attention(q, k, v, query_blocks=qbs)
    assert np.abs(mo - do).max() < 1e-12 and np.abs(ml - dl).max() < 1e-12
    # a strict prefix of key blocks = non-causal dense attention on physically truncated K/V
    sets = [[[0, 1, 2]] for _ in range(q.shape[0])]
    mo, ml = O.masked_attention(q, k, v, sets, query_blocks=[6])
    do6, dl6 = O.dense_attention(np.ascontiguousarray(q[:, 768:896]), k[:, :384], v[:, :384], causal=False,
                                 query_blocks=[0])
    assert np.abs(mo - do6).max() < 1e-12 and np.abs(ml - dl6).max() < 1e-12


# ---------------------------------------------------------------- OSK, skipping off
def _full_lists(hq, nqb, rng=None):
    order = np.full((hq, nqb, nqb), -1, np.int32)
    count = np.zeros((hq, nqb), np.int32)
    for h in range(hq):
        for i in range(nqb):
            ids = np.arange(i + 1)
            if rng is not None:
                ids = rng.permutation(ids)
            order[h, i, :i + 1] = ids
            count[h, i] = i + 1
    return order, count


def test_full_budget_osk_is_dense_in_any_order(small):
    """Property 2 (Eq. 4): with every block listed and Stage 2 off the result is dense attention."""
    q, k, v, _ = small
    do, dl = O.dense_attention(q, k, v)
    for rng in (None, np.random.default_rng(1), np.random.default_rng(2)):
        order, count = _full_lists(q.shape[0], 8, rng)
        r = O.osk_attention(q, k, v, order, count, skip_scale=2000.0, tightened_budget=1.0)
        assert np.abs(r["out"] - do).max() < 1e-12 and np.abs(r["lse"] - dl).max() < 1e-12
        assert (r["visited"] == count).all() and (r["scored"] == count).all()
        r2 = O.osk_attention(q, k, v, order, count, skip_scale=-1.0, tightened_budget=1.0)
        assert np.abs(r2["out"] - do).max() < 1e-12


def test_ordered_traversal_of_a_mask_is_masked_attention(small):
    q, k, v, _ = small
    rng = np.random.default_rng(3)
    hq, nqb = q.shape[0], 8
    order = np.full((hq, nqb, nqb), -1, np.int32)
    count = np.zeros((hq, nqb), np.int32)
    sets = [[None] * nqb for _ in range(hq)]
    for h in range(hq):
        for i in range(nqb):
            c = int(rng.integers(1, i + 2))
            ids = rng.choice(i + 1, size=c, replace=False)
            order[h, i, :c], count[h, i], sets[h][i] = ids, c, ids
    r = O.osk_attention(q, k, v, order, count, tightened_budget=1.0)
    mo, ml = O.masked_attention(q, k, v, sets)
    assert np.abs(r["out"] - mo).max() < 1e-12 and np.abs(r["lse"] - ml).max() < 1e-12


# ---------------------------------------------------------------- OSK, skip rule
def _two_block_case(a, b, veto_row=None, block=4, d=4):
    """Key block A has every logit a, key block B every logit b (non-causal, one head)."""
    q = np.zeros((1, block, d)); q[0, :, 0] = math.sqrt(d)
    if veto_row is not None:
        q[0, veto_row, 0] = -math.sqrt(d)           # on this row block B lies ABOVE block A
    k = np.zeros((1, 2 * block, d)); k[0, :block, 0] = a; k[0, block:, 0] = b
    v = np.zeros((1, 2 * block, d)); v[0, :block] = 1.0; v[0, block:] = -2.0
    return q, k, v


def _run_two(q, k, v, first, delta, n_for_theta):
    # N of the call is 2*block; choose delta so that ln(delta/N) = theta
    order = np.array([[[first, 1 - first]]], np.int32)
    count = np.array([[2]], np.int32)
    return O.osk_attention(q, k, v, order, count, skip_scale=delta, tightened_budget=0.999999,
                           causal=False, block=q.shape[1])


def test_skip_rule_depends_on_order_running_max():
    """Limitation 2.1: the test is against the RUNNING maximum, so (A,B) can skip B but (B,A) skips nothing."""
    a, b = 3.0, 0.5
    q, k, v = _two_block_case(a, b)
    n = k.shape[1]
    theta = -1.0                                     # b - a = -2.5 < theta  -> B negligible after A
    delta = n * math.exp(theta)
    r = _run_two(q, k, v, 0, delta, n)
    assert r["decisions"][(0, 0)] == [True, False] and r["visited"][0, 0] == 1
    assert np.allclose(r["out"], 1.0, atol=1e-15)                       # only A's values
    assert np.allclose(r["lse"], a + math.log(4), atol=1e-14)
    assert np.allclose(r["gaps"][(0, 0)], [0.0, b - a], atol=1e-15)
    r = _run_two(q, k, v, 1, delta, n)               # B first: both raise the running max
    assert r["decisions"][(0, 0)] == [True, True]
    w = math.exp(b) / (math.exp(a) + math.exp(b))
    assert np.allclose(r["out"], (1 - w) * 1.0 + w * -2.0, atol=1e-14)
    # a milder threshold keeps B even after A (b - a >= theta)
    r = _run_two(q, k, v, 0, n * math.exp(-3.0), n)
    assert r["decisions"][(0, 0)] == [True, True]
    assert np.allclose(r["out"], (1 - w) * 1.0 + w * -2.0, atol=1e-14)
    # boundary: equality is NOT a skip (strict inequality in Eq. 5)
    r = _run_two(q, k, v, 0, n * math.exp(-2.5), n)
    gap = r["gaps"][(0, 0)][1]
    assert r["decisions"][(0, 0)][1] == (not gap < math.log(n * math.exp(-2.5) / n))


def test_skip_rule_single_row_veto():
    """Limitation 2.2 (bucket effect): one row on which B is not negligible vetoes the skip."""
    q, k, v = _two_block_case(3.0, 0.5, veto_row=2)
    n = k.shape[1]
    r = _run_two(q, k, v, 0, n * math.exp(-1.0), n)
    assert r["decisions"][(0, 0)] == [True, True]
    assert r["gaps"][(0, 0)][1] == 0.0               # B raised the maximum of the veto row


@pytest.fixture(scope="module")
def kap_lists(small):
    q, k, v, _ = small
    return O.kap_select(q, k, s=8, budget=1.0)


def test_online_and_offline_gaps_agree_and_sets_are_nested(small, kap_lists):
    q, k, v, _ = small
    order, count = kap_lists
    n = q.shape[1]
    prev_sets = None
    for delta in (1e-9, 50.0, 200.0, 600.0):
        r = O.osk_attention(q, k, v, order, count, skip_scale=delta, tightened_budget=0.999999)
        theta = math.log(delta / n)
        sets = {}
        for (h, i), dec in r["decisions"].items():
            off = O.osk_gaps_offline(q, k, order, count, h, i)
            assert np.array_equal(np.asarray(r["gaps"][(h, i)]), off)
            assert dec == [not g < theta for g in off]
            assert dec[0]                                   # the first listed block is always computed
            sets[(h, i)] = {int(order[h, i, kk]) for kk, c in enumerate(dec) if c}
        if delta == 1e-9:
            assert all(len(s) == count[h, i] for (h, i), s in sets.items())   # Delta -> 0+ skips nothing
        if prev_sets is not None:                           # larger Delta -> subset
            assert all(sets[key] <= prev_sets[key] for key in sets)
        prev_sets = sets
        # the output is masked attention over the computed set
        bs = [[sorted(sets[(h, i)]) for i in range(n // 128)] for h in range(q.shape[0])]
        mo, ml = O.masked_attention(q, k, v, bs)
        assert np.abs(r["out"] - mo).max() < 1e-12 and np.abs(r["lse"] - ml).max() < 1e-12
    assert any(len(s) < count[h, i] for (h, i), s in prev_sets.items())       # something was skipped


def test_hrm_first_order_makes_later_gaps_order_free(small, kap_lists):
    """After the blocks holding a row maximum have been visited the running maximum is the
    maximum over the whole list, so the statistic no longer depends on the order."""
    q, k, v, _ = small
    order, count = kap_lists
    h, i = 1, 7
    cnt = int(count[h, i])
    mloc = np.stack([(q[h, i * 128:(i + 1) * 128] @ k[0, j * 128:(j + 1) * 128].T / math.sqrt(128))
                     for j in order[h, i, :cnt]])
    mloc[list(order[h, i, :cnt]).index(i)] = np.where(np.tri(128, dtype=bool), mloc[list(order[h, i, :cnt]).index(i)], -np.inf)
    mloc = mloc.max(axis=2)
    gstar = (mloc - mloc.max(axis=0)).max(axis=1)
    gaps = O.osk_gaps_offline(q, k, order, count, h, i)
    owners = set(np.argmax(mloc, axis=0))             # list positions that own some row's maximum
    last = max(owners)
    assert np.allclose(gaps[last:], gstar[last:], atol=0)
    assert (gaps >= gstar - 1e-15).all()              # Eq. (6): running max <= global max


def test_cap_on_computed_blocks(small, kap_lists):
    q, k, v, _ = small
    order, count = kap_lists
    n = q.shape[1]
    delta, tb = 200.0, 0.3
    theta = math.log(delta / n)
    r = O.osk_attention(q, k, v, order, count, skip_scale=delta, tightened_budget=tb)
    for (h, i), dec in r["decisions"].items():
        off = O.osk_gaps_offline(q, k, order, count, h, i)
        cap = min(int(count[h, i]), O.budget_count(tb, i + 1))
        want = [kk for kk, g in enumerate(off) if not g < theta][:cap]
        got = [kk for kk, c in enumerate(dec) if c]
        assert got == want and r["visited"][h, i // 1] == len(want)
        if len(want) == cap:                            # the walk stops right after the cap-th computed block
            assert len(dec) == want[-1] + 1
    # a cap that cannot bind changes nothing
    ra = O.osk_attention(q, k, v, order, count, skip_scale=delta, tightened_budget=0.999999)
    assert all(ra["decisions"][key] == [not g < theta for g in O.osk_gaps_offline(q, k, order, count, *key)]
               for key in ra["decisions"])
    # threshold off, cap on: the first C_i listed blocks
    rb = O.osk_attention(q, k, v, order, count, skip_scale=-1.0, tightened_budget=tb)
    for (h, i), dec in rb["decisions"].items():
        assert dec == [True] * min(int(count[h, i]), O.budget_count(tb, i + 1))


def test_skip_scale_not_below_n_is_rejected(small, kap_lists):
    q, k, v, _ = small
    with pytest.raises(ValueError):
        O.osk_attention(q, k, v, *kap_lists, skip_scale=float(q.shape[1]), tightened_budget=0.5)


# ---------------------------------------------------------------- KAP scores and flags
def test_literal_and_cancelled_forms_agree(small):
    q, k, v, _ = small
    for s in (4, 8, 16):
        for h in range(q.shape[0]):
            for i in (0, 1, 4, 7):
                a, fa, _ = O.kap_scores(q, k, h, i, s)
                b, fb = O.kap_scores_literal(q, k, h, i, s)
                assert np.abs(a - b).max() <= 1e-12 * max(1.0, a.max())
                assert np.array_equal(fa, fb)


def test_score_and_flag_invariants(small):
    q, k, v, _ = small
    for s in (8, 32):
        R = 128 // s
        for h in range(q.shape[0]):
            for i in range(8):
                sc, fl, M = O.kap_scores(q, k, h, i, s)
                assert (sc > 0).all() and (sc <= R).all()
                assert (sc[fl] >= 1.0).all()
                assert 1 <= fl.sum() <= R
                # every sampled row's maximum lies in some flagged block
                assert fl[np.argmax(M, axis=1)].all()


def test_block_scores_from_explicit_index_sets():
    """Eqs. (9)-(12) written out token by token: sampled query rows Q_i = {r : r div R = i}, sampled keys of a key
    block K_j = {c : c div R = j}, sampled row r is token r*s (likewise for keys), causal mask c <= r.  Scalar
    loops over plain Python floats that share nothing with the oracle's vectorised gather, reshape and max: a
    wrong axis or a wrong grouping of the sampled keys into blocks in `kap_scores` fails here."""
    q, k, _, _ = _inputs(seed=11, hq=2, hkv=1, n=512, needles=1)
    n, d = q.shape[1], q.shape[2]
    for s in (8, 32):
        R = 128 // s
        for h, i in ((0, 0), (0, 2), (1, 3)):
            rows = [r for r in range(n // s) if r // R == i]                      # Q_i
            J = i + 1
            P = {}                                                                # (r, j) -> max_c softmax(z)[r, c]
            for r in rows:
                cs = [c for c in range(n // s) if c <= r]                         # causal: sampled key not after the row
                z = {c: math.fsum(q[h, r * s, e] * k[0, c * s, e] for e in range(d)) / math.sqrt(d) for c in cs}
                zmax = max(z.values())
                den = math.fsum(math.exp(z[c] - zmax) for c in cs)                # Eq. 8: softmax over the sampled keys
                for j in range(J):
                    Kj = [c for c in cs if c // R == j]                           # K_j
                    P[r, j] = max(math.exp(z[c] - zmax) / den for c in Kj) if Kj else 0.0     # Eq. 9: MaxPool
            want_s, want_h = [], []
            for j in range(J):
                pbar = [P[r, j] / max(P[r, jj] for jj in range(J)) for r in rows]            # Eq. 10: MaxNorm
                want_s.append(math.fsum(pbar))                                               # Eq. 11
                want_h.append(any(x == 1.0 for x in pbar))                                   # Eq. 12
            got_s, got_h, _ = O.kap_scores(q, k, h, i, s)
            assert np.allclose(got_s, want_s, rtol=1e-12, atol=0)
            assert list(got_h) == want_h


def test_single_sample_per_block_reduces_to_argsort(small):
    """s = b: one sampled row and key per block, so exactly one HRM block and the list is
    that block followed by the others in descending order of the sampled logit."""
    q, k, v, _ = small
    order, count = O.kap_select(q, k, s=128, budget=1.0)
    for h in range(q.shape[0]):
        z = (q[h, ::128] @ k[0, ::128].T) / math.sqrt(128)
        for i in range(8):
            ref = np.argsort(-z[i, :i + 1], kind="stable")
            assert list(order[h, i, :i + 1]) == list(ref)
            _, fl, _ = O.kap_scores(q, k, h, i, 128)
            assert fl.sum() == 1 and fl[ref[0]]


def test_token_granularity_reduces_to_exact_logit_argsort():
    """b = 1, s = 1: every block is one token, the list is the argsort of the true logits."""
    rng = np.random.default_rng(5)
    q = rng.standard_normal((1, 24, 8)); k = rng.standard_normal((1, 24, 8))
    order, count = O.kap_select(q, k, s=1, budget=1.0, block=1)
    z = (q[0] @ k[0].T) / math.sqrt(8)
    for i in range(24):
        assert list(order[0, i, :i + 1]) == list(np.argsort(-z[i, :i + 1], kind="stable"))


# ---------------------------------------------------------------- KAP lists
def test_lists_against_bruteforce_lexsort(small):
    q, k, v, _ = small
    for budget in (0.2, 0.5, 1.0):
        order, count = O.kap_select(q, k, s=8, budget=budget)
        for h in range(q.shape[0]):
            for i in range(8):
                sc, fl, _ = O.kap_scores(q, k, h, i, 8)
                ref = np.lexsort((np.arange(i + 1), -sc, ~fl))      # last key is the primary one
                K = math.ceil(Fraction(budget).limit_denominator(1000) * (i + 1))
                K = max(1, min(i + 1, K))
                assert count[h, i] == K
                assert list(order[h, i, :K]) == list(ref[:K])
                assert (order[h, i, K:] == -1).all()


def test_list_structure_and_prefix_property(small):
    q, k, v, _ = small
    full, cfull = O.kap_select(q, k, s=8, budget=1.0)
    for budget in (0.1, 0.25, 0.5):
        order, count = O.kap_select(q, k, s=8, budget=budget)
        for h in range(q.shape[0]):
            for i in range(8):
                c = count[h, i]
                ids = order[h, i, :c]
                assert len(set(ids)) == c and ids.min() >= 0 and ids.max() <= i
                assert list(ids) == list(full[h, i, :c])            # lists are nested across budgets
                sc, fl, _ = O.kap_scores(q, k, h, i, 8)
                f = fl[ids]
                assert not (np.diff(f.astype(int)) > 0).any()       # flagged blocks first
                for grp in (ids[f], ids[~f]):
                    assert (np.diff(sc[grp]) <= 0).all()
    for h in range(q.shape[0]):
        for i in range(8):
            assert sorted(full[h, i, :i + 1]) == list(range(i + 1))


def test_ties_break_by_ascending_block_id():
    sc = np.array([0.5, 2.0, 0.5, 2.0, 0.5])
    fl = np.array([False, True, True, False, False])
    assert O.flag_grouped_order(sc, fl) == [1, 2, 3, 0, 4]


def test_budget_count_is_exact_ceiling():
    for b in (0.5, 0.25, 0.125, 0.2, 0.1, 0.08, 0.04, 0.0625, 1.0, 0.05, 0.025, 0.03125):
        for J in list(range(1, 300)) + [511, 512, 1000, 1024]:
            want = max(1, min(J, math.ceil(Fraction(str(b)) * J)))
            assert O.budget_count(b, J) == want, (b, J)


# ---------------------------------------------------------------- Top-p retention (Sec. 4.2 / Sec. C.1)
def test_topp_count_closed_forms():
    # equal scores: the prefix sum is k, so K = ceil(p * J) (p * J not an integer here)
    assert O.topp_count(np.ones(40), 0.33)[0] == 14
    # p * J an integer: the prefix that reaches the threshold exactly is enough (>=), margin 0
    kept, margin = O.topp_count(np.ones(40), 0.35)
    assert kept == 14 and margin == 0.0
    # geometric scores 2^-t (exact in binary): sum of k terms is 2 - 2^(1-k); 0.9 * total = 1.79999..:
    # three terms give 1.75, four give 1.875
    kept, margin = O.topp_count(0.5 ** np.arange(20), 0.9)
    assert kept == 4
    total = 2.0 - 2.0 ** -19
    assert margin == pytest.approx(min(1.875 - 0.9 * total, 0.9 * total - 1.75) / total, rel=1e-12)
    # p = 1 keeps everything, a vanishing p keeps the first entry only
    rng = np.random.default_rng(5)
    sc = rng.random(57) + 0.01
    assert O.topp_count(sc, 1.0)[0] == 57 and O.topp_count(sc, 1e-12)[0] == 1
    # monotone in p and minimal: one entry fewer does not reach the threshold
    last = 1
    for p_ in np.linspace(0.05, 0.99, 40):
        kept, _ = O.topp_count(sc, p_)
        assert kept >= last
        assert math.fsum(sc[:kept]) >= p_ * math.fsum(sc) * (1 - 1e-14)
        assert kept == 1 or math.fsum(sc[:kept - 1]) < p_ * math.fsum(sc) * (1 + 1e-14)
        last = kept


def test_topp_is_cumulated_along_the_flag_grouped_order():
    # an HRM block with a small score comes first in rho and counts toward the prefix: scores (0.1*, 5, 4),
    # p = 0.5 -> threshold 4.55: rho = (0, 1, 2), prefix sums 0.1, 5.1 -> two blocks; by score alone one would do
    scores, flags = np.array([0.1, 5.0, 4.0]), np.array([True, False, False])
    rho = O.flag_grouped_order(scores, flags)
    assert rho == [0, 1, 2]
    assert O.topp_count(scores[rho], 0.5)[0] == 2
    assert O.topp_count(np.sort(scores)[::-1], 0.5)[0] == 1


def test_kap_select_with_topp(small):
    q, k, _, _ = small
    nqb = q.shape[1] // 128
    full, cfull = O.kap_select(q, k, s=8, budget=1.0)
    # p = 1: whole candidate set; tiny p: the first entry; the list is always a prefix of the budget-1 list
    _, c1 = O.kap_select(q, k, s=8, budget=1.0, top_p=1.0)
    assert (c1 == cfull).all()
    _, c0 = O.kap_select(q, k, s=8, budget=1.0, top_p=1e-9)
    assert (c0 == 1).all()
    order, count, audit = O.kap_select(q, k, s=8, budget=1.0, top_p=0.9, audit=True)
    for h in range(q.shape[0]):
        for i in range(nqb):
            kept = count[h, i]
            assert 1 <= kept <= i + 1
            assert (order[h, i, :kept] == full[h, i, :kept]).all() and (order[h, i, kept:] == -1).all()
            # the definition, summed independently (exactly rounded sums) over the scores of the kept blocks
            scores, flags, _ = O.kap_scores(q, k, h, i, 8)
            total = math.fsum(scores)
            assert math.fsum(scores[order[h, i, :kept]]) >= 0.9 * total * (1 - 1e-13)
            if kept > 1:
                assert math.fsum(scores[order[h, i, :kept - 1]]) < 0.9 * total * (1 + 1e-13)
    assert np.isfinite(audit["topp_margin"]).all()
    # the budget count caps the Top-p count
    _, ccap = O.kap_select(q, k, s=8, budget=0.25, top_p=0.9)
    _, cb = O.kap_select(q, k, s=8, budget=0.25)
    assert (ccap == np.minimum(count, cb)).all()


# ---------------------------------------------------------------- wide query blocks (block_q = 256 variant)
def test_wide_block_scores_are_the_sum_over_its_row_tiles(small):
    """The sum over sampled rows of Eq. (11) splits over the two 128-row tiles, the flag of Eq. (12) is their OR;
    a key block wholly after a tile gets nothing from it."""
    q, k, _, _ = small
    for h in range(q.shape[0]):
        for big in range(q.shape[1] // 256):
            scores, flags, M = O.kap_scores_wide(q, k, h, big, 8)
            s0, f0, _ = O.kap_scores(q, k, h, 2 * big, 8)
            s1, f1, _ = O.kap_scores(q, k, h, 2 * big + 1, 8)
            assert len(scores) == 2 * big + 2
            assert np.abs(scores - (np.append(s0, 0.0) + s1)).max() < 1e-12
            assert np.array_equal(flags, np.append(f0, False) | f1)
            assert np.isneginf(M[:16, 2 * big + 1]).all()                    # the first tile never sees the last block
    # with a single tile the wide routine is the ordinary one
    sw, fw, _ = O.kap_scores_wide(q, k, 1, 5, 8, tiles=1)
    sn, fn, _ = O.kap_scores(q, k, 1, 5, 8)
    assert np.array_equal(sw, sn) and np.array_equal(fw, fn)


def test_wide_block_lists(small):
    q, k, _, _ = small
    nqb = q.shape[1] // 128
    order, count = O.kap_select_wide(q, k, s=8, budget=0.6)
    for h in range(q.shape[0]):
        for big in range(nqb // 2):
            scores, flags, _ = O.kap_scores_wide(q, k, h, big, 8)
            # the ranking by brute force: HRM group first, then by score, ties by id
            J = 2 * big + 2
            rank = sorted(range(J), key=lambda j: (not flags[j], -scores[j], j))[:O.budget_count(0.6, J)]
            hi = order[h, 2 * big + 1, :count[h, 2 * big + 1]].tolist()
            lo = order[h, 2 * big, :count[h, 2 * big]].tolist()
            assert hi == rank
            assert lo == [j for j in rank if j != 2 * big + 1] and all(j <= 2 * big for j in lo)
    # one tile per block: the ordinary lists
    o1, c1 = O.kap_select_wide(q, k, s=8, budget=0.6, tiles=1)
    o0, c0 = O.kap_select(q, k, s=8, budget=0.6, order_stride=nqb)
    assert np.array_equal(o1, o0) and np.array_equal(c1, c0)


# ---------------------------------------------------------------- paged K/V
def test_paged_view_hand_example_and_round_trip():
    from synth.generator import scatter_to_pages
    # two KV heads, four tokens, page size 2: logical page 0 -> physical 2, logical page 1 -> physical 0
    pool = np.arange(3 * 2 * 2 * 1).reshape(3, 2, 2, 1)
    view = O.paged_view(pool, np.array([2, 0]), 4)
    assert view[:, :, 0].tolist() == [[8, 9, 0, 1], [10, 11, 2, 3]]
    rng = np.random.default_rng(1)
    x = rng.integers(0, 2 ** 16, size=(3, 1024, 8), dtype=np.uint16)
    for page_size in (16, 64, 128, 256):
        pool, table = scatter_to_pages(x, page_size, seed=5)
        assert len(set(table.tolist())) == 1024 // page_size and pool.shape[0] == 1024 // page_size + 3
        assert np.array_equal(O.paged_view(pool, table, 1024), x)
        assert not np.array_equal(table, np.arange(1024 // page_size))          # really permuted


# ---------------------------------------------------------------- list utilities (remapping analysis, logical mask)
def test_list_utilities_against_hand_example_and_bruteforce():
    order = np.array([[[0, -1, -1, -1], [1, 0, -1, -1], [2, 0, 1, -1]]], np.int32)      # causal lists, nQB = 3
    count = np.array([[1, 2, 3]], np.int32)
    assert O.lists_reordered(order, count).tolist() == [[[0, -1, -1, -1], [0, 1, -1, -1], [0, 1, 2, -1]]]
    assert O.lists_reordered(order, count, descending=True).tolist() == [[[0, -1, -1, -1], [1, 0, -1, -1], [2, 1, 0, -1]]]
    # bit packing: block 33 is bit 1 of word 1, block 5 is bit 5 of word 0
    big = np.full((1, 40, 40), -1, np.int32)
    cnt = np.ones((1, 40), np.int32)
    big[0, :, 0] = 0
    big[0, 39, :3] = [33, 0, 5]
    cnt[0, 39] = 3
    mask = O.lists_to_mask(big, cnt, 40)
    assert mask.shape == (1, 40, 2) and mask[0, 39].tolist() == [0x21, 0x2] and mask[0, 7].tolist() == [1, 0]
    # round trip on random causal sets: mask -> walk gives the ascending list; non-candidate bits are ignored
    rng = np.random.default_rng(3)
    nqb = 70
    order = np.full((2, nqb, nqb), -1, np.int32)
    count = np.zeros((2, nqb), np.int32)
    for h in range(2):
        for i in range(nqb):
            ids = rng.permutation(i + 1)[:rng.integers(1, i + 2)]
            order[h, i, :len(ids)] = ids
            count[h, i] = len(ids)
    mask = O.lists_to_mask(order, count, nqb)
    for h in range(2):
        for i in range(nqb):
            assert {j for j in range(nqb) if (int(mask[h, i, j // 32]) >> (j % 32)) & 1} == set(order[h, i, :count[h, i]].tolist())
    noisy = mask.copy()
    noisy[:, :5, 2] = 0xffffffff                                             # blocks 64.. are no candidates of rows 0..4
    back, bcount = O.mask_to_lists(noisy, nqb)
    assert np.array_equal(back, O.lists_reordered(order, count)) and np.array_equal(bcount, count)


def test_natural_order_keeps_the_set_but_changes_the_decisions(small):
    """Order invariance (Eq. 4) holds with Stage 2 off; with the skip rule on, the visiting order matters
    (Sec. 3.3, Limitation 2): the remapping analysis rests on exactly this."""
    q, k, v, _ = small
    order, count = O.kap_select(q, k, s=8, budget=0.75)
    nat = O.lists_reordered(order, count)
    a = O.osk_attention(q, k, v, order, count, tightened_budget=1.0)
    b = O.osk_attention(q, k, v, nat, count, tightened_budget=1.0)
    assert np.abs(a["out"] - b["out"]).max() < 1e-12
    c = O.osk_attention(q, k, v, order, count, skip_scale=300.0, tightened_budget=0.999)
    d = O.osk_attention(q, k, v, nat, count, skip_scale=300.0, tightened_budget=0.999)
    assert c["visited"].sum() < d["visited"].sum()          # HRM-first order lets more blocks fall below the threshold


def test_planted_structure_is_recalled():
    q, k, v, planted = _inputs(seed=11, hq=4, hkv=1, n=2048, needles=3)
    order, count = O.kap_select(q, k, s=8, budget=0.35)
    for h in range(4):
        for i in range(8, 16):
            ids = set(order[h, i, :count[h, i]])
            assert 0 in ids and i - 1 in ids                        # sink and local band
        for j, t in zip(planted["needle_key_blocks"][0], planted["needle_targets"][0]):
            if t >= 3:
                assert j in set(order[h, t, :count[h, t]])          # the needle, at its target block


def test_frozen_oracle_outputs():
    """The stored values were written by tests/golden/make_golden.py from the oracle alone."""
    import json
    import os
    with open(os.path.join(os.path.dirname(__file__), "golden", "oracle_tiny.json")) as f:
        doc = json.load(f)
    q, k, v, _ = _inputs()
    order, count = O.kap_select(q, k, s=8, budget=0.5)
    assert order.tolist() == doc["order"] and count.tolist() == doc["count"]
    r = O.osk_attention(q, k, v, order, count, skip_scale=200.0, tightened_budget=0.3)
    assert r["visited"].tolist() == doc["visited"] and r["scored"].tolist() == doc["scored"]
    assert np.allclose(r["out"][1, 1000, :4], doc["out_sample"], atol=1e-13)
    assert np.allclose(r["lse"][0, ::128], doc["lse_sample"], atol=1e-13)
