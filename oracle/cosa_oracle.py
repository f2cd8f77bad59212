"""fp64 CPU oracle for the CoSA hot path (KAP selection/ordering + OSK attention).

TEST INFRASTRUCTURE ONLY.  This is a plain, slow restatement of what the paper
defines, written to be checked against the paper by eye.  It shares no code with
the CUDA path and must never be imported by the product package; only the test
suite, the smoke check and the benchmark's CPU-baseline leg call it.

All arithmetic is float64 on inputs that are bf16 values widened exactly.
Block ids, list positions and row indices are 0-based (the paper is 1-based).

Parity status: every function here is pinned by the CPU tests (closed forms,
library routines, brute force, order invariance, hand-built skip cases).  The
paper prints no worked numeric example, so no value fixture comes from it; the
conventions the paper leaves open (sampling offset, tie-break, budget rounding,
the computed-block cap) are this build's readings and are "parity unpinned" as
conventions -- they are stated next to the code that takes them.

Functions
  dense_attention     Sec. 3.1, Eqs. (1)-(2): softmax(QK^T/sqrt d)V, the plain definition
  masked_attention    Sec. 3.2, Eq. (3): the same restricted to a set of key blocks
  kap_scores          Sec. 4.2, Eqs. (8)-(12); Algorithm A steps 2-4
  kap_scores_literal  the same with the softmax written out (identity check)
  kap_select          Eqs. (13)-(14); Algorithm A step 5
  osk_attention       Algorithm A steps 7-21 with the skip rule of Eq. (5)
  osk_gaps_offline    closed form of the skip statistic, independent of decisions
"""
from __future__ import annotations

import math

import numpy as np

NEG_INF = -np.inf


# ----------------------------------------------------------------------------
# budgets (this build's reading; the paper only says K_i = B x J, Eq. 14)
# ----------------------------------------------------------------------------
def budget_count(budget: float, candidates: int) -> int:
    """ceil(budget * candidates) in exact integer arithmetic, clamped to [1, candidates].

    The fraction is first truncated to 20 fractional bits of its float32 value, so
    that a CPU and a GPU evaluate the very same integer expression.
    """
    fx = int(math.floor(float(np.float32(budget)) * (1 << 20)))
    kept = (fx * candidates + (1 << 20) - 1) >> 20
    return max(1, min(candidates, kept))


def n_candidates(i: int, n_kblocks: int, causal: bool) -> int:
    """Causal candidates of query block i are key blocks j <= i (Algorithm A step 5)."""
    return i + 1 if causal else n_kblocks


# ----------------------------------------------------------------------------
# dense and masked attention: the plain definitions
# ----------------------------------------------------------------------------
def _attend_rows(q_rows, k_all, v_all, key_ok, scale):
    """softmax over the permitted keys for a set of query rows.

    q_rows [T,d], k_all/v_all [U,d], key_ok [T,U] bool.  Returns O [T,d], lse [T],
    and the probabilities [T,U] (for the rows-sum-to-one pin)."""
    logits = (q_rows @ k_all.T) * scale
    logits = np.where(key_ok, logits, NEG_INF)
    mx = logits.max(axis=1, keepdims=True)
    e = np.exp(logits - mx)
    denom = e.sum(axis=1, keepdims=True)
    p = e / denom
    return p @ v_all, (mx + np.log(denom))[:, 0], p


def dense_attention(q, k, v, causal=True, block=128, query_blocks=None, return_probs=False):
    """O[h,t] = sum_u softmax_u(q_t.k_u / sqrt d) v_u with u <= t if causal (Eqs. 1-2).

    q [Hq,N,d], k,v [Hkv,N,d] float64; query head h reads KV head h // (Hq/Hkv).
    `query_blocks` restricts the evaluation to some blocks of `block` query rows
    (the result arrays then hold only those rows, in the given order)."""
    hq, n, d = q.shape
    G = hq // k.shape[0]
    scale = 1.0 / math.sqrt(d)
    qbs = list(range(n // block)) if query_blocks is None else list(query_blocks)
    out = np.zeros((hq, len(qbs) * block, d))
    lse = np.zeros((hq, len(qbs) * block))
    probs = []
    for h in range(hq):
        g = h // G
        for a, i in enumerate(qbs):
            t = np.arange(i * block, (i + 1) * block)
            hi = (i + 1) * block if causal else k.shape[1]
            u = np.arange(hi)
            ok = (u[None, :] <= t[:, None]) if causal else np.ones((block, hi), bool)
            o, l, p = _attend_rows(q[h, t], k[g, :hi], v[g, :hi], ok, scale)
            out[h, a * block:(a + 1) * block] = o
            lse[h, a * block:(a + 1) * block] = l
            if return_probs:
                probs.append(p)
    return (out, lse, probs) if return_probs else (out, lse)


def masked_attention(q, k, v, block_sets, causal=True, block=128, query_blocks=None):
    """Attention restricted to the keys of the listed key blocks (Eq. 3).

    block_sets[h][a] is an iterable of key-block ids for query head h and the a-th
    entry of `query_blocks`; order and repetition do not matter.  Inside block j == i
    the token-level causal mask u <= t applies."""
    hq, n, d = q.shape
    G = hq // k.shape[0]
    scale = 1.0 / math.sqrt(d)
    qbs = list(range(n // block)) if query_blocks is None else list(query_blocks)
    out = np.zeros((hq, len(qbs) * block, d))
    lse = np.zeros((hq, len(qbs) * block))
    for h in range(hq):
        g = h // G
        for a, i in enumerate(qbs):
            js = sorted(set(int(j) for j in block_sets[h][a]))
            t = np.arange(i * block, (i + 1) * block)
            u = np.concatenate([np.arange(j * block, (j + 1) * block) for j in js])
            ok = (u[None, :] <= t[:, None]) if causal else np.ones((block, len(u)), bool)
            o, l, _ = _attend_rows(q[h, t], k[g, u], v[g, u], ok, scale)
            out[h, a * block:(a + 1) * block] = o
            lse[h, a * block:(a + 1) * block] = l
    return out, lse


# ----------------------------------------------------------------------------
# KAP: scores, flags, ordering
# ----------------------------------------------------------------------------
def _sampled_logits(q, k, h, g, i, s, block, causal):
    """Algorithm A step 2 for query block i: strided rows, scaled logits, causal mask.

    Sampled query rows r in [iR,(i+1)R) are tokens r*s; sampled keys c are tokens
    c*s; key c belongs to key block c // R.  Returns z [R, J*R] with -inf where the
    sampled key lies after the sampled query, and J."""
    n, d = q.shape[1], q.shape[2]
    R = block // s
    J = n_candidates(i, n // block, causal)
    r = np.arange(i * R, (i + 1) * R)
    c = np.arange(J * R)
    z = (q[h, r * s] @ k[g, c * s].T) * (1.0 / math.sqrt(d))
    if causal:
        z = np.where(c[None, :] <= r[:, None], z, NEG_INF)
    return z, J


def kap_scores(q, k, h, i, s=8, block=128, causal=True):
    """Block scores s_ij and HRM flags h_ij of query head h, query block i (Eqs. 8-12).

    The softmax denominator of a sampled row is common to all of that row's keys and
    cancels in P[r,j] / max_j' P[r,j'], so Pbar[r,j] = exp(M[r,j] - M*[r]) with
    M[r,j] the largest logit of row r inside key block j and M*[r] the row's largest
    logit overall.  The HRM flag asks whether some row attains Pbar = 1, i.e. whether
    M[r,j] == M*[r] for some r.  Returns (scores [J], flags [J] bool, M [R,J])."""
    G = q.shape[0] // k.shape[0]
    R = block // s
    z, J = _sampled_logits(q, k, h, h // G, i, s, block, causal)
    M = z.reshape(R, J, R).max(axis=2)            # MaxPool over the sampled keys of block j
    Mstar = M.max(axis=1)                         # the row's maximum over blocks
    Pbar = np.exp(M - Mstar[:, None])             # MaxNorm
    scores = np.zeros(J)
    for r in range(R):                            # sum over the sampled rows of block i
        scores += Pbar[r]
    flags = (M == Mstar[:, None]).any(axis=0)
    return scores, flags, M


def kap_scores_literal(q, k, h, i, s=8, block=128, causal=True):
    """Eqs. (8)-(12) with the softmax written out, no cancellation."""
    G = q.shape[0] // k.shape[0]
    R = block // s
    z, J = _sampled_logits(q, k, h, h // G, i, s, block, causal)
    e = np.exp(z - z.max(axis=1, keepdims=True))
    S_hat = e / e.sum(axis=1, keepdims=True)      # Softmax over the (causal) sampled keys
    P = S_hat.reshape(R, J, R).max(axis=2)        # MaxPool
    Pbar = P / P.max(axis=1, keepdims=True)       # MaxNorm
    scores = Pbar.sum(axis=0)
    flags = (Pbar.max(axis=0) == 1.0)
    return scores, flags


def kap_scores_wide(q, k, h, big, s=8, block=128, tiles=2, causal=True):
    """Scores and flags of a query block of tiles*block rows against key blocks of `block`
    rows (Sec. C.1 names b = 128 for both; this is the wider-query variant): Eqs. (8)-(12)
    with the sum of Eq. (11) and the "some row" of Eq. (12) running over all sampled rows of
    the wide block.  Candidates when causal: the key blocks holding a key that some row of
    the block may see, j < tiles * (big + 1).  Returns (scores [J], flags [J], M [tiles*R, J])."""
    G = q.shape[0] // k.shape[0]
    n, d = q.shape[1], q.shape[2]
    R = block // s
    rows = tiles * R
    J = tiles * (big + 1) if causal else n // block
    r = np.arange(big * rows, (big + 1) * rows)
    c = np.arange(J * R)
    z = (q[h, r * s] @ k[h // G, c * s].T) * (1.0 / math.sqrt(d))
    if causal:
        z = np.where(c[None, :] <= r[:, None], z, NEG_INF)
    M = z.reshape(rows, J, R).max(axis=2)
    Mstar = M.max(axis=1)
    Pbar = np.exp(M - Mstar[:, None])             # 0 where a row sees nothing of block j
    scores = np.zeros(J)
    for rr in range(rows):
        scores += Pbar[rr]
    flags = (M == Mstar[:, None]).any(axis=0)
    return scores, flags, M


def kap_select_wide(q, k, s=8, budget=0.25, causal=True, block=128, tiles=2, order_stride=None, heads=None,
                    wide_blocks=None, top_p=None):
    """Stage-1 lists when one ranking is made per query block of tiles*block rows and shared by
    its `tiles` row tiles of `block` rows (the block_q = 256 variant).  The wide block keeps the
    first K = budget_count(budget, candidates) entries of its flag-grouped order; row tile t of
    the block gets those entries in that order minus the key blocks that lie wholly after it
    (when causal).  Returns per-tile (order [Hq, N/block, order_stride], count [Hq, N/block])."""
    hq, n, _ = q.shape
    nqb = n // block
    nbig = nqb // tiles
    if order_stride is None:
        order_stride = nqb
    order = np.full((hq, nqb, order_stride), -1, np.int32)
    count = np.zeros((hq, nqb), np.int32)
    for h in (range(hq) if heads is None else heads):
        for big in (range(nbig) if wide_blocks is None else wide_blocks):
            scores, flags, _ = kap_scores_wide(q, k, h, big, s, block, tiles, causal)
            rho = flag_grouped_order(scores, flags)
            n_keep = budget_count(budget, len(rho))
            if top_p is not None:
                n_keep = min(n_keep, topp_count(scores[rho], top_p)[0])
            kept = rho[:n_keep]
            for t in range(tiles):
                i = big * tiles + t
                ids = [j for j in kept if (not causal) or j <= i]
                order[h, i, :len(ids)] = ids
                count[h, i] = len(ids)
    return order, count


def flag_grouped_order(scores, flags):
    """rho_i of Eq. (13): HRM blocks first, each group by descending score.
    Equal scores inside a group are ordered by ascending block id (this build's
    tie-break; the paper states none)."""
    ids = list(range(len(scores)))
    ids.sort(key=lambda j: (0 if flags[j] else 1, -scores[j], j))
    return ids


def topp_count(scores_in_order, top_p: float):
    """Top-p retention of Stage 1 (Sec. 4.2, text after Eq. 13; Sec. C.1: p = 0.95 for Qwen).

    `scores_in_order` are the block scores s_ij taken along the computation order rho_i.
    K_i is the length of the shortest prefix of rho_i whose scores sum to at least
    top_p times the sum over all candidates (cumulated along rho_i, i.e. with the HRM
    group first: the paper "retains the leading entries" of that order).  Returns
    (K_i, margin): margin is the relative distance |cum - top_p*total| / total of the
    closest of the two prefix sums that decide K_i (at K_i and at K_i - 1)."""
    c = np.cumsum(np.asarray(scores_in_order, np.float64))
    total = float(c[-1])
    thr = float(top_p) * total
    kept = len(c)
    for t in range(len(c)):
        if c[t] >= thr:
            kept = t + 1
            break
    gaps = [abs(float(c[kept - 1]) - thr)]
    if kept >= 2:
        gaps.append(abs(float(c[kept - 2]) - thr))
    return kept, min(gaps) / max(total, 1e-300)


def kap_select(q, k, s=8, budget=0.25, causal=True, block=128, heads=None, query_blocks=None,
               order_stride=None, audit=False, top_p=None):
    """Ordered Stage-1 visit lists M_KAP (Eq. 14): order[h,i,:count] then -1 padding.

    Returns (order int32 [Hq,nQB,order_stride], count int32 [Hq,nQB]) and, if `audit`,
    a dict with the smallest decision margins met (relative gap between adjacent list
    entries of one group up to and including the retention boundary; absolute gap
    between the two largest block maxima of a sampled row).

    `top_p` (None = off): K_i is the Top-p count of topp_count(), still capped by the
    budget count (budget = 1 leaves Top-p alone); the audit then also holds the per-list
    margins of that decision ("topp_margin" [Hq,nQB], inf where the cap decided)."""
    hq, n, _ = q.shape
    nqb = n // block
    nkb = nqb
    if order_stride is None:
        order_stride = max(budget_count(budget, n_candidates(i, nkb, causal)) for i in range(nqb))
    order = np.full((hq, nqb, order_stride), -1, np.int32)
    count = np.zeros((hq, nqb), np.int32)
    min_rel_gap, min_top2 = np.inf, np.inf
    topp_margin = np.full((hq, nqb), np.inf)
    for h in (range(hq) if heads is None else heads):
        for i in (range(nqb) if query_blocks is None else query_blocks):
            scores, flags, M = kap_scores(q, k, h, i, s, block, causal)
            rho = flag_grouped_order(scores, flags)
            K_i = budget_count(budget, len(rho))
            if top_p is not None:
                K_p, margin = topp_count(scores[rho], top_p)
                if K_p <= K_i:
                    K_i = K_p
                    topp_margin[h, i] = margin
            order[h, i, :K_i] = rho[:K_i]
            count[h, i] = K_i
            if audit:
                for a in range(min(K_i, len(rho) - 1)):
                    ja, jb = rho[a], rho[a + 1]
                    if flags[ja] == flags[jb]:
                        gap = (scores[ja] - scores[jb]) / max(scores[ja], 1e-300)
                        min_rel_gap = min(min_rel_gap, gap)
                if M.shape[1] > 1:
                    top = np.sort(M, axis=1)
                    min_top2 = min(min_top2, float((top[:, -1] - top[:, -2]).min()))
    if audit:
        return order, count, {"min_rel_score_gap": float(min_rel_gap), "min_row_top2_gap": float(min_top2),
                              "topp_margin": topp_margin}
    return order, count


# ----------------------------------------------------------------------------
# Paged K/V (Sec. C.1: a logical block of b = 128 tokens is resolved through one or more
# physical pages of b_p tokens)
# ----------------------------------------------------------------------------
def paged_view(pool, table, n):
    """The logical [Hkv, N, d] tensor behind a page pool [P, Hkv, b_p, d] and a page table
    [N / b_p]: token t of KV head g is pool[table[t div b_p], g, t mod b_p].  Everything the
    method computes is defined on this view."""
    page_size = pool.shape[2]
    out = np.empty((pool.shape[1], n, pool.shape[3]), pool.dtype)
    for t in range(n // page_size):
        out[:, t * page_size:(t + 1) * page_size] = pool[int(table[t])]
    return out


# ----------------------------------------------------------------------------
# List utilities for the remapping analysis (Sec. 5.3 "Effect of remapping") and the
# logical-mask comparison (Sec. D "Kernel Microbenchmark")
# ----------------------------------------------------------------------------
def lists_reordered(order, count, descending=False):
    """The same kept sets visited in natural page order (ascending block id: execution
    "without remapping") or in descending id order; padding stays -1."""
    out = np.full_like(order, -1)
    for h in range(order.shape[0]):
        for i in range(order.shape[1]):
            ids = sorted(int(x) for x in order[h, i, :count[h, i]])
            if descending:
                ids.reverse()
            out[h, i, :len(ids)] = ids
    return out


def lists_to_mask(order, count, n_kblocks):
    """The binary block mask of Eq. (3) for the kept sets: uint32 words [Hq,nQB,ceil(nKB/32)],
    block j is bit (j mod 32) of word (j div 32)."""
    words = (n_kblocks + 31) // 32
    mask = np.zeros(order.shape[:2] + (words,), np.uint32)
    for h in range(order.shape[0]):
        for i in range(order.shape[1]):
            for j in order[h, i, :count[h, i]]:
                mask[h, i, int(j) // 32] |= np.uint32(1 << (int(j) % 32))
    return mask


def mask_to_lists(mask, n_kblocks, causal=True, order_stride=None):
    """The visiting sequence of a kernel that walks the candidates j = 0, 1, ... and skips the
    ones whose mask bit is clear ("logical skipping"): the kept ids in ascending order.  Bits of
    non-candidates (j > i when causal, j >= nKB) are ignored."""
    hq, nqb, _ = mask.shape
    order_stride = order_stride or n_kblocks
    order = np.full((hq, nqb, order_stride), -1, np.int32)
    count = np.zeros((hq, nqb), np.int32)
    for h in range(hq):
        for i in range(nqb):
            ids = [j for j in range(n_candidates(i, n_kblocks, causal)) if (int(mask[h, i, j // 32]) >> (j % 32)) & 1]
            order[h, i, :len(ids)] = ids
            count[h, i] = len(ids)
    return order, count


# ----------------------------------------------------------------------------
# OSK: ordered traversal with the in-kernel skip
# ----------------------------------------------------------------------------
def skip_threshold(skip_scale: float, n: int) -> float:
    """ln(Delta / N) of Eq. (5); N is the sequence length of the call."""
    return math.log(skip_scale / n)


def _block_logits(q, k, h, g, i, j, block, causal, scale):
    """S_ij = Q_i K_j^T / sqrt d, with the token-level causal mask on the diagonal block."""
    S = (q[h, i * block:(i + 1) * block] @ k[g, j * block:(j + 1) * block].T) * scale
    if causal and j == i:
        t = np.arange(block)
        S = np.where(t[None, :] <= t[:, None], S, NEG_INF)
    return S


def osk_attention(q, k, v, order, count, skip_scale=2000.0, tightened_budget=1.0, causal=True,
                  block=128, heads=None, query_blocks=None):
    """Algorithm A steps 7-21 for every (query head, query block).

    For list position kk: j = order[h,i,kk]; S = Q_i K_j^T / sqrt d; m_loc = rowmax S;
    m' = m; m = max(m, m_loc); gap = max_r (m_loc[r] - m[r]); the block is skipped
    (nothing added to l or O) iff Delta > 0 and gap < ln(Delta/N)  (Eq. 5, the running
    maximum already includes the block under test).  Otherwise P = exp(S - m),
    l = exp(m'-m) l + rowsum P, O = diag(exp(m'-m)) O + P V_j.  Finally O /= l.

    `tightened_budget` (this build's reading, not in the paper, where the overall budget
    is an outcome): >= 1 switches Stage 2 off altogether; otherwise the walk also stops
    once ceil(tightened_budget * candidates) blocks have been computed (clamped to
    [1, count]).  skip_scale <= 0 switches the threshold test off (the paper's Delta=-1).

    Returns dict: out [Hq,nQ*b,d], lse (natural log of the summed exp of the scaled
    logits over the computed keys), visited (computed blocks), scored (blocks whose
    logits were formed), decisions (list of bool per scored position: True = computed),
    gaps (the statistic of every scored position)."""
    hq, nq, d = q.shape
    n = k.shape[1]                     # N of Eq. (5): the context length (nq == n in prefill)
    G = hq // k.shape[0]
    nkb = n // block
    scale = 1.0 / math.sqrt(d)
    stage2 = tightened_budget < 1.0
    use_rule = stage2 and skip_scale > 0
    if use_rule and not skip_scale < n:
        raise ValueError("skip_scale >= N would skip the first block")
    theta = skip_threshold(skip_scale, n) if use_rule else None
    hs = list(range(hq)) if heads is None else list(heads)
    qbs = list(range(nq // block)) if query_blocks is None else list(query_blocks)
    out = np.zeros((hq, len(qbs) * block, d))
    lse = np.zeros((hq, len(qbs) * block))
    visited = np.zeros((hq, len(qbs)), np.int32)
    scored = np.zeros((hq, len(qbs)), np.int32)
    decisions = {}
    gaps = {}
    for h in hs:
        g = h // G
        for a, i in enumerate(qbs):
            cnt = int(count[h, i])
            cap = cnt
            if stage2:
                cap = min(cnt, budget_count(tightened_budget, n_candidates(i, nkb, causal)))
            m = np.full(block, NEG_INF)
            l = np.zeros(block)
            O = np.zeros((block, d))
            computed = 0
            dec, gp = [], []
            for kk in range(cnt):
                if computed == cap:
                    break
                j = int(order[h, i, kk])
                S = _block_logits(q, k, h, g, i, j, block, causal, scale)
                m_loc = S.max(axis=1)
                m_prev = m
                m = np.maximum(m, m_loc)
                gap = float((m_loc - m).max())
                gp.append(gap)
                if use_rule and gap < theta:
                    dec.append(False)
                    continue
                P = np.exp(S - m[:, None])
                alpha = np.exp(m_prev - m)
                l = alpha * l + P.sum(axis=1)
                O = alpha[:, None] * O + P @ v[g, j * block:(j + 1) * block]
                computed += 1
                dec.append(True)
            out[h, a * block:(a + 1) * block] = O / l[:, None]
            lse[h, a * block:(a + 1) * block] = m + np.log(l)
            visited[h, a] = computed
            scored[h, a] = len(dec)
            decisions[(h, i)] = dec
            gaps[(h, i)] = gp
    return {"out": out, "lse": lse, "visited": visited, "scored": scored,
            "decisions": decisions, "gaps": gaps}


def osk_gaps_offline(q, k, order, count, h, i, causal=True, block=128):
    """gap_kk = max_r ( m_loc_kk[r] - max_{kk' <= kk} m_loc_kk'[r] ) for every list position.

    A skipped block lies below the running maximum on every row, so it never moves the
    maximum: the statistic of each position does not depend on earlier decisions or on
    Delta, and can be evaluated over the whole list at once."""
    G = q.shape[0] // k.shape[0]
    d = q.shape[2]
    scale = 1.0 / math.sqrt(d)
    cnt = int(count[h, i])
    mloc = np.stack([_block_logits(q, k, h, h // G, i, int(order[h, i, kk]), block, causal, scale).max(axis=1)
                     for kk in range(cnt)])
    run = np.maximum.accumulate(mloc, axis=0)
    return (mloc - run).max(axis=1)
