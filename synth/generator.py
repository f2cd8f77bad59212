"""Seeded synthetic Q/K/V with planted attention structure.

This module only draws random numbers and plants structure; it holds none of
the method's arithmetic (no scoring, no softmax, no selection).  Both the CPU
oracle's tests and the CUDA path's tests read their inputs from here, so the
two sides always see the same bf16 bit patterns.

Recipe (per KV head g, block size b, blk(t) = t // b):
  Q[h,t] = n + alpha * (u_g + w_{g,blk(t)})                    n ~ N(0, I)
  K[g,t] = n + [blk(t)=0] * sigma * u_g + tau * sum_{m<W} w_{g,blk(t)+m}
  needles: P key blocks j_n (distinct, >= 1) each paired with a distinct
           target query block t_n >= j_n; every key of block j_n is set to
           0.5 * mean(bf16 Q rows of block t_n over the G heads of the group)
  V[g,t] = n
u_g and w_{g,i} are unit vectors.  Key block 0 is the sink, key block j serves
query blocks j..j+W-1 (local band), needle blocks are vertical lines that peak
at their target query block.  Everything is rounded to bf16 (round to nearest
even) and returned as uint16 bit patterns.
"""
from __future__ import annotations

from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass

import numpy as np


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round fp32 to bf16 (nearest even) and return the 16-bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    rounded = u + (np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1)))
    return (rounded >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32)


def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    return bf16_bits_to_f32(bits).astype(np.float64)


@dataclass(frozen=True)
class Structure:
    """Planted-structure parameters of one synthetic attention layer."""
    band: int = 2          # W: local band width in blocks
    needles: int = 3       # P: needle key blocks per KV head
    alpha: float = 8.0     # amplitude of the planted query direction
    sigma: float = 10.0    # sink amplitude on key block 0
    tau: float = 8.0       # band amplitude


def _rng(seed: int, stream: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[seed, stream]))


def _unit(v: np.ndarray) -> np.ndarray:
    return v / np.linalg.norm(v, axis=-1, keepdims=True)


def plan_needles(seed: int, g: int, n_blocks: int, needles: int):
    """Distinct needle key blocks j_n >= 1 with distinct targets t_n >= j_n."""
    rng = _rng(seed, 7_000_000 + g)
    P = min(needles, max(n_blocks - 1, 0))
    if P == 0:
        return np.zeros(0, np.int64), np.zeros(0, np.int64)
    targets = np.sort(rng.choice(np.arange(1, n_blocks), size=P, replace=False))
    keys = []
    used = set()
    for t in targets:                       # ascending targets: a free j <= t always exists
        free = [j for j in range(1, int(t) + 1) if j not in used]
        j = free[int(rng.integers(0, len(free)))]
        used.add(j)
        keys.append(j)
    return np.asarray(keys, np.int64), targets.astype(np.int64)


def make_qkv(seed: int, hq: int, hkv: int, n: int, d: int = 128, block: int = 128,
             st: Structure = Structure(), threads: int = 8):
    """Return (q, k, v) as uint16 bf16 bit patterns of shapes
    [hq, n, d], [hkv, n, d], [hkv, n, d], plus a dict describing what was planted."""
    assert hq % hkv == 0 and n % block == 0
    G = hq // hkv
    nb = n // block
    q = np.empty((hq, n, d), np.uint16)
    k = np.empty((hkv, n, d), np.uint16)
    v = np.empty((hkv, n, d), np.uint16)
    planted = {"needle_key_blocks": [], "needle_targets": []}

    dirs = []
    for g in range(hkv):
        r = _rng(seed, 1_000_000 + g)
        u = _unit(r.standard_normal(d))
        w = _unit(r.standard_normal((nb + st.band, d)))
        w[nb:] = 0.0                        # band does not extend past the sequence
        dirs.append((u.astype(np.float32), w.astype(np.float32)))

    def fill_q(h):
        g = h // G
        u, w = dirs[g]
        x = _rng(seed, 2_000_000 + h).standard_normal((n, d), dtype=np.float32)
        x = x.reshape(nb, block, d)
        x += (st.alpha * (u[None, :] + w[:nb]))[:, None, :]
        q[h] = f32_to_bf16_bits(x.reshape(n, d))

    def fill_k(g):
        u, w = dirs[g]
        x = _rng(seed, 3_000_000 + g).standard_normal((n, d), dtype=np.float32)
        x = x.reshape(nb, block, d)
        bandsum = np.zeros((nb, d), np.float32)
        for m in range(st.band):
            bandsum += w[m:m + nb]
        x += (st.tau * bandsum)[:, None, :]
        x[0] += st.sigma * u[None, :]
        k[g] = f32_to_bf16_bits(x.reshape(n, d))

    def fill_v(g):
        x = _rng(seed, 4_000_000 + g).standard_normal((n, d), dtype=np.float32)
        v[g] = f32_to_bf16_bits(x)

    with ThreadPoolExecutor(max_workers=threads) as ex:
        list(ex.map(fill_q, range(hq)))
        list(ex.map(fill_k, range(hkv)))
        list(ex.map(fill_v, range(hkv)))

    for g in range(hkv):
        jn, tn = plan_needles(seed, g, nb, st.needles)
        for j, t in zip(jn, tn):
            rows = bf16_bits_to_f32(q[g * G:(g + 1) * G, t * block:(t + 1) * block, :])
            qbar = rows.reshape(-1, d).mean(axis=0, dtype=np.float64).astype(np.float32)
            k[g, j * block:(j + 1) * block, :] = f32_to_bf16_bits(0.5 * qbar)[None, :]
        planted["needle_key_blocks"].append(jn)
        planted["needle_targets"].append(tn)
    return q, k, v, planted


def scatter_to_pages(x_bits: np.ndarray, page_size: int, seed: int, spare_pages: int = 3):
    """Lay a dense [Hkv, N, d] tensor out as a paged pool (layout only, no arithmetic).

    Returns (pool [P, Hkv, page_size, d] uint16, table [N / page_size] int32): logical page t of every
    KV head lives in physical page table[t]; the pages are a seeded random permutation and the
    pool holds a few unused pages filled with a recognisable bit pattern."""
    hkv, n, d = x_bits.shape
    assert n % page_size == 0
    n_pages = n // page_size
    rng = np.random.Generator(np.random.Philox(key=[seed, 77]))
    phys = rng.permutation(n_pages + spare_pages)[:n_pages].astype(np.int32)
    pool = np.full((n_pages + spare_pages, hkv, page_size, d), 0x7FC0, np.uint16)   # bf16 NaN in unused pages
    pool[phys] = x_bits.reshape(hkv, n_pages, page_size, d).transpose(1, 0, 2, 3)
    return pool, phys
