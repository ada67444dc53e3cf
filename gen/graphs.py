"""Seeded synthetic graphs with the shapes of the paper's workloads.

Every generator returns an undirected simple graph (no self-loops, no parallel
edges) as a symmetric CSR pair ``(rowptr int64[n+1], col int32[nnz])`` whose
column indices ascend inside each row.  ``nnz`` counts both directions of every
undirected edge, the convention of the paper's average-degree figures (Section
5.3: 2 * #Edges / #Vertices of Table 1).

Nothing here belongs to the method under test: there is no partitioning, no
sampling, no normalization and no network arithmetic in this package.  It only
draws inputs, so the CPU checker and the CUDA library can both be fed the same
bytes.
"""
from __future__ import annotations

import numpy as np


def _rng(seed: int) -> np.random.Generator:
    # Philox is counter-based: the stream depends on the seed only, never on
    # the machine or on the thread count.
    return np.random.Generator(np.random.Philox(int(seed)))


def csr_from_undirected(n: int, lo: np.ndarray, hi: np.ndarray):
    """Symmetric CSR from unique undirected pairs ``lo < hi``."""
    src = np.concatenate([lo, hi]).astype(np.int64, copy=False)
    dst = np.concatenate([hi, lo]).astype(np.int64, copy=False)
    key = src * np.int64(n) + dst
    key.sort()
    src = key // np.int64(n)
    col = (key - src * np.int64(n)).astype(np.int32)
    counts = np.bincount(src, minlength=n)
    rowptr = np.zeros(n + 1, dtype=np.int64)
    np.cumsum(counts, out=rowptr[1:])
    return rowptr, col


def _dedupe_sorted(keys: np.ndarray) -> np.ndarray:
    keys.sort()
    if keys.size == 0:
        return keys
    keep = np.empty(keys.size, dtype=bool)
    keep[0] = True
    np.not_equal(keys[1:], keys[:-1], out=keep[1:])
    return keys[keep]


def sbm(n_blocks: int, block_size: int, avg_degree: float, ratio: float, seed: int):
    """Stochastic block model with equal blocks laid out as contiguous id ranges.

    ``ratio`` = p_in / p_out; the two probabilities are solved from the wanted
    average degree: avg = p_in (b - 1) + p_out (n - b).
    Returns (rowptr, col, block) with block[v] = v // block_size.
    """
    n = n_blocks * block_size
    p_out = avg_degree / (ratio * (block_size - 1) + (n - block_size))
    p_in = ratio * p_out
    rng = _rng(seed)
    los, his = [], []
    for a in range(n_blocks):
        for b in range(a, n_blocks):
            p = p_in if a == b else p_out
            # number of candidate pairs in this block pair, then a binomial
            # count and that many distinct pair indices
            pairs = block_size * (block_size - 1) // 2 if a == b else block_size * block_size
            k = int(rng.binomial(pairs, p))
            if k == 0:
                continue
            idx = rng.choice(pairs, size=k, replace=False)
            if a == b:
                # unrank idx into (i < j) inside the block
                i = np.floor((np.sqrt(8.0 * idx + 1.0) + 1.0) / 2.0).astype(np.int64)
                # guard the float unranking at triangle boundaries
                i = np.where(i * (i - 1) // 2 > idx, i - 1, i)
                i = np.where((i + 1) * i // 2 <= idx, i + 1, i)
                j = idx - i * (i - 1) // 2
                lo_, hi_ = j + a * block_size, i + a * block_size
            else:
                lo_ = idx // block_size + a * block_size
                hi_ = idx % block_size + b * block_size
            los.append(lo_.astype(np.int64))
            his.append(hi_.astype(np.int64))
    lo = np.concatenate(los) if los else np.zeros(0, np.int64)
    hi = np.concatenate(his) if his else np.zeros(0, np.int64)
    rowptr, col = csr_from_undirected(n, lo, hi)
    block = (np.arange(n) // block_size).astype(np.int32)
    return rowptr, col, block


def _pareto_weights(n: int, gamma: float, total: float, rng: np.random.Generator) -> np.ndarray:
    """Expected degrees w ~ Pareto(tail exponent gamma), capped at sqrt(total),
    scaled so that sum(w) = total."""
    u = rng.random(n)
    shape = gamma - 1.0
    base = (1.0 - u) ** (-1.0 / shape)  # Pareto with minimum 1
    cap = np.sqrt(total)
    lo, hi = 1e-6, total
    for _ in range(200):  # bisection on the minimum weight
        mid = 0.5 * (lo + hi)
        s = np.minimum(base * mid, cap).sum()
        if s < total:
            lo = mid
        else:
            hi = mid
    return np.minimum(base * hi, cap)


def chung_lu_communities(n: int, target_nnz: int, gamma: float, n_comm: int, mu: float, seed: int):
    """Chung-Lu power-law graph whose ids are ordered by community.

    Communities are ``n_comm`` contiguous id ranges of near-equal size.  Every
    undirected edge draws endpoint u with probability proportional to w_u and
    endpoint v proportional to w_v inside u's community with probability ``mu``,
    over the whole graph otherwise.  Loops and repeats are dropped; drawing goes
    on until at least ``target_nnz / 2`` distinct pairs exist and a seeded
    subset of exactly that many is kept.
    Returns (rowptr, col, community).
    """
    rng = _rng(seed)
    want = int(target_nnz) // 2
    w = _pareto_weights(n, gamma, float(target_nnz), rng)
    bounds = (np.arange(n_comm + 1, dtype=np.int64) * n) // n_comm
    community = (np.searchsorted(bounds, np.arange(n), side="right") - 1).astype(np.int32)
    cw = np.concatenate([[0.0], np.cumsum(w)])
    c_lo = cw[bounds[:-1]]
    c_hi = cw[bounds[1:]]
    prob = w / w.sum()
    have = np.zeros(0, dtype=np.int64)
    deficit = want
    rounds = 0
    while have.size < want:
        rounds += 1
        if rounds > 64:
            raise RuntimeError("graph too dense for the requested nnz")
        draw = int(deficit * 1.25) + 1024
        # endpoint u: a multinomial count per vertex (sorted by construction)
        u = np.repeat(np.arange(n, dtype=np.int64), rng.multinomial(draw, prob))
        cu = community[u]
        inside = rng.random(draw) < mu
        r = rng.random(draw)
        q = np.where(inside, c_lo[cu] + r * (c_hi[cu] - c_lo[cu]), r * cw[-1])
        v = np.searchsorted(cw, q, side="right") - 1
        np.clip(v, 0, n - 1, out=v)
        ok = u != v
        lo = np.minimum(u, v)[ok]
        hi = np.maximum(u, v)[ok]
        have = _dedupe_sorted(np.concatenate([have, lo * np.int64(n) + hi]))
        deficit = max(want - have.size, 0)
    if have.size > want:
        drop = rng.choice(have.size, size=have.size - want, replace=False)
        keep = np.ones(have.size, dtype=bool)
        keep[drop] = False
        have = have[keep]
    lo = have // np.int64(n)
    hi = have - lo * np.int64(n)
    rowptr, col = csr_from_undirected(n, lo, hi)
    return rowptr, col, community


def permutation_graph(n: int, k: int, seed: int):
    """Near-regular graph without locality: the union of ``k`` seeded random
    permutations (v, pi_j(v)), symmetrised, loops and repeats dropped; degrees
    come out close to 2k."""
    rng = _rng(seed)
    base = np.arange(n, dtype=np.int64)
    keys = []
    for _ in range(k):
        pi = rng.permutation(n).astype(np.int64)
        ok = pi != base
        lo = np.minimum(base, pi)[ok]
        hi = np.maximum(base, pi)[ok]
        keys.append(lo * np.int64(n) + hi)
    have = _dedupe_sorted(np.concatenate(keys))
    lo = have // np.int64(n)
    hi = have - lo * np.int64(n)
    return csr_from_undirected(n, lo, hi)


def from_edge_list(n: int, edges):
    """Small hand-written graphs for tests: iterable of undirected (a, b)."""
    e = np.asarray(list(edges), dtype=np.int64).reshape(-1, 2)
    lo = np.minimum(e[:, 0], e[:, 1])
    hi = np.maximum(e[:, 0], e[:, 1])
    ok = lo != hi
    keys = _dedupe_sorted(lo[ok] * np.int64(n) + hi[ok])
    lo = keys // np.int64(n)
    hi = keys - lo * np.int64(n)
    return csr_from_undirected(n, lo, hi)


def erdos_renyi(n: int, p: float, seed: int):
    """G(n, p) for small test graphs (dense Bernoulli draw)."""
    rng = _rng(seed)
    upper = np.triu(rng.random((n, n)) < p, k=1)
    lo, hi = np.nonzero(upper)
    return csr_from_undirected(n, lo.astype(np.int64), hi.astype(np.int64))


def cut_fraction(rowptr: np.ndarray, col: np.ndarray, part: np.ndarray) -> float:
    """Share of directed non-zeros whose endpoints lie in different parts."""
    n = rowptr.size - 1
    src = np.repeat(np.arange(n), np.diff(rowptr))
    if col.size == 0:
        return 0.0
    return float(np.count_nonzero(part[src] != part[col])) / float(col.size)
