"""Pins for the checker's graph steps: selection key, partition assignment,
Algorithm 1 and the augmented partition graph.  Everything here is compared
with something other than the checker itself: printed values of the paper,
published test vectors, a hand-worked example, closed forms, or a dense
brute-force restatement on tiny graphs."""
import os

import numpy as np
import pytest

from gen import graphs
from oracle import oracle

GOLD = os.path.join(os.path.dirname(__file__), "golden")
M64 = (1 << 64) - 1


def _rows(name):
    with open(os.path.join(GOLD, name)) as fh:
        return [ln.split() for ln in fh if ln.strip() and not ln.startswith("#")]


# ----------------------------------------------------------------- key ---
def _mix_py(z):
    z ^= z >> 30
    z = (z * 0xBF58476D1CE4E5B9) & M64
    z ^= z >> 27
    z = (z * 0x94D049BB133111EB) & M64
    z ^= z >> 31
    return z


def _key_py(seed, w0, w1, w2, w3, v):
    h = _mix_py(seed)
    for w in (w0, w1, w2, w3):
        h = _mix_py(h ^ w)
    return _mix_py(h ^ v)


def test_mix_matches_published_splitmix64_vectors():
    want = [int(r[0], 16) for r in _rows("splitmix64_vectors.txt")]
    got = [_mix_py(((i + 1) * 0x9E3779B97F4A7C15) & M64) for i in range(3)]
    assert got == want
    # the C key is that mix applied word by word
    for args in [(0, 0, 0, 0, 0, 0), (20201209, 2, 1, 4, 3, 99), (M64, M64, 5, 6, 7, 123456789)]:
        assert oracle.key(*args) == _key_py(*args)


def test_key_is_injective_and_spread():
    ks = np.array([oracle.key(7, 2, 0, 1, 1, v) for v in range(4096)], dtype=np.uint64)
    assert np.unique(ks).size == ks.size
    # top byte roughly uniform: chi-square with 255 dof, mean 255, sd about 22.6
    counts = np.bincount((ks >> np.uint64(56)).astype(np.int64), minlength=256)
    chi2 = ((counts - 16.0) ** 2 / 16.0).sum()
    assert chi2 < 255 + 6 * 22.6


# ----------------------------------------------------------- partition ---
@pytest.mark.parametrize("n,m", [(10, 3), (2000, 7), (5, 5), (17, 1)])
def test_range_partition_is_balanced_and_monotone(n, m):
    part = oracle.partition(n, m, oracle.PART_RANGE)
    sizes = np.bincount(part, minlength=m)
    assert sizes.sum() == n and sizes.max() - sizes.min() <= 1
    assert np.all(np.diff(part) >= 0)
    assert abs(sizes - n / m).max() < 1


def test_hash_partition_is_a_balanced_permutation_cut():
    n, m = 1001, 4
    part = oracle.partition(n, m, oracle.PART_HASH, seed=11)
    sizes = np.bincount(part, minlength=m)
    assert sizes.max() - sizes.min() <= 1
    # independent restatement: rank by key, cut ranks with floor(r m / n)
    ks = [_key_py(11, 1, 0, 0, 0, v) for v in range(n)]
    order = sorted(range(n), key=lambda v: ks[v])
    want = np.empty(n, dtype=np.int32)
    for r, v in enumerate(order):
        want[v] = (r * m) // n
    assert np.array_equal(part, want)
    assert not np.array_equal(part, oracle.partition(n, m, oracle.PART_HASH, seed=12))


def test_user_partition_is_copied_and_checked():
    u = np.array([1, 0, 1, 1, 0], dtype=np.int32)
    assert np.array_equal(oracle.partition(5, 2, oracle.PART_USER, user=u), u)
    with pytest.raises(ValueError):
        oracle.partition(5, 2, oracle.PART_USER, user=np.array([0, 2, 0, 0, 0], dtype=np.int32))


# ----------------------------------------------------------------- nts ---
def test_nts_reproduces_the_papers_overhead_figures():
    """Section 3.1 example and the overhead column of Tables 2 and 4."""
    n_total = 6_000_000  # divisible by 3, 5, 20 and large enough for the printed digits
    for m, o, per_op, overhead, digits in _rows("overhead_table.txt"):
        m, o, per_op, overhead, digits = int(m), float(o), float(per_op), float(overhead), int(digits)
        n_p = n_total // m
        k = oracle.nts(n_p, m, int(round(o * 10_000)))
        assert abs(100.0 * k / n_p - per_op) < 1e-3
        got = 100.0 * (m - 1) * k * m / (n_total * m)   # all halos of all partitions / (M N)
        # the paper truncates or rounds to the digits it prints
        assert abs(got - overhead) <= 0.5 * 10 ** (-digits) + 0.05


def test_nts_floor_and_single_partition():
    assert oracle.nts(4, 2, 500_000) == 2
    assert oracle.nts(7, 3, 100_000) == 0          # 0.35 -> 0
    assert oracle.nts(1000, 1, 500_000) == 0       # M = 1: nothing to sample from
    assert oracle.nts(46593, 5, 100_000) == 1164


# --------------------------------------------------------- Algorithm 1 ---
def _path8():
    return graphs.from_edge_list(8, [(i, i + 1) for i in range(7)])


def test_hand_worked_path_example():
    rows = {r[0]: [int(x) for x in r[1:]] for r in _rows("path8_example.txt")}
    rowptr, col = _path8()
    part, parts = oracle.build_partitions(rowptr, col, 2, 500_000, seed=3, mode=oracle.PART_RANGE)
    assert part.tolist() == [0, 0, 0, 0, 1, 1, 1, 1]
    assert parts[0].members.tolist() == rows["p0_members"]
    assert parts[1].members.tolist() == rows["p1_members"]
    assert parts[0].depth_by_op[1] == rows["depth"][0] and parts[1].depth_by_op[0] == rows["depth"][0]
    # the same for any seed: no draw is left to chance in this example
    for seed in range(5):
        _, q = oracle.build_partitions(rowptr, col, 2, 500_000, seed=seed)
        assert q[0].members.tolist() == rows["p0_members"]


def _brute_levels(adj, part, p, op):
    """BFS levels of op seen from p via dense boolean algebra."""
    in_p, in_op = part == p, part == op
    seen = np.zeros(adj.shape[0], dtype=bool)
    level = (adj[in_p].any(axis=0)) & in_op
    out = []
    while level.any():
        out.append(np.flatnonzero(level))
        seen |= level
        level = adj[level].any(axis=0) & in_op & ~seen
    return out


def _brute_sample(adj, part, p, op, k, seed):
    taken, depth = [], 0
    for lvl_no, lvl in enumerate(_brute_levels(adj, part, p, op), start=1):
        if k <= 0:
            break
        depth = lvl_no
        if lvl.size >= k:
            ks = sorted(lvl.tolist(), key=lambda v: _key_py(seed, 2, p, op, lvl_no, v))
            taken += ks[:k]
            k = 0
        else:
            taken += lvl.tolist()
            k -= lvl.size
    return sorted(taken), depth


@pytest.mark.parametrize("n,prob,m,o_ppm,seed,expect_multi", [
    (40, 0.08, 2, 500_000, 1, False), (64, 0.04, 3, 900_000, 2, False), (48, 0.03, 4, 1_000_000, 3, True),
    (30, 0.30, 3, 400_000, 4, False), (64, 0.02, 2, 2_000_000, 5, True), (50, 0.05, 5, 1_200_000, 6, False),
    (64, 0.03, 2, 1_000_000, 7, True), (30, 0.30, 3, 100_000, 4, False),
])
def test_algorithm1_against_dense_brute_force(n, prob, m, o_ppm, seed, expect_multi):
    rowptr, col = graphs.erdos_renyi(n, prob, 100 + seed)
    adj = np.zeros((n, n), dtype=bool)
    adj[np.repeat(np.arange(n), np.diff(rowptr)), col] = True
    for mode in (oracle.PART_RANGE, oracle.PART_HASH):
        part, parts = oracle.build_partitions(rowptr, col, m, o_ppm, seed=seed, mode=mode)
        multi_level = False
        for pt in parts:
            assert np.array_equal(pt.owned, np.flatnonzero(part == pt.p))
            k = (o_ppm * pt.n_owned) // (1_000_000 * (m - 1))
            assert pt.nts == k
            halo_all = []
            for op in range(m):
                if op == pt.p:
                    continue
                want, depth = _brute_sample(adj, part, pt.p, op, k, seed)
                assert pt.halo_by_op[op].tolist() == want
                assert pt.depth_by_op[op] == depth
                multi_level |= depth > 1
                # invariants: inside op, size = min(nts, reachable), whole earlier levels
                reach = _brute_levels(adj, part, pt.p, op)
                n_reach = sum(l.size for l in reach)
                assert len(want) == min(k, n_reach)
                assert all(part[v] == op for v in want)
                got = set(want)
                for lvl in reach[:max(depth - 1, 0)]:
                    assert set(lvl.tolist()) <= got
                halo_all += want
            assert len(set(halo_all)) == len(halo_all)
            assert pt.members.tolist() == pt.owned.tolist() + sorted(halo_all)
        if expect_multi:
            assert multi_level  # the sparse cases must exercise the recursive branch


def test_zero_overlap_and_single_partition_add_nothing():
    rowptr, col = graphs.erdos_renyi(30, 0.2, 9)
    _, parts = oracle.build_partitions(rowptr, col, 3, 0, seed=1)
    assert all(pt.n == pt.n_owned for pt in parts)
    _, parts = oracle.build_partitions(rowptr, col, 1, 500_000, seed=1)
    assert parts[0].n == 30 and parts[0].nts == 0


def test_saturated_overlap_on_connected_graph_gives_whole_graph():
    """M = 2, connected G, nts >= |op|: both augmented partitions are all of G."""
    n = 24
    rowptr, col = graphs.from_edge_list(n, [(i, (i + 1) % n) for i in range(n)] + [(0, 12), (3, 17)])
    _, parts = oracle.build_partitions(rowptr, col, 2, 1_000_000, seed=5)
    for pt in parts:
        assert sorted(pt.members.tolist()) == list(range(n))
        assert pt.nnz == col.size + n


def test_unreachable_partition_contributes_nothing():
    # two components: {0..3} path and {4..7} path; partitions = components
    rowptr, col = graphs.from_edge_list(8, [(0, 1), (1, 2), (2, 3), (4, 5), (5, 6), (6, 7)])
    _, parts = oracle.build_partitions(rowptr, col, 2, 1_000_000, seed=5)
    assert parts[0].members.tolist() == [0, 1, 2, 3] and parts[0].depth_by_op[1] == 0


def test_last_level_choice_is_uniform_over_seeds():
    """Star from partition 0 into 12 vertices of partition 1; draw 3 of them."""
    n = 16
    edges = [(0, 4 + j) for j in range(12)] + [(1, 2), (2, 3), (0, 1)]
    rowptr, col = graphs.from_edge_list(n, edges)
    user = np.array([0] * 4 + [1] * 12, dtype=np.int32)
    counts = np.zeros(n, dtype=np.int64)
    trials = 2000
    for seed in range(trials):
        _, parts = oracle.build_partitions(rowptr, col, 2, 750_000, seed=seed, mode=oracle.PART_USER, user=user)
        h = parts[0].halo_by_op[1]
        assert h.size == 3
        counts[h] += 1
    expect = trials * 3 / 12.0
    chi2 = ((counts[4:] - expect) ** 2 / expect).sum()
    assert counts[:4].sum() == 0
    assert chi2 < 11 + 6 * np.sqrt(22)  # 11 dof (loose: the draws within a seed are dependent)


def test_overhead_identity_when_unsaturated(small_wl):
    """Each halo holds (M-1) nts vertices, i.e. an overhead of O / M of N per
    partition (the paper's 2 % at M = 5, O = 10 %)."""
    w = small_wl
    _, parts = oracle.build_partitions(w.rowptr, w.col, w.m, w.overlap_ppm, w.seed, w.part_mode)
    halo = sum(pt.n - pt.n_owned for pt in parts)
    assert halo == sum((w.m - 1) * pt.nts for pt in parts)
    for pt in parts:
        assert abs((pt.n - pt.n_owned) / w.n - 0.1 / w.m) < 1e-3


# ---------------------------------------------- augmented partition graph ---
def _dense_ahat(adj_sub):
    a = adj_sub.astype(np.float64) + np.eye(adj_sub.shape[0])
    d = a.sum(axis=1)
    return a / np.sqrt(np.outer(d, d))


def _to_dense(rp, cc, vv, n):
    a = np.zeros((n, n))
    a[np.repeat(np.arange(n), np.diff(rp)), cc] = vv
    return a


@pytest.mark.parametrize("seed", [1, 2, 3])
def test_induced_graph_and_weights_against_dense(seed):
    n = 60
    rowptr, col = graphs.erdos_renyi(n, 0.1, seed)
    adj = np.zeros((n, n), dtype=bool)
    adj[np.repeat(np.arange(n), np.diff(rowptr)), col] = True
    _, parts = oracle.build_partitions(rowptr, col, 3, 600_000, seed=seed, mode=oracle.PART_HASH)
    for pt in parts:
        s = pt.members
        want = _dense_ahat(adj[np.ix_(s, s)])
        got = _to_dense(pt.rowptr, pt.col, pt.val, pt.n)
        assert np.allclose(got, want, rtol=0, atol=1e-15)
        assert np.array_equal(got != 0, want != 0)
        # columns ascend, self-loop present, nnz = 2 E + n
        for i in range(pt.n):
            c = pt.col[pt.rowptr[i]:pt.rowptr[i + 1]]
            assert np.all(np.diff(c) > 0) and i in c
        assert pt.nnz == 2 * int(np.triu(adj[np.ix_(s, s)], 1).sum()) + pt.n
        # the real transpose equals the matrix itself on symmetric input
        assert np.array_equal(pt.t_rowptr, pt.rowptr) and np.array_equal(pt.t_col, pt.col)
        assert np.array_equal(pt.t_val, pt.val)
        # A_hat sqrt(d) = sqrt(d): eigenvalue 1
        d = np.diff(pt.rowptr).astype(np.float64)
        assert np.allclose(got @ np.sqrt(d), np.sqrt(d), atol=1e-12)


def test_transpose_of_a_non_symmetric_matrix():
    rp = np.array([0, 2, 3, 3], dtype=np.int64)
    cc = np.array([1, 3, 0], dtype=np.int64)
    vv = np.array([1.0, 2.0, 3.0])
    trp, tc, tv = oracle.transpose(3, 4, rp, cc, vv)
    dense = np.zeros((3, 4)); dense[0, 1], dense[0, 3], dense[1, 0] = 1, 2, 3
    got = np.zeros((4, 3)); got[np.repeat(np.arange(4), np.diff(trp)), tc] = tv
    assert np.array_equal(got, dense.T)


def test_normalization_closed_forms():
    # complete graph K_6: every entry 1/6
    n = 6
    rowptr, col = graphs.from_edge_list(n, [(i, j) for i in range(n) for j in range(i + 1, n)])
    rp, cc, vv = oracle.induced(rowptr, col, np.arange(n))
    assert vv.size == n * n and np.allclose(vv, 1.0 / n, atol=1e-16)
    # cycle (2-regular): (A + I) / 3, row sums 1
    n = 9
    rowptr, col = graphs.from_edge_list(n, [(i, (i + 1) % n) for i in range(n)])
    rp, cc, vv = oracle.induced(rowptr, col, np.arange(n))
    assert np.allclose(vv, 1.0 / 3.0, atol=1e-16)
    assert np.allclose(np.add.reduceat(vv, rp[:-1]), 1.0)
    # path of six, the augmented partition of the hand-worked example
    rowptr, col = _path8()
    _, parts = oracle.build_partitions(rowptr, col, 2, 500_000, seed=0)
    a = _to_dense(parts[0].rowptr, parts[0].col, parts[0].val, 6)
    assert abs(a[0, 0] - 0.5) < 1e-15 and abs(a[0, 1] - 1 / np.sqrt(6)) < 1e-15
    assert abs(a[1, 1] - 1 / 3) < 1e-15 and abs(a[1, 2] - 1 / 3) < 1e-15
    assert np.array_equal(a, a.T)


def test_degrees_are_counted_inside_the_augmented_partition():
    # star: centre 0 with leaves 1..5; partition {0,1,2} | {3,4,5}, no overlap:
    # inside partition 0 the centre has degree 2 (+1 self-loop), not 5
    rowptr, col = graphs.from_edge_list(6, [(0, j) for j in range(1, 6)])
    _, parts = oracle.build_partitions(rowptr, col, 2, 0, seed=0)
    a = _to_dense(parts[0].rowptr, parts[0].col, parts[0].val, 3)
    assert abs(a[0, 0] - 1 / 3) < 1e-15 and abs(a[0, 1] - 1 / np.sqrt(6)) < 1e-15
    # partition 1 holds three isolated leaves: identity
    assert np.array_equal(_to_dense(parts[1].rowptr, parts[1].col, parts[1].val, 3), np.eye(3))


def test_validate_rejects_bad_graphs():
    oracle.validate(*_path8())
    with pytest.raises(ValueError):      # not symmetric
        oracle.validate(np.array([0, 1, 1], dtype=np.int64), np.array([1], dtype=np.int32))
    with pytest.raises(ValueError):      # self-loop
        oracle.validate(np.array([0, 1], dtype=np.int64), np.array([0], dtype=np.int32))


def test_spmm_against_dense():
    rng = np.random.default_rng(0)
    rowptr, col = graphs.erdos_renyi(37, 0.2, 4)
    rp, cc, vv = oracle.induced(rowptr, col, np.arange(37))
    x = rng.standard_normal((37, 5))
    assert np.allclose(oracle.spmm(rp, cc, vv, x), _to_dense(rp, cc, vv, 37) @ x, atol=1e-14)
