"""Named synthetic workloads: graph + features + labels + mask + initial weights.

The shapes, sizes and value distributions follow the paper's two datasets
(Table 1: a dense 233K-vertex graph with 602 features and 41 labels; a sparse
2.4M-vertex graph with 100 features) and its hyper-parameters (Section 4.1: two
layers, 128 hidden units, Adam, learning rate 0.02).  The datasets themselves
are not available, so seeded random graphs stand in for them.

Only inputs are made here.  Partitioning, sampling, normalization and training
are the business of the code under test and of its checker.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

from . import graphs

BASE_SEED = 20201204
# sub-streams of the base seed
S_GRAPH, S_FEAT, S_LABEL, S_WEIGHT, S_PART = 1, 2, 3, 4, 5

PART_RANGE, PART_HASH, PART_USER = 0, 1, 2


@dataclass
class Workload:
    name: str
    n: int
    rowptr: np.ndarray          # int64 [n+1]
    col: np.ndarray             # int32 [nnz]
    x: np.ndarray               # float32 [n, f]
    y: np.ndarray               # int32 [n]
    train_mask: np.ndarray      # uint8 [n]
    dims: list                  # [f, hidden..., c]
    w0: list                    # float32 [dims[l], dims[l+1]] per layer
    b0: list                    # float32 [dims[l+1]] per layer
    m: int                      # number of partitions M
    overlap_ppm: int            # overlap threshold O of Algorithm 1, in parts per million
    part_mode: int
    user_part: np.ndarray | None
    seed: int                   # seed of the partition / sampling keys
    lr: float
    epochs: int
    beta1: float = 0.9
    beta2: float = 0.999
    eps: float = 1e-8
    loss_on_halo: int = 1
    stats: dict = field(default_factory=dict)

    @property
    def nnz(self) -> int:
        return int(self.col.size)


def class_features(cls: np.ndarray, n_classes: int, f: int, seed: int, mean_scale: float = 0.5) -> np.ndarray:
    """x_v = mu_{class(v)} + N(0, I_f), mu_c ~ mean_scale * N(0, I_f); float32."""
    rng = graphs._rng(seed)
    mu = (mean_scale * rng.standard_normal((n_classes, f))).astype(np.float32)
    x = rng.standard_normal((cls.size, f), dtype=np.float32)
    x += mu[cls]
    return x


def bernoulli_mask(n: int, p: float, seed: int) -> np.ndarray:
    return (graphs._rng(seed).random(n) < p).astype(np.uint8)


def noisy_labels(cls: np.ndarray, n_classes: int, noise: float, seed: int) -> np.ndarray:
    rng = graphs._rng(seed)
    y = cls.astype(np.int32).copy()
    flip = rng.random(y.size) < noise
    y[flip] = rng.integers(0, n_classes, size=int(flip.sum()), dtype=np.int32)
    return y


def glorot(dims, seed: int):
    """Glorot-uniform weights, zero biases (float32)."""
    rng = graphs._rng(seed)
    w0, b0 = [], []
    for fi, fo in zip(dims[:-1], dims[1:]):
        lim = np.sqrt(6.0 / (fi + fo))
        w0.append(rng.uniform(-lim, lim, size=(fi, fo)).astype(np.float32))
        b0.append(np.zeros(fo, dtype=np.float32))
    return w0, b0


def _finish(name, rowptr, col, cls, n_classes, f, hidden, m, overlap_ppm, part_mode, user_part,
            lr, epochs, mask_p, label_noise, seed, stats=None) -> Workload:
    n = rowptr.size - 1
    x = class_features(cls, n_classes, f, seed + S_FEAT)
    y = noisy_labels(cls, n_classes, label_noise, seed + S_LABEL)
    mask = bernoulli_mask(n, mask_p, seed + S_LABEL + 1000)
    dims = [f] + list(hidden) + [n_classes]
    w0, b0 = glorot(dims, seed + S_WEIGHT)
    st = dict(stats or {})
    deg = np.diff(rowptr)
    st.update(n=int(n), nnz=int(col.size), avg_degree=float(col.size) / max(n, 1),
              max_degree=int(deg.max()) if n else 0, min_degree=int(deg.min()) if n else 0)
    return Workload(name, n, rowptr, col, x, y, mask, dims, w0, b0, m, overlap_ppm, part_mode,
                    user_part, seed + S_PART, lr, epochs, stats=st)


def tiny(seed: int = BASE_SEED) -> Workload:
    """5-block SBM, 2 000 vertices, average degree 8, 64 features, 5 classes,
    hidden 16, two partitions by community block, 10 epochs at lr 0.01."""
    rowptr, col, block = graphs.sbm(5, 400, 8.0, 10.0, seed + S_GRAPH)
    user = ((block.astype(np.int64) * 2) // 5).astype(np.int32)  # blocks {0,1,2} | {3,4}
    return _finish("tiny", rowptr, col, block, 5, 64, [16], 2, 100_000, PART_USER, user,
                   0.01, 10, 0.5, 0.0, seed)


def small(seed: int = BASE_SEED) -> Workload:
    """20-block SBM, 20 000 vertices, average degree 20, 500 features, 20
    classes, hidden 64, four range partitions, 50 epochs."""
    rowptr, col, block = graphs.sbm(20, 1000, 20.0, 10.0, seed + S_GRAPH)
    return _finish("small", rowptr, col, block, 20, 500, [64], 4, 100_000, PART_RANGE, None,
                   0.02, 50, 0.5, 0.0, seed)


def power_law(name: str, n: int, target_nnz: int, f: int, n_classes: int, hidden, m: int, epochs: int,
              n_comm: int, mu: float = 0.86, gamma: float = 2.1, overlap_ppm: int = 100_000,
              seed: int = BASE_SEED) -> Workload:
    rowptr, col, comm = graphs.chung_lu_communities(n, target_nnz, gamma, n_comm, mu, seed + S_GRAPH)
    cls = (comm % n_classes).astype(np.int32)
    part = ((np.arange(n, dtype=np.int64) * m) // n).astype(np.int32)
    stats = {"cut_fraction_range": graphs.cut_fraction(rowptr, col, part), "communities": n_comm, "mu": mu,
             "gamma": gamma}
    return _finish(name, rowptr, col, cls, n_classes, f, hidden, m, overlap_ppm, PART_RANGE, None,
                   0.02, epochs, 0.66, 0.03, seed, stats)


def paper_scale(seed: int = BASE_SEED, scale: float = 1.0) -> Workload:
    """232 965 vertices, 114.6 M directed non-zeros (average degree about 492),
    602 features, 41 classes, hidden 128, five partitions.  ``scale`` < 1
    shrinks the vertex count by ``scale`` and the average degree by its square
    root, for tests."""
    n = int(round(232_965 * scale))
    nnz = int(round(114_600_000 * scale ** 1.5))
    # 41 communities and mu = 0.94: after duplicate rejection inside the dense
    # communities a five-way range split cuts about 11 % of the edges, the
    # share the paper reports for its 233K-vertex dataset (Section 1).
    return power_law("paper_scale" if scale == 1.0 else f"paper_scale_x{scale:g}", n, nnz, 602, 41, [128], 5,
                     200, 41, mu=0.94, seed=seed)


def large_sparse(seed: int = BASE_SEED, scale: float = 1.0) -> Workload:
    """2.45 M vertices, 123.7 M directed non-zeros (average degree about 50),
    100 features, 47 classes, three layers with hidden 256, ten partitions."""
    n = int(round(2_450_000 * scale))
    nnz = int(round(123_700_000 * scale ** 1.5))
    n_comm = max(47, int(round(1504 * scale / 47.0)) * 47)
    return power_law("large_sparse" if scale == 1.0 else f"large_sparse_x{scale:g}", n, nnz, 100, 47, [256, 256],
                     10, 100, n_comm, seed=seed)


def sweep_graph(graph: str, seed: int = BASE_SEED, scale: float = 1.0):
    """The graph of a sweep point: ("paper" | "regular") -> (rowptr, col, cls_source)."""
    if graph == "paper":
        n = int(round(232_965 * scale))
        rowptr, col, comm = graphs.chung_lu_communities(n, int(round(114_600_000 * scale ** 1.5)), 2.1, 41, 0.94,
                                                        seed + S_GRAPH)
        return rowptr, col, comm
    if graph == "regular":
        n = int(round(1_000_000 * scale))
        rowptr, col = graphs.permutation_graph(n, 16, seed + S_GRAPH)
        return rowptr, col, np.arange(n, dtype=np.int64)
    raise ValueError(graph)


def sweep_point(graph: str, width: int, m: int, seed: int = BASE_SEED, scale: float = 1.0, prebuilt=None) -> Workload:
    """One point of the SpMM/GEMM sweep: a single GCN layer of equal input and
    output width on the paper-scale graph or on the degree-32 random graph.
    ``prebuilt`` = result of sweep_graph, to reuse one graph for several widths."""
    rowptr, col, src = prebuilt if prebuilt is not None else sweep_graph(graph, seed, scale)
    cls = (src % min(width, 32)).astype(np.int32)
    return _finish(f"sweep_{graph}_f{width}_m{m}", rowptr, col, cls, width, width, [], m, 100_000 if m > 1 else 0,
                   PART_RANGE, None, 0.02, 1, 0.66, 0.0, seed)


def sage_weights(dims, seed: int):
    """Initial parameters of the two-layer mean-aggregator model: per layer a self and a neighbour matrix
    (Glorot-uniform over the stacked [2 din x dout] matrix) and a zero bias (float32)."""
    rng = graphs._rng(seed)
    w_self, w_neigh, b = [], [], []
    for fi, fo in zip(dims[:-1], dims[1:]):
        lim = np.sqrt(6.0 / (2 * fi + fo))
        w_self.append(rng.uniform(-lim, lim, size=(fi, fo)).astype(np.float32))
        w_neigh.append(rng.uniform(-lim, lim, size=(fi, fo)).astype(np.float32))
        b.append(np.zeros(fo, dtype=np.float32))
    return w_self, w_neigh, b


def by_name(name: str, **kw) -> Workload:
    return {"tiny": tiny, "small": small, "paper_scale": paper_scale, "large_sparse": large_sparse}[name](**kw)
