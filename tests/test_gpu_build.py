"""GPU parity of gcnsa_build_partitions run in CUDA kernels (the default builder).

Two comparisons, both bit-exact (integer, index and byte work):
  * against the fp64 checker: partition assignment, the vertex sets Algorithm 1
    selects, BFS depths, CSR and transposed CSR of every extended partition,
    the number of loss-carrying vertices;
  * against the library's host-side builder, which the CPU suite pins to the
    checker: everything above plus the scheduling structures only the library
    has (row orders, hub-row counts, loss rows, transposed CSR over the loss
    columns), labels, masks and the gathered feature rows.
Cases cover range / hash / caller-given assignments, no overlap, saturated
overlap, deep breadth-first walks (paths, rings), one partition, partitions
another cannot reach, both loss_on_halo settings, and the error codes of the
device-side input checks."""
import numpy as np
import pytest
import torch

from gen import configs, graphs
from oracle import oracle
from paper_2012_04930_b200 import gcnsa

pytestmark = pytest.mark.gpu


def _build(builder, rowptr, col, x, y, mask, c, m, o_ppm, seed, mode, user, loh):
    env = gcnsa.make_env(0)
    return gcnsa.Parts(env, rowptr, col, x, y, mask, c, m, o_ppm, seed, mode, user, loh, builder=builder)


def _against_checker(parts, rowptr, col, m, o_ppm, seed, mode, user, mask, loh):
    part, ref = oracle.build_partitions(rowptr, col, m, o_ppm, seed, mode, user)
    assert np.array_equal(parts.assignment(), part)
    for p, pt in enumerate(ref):
        i = parts.info(p)
        e = parts.export(p)
        assert (i.n_owned, i.n_halo, i.n, i.nnz, i.nts) == (pt.n_owned, pt.n - pt.n_owned, pt.n, pt.nnz, pt.nts)
        assert np.array_equal(e["members"], pt.members)
        for k in ("rowptr", "col", "t_rowptr", "t_col"):
            assert np.array_equal(e[k], getattr(pt, k)), (p, k)
        for op in range(m):
            assert e["depth"][op] == (0 if op == p else pt.depth_by_op[op]), (p, op)
        assert i.max_depth == max([0] + list(pt.depth_by_op.values()))
        assert i.n_train == int(oracle.train_set(pt, mask[pt.members], loh).sum())
        if pt.val.size:      # an empty partition has no entries
            assert np.abs(e["val"] - pt.val).max() <= 2e-7 * pt.val.max()
            assert np.abs(e["t_val"] - pt.t_val).max() <= 2e-7 * pt.t_val.max()


def _same(dev, host, m):
    assert np.array_equal(dev.assignment(), host.assignment())
    for p in range(m):
        a, b = dev.info(p), host.info(p)
        for k in ("n_owned", "n_halo", "n", "nnz", "nts", "n_train", "max_depth"):
            assert getattr(a, k) == getattr(b, k), (p, k, getattr(a, k), getattr(b, k))
        ea, eb = dev.export(p), host.export(p)
        for k in ea:
            assert np.array_equal(ea[k], eb[k]), (p, k)      # values too: same kernel, same inputs
        sa, sb = dev.export_schedule(p), host.export_schedule(p)
        for k in sa:
            assert np.array_equal(sa[k], sb[k]), (p, k)
        assert np.array_equal(dev.features(p), host.features(p)), p


def _case(rowptr, col, m, o_ppm, seed, mode, user=None, loh=1, f=5, c=4):
    n = rowptr.size - 1
    rng = np.random.default_rng(1000 + seed)
    x = rng.standard_normal((n, f)).astype(np.float32)
    y = rng.integers(0, c, n).astype(np.int32)
    mask = (rng.random(n) < 0.5).astype(np.uint8)
    dev = _build(gcnsa.BUILD_DEVICE, rowptr, col, x, y, mask, c, m, o_ppm, seed, mode, user, loh)
    host = _build(gcnsa.BUILD_HOST, rowptr, col, x, y, mask, c, m, o_ppm, seed, mode, user, loh)
    _against_checker(dev, rowptr, col, m, o_ppm, seed, mode, user, mask, loh)
    _same(dev, host, m)
    # the gathered rows are the caller's rows
    for p in range(m):
        assert np.array_equal(dev.features(p), x[dev.members(p)])
    dev.close(); host.close()


@pytest.mark.parametrize("n,prob,m,o_ppm,seed,mode", [
    (64, 0.03, 2, 1_000_000, 7, 0), (64, 0.02, 2, 2_000_000, 5, 1), (48, 0.03, 4, 1_000_000, 3, 1),
    (200, 0.02, 5, 500_000, 11, 0), (200, 0.01, 3, 3_000_000, 12, 1), (30, 0.3, 3, 100_000, 4, 0),
    (90, 0.05, 1, 500_000, 13, 0), (120, 0.04, 6, 0, 14, 1), (5000, 0.002, 7, 300_000, 15, 1),
    (3000, 0.004, 40, 900_000, 16, 1), (2600, 0.003, 33, 250_000, 17, 0),
])
def test_random_graphs(n, prob, m, o_ppm, seed, mode):
    rowptr, col = graphs.erdos_renyi(n, prob, 300 + seed)
    for loh in (1, 0):
        _case(rowptr, col, m, o_ppm, seed, mode, loh=loh)


@pytest.mark.parametrize("n,m,o_ppm", [(64, 2, 500_000), (1000, 4, 900_000), (257, 3, 2_000_000)])
def test_paths_and_rings_walk_many_levels(n, m, o_ppm):
    path = graphs.from_edge_list(n, [(i, i + 1) for i in range(n - 1)])
    ring = graphs.from_edge_list(n, [(i, (i + 1) % n) for i in range(n)])
    for rowptr, col in (path, ring):
        _case(rowptr, col, m, o_ppm, 21, gcnsa.PART_RANGE)
        _case(rowptr, col, m, o_ppm, 22, gcnsa.PART_HASH)


def test_unreachable_partition_and_isolated_vertices():
    # two components: partition 1 cannot be reached from partition 0; vertices 28..31 have no edges at all
    edges = [(i, i + 1) for i in range(0, 15)] + [(i, i + 1) for i in range(16, 27)]
    rowptr, col = graphs.from_edge_list(32, edges)
    _case(rowptr, col, 2, 1_000_000, 31, gcnsa.PART_RANGE)
    _case(rowptr, col, 4, 1_000_000, 32, gcnsa.PART_RANGE)


def test_caller_given_assignment_tiny(tiny_wl):
    w = tiny_wl
    dev = _build(gcnsa.BUILD_DEVICE, w.rowptr, w.col, w.x, w.y, w.train_mask, w.dims[-1], w.m, w.overlap_ppm, w.seed,
                 w.part_mode, w.user_part, w.loss_on_halo)
    host = _build(gcnsa.BUILD_HOST, w.rowptr, w.col, w.x, w.y, w.train_mask, w.dims[-1], w.m, w.overlap_ppm, w.seed,
                  w.part_mode, w.user_part, w.loss_on_halo)
    _against_checker(dev, w.rowptr, w.col, w.m, w.overlap_ppm, w.seed, w.part_mode, w.user_part, w.train_mask,
                     w.loss_on_halo)
    _same(dev, host, w.m)
    dev.close(); host.close()


@pytest.mark.parametrize("name,kw", [("small", {}), ("paper_scale", {"scale": 0.02}), ("large_sparse", {"scale": 0.02})])
def test_workloads(name, kw):
    w = configs.by_name(name, **kw)
    for mode, o_ppm in ((w.part_mode, w.overlap_ppm), (gcnsa.PART_HASH, 500_000)):
        user = w.user_part if mode == w.part_mode else None
        dev = _build(gcnsa.BUILD_DEVICE, w.rowptr, w.col, w.x, w.y, w.train_mask, w.dims[-1], w.m, o_ppm, w.seed, mode,
                     user, w.loss_on_halo)
        host = _build(gcnsa.BUILD_HOST, w.rowptr, w.col, w.x, w.y, w.train_mask, w.dims[-1], w.m, o_ppm, w.seed, mode,
                      user, w.loss_on_halo)
        _against_checker(dev, w.rowptr, w.col, w.m, o_ppm, w.seed, mode, user, w.train_mask, w.loss_on_halo)
        _same(dev, host, w.m)
        dev.close(); host.close()


def test_feature_rows_with_a_leading_dimension():
    """ldx > f on the caller's side: only the first f columns of every row are features."""
    rowptr, col = graphs.erdos_renyi(300, 0.03, 77)
    rng = np.random.default_rng(5)
    wide = rng.standard_normal((300, 11)).astype(np.float32)
    y = rng.integers(0, 3, 300).astype(np.int32)
    mask = np.ones(300, np.uint8)
    import ctypes as C
    L = gcnsa.lib()
    env = gcnsa.make_env(0)
    rp, cl = rowptr.astype(np.int64), col.astype(np.int32)
    g = gcnsa.Graph(n=300, nnz=cl.size, rowptr=rp.ctypes.data, col=cl.ctypes.data, f=7, x=wide.ctypes.data, ldx=11, c=3,
                    y=y.ctypes.data, train_mask=mask.ctypes.data)
    o = gcnsa.PartOpts(m=3, overlap_ppm=200_000, seed=9, part_mode=gcnsa.PART_RANGE, user_part=None, loss_on_halo=1,
                       builder=gcnsa.BUILD_DEVICE)
    h = C.c_void_p()
    assert L.gcnsa_build_partitions(C.byref(env), C.byref(g), C.byref(o), C.byref(h)) == 0
    for p in range(3):
        info = gcnsa.PartInfo()
        assert L.gcnsa_parts_info(h, p, C.byref(info)) == 0
        mem = np.empty(info.n, np.int64)
        ph = gcnsa.PartHost(members=mem.ctypes.data)
        assert L.gcnsa_parts_export(h, p, C.byref(ph)) == 0
        got = np.empty((info.n, 7), np.float32)
        assert L.gcnsa_parts_get_features(h, p, got.ctypes.data) == 0
        assert np.array_equal(got, wide[mem, :7])
    L.gcnsa_parts_destroy(h)


def test_device_side_input_checks_return_codes():
    x = np.zeros((3, 2), np.float32); y = np.zeros(3, np.int32); mk = np.ones(3, np.uint8)
    env = gcnsa.make_env(0)

    def code(rowptr, col, yy=y, **kw):
        args = dict(n_classes=2, m=1, overlap_ppm=0, seed=0)
        args.update(kw)
        with pytest.raises(gcnsa.GcnsaError) as ei:
            gcnsa.Parts(env, np.array(rowptr, np.int64), np.array(col, np.int32), x, yy, mk, **args)
        return ei.value.code

    assert code([0, 1, 1, 1], [1]) == gcnsa.ERR_NOT_SYMMETRIC
    assert code([0, 1, 1, 1], [0]) == gcnsa.ERR_SELF_LOOP_OR_DUP
    assert code([0, 2, 3, 4], [1, 1, 0, 0]) == gcnsa.ERR_SELF_LOOP_OR_DUP
    assert code([0, 2, 3, 4], [2, 1, 0, 0]) == gcnsa.ERR_ARG            # row not ascending
    assert code([0, 1, 2, 2], [1, 7]) == gcnsa.ERR_ARG                  # column out of range
    assert code([0, 2, 1, 2], [1, 0]) == gcnsa.ERR_ARG                  # row pointers decrease
    assert code([0, 1, 2, 2], [1, 0], m=4) == gcnsa.ERR_ARG             # more partitions than vertices
    assert code([0, 1, 2, 2], [1, 0], m=2, part_mode=gcnsa.PART_USER, user_part=np.array([0, 5, 0])) == gcnsa.ERR_LABEL_RANGE
    assert code([0, 1, 2, 2], [1, 0], yy=np.array([0, 3, 0], np.int32)) == gcnsa.ERR_LABEL_RANGE
    # and the context is still healthy: a valid build follows
    p = gcnsa.Parts(env, np.array([0, 1, 2, 2], np.int64), np.array([1, 0], np.int32), x, y, mk, 2, 1, 0, 0)
    assert p.info(0).n == 3 and p.info(0).nnz == 5
    p.close()
    torch.cuda.synchronize()


def test_empty_partition_and_edgeless_graph_build_and_train():
    """Degenerate inputs: a caller-given assignment that leaves partition 1 empty, and a graph without edges
    (every extended partition is then its owned vertices with self-loops only).  Both builders agree with the
    checker, and an epoch runs on them (an empty partition contributes loss 0 and no gradient)."""
    rng = np.random.default_rng(3)
    cases = []
    rowptr, col = graphs.erdos_renyi(60, 0.08, 5)
    user = np.where(np.arange(60) < 25, 0, 2).astype(np.int32)          # nobody in partition 1
    cases.append((rowptr, col, 3, 400_000, gcnsa.PART_USER, user))
    cases.append((np.zeros(8, np.int64), np.zeros(0, np.int32), 2, 500_000, gcnsa.PART_RANGE, None))
    for rowptr, col, m, o_ppm, mode, user in cases:
        n = rowptr.size - 1
        x = rng.standard_normal((n, 6)).astype(np.float32)
        y = rng.integers(0, 3, n).astype(np.int32)
        mask = np.ones(n, np.uint8)
        dev = _build(gcnsa.BUILD_DEVICE, rowptr, col, x, y, mask, 3, m, o_ppm, 41, mode, user, 1)
        host = _build(gcnsa.BUILD_HOST, rowptr, col, x, y, mask, 3, m, o_ppm, 41, mode, user, 1)
        _against_checker(dev, rowptr, col, m, o_ppm, 41, mode, user, mask, 1)
        _same(dev, host, m)
        env = gcnsa.make_env(0)
        w0 = [rng.standard_normal((6, 4)).astype(np.float32), rng.standard_normal((4, 3)).astype(np.float32)]
        losses = []
        for parts in (dev, host):
            for fact in (0, 1):
                model = gcnsa.Model(env, parts, [6, 4, 3], w0, None, **{**gcnsa.PLAIN, 'gemm_mode': gcnsa.GEMM_TF32X3,
                                                                      'factored_norm': fact})
                loss = torch.zeros(1, device="cuda")
                model.epoch(loss.data_ptr())
                model.epoch(loss.data_ptr())
                losses.append(loss.item())
                assert np.isfinite(losses[-1])
                model.close()
        assert max(losses) - min(losses) <= 1e-5 * max(abs(l) for l in losses)
        dev.close(); host.close()
