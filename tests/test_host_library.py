"""CPU-side tests of the CUDA library: it loads, exports every symbol the
header declares, reports argument and graph errors as codes, fails loudly
without a GPU, and its host builder (partition assignment, Algorithm 1,
structure of the extended partitions) agrees bit for bit with the checker."""
import os
import re

import numpy as np
import pytest

from gen import configs, graphs
from oracle import oracle
from paper_2012_04930_b200 import gcnsa

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _has_gpu():
    import torch
    return torch.cuda.is_available()


def test_library_exports_every_declared_symbol():
    hdr = open(os.path.join(ROOT, "include", "gcnsa.h")).read()
    hdr = re.sub(r"/\*.*?\*/", "", hdr, flags=re.S)
    declared = set(re.findall(r"\b(gcnsa_[a-z0-9_]+)\s*\(", hdr))
    assert {"gcnsa_build_partitions", "gcnsa_forward", "gcnsa_backward", "gcnsa_step"} <= declared
    L = gcnsa.lib()
    for name in sorted(declared):
        assert hasattr(L, name), f"{name} declared in gcnsa.h but not exported"
    assert declared == set(gcnsa.exported_symbols()), declared ^ set(gcnsa.exported_symbols())


def test_error_texts():
    L = gcnsa.lib()
    assert L.gcnsa_strerror(0) == b"ok"
    for code in range(-9, 0):
        assert L.gcnsa_strerror(code) not in (b"ok", b"unknown error")
    assert L.gcnsa_strerror(-99) == b"unknown error"


def _plan(w, **kw):
    args = dict(m=w.m, overlap_ppm=w.overlap_ppm, seed=w.seed, part_mode=w.part_mode, user_part=w.user_part,
                loss_on_halo=w.loss_on_halo)
    args.update(kw)
    return gcnsa.Plan(w.rowptr, w.col, w.x, w.y, w.train_mask, w.dims[-1], **args)


def _compare(plan, rowptr, col, m, o_ppm, seed, mode, user, mask, loss_on_halo=1):
    part, parts = oracle.build_partitions(rowptr, col, m, o_ppm, seed, mode, user)
    assert np.array_equal(plan.assignment(), part)
    for p, pt in enumerate(parts):
        i = plan.info(p)
        e = plan.export(p)
        assert (i.n_owned, i.n_halo, i.n, i.nnz, i.nts) == (pt.n_owned, pt.n - pt.n_owned, pt.n, pt.nnz, pt.nts)
        assert np.array_equal(e["members"], pt.members)
        assert np.array_equal(e["rowptr"], pt.rowptr) and np.array_equal(e["col"], pt.col)
        assert np.array_equal(e["t_rowptr"], pt.t_rowptr) and np.array_equal(e["t_col"], pt.t_col)
        for op in range(m):
            assert e["depth"][op] == (0 if op == p else pt.depth_by_op[op])
        assert i.max_depth == max([0] + list(pt.depth_by_op.values()))
        t = oracle.train_set(pt, mask[pt.members], loss_on_halo)
        assert i.n_train == int(t.sum())


def test_host_builder_matches_checker_on_tiny_and_small(tiny_wl, small_wl):
    for w in (tiny_wl, small_wl):
        pl = _plan(w)
        _compare(pl, w.rowptr, w.col, w.m, w.overlap_ppm, w.seed, w.part_mode, w.user_part, w.train_mask)
        pl.close()


@pytest.mark.parametrize("n,prob,m,o_ppm,seed,mode", [
    (64, 0.03, 2, 1_000_000, 7, 0), (64, 0.02, 2, 2_000_000, 5, 1), (48, 0.03, 4, 1_000_000, 3, 1),
    (200, 0.02, 5, 500_000, 11, 0), (200, 0.01, 3, 3_000_000, 12, 1), (30, 0.3, 3, 100_000, 4, 0),
    (90, 0.05, 1, 500_000, 13, 0), (120, 0.04, 6, 0, 14, 1),
])
def test_host_builder_matches_checker_on_random_graphs(n, prob, m, o_ppm, seed, mode):
    rowptr, col = graphs.erdos_renyi(n, prob, 300 + seed)
    rng = np.random.default_rng(seed)
    x = rng.standard_normal((n, 3)).astype(np.float32)
    y = rng.integers(0, 4, n).astype(np.int32)
    mask = (rng.random(n) < 0.5).astype(np.uint8)
    for loh in (1, 0):
        pl = gcnsa.Plan(rowptr, col, x, y, mask, 4, m, o_ppm, seed, mode, None, loh)
        _compare(pl, rowptr, col, m, o_ppm, seed, mode, None, mask, loh)
        pl.close()


def test_host_builder_on_scaled_power_law_graph():
    w = configs.paper_scale(scale=0.02)
    pl = _plan(w)
    _compare(pl, w.rowptr, w.col, w.m, w.overlap_ppm, w.seed, w.part_mode, w.user_part, w.train_mask)
    # a hash partition of the same graph (worst-case cut) and a large overlap
    pl2 = _plan(w, part_mode=gcnsa.PART_HASH, overlap_ppm=500_000)
    _compare(pl2, w.rowptr, w.col, w.m, 500_000, w.seed, gcnsa.PART_HASH, None, w.train_mask)


def test_graph_errors_are_codes():
    x = np.zeros((3, 2), np.float32); y = np.zeros(3, np.int32); mk = np.ones(3, np.uint8)

    def code(rowptr, col, **kw):
        args = dict(n_classes=2, m=1, overlap_ppm=0, seed=0)
        args.update(kw)
        with pytest.raises(gcnsa.GcnsaError) as ei:
            gcnsa.Plan(np.array(rowptr, np.int64), np.array(col, np.int32), x, y, mk, **args)
        return ei.value.code

    assert code([0, 1, 1, 1], [1]) == gcnsa.ERR_NOT_SYMMETRIC
    assert code([0, 1, 1, 1], [0]) == gcnsa.ERR_SELF_LOOP_OR_DUP
    assert code([0, 2, 3, 4], [1, 1, 0, 0]) == gcnsa.ERR_SELF_LOOP_OR_DUP
    assert code([0, 2, 3, 4], [2, 1, 0, 0]) == gcnsa.ERR_ARG            # row not ascending
    assert code([0, 1, 2, 2], [1, 7]) == gcnsa.ERR_ARG                  # column out of range
    assert code([0, 1, 2, 2], [1, 0], m=4) == gcnsa.ERR_ARG             # more partitions than vertices
    assert code([0, 1, 2, 2], [1, 0], m=0) == gcnsa.ERR_ARG
    assert code([0, 1, 2, 2], [1, 0], n_classes=0) == gcnsa.ERR_ARG
    assert code([0, 1, 2, 2], [1, 0], m=2, part_mode=gcnsa.PART_USER, user_part=np.array([0, 5, 0])) == gcnsa.ERR_LABEL_RANGE
    assert code([0, 1, 2, 2], [1, 0], m=2, part_mode=gcnsa.PART_USER) == gcnsa.ERR_ARG  # user_part missing
    assert code([0, 1, 2, 2], [1, 0], part_mode=9) == gcnsa.ERR_ARG
    assert code([0, 1, 2, 2], [1, 0], order_window=100) == gcnsa.ERR_ARG       # windows of fewer than 256 rows
    with pytest.raises(gcnsa.GcnsaError) as ei:
        gcnsa.Plan(np.array([0, 1, 2, 2], np.int64), np.array([1, 0], np.int32), x, np.array([0, 3, 0], np.int32), mk,
                   2, 1, 0, 0)
    assert ei.value.code == gcnsa.ERR_LABEL_RANGE


@pytest.mark.skipif(_has_gpu(), reason="checks the behaviour without a GPU")
def test_device_path_fails_loudly_without_a_gpu(tiny_wl):
    """No CPU fallback: building the device-resident partitions must raise."""
    w = tiny_wl
    env = gcnsa.Env()
    env.device = 0
    with pytest.raises(gcnsa.GcnsaError) as ei:
        gcnsa.Parts(env, w.rowptr, w.col, w.x, w.y, w.train_mask, w.dims[-1], w.m, w.overlap_ppm, w.seed, w.part_mode,
                    w.user_part)
    assert ei.value.code in (gcnsa.ERR_CUDA, gcnsa.ERR_ARCH)


def test_product_code_never_touches_the_checker():
    """The library and its binding must not import, link or read oracle/."""
    pkg = os.path.join(ROOT, "paper_2012_04930_b200")
    for dirpath, _, files in os.walk(pkg):
        for fn in files:
            if fn.endswith((".py", ".cu", ".cpp", ".h")):
                text = open(os.path.join(dirpath, fn)).read()
                assert "oracle" not in text, f"{fn} mentions the checker"


def _length_class(n):
    """Lengths below 32 are a class each; longer ones share a class with the lengths that have the same five
    leading bits (written here from that sentence, not from the library's code)."""
    if n < 32:
        return n
    e = int(n).bit_length() - 1
    return 32 + (e - 5) * 16 + ((n >> (e - 4)) & 15)


def _check_order(order, lens, thr, n_long, window=None):
    """Hub rows (at least thr entries) first, by descending length class; then the other rows window by window
    (a window = `window` consecutive rows, None = one window), inside a window by descending class; rows of one
    class in index order."""
    n = lens.size
    assert np.array_equal(np.sort(order), np.arange(n)), "a processing order is a permutation of the rows"
    ln = lens[order]
    assert n_long == int((lens >= thr).sum()) and np.all(ln[:n_long] >= thr) and np.all(ln[n_long:] < thr)
    rest = order[n_long:]
    win = rest // window if window else np.zeros(rest.size, np.int64)
    assert np.all(np.diff(win) >= 0), "windows come in ascending order"
    segments = [order[:n_long]] + [rest[win == k] for k in np.unique(win)]
    for seg in segments:
        cls = np.array([_length_class(int(v)) for v in lens[seg]])
        assert np.all(np.diff(cls) <= 0), "length classes descend"
        same = np.diff(cls) == 0
        assert np.all(np.diff(seg)[same] > 0), "rows of one class come in index order"


@pytest.mark.parametrize("name,kw,o_ppm", [("small", {}, 100_000), ("paper_scale", {"scale": 0.02}, 500_000),
                                           ("large_sparse", {"scale": 0.01}, 100_000)])
def test_host_builder_scheduling_structures(name, kw, o_ppm):
    """Row orders (hub rows first, then window by window by descending length class, ties by index), the loss rows
    in that order, and the transposed CSR restricted to the loss columns, each rebuilt here with numpy from the
    checker's CSR.  The default (one window for partitions this small), windows of 256 and 1 000 rows, one window."""
    w = configs.by_name(name, **kw)
    for loh, ow, window in ((1, 0, None), (0, 256, 256), (1, -1, None), (1, 1000, 1000)):   # 0: under 131 072 rows, one window
        pl = _plan(w, overlap_ppm=o_ppm, loss_on_halo=loh, order_window=ow)
        _, parts = oracle.build_partitions(w.rowptr, w.col, w.m, o_ppm, w.seed, w.part_mode, w.user_part)
        for p, pt in enumerate(parts):
            s = pl.export_schedule(p)
            thr = max(1024, pt.nnz // 8192)
            lens, t_lens = np.diff(pt.rowptr), np.diff(pt.t_rowptr)
            _check_order(s["order"], lens, thr, s["n_long"], window)
            _check_order(s["t_order"], t_lens, thr, s["t_n_long"], window)
            carries = oracle.train_set(pt, w.train_mask[pt.members], loh).astype(bool)
            assert np.array_equal(s["m_order"], s["order"][carries[s["order"]]])
            assert s["m_nnz"] == int(lens[carries].sum()) and s["m_n_long"] == int((lens[carries] >= thr).sum())
            keep = carries[pt.t_col]                       # entries of the transposed CSR whose column carries loss
            assert np.array_equal(s["tm_col"], pt.t_col[keep])
            t_row = np.repeat(np.arange(pt.n), t_lens)
            tm_lens = np.bincount(t_row[keep], minlength=pt.n)
            assert np.array_equal(s["tm_rowptr"], np.concatenate([[0], np.cumsum(tm_lens)]))
            assert s["tm_nnz"] == int(keep.sum())
            _check_order(s["tm_order"], tm_lens, max(1024, s["tm_nnz"] // 8192), s["tm_n_long"], window)
        pl.close()


def test_hub_rows_lead_the_processing_order():
    """A star of 3 000 leaves next to a ring: the centre's row (3 001 entries, above the 1 024-entry threshold) is
    the one hub row and comes first in both orders."""
    n = 3_400
    edges = [(0, j) for j in range(1, 3_001)] + [(j, j + 1) for j in range(3_001, n - 1)] + [(n - 1, 3_001)]
    rowptr, col = graphs.from_edge_list(n, edges)
    x = np.zeros((n, 2), np.float32); y = np.zeros(n, np.int32); mk = np.ones(n, np.uint8)
    pl = gcnsa.Plan(rowptr, col, x, y, mk, 2, 1, 0, 0)
    e, s = pl.export(0), pl.export_schedule(0)
    lens = np.diff(e["rowptr"])
    assert (s["n_long"], s["t_n_long"], s["m_n_long"], s["tm_n_long"]) == (1, 1, 1, 1)
    assert s["order"][0] == 0 and s["t_order"][0] == 0 and s["m_order"][0] == 0 and s["tm_order"][0] == 0
    _check_order(s["order"], lens, 1024, 1)
    pl.close()


def test_large_partitions_get_windows_of_8192_rows_by_default():
    """From 131 072 rows on, the library cuts the processing order into windows of 8 192 consecutive rows."""
    n = 140_000
    rng = np.random.default_rng(0)
    extra = [(int(a), int(b)) for a, b in zip(rng.integers(0, n, 60_000), rng.integers(0, n, 60_000)) if a != b]
    rowptr, col = graphs.from_edge_list(n, [(j, (j + 1) % n) for j in range(n)] + extra)
    x = np.zeros((n, 1), np.float32); y = np.zeros(n, np.int32); mk = np.ones(n, np.uint8)
    pl = gcnsa.Plan(rowptr, col, x, y, mk, 1, 1, 0, 0)
    e, s = pl.export(0), pl.export_schedule(0)
    lens = np.diff(e["rowptr"])
    _check_order(s["order"], lens, 1024, 0, window=8192)
    assert len(np.unique(s["order"][:8192] // 8192)) == 1 and lens[s["order"][0]] == lens[:8192].max()
    pl.close()


def test_calls_that_need_no_device():
    """The dense-product path counters and the default option set are host-side state."""
    tc, fb = gcnsa.gemm_path_counts()
    assert tc >= 0 and fb >= 0
    o = gcnsa.ModelOpts()
    o.gemm_mode, o.lr = 77, -1.0
    gcnsa.lib().gcnsa_model_opts_default(o)
    got = {k: getattr(o, k) for k in gcnsa.MEASURED}
    assert got == gcnsa.MEASURED, "the binding's MEASURED set must be what the library calls its default"
    assert (o.n_layers, o.use_bias, o.agg_mode, o.cache_ax) == (2, 1, gcnsa.AGG_GRAD_AVG, 0)
    assert abs(o.lr - 0.02) < 1e-9 and abs(o.beta1 - 0.9) < 1e-7 and abs(o.beta2 - 0.999) < 1e-7 and 0 < o.eps < 1e-7
    import ctypes as C
    assert gcnsa.lib().gcnsa_gemm_path_counts(None, C.byref(C.c_int64())) == gcnsa.ERR_ARG


def test_op_arguments_are_rejected_before_any_device_work():
    """Misaligned or inconsistent operands give GCNSA_ERR_ARG on the host; no kernel is launched for them (the
    pointers below are made-up addresses that are never dereferenced)."""
    import ctypes as C
    L = gcnsa.lib()
    base = 0x7f0000000000
    before = gcnsa.launch_count()

    def colsum_scaled(g, ldg, scaled, lds, f=41, scratch=base + 0x100000, sbytes=1 << 20, rs=base + 0x200000):
        return L.gcnsa_op_colsum_scaled(None, 100, f, g, ldg, base + 0x300000, 0, scratch, sbytes, rs, scaled, lds)

    assert colsum_scaled(base + 4, 44, base + 0x400000, 44) == gcnsa.ERR_ARG        # g not 16-byte aligned
    assert colsum_scaled(base, 44, base + 0x400008, 44) == gcnsa.ERR_ARG            # scaled not 16-byte aligned
    assert colsum_scaled(base, 43, base + 0x400000, 44) == gcnsa.ERR_ARG            # pitch of g not a multiple of 4
    assert colsum_scaled(base, 44, base + 0x400000, 42) == gcnsa.ERR_ARG            # pitch of scaled
    assert colsum_scaled(base, 44, base + 0x400000, 40) == gcnsa.ERR_ARG            # scaled rows shorter than f
    assert colsum_scaled(base, 44, None, 44) == gcnsa.ERR_ARG
    assert colsum_scaled(base, 44, base + 0x400000, 44, rs=None) == gcnsa.ERR_ARG
    assert colsum_scaled(base, 44, base + 0x400000, 44, sbytes=16) == gcnsa.ERR_ARG  # scratch too small
    # sparse product: unaligned x, pitch not a multiple of 4, mask without a buffer
    def spmm(x, ldx, y, ldy, epi=gcnsa.EPI_NONE, aux=None, ldaux=0):
        return L.gcnsa_op_spmm(None, 10, base, base + 0x1000, base + 0x2000, None, 0, x, ldx, 8, epi, aux, ldaux, y, ldy)
    assert spmm(base + 0x10004, 8, base + 0x20000, 8) == gcnsa.ERR_ARG
    assert spmm(base + 0x10000, 9, base + 0x20000, 8) == gcnsa.ERR_ARG
    assert spmm(base + 0x10000, 8, base + 0x20000, 8, epi=gcnsa.EPI_MASK) == gcnsa.ERR_ARG
    assert spmm(base + 0x10000, 8, base + 0x20000, 8, epi=99) == gcnsa.ERR_ARG
    assert L.gcnsa_op_colsum_static(None, 10, gcnsa.COLSUM_STATIC_MAX_F + 1, base, 2048, base + 0x10000, 0) == gcnsa.ERR_TOO_LARGE
    # masked product with column sums: missing mask / sums / scratch, short pitches, unaligned or short scratch
    need = gcnsa.op_gemm_mask_colsum_scratch(300, 41)
    assert need % 256 == 0 and need >= 4 * 4 * 3 * 44                    # a row of partial sums per warp and row tile

    def fused(mask=base + 0x30000, ldmask=44, out=base + 0x40000, scratch=base + 0x100000, sbytes=need, ldc=44, mode=gcnsa.GEMM_TF32X3):
        return L.gcnsa_op_gemm_mask_colsum(None, mode, 0, 1, 300, 41, 64, base, 64, base + 0x10000, 64, base + 0x20000, ldc,
                                           mask, ldmask, None, out, 0, scratch, sbytes, None, 0)
    assert fused(mask=None) == gcnsa.ERR_ARG
    assert fused(out=None) == gcnsa.ERR_ARG
    assert fused(ldmask=40) == gcnsa.ERR_ARG
    assert fused(ldc=40) == gcnsa.ERR_ARG
    assert fused(scratch=None) == gcnsa.ERR_ARG
    assert fused(scratch=base + 0x100010) == gcnsa.ERR_ARG
    assert fused(sbytes=need - 256) == gcnsa.ERR_ARG
    assert fused(mode=7) == gcnsa.ERR_ARG
    # gather probe: short or unaligned rows, window outside the matrix, negative counts, missing buffers
    def probe(x=base, ldx=128, n=1000, window=64, hit=4, rounds=1, out=base + 0x1000000, obytes=1 << 30):
        return L.gcnsa_op_gather_probe(None, x, ldx, n, window, hit, rounds, out, obytes)
    assert probe(x=None) == gcnsa.ERR_ARG and probe(out=None) == gcnsa.ERR_ARG
    assert probe(ldx=124) == gcnsa.ERR_ARG and probe(ldx=130) == gcnsa.ERR_ARG and probe(x=base + 8) == gcnsa.ERR_ARG
    assert probe(window=0) == gcnsa.ERR_ARG and probe(window=1001) == gcnsa.ERR_ARG and probe(n=0) == gcnsa.ERR_ARG
    assert probe(hit=-1) == gcnsa.ERR_ARG and probe(rounds=-1) == gcnsa.ERR_ARG
    assert L.gcnsa_op_gather_probe_warps(None) == gcnsa.ERR_ARG
    assert gcnsa.launch_count() == before
