"""GPU parity of the single kernels, called through the C-ABI on caller-owned
device buffers and compared element by element with the fp64 checker.

Tolerance (fp32 kernels against fp64): max |got - want| <= 1e-4 * max |want|
per tensor, the bound the training path is held to; integer work is exact."""
import numpy as np
import pytest
import torch

from gen import graphs
from oracle import oracle
from paper_2012_04930_b200 import gcnsa

pytestmark = pytest.mark.gpu
TOL = 1e-4


def _close(got, want, tol=TOL, what=""):
    got = np.asarray(got, dtype=np.float64)
    want = np.asarray(want, dtype=np.float64)
    assert got.shape == want.shape, (what, got.shape, want.shape)
    if want.size == 0:
        return
    scale = max(np.abs(want).max(), 1e-30)
    err = np.abs(got - want).max()
    assert err <= tol * scale, f"{what}: max err {err:.3e} vs scale {scale:.3e}"


def _dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def _padded(a, ld):
    """Host [n x f] -> device [n x ld] with zero pad columns; returns the tensor."""
    t = torch.zeros((a.shape[0], ld), dtype=torch.float32, device="cuda")
    t[:, :a.shape[1]] = torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).cuda()
    return t


def _ld(f):
    return (f + 3) // 4 * 4


def _graph(kind, seed):
    if kind == "er":
        rowptr, col = graphs.erdos_renyi(777, 0.03, seed)          # ragged: 777 rows, not a multiple of 8
    elif kind == "powerlaw":
        rowptr, col, _ = graphs.chung_lu_communities(3001, 240_000, 2.1, 7, 0.8, seed)  # hubs of > 32 and > 1000 nnz
    else:
        rowptr, col = graphs.from_edge_list(50, [(0, j) for j in range(1, 40)])        # star + isolated vertices
    rp, cc, vv = oracle.induced(rowptr, col, np.arange(rowptr.size - 1))
    return rp, cc, vv


@pytest.mark.parametrize("kind", ["er", "powerlaw", "star"])
@pytest.mark.parametrize("f", [1, 3, 4, 16, 41, 47, 64, 100, 128, 130, 256, 602, 700])
def test_spmm_matches_checker(kind, f):
    rp, cc, vv = _graph(kind, 5)
    n = rp.size - 1
    rng = np.random.default_rng(f)
    x = rng.standard_normal((n, f)).astype(np.float32)
    want = oracle.spmm(rp, cc, vv, x.astype(np.float64))
    ld = _ld(f)
    xd = _padded(x, ld)
    yd = torch.full((n, ld), 7.0, device="cuda")
    order = torch.from_numpy(np.argsort(-np.diff(rp), kind="stable").astype(np.int32)).cuda()
    d_rp, d_cc, d_vv = _dev(rp.astype(np.int32)), _dev(cc.astype(np.int32)), _dev(vv.astype(np.float32))
    # plain order, longest-first order, and the 37 longest rows handled by a thread block each
    for ordr, n_long in ((None, 0), (order, 0), (order, min(n, 37))):
        yd.fill_(7.0)
        gcnsa.op_spmm(d_rp, d_cc, d_vv, xd, f, yd, order=ordr, n_long=n_long)
        torch.cuda.synchronize()
        _close(yd[:, :f].cpu().numpy(), want, what=f"spmm {kind} f={f}")
        assert torch.all(yd[:, f:] == 0), "pad columns must come out zero"


@pytest.mark.parametrize("f", [1, 41, 64, 128, 300])
def test_pattern_spmm_is_the_factored_normalized_product(f):
    """A_hat X = diag(d^-1/2) (A + I) (diag(d^-1/2) X) (Section 4.1 footnote): the unit-weight product with
    scaled source rows and scaled result rows equals the checker's product with the stored values; without a
    row scale it is the plain neighbour sum."""
    rp, cc, vv = _graph("powerlaw", 5)
    n = rp.size - 1
    rng = np.random.default_rng(100 + f)
    x = rng.standard_normal((n, f)).astype(np.float32)
    bias = rng.standard_normal(f).astype(np.float32)
    want = oracle.spmm(rp, cc, vv, x.astype(np.float64))
    ones = oracle.spmm(rp, cc, np.ones_like(vv), x.astype(np.float64))
    dinv = (1.0 / np.sqrt(np.diff(rp).astype(np.float64))).astype(np.float32)
    ld = _ld(f)
    xs = _padded(x * dinv[:, None], ld)
    yd = torch.full((n, ld), 7.0, device="cuda")
    order = torch.from_numpy(np.argsort(-np.diff(rp), kind="stable").astype(np.int32)).cuda()
    d_rp, d_cc = _dev(rp.astype(np.int32)), _dev(cc.astype(np.int32))
    for ordr, n_long in ((None, 0), (order, 0), (order, min(n, 37))):
        yd.fill_(7.0)
        gcnsa.op_spmm_pattern(d_rp, d_cc, xs, f, yd, row_scale=_dev(dinv), order=ordr, n_long=n_long)
        _close(yd[:, :f].cpu().numpy(), want, what=f"pattern spmm f={f}")
        assert torch.all(yd[:, f:] == 0), "pad columns must come out zero"
    gcnsa.op_spmm_pattern(d_rp, d_cc, xs, f, yd, row_scale=_dev(dinv), epi=gcnsa.EPI_BIAS_RELU, aux=_dev(bias), order=order,
                          n_long=3)
    _close(yd[:, :f].cpu().numpy(), np.maximum(want + bias, 0), what="pattern spmm, scale before bias + relu")
    gcnsa.op_spmm_pattern(d_rp, d_cc, _padded(x, ld), f, yd)
    _close(yd[:, :f].cpu().numpy(), ones, what="neighbour sum")


def test_spmm_epilogues_and_transposed_product():
    rp, cc, vv = _graph("powerlaw", 9)
    n = rp.size - 1
    # a non-symmetric matrix: scale every row differently, then use its real transpose
    rng = np.random.default_rng(1)
    vv = vv * np.repeat(rng.uniform(0.5, 2.0, n), np.diff(rp))
    trp, tc, tv = oracle.transpose(n, n, rp, cc, vv)
    f = 44
    x = rng.standard_normal((n, f)).astype(np.float32)
    bias = rng.standard_normal(f).astype(np.float32)
    maskm = rng.standard_normal((n, f)).astype(np.float32)
    base = oracle.spmm(trp, tc, tv, x.astype(np.float64))
    xd, yd = _padded(x, f), torch.empty((n, f), device="cuda")
    args = (_dev(trp.astype(np.int32)), _dev(tc.astype(np.int32)), _dev(tv.astype(np.float32)), xd, f, yd)
    gcnsa.op_spmm(*args, epi=gcnsa.EPI_BIAS, aux=_dev(bias))
    _close(yd.cpu().numpy(), base + bias, what="bias")
    gcnsa.op_spmm(*args, epi=gcnsa.EPI_BIAS_RELU, aux=_dev(bias))
    _close(yd.cpu().numpy(), np.maximum(base + bias, 0), what="bias+relu")
    gcnsa.op_spmm(*args, epi=gcnsa.EPI_BIAS_RELU, aux=None)
    _close(yd.cpu().numpy(), np.maximum(base, 0), what="relu")
    gcnsa.op_spmm(*args, epi=gcnsa.EPI_MASK, aux=_dev(maskm))
    _close(yd.cpu().numpy(), base * (maskm > 0), what="mask")


def test_spmm_edge_cases_and_argument_errors():
    z = torch.zeros(4, dtype=torch.int32, device="cuda")
    zf = torch.zeros((4, 4), device="cuda")
    # zero rows: nothing launched, no error
    gcnsa.op_spmm(torch.zeros(1, dtype=torch.int32, device="cuda"), z, zf.view(-1), zf, 4, zf)
    rp = _dev(np.array([0, 0, 1, 1], np.int32))     # empty rows around one entry
    y = torch.full((3, 4), 5.0, device="cuda")
    gcnsa.op_spmm(rp, _dev(np.array([2], np.int32)), _dev(np.array([2.0], np.float32)),
                  _dev(np.arange(12, dtype=np.float32).reshape(3, 4)), 4, y)
    assert y.cpu().tolist() == [[0, 0, 0, 0], [16, 18, 20, 22], [0, 0, 0, 0]]
    with pytest.raises(gcnsa.GcnsaError) as ei:     # leading dimension not a multiple of 4
        gcnsa.op_spmm(rp, z, zf.view(-1), torch.zeros((3, 5), device="cuda"), 5, torch.zeros((3, 5), device="cuda"))
    assert ei.value.code == gcnsa.ERR_ARG
    with pytest.raises(gcnsa.GcnsaError):           # mask epilogue without a mask
        gcnsa.op_spmm(rp, z, zf.view(-1), zf, 4, y, epi=gcnsa.EPI_MASK)


GEMM_SHAPES = [(1, 1, 1), (5, 3, 2), (130, 41, 602), (257, 128, 64), (64, 64, 16), (300, 47, 256), (129, 130, 131)]


@pytest.mark.parametrize("m,n,k", GEMM_SHAPES)
@pytest.mark.parametrize("ta,tb", [(0, 0), (1, 0), (0, 1), (1, 1)])
def test_gemm_matches_fp64(m, n, k, ta, tb):
    rng = np.random.default_rng(m * 7 + n)
    a = rng.standard_normal((k, m) if ta else (m, k)).astype(np.float32)
    b = rng.standard_normal((n, k) if tb else (k, n)).astype(np.float32)
    want = (a.T if ta else a).astype(np.float64) @ (b.T if tb else b).astype(np.float64)
    for pad in (True, False):  # 16-byte aligned rows (vector loads) and dense odd rows (scalar loads)
        ad = _padded(a, _ld(a.shape[1])) if pad else _dev(a)
        bd = _padded(b, _ld(b.shape[1])) if pad else _dev(b)
        cd = torch.full((m, _ld(n)), 3.0, device="cuda")
        gcnsa.op_gemm(ad, bd, cd, m, n, k, ta=ta, tb=tb)
        _close(cd[:, :n].cpu().numpy(), want, what=f"gemm {m}x{n}x{k} ta={ta} tb={tb} pad={pad}")
        assert torch.all(cd[:, n:] == 0)


def test_gemm_split_k_accumulate_and_epilogues():
    rng = np.random.default_rng(3)
    # H^T dT with the row count of a partition as the inner dimension
    kk, m, n = 20_011, 130, 41
    h = rng.standard_normal((kk, m)).astype(np.float32)
    dt = rng.standard_normal((kk, n)).astype(np.float32)
    c0 = rng.standard_normal((m, n)).astype(np.float32)
    want = c0 + h.astype(np.float64).T @ dt.astype(np.float64)
    wsb = gcnsa.op_gemm_workspace(1, 0, m, n, kk)
    assert wsb > 0, "a tall-skinny product should be split along k"
    ws = torch.empty(wsb // 4, device="cuda")
    hd, dtd = _padded(h, _ld(m)), _padded(dt, _ld(n))
    outs = []
    for _ in range(2):
        cd = _padded(c0, _ld(n))
        gcnsa.op_gemm(hd, dtd, cd, m, n, kk, ta=1, accumulate=1, workspace=ws)
        outs.append(cd.clone())
    _close(outs[0][:, :n].cpu().numpy(), want, what="split-k accumulate")
    assert torch.equal(outs[0], outs[1]), "split-k must be run-to-run identical"
    cd = _padded(c0, _ld(n))                       # without workspace: unsplit, same result within tolerance
    gcnsa.op_gemm(hd, dtd, cd, m, n, kk, ta=1, accumulate=1)
    _close(cd[:, :n].cpu().numpy(), want, what="unsplit accumulate")
    # epilogues
    a = rng.standard_normal((300, 70)).astype(np.float32)
    b = rng.standard_normal((70, 50)).astype(np.float32)
    bias = rng.standard_normal(50).astype(np.float32)
    mk = rng.standard_normal((300, 50)).astype(np.float32)
    base = a.astype(np.float64) @ b.astype(np.float64)
    ad, bd, cd = _padded(a, 72), _padded(b, 52), torch.empty((300, 52), device="cuda")
    gcnsa.op_gemm(ad, bd, cd, 300, 50, 70, epi=gcnsa.EPI_BIAS, aux=_dev(bias))
    _close(cd[:, :50].cpu().numpy(), base + bias, what="bias")
    gcnsa.op_gemm(ad, bd, cd, 300, 50, 70, epi=gcnsa.EPI_BIAS_RELU, aux=_dev(bias))
    _close(cd[:, :50].cpu().numpy(), np.maximum(base + bias, 0), what="bias relu")
    gcnsa.op_gemm(ad, bd, cd, 300, 50, 70, epi=gcnsa.EPI_MASK, aux=_padded(mk, 52))
    _close(cd[:, :50].cpu().numpy(), base * (mk > 0), what="mask")
    rs = rng.uniform(0.1, 2.0, 300).astype(np.float32)
    gcnsa.op_gemm(ad, bd, cd, 300, 50, 70, epi=gcnsa.EPI_ROWSCALE, aux=_dev(rs))
    _close(cd[:, :50].cpu().numpy(), base * rs[:, None], what="row scale")
    with pytest.raises(gcnsa.GcnsaError):
        gcnsa.op_gemm(ad, bd, cd, 300, 50, 70, epi=gcnsa.EPI_ROWSCALE)          # no scale vector


@pytest.mark.parametrize("n,c", [(1, 1), (7, 5), (1000, 41), (20_003, 47), (513, 300)])
def test_softmax_cross_entropy(n, c):
    rng = np.random.default_rng(n + c)
    z = (rng.standard_normal((n, c)) * 3).astype(np.float32)
    y = rng.integers(0, c, n).astype(np.int32)
    mask = (rng.random(n) < 0.6).astype(np.uint8)
    nt = int(mask.sum())
    z64 = z.astype(np.float64)
    lse = np.log(np.exp(z64 - z64.max(1, keepdims=True)).sum(1)) + z64.max(1)
    want_loss = ((lse - z64[np.arange(n), y]) * mask).sum() / max(nt, 1)
    soft = np.exp(z64 - lse[:, None])
    soft[np.arange(n), y] -= 1
    want_g = soft * mask[:, None] / max(nt, 1)
    ld = _ld(c)
    zd, gd = _padded(z, ld), torch.full((n, ld), 9.0, device="cuda")
    loss = torch.full((1,), 9.0, device="cuda")
    sc = torch.empty(gcnsa.op_softmax_ce_scratch(n) // 4 + 1, device="cuda")
    gcnsa.op_softmax_ce(zd, c, _dev(y), _dev(mask), nt, loss, gd, sc)
    _close(gd[:, :c].cpu().numpy(), want_g, what="dlogits")
    assert torch.all(gd[:, c:] == 0)
    assert abs(loss.item() - want_loss) <= 1e-5 * max(abs(want_loss), 1e-6)
    # empty training set: zero loss, zero gradient
    gcnsa.op_softmax_ce(zd, c, _dev(y), _dev(np.zeros(n, np.uint8)), 0, loss, gd, sc)
    assert loss.item() == 0.0 and torch.all(gd == 0)


def test_softmax_cross_entropy_extreme_logits():
    z = np.array([[1e4, -1e4, 0.0], [-80.0, -90.0, -100.0]], np.float32)
    y = np.array([1, 0], np.int32)
    gd, loss = torch.empty((2, 4), device="cuda"), torch.empty(1, device="cuda")
    sc = torch.empty(64, device="cuda")
    gcnsa.op_softmax_ce(_padded(z, 4), 3, _dev(y), _dev(np.ones(2, np.uint8)), 2, loss, gd, sc)
    assert np.isfinite(loss.item()) and torch.isfinite(gd).all()
    assert abs(loss.item() - (2e4 + np.log1p(np.exp(-10.0) + np.exp(-20.0))) / 2) < 1e-2


@pytest.mark.parametrize("n,f", [(1, 1), (1000, 41), (50_001, 128), (300, 602)])
def test_colsum(n, f):
    rng = np.random.default_rng(n)
    g = rng.standard_normal((n, f)).astype(np.float32)
    out0 = rng.standard_normal(f).astype(np.float32)
    gd = _padded(g, _ld(f))
    sc = torch.empty(gcnsa.op_colsum_scratch(n, f) // 4 + 1, device="cuda")
    out = _dev(out0)
    gcnsa.op_colsum(gd, f, out, 1, sc)
    _close(out.cpu().numpy(), out0 + g.astype(np.float64).sum(0), what="colsum accumulate")
    gcnsa.op_colsum(gd, f, out, 0, sc)
    _close(out.cpu().numpy(), g.astype(np.float64).sum(0), what="colsum")
    # the same sums with the row-scaled copy written on the way, out of place and in place
    rs = rng.uniform(0.1, 2.0, n).astype(np.float32)
    want_scaled = g.astype(np.float64) * rs[:, None].astype(np.float64)
    side = torch.full((n, _ld(f) + 4), 9.0, device="cuda")
    plain = out.clone()
    gcnsa.op_colsum_scaled(gd, f, out, 0, sc, _dev(rs), side)
    assert torch.equal(out, plain), "the sums must not depend on the side output"
    _close(side[:, :f].cpu().numpy(), want_scaled, tol=1e-6, what="scaled copy")
    assert torch.all(side[:, _ld(f):] == 9.0), "columns beyond the last float4 chunk stay untouched"
    gcnsa.op_colsum_scaled(gd, f, out, 0, sc, _dev(rs), gd)
    assert torch.equal(out, plain)
    _close(gd[:, :f].cpu().numpy(), want_scaled, tol=1e-6, what="scaled in place")


def test_adam_against_checker():
    rng = np.random.default_rng(0)
    p0 = rng.standard_normal(10_001).astype(np.float32)
    opt = oracle.Adam([p0.astype(np.float64)], lr=0.02)
    theta, m, v = _dev(p0), torch.zeros(10_001, device="cuda"), torch.zeros(10_001, device="cuda")
    cur = [p0.astype(np.float64)]
    for t in range(1, 6):
        gs = rng.standard_normal(10_001).astype(np.float32)
        gsum = _dev(gs)
        gcnsa.op_adam(theta, gsum, m, v, 1.0 / 5.0, 0.02, 0.9, 0.999, 1e-8, t)
        cur = opt.step(cur, [gs.astype(np.float64) / 5.0])
        _close(theta.cpu().numpy(), cur[0], tol=1e-5, what=f"adam t={t}")
        assert torch.all(gsum == 0), "the gradient sum must be cleared"


def test_normalize_kernel():
    rp, cc, vv = _graph("powerlaw", 2)
    deg = np.diff(rp).astype(np.int32)
    val = torch.empty(cc.size, device="cuda")
    gcnsa.op_normalize(_dev(rp.astype(np.int32)), _dev(cc.astype(np.int32)), _dev(deg), val)
    got = val.cpu().numpy().astype(np.float64)
    assert np.abs(got - vv).max() <= 2e-7 * vv.max()


# ------------------------------------------------ tensor-core GEMM (3xTF32) ---
TC_SHAPES = [(1, 1, 1), (130, 41, 602), (257, 128, 64), (300, 47, 256), (129, 130, 131), (1000, 128, 602),
             (128, 64, 32), (512, 256, 96), (300, 256, 256), (260, 602, 100), (1000, 300, 70),
             # more tiles than SMs: every CTA walks several work items (three and more wrap the phase of the two
             # accumulator buffers and of the stage ring), the last ones ragged
             (57_000, 128, 96), (20_011, 300, 200), (40_003, 41, 130), (19_000, 128, 33)]


@pytest.mark.parametrize("m,n,k", TC_SHAPES)
@pytest.mark.parametrize("ta,tb", [(0, 0), (1, 0), (0, 1), (1, 1)])
def test_tensor_core_gemm_matches_fp64(m, n, k, ta, tb):
    rng = np.random.default_rng(m * 11 + n + k)
    a = rng.standard_normal((k, m) if ta else (m, k)).astype(np.float32)
    b = rng.standard_normal((n, k) if tb else (k, n)).astype(np.float32)
    want = (a.T if ta else a).astype(np.float64) @ (b.T if tb else b).astype(np.float64)
    ad, bd = _padded(a, _ld(a.shape[1])), _padded(b, _ld(b.shape[1]))
    cd = torch.full((m, _ld(n)), 3.0, device="cuda")
    ws = torch.empty(gcnsa.op_gemm_workspace(ta, tb, m, n, k, gcnsa.GEMM_TF32X3) // 4 + 64, device="cuda")
    before = gcnsa.launch_count()
    tc0, fb0 = gcnsa.gemm_path_counts()
    gcnsa.op_gemm(ad, bd, cd, m, n, k, ta=ta, tb=tb, workspace=ws, mode=gcnsa.GEMM_TF32X3)
    assert gcnsa.tc_status() == 0
    assert gcnsa.launch_count() > before
    assert gcnsa.gemm_path_counts() == (tc0 + 1, fb0), "the tensor-core kernel must have taken this product"
    # three TF32 products give fp32-level accuracy (a few 1e-6 of max at K = 602): far inside the 1e-4 bar
    _close(cd[:, :n].cpu().numpy(), want, tol=1e-5, what=f"tc gemm {m}x{n}x{k} ta={ta} tb={tb}")
    assert torch.all(cd[:, n:_ld(n)] == 0)


def test_tensor_core_gemm_split_k_epilogues_and_fallback():
    rng = np.random.default_rng(5)
    kk, m, n = 20_011, 130, 41                       # H^T dT: inner dimension = rows of a partition
    h = rng.standard_normal((kk, m)).astype(np.float32)
    dt = rng.standard_normal((kk, n)).astype(np.float32)
    c0 = rng.standard_normal((m, n)).astype(np.float32)
    want = c0 + h.astype(np.float64).T @ dt.astype(np.float64)
    ws = torch.empty(gcnsa.op_gemm_workspace(1, 0, m, n, kk, gcnsa.GEMM_TF32X3) // 4 + 64, device="cuda")
    hd, dtd = _padded(h, _ld(m)), _padded(dt, _ld(n))
    outs = []
    for _ in range(2):
        cd = _padded(c0, _ld(n))
        gcnsa.op_gemm(hd, dtd, cd, m, n, kk, ta=1, accumulate=1, workspace=ws, mode=gcnsa.GEMM_TF32X3)
        outs.append(cd.clone())
    assert gcnsa.tc_status() == 0
    _close(outs[0][:, :n].cpu().numpy(), want, tol=2e-5, what="tc split-k accumulate")
    assert torch.equal(outs[0], outs[1])
    # epilogues
    a = rng.standard_normal((300, 70)).astype(np.float32)
    b = rng.standard_normal((50, 70)).astype(np.float32)
    bias = rng.standard_normal(50).astype(np.float32)
    mk = rng.standard_normal((300, 50)).astype(np.float32)
    base = a.astype(np.float64) @ b.astype(np.float64).T
    ad, bd, cd = _padded(a, 72), _padded(b, 72), torch.empty((300, 52), device="cuda")
    gcnsa.op_gemm(ad, bd, cd, 300, 50, 70, tb=1, epi=gcnsa.EPI_BIAS_RELU, aux=_dev(bias), workspace=ws, mode=gcnsa.GEMM_TF32X3)
    _close(cd[:, :50].cpu().numpy(), np.maximum(base + bias, 0), tol=2e-5, what="tc bias relu")
    gcnsa.op_gemm(ad, bd, cd, 300, 50, 70, tb=1, epi=gcnsa.EPI_MASK, aux=_padded(mk, 52), workspace=ws, mode=gcnsa.GEMM_TF32X3)
    _close(cd[:, :50].cpu().numpy(), base * (mk > 0), tol=2e-5, what="tc mask")
    rs = rng.uniform(0.1, 2.0, 300).astype(np.float32)
    gcnsa.op_gemm(ad, bd, cd, 300, 50, 70, tb=1, epi=gcnsa.EPI_ROWSCALE, aux=_dev(rs), workspace=ws, mode=gcnsa.GEMM_TF32X3)
    _close(cd[:, :50].cpu().numpy(), base * rs[:, None], tol=2e-5, what="tc row scale")
    # a wide, 16-byte aligned result takes the float4 epilogue
    b2 = rng.standard_normal((128, 70)).astype(np.float32)
    c2 = torch.empty((300, 128), device="cuda")
    gcnsa.op_gemm(ad, _padded(b2, 72), c2, 300, 128, 70, tb=1, epi=gcnsa.EPI_ROWSCALE, aux=_dev(rs), workspace=ws,
                  mode=gcnsa.GEMM_TF32X3)
    _close(c2.cpu().numpy(), (a.astype(np.float64) @ b2.astype(np.float64).T) * rs[:, None], tol=2e-5,
           what="tc row scale, float4 epilogue")
    # rows that are not 16-byte aligned cannot go through TMA: the call falls back to the fp32 FMA kernel
    a_odd, b_odd = _dev(a[:, :67].copy()), _dev(b[:, :67].copy())
    tc0, fb0 = gcnsa.gemm_path_counts()
    gcnsa.op_gemm(a_odd, b_odd, cd, 300, 50, 67, tb=1, workspace=ws, mode=gcnsa.GEMM_TF32X3)
    _close(cd[:, :50].cpu().numpy(), a[:, :67].astype(np.float64) @ b[:, :67].astype(np.float64).T, what="fallback")
    assert gcnsa.gemm_path_counts() == (tc0, fb0 + 1), "unaligned rows: the fp32 FMA kernel, and it is counted"
    # too little workspace for the k-slices: fallback as well; fp32 mode counts in neither
    gcnsa.op_gemm(hd, dtd, _padded(c0, _ld(n)), m, n, kk, ta=1, accumulate=1, workspace=None, mode=gcnsa.GEMM_TF32X3)
    assert gcnsa.gemm_path_counts() == (tc0, fb0 + 2)
    gcnsa.op_gemm(ad, bd, cd, 300, 50, 70, tb=1, workspace=ws, mode=gcnsa.GEMM_FP32)
    assert gcnsa.gemm_path_counts() == (tc0, fb0 + 2)
    assert gcnsa.tc_status() == 0
    gcnsa.tc_clear()
    assert gcnsa.tc_status() == 0


def test_plain_tf32_products_are_outside_the_bar_of_the_training_path():
    """GEMM_TF32 issues one TF32 product per term on the same kernel.  Measured here so that the choice of the
    three-term split stays checked: the error is tens of times that of the split and above the 1e-4 of the largest
    entry that the training path is held to."""
    rng = np.random.default_rng(3)
    worst = {}
    for m, n, k in ((1000, 128, 602), (2000, 41, 128), (3000, 128, 47)):
        a = rng.standard_normal((m, k)).astype(np.float32)
        b = rng.standard_normal((k, n)).astype(np.float32)
        want = a.astype(np.float64) @ b.astype(np.float64)
        ad, bd = _padded(a, _ld(k)), _padded(b, _ld(n))
        ws = torch.empty(gcnsa.op_gemm_workspace(0, 0, m, n, k, gcnsa.GEMM_TF32X3) // 4 + 64, device="cuda")
        for mode in (gcnsa.GEMM_TF32, gcnsa.GEMM_TF32X3):
            cd = torch.empty((m, _ld(n)), device="cuda")
            gcnsa.op_gemm(ad, bd, cd, m, n, k, workspace=ws, mode=mode)
            err = np.abs(cd[:, :n].cpu().numpy() - want).max() / np.abs(want).max()
            worst[mode] = max(worst.get(mode, 0.0), err)
    assert gcnsa.tc_status() == 0
    assert worst[gcnsa.GEMM_TF32X3] <= 1e-5
    assert 1e-4 < worst[gcnsa.GEMM_TF32] < 5e-3, worst


@pytest.mark.parametrize("m", [777, 30_011])
@pytest.mark.parametrize("ta,tb", [(0, 0), (0, 1), (1, 0)])
def test_tensor_core_gemm_wide_results_with_epilogues(ta, tb, m):
    """Results wider than 128 columns, with one work item per CTA (777 rows) and with three to four (30 011 rows:
    the epilogue of one item runs beside the products of the next): every epilogue, accumulation and a ragged edge."""
    rng = np.random.default_rng(17 + ta + 2 * tb)
    n, k = 256, 200
    a = rng.standard_normal((k, m) if ta else (m, k)).astype(np.float32)
    b = rng.standard_normal((n, k) if tb else (k, n)).astype(np.float32)
    base = (a.T if ta else a).astype(np.float64) @ (b.T if tb else b).astype(np.float64)
    ad, bd = _padded(a, _ld(a.shape[1])), _padded(b, _ld(b.shape[1]))
    ws = torch.empty(gcnsa.op_gemm_workspace(ta, tb, m, n, k, gcnsa.GEMM_TF32X3) // 4 + 64, device="cuda")
    bias = rng.standard_normal(n).astype(np.float32)
    mk = rng.standard_normal((m, n)).astype(np.float32)
    rs = rng.uniform(0.1, 2.0, m).astype(np.float32)
    c0 = rng.standard_normal((m, n)).astype(np.float32)
    tc0, fb0 = gcnsa.gemm_path_counts()
    for epi, aux, want in ((gcnsa.EPI_NONE, None, base), (gcnsa.EPI_BIAS_RELU, _dev(bias), np.maximum(base + bias, 0)),
                           (gcnsa.EPI_MASK, _padded(mk, n), base * (mk > 0)), (gcnsa.EPI_ROWSCALE, _dev(rs), base * rs[:, None])):
        cd = torch.full((m, n), 5.0, device="cuda")
        gcnsa.op_gemm(ad, bd, cd, m, n, k, ta=ta, tb=tb, epi=epi, aux=aux, workspace=ws, mode=gcnsa.GEMM_TF32X3)
        _close(cd.cpu().numpy(), want, tol=1e-5, what=f"wide result, epilogue {epi}")
    cd = _dev(c0)
    gcnsa.op_gemm(ad, bd, cd, m, n, k, ta=ta, tb=tb, accumulate=1, workspace=ws, mode=gcnsa.GEMM_TF32X3)
    _close(cd.cpu().numpy(), c0 + base, tol=1e-5, what="wide result, accumulate")
    # 250 of 256 columns (the last float4 chunks of the tile lie outside the matrix), unpadded result rows
    cd = torch.full((m, 252), 5.0, device="cuda")
    gcnsa.op_gemm(ad, bd, cd, m, 250, k, ta=ta, tb=tb, workspace=ws, mode=gcnsa.GEMM_TF32X3)
    _close(cd[:, :250].cpu().numpy(), base[:, :250], tol=1e-5, what="wide result, ragged columns")
    assert torch.all(cd[:, 250:] == 0)
    assert gcnsa.gemm_path_counts() == (tc0 + 6, fb0) and gcnsa.tc_status() == 0


@pytest.mark.parametrize("mode", [gcnsa.GEMM_TF32X3, gcnsa.GEMM_FP32])
@pytest.mark.parametrize("m,n,k,scale", [(777, 256, 200, True), (30_011, 128, 41, True), (30_011, 256, 47, False),
                                        (5_000, 41, 128, True), (40_003, 100, 256, True), (300, 130, 64, False)])
def test_masked_product_with_column_sums_and_row_scale(m, n, k, scale, mode):
    """C = (A W^T) .* [mask > 0], column sums of C added to `out`, rows of C scaled afterwards: the gradient of a
    hidden layer with the bias gradient of the layer below, against fp64.  With one work item per CTA and with
    several, results narrower and wider than a tile, a ragged last float4; on the tensor-core kernel in its
    epilogue, on the fp32 path as product + column-sum kernel."""
    rng = np.random.default_rng(m + 3 * n + k)
    a = rng.standard_normal((m, k)).astype(np.float32)
    wt = rng.standard_normal((n, k)).astype(np.float32)         # stored transposed: tb = 1
    mk = rng.standard_normal((m, n)).astype(np.float32)
    rs = rng.uniform(0.1, 2.0, m).astype(np.float32)
    out0 = rng.standard_normal(n).astype(np.float32)
    base = (a.astype(np.float64) @ wt.astype(np.float64).T) * (mk > 0)
    ad, bd, md = _padded(a, _ld(k)), _padded(wt, _ld(k)), _padded(mk, _ld(n))
    cd = torch.full((m, _ld(n)), 7.0, device="cuda")
    out = _dev(out0)
    ws = torch.empty(gcnsa.op_gemm_workspace(0, 1, m, n, k, mode) // 4 + 64, device="cuda")
    sc = torch.empty(gcnsa.op_gemm_mask_colsum_scratch(m, n) // 4, device="cuda")
    tc0, fb0 = gcnsa.gemm_path_counts()
    gcnsa.op_gemm_mask_colsum(ad, bd, cd, m, n, k, md, out, row_scale=_dev(rs) if scale else None, tb=1, accumulate=1,
                              scratch=sc, workspace=ws, mode=mode)
    want_c = base * rs[:, None] if scale else base
    _close(cd[:, :n].cpu().numpy(), want_c, tol=1e-5, what="masked product")
    assert torch.all(cd[:, n:_ld(n)] == 0)
    _close(out.cpu().numpy(), out0 + base.sum(axis=0), tol=2e-5, what="column sums of the unscaled product")
    if mode == gcnsa.GEMM_TF32X3:
        assert gcnsa.gemm_path_counts() == (tc0 + 1, fb0) and gcnsa.tc_status() == 0
    # the same sums every time
    out2 = _dev(out0)
    gcnsa.op_gemm_mask_colsum(ad, bd, cd, m, n, k, md, out2, row_scale=_dev(rs) if scale else None, tb=1, accumulate=1,
                              scratch=sc, workspace=ws, mode=mode)
    assert torch.equal(out, out2)
    # without accumulate the sums replace what was there
    out3 = torch.full((n,), 5.0, device="cuda")
    gcnsa.op_gemm_mask_colsum(ad, bd, cd, m, n, k, md, out3, tb=1, scratch=sc, workspace=ws, mode=mode)
    _close(out3.cpu().numpy(), base.sum(axis=0), tol=2e-5, what="column sums, not accumulated")


def _probe_reference(x, n_rows, window_rows, hit_every, rounds, warps):
    """The gather probe's documented draws, in integer numpy, and the lane-wise sums of the rows they name."""
    w = np.arange(warps, dtype=np.uint64)
    s = (np.uint64(0x9E3779B9) * (w + np.uint64(1))) & np.uint64(0xFFFFFFFF)
    base = ((w // np.uint64(8)) * np.uint64(977)) % np.uint64(n_rows - window_rows + 1)
    acc = np.zeros((warps, 128), np.float64)
    for _ in range(rounds):
        for u in range(16):
            s = (s * np.uint64(1664525) + np.uint64(1013904223)) & np.uint64(0xFFFFFFFF)
            s = s ^ (s >> np.uint64(15))
            near = hit_every > 0 and u % hit_every == 0
            r = base + ((s * np.uint64(window_rows)) >> np.uint64(32)) if near else (s * np.uint64(n_rows)) >> np.uint64(32)
            acc += x[r.astype(np.int64), :128]
    return acc


@pytest.mark.parametrize("hit_every", [0, 1, 4])
def test_gather_probe_gathers_the_documented_rows(hit_every):
    """The measuring stick of the sparse products: its sums are those of the rows its generator names (small integer
    entries, so fp32 sums are exact), for every mix of window and whole-matrix draws."""
    rng = np.random.default_rng(9 + hit_every)
    n_rows, ld, window, rounds = 3_001, 132, 64, 3
    x = rng.integers(-8, 9, size=(n_rows, ld)).astype(np.float32)
    warps = gcnsa.gather_probe_warps()
    assert warps % 8 == 0 and warps >= 8
    out = torch.full((warps, 128), -1.0, device="cuda")
    before = gcnsa.launch_count()
    gcnsa.op_gather_probe(_dev(x), n_rows, window, hit_every, rounds, out)
    assert gcnsa.launch_count() == before + 1
    want = _probe_reference(x, n_rows, window, hit_every, rounds, warps)
    assert np.array_equal(out.cpu().numpy().astype(np.float64), want)
    for bad in (dict(window_rows=0), dict(window_rows=n_rows + 1), dict(hit_every=-1), dict(rounds=-1)):
        kw = dict(window_rows=window, hit_every=hit_every, rounds=rounds)
        kw.update(bad)
        with pytest.raises(gcnsa.GcnsaError):
            gcnsa.op_gather_probe(_dev(x), n_rows, kw["window_rows"], kw["hit_every"], kw["rounds"], out)
    with pytest.raises(gcnsa.GcnsaError):
        gcnsa.op_gather_probe(_dev(x), n_rows, window, hit_every, rounds, out[:8])
