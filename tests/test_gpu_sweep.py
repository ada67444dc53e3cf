"""Parity of the sweep configuration: one GCN layer of equal input and output
width (forward + backward + step), on the dense power-law graph and on the
degree-32 random graph, at 1, 5 and 16 partitions and narrow to wide feature
widths, against the fp64 checker.  Reduced graphs for the grid of cases; one
point on the complete 1 M-vertex degree-32 graph, where the gathered matrix
exceeds L2 and the sparse product runs against the HBM roof."""
import numpy as np
import pytest
import torch

from gen import configs
from oracle import oracle
from paper_2012_04930_b200 import gcnsa

from parity_helpers import TOL, close

pytestmark = pytest.mark.gpu

_GRAPHS = {}


def _graph(kind, scale):
    if (kind, scale) not in _GRAPHS:
        _GRAPHS[(kind, scale)] = configs.sweep_graph(kind, scale=scale)
    return _GRAPHS[(kind, scale)]


def _one_layer_step(w, gemm_mode, check_structure=True, **opts):
    assert len(w.dims) == 2 and w.dims[0] == w.dims[1]
    env = gcnsa.make_env(0)
    parts = gcnsa.Parts(env, w.rowptr, w.col, w.x, w.y, w.train_mask, w.dims[-1], w.m, w.overlap_ppm, w.seed,
                        w.part_mode, w.user_part, w.loss_on_halo)
    model = gcnsa.Model(env, parts, w.dims, w.w0, w.b0, lr=w.lr, beta1=w.beta1, beta2=w.beta2, eps=w.eps,
                        gemm_mode=gemm_mode, epoch_graph=0, **opts)
    part, rparts = oracle.build_partitions(w.rowptr, w.col, w.m, w.overlap_ppm, w.seed, w.part_mode, w.user_part)
    assert np.array_equal(parts.assignment(), part)
    ws = [w.w0[0].astype(np.float64)]
    bs = [w.b0[0].astype(np.float64)]
    gw, gb = np.zeros_like(ws[0]), np.zeros_like(bs[0])
    losses = torch.zeros(w.m, device="cuda")
    want_losses = []
    tc0, fb0 = gcnsa.gemm_path_counts()
    for pt in rparts:
        p = pt.p
        if check_structure:
            e = parts.export(p)
            assert np.array_equal(e["members"], pt.members)
            for k in ("rowptr", "col", "t_rowptr", "t_col"):
                assert np.array_equal(e[k], getattr(pt, k)), k
            assert np.abs(e["val"] - pt.val).max() <= 2e-7 * pt.val.max()
        fw = oracle.forward(pt, w.x[pt.members], ws, bs, w.y[pt.members], w.train_mask[pt.members], w.loss_on_halo)
        bw = oracle.backward(pt, fw, ws, w.y[pt.members])     # a single layer: no ReLU on the way back
        model.forward(p, losses[p:p + 1].data_ptr())
        logits = model.get(gcnsa.GET_ACT, 1, rows=pt.n)
        if opts.get("loss_rows_only"):
            t = fw["t"]
            close(logits[t], fw["Z"][0][t], what=f"p{p} logits on the loss rows")
        else:
            close(logits, fw["Z"][0], what=f"p{p} logits")
        close(model.get(gcnsa.GET_DLOGITS, rows=pt.n), bw["G"][0], what=f"p{p} dlogits")
        model.backward(p)
        gw += bw["dW"][0]; gb += bw["db"][0]
        want_losses.append(fw["loss"])
    assert np.allclose(losses.cpu().numpy(), want_losses, rtol=2e-5)
    close(model.get(gcnsa.GET_GRAD_W, 0), gw, what="dW")
    close(model.get(gcnsa.GET_GRAD_B, 0), gb, what="db")
    if gemm_mode == gcnsa.GEMM_TF32X3:
        tc1, fb1 = gcnsa.gemm_path_counts()
        assert tc1 > tc0 and fb1 == fb0
    g_own = [model.get(gcnsa.GET_GRAD_W, 0).astype(np.float64), model.get(gcnsa.GET_GRAD_B, 0).astype(np.float64)]
    model.step()
    # Adam's first step moves an entry by about lr * sign(g): entries whose gradient is below fp32 resolution have no
    # determined sign, so the checker's step on its own gradient is compared where |g| >= 1e-3 max|g|, and its step on
    # the kernel's gradient everywhere
    ref = oracle.Adam(ws + bs, w.lr, w.beta1, w.beta2, w.eps).step(ws + bs, [gw / w.m, gb / w.m])
    own = oracle.Adam(ws + bs, w.lr, w.beta1, w.beta2, w.eps).step(ws + bs, [g / w.m for g in g_own])
    for got, r, o, g in zip((model.get(gcnsa.GET_W, 0), model.get(gcnsa.GET_B, 0)), ref, own, (gw, gb)):
        scale = max(np.abs(r).max(), w.lr)
        assert np.abs(got - o).max() <= 1e-5 * scale
        firm = np.abs(g) >= 1e-3 * np.abs(g).max()
        if firm.any():
            assert np.abs(got - r)[firm].max() <= TOL * scale
    assert gcnsa.tc_status() == 0
    model.close(); parts.close()


@pytest.mark.parametrize("gemm_mode", [gcnsa.GEMM_FP32, gcnsa.GEMM_TF32X3])
@pytest.mark.parametrize("width", [16, 64, 602])
@pytest.mark.parametrize("m", [1, 5, 16])
@pytest.mark.parametrize("kind", ["regular", "paper"])
def test_sweep_points_match_checker(kind, m, width, gemm_mode):
    w = configs.sweep_point(kind, width, m, scale=0.02, prebuilt=_graph(kind, 0.02))
    _one_layer_step(w, gemm_mode, factored_norm=1, loss_rows_only=0)


@pytest.mark.parametrize("kind,m,width", [("regular", 5, 128), ("paper", 16, 256)])
def test_sweep_points_in_the_other_option_sets(kind, m, width):
    """Stored values instead of the factored normalization, and the last (here: only) layer on the loss rows only."""
    w = configs.sweep_point(kind, width, m, scale=0.02, prebuilt=_graph(kind, 0.02))
    _one_layer_step(w, gcnsa.GEMM_TF32X3, factored_norm=0, loss_rows_only=0)
    _one_layer_step(w, gcnsa.GEMM_TF32X3, factored_norm=1, loss_rows_only=1)


def test_sweep_point_on_the_complete_regular_graph():
    """1 M vertices, degree about 32, one partition, width 128: the gathered matrix (512 MB) exceeds L2."""
    w = configs.sweep_point("regular", 128, 1)
    assert w.n == 1_000_000 and 31.0 < w.nnz / w.n <= 32.0
    _one_layer_step(w, gcnsa.GEMM_TF32X3, factored_norm=1, loss_rows_only=0)
