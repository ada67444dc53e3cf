"""Parity at the benchmark's full sizes, in the launch configuration bench.py
times (tensor-core GEMMs): the paper-scale workload (232 965 vertices, 114.6 M non-zeros, 602 ->
128 -> 41, five partitions) and the large sparse one (2.45 M vertices, 123.7 M
non-zeros, 100 -> 256 -> 256 -> 47, ten partitions).  The checker is fast
enough to compute whole partitions at these sizes, so tensors are compared in
full rather than sampled."""
import numpy as np
import pytest
import torch

from gen import configs
from oracle import oracle
from paper_2012_04930_b200 import gcnsa

from parity_helpers import TOL, close as _close, relu_decisions as _relu_decisions

pytestmark = pytest.mark.gpu


# "plain": every option off.  "bench": the launch configuration bench.py times (last-layer logits only on the
# rows that carry loss, normalization factored out of the sparse products, recorded epoch).
CONFIGS = {"plain": dict(loss_rows_only=0, factored_norm=0, epoch_graph=0),
           "bench": dict(loss_rows_only=1, factored_norm=1, epoch_graph=1)}


def _make(w, config, gemm_mode=gcnsa.GEMM_TF32X3):
    env = gcnsa.make_env(0)   # torch's current stream: the caller makes a side stream current for "bench"
    parts = gcnsa.Parts(env, w.rowptr, w.col, w.x, w.y, w.train_mask, w.dims[-1], w.m, w.overlap_ppm, w.seed,
                        w.part_mode, w.user_part, w.loss_on_halo)
    model = gcnsa.Model(env, parts, w.dims, w.w0, w.b0, lr=w.lr, beta1=w.beta1, beta2=w.beta2, eps=w.eps,
                        gemm_mode=gemm_mode, **CONFIGS[config])
    return env, parts, model


def _structure(parts, part, rparts):
    assert np.array_equal(parts.assignment(), part)
    for pt in rparts:
        e = parts.export(pt.p)
        assert np.array_equal(e["members"], pt.members)
        for k in ("rowptr", "col", "t_rowptr", "t_col"):
            assert np.array_equal(e[k], getattr(pt, k)), k
        assert np.abs(e["val"] - pt.val).max() <= 2e-7 * pt.val.max()
        assert np.abs(e["t_val"] - pt.t_val).max() <= 2e-7 * pt.t_val.max()
        assert [int(d) for i, d in enumerate(e["depth"]) if i != pt.p] == [pt.depth_by_op[op] for op in sorted(pt.depth_by_op)]


def _one_epoch(w, model, parts, rparts, check_acts_on, loss_rows_only=False):
    """Forward + backward on every partition on both sides; returns the
    checker's gradient sums and losses after comparing tensors."""
    L = len(w.w0)
    ws = [a.astype(np.float64) for a in w.w0]
    bs = [b.astype(np.float64) for b in w.b0]
    gw = [np.zeros_like(a) for a in ws]
    gb = [np.zeros_like(b) for b in bs]
    losses_ref, losses = [], torch.zeros(w.m, device="cuda")
    for pt in rparts:
        p = pt.p
        fw = oracle.forward(pt, w.x[pt.members], ws, bs, w.y[pt.members], w.train_mask[pt.members], w.loss_on_halo)
        model.forward(p, losses[p:p + 1].data_ptr())
        h_gpu = [model.get(gcnsa.GET_ACT, l, rows=pt.n) for l in range(1, L)]
        if p in check_acts_on:
            for l in range(1, L):
                _close(h_gpu[l - 1], fw["H"][l], what=f"p{p} H{l}")
            logits = model.get(gcnsa.GET_ACT, L, rows=pt.n)
            if loss_rows_only:   # the other rows are not computed
                t = oracle.train_set(pt, w.train_mask[pt.members], w.loss_on_halo).astype(bool)
                _close(logits[t], fw["H"][L][t], what=f"p{p} logits on the loss rows")
            else:
                _close(logits, fw["H"][L], what=f"p{p} logits")
        bw = oracle.backward(pt, fw, ws, w.y[pt.members], relu_on=_relu_decisions(fw, h_gpu))
        if p in check_acts_on:
            _close(model.get(gcnsa.GET_DLOGITS, rows=pt.n), bw["G"][L - 1], what=f"p{p} dlogits")
        model.backward(p)
        for l in range(L):
            gw[l] += bw["dW"][l]; gb[l] += bw["db"][l]
        losses_ref.append(fw["loss"])
    assert np.allclose(losses.cpu().numpy(), losses_ref, rtol=2e-5)
    for l in range(L):
        _close(model.get(gcnsa.GET_GRAD_W, l), gw[l], what=f"dW{l}")
        _close(model.get(gcnsa.GET_GRAD_B, l), gb[l], what=f"db{l}")
    return ws, bs, gw, gb, losses_ref


def _check_step(w, model, ws, bs, gw, gb):
    """After gcnsa_step: Adam's first step moves every entry by about
    lr * sign(g), so an entry whose gradient is below fp32 resolution has no
    determined sign.  Entries with |g| >= 1e-3 max|g| are compared with the
    checker's step on the checker's gradient; all entries are compared with
    the checker's step on the kernel's own gradient."""
    L = len(ws)
    g_gpu = [model.get(gcnsa.GET_GRAD_W, l).astype(np.float64) for l in range(L)] + \
            [model.get(gcnsa.GET_GRAD_B, l).astype(np.float64) for l in range(L)]
    model.step()
    new_ref = oracle.Adam(ws + bs, w.lr, w.beta1, w.beta2, w.eps).step(ws + bs, [g / w.m for g in gw + gb])
    new_own = oracle.Adam(ws + bs, w.lr, w.beta1, w.beta2, w.eps).step(ws + bs, [g / w.m for g in g_gpu])
    got = [model.get(gcnsa.GET_W, l) for l in range(L)] + [model.get(gcnsa.GET_B, l) for l in range(L)]
    for i, (a, ref, own, g) in enumerate(zip(got, new_ref, new_own, gw + gb)):
        scale = max(np.abs(ref).max(), w.lr)
        assert np.abs(a - own).max() <= 1e-5 * scale, f"param {i}: Adam kernel differs on its own gradient"
        firm = np.abs(g) >= 1e-3 * np.abs(g).max()
        assert firm.mean() > 0.98
        assert np.abs(a - ref)[firm].max() <= TOL * scale, f"param {i} after one step"
    return new_ref


@pytest.mark.parametrize("config", ["plain", "bench"])
def test_paper_scale_epoch_matches_checker(config):
    # a recorded epoch needs a stream other than the legacy default stream, as in bench.py
    stream = torch.cuda.Stream() if CONFIGS[config].get("epoch_graph") else torch.cuda.current_stream()
    with torch.cuda.stream(stream):
        _paper_scale_epoch_matches_checker(config)


def _paper_scale_epoch_matches_checker(config):
    w = configs.paper_scale()
    assert (w.n, w.nnz, w.dims, w.m) == (232_965, 114_600_000, [602, 128, 41], 5)
    env, parts, model = _make(w, config)
    part, rparts = oracle.build_partitions(w.rowptr, w.col, w.m, w.overlap_ppm, w.seed, w.part_mode, w.user_part)
    _structure(parts, part, rparts)
    for pt in rparts:
        i = parts.info(pt.p)
        assert (i.n_owned, i.n_halo, i.nts) == (pt.n_owned, 4 * 1164, 1164)   # 2.5 % of N_p from each of 4 others
    ws, bs, gw, gb, losses = _one_epoch(w, model, parts, rparts, check_acts_on={0, 3},
                                        loss_rows_only=config == "bench")
    new = _check_step(w, model, ws, bs, gw, gb)
    # the loss curve: 50 epochs in the configuration the benchmark times (the checker needs about four seconds per
    # epoch on 16 cores), 3 on the plain path
    _loss_curve(w, model, rparts, ws, bs, gw, gb, new, epochs=50 if config == "bench" else 3)
    assert gcnsa.tc_status() == 0
    model.close(); parts.close()


def _loss_curve(w, model, rparts, ws, bs, gw, gb, after_first, epochs):
    """Epochs 2 .. `epochs` on both sides (epoch 1 was the step-by-step comparison): the epoch loss within 1e-3
    relative at every epoch."""
    L = len(ws)
    opt = oracle.Adam(ws + bs, w.lr, w.beta1, w.beta2, w.eps)
    opt.step(ws + bs, [g / w.m for g in gw + gb])
    ws, bs = after_first[:L], after_first[L:]
    loss = torch.zeros(1, device="cuda")
    xs = [w.x[pt.members].astype(np.float64) for pt in rparts]
    ys = [w.y[pt.members] for pt in rparts]
    mks = [w.train_mask[pt.members] for pt in rparts]
    for e in range(1, epochs):
        ws, bs, want, _ = oracle.epoch(rparts, xs, ys, mks, ws, bs, opt, w.loss_on_halo)
        model.epoch(loss.data_ptr())
        assert abs(loss.item() - want) <= 1e-3 * abs(want), (e, loss.item(), want)


@pytest.mark.parametrize("config", ["plain", "bench"])
def test_large_sparse_epoch_matches_checker(config):
    # a recorded epoch needs a stream other than the legacy default stream, as in bench.py
    stream = torch.cuda.Stream() if CONFIGS[config].get("epoch_graph") else torch.cuda.current_stream()
    with torch.cuda.stream(stream):
        _large_sparse_epoch_matches_checker(config)


def _large_sparse_epoch_matches_checker(config):
    w = configs.large_sparse()
    assert (w.n, w.nnz, w.dims, w.m) == (2_450_000, 123_700_000, [100, 256, 256, 47], 10)
    env, parts, model = _make(w, config)
    part, rparts = oracle.build_partitions(w.rowptr, w.col, w.m, w.overlap_ppm, w.seed, w.part_mode, w.user_part)
    _structure(parts, part, rparts)
    ws, bs, gw, gb, losses = _one_epoch(w, model, parts, rparts, check_acts_on={0, 7},
                                        loss_rows_only=config == "bench")
    new = _check_step(w, model, ws, bs, gw, gb)
    if config == "bench":   # five more epochs of the loss curve
        _loss_curve(w, model, rparts, ws, bs, gw, gb, new, epochs=6)
    assert gcnsa.tc_status() == 0
    model.close(); parts.close()
