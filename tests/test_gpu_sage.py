"""GPU parity of the GraphSAGE variant (mean aggregator, sampled neighbours,
mini-batches, per-worker Adam, parameters averaged per epoch) through the C-ABI
against the fp64 checker on the same seeded inputs.

Bars: batch membership and sampled neighbour sets identical (compared as sets:
every draw is a set of unique keys); embeddings, logits, gradients within
1e-4 * max|reference|; epoch loss within 1e-3 relative at every epoch."""
import numpy as np
import pytest
import torch

from gen import configs
from oracle import oracle, sage
from paper_2012_04930_b200 import gcnsa

from parity_helpers import TOL, ambiguous_units, close

pytestmark = pytest.mark.gpu


def _setup(w, hidden, fanout, batch, lr, gemm_mode):
    dims = [w.dims[0], hidden, w.dims[-1]]
    ws, wn, bs = configs.sage_weights(dims, w.seed + 77)
    env = gcnsa.make_env(0)
    parts = gcnsa.Parts(env, w.rowptr, w.col, w.x, w.y, w.train_mask, w.dims[-1], w.m, w.overlap_ppm, w.seed,
                        w.part_mode, w.user_part, w.loss_on_halo)
    model = gcnsa.Sage(env, parts, dims, ws, wn, bs, fanout=fanout, batch=batch, lr=lr, seed=w.seed, gemm_mode=gemm_mode)
    _, rparts = oracle.build_partitions(w.rowptr, w.col, w.m, w.overlap_ppm, w.seed, w.part_mode, w.user_part)
    params = [ws[0].astype(np.float64), wn[0].astype(np.float64), bs[0].astype(np.float64),
              ws[1].astype(np.float64), wn[1].astype(np.float64), bs[1].astype(np.float64)]
    xs = [w.x[pt.members].astype(np.float64) for pt in rparts]
    ys = [w.y[pt.members] for pt in rparts]
    trs = [oracle.train_set(pt, w.train_mask[pt.members], w.loss_on_halo) for pt in rparts]
    return env, parts, model, rparts, params, xs, ys, trs


def _relu_decisions(fw, e):
    """ReLU on / off per hidden unit for the checker's backward pass: its own sign of z, except where |z| is
    within fp32 resolution of zero (parity_helpers.ambiguous_units, from the checker's values alone); there the
    kernel's decision is taken, after checking that its value is equally tiny.  Away from zero both must agree."""
    z = fw["z1"]
    amb = ambiguous_units([z])[0]
    on = z > 0.0
    seen = np.zeros(z.shape[0], bool)
    for j, v in enumerate(e["vertices"]):
        if v < 0:
            continue
        k = fw["where"][int(v)]
        h = e["hidden"][j]
        assert np.all(np.abs(h[amb[k]]) < 2e-5 * np.abs(z).max())
        assert np.array_equal((h > 0)[~amb[k]], on[k][~amb[k]]), "ReLU decisions differ away from zero"
        if not seen[k]:
            on[k] = np.where(amb[k], h > 0, on[k])
            seen[k] = True
    assert amb.sum() <= 1e-3 * z.size + 2
    return on


def _gpu_params(model, base):
    return [model.get(base + k, l) for l in (0, 1) for k in (0, 1, 2)]


def _check_batch(model, pt, x, y, params, tg, seed, epoch, fanout, p, b):
    """One batch on both sides: membership, both layers' sample sets, embeddings, logits, loss, logit gradient and
    the six parameter gradients."""
    fw = sage.batch_forward(pt, x, params, tg, y, seed, epoch, fanout)
    model.run_batch(p, epoch, b, apply=False)
    e = model.batch_export()
    grads, g = sage.batch_backward(fw, x, params, relu_on=_relu_decisions(fw, e))
    nb, r1, r2 = tg.size, fanout[0], fanout[1]
    assert e["nb"] == nb and np.array_equal(e["vertices"][:nb], tg), "batch membership and order"
    # the output layer's samples: slots nb + i r2 + s
    slots = e["vertices"][nb:].reshape(nb, r2)
    for i in range(nb):
        c = int(e["count2"][i])
        assert c == fw["c2"][i] and sorted(slots[i, :c]) == list(fw["s2"][i, :c]) and np.all(slots[i, c:] == -1)
    # the hidden layer's samples and embeddings, row by row against the checker's record of that vertex
    for j, v in enumerate(e["vertices"]):
        if v < 0:
            assert e["count1"][j] == 0
            continue
        k = fw["where"][int(v)]
        c = int(e["count1"][j])
        assert c == fw["c1"][k] and sorted(e["samples1"][j, :c]) == list(fw["s1"][k, :c])
    valid = e["vertices"] >= 0
    rows = np.array([fw["where"][int(v)] for v in e["vertices"][valid]])
    close(e["hidden"][valid], fw["h1"][rows], what=f"p{p} b{b} hidden layer")
    close(e["logits"], fw["logits"], what=f"p{p} b{b} logits")
    close(e["dlogits"], g, what=f"p{p} b{b} dlogits")
    assert abs(float(e["loss"][0]) - fw["loss"]) <= 1e-5 * abs(fw["loss"])
    for got, want, nm in zip(_gpu_params(model, gcnsa.SAGE_GRAD_W_SELF), grads,
                             ("dWs1", "dWn1", "db1", "dWs2", "dWn2", "db2")):
        close(got, want, what=f"p{p} b{b} {nm}")


@pytest.mark.parametrize("gemm_mode", [gcnsa.GEMM_FP32, gcnsa.GEMM_TF32X3])
@pytest.mark.parametrize("name,hidden,fanout,batch", [("tiny", 16, (5, 3), 64), ("tiny", 16, (25, 10), 256),
                                                      ("small", 64, (25, 10), 256), ("small", 32, (2, 40), 100)])
def test_one_batch_matches_checker(name, hidden, fanout, batch, gemm_mode, tiny_wl, small_wl):
    w = tiny_wl if name == "tiny" else small_wl
    env, parts, model, rparts, params, xs, ys, trs = _setup(w, hidden, fanout, batch, 0.01, gemm_mode)
    tc0, fb0 = gcnsa.gemm_path_counts()
    for p, epoch in ((0, 0), (w.m - 1, 3)):
        pt = rparts[p]
        want_batches = sage.batches(pt, trs[p], w.seed, epoch, batch)
        assert model.n_batches(p) == len(want_batches)
        for b in sorted({0, len(want_batches) - 1}):         # a full batch and the ragged last one
            _check_batch(model, pt, xs[p], ys[p], params, want_batches[b], w.seed, epoch, fanout, p, b)
    if gemm_mode == gcnsa.GEMM_TF32X3:
        tc1, fb1 = gcnsa.gemm_path_counts()
        assert tc1 > tc0 and fb1 == fb0 and gcnsa.tc_status() == 0
    # one Adam step of worker 0 on the last computed gradient of a fresh batch
    pt = rparts[0]
    tg = sage.batches(pt, trs[0], w.seed, 0, batch)[0]
    fw = sage.batch_forward(pt, xs[0], params, tg, ys[0], w.seed, 0, fanout)
    model.run_batch(0, 0, 0, apply=False)
    grads, _ = sage.batch_backward(fw, xs[0], params, relu_on=_relu_decisions(fw, model.batch_export()))
    g_own = [a.astype(np.float64) for a in _gpu_params(model, gcnsa.SAGE_GRAD_W_SELF)]
    model.run_batch(0, 0, 0, apply=True)
    ref = oracle.Adam(params, 0.01).step(params, grads)
    own = oracle.Adam(params, 0.01).step(params, g_own)
    for got, r, o, gr in zip(_gpu_params(model, gcnsa.SAGE_WORK_W_SELF), ref, own, grads):
        scale = max(np.abs(r).max(), 0.01)
        assert np.abs(got - o).max() <= 1e-5 * scale          # the kernel's step on its own gradient
        firm = np.abs(gr) >= 1e-3 * np.abs(gr).max()          # where the sign of the gradient is determined in fp32
        if firm.any():
            assert np.abs(got - r)[firm].max() <= TOL * scale
    for got, p0 in zip(_gpu_params(model, gcnsa.SAGE_W_SELF), params):
        assert np.array_equal(got, p0.astype(np.float32)), "the aggregated parameters move at the end of an epoch only"
    model.close(); parts.close()


@pytest.mark.parametrize("name,hidden,fanout,batch,epochs,lr", [("tiny", 16, (25, 10), 256, 10, 0.003),
                                                               ("small", 64, (25, 10), 256, 5, 0.0005)])
def test_loss_curve_and_averaged_parameters_match_checker(name, hidden, fanout, batch, epochs, lr, tiny_wl, small_wl):
    w = tiny_wl if name == "tiny" else small_wl
    env, parts, model, rparts, params, xs, ys, trs = _setup(w, hidden, fanout, batch, lr, gcnsa.GEMM_TF32X3)
    opts = [oracle.Adam(params, lr) for _ in rparts]
    loss = torch.zeros(1, device="cuda")
    first = None
    for e in range(epochs):
        params, want = sage.epoch(rparts, xs, ys, trs, params, opts, w.seed, e, fanout, batch)
        model.epoch(loss.data_ptr())
        got = loss.item()
        assert abs(got - want) <= 1e-3 * abs(want), (e, got, want)
        first = want if first is None else first
    assert want < first, "training must reduce the loss"
    assert model.epochs_done == epochs and gcnsa.tc_status() == 0
    for got, ref, nm in zip(_gpu_params(model, gcnsa.SAGE_W_SELF), params, ("Ws1", "Wn1", "b1", "Ws2", "Wn2", "b2")):
        close(got, ref, tol=5e-3, what=f"{nm} after {epochs} epochs")
    model.close(); parts.close()


def test_batches_at_paper_scale_match_checker():
    """The configuration the benchmark's GraphSAGE line times (232 965 vertices, 602 -> 128 -> 41, fan-outs 25 / 10,
    batches of 256, tensor-core products): the first, a middle and the ragged last batch of two workers, in two
    different epochs, against the checker."""
    w = configs.paper_scale()
    fanout, batch = (25, 10), 256
    env, parts, model, rparts, params, xs, ys, trs = _setup(w, 128, fanout, batch, 1e-4, gcnsa.GEMM_TF32X3)
    tc0, fb0 = gcnsa.gemm_path_counts()
    for p, epoch in ((1, 0), (4, 2)):
        pt = rparts[p]
        want_batches = sage.batches(pt, trs[p], w.seed, epoch, batch)
        assert model.n_batches(p) == len(want_batches) > 100
        for b in (0, len(want_batches) // 2, len(want_batches) - 1):
            _check_batch(model, pt, xs[p], ys[p], params, want_batches[b], w.seed, epoch, fanout, p, b)
    tc1, fb1 = gcnsa.gemm_path_counts()
    assert tc1 > tc0 and fb1 == fb0 and gcnsa.tc_status() == 0
    model.close(); parts.close()


def test_recorded_batches_equal_plain_launches(small_wl):
    """batch_graph: a worker's full-size batches replay one recorded kernel sequence whose batch index and epoch
    live in device memory.  Losses, parameters and the launch counter equal those of plain launches, bit for bit,
    over three epochs (ten full batches and a ragged one per worker)."""
    w = small_wl
    dims = [w.dims[0], 64, w.dims[-1]]
    ws, wn, bs = configs.sage_weights(dims, w.seed + 77)
    results = []
    with torch.cuda.stream(torch.cuda.Stream()):      # a recording needs a stream other than the legacy default one
        for batch_graph in (0, 1):
            env = gcnsa.make_env(0)
            parts = gcnsa.Parts(env, w.rowptr, w.col, w.x, w.y, w.train_mask, w.dims[-1], w.m, w.overlap_ppm, w.seed,
                                w.part_mode, w.user_part, w.loss_on_halo)
            model = gcnsa.Sage(env, parts, dims, ws, wn, bs, fanout=(25, 10), batch=256, lr=5e-4, seed=w.seed,
                               gemm_mode=gcnsa.GEMM_TF32X3, batch_graph=batch_graph)
            assert all(model.n_batches(p) >= 5 for p in range(w.m))
            loss = torch.zeros(1, device="cuda")
            losses, n0 = [], gcnsa.launch_count()
            for _ in range(3):
                model.epoch(loss.data_ptr())
                losses.append(loss.item())
            launches = gcnsa.launch_count() - n0
            results.append((losses, _gpu_params(model, gcnsa.SAGE_W_SELF), launches))
            assert gcnsa.tc_status() == 0
            model.close(); parts.close()
    (l0, p0, n0), (l1, p1, n1) = results
    assert l0 == l1, (l0, l1)
    for a, b in zip(p0, p1):
        assert np.array_equal(a, b)
    # the recorded sequence has one kernel more per full batch (its first, which advances the index and takes the
    # batch's vertices, where the plain sequence has a copy) and one per worker and epoch that resets the index
    assert n1 > n0


def test_runs_are_bitwise_reproducible_and_arguments_are_checked(tiny_wl):
    w = tiny_wl
    outs = []
    for _ in range(2):
        env, parts, model, *_ = _setup(w, 16, (4, 3), 128, 0.01, gcnsa.GEMM_TF32X3)
        for _ in range(2):
            model.epoch()
        outs.append(_gpu_params(model, gcnsa.SAGE_W_SELF))
        if len(outs) == 2:
            for bad in (lambda: model.run_batch(0, 0, 10_000), lambda: model.run_batch(9, 0, 0),
                        lambda: model.run_batch(0, -1, 0), lambda: model.get(99, 0), lambda: model.get(0, 2)):
                with pytest.raises(gcnsa.GcnsaError) as ei:
                    bad()
                assert ei.value.code == gcnsa.ERR_ARG
        model.close(); parts.close()
    for a, b in zip(*outs):
        assert np.array_equal(a, b)
    env = gcnsa.make_env(0)
    parts = gcnsa.Parts(env, w.rowptr, w.col, w.x, w.y, w.train_mask, w.dims[-1], w.m, w.overlap_ppm, w.seed, w.part_mode,
                        w.user_part)
    ws, wn, bs = configs.sage_weights([64, 16, 5], 1)
    for kw in (dict(batch=0), dict(fanout=(-1, 3)), dict(lr=0.0)):
        with pytest.raises(gcnsa.GcnsaError) as ei:
            gcnsa.Sage(env, parts, [64, 16, 5], ws, wn, bs, **kw)
        assert ei.value.code == gcnsa.ERR_ARG
    with pytest.raises(gcnsa.GcnsaError):
        gcnsa.Sage(env, parts, [63, 16, 5], ws, wn, bs)        # width does not match the partitions
    parts.close()
