"""GPU parity of the whole path through the C-ABI: gcnsa_build_partitions,
gcnsa_forward, gcnsa_backward, gcnsa_step against the fp64 checker on the same
seeded inputs.

Bars: bit-exact partition assignment, sampled vertex sets, CSR and transposed
CSR indices; fp32 tensors within 1e-4 * max|reference| after one step; epoch
loss within 1e-3 relative at every epoch."""
import numpy as np
import pytest
import torch

from gen import configs
from oracle import oracle
from paper_2012_04930_b200 import gcnsa

from parity_helpers import TOL, close as _close, relu_decisions as _relu_decisions

pytestmark = pytest.mark.gpu


def _make(w, **kw):
    env = gcnsa.make_env(0)
    parts = gcnsa.Parts(env, w.rowptr, w.col, w.x, w.y, w.train_mask, w.dims[-1], w.m, w.overlap_ppm, w.seed,
                        w.part_mode, w.user_part, kw.get("loss_on_halo", w.loss_on_halo))
    model = gcnsa.Model(env, parts, w.dims, w.w0, w.b0, use_bias=kw.get("use_bias", 1), lr=w.lr, beta1=w.beta1,
                        beta2=w.beta2, eps=w.eps, gemm_mode=kw.get("gemm_mode", gcnsa.GEMM_FP32),
                        factored_norm=kw.get("factored_norm", 0), loss_rows_only=0, epoch_graph=0)
    return env, parts, model


def _check_structure(parts, ref_part, ref_parts):
    assert np.array_equal(parts.assignment(), ref_part)
    for p, pt in enumerate(ref_parts):
        e = parts.export(p)
        i = parts.info(p)
        assert (i.n_owned, i.n, i.nnz, i.nts) == (pt.n_owned, pt.n, pt.nnz, pt.nts)
        assert np.array_equal(e["members"], pt.members)
        for k in ("rowptr", "col", "t_rowptr", "t_col"):
            assert np.array_equal(e[k], getattr(pt, k)), k
        assert np.abs(e["val"] - pt.val).max() <= 2e-7 * pt.val.max()
        assert np.abs(e["t_val"] - pt.t_val).max() <= 2e-7 * pt.t_val.max()


@pytest.mark.parametrize("factored_norm", [0, 1])
@pytest.mark.parametrize("gemm_mode", [gcnsa.GEMM_FP32, gcnsa.GEMM_TF32X3])
@pytest.mark.parametrize("name", ["tiny", "small", "small_seed_7", "small_seed_123457"])
def test_one_step_matches_checker(name, gemm_mode, factored_norm, tiny_wl, small_wl):
    if name.startswith("small_seed_"):       # other draws of graph, features, weights and sampling keys
        w = configs.small(seed=int(name.rsplit("_", 1)[1]))
    else:
        w = tiny_wl if name == "tiny" else small_wl
    ref = oracle.train(w, epochs=1, keep_first=True)
    env, parts, model = _make(w, gemm_mode=gemm_mode, factored_norm=factored_norm)
    _check_structure(parts, ref["part"], ref["parts"])
    recs, _, _ = ref["first"]
    L = len(w.w0)
    ws0 = [a.astype(np.float64) for a in w.w0]
    bs0 = [b.astype(np.float64) for b in w.b0]
    gw = [np.zeros_like(a) for a in ws0]
    gb = [np.zeros_like(b) for b in bs0]
    losses = torch.zeros(w.m, device="cuda")
    for p, pt in enumerate(ref["parts"]):
        model.forward(p, losses[p:p + 1].data_ptr())
        fw, _ = recs[p]
        h_gpu = [model.get(gcnsa.GET_ACT, l, rows=pt.n) for l in range(1, L + 1)]
        for l in range(1, L + 1):
            _close(h_gpu[l - 1], fw["H"][l], what=f"p{p} H{l}")
        bw = oracle.backward(pt, fw, ws0, w.y[pt.members], relu_on=_relu_decisions(fw, h_gpu[:-1]))
        _close(model.get(gcnsa.GET_DLOGITS, rows=pt.n), bw["G"][L - 1], what=f"p{p} dlogits")
        model.backward(p)
        for l in range(L):
            gw[l] += bw["dW"][l]; gb[l] += bw["db"][l]
    assert np.allclose(losses.cpu().numpy(), [r[0]["loss"] for r in recs], rtol=1e-5)
    for l in range(L):  # the gradient sum before the step
        _close(model.get(gcnsa.GET_GRAD_W, l), gw[l], what=f"dW{l}")
        _close(model.get(gcnsa.GET_GRAD_B, l), gb[l], what=f"db{l}")
    g_own = [model.get(gcnsa.GET_GRAD_W, l).astype(np.float64) for l in range(L)] + \
            [model.get(gcnsa.GET_GRAD_B, l).astype(np.float64) for l in range(L)]
    model.step()
    assert model.t == 1 and gcnsa.tc_status() == 0
    # Adam's first step moves every entry by about lr * sign(g): an entry whose gradient is below fp32
    # resolution has no determined sign.  Entries with |g| >= 1e-3 max|g| are compared with the checker's step
    # on the checker's gradient; every entry is compared with the checker's step on the kernel's own gradient.
    opt = oracle.Adam(ws0 + bs0, w.lr, w.beta1, w.beta2, w.eps)
    new = opt.step(ws0 + bs0, [g / w.m for g in gw + gb])
    own = oracle.Adam(ws0 + bs0, w.lr, w.beta1, w.beta2, w.eps).step(ws0 + bs0, [g / w.m for g in g_own])
    got = [model.get(gcnsa.GET_W, l) for l in range(L)] + [model.get(gcnsa.GET_B, l) for l in range(L)]
    for i, (a, ref, mine, g) in enumerate(zip(got, new, own, gw + gb)):
        scale = max(np.abs(ref).max(), w.lr)
        assert np.abs(a - mine).max() <= 1e-5 * scale, f"param {i}: Adam kernel on its own gradient"
        firm = np.abs(g) >= 1e-3 * np.abs(g).max()
        assert firm.mean() >= 0.9
        assert np.abs(a - ref)[firm].max() <= TOL * scale, f"param {i} after one step"
    for l in range(L):
        assert np.all(model.get(gcnsa.GET_GRAD_W, l) == 0)
        _close(model.get(gcnsa.GET_ADAM_M_W, l), opt.m[l], what=f"adam m W{l}")
        _close(model.get(gcnsa.GET_ADAM_V_W, l), opt.v[l], what=f"adam v W{l}")
    model.close(); parts.close()


@pytest.mark.parametrize("factored_norm", [0, 1])
@pytest.mark.parametrize("gemm_mode", [gcnsa.GEMM_FP32, gcnsa.GEMM_TF32X3])
@pytest.mark.parametrize("name,epochs", [("tiny", 10), ("small", 50)])
def test_loss_curve_matches_checker(name, epochs, gemm_mode, factored_norm, tiny_wl, small_wl):
    w = tiny_wl if name == "tiny" else small_wl
    ref = oracle.train(w, epochs=epochs)
    env, parts, model = _make(w, gemm_mode=gemm_mode, factored_norm=factored_norm)
    loss = torch.zeros(1, device="cuda")
    got = []
    for _ in range(epochs):
        model.epoch(loss.data_ptr())
        got.append(loss.item())
    got, want = np.array(got), np.array(ref["losses"])
    assert np.abs(got - want).max() <= 1e-3 * np.abs(want).max(), (got, want)
    assert np.all(np.abs(got - want) <= 1e-3 * np.abs(want) + 1e-6)
    model.close(); parts.close()


def test_three_layers_with_a_widening_layer_and_options():
    """Deeper variant: 100 -> 256 -> 256 -> 47 runs the first layer as
    (A_hat H) W and the others as A_hat (H W); also without bias, with the
    loss restricted to owned vertices, and with the normalization factored out
    of the sparse products."""
    w = configs.large_sparse(scale=0.004)
    for use_bias, loh, mode, fact in ((1, 1, gcnsa.GEMM_FP32, 0), (0, 0, gcnsa.GEMM_TF32X3, 1), (1, 1, gcnsa.GEMM_TF32X3, 1)):
        w.loss_on_halo = loh
        if not use_bias:
            w.b0 = [np.zeros_like(b) for b in w.b0]
        env, parts, model = _make(w, use_bias=use_bias, loss_on_halo=loh, gemm_mode=mode, factored_norm=fact)
        part, rparts = oracle.build_partitions(w.rowptr, w.col, w.m, w.overlap_ppm, w.seed, w.part_mode, w.user_part)
        _check_structure(parts, part, rparts)
        ws = [a.astype(np.float64) for a in w.w0]
        bs = [b.astype(np.float64) for b in w.b0]
        gw = [np.zeros_like(a) for a in ws]
        gb = [np.zeros_like(b) for b in bs]
        for p, pt in enumerate(rparts):
            fw = oracle.forward(pt, w.x[pt.members], ws, bs if use_bias else None, w.y[pt.members],
                                w.train_mask[pt.members], loh)
            model.forward(p)
            h_gpu = [model.get(gcnsa.GET_ACT, l, rows=pt.n) for l in range(1, 4)]
            for l in range(1, 4):
                _close(h_gpu[l - 1], fw["H"][l], what=f"p{p} H{l}")
            bw = oracle.backward(pt, fw, ws, w.y[pt.members], relu_on=_relu_decisions(fw, h_gpu[:-1]))
            model.backward(p)
            for l in range(3):
                gw[l] += bw["dW"][l]; gb[l] += bw["db"][l]
        for l in range(3):
            _close(model.get(gcnsa.GET_GRAD_W, l), gw[l], what=f"dW{l}")
            if use_bias:
                _close(model.get(gcnsa.GET_GRAD_B, l), gb[l], what=f"db{l}")
            else:
                assert np.all(model.get(gcnsa.GET_GRAD_B, l) == 0)
        model.close(); parts.close()


def test_runs_are_bitwise_reproducible(small_wl):
    outs = []
    for _ in range(2):
        env, parts, model = _make(small_wl)
        for _ in range(3):
            model.epoch()
        outs.append([model.get(gcnsa.GET_W, l) for l in range(2)])
        model.close(); parts.close()
    for a, b in zip(*outs):
        assert np.array_equal(a, b)


def test_call_order_errors_and_checkpoint(tiny_wl):
    w = tiny_wl
    env, parts, model = _make(w)
    with pytest.raises(gcnsa.GcnsaError) as ei:
        model.backward(0)                      # no forward yet
    assert ei.value.code == gcnsa.ERR_ORDER
    with pytest.raises(gcnsa.GcnsaError) as ei:
        model.step()                           # nothing accumulated
    assert ei.value.code == gcnsa.ERR_ORDER
    model.forward(0)
    with pytest.raises(gcnsa.GcnsaError) as ei:
        model.backward(1)                      # forward was on another partition
    assert ei.value.code == gcnsa.ERR_ORDER
    with pytest.raises(gcnsa.GcnsaError) as ei:
        model.forward(5)
    assert ei.value.code == gcnsa.ERR_ARG
    model.backward(0)
    with pytest.raises(gcnsa.GcnsaError):
        model.step()                           # only one of two partitions
    model.forward(1); model.backward(1); model.step()
    # checkpoint: 2 epochs, save, 2 more  ==  restore into a fresh model, 2 more
    model.epoch()
    state = {(what, l): model.get(what, l) for what in range(8) for l in range(2)}
    t = model.t
    model.epoch(); model.epoch()
    want = [model.get(gcnsa.GET_W, l) for l in range(2)]
    env2, parts2, model2 = _make(w)
    for (what, l), v in state.items():
        model2.set(what, l, v)
    model2.t = t
    model2.epoch(); model2.epoch()
    for l in range(2):
        assert np.array_equal(model2.get(gcnsa.GET_W, l), want[l])
    for m_, p_ in ((model, parts), (model2, parts2)):
        m_.close(); p_.close()


def test_epoch_from_host_buffers_matches_resident_epoch(small_wl):
    w = small_wl
    env, parts, model = _make(w)
    env2, parts2, model2 = _make(w)
    xs = [torch.from_numpy(np.ascontiguousarray(w.x[parts.members(p)])).pin_memory() for p in range(w.m)]
    loss_h = np.zeros(1, np.float32)
    loss_d = torch.zeros(1, device="cuda")
    for _ in range(3):
        model.epoch_host([x.data_ptr() for x in xs], loss_h)
        model2.epoch(loss_d.data_ptr())
        assert loss_h[0] == loss_d.item()
    for l in range(2):
        assert np.array_equal(model.get(gcnsa.GET_W, l), model2.get(gcnsa.GET_W, l))
    for m_, p_ in ((model, parts), (model2, parts2)):
        m_.close(); p_.close()


def test_single_partition_and_zero_overlap(tiny_wl):
    """M = 1 (no sampling at all) and O = 0 (isolated partitions) are the
    method's degenerate cases."""
    import copy
    for m, o_ppm, mode in ((1, 100_000, configs.PART_RANGE), (3, 0, configs.PART_HASH)):
        w = copy.copy(tiny_wl)
        w.m, w.overlap_ppm, w.part_mode, w.user_part, w.epochs = m, o_ppm, mode, None, 2
        ref = oracle.train(w)
        env, parts, model = _make(w)
        assert all(parts.info(p).n_halo == 0 for p in range(m))
        loss = torch.zeros(1, device="cuda")
        for e in range(2):
            model.epoch(loss.data_ptr())
            assert abs(loss.item() - ref["losses"][e]) <= 1e-3 * ref["losses"][e]
        for l in range(2):
            _close(model.get(gcnsa.GET_W, l), ref["ws"][l], tol=2e-4, what=f"W{l}")
        model.close(); parts.close()


def test_profile_counters(small_wl):
    env, parts, model = _make(small_wl)
    model.profile(True)
    before = gcnsa.launch_count()
    model.epoch()
    pr = model.profile_read()
    assert pr["spmm"]["launches"] == 4 * small_wl.m and pr["spmm"]["ms"] > 0
    assert pr["gemm"]["launches"] >= 5 * small_wl.m
    assert sum(v["launches"] for v in pr.values()) == gcnsa.launch_count() - before
    nnz = sum(parts.info(p).nnz for p in range(small_wl.m))
    # the last layer's transposed product skips the columns that carry no loss, hence "<="
    assert 2.0 * nnz * (64 + 64 + 20) < pr["spmm"]["flops"] <= 2.0 * nnz * (64 + 64 + 20 + 20)
    model.close(); parts.close()


@pytest.mark.parametrize("name,epochs", [("tiny", 10), ("small", 20)])
def test_parameter_averaging_mode_matches_checker(name, epochs, tiny_wl, small_wl):
    """Section 3.2 as written: every partition takes its own Adam step (own
    moments) from the aggregated parameters; the parameters are averaged."""
    w = tiny_wl if name == "tiny" else small_wl
    env = gcnsa.make_env(0)
    parts = gcnsa.Parts(env, w.rowptr, w.col, w.x, w.y, w.train_mask, w.dims[-1], w.m, w.overlap_ppm, w.seed,
                        w.part_mode, w.user_part, w.loss_on_halo)
    model = gcnsa.Model(env, parts, w.dims, w.w0, w.b0, lr=w.lr, beta1=w.beta1, beta2=w.beta2, eps=w.eps,
                        gemm_mode=gcnsa.GEMM_TF32X3, agg_mode=gcnsa.AGG_PARAM_AVG, factored_norm=1, loss_rows_only=0,
                        epoch_graph=0)
    _, rparts = oracle.build_partitions(w.rowptr, w.col, w.m, w.overlap_ppm, w.seed, w.part_mode, w.user_part)
    xs = [w.x[pt.members].astype(np.float64) for pt in rparts]
    ys = [w.y[pt.members] for pt in rparts]
    mks = [w.train_mask[pt.members] for pt in rparts]
    ws = [a.astype(np.float64) for a in w.w0]
    bs = [b.astype(np.float64) for b in w.b0]
    opts = [oracle.Adam(ws + bs, w.lr, w.beta1, w.beta2, w.eps) for _ in rparts]
    loss = torch.zeros(1, device="cuda")
    L = len(ws)
    for e in range(epochs):
        ws, bs, want = oracle.epoch_param_avg(rparts, xs, ys, mks, ws, bs, opts, w.loss_on_halo)
        model.epoch(loss.data_ptr())
        assert abs(loss.item() - want) <= 1e-3 * abs(want), (e, loss.item(), want)
        if e == 0:
            # the first step moves each entry by about lr * sign(g_p) per partition: compare where every
            # partition's gradient sign is determined, i.e. away from |first moment| ~ 0
            for l in range(L):
                got = model.get(gcnsa.GET_W, l)
                firm = np.ones(got.shape, bool)
                for o in opts:
                    firm &= np.abs(o.m[l]) >= 1e-3 * np.abs(o.m[l]).max()
                assert firm.mean() > 0.9
                assert np.abs(got - ws[l])[firm].max() <= 1e-4 * np.abs(ws[l]).max()
            for p, o in enumerate(opts):      # every partition keeps its own moments
                model.select_partition(p)
                for l in range(L):
                    _close(model.get(gcnsa.GET_ADAM_M_W, l), o.m[l], what=f"m p{p} W{l}")
                    _close(model.get(gcnsa.GET_ADAM_V_W, l), o.v[l], what=f"v p{p} W{l}")
    assert model.t == epochs and gcnsa.tc_status() == 0
    for l in range(L):
        _close(model.get(gcnsa.GET_W, l), ws[l], tol=2e-3, what=f"W{l} after {epochs} epochs")
    model.close(); parts.close()


def test_full_graph_evaluation_matches_checker(small_wl):
    """Micro-F1 on the complete graph (Section 2.2): train on the extended
    partitions, copy the parameters into a model built on the un-partitioned
    graph, predict, count.  Predictions are compared with the checker's argmax
    on the same parameters; rows whose two best logits are closer than fp32
    resolution may go either way."""
    w = small_wl
    env, parts, model = _make(w, gemm_mode=gcnsa.GEMM_TF32X3)
    for _ in range(15):
        model.epoch()
    full = gcnsa.Parts(env, w.rowptr, w.col, w.x, w.y, w.train_mask, w.dims[-1], 1, 0, w.seed, gcnsa.PART_RANGE)
    # the evaluating model uses the options bench.py trains with: evaluation still has to compute every row
    ev = gcnsa.Model(env, full, w.dims, w.w0, w.b0, **gcnsa.MEASURED)
    ev.copy_params_from(model)
    test_mask = (1 - w.train_mask).astype(np.uint8)
    correct, total, pred = ev.evaluate(full, 0, test_mask)
    ws = [model.get(gcnsa.GET_W, l).astype(np.float64) for l in range(2)]
    bs = [model.get(gcnsa.GET_B, l).astype(np.float64) for l in range(2)]
    _, (pt,) = oracle.build_partitions(w.rowptr, w.col, 1, 0, w.seed)
    want_pred, logits = oracle.predict(pt, w.x.astype(np.float64), ws, bs)
    top2 = np.sort(logits, axis=1)[:, -2:]
    firm = (top2[:, 1] - top2[:, 0]) > 1e-4 * np.abs(logits).max()
    assert firm.mean() > 0.99
    assert np.array_equal(pred[firm], want_pred[firm])
    f1, tp, fp, fn = oracle.micro_f1(want_pred, w.y, test_mask, w.dims[-1])
    assert total == int(test_mask.sum()) == tp + fn
    assert abs(correct - tp) <= int((~firm & test_mask.astype(bool)).sum())
    assert correct / total > 0.8          # the synthetic classes are learnable: training worked
    # no mask = every vertex; evaluation leaves the training state alone
    c_all, t_all, _ = ev.evaluate(full, 0)
    assert t_all == w.n and c_all >= correct
    with pytest.raises(gcnsa.GcnsaError):   # a model built for smaller partitions cannot take the full graph
        model.evaluate(full, 0)
    model.epoch()
    for m_, p_ in ((ev, full), (model, parts)):
        m_.close(); p_.close()


def test_loss_rows_only_gives_the_same_training(small_wl):
    """With loss_rows_only the last layer is computed on the rows that carry
    loss only; training (losses, parameters) must be bit-identical, and an
    evaluation in between still sees every row."""
    w = small_wl
    env = gcnsa.make_env(0)
    parts = gcnsa.Parts(env, w.rowptr, w.col, w.x, w.y, w.train_mask, w.dims[-1], w.m, w.overlap_ppm, w.seed,
                        w.part_mode, w.user_part, w.loss_on_halo)
    models = [gcnsa.Model(env, parts, w.dims, w.w0, w.b0, lr=w.lr, gemm_mode=gcnsa.GEMM_TF32X3, loss_rows_only=k,
                          factored_norm=0, epoch_graph=0) for k in (0, 1)]
    loss = torch.zeros(2, device="cuda")
    for e in range(5):
        for k, m_ in enumerate(models):
            m_.epoch(loss[k:k + 1].data_ptr())
        assert loss[0].item() == loss[1].item()
        if e == 2:
            a = models[0].evaluate(parts, 1)
            b = models[1].evaluate(parts, 1)
            assert a[0] == b[0] and np.array_equal(a[2], b[2])
    for l in range(2):
        assert np.array_equal(models[0].get(gcnsa.GET_W, l), models[1].get(gcnsa.GET_W, l))
    for m_ in models:
        m_.close()
    parts.close()


@pytest.mark.parametrize("agg_mode", [gcnsa.AGG_GRAD_AVG, gcnsa.AGG_PARAM_AVG])
def test_recorded_epoch_equals_plain_launches(small_wl, agg_mode):
    """epoch_graph replays one recorded epoch: losses, parameters, step count
    and the launch counter must be those of plain launches, also after the
    step count is set by hand, while profiling, and with another loss pointer."""
    w = small_wl
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        env = gcnsa.make_env(0)
        assert env.stream          # a stream of its own, not the legacy default stream (NULL)
        parts = gcnsa.Parts(env, w.rowptr, w.col, w.x, w.y, w.train_mask, w.dims[-1], w.m, w.overlap_ppm, w.seed,
                            w.part_mode, w.user_part, w.loss_on_halo)
        models = [gcnsa.Model(env, parts, w.dims, w.w0, w.b0, lr=w.lr, gemm_mode=gcnsa.GEMM_TF32X3, agg_mode=agg_mode,
                              loss_rows_only=1, factored_norm=0, epoch_graph=k) for k in (0, 1)]
        loss = torch.zeros(3, device="cuda")
        counts = [0, 0]
        for e in range(8):
            if e == 3:
                for m_ in models:
                    m_.t = 40            # as after restoring a checkpoint
            if e == 5:
                models[1].profile(True)  # profiling suspends the replay
            if e == 6:
                models[1].profile(False)
            for k, m_ in enumerate(models):
                before = gcnsa.launch_count()
                m_.epoch(loss[2 if (k == 1 and e == 7) else k:].data_ptr())
                counts[k] = gcnsa.launch_count() - before
            stream.synchronize()
            got = loss[2].item() if e == 7 else loss[1].item()
            assert loss[0].item() == got, e
            assert counts[0] == counts[1] > 0
            assert models[0].t == models[1].t
        for what in (gcnsa.GET_W, gcnsa.GET_B):
            for l in range(2):
                assert np.array_equal(models[0].get(what, l), models[1].get(what, l))
        assert gcnsa.tc_status() == 0
        for m_ in models:
            m_.close()
        parts.close()


def test_recorded_epoch_on_the_default_stream_falls_back(tiny_wl):
    """The legacy default stream cannot be recorded: epoch_graph then runs
    plain launches with the same results."""
    w = tiny_wl
    env = gcnsa.make_env(0)
    if env.stream:
        pytest.skip("torch's current stream is not the default stream")
    parts = gcnsa.Parts(env, w.rowptr, w.col, w.x, w.y, w.train_mask, w.dims[-1], w.m, w.overlap_ppm, w.seed,
                        w.part_mode, w.user_part, w.loss_on_halo)
    models = [gcnsa.Model(env, parts, w.dims, w.w0, w.b0, lr=w.lr, **{**gcnsa.PLAIN, "epoch_graph": k}) for k in (0, 1)]
    for _ in range(3):
        for m_ in models:
            m_.epoch()
    for l in range(2):
        assert np.array_equal(models[0].get(gcnsa.GET_W, l), models[1].get(gcnsa.GET_W, l))
    for m_ in models:
        m_.close()
    parts.close()


@pytest.mark.parametrize("epoch_graph", [0, 1])
def test_cached_aggregated_features_give_the_same_training(epoch_graph, small_wl):
    """cache_ax keeps A_hat X of every partition and runs layer 1 as (A_hat X) W (Section 4.1: the same
    H^1 = sigma(A_hat X W^1), multiplied in the other order): gradients and loss curve match the checker, and a
    partition whose feature rows are rewritten gets its product recomputed."""
    w = small_wl
    epochs = 12
    ref = oracle.train(w, epochs=epochs, keep_first=True)
    stream = torch.cuda.Stream() if epoch_graph else torch.cuda.current_stream()
    with torch.cuda.stream(stream):
        env = gcnsa.make_env(0)
        parts = gcnsa.Parts(env, w.rowptr, w.col, w.x, w.y, w.train_mask, w.dims[-1], w.m, w.overlap_ppm, w.seed,
                            w.part_mode, w.user_part, w.loss_on_halo)
        kw = dict(lr=w.lr, beta1=w.beta1, beta2=w.beta2, eps=w.eps, gemm_mode=gcnsa.GEMM_TF32X3, loss_rows_only=1,
                  factored_norm=1, epoch_graph=epoch_graph)
        cached = gcnsa.Model(env, parts, w.dims, w.w0, w.b0, cache_ax=1, **kw)
        # gradient sum of the first epoch against the checker's
        recs, _, _ = ref["first"]
        L = len(w.w0)
        ws0 = [a.astype(np.float64) for a in w.w0]
        gw = [np.zeros_like(a) for a in ws0]
        for p, pt in enumerate(ref["parts"]):
            cached.forward(p)
            fw, _ = recs[p]
            h1 = cached.get(gcnsa.GET_ACT, 1, rows=pt.n)
            _close(h1, fw["H"][1], what=f"p{p} H1 from the cached product")
            bw = oracle.backward(pt, fw, ws0, w.y[pt.members], relu_on=_relu_decisions(fw, [h1]))
            cached.backward(p)
            for l in range(L):
                gw[l] += bw["dW"][l]
        for l in range(L):
            _close(cached.get(gcnsa.GET_GRAD_W, l), gw[l], what=f"dW{l}")
        cached.step()
        # loss curve of the following epochs (the first one is spent above)
        loss = torch.zeros(1, device="cuda")
        for e in range(1, epochs):
            cached.epoch(loss.data_ptr())
            assert abs(loss.item() - ref["losses"][e]) <= 1e-3 * abs(ref["losses"][e]), (e, loss.item(), ref["losses"][e])
        # rewrite one partition's feature rows: the cached product must follow
        plain = gcnsa.Model(env, parts, w.dims, w.w0, w.b0, **kw)
        for l in range(L):
            for what in (gcnsa.GET_W, gcnsa.GET_B):
                plain.set(what, l, cached.get(what, l))
        newx = np.ascontiguousarray(w.x[parts.members(1)] * np.float32(0.5))
        parts.set_features(1, newx.ctypes.data)
        la, lb = torch.zeros(1, device="cuda"), torch.zeros(1, device="cuda")
        cached.forward(1, la.data_ptr()); plain.forward(1, lb.data_ptr())
        _close(cached.get(gcnsa.GET_ACT, 1, rows=parts.info(1).n), plain.get(gcnsa.GET_ACT, 1, rows=parts.info(1).n),
               what="H1 after the feature rows changed")
        assert abs(la.item() - lb.item()) <= 1e-5 * abs(lb.item())
        cached.close(); plain.close(); parts.close()
