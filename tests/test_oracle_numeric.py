"""Pins for the checker's dense steps: forward, loss, backward, Adam, epoch.
Each is compared with something that shares nothing with it: a dense
restatement, central finite differences, torch CPU autograd on a dense
normalized adjacency, torch.optim.Adam, closed forms."""
import numpy as np
import pytest
import torch

from gen import graphs
from oracle import oracle


def _setup(n=50, prob=0.12, m=2, o_ppm=400_000, dims=(7, 6, 5, 4), seed=3, p=0):
    rng = np.random.default_rng(seed)
    rowptr, col = graphs.erdos_renyi(n, prob, seed)
    _, parts = oracle.build_partitions(rowptr, col, m, o_ppm, seed=seed)
    pt = parts[p]
    x = rng.standard_normal((n, dims[0]))[pt.members]
    y = rng.integers(0, dims[-1], size=n)[pt.members]
    mask = (rng.random(n) < 0.6).astype(np.uint8)[pt.members]
    ws = [rng.standard_normal((a, b)) * 0.4 for a, b in zip(dims[:-1], dims[1:])]
    bs = [rng.standard_normal(b) * 0.1 for b in dims[1:]]
    return pt, x, y, mask, ws, bs


def _dense(pt):
    a = np.zeros((pt.n, pt.n))
    a[np.repeat(np.arange(pt.n), np.diff(pt.rowptr)), pt.col] = pt.val
    return a


def _loss_dense(a, x, ws, bs, y, t):
    h = x
    for l, (w, b) in enumerate(zip(ws, bs)):
        z = a @ h @ w + b
        h = np.maximum(z, 0) if l < len(ws) - 1 else z
    if t.sum() == 0:
        return 0.0
    p = np.exp(h - h.max(1, keepdims=True))
    p /= p.sum(1, keepdims=True)
    return float(-(np.log(p[np.arange(len(y)), y]) * t).sum() / t.sum())


@pytest.mark.parametrize("loss_on_halo", [1, 0])
def test_forward_against_dense(loss_on_halo):
    pt, x, y, mask, ws, bs = _setup()
    assert pt.n > pt.n_owned
    fw = oracle.forward(pt, x, ws, bs, y, mask, loss_on_halo)
    a = _dense(pt)
    h = x
    for l in range(3):
        z = a @ h @ ws[l] + bs[l]
        assert np.allclose(fw["Z"][l], z, atol=1e-12)
        h = np.maximum(z, 0) if l < 2 else z
        assert np.allclose(fw["H"][l + 1], h, atol=1e-12)
    t = mask.astype(bool).copy()
    if not loss_on_halo:
        t[pt.n_owned:] = False
    assert abs(fw["loss"] - _loss_dense(a, x, ws, bs, y, t)) < 1e-12
    if not loss_on_halo:
        assert fw["nt"] == int(mask[:pt.n_owned].sum())


def test_identity_adjacency_reduces_to_a_plain_mlp():
    # a graph with no edges: A_hat = I, so the network is an MLP on the rows
    rowptr, col = graphs.from_edge_list(9, [])
    _, parts = oracle.build_partitions(rowptr, col, 1, 0, seed=0)
    rng = np.random.default_rng(0)
    x, w1, w2 = rng.standard_normal((9, 4)), rng.standard_normal((4, 3)), rng.standard_normal((3, 2))
    fw = oracle.forward(parts[0], x, [w1, w2], [np.zeros(3), np.zeros(2)], np.zeros(9, int), np.ones(9, np.uint8))
    assert np.allclose(fw["Z"][1], np.maximum(x @ w1, 0) @ w2, atol=1e-13)


def test_backward_against_finite_differences():
    pt, x, y, mask, ws, bs = _setup()
    fw = oracle.forward(pt, x, ws, bs, y, mask)
    bw = oracle.backward(pt, fw, ws, y)
    a, t = _dense(pt), mask.astype(bool)
    h = 1e-6
    for l in range(3):
        for arr, grad in ((ws[l], bw["dW"][l]), (bs[l], bw["db"][l])):
            num = np.zeros_like(arr)
            it = np.nditer(arr, flags=["multi_index"])
            for _ in it:
                i = it.multi_index
                old = arr[i]
                arr[i] = old + h
                lp = _loss_dense(a, x, ws, bs, y, t)
                arr[i] = old - h
                lm = _loss_dense(a, x, ws, bs, y, t)
                arr[i] = old
                num[i] = (lp - lm) / (2 * h)
            assert np.abs(num - grad).max() <= 1e-6 * max(np.abs(num).max(), 1e-3)


@pytest.mark.parametrize("loss_on_halo", [1, 0])
def test_backward_against_torch_autograd(loss_on_halo):
    pt, x, y, mask, ws, bs = _setup(n=70, dims=(9, 8, 6), seed=8, m=3, p=1)
    fw = oracle.forward(pt, x, ws, bs, y, mask, loss_on_halo)
    bw = oracle.backward(pt, fw, ws, y)
    a = torch.tensor(_dense(pt))
    tw = [torch.tensor(w, requires_grad=True) for w in ws]
    tb = [torch.tensor(b, requires_grad=True) for b in bs]
    h = torch.tensor(x)
    for l in range(len(ws)):
        h = a @ h @ tw[l] + tb[l]
        if l < len(ws) - 1:
            h = torch.relu(h)
    t = torch.tensor(mask.astype(bool))
    if not loss_on_halo:
        t[pt.n_owned:] = False
    loss = torch.nn.functional.cross_entropy(h[t], torch.tensor(y, dtype=torch.long)[t], reduction="mean")
    loss.backward()
    assert abs(float(loss.detach()) - fw["loss"]) < 1e-12
    for l in range(len(ws)):
        assert np.allclose(bw["dW"][l], tw[l].grad.numpy(), atol=1e-12)
        assert np.allclose(bw["db"][l], tb[l].grad.numpy(), atol=1e-12)


def test_empty_training_set_gives_zero_loss_and_gradients():
    pt, x, y, mask, ws, bs = _setup()
    fw = oracle.forward(pt, x, ws, bs, y, np.zeros_like(mask))
    bw = oracle.backward(pt, fw, ws, y)
    assert fw["loss"] == 0.0
    assert all(np.all(g == 0) for g in bw["dW"] + bw["db"])


def test_adam_first_step_closed_form_and_torch():
    rng = np.random.default_rng(1)
    p0 = [rng.standard_normal((4, 3)), rng.standard_normal(3)]
    opt = oracle.Adam(p0, lr=0.02)
    g = [rng.standard_normal((4, 3)), rng.standard_normal(3)]
    p1 = opt.step(p0, g)
    # t = 1: m_hat = g, v_hat = g^2, so the move is -lr g / (|g| + eps)
    for a, b, gg in zip(p0, p1, g):
        assert np.allclose(b - a, -0.02 * gg / (np.abs(gg) + 1e-8), atol=1e-15)
    # several steps against torch.optim.Adam in fp64
    tp = [torch.tensor(a.copy(), requires_grad=True) for a in p0]
    topt = torch.optim.Adam(tp, lr=0.02, betas=(0.9, 0.999), eps=1e-8)
    cur = p0
    opt = oracle.Adam(p0, lr=0.02)
    for step in range(5):
        g = [rng.standard_normal((4, 3)), rng.standard_normal(3)]
        cur = opt.step(cur, g)
        for t_, gg in zip(tp, g):
            t_.grad = torch.tensor(gg)
        topt.step()
        for a, t_ in zip(cur, tp):
            assert np.allclose(a, t_.detach().numpy(), atol=1e-13)


def test_epoch_average_of_identical_partitions_and_full_coverage():
    """M = 2 with saturated overlap on a connected graph: both augmented
    partitions are the whole graph (relabelled), so one epoch equals one
    full-batch step on the single graph."""
    n = 24
    rowptr, col = graphs.from_edge_list(n, [(i, (i + 1) % n) for i in range(n)] + [(0, 12), (3, 17), (5, 20)])
    rng = np.random.default_rng(2)
    x = rng.standard_normal((n, 5)); y = rng.integers(0, 3, n); mask = np.ones(n, np.uint8)
    ws = [rng.standard_normal((5, 4)) * 0.5, rng.standard_normal((4, 3)) * 0.5]
    bs = [np.zeros(4), np.zeros(3)]
    _, two = oracle.build_partitions(rowptr, col, 2, 1_000_000, seed=1)
    _, one = oracle.build_partitions(rowptr, col, 1, 0, seed=1)
    assert all(pt.n == n for pt in two)

    def run(parts):
        opt = oracle.Adam(ws + bs, 0.02)
        return oracle.epoch(parts, [x[pt.members] for pt in parts], [y[pt.members] for pt in parts],
                            [mask[pt.members] for pt in parts], ws, bs, opt)

    w2, b2, l2, _ = run(two)
    w1, b1, l1, _ = run(one)
    assert abs(l1 - l2) < 1e-12
    for a, b in zip(w1 + b1, w2 + b2):
        assert np.allclose(a, b, atol=1e-12)


def test_training_reduces_the_loss(tiny_wl):
    r = oracle.train(tiny_wl)
    assert len(r["losses"]) == 10
    assert r["losses"][0] > np.log(5) * 0.8 and r["losses"][-1] < 0.6 * r["losses"][0]
    assert all(b < a for a, b in zip(r["losses"], r["losses"][1:]))


def test_parameter_averaging_epoch_against_torch_and_special_cases():
    """Section 3.2 as written: per-worker Adam step from the aggregated
    parameters, then the mean of the workers' parameters.  Checked against
    torch.optim.Adam per worker on dense matrices, and against the cases where
    it must coincide with the gradient-averaging epoch."""
    n = 40
    rowptr, col = graphs.erdos_renyi(n, 0.15, 21)
    rng = np.random.default_rng(4)
    x = rng.standard_normal((n, 6)); y = rng.integers(0, 3, n); mask = (rng.random(n) < 0.7).astype(np.uint8)
    ws = [rng.standard_normal((6, 5)) * 0.4, rng.standard_normal((5, 3)) * 0.4]
    bs = [rng.standard_normal(5) * 0.1, rng.standard_normal(3) * 0.1]
    _, parts = oracle.build_partitions(rowptr, col, 3, 500_000, seed=2)
    xs = [x[pt.members] for pt in parts]; ys = [y[pt.members] for pt in parts]; mks = [mask[pt.members] for pt in parts]
    opts = [oracle.Adam(ws + bs, 0.02) for _ in parts]
    # torch: one model copy and one Adam per worker, two epochs
    tw = [[torch.tensor(a.copy(), requires_grad=True) for a in ws + bs] for _ in parts]
    topt = [torch.optim.Adam(t, lr=0.02) for t in tw]
    cur_w, cur_b = ws, bs
    for epoch in range(2):
        cur_w, cur_b, loss = oracle.epoch_param_avg(parts, xs, ys, mks, cur_w, cur_b, opts)
        for pt, t, o, xx, yy, mm in zip(parts, tw, topt, xs, ys, mks):
            a = torch.tensor(_dense(pt))
            h = torch.relu(a @ torch.tensor(xx) @ t[0] + t[2])
            z = a @ h @ t[1] + t[3]
            sel = torch.tensor(mm.astype(bool))
            o.zero_grad()
            torch.nn.functional.cross_entropy(z[sel], torch.tensor(yy, dtype=torch.long)[sel]).backward()
            o.step()
        with torch.no_grad():
            mean = [sum(t[i] for t in tw) / len(tw) for i in range(4)]
            for t in tw:
                for i in range(4):
                    t[i].copy_(mean[i])
        for got, want in zip(cur_w + cur_b, [mean[0], mean[1], mean[2], mean[3]]):
            assert np.allclose(got, want.numpy(), atol=1e-12)
    # one worker: parameter averaging == gradient averaging
    _, one = oracle.build_partitions(rowptr, col, 1, 0, seed=2)
    a_w, a_b, a_l = oracle.epoch_param_avg(one, [x], [y], [mask], ws, bs, [oracle.Adam(ws + bs, 0.02)])
    g_w, g_b, g_l, _ = oracle.epoch(one, [x], [y], [mask], ws, bs, oracle.Adam(ws + bs, 0.02))
    assert a_l == g_l and all(np.array_equal(p, q) for p, q in zip(a_w + a_b, g_w + g_b))
    # first epoch with Adam: each worker moves by about lr * sign(g_p), so the mean differs from one step on the
    # mean gradient wherever the workers' gradient signs disagree
    p_w, _, _ = oracle.epoch_param_avg(parts, xs, ys, mks, ws, bs, [oracle.Adam(ws + bs, 0.02) for _ in parts])
    q_w, _, _, _ = oracle.epoch(parts, xs, ys, mks, ws, bs, oracle.Adam(ws + bs, 0.02))
    assert not np.allclose(p_w[0], q_w[0], atol=1e-4)
    assert np.abs(p_w[0] - ws[0]).max() <= 0.02 + 1e-9


def test_micro_f1_hand_case_and_equals_accuracy():
    """Section 2.2 metric.  Hand case: y = [0,0,1,1,2], pred = [0,1,1,1,0] over
    all five: TP = 3 (positions 0,2,3), every miss is one FP and one FN (2
    each), precision = recall = 3/5 -> F1 = 0.6 = accuracy."""
    f1, tp, fp, fn = oracle.micro_f1([0, 1, 1, 1, 0], [0, 0, 1, 1, 2], [1, 1, 1, 1, 1], 3)
    assert (tp, fp, fn) == (3, 2, 2) and abs(f1 - 0.6) < 1e-15
    f1, tp, fp, fn = oracle.micro_f1([0, 1, 1, 1, 0], [0, 0, 1, 1, 2], [1, 0, 1, 0, 1], 3)   # masked subset
    assert (tp, fp, fn) == (2, 1, 1) and abs(f1 - 2 / 3) < 1e-15
    rng = np.random.default_rng(0)
    y, p, m = rng.integers(0, 7, 500), rng.integers(0, 7, 500), rng.random(500) < 0.4
    f1, *_ = oracle.micro_f1(p, y, m, 7)
    assert abs(f1 - np.mean(p[m] == y[m])) < 1e-15          # single-label: micro-F1 is the accuracy
    assert oracle.micro_f1([1, 1], [0, 0], [1, 1], 2)[0] == 0.0


def test_predict_is_argmax_of_dense_forward():
    pt, x, y, mask, ws, bs = _setup()
    pred, logits = oracle.predict(pt, x, ws, bs)
    a, h = _dense(pt), x
    for l in range(3):
        h = a @ h @ ws[l] + bs[l]
        if l < 2:
            h = np.maximum(h, 0)
    assert np.allclose(logits, h, atol=1e-12) and np.array_equal(pred, h.argmax(1))


# ---- backward(relu_on=...): the ReLU decision handed in from outside (ReLU'(0) reading: derivative 0 at z <= 0;
# a parity test hands in the fp32 path's decision for units whose |z| is below fp32 resolution) ----
def _loss_dense_forced(a, x, ws, bs, y, t, forced):
    """The dense loss with some hidden units' ReLU replaced by a fixed linear piece: forced[(l, i, j)] = True
    makes unit (i, j) of hidden layer l the identity, False makes it zero, whatever the sign of z."""
    h = x
    for l, (w, b) in enumerate(zip(ws, bs)):
        z = a @ h @ w + b
        if l < len(ws) - 1:
            h = np.maximum(z, 0)
            for (fl, i, j), on in forced.items():
                if fl == l:
                    h[i, j] = z[i, j] if on else 0.0
        else:
            h = z
    p = np.exp(h - h.max(1, keepdims=True))
    p /= p.sum(1, keepdims=True)
    return float(-(np.log(p[np.arange(len(y)), y]) * t).sum() / t.sum())


def test_backward_with_the_checkers_own_relu_decisions_is_bitwise_the_default():
    pt, x, y, mask, ws, bs = _setup()
    fw = oracle.forward(pt, x, ws, bs, y, mask)
    a = oracle.backward(pt, fw, ws, y)
    b = oracle.backward(pt, fw, ws, y, relu_on=[z > 0.0 for z in fw["Z"][:-1]])
    for k in ("dW", "db", "G"):
        for u, v in zip(a[k], b[k]):
            assert np.array_equal(u, v)


@pytest.mark.parametrize("which", ["off_in_layer_0", "on_in_layer_0", "off_in_layer_1", "on_in_layer_1", "both_layers"])
def test_backward_with_flipped_relu_decisions_against_finite_differences(which):
    """Flipping a unit's decision must give the gradient of the loss in which that unit's ReLU is the other linear
    piece.  Units are picked in both hidden layers of the three-layer case, so that a decision list applied to the
    wrong layer, transposed, or ignored shows up."""
    pt, x, y, mask, ws, bs = _setup()
    fw = oracle.forward(pt, x, ws, bs, y, mask)
    a, t = _dense(pt), mask.astype(bool)
    on = [z > 0.0 for z in fw["Z"][:-1]]
    forced = {}

    def pick(l, want_positive, nth=0):
        z = fw["Z"][l]
        rows = np.flatnonzero(t)                      # a unit in a row that carries loss, so that it matters
        cand = [(i, j) for i in rows for j in range(z.shape[1]) if (z[i, j] > 0.05) == want_positive and abs(z[i, j]) > 0.05]
        return cand[nth]

    if which in ("off_in_layer_0", "both_layers"):
        i, j = pick(0, True)
        forced[(0, i, j)] = False
    if which == "on_in_layer_0":
        i, j = pick(0, False)
        forced[(0, i, j)] = True
    if which == "off_in_layer_1":
        i, j = pick(1, True)
        forced[(1, i, j)] = False
    if which in ("on_in_layer_1", "both_layers"):
        i, j = pick(1, False, nth=1)
        forced[(1, i, j)] = True
    for (l, i, j), v in forced.items():
        assert on[l][i, j] != v                      # it is a flip
        on[l][i, j] = v
    bw = oracle.backward(pt, fw, ws, y, relu_on=on)
    plain = oracle.backward(pt, fw, ws, y)
    assert any(not np.allclose(p, q, rtol=1e-9, atol=0) for p, q in zip(plain["dW"], bw["dW"])), "the flip must matter"
    # the forward values feeding the backward pass are those of the forced function only if the forced units keep
    # their forward value; the oracle's backward takes fw as given, so compare with finite differences of the
    # forced loss around the same parameters, where the flipped units change the activations too
    fwf = _forward_forced(pt, x, ws, bs, y, mask, forced)
    bwf = oracle.backward(pt, fwf, ws, y, relu_on=on)
    h = 1e-6
    for l in range(3):
        for arr, grad in ((ws[l], bwf["dW"][l]), (bs[l], bwf["db"][l])):
            num = np.zeros_like(arr)
            it = np.nditer(arr, flags=["multi_index"])
            for _ in it:
                idx = it.multi_index
                old = arr[idx]
                arr[idx] = old + h
                lp = _loss_dense_forced(a, x, ws, bs, y, t, forced)
                arr[idx] = old - h
                lm = _loss_dense_forced(a, x, ws, bs, y, t, forced)
                arr[idx] = old
                num[idx] = (lp - lm) / (2 * h)
            assert np.abs(num - grad).max() <= 1e-6 * max(np.abs(num).max(), 1e-3), (which, l)


def _forward_forced(pt, x, ws, bs, y, mask, forced):
    """oracle.forward's record for the forced function: the same fields, with the forced units' activations set
    to their linear piece (dense restatement of the layers, the loss fields taken from the checker's formula)."""
    a = _dense(pt)
    h = x
    S, Z, H = [], [], [h]
    for l, (w, b) in enumerate(zip(ws, bs)):
        s = a @ h
        z = s @ w + b
        if l < len(ws) - 1:
            h = np.maximum(z, 0)
            for (fl, i, j), on in forced.items():
                if fl == l:
                    h[i, j] = z[i, j] if on else 0.0
        else:
            h = z
        S.append(s); Z.append(z); H.append(h)
    t = mask.astype(bool)
    zmax = Z[-1].max(axis=1, keepdims=True)
    lse = zmax[:, 0] + np.log(np.exp(Z[-1] - zmax).sum(axis=1))
    return {"S": S, "Z": Z, "H": H, "t": t, "nt": int(t.sum()), "lse": lse, "loss": None}


def test_backward_rejects_malformed_relu_decisions():
    pt, x, y, mask, ws, bs = _setup()
    fw = oracle.forward(pt, x, ws, bs, y, mask)
    good = [z > 0.0 for z in fw["Z"][:-1]]
    with pytest.raises(ValueError):
        oracle.backward(pt, fw, ws, y, relu_on=good[:1])                 # one array too few
    with pytest.raises(ValueError):
        oracle.backward(pt, fw, ws, y, relu_on=good + [good[0]])         # one too many
    with pytest.raises(ValueError):
        oracle.backward(pt, fw, ws, y, relu_on=[good[0].T, good[1]])     # transposed
    with pytest.raises(ValueError):
        oracle.backward(pt, fw, ws, y, relu_on=[good[0][:, :1], good[1]])  # would broadcast silently
    with pytest.raises(ValueError):
        oracle.backward(pt, fw, ws, y, relu_on=[good[0].astype(np.float64), good[1]])  # not boolean
