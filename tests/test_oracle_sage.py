"""Pins for the GraphSAGE checker (oracle/sage.py): the sampled sets against a
brute-force restatement, the layers against dense sampled operators, gradients
against finite differences and torch CPU autograd, the full-neighbourhood case
against the textbook mean aggregator, the batching against a sort, the epoch
against torch.optim.Adam per worker."""
import numpy as np
import pytest
import torch

from gen import graphs
from oracle import oracle, sage


def _case(n=60, prob=0.15, m=2, o_ppm=300_000, f=6, hidden=5, c=4, seed=5, p=0):
    rng = np.random.default_rng(seed)
    rowptr, col = graphs.erdos_renyi(n, prob, seed)
    _, parts = oracle.build_partitions(rowptr, col, m, o_ppm, seed=seed)
    pt = parts[p]
    x = rng.standard_normal((n, f))[pt.members]
    y = rng.integers(0, c, size=n)[pt.members]
    train = (rng.random(n) < 0.7)[pt.members]
    params = [rng.standard_normal((f, hidden)) * 0.4, rng.standard_normal((f, hidden)) * 0.4, rng.standard_normal(hidden) * 0.1,
              rng.standard_normal((hidden, c)) * 0.4, rng.standard_normal((hidden, c)) * 0.4, rng.standard_normal(c) * 0.1]
    return pt, x, y, train, params


def _neighbors(pt, v):
    row = pt.col[pt.rowptr[v]:pt.rowptr[v + 1]]
    return [int(u) for u in row if u != v]


def _brute_sample(pt, seed, epoch, layer, v, r):
    nb = _neighbors(pt, v)
    if len(nb) <= r:
        return sorted(nb)
    keyed = sorted(nb, key=lambda u: oracle.key(seed, 3, pt.p, epoch * 256 + layer, v, u))
    return sorted(keyed[:r])


@pytest.mark.parametrize("r", [0, 1, 3, 7, 100])
def test_sampled_sets_against_brute_force(r):
    pt, *_ = _case()
    vs = np.array(list(range(pt.n)) + [-1, 0, 0])
    for epoch, layer in ((0, 1), (0, 2), (3, 1)):
        ids, cnt = sage.sample_neighbors(pt, 99, epoch, layer, vs, r)
        for i, v in enumerate(vs):
            want = [] if v < 0 else _brute_sample(pt, 99, epoch, layer, int(v), r)
            assert cnt[i] == len(want) and list(ids[i, :cnt[i]]) == want and np.all(ids[i, cnt[i]:] == -1)
            assert v not in want
    # the draw depends on (seed, p, epoch, layer, v) only, and changes with each of them
    a, _ = sage.sample_neighbors(pt, 99, 0, 1, vs, 3)
    if r == 3:
        assert np.array_equal(a[-1], a[0]) and np.array_equal(a[-2], a[0])
        for other in (sage.sample_neighbors(pt, 98, 0, 1, vs, 3)[0], sage.sample_neighbors(pt, 99, 1, 1, vs, 3)[0],
                      sage.sample_neighbors(pt, 99, 0, 2, vs, 3)[0]):
            assert not np.array_equal(other, a)


def test_the_draw_is_uniform_over_the_neighbours():
    """Chi-square on how often each neighbour of one vertex is drawn over many epochs."""
    pt, *_ = _case(n=40, prob=0.5, m=1, o_ppm=0)
    v = int(np.argmax(np.diff(pt.rowptr)))
    nb = _neighbors(pt, v)
    assert len(nb) >= 12
    hits = {u: 0 for u in nb}
    trials, r = 3000, 4
    for e in range(trials):
        ids, cnt = sage.sample_neighbors(pt, 7, e, 1, [v], r)
        assert cnt[0] == r and len(set(ids[0])) == r
        for u in ids[0]:
            hits[int(u)] += 1
    expect = trials * r / len(nb)
    chi2 = sum((h - expect) ** 2 / expect for h in hits.values())
    assert chi2 < 3.0 * len(nb)            # the mean of chi-square is len(nb) - 1


def _dense_operators(pt, fw, r_cols):
    """P1 [need x n], P2 [targets x need], T [targets x need] built from the recorded samples alone."""
    need, targets = fw["need"], fw["targets"]
    p1 = np.zeros((need.size, pt.n))
    for j in range(need.size):
        for u in fw["s1"][j, :fw["c1"][j]]:
            p1[j, u] = 1.0 / fw["c1"][j]
    pos = {int(v): j for j, v in enumerate(need)}
    p2 = np.zeros((targets.size, need.size))
    sel = np.zeros((targets.size, need.size))
    for i, v in enumerate(targets):
        sel[i, pos[int(v)]] = 1.0
        for u in fw["s2"][i, :fw["c2"][i]]:
            p2[i, pos[int(u)]] = 1.0 / fw["c2"][i]
    return p1, p2, sel


def test_batch_forward_and_backward_against_torch_autograd_on_dense_operators():
    pt, x, y, train, params = _case()
    targets = np.flatnonzero(train)[:17]
    fw = sage.batch_forward(pt, x, params, targets, y, 11, 2, (3, 2))
    grads, _ = sage.batch_backward(fw, x, params)
    assert (fw["c1"] <= 3).all() and (fw["c2"] <= 2).all() and fw["c1"].max() == 3
    p1, p2, sel = _dense_operators(pt, fw, None)
    tp = [torch.tensor(a, requires_grad=True) for a in params]
    xt = torch.tensor(x)
    h1 = torch.relu(xt[fw["need"]] @ tp[0] + torch.tensor(p1) @ xt @ tp[1] + tp[2])
    logits = torch.tensor(sel) @ h1 @ tp[3] + torch.tensor(p2) @ h1 @ tp[4] + tp[5]
    loss = torch.nn.functional.cross_entropy(logits, torch.tensor(y[targets], dtype=torch.long))
    loss.backward()
    assert np.allclose(fw["logits"], logits.detach().numpy(), atol=1e-12)
    assert abs(fw["loss"] - float(loss.detach())) < 1e-12
    for g, t in zip(grads, tp):
        assert np.allclose(g, t.grad.numpy(), atol=1e-12)


def test_batch_backward_against_finite_differences():
    pt, x, y, train, params = _case(seed=9)
    targets = np.flatnonzero(train)[3:14]
    fw = sage.batch_forward(pt, x, params, targets, y, 4, 0, (4, 3))
    grads, _ = sage.batch_backward(fw, x, params)
    h = 1e-6
    for arr, grad in zip(params, grads):
        num = np.zeros_like(arr)
        it = np.nditer(arr, flags=["multi_index"])
        for _ in it:
            i = it.multi_index
            old = arr[i]
            arr[i] = old + h
            lp = sage.batch_forward(pt, x, params, targets, y, 4, 0, (4, 3))["loss"]
            arr[i] = old - h
            lm = sage.batch_forward(pt, x, params, targets, y, 4, 0, (4, 3))["loss"]
            arr[i] = old
            num[i] = (lp - lm) / (2 * h)
        assert np.abs(num - grad).max() <= 1e-6 * max(np.abs(num).max(), 1e-3)


def test_full_neighbourhoods_give_the_textbook_mean_aggregator():
    """With fan-outs at least the largest degree nothing is random: H1 = relu(X Ws1 + D^-1 A X Wn1 + b1) and
    logits = H1 Ws2 + D^-1 A H1 Wn2 + b2 on the whole partition, A without self-loops, empty rows giving 0."""
    pt, x, y, train, params = _case(n=45, prob=0.05, m=1, o_ppm=0, seed=2)
    a = np.zeros((pt.n, pt.n))
    for v in range(pt.n):
        a[v, _neighbors(pt, v)] = 1.0
    deg = a.sum(1)
    assert (deg == 0).any(), "the case should contain an isolated vertex"
    mean = a / np.maximum(deg, 1.0)[:, None]
    ws1, wn1, b1, ws2, wn2, b2 = params
    h1 = np.maximum(x @ ws1 + mean @ x @ wn1 + b1, 0.0)
    want = h1 @ ws2 + mean @ h1 @ wn2 + b2
    targets = np.arange(pt.n)
    fw = sage.batch_forward(pt, x, params, targets, y, 1, 0, (1000, 1000))
    assert np.allclose(fw["logits"], want, atol=1e-12)


def test_batches_are_the_training_vertices_in_key_order():
    pt, x, y, train, params = _case()
    for epoch in (0, 1):
        bs = sage.batches(pt, train, 5, epoch, 8)
        flat = np.concatenate(bs)
        assert sorted(flat) == list(np.flatnonzero(train)) and all(len(b) == 8 for b in bs[:-1]) and 1 <= len(bs[-1]) <= 8
        keys = [oracle.key(5, 4, pt.p, epoch, 0, int(v)) for v in flat]
        assert keys == sorted(keys)
    assert not np.array_equal(np.concatenate(sage.batches(pt, train, 5, 0, 8)), np.concatenate(sage.batches(pt, train, 5, 1, 8)))
    assert sage.batches(pt, np.zeros_like(train), 5, 0, 8) == []


def test_epoch_against_torch_adam_per_worker():
    """Two workers, two epochs: every batch one Adam step on the worker's copy (own state), parameters averaged."""
    n, m = 50, 2
    rng = np.random.default_rng(3)
    rowptr, col = graphs.erdos_renyi(n, 0.15, 3)
    _, parts = oracle.build_partitions(rowptr, col, m, 400_000, seed=3)
    x = rng.standard_normal((n, 5)); y = rng.integers(0, 3, n); train = rng.random(n) < 0.8
    params = [rng.standard_normal((5, 4)) * 0.4, rng.standard_normal((5, 4)) * 0.4, np.zeros(4),
              rng.standard_normal((4, 3)) * 0.4, rng.standard_normal((4, 3)) * 0.4, np.zeros(3)]
    xs = [x[pt.members] for pt in parts]; ys = [y[pt.members] for pt in parts]; trs = [train[pt.members] for pt in parts]
    opts = [oracle.Adam(params, 0.01) for _ in parts]
    tw = [[torch.tensor(a.copy(), requires_grad=True) for a in params] for _ in parts]
    topt = [torch.optim.Adam(t, lr=0.01) for t in tw]
    cur = params
    for e in range(2):
        cur, loss = sage.epoch(parts, xs, ys, trs, cur, opts, 21, e, (3, 2), 7)
        want_losses = []
        for pt, xx, yy, tr, t, o in zip(parts, xs, ys, trs, tw, topt):
            total = 0.0
            for tg in sage.batches(pt, tr, 21, e, 7):
                now = [a.detach().numpy() for a in t]
                fw = sage.batch_forward(pt, xx, now, tg, yy, 21, e, (3, 2))     # only its recorded samples are used
                p1, p2, sel = _dense_operators(pt, fw, None)
                xt = torch.tensor(xx)
                h1 = torch.relu(xt[fw["need"]] @ t[0] + torch.tensor(p1) @ xt @ t[1] + t[2])
                logits = torch.tensor(sel) @ h1 @ t[3] + torch.tensor(p2) @ h1 @ t[4] + t[5]
                l = torch.nn.functional.cross_entropy(logits, torch.tensor(yy[tg], dtype=torch.long))
                o.zero_grad(); l.backward(); o.step()
                total += float(l.detach()) * tg.size
            want_losses.append(total / int(tr.sum()))
        with torch.no_grad():
            mean = [sum(t[i] for t in tw) / m for i in range(6)]
            for t in tw:
                for i in range(6):
                    t[i].copy_(mean[i])
        assert abs(loss - np.mean(want_losses)) < 1e-12
        for got, want in zip(cur, mean):
            assert np.allclose(got, want.numpy(), atol=1e-12)


def test_backward_with_given_relu_decisions():
    """batch_backward(relu_on=...): bitwise the default on the checker's own signs; with flipped units it is the
    gradient of the network whose hidden activation is z * mask for that fixed mask (torch autograd); malformed
    masks are rejected."""
    pt, x, y, train, params = _case(seed=12)
    targets = np.flatnonzero(train)[:15]
    fw = sage.batch_forward(pt, x, params, targets, y, 3, 1, (3, 2))
    own = fw["z1"] > 0.0
    a, _ = sage.batch_backward(fw, x, params)
    b, _ = sage.batch_backward(fw, x, params, relu_on=own)
    assert all(np.array_equal(u, v) for u, v in zip(a, b))
    mask = own.copy()
    tj = fw["tj"]
    on_units = np.argwhere(own[tj] & (fw["z1"][tj] > 0.05))
    off_units = np.argwhere(~own[tj] & (fw["z1"][tj] < -0.05))
    i, c = on_units[0]; mask[tj[i], c] = False            # an active unit of a batch vertex switched off
    i, c = off_units[1]; mask[tj[i], c] = True            # an inactive one switched on
    p1, p2, sel = _dense_operators(pt, fw, None)
    tp = [torch.tensor(v, requires_grad=True) for v in params]
    xt = torch.tensor(x)
    z1 = xt[fw["need"]] @ tp[0] + torch.tensor(p1) @ xt @ tp[1] + tp[2]
    h1 = z1 * torch.tensor(mask.astype(np.float64))
    logits = torch.tensor(sel) @ h1 @ tp[3] + torch.tensor(p2) @ h1 @ tp[4] + tp[5]
    loss = torch.nn.functional.cross_entropy(logits, torch.tensor(y[targets], dtype=torch.long))
    loss.backward()
    # the checker's record of the same function: the forward values of the forced network
    forced = dict(fw)
    forced["h1"] = h1.detach().numpy()
    forced["m2"] = p2 @ forced["h1"]
    forced["logits"] = logits.detach().numpy()
    zmax = forced["logits"].max(axis=1, keepdims=True)
    forced["lse"] = zmax[:, 0] + np.log(np.exp(forced["logits"] - zmax).sum(axis=1))
    grads, _ = sage.batch_backward(forced, x, params, relu_on=mask)
    plain, _ = sage.batch_backward(forced, x, params)
    assert not np.allclose(plain[0], grads[0], rtol=1e-9, atol=0), "the flips must matter"
    for g, t in zip(grads, tp):
        assert np.allclose(g, t.grad.numpy(), atol=1e-12)
    for bad in (mask[:, :2], mask.T, mask.astype(np.float64), mask[:-1]):
        with pytest.raises(ValueError):
            sage.batch_backward(fw, x, params, relu_on=bad)
