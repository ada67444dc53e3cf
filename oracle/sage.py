"""CPU checker for the GraphSAGE variant (Section 4.1, "Investigated GCNs"):
fp64, plain numpy, by the definitions.

TEST INFRASTRUCTURE ONLY: nothing in the CUDA library or its binding may import
this module; it shares no code with the CUDA path.

What the paper fixes: sampling of a fixed number of neighbours, the element-wise
mean as propagation rule, 2 layers, mini-batches of 256, Adam, learning rates
1e-4 / 2e-4 (Section 4.1); one model copy per worker, trained on the worker's
extended partition for an epoch, parameters averaged at the end of every epoch
(Section 3.2).  What it leaves open, and the reading taken here:

  layer      h_v^k = sigma(h_v^{k-1} Ws^k + mean_{u in S_k(v)} h_u^{k-1} Wn^k + b^k),
             the mean aggregator of the GraphSAGE publication (its concatenation
             [h_v, mean] times one matrix, written as two matrices); ReLU for
             k < K, the last layer's output goes to softmax cross-entropy; no
             normalisation of the embeddings
  fan-out    r_1, r_2 are inputs (the workloads use 25 and 10, the values of the
             GraphSAGE publication)
  sample     S_k(v): uniform without replacement among the neighbours of v inside
             the extended partition, v itself excluded; all of them when there
             are at most r_k; the r_k smallest selection keys (gcnsa_oracle.c);
             an empty neighbourhood has mean 0
  batches    the training vertices T_p in ascending order of the key
             key(seed; 4, p, epoch, 0; v), cut into consecutive groups of `batch`
  training   every batch is one Adam step on worker p's copy of the parameters
             (Adam state kept per worker across epochs); batch loss = mean
             cross-entropy over the batch
  epoch loss mean over partitions of (sum of the batch losses weighted by batch
             size) / |T_p|
"""
from __future__ import annotations

import numpy as np

from . import oracle

TAG_BATCH = 4


def sample_neighbors(pt, seed, epoch, layer, vs, r):
    """S_layer(v) for every v in vs (local ids, -1 = none) -> (ids [len(vs) x r] padded with -1, counts)."""
    L = oracle.lib()
    vs = np.ascontiguousarray(vs, dtype=np.int64)
    out = np.empty((vs.size, max(r, 0)), dtype=np.int64)
    cnt = np.empty(vs.size, dtype=np.int64)
    rp, cc = np.ascontiguousarray(pt.rowptr, np.int64), np.ascontiguousarray(pt.col, np.int64)
    oracle._check(L.gcnsa_o_sample_neighbors(pt.n, oracle._p(rp), oracle._p(cc), seed, pt.p, epoch, layer, vs.size,
                                             oracle._p(vs), r, oracle._p(out), oracle._p(cnt)))
    return out, cnt


def batches(pt, train, seed, epoch, batch):
    """The training vertices of the partition in key order, cut into batches."""
    t = np.flatnonzero(train)
    keys = np.array([oracle.key(seed, TAG_BATCH, pt.p, epoch, 0, int(v)) for v in t], dtype=np.uint64)
    order = t[np.argsort(keys, kind="stable")]
    return [order[i:i + batch] for i in range(0, order.size, batch)]


def batch_forward(pt, x, params, targets, y, seed, epoch, fanout):
    """Forward pass of one mini-batch by the definition.  params = (Ws1, Wn1, b1, Ws2, Wn2, b2)."""
    ws1, wn1, b1, ws2, wn2, b2 = params
    r1, r2 = fanout
    targets = np.asarray(targets, dtype=np.int64)
    s2, c2 = sample_neighbors(pt, seed, epoch, 2, targets, r2)            # who the output layer aggregates
    need = np.unique(np.concatenate([targets, s2[s2 >= 0]]))              # vertices whose h^1 is needed
    s1, c1 = sample_neighbors(pt, seed, epoch, 1, need, r1)               # who the hidden layer aggregates
    m1 = np.zeros((need.size, x.shape[1]))
    for j in range(need.size):
        if c1[j] > 0:
            m1[j] = x[s1[j, :c1[j]]].mean(axis=0)
    z1 = x[need] @ ws1 + m1 @ wn1 + b1
    h1 = np.maximum(z1, 0.0)
    where = {int(v): j for j, v in enumerate(need)}
    tj = np.array([where[int(v)] for v in targets], dtype=np.int64)
    m2 = np.zeros((targets.size, h1.shape[1]))
    for i in range(targets.size):
        if c2[i] > 0:
            m2[i] = h1[[where[int(u)] for u in s2[i, :c2[i]]]].mean(axis=0)
    logits = h1[tj] @ ws2 + m2 @ wn2 + b2
    zmax = logits.max(axis=1, keepdims=True)
    lse = zmax[:, 0] + np.log(np.exp(logits - zmax).sum(axis=1))
    yt = np.asarray(y, dtype=np.int64)[targets]
    losses = lse - logits[np.arange(targets.size), yt]
    return {"targets": targets, "s2": s2, "c2": c2, "need": need, "s1": s1, "c1": c1, "m1": m1, "z1": z1, "h1": h1,
            "tj": tj, "where": where, "m2": m2, "logits": logits, "lse": lse, "yt": yt, "loss": float(losses.mean()),
            "loss_sum": float(losses.sum())}


def batch_backward(fw, x, params, relu_on=None):
    """Gradients of the batch loss (mean cross-entropy) w.r.t. the six parameters: the chain rule.

    ReLU'(z) = [z > 0].  ``relu_on`` (optional boolean array shaped like fw["z1"]) replaces that decision: a parity
    test passes the decision the fp32 path took for the few units whose |z| lies below fp32 resolution, where the
    sign of z is not determined, so that both sides differentiate the same piecewise-linear function."""
    ws1, wn1, b1, ws2, wn2, b2 = params
    if relu_on is not None:
        relu_on = np.asarray(relu_on)
        if relu_on.shape != fw["z1"].shape or relu_on.dtype != np.bool_:
            raise ValueError(f"relu_on must be a boolean array of shape {fw['z1'].shape}")
    nb = fw["targets"].size
    g = np.exp(fw["logits"] - fw["lse"][:, None])
    g[np.arange(nb), fw["yt"]] -= 1.0
    g /= nb                                                   # d loss / d logits
    h1, tj = fw["h1"], fw["tj"]
    d_ws2 = h1[tj].T @ g
    d_wn2 = fw["m2"].T @ g
    d_b2 = g.sum(axis=0)
    dh1 = np.zeros_like(h1)
    np.add.at(dh1, tj, g @ ws2.T)                             # through the vertex's own embedding
    dm2 = g @ wn2.T
    for i in range(nb):                                       # through the mean over S_2(v)
        c = fw["c2"][i]
        for u in fw["s2"][i, :c]:
            dh1[fw["where"][int(u)]] += dm2[i] / c
    dz1 = dh1 * ((fw["z1"] > 0.0) if relu_on is None else relu_on)
    d_ws1 = x[fw["need"]].T @ dz1
    d_wn1 = fw["m1"].T @ dz1
    d_b1 = dz1.sum(axis=0)
    return [d_ws1, d_wn1, d_b1, d_ws2, d_wn2, d_b2], g


def epoch(parts, xs, ys, trains, params, opts, seed, epoch_index, fanout, batch):
    """One epoch of the master-worker scheme (Section 3.2) with mini-batch workers: worker p starts from the
    aggregated parameters, takes one Adam step per batch of its extended partition (its own Adam state opts[p]),
    and the master averages the workers' parameters.  Returns (params, epoch loss)."""
    acc = [np.zeros_like(a, dtype=np.float64) for a in params]
    losses = []
    for pt, x, y, tr, opt in zip(parts, xs, ys, trains, opts):
        cur = [np.array(a, dtype=np.float64) for a in params]
        total, count = 0.0, 0
        for tg in batches(pt, tr, seed, epoch_index, batch):
            fw = batch_forward(pt, x, cur, tg, y, seed, epoch_index, fanout)
            grads, _ = batch_backward(fw, x, cur)
            cur = opt.step(cur, grads)
            total += fw["loss_sum"]
            count += tg.size
        for a, c in zip(acc, cur):
            a += c
        losses.append(total / count if count else 0.0)
    return [a / len(parts) for a in acc], float(np.mean(losses))
