"""CPU checker ("oracle") for subgraph-approximation GCN training: fp64, plain.

TEST INFRASTRUCTURE ONLY.  Nothing in the CUDA library or its Python binding
may import this module; only the tests, the smoke check and the benchmark's
CPU-baseline leg do.  It shares no code with the CUDA path.

The graph steps (selection key, partition assignment, Algorithm 1, the
augmented partition graph with its normalized weights, transpose, SpMM) are
plain C in ``gcnsa_oracle.c``; the dense steps below are numpy in fp64, one
statement per formula:

  forward   H^l = sigma(A_hat H^{l-1} W^l + b^l), H^0 = X    (Section 4.1)
  loss      mean over the training vertices of softmax cross-entropy
            (vertex classification, Section 2.2)
  backward  the chain rule applied to the two lines above
  step      average of the partition gradients (the paper's epoch-end
            aggregation, Section 3.2, applied to gradients), then Adam
            (Kingma and Ba, Algorithm 1 with bias correction)

Pinned by tests/test_oracle_*.py: hand-worked Algorithm 1 example, brute-force
dense level sets, closed-form normalization, dense A_hat H W, finite
differences, torch CPU autograd and torch.optim.Adam.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SO = os.path.join(_HERE, "libgcnsa_oracle.so")
_SRC = os.path.join(_HERE, "gcnsa_oracle.c")

PART_RANGE, PART_HASH, PART_USER = 0, 1, 2

ERR = {-1: "bad argument", -2: "out of memory", -3: "user partition id out of range",
       -4: "graph not symmetric", -5: "self-loop or repeated edge"}


def build(force: bool = False) -> str:
    """Compile the C part with gcc (OpenMP over SpMM rows)."""
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-o", _SO, _SRC, "-lm"])
    return _SO


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = ctypes.CDLL(build())
        i64, u64, i32, vp = ctypes.c_int64, ctypes.c_uint64, ctypes.c_int32, ctypes.c_void_p
        L.gcnsa_o_key.restype = u64
        L.gcnsa_o_key.argtypes = [u64] * 6
        L.gcnsa_o_partition.restype = ctypes.c_int
        L.gcnsa_o_partition.argtypes = [i64, i64, ctypes.c_int, u64, vp, vp]
        L.gcnsa_o_sample.restype = i64
        L.gcnsa_o_sample.argtypes = [i64, vp, vp, vp, ctypes.c_int, ctypes.c_int, i64, u64, vp, vp]
        L.gcnsa_o_nts.restype = i64
        L.gcnsa_o_nts.argtypes = [i64, i64, i64]
        L.gcnsa_o_induced.restype = ctypes.c_int
        L.gcnsa_o_induced.argtypes = [i64, vp, vp, vp, i64, vp, vp, vp]
        L.gcnsa_o_transpose.restype = ctypes.c_int
        L.gcnsa_o_transpose.argtypes = [i64, i64, vp, vp, vp, vp, vp, vp]
        L.gcnsa_o_spmm.restype = ctypes.c_int
        L.gcnsa_o_spmm.argtypes = [i64, vp, vp, vp, vp, i64, vp]
        L.gcnsa_o_validate.restype = ctypes.c_int
        L.gcnsa_o_validate.argtypes = [i64, vp, vp]
        L.gcnsa_o_sample_neighbors.restype = ctypes.c_int
        L.gcnsa_o_sample_neighbors.argtypes = [i64, vp, vp, u64, u64, u64, u64, i64, vp, i64, vp, vp]
        _lib = L
    return _lib


def _p(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _check(rc):
    if rc < 0:
        raise ValueError(ERR.get(int(rc), f"oracle error {rc}"))
    return rc


def _c(a, dt):
    return np.ascontiguousarray(a, dtype=dt)


# ------------------------------------------------------------ graph steps ---
def key(seed, w0, w1, w2, w3, v) -> int:
    return int(lib().gcnsa_o_key(seed, w0, w1, w2, w3, v))


def validate(rowptr, col):
    rowptr, col = _c(rowptr, np.int64), _c(col, np.int32)
    _check(lib().gcnsa_o_validate(rowptr.size - 1, _p(rowptr), _p(col)))


def partition(n, m, mode=PART_RANGE, seed=0, user=None) -> np.ndarray:
    part = np.empty(n, dtype=np.int32)
    u = None if user is None else _c(user, np.int32)
    _check(lib().gcnsa_o_partition(n, m, mode, seed, _p(u), _p(part)))
    return part


def nts(n_p, m, overlap_ppm) -> int:
    return int(lib().gcnsa_o_nts(n_p, m, overlap_ppm))


def sample(rowptr, col, part, p, op, n_to_sample, seed):
    """Algorithm 1 for one (p, op) pair -> (sorted halo ids, BFS levels used)."""
    rowptr, col, part = _c(rowptr, np.int64), _c(col, np.int32), _c(part, np.int32)
    out = np.empty(max(int(n_to_sample), 1), dtype=np.int64)
    depth = np.zeros(1, dtype=np.int32)
    k = _check(lib().gcnsa_o_sample(rowptr.size - 1, _p(rowptr), _p(col), _p(part), p, op, int(n_to_sample),
                                    seed, _p(out), _p(depth)))
    return out[:k].copy(), int(depth[0])


def induced(rowptr, col, members):
    """Augmented partition graph on ``members`` (local order) -> CSR rowptr,
    col (int64) and D^-1/2 (A+I) D^-1/2 values (float64)."""
    rowptr, col, members = _c(rowptr, np.int64), _c(col, np.int32), _c(members, np.int64)
    n, n_loc = rowptr.size - 1, members.size
    rp = np.zeros(n_loc + 1, dtype=np.int64)
    _check(lib().gcnsa_o_induced(n, _p(rowptr), _p(col), _p(members), n_loc, _p(rp), None, None))
    cc = np.empty(int(rp[-1]), dtype=np.int64)
    vv = np.empty(int(rp[-1]), dtype=np.float64)
    _check(lib().gcnsa_o_induced(n, _p(rowptr), _p(col), _p(members), n_loc, _p(rp), _p(cc), _p(vv)))
    return rp, cc, vv


def transpose(n_rows, n_cols, rowptr, col, val):
    rowptr, col, val = _c(rowptr, np.int64), _c(col, np.int64), _c(val, np.float64)
    trp = np.zeros(n_cols + 1, dtype=np.int64)
    tc = np.empty(col.size, dtype=np.int64)
    tv = np.empty(col.size, dtype=np.float64)
    _check(lib().gcnsa_o_transpose(n_rows, n_cols, _p(rowptr), _p(col), _p(val), _p(trp), _p(tc), _p(tv)))
    return trp, tc, tv


def spmm(rowptr, col, val, x):
    """Y = A X by the definition."""
    rowptr, col, val = _c(rowptr, np.int64), _c(col, np.int64), _c(val, np.float64)
    x = _c(x, np.float64)
    y = np.empty((rowptr.size - 1, x.shape[1]), dtype=np.float64)
    _check(lib().gcnsa_o_spmm(rowptr.size - 1, _p(rowptr), _p(col), _p(val), _p(x), x.shape[1], _p(y)))
    return y


class Partition:
    """One augmented partition P_o[p] with its graph."""

    def __init__(self, p, owned, halo_by_op, depth_by_op, nts_, members, rp, cc, vv, trp, tc, tv):
        self.p = p
        self.owned = owned                  # global ids, ascending
        self.halo_by_op = halo_by_op        # {op: sorted global ids}
        self.depth_by_op = depth_by_op      # {op: BFS levels used}
        self.nts = nts_
        self.members = members              # local -> global, owned then halo
        self.n_owned = owned.size
        self.n = members.size
        self.rowptr, self.col, self.val = rp, cc, vv
        self.t_rowptr, self.t_col, self.t_val = trp, tc, tv

    @property
    def nnz(self):
        return int(self.col.size)


def build_partitions(rowptr, col, m, overlap_ppm, seed, mode=PART_RANGE, user=None, only=None):
    """Partition assignment, Algorithm 1 for every ordered pair, and the
    augmented partition graphs.  ``only`` = iterable of partition ids to build
    (all when None).  Returns (part, [Partition])."""
    rowptr, col = _c(rowptr, np.int64), _c(col, np.int32)
    n = rowptr.size - 1
    part = partition(n, m, mode, seed, user)
    out = []
    for p in (range(m) if only is None else only):
        owned = np.flatnonzero(part == p).astype(np.int64)
        k = nts(owned.size, m, overlap_ppm)
        halo_by_op, depth_by_op = {}, {}
        for op in range(m):                       # for op in P \ p
            if op == p:
                continue
            halo_by_op[op], depth_by_op[op] = sample(rowptr, col, part, p, op, k, seed)
        halo = np.sort(np.concatenate([halo_by_op[op] for op in sorted(halo_by_op)] + [np.zeros(0, np.int64)]))
        members = np.concatenate([owned, halo])
        rp, cc, vv = induced(rowptr, col, members)
        trp, tc, tv = transpose(members.size, members.size, rp, cc, vv)
        out.append(Partition(p, owned, halo_by_op, depth_by_op, k, members, rp, cc, vv, trp, tc, tv))
    return part, out


# ------------------------------------------------------------ dense steps ---
def train_set(pt: Partition, mask_local, loss_on_halo=1):
    """T_p: the masked vertices of the partition that carry loss."""
    t = np.asarray(mask_local).astype(bool).copy()
    if not loss_on_halo:
        t[pt.n_owned:] = False
    return t


def forward(pt: Partition, x_local, ws, bs, y_local, mask_local, loss_on_halo=1):
    """Section 4.1: H^l = sigma(A_hat H^{l-1} W^l + b^l); sigma = ReLU between
    layers, the last layer's output goes to softmax cross-entropy.
    Returns dict with S[l] = A_hat H^{l-1}, Z[l], H[l], loss."""
    h = np.asarray(x_local, dtype=np.float64)
    S, Z, H = [], [], [h]
    n_layers = len(ws)
    for l in range(n_layers):
        s = spmm(pt.rowptr, pt.col, pt.val, h)              # A_hat H^{l-1}
        z = s @ np.asarray(ws[l], np.float64)               # ... W^l
        if bs is not None and bs[l] is not None:
            z = z + np.asarray(bs[l], np.float64)[None, :]
        h = np.maximum(z, 0.0) if l < n_layers - 1 else z
        S.append(s); Z.append(z); H.append(h)
    t = train_set(pt, mask_local, loss_on_halo)
    nt = int(t.sum())
    logits = Z[-1]
    zmax = logits.max(axis=1, keepdims=True)
    lse = zmax[:, 0] + np.log(np.exp(logits - zmax).sum(axis=1))
    picked = logits[np.arange(pt.n), np.asarray(y_local, dtype=np.int64)]
    loss = float(((lse - picked) * t).sum() / nt) if nt > 0 else 0.0
    return {"S": S, "Z": Z, "H": H, "loss": loss, "t": t, "nt": nt, "lse": lse}


def backward(pt: Partition, fw, ws, y_local, relu_on=None):
    """Gradients of the partition loss w.r.t. every W^l and b^l (chain rule).

    ReLU'(z) = [z > 0].  ``relu_on`` (optional, one boolean array per hidden
    layer) replaces that decision: a parity test passes the decision the fp32
    path took for the few units whose |z| lies below fp32 resolution, where
    the sign of z is not determined, so that both sides differentiate the same
    piecewise-linear function."""
    n_layers = len(ws)
    if relu_on is not None:
        if len(relu_on) != n_layers - 1:
            raise ValueError(f"relu_on needs one array per hidden layer ({n_layers - 1}), got {len(relu_on)}")
        relu_on = [np.asarray(on) for on in relu_on]
        for l, on in enumerate(relu_on):
            if on.shape != fw["Z"][l].shape or on.dtype != np.bool_:
                raise ValueError(f"relu_on[{l}] must be a boolean array of shape {fw['Z'][l].shape}")
    logits = fw["Z"][-1]
    nt, t = fw["nt"], fw["t"]
    g = np.zeros_like(logits)
    if nt > 0:
        soft = np.exp(logits - fw["lse"][:, None])
        soft[np.arange(pt.n), np.asarray(y_local, dtype=np.int64)] -= 1.0
        g = soft * t[:, None] / nt
    dW, db, G = [None] * n_layers, [None] * n_layers, [None] * n_layers
    for l in range(n_layers - 1, -1, -1):
        G[l] = g
        dW[l] = fw["S"][l].T @ g                             # (A_hat H^{l-1})^T G^l
        db[l] = g.sum(axis=0)
        if l > 0:
            ds = g @ np.asarray(ws[l], np.float64).T         # G^l W^l^T
            dh = spmm(pt.t_rowptr, pt.t_col, pt.t_val, ds)   # A_hat^T ...
            on = (fw["Z"][l - 1] > 0.0) if relu_on is None else relu_on[l - 1]
            g = dh * on                                      # ReLU'(z) = [z > 0]
    return {"dW": dW, "db": db, "G": G}


class Adam:
    """theta <- theta - lr * m_hat / (sqrt(v_hat) + eps), fp64."""

    def __init__(self, params, lr, beta1=0.9, beta2=0.999, eps=1e-8):
        self.lr, self.b1, self.b2, self.eps = lr, beta1, beta2, eps
        self.m = [np.zeros_like(p, dtype=np.float64) for p in params]
        self.v = [np.zeros_like(p, dtype=np.float64) for p in params]
        self.t = 0

    def step(self, params, grads):
        self.t += 1
        out = []
        for i, (p, g) in enumerate(zip(params, grads)):
            self.m[i] = self.b1 * self.m[i] + (1.0 - self.b1) * g
            self.v[i] = self.b2 * self.v[i] + (1.0 - self.b2) * g * g
            m_hat = self.m[i] / (1.0 - self.b1 ** self.t)
            v_hat = self.v[i] / (1.0 - self.b2 ** self.t)
            out.append(p - self.lr * m_hat / (np.sqrt(v_hat) + self.eps))
        return out


def epoch(parts, xs, ys, masks, ws, bs, opt: Adam, loss_on_halo=1, keep=False):
    """One epoch: forward + backward on every augmented partition at the same
    parameters, unweighted mean of the partition gradients, one Adam step.
    Returns (ws, bs, mean partition loss, per-partition records if keep)."""
    m = len(parts)
    L = len(ws)
    gw = [np.zeros_like(w, dtype=np.float64) for w in ws]
    gb = [np.zeros_like(b, dtype=np.float64) for b in bs]
    losses, recs = [], []
    for pt, x, y, mk in zip(parts, xs, ys, masks):
        fw = forward(pt, x, ws, bs, y, mk, loss_on_halo)
        bw = backward(pt, fw, ws, y)
        for l in range(L):
            gw[l] += bw["dW"][l]
            gb[l] += bw["db"][l]
        losses.append(fw["loss"])
        if keep:
            recs.append((fw, bw))
    gw = [g / m for g in gw]
    gb = [g / m for g in gb]
    new = opt.step(list(ws) + list(bs), gw + gb)
    return new[:L], new[L:], float(np.mean(losses)), (recs, gw, gb)


def epoch_param_avg(parts, xs, ys, masks, ws, bs, opts, loss_on_halo=1):
    """One epoch of the master-worker scheme as Section 3.2 states it: every
    worker starts from the aggregated parameters, trains on its own extended
    partition for the epoch (full batch: one Adam step, with the worker's own
    Adam state ``opts[p]``), and the master averages the workers' parameters.
    Returns (ws, bs, mean partition loss)."""
    m, L = len(parts), len(ws)
    acc = [np.zeros_like(w, dtype=np.float64) for w in list(ws) + list(bs)]
    losses = []
    for pt, x, y, mk, opt in zip(parts, xs, ys, masks, opts):
        fw = forward(pt, x, ws, bs, y, mk, loss_on_halo)
        bw = backward(pt, fw, ws, y)
        w_i = opt.step(list(ws) + list(bs), bw["dW"] + bw["db"])      # W_i^k
        for a, w in zip(acc, w_i):
            a += w
        losses.append(fw["loss"])
    agg = [a / m for a in acc]                                          # W_agg^k
    return agg[:L], agg[L:], float(np.mean(losses))


def predict(pt: Partition, x_local, ws, bs):
    """Predicted class per vertex: argmax of the last layer's output (ties to
    the lowest class index), and the logits."""
    n = pt.n
    fw = forward(pt, x_local, ws, bs, np.zeros(n, dtype=np.int64), np.zeros(n, dtype=np.uint8))
    logits = fw["Z"][-1]
    return np.argmax(logits, axis=1), logits


def micro_f1(pred, y, mask, n_classes):
    """Micro-averaged F1 (Section 2.2: "the micro-averaged harmonic mean of
    precision and recall, which we call accuracy"): true positives, false
    positives and false negatives are summed over the classes before the
    harmonic mean is taken.  Returns (f1, tp, fp, fn)."""
    sel = np.asarray(mask).astype(bool)
    p, t = np.asarray(pred)[sel], np.asarray(y)[sel]
    tp = fp = fn = 0
    for c in range(n_classes):
        tp += int(np.sum((p == c) & (t == c)))
        fp += int(np.sum((p == c) & (t != c)))
        fn += int(np.sum((p != c) & (t == c)))
    if tp == 0:
        return 0.0, tp, fp, fn
    precision, recall = tp / (tp + fp), tp / (tp + fn)
    return 2 * precision * recall / (precision + recall), tp, fp, fn


def train(wl, epochs=None, keep_first=False):
    """Run a whole workload (an object with the fields of gen.configs.Workload)."""
    part, parts = build_partitions(wl.rowptr, wl.col, wl.m, wl.overlap_ppm, wl.seed, wl.part_mode, wl.user_part)
    xs = [wl.x[pt.members].astype(np.float64) for pt in parts]
    ys = [wl.y[pt.members] for pt in parts]
    mks = [wl.train_mask[pt.members] for pt in parts]
    ws = [w.astype(np.float64) for w in wl.w0]
    bs = [b.astype(np.float64) for b in wl.b0]
    opt = Adam(ws + bs, wl.lr, wl.beta1, wl.beta2, wl.eps)
    losses, first = [], None
    for e in range(wl.epochs if epochs is None else epochs):
        ws, bs, loss, rec = epoch(parts, xs, ys, mks, ws, bs, opt, wl.loss_on_halo, keep=(keep_first and e == 0))
        if keep_first and e == 0:
            first = rec
        losses.append(loss)
    return {"part": part, "parts": parts, "ws": ws, "bs": bs, "losses": losses, "first": first, "opt": opt}
