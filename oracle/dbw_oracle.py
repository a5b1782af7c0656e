"""CPU oracle for one round of consensus SGD with dynamic backup workers (cb-DyBW).

TEST INFRASTRUCTURE ONLY.  This is a plain, slow, double-precision restatement of
the paper's round, written to be checked against the paper by eye.  It shares no
code with the CUDA library, imports nothing from it, and must never be reachable
from the product path; only the tests, the smoke check and the benchmark's CPU
baseline leg call it.

Conventions (paper, Section 2): N workers on an undirected connected graph given
as sorted CSR (rowptr, col) without self loops; row i of X (N x d) is worker i's
parameter vector w_i (the paper stores workers as columns of W; this is its
transpose); deg_i neighbours, b_i backup workers, p_i = deg_i - b_i neighbours
waited for; t_i the time at which worker i's local update is available.

Every function is pinned by something other than itself; what pins which is
listed in tests/test_oracle_pins.py: invariants, closed forms, brute force on
tiny inputs, finite differences and hand-derived examples.  The paper prints no
worked numerical round, so none of the pins is a value printed by the paper.
"""
from __future__ import annotations

import numpy as np

METROPOLIS = "metropolis"
UNIFORM = "uniform"
LOCAL_THEN_MIX = "local_then_mix"      # Algorithm 1 / Eqs. 4-5
MIX_THEN_CORRECT = "mix_then_correct"  # Eq. 3 restricted to the kept set


# ---------------------------------------------------------------------------
# Section 2.2: worker j waits for the first p_j(k) updates of its neighbours
# ---------------------------------------------------------------------------

def select_fastest(rowptr, col, t, b, t_edge=None):
    """Kept-neighbour mask, aligned with `col` (1 = waited for, 0 = backup).

    Section 2.2: worker i keeps the first p_i = deg_i - b_i updates to arrive.
    The update of neighbour j arrives at t_j; equal times are ordered by the
    lower worker index.  With `t_edge` (aligned with `col`) the update of
    col[e] arrives at worker i at t_edge[e] instead (per-link delays).
    """
    n = len(rowptr) - 1
    kept = np.zeros(len(col), dtype=np.uint8)
    for i in range(n):
        lo, hi = int(rowptr[i]), int(rowptr[i + 1])
        deg = hi - lo
        p = deg - int(b[i])
        if p < 0 or p > deg:
            raise ValueError("b out of range for worker %d" % i)
        arrive = (lambda e: float(t_edge[e])) if t_edge is not None else (lambda e: float(t[col[e]]))
        order = sorted(range(lo, hi), key=lambda e: (arrive(e), int(col[e])))
        for e in order[:p]:
            kept[e] = 1
    return kept


# ---------------------------------------------------------------------------
# Section 3.2.2: T_j(k) = max{t_i : i in S_j(k)}, V' = union of the S_i,
# T(k) = max{T_j : j in V'}
# ---------------------------------------------------------------------------

def round_times(rowptr, col, t, b, kept, t_edge=None):
    """(T_nbr, T_worker, T_round) of one round.

    T_nbr[i]    = max arrival time over the kept neighbours of i (0.0 when p_i = 0);
    a worker participates when it waits for someone or someone waits for it;
    T_worker[i] = max(t_i, T_nbr[i]) when p_i >= 1, t_i when it only participates
                  through others, 0.0 when it does not participate;
    T_round     = max of T_worker over the participating workers (0.0 if none).
    Without per-link delays this is the max of t over the participating workers,
    because every kept neighbour participates itself.
    """
    n = len(rowptr) - 1
    t = np.asarray(t, dtype=np.float64)
    p = np.diff(rowptr) - np.asarray(b)
    T_nbr = np.zeros(n)
    waited_for = np.zeros(n, dtype=bool)
    for i in range(n):
        for e in range(int(rowptr[i]), int(rowptr[i + 1])):
            if kept[e]:
                j = int(col[e])
                waited_for[j] = True
                T_nbr[i] = max(T_nbr[i], t[j] if t_edge is None else t_edge[e])
    T_worker = np.zeros(n)
    T_round = 0.0
    for i in range(n):
        participating = p[i] >= 1 or waited_for[i]
        if p[i] >= 1:
            T_worker[i] = max(t[i], T_nbr[i])
        elif participating:
            T_worker[i] = t[i]
        if participating:
            T_round = max(T_round, T_worker[i])
    return T_nbr, T_worker, T_round


# ---------------------------------------------------------------------------
# Assumption 1: Metropolis weights on the kept links
# ---------------------------------------------------------------------------

def mixing_weights(rowptr, col, b, kept, rule=METROPOLIS):
    """(w_self (N,), w_edge (nnz,)) — the weight worker i puts on itself and on col[e].

    METROPOLIS (Assumption 1): w_ij = 1 / (1 + max{p_i, p_j}) for kept j,
    w_ii = 1 - sum of the kept w_ij, 0 for backups.
    UNIFORM: w_ii = w_ij = 1 / (1 + p_i) over self and the kept neighbours.
    """
    n = len(rowptr) - 1
    p = np.diff(rowptr) - np.asarray(b)
    w_edge = np.zeros(len(col))
    w_self = np.zeros(n)
    for i in range(n):
        s = 0.0
        for e in range(int(rowptr[i]), int(rowptr[i + 1])):
            if kept[e]:
                j = int(col[e])
                if rule == METROPOLIS:
                    w_edge[e] = 1.0 / (1.0 + max(int(p[i]), int(p[j])))
                elif rule == UNIFORM:
                    w_edge[e] = 1.0 / (1.0 + int(p[i]))
                else:
                    raise ValueError(rule)
                s += w_edge[e]
        w_self[i] = 1.0 - s if rule == METROPOLIS else 1.0 / (1.0 + int(p[i]))
    return w_self, w_edge


# ---------------------------------------------------------------------------
# Eqs. 4-5 (Algorithm 1) and Eq. 3
# ---------------------------------------------------------------------------

def mix_update(rowptr, col, X, G, w_self, w_edge, lr, order=LOCAL_THEN_MIX):
    """New parameters X' (N x d, float64), all read from the OLD X.

    LOCAL_THEN_MIX (Eqs. 4-5): xt_j = x_j - lr_j g_j for every j, then
        x'_i = w_ii xt_i + sum over kept j of w_ij xt_j.
    MIX_THEN_CORRECT (Eq. 3 over the kept set):
        x'_i = w_ii x_i + sum over kept j of w_ij x_j - lr_i g_i.
    `lr` is a scalar or one value per worker.  Any subset of columns may be
    passed: the update is independent per column.
    """
    X = np.asarray(X, dtype=np.float64)
    G = np.asarray(G, dtype=np.float64)
    n = X.shape[0]
    lr = np.broadcast_to(np.asarray(lr, dtype=np.float64), (n,))
    out = np.zeros_like(X)
    if order == LOCAL_THEN_MIX:
        Xt = X - lr[:, None] * G
        for i in range(n):
            acc = w_self[i] * Xt[i]
            for e in range(int(rowptr[i]), int(rowptr[i + 1])):
                if w_edge[e] != 0.0:
                    acc = acc + w_edge[e] * Xt[int(col[e])]
            out[i] = acc
    elif order == MIX_THEN_CORRECT:
        for i in range(n):
            acc = w_self[i] * X[i]
            for e in range(int(rowptr[i]), int(rowptr[i + 1])):
                if w_edge[e] != 0.0:
                    acc = acc + w_edge[e] * X[int(col[e])]
            out[i] = acc - lr[i] * G[i]
    else:
        raise ValueError(order)
    return out


# ---------------------------------------------------------------------------
# Section 4: distributed threshold-based update rule (DTUR), Algorithm 2
# ---------------------------------------------------------------------------

def spanning_links(rowptr, col):
    """The link set P: a spanning tree (N - 1 links, the fewest that connect all nodes).

    Breadth-first search from worker 0, neighbours visited in ascending index;
    links are listed in the order their far end is discovered.
    """
    n = len(rowptr) - 1
    seen = np.zeros(n, dtype=bool)
    seen[0] = True
    queue = [0]
    links = []
    head = 0
    while head < len(queue):
        u = queue[head]
        head += 1
        for e in range(int(rowptr[u]), int(rowptr[u + 1])):
            v = int(col[e])
            if not seen[v]:
                seen[v] = True
                links.append((u, v))
                queue.append(v)
    if len(links) != n - 1:
        raise ValueError("graph is not connected")
    return links


class Dtur:
    """State of Algorithm 2: the links P, the covered set P' and the position in the epoch."""

    def __init__(self, rowptr, col):
        self.rowptr = np.asarray(rowptr)
        self.col = np.asarray(col)
        self.links = spanning_links(rowptr, col)
        self.covered = [False] * len(self.links)
        self.step = 0          # links covered so far in this epoch
        self.last_link = -1    # position in P of the link credited by the last call

    def update_backups(self, t):
        """(b, theta) for the round whose arrival times are t.

        theta = the earliest establishment time max(t_u, t_v) among links of P
        not yet in P' (first such link on ties); that link joins P'; after
        |P| iterations P' is emptied.  Then (threshold rule of Section 4.1)
        worker j waits for the neighbours with t_i <= theta if t_j <= theta,
        and for nobody otherwise; b_j = deg_j - p_j.
        """
        t = np.asarray(t, dtype=np.float64)
        best, theta = -1, np.inf
        for pos, (u, v) in enumerate(self.links):
            if not self.covered[pos]:
                est = max(t[u], t[v])
                if est < theta:
                    best, theta = pos, est
        self.covered[best] = True
        self.last_link = best
        self.step += 1
        if self.step == len(self.links):
            self.covered = [False] * len(self.links)
            self.step = 0
        n = len(self.rowptr) - 1
        b = np.zeros(n, dtype=np.int32)
        for j in range(n):
            lo, hi = int(self.rowptr[j]), int(self.rowptr[j + 1])
            p = 0
            if t[j] <= theta:
                p = sum(1 for e in range(lo, hi) if t[self.col[e]] <= theta)
            b[j] = (hi - lo) - p
        return b, float(theta)


# ---------------------------------------------------------------------------
# Eq. 2 (mini-batch stochastic gradient) for an MLP with softmax cross-entropy
# ---------------------------------------------------------------------------

def unpack_layers(x, layers):
    """Split a logical parameter row into [(W_l [out][in], b_l [out]), ...]."""
    params = []
    off = 0
    for l in range(len(layers) - 1):
        fin, fout = layers[l], layers[l + 1]
        W = np.asarray(x[off: off + fout * fin], dtype=np.float64).reshape(fout, fin)
        off += fout * fin
        bias = np.asarray(x[off: off + fout], dtype=np.float64)
        off += fout
        params.append((W, bias))
    assert off == len(x)
    return params


def mlp_loss(x, layers, feats, labels):
    """Mean softmax cross-entropy of the ReLU MLP with parameter row x on a batch."""
    a = np.asarray(feats, dtype=np.float64)
    params = unpack_layers(x, layers)
    for l, (W, bias) in enumerate(params):
        z = a @ W.T + bias
        a = np.maximum(z, 0.0) if l < len(params) - 1 else z
    zmax = a.max(axis=1, keepdims=True)
    lse = zmax[:, 0] + np.log(np.exp(a - zmax).sum(axis=1))
    return float(np.mean(lse - a[np.arange(len(labels)), np.asarray(labels)]))


def mlp_grad(x, layers, feats, labels, relu_on=None, margins=None):
    """(g, loss): g = mean over the batch of grad f(x; sample) in the layout of x (Eq. 2).

    At a pre-activation of exactly zero ReLU has the sub-differential [0, 1]; this function takes 0 there.
    A finite-precision implementation may see a pre-activation that is zero up to rounding on either side,
    and both choices are then valid.  `relu_on` maps (layer, sample, unit) (layer = 1 .. L-1, the index of
    the activation) to True / False and forces that unit on (a = z, derivative 1) or off (a = 0, derivative
    0); tests use it to compare at a pre-activation closer to zero than fp32 accumulation resolves.
    `margins`, if a list, receives per hidden layer the array |z| / (|a| |W|^T + |b|): how far, relative to
    the size of its terms, each pre-activation is from the kink."""
    a0 = np.asarray(feats, dtype=np.float64)
    labels = np.asarray(labels)
    B = a0.shape[0]
    params = unpack_layers(x, layers)
    acts = [a0]
    on = []
    a = a0
    for l, (W, bias) in enumerate(params):
        z = a @ W.T + bias
        if l < len(params) - 1:
            if margins is not None:
                margins.append(np.abs(z) / np.maximum(np.abs(a) @ np.abs(W).T + np.abs(bias), 1e-300))
            active = z > 0.0                      # ReLU'(0) = 0
            for (ll, smp, unit), val in (relu_on or {}).items():
                if ll == l + 1:
                    active[smp, unit] = bool(val)
            on.append(active)
            a = np.where(active, z, 0.0)
        else:
            a = z
        acts.append(a)
    logits = acts[-1]
    zmax = logits.max(axis=1, keepdims=True)
    e = np.exp(logits - zmax)
    prob = e / e.sum(axis=1, keepdims=True)
    lse = zmax[:, 0] + np.log(e.sum(axis=1))
    loss = float(np.mean(lse - logits[np.arange(B), labels]))
    dz = prob.copy()
    dz[np.arange(B), labels] -= 1.0
    dz /= B
    grads = [None] * len(params)
    for l in range(len(params) - 1, -1, -1):
        W, _ = params[l]
        grads[l] = (dz.T @ acts[l], dz.sum(axis=0))
        if l > 0:
            da = dz @ W
            dz = da * on[l - 1]
    g = np.concatenate([np.concatenate([gw.ravel(), gb]) for gw, gb in grads])
    return g, loss


# ---------------------------------------------------------------------------
# Algorithm 1: one iteration
# ---------------------------------------------------------------------------

def dbw_round(rowptr, col, X, t, b, lr, G=None, layers=None, feats=None, labels=None,
              rule=METROPOLIS, order=LOCAL_THEN_MIX):
    """One round for all workers.

    Gradients come from `G` (N x d) when given, otherwise worker i's mini-batch
    gradient is computed from feats[i] (B x in), labels[i] (B).  Returns a dict
    with X', G, loss (N,), kept, T_nbr, T_worker, T_round, w_self, w_edge.
    """
    X = np.asarray(X, dtype=np.float64)
    n = X.shape[0]
    loss = np.zeros(n)
    if G is None:
        G = np.zeros_like(X)
        for i in range(n):
            G[i], loss[i] = mlp_grad(X[i], layers, feats[i], labels[i])
    kept = select_fastest(rowptr, col, t, b)
    T_nbr, T_worker, T_round = round_times(rowptr, col, t, b, kept)
    w_self, w_edge = mixing_weights(rowptr, col, b, kept, rule)
    Xn = mix_update(rowptr, col, X, G, w_self, w_edge, lr, order)
    return dict(X=Xn, G=np.asarray(G, dtype=np.float64), loss=loss, kept=kept, T_nbr=T_nbr,
                T_worker=T_worker, T_round=T_round, w_self=w_self, w_edge=w_edge)
