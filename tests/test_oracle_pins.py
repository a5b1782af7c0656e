"""Pins for the CPU oracle: what the paper and the mathematics fix, not the oracle's own formulas.

select_fastest   <- brute force over all subsets; rank-count characterisation; hand example
mixing_weights   <- hand example (Assumption 1); rows sum to 1; doubly stochastic when kept is symmetric
mix_update       <- hand example (Eqs. 4-5 and Eq. 3); dense [W - G eta] P product (compact form);
                    network-mean recursion y(k+1) = y(k) - (eta/N) sum g; consensus limit (Corollary 1);
                    complete graph averages in one round; p_i = 0 keeps the local step; N = 2 average
round_times      <- hand example; T <= max t, = max t when every p >= 1; = theta under DTUR
Dtur             <- hand example; theta is the credited link's establishment time; symmetric masks;
                    each epoch credits every link of P once and its kept links connect the graph
mlp_grad         <- central finite differences of an independently written loss; softmax-regression
                    closed form X^T (softmax - Y) / B; the sub-gradient choice at a ReLU kink (relu_on) by
                    one-sided differences, the margins by a unit placed exactly on the kink
mlp_loss         <- the independently written loss
spanning_links   <- hand example (the link list of a 4-worker path); N - 1 links that connect the graph (Dtur invariants)
dbw_round        <- hand example; the network-mean recursion, the consensus limit and the special cases run through it
"""
import itertools
import json
import os
from fractions import Fraction

import numpy as np
import pytest

from oracle import dbw_oracle as orc
from workloads import configs as wl

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _frac(v):
    return np.array([float(Fraction(s)) for s in v])


def _dense_P(rowptr, col, w_self, w_edge):
    """M[i, j] = weight worker i puts on worker j."""
    n = len(rowptr) - 1
    M = np.zeros((n, n))
    for i in range(n):
        M[i, i] = w_self[i]
        for e in range(rowptr[i], rowptr[i + 1]):
            M[i, col[e]] = w_edge[e]
    return M


# ----------------------------------------------------------------------------- hand examples

def test_hand_example_round():
    g = json.load(open(os.path.join(GOLD, "hand_example_star4.json")))
    rowptr, col = np.array(g["rowptr"]), np.array(g["col"])
    t, b = np.array(g["t"]), np.array(g["b"])
    kept = orc.select_fastest(rowptr, col, t, b)
    assert kept.tolist() == g["kept"]
    ws, we = orc.mixing_weights(rowptr, col, b, kept, orc.METROPOLIS)
    np.testing.assert_allclose(ws, _frac(g["w_self_metropolis"]), rtol=0, atol=1e-15)
    np.testing.assert_allclose(we, _frac(g["w_edge_metropolis"]), rtol=0, atol=1e-15)
    X = np.array(g["X"])[:, None]
    G = np.array(g["G"])[:, None]
    out = orc.mix_update(rowptr, col, X, G, ws, we, g["lr"], orc.LOCAL_THEN_MIX)
    np.testing.assert_allclose(out[:, 0], _frac(g["X_local_then_mix_metropolis"]), rtol=0, atol=1e-14)
    out = orc.mix_update(rowptr, col, X, G, ws, we, g["lr"], orc.MIX_THEN_CORRECT)
    np.testing.assert_allclose(out[:, 0], _frac(g["X_mix_then_correct_metropolis"]), rtol=0, atol=1e-14)
    ws, we = orc.mixing_weights(rowptr, col, b, kept, orc.UNIFORM)
    out = orc.mix_update(rowptr, col, X, G, ws, we, g["lr"], orc.LOCAL_THEN_MIX)
    np.testing.assert_allclose(out[:, 0], _frac(g["X_local_then_mix_uniform"]), rtol=0, atol=1e-14)
    T_nbr, T_worker, T_round = orc.round_times(rowptr, col, t, b, kept)
    assert T_nbr.tolist() == g["T_nbr"]
    assert T_worker.tolist() == g["T_worker"]
    assert T_round == g["T_round"]
    r = orc.dbw_round(rowptr, col, X, t, b, g["lr"], G=G)
    np.testing.assert_allclose(r["X"][:, 0], _frac(g["X_local_then_mix_metropolis"]), rtol=0, atol=1e-14)


def test_hand_example_dtur():
    g = json.load(open(os.path.join(GOLD, "hand_example_dtur_path4.json")))
    rowptr, col = np.array(g["rowptr"]), np.array(g["col"])
    assert [list(l) for l in orc.spanning_links(rowptr, col)] == g["links"]
    d = orc.Dtur(rowptr, col)
    for r in g["rounds"]:
        b, theta = d.update_backups(np.array(r["t"]))
        assert theta == r["theta"] and d.last_link == r["link"] and b.tolist() == r["b"]


# ----------------------------------------------------------------------------- selection

def _small_graphs():
    out = [wl.ring(3), wl.ring(5), wl.path(4), wl.complete(4), wl.complete(5)]
    for s in range(4):
        out.append(wl.erdos_renyi_connected(6, 0.5, 100 + s))
    return out


@pytest.mark.parametrize("ties", [False, True])
def test_selection_brute_force(ties):
    rng = np.random.default_rng(7)
    for rowptr, col in _small_graphs():
        n = len(rowptr) - 1
        deg = np.diff(rowptr)
        for trial in range(6):
            t = rng.integers(0, 3, size=n).astype(np.float64) if ties else rng.random(n)
            for b in itertools.product(*[range(int(dg) + 1) for dg in deg]) if n <= 4 else \
                    [rng.integers(0, deg + 1) for _ in range(20)]:
                b = np.array(b)
                kept = orc.select_fastest(rowptr, col, t, b)
                for i in range(n):
                    nb = [int(col[e]) for e in range(rowptr[i], rowptr[i + 1])]
                    p = int(deg[i] - b[i])
                    # brute force: among all subsets of size p, the one whose sorted
                    # (time, index) keys are lexicographically smallest
                    best = min(itertools.combinations(nb, p),
                               key=lambda s: sorted((t[j], j) for j in s))
                    got = [int(col[e]) for e in range(rowptr[i], rowptr[i + 1]) if kept[e]]
                    assert sorted(best) == got
                    # rank characterisation: kept iff fewer than p neighbours come strictly before
                    for e in range(rowptr[i], rowptr[i + 1]):
                        j = int(col[e])
                        before = sum((t[q], q) < (t[j], j) for q in nb)
                        assert bool(kept[e]) == (before < p)


def test_selection_rejects_bad_b():
    rowptr, col = wl.ring(4)
    with pytest.raises(ValueError):
        orc.select_fastest(rowptr, col, np.zeros(4), np.array([0, 3, 0, 0]))
    with pytest.raises(ValueError):
        orc.select_fastest(rowptr, col, np.zeros(4), np.array([0, -1, 0, 0]))


# ----------------------------------------------------------------------------- weights and the update

def _random_problem(rowptr, col, d, seed):
    rng = np.random.default_rng(seed)
    n = len(rowptr) - 1
    return rng.standard_normal((n, d)), rng.standard_normal((n, d)), 1.0 + rng.random(n)


@pytest.mark.parametrize("rule", [orc.METROPOLIS, orc.UNIFORM])
def test_rows_sum_to_one_and_self_weight_positive(rule):
    rng = np.random.default_rng(3)
    for rowptr, col in _small_graphs() + [wl.random_regular(16, 4, 5)]:
        n = len(rowptr) - 1
        deg = np.diff(rowptr)
        for _ in range(5):
            b = rng.integers(0, deg + 1)
            t = rng.random(n)
            kept = orc.select_fastest(rowptr, col, t, b)
            ws, we = orc.mixing_weights(rowptr, col, b, kept, rule)
            M = _dense_P(rowptr, col, ws, we)
            np.testing.assert_allclose(M.sum(axis=1), 1.0, atol=1e-14)
            p = deg - b
            assert np.all(ws >= 1.0 / (1.0 + p) - 1e-15)
            assert np.all(we[kept == 0] == 0.0)


@pytest.mark.parametrize("order", [orc.LOCAL_THEN_MIX, orc.MIX_THEN_CORRECT])
def test_full_participation_doubly_stochastic_and_mean_follows_sgd(order):
    """b = 0: P is doubly stochastic (Assumption 1) and the network mean obeys
    y(k+1) = y(k) - (eta/N) sum_j g_j (proof sketch of Theorem 1)."""
    for rowptr, col in _small_graphs() + [wl.random_regular(32, 4, 2), wl.erdos_renyi_connected(24, 0.2, 9)]:
        n = len(rowptr) - 1
        X, G, t = _random_problem(rowptr, col, 7, 11)
        b = np.zeros(n, dtype=int)
        kept = orc.select_fastest(rowptr, col, t, b)
        assert kept.all()
        ws, we = orc.mixing_weights(rowptr, col, b, kept)
        M = _dense_P(rowptr, col, ws, we)
        np.testing.assert_allclose(M.sum(axis=0), 1.0, atol=1e-13)
        np.testing.assert_allclose(M, M.T, atol=0)
        lr = 0.3
        Xn = orc.mix_update(rowptr, col, X, G, ws, we, lr, order)
        np.testing.assert_allclose(Xn.mean(axis=0), X.mean(axis=0) - lr * G.mean(axis=0), atol=1e-12)


def test_update_matches_dense_compact_form():
    """Compact form of Eqs. 4-5: W(k) = [W(k-1) - G(k-1) eta(k)] P(k), workers as columns,
    with per-worker learning rates; and Eq. 3: W P - G eta."""
    rng = np.random.default_rng(5)
    for rowptr, col in _small_graphs() + [wl.random_regular(16, 6, 3)]:
        n = len(rowptr) - 1
        deg = np.diff(rowptr)
        X, G, t = _random_problem(rowptr, col, 5, 21)
        b = rng.integers(0, deg + 1)
        lr = 0.1 + rng.random(n)
        for rule in (orc.METROPOLIS, orc.UNIFORM):
            kept = orc.select_fastest(rowptr, col, t, b)
            ws, we = orc.mixing_weights(rowptr, col, b, kept, rule)
            M = _dense_P(rowptr, col, ws, we)          # M[i, j]: weight of j in worker i's average
            P = M.T                                    # paper: column j of P holds worker j's weights
            W = X.T                                    # d x N
            Wn = (W - G.T @ np.diag(lr)) @ P
            np.testing.assert_allclose(orc.mix_update(rowptr, col, X, G, ws, we, lr), Wn.T, atol=1e-13)
            Wn3 = W @ P - G.T @ np.diag(lr)
            np.testing.assert_allclose(
                orc.mix_update(rowptr, col, X, G, ws, we, lr, orc.MIX_THEN_CORRECT), Wn3.T, atol=1e-13)


def test_consensus_limit_zero_gradients():
    """Corollary 1 / Lemma 1: with G = 0 and b = 0 every row tends geometrically to the initial mean."""
    rowptr, col = wl.random_regular(16, 4, 8)
    n = 16
    X, _, t = _random_problem(rowptr, col, 6, 4)
    G = np.zeros_like(X)
    mean0 = X.mean(axis=0)
    b = np.zeros(n, dtype=int)
    dev = []
    for k in range(200):
        r = orc.dbw_round(rowptr, col, X, t, b, 0.05, G=G)
        X = r["X"]
        dev.append(np.abs(X - mean0).max())
        np.testing.assert_allclose(X.mean(axis=0), mean0, atol=1e-12)
    assert dev[-1] < 1e-10
    assert all(dev[k + 1] <= dev[k] + 1e-15 for k in range(len(dev) - 1))
    assert dev[100] < dev[50] * 1e-2 < dev[0] * 1e-4


def test_complete_graph_averages_in_one_round():
    """Complete graph, b = 0: every weight is 1/N, so one round gives the mean of the stepped rows."""
    rowptr, col = wl.complete(6)
    X, G, t = _random_problem(rowptr, col, 4, 2)
    r = orc.dbw_round(rowptr, col, X, t, np.zeros(6, dtype=int), 0.2, G=G)
    np.testing.assert_allclose(r["w_self"], 1 / 6, atol=1e-15)
    np.testing.assert_allclose(r["X"], np.tile((X - 0.2 * G).mean(axis=0), (6, 1)), atol=1e-13)


def test_special_cases():
    # p_i = 0: the worker keeps exactly its own local step (both orders)
    rowptr, col = wl.ring(5)
    X, G, t = _random_problem(rowptr, col, 3, 1)
    b = np.array([2, 0, 1, 0, 2])
    for order in (orc.LOCAL_THEN_MIX, orc.MIX_THEN_CORRECT):
        r = orc.dbw_round(rowptr, col, X, t, b, 0.1, G=G, order=order)
        for i in (0, 4):
            np.testing.assert_allclose(r["X"][i], X[i] - 0.1 * G[i], atol=1e-15)
    # N = 2, b = 0: both rows become the average of the two stepped rows
    rowptr, col = wl.path(2)
    X, G, t = _random_problem(rowptr, col, 3, 6)
    r = orc.dbw_round(rowptr, col, X, t, np.zeros(2, dtype=int), 0.1, G=G)
    avg = 0.5 * ((X[0] - 0.1 * G[0]) + (X[1] - 0.1 * G[1]))
    np.testing.assert_allclose(r["X"], np.stack([avg, avg]), atol=1e-15)


# ----------------------------------------------------------------------------- times and DTUR

def test_round_time_bounds():
    rng = np.random.default_rng(12)
    for rowptr, col in _small_graphs() + [wl.random_regular(16, 4, 5)]:
        n = len(rowptr) - 1
        deg = np.diff(rowptr)
        for _ in range(10):
            t = rng.random(n)
            b = rng.integers(0, deg + 1)
            kept = orc.select_fastest(rowptr, col, t, b)
            T_nbr, T_worker, T_round = orc.round_times(rowptr, col, t, b, kept)
            assert T_round <= t.max()
            if np.all(deg - b >= 1):
                assert T_round == t.max()
            assert np.all(T_worker <= max(T_round, 0.0))
            # T_nbr is the p-th order statistic of the neighbours' times
            for i in range(n):
                p = deg[i] - b[i]
                ts = sorted(t[col[rowptr[i]:rowptr[i + 1]]])
                assert T_nbr[i] == (ts[p - 1] if p >= 1 else 0.0)


@pytest.mark.parametrize("cfg", [1, 2])
def test_dtur_invariants(cfg):
    w = wl.make_workload(cfg)
    rowptr, col, n = w.rowptr, w.col, w.N
    deg = np.diff(rowptr)
    times = wl.arrival_times(w, 3 * (n - 1) + 5)
    dt = orc.Dtur(rowptr, col)
    links = dt.links
    assert len(links) == n - 1
    credited = []
    epoch_edges = set()
    X = np.random.default_rng(1).standard_normal((n, 3))
    G = np.random.default_rng(2).standard_normal((n, 3))
    for k in range(times.shape[0]):
        t = times[k]
        b, theta = dt.update_backups(t)
        u, v = links[dt.last_link]
        assert theta == max(t[u], t[v])                      # establishment time of the credited link
        credited.append(dt.last_link)
        kept = orc.select_fastest(rowptr, col, t, b)
        # top-p selection returns exactly the on-time neighbours of on-time workers
        for i in range(n):
            for e in range(rowptr[i], rowptr[i + 1]):
                assert bool(kept[e]) == (t[i] <= theta and t[col[e]] <= theta)
                if kept[e]:
                    epoch_edges.add((i, int(col[e])))
        assert kept[np.searchsorted(col[rowptr[u]:rowptr[u + 1]], v) + rowptr[u]] == 1
        # symmetric kept relation -> doubly stochastic P -> mean follows SGD even with b > 0
        ws, we = orc.mixing_weights(rowptr, col, b, kept)
        M = _dense_P(rowptr, col, ws, we)
        np.testing.assert_allclose(M, M.T, atol=0)
        np.testing.assert_allclose(M.sum(axis=0), 1.0, atol=1e-13)
        Xn = orc.mix_update(rowptr, col, X, G, ws, we, 0.05)
        np.testing.assert_allclose(Xn.mean(axis=0), X.mean(axis=0) - 0.05 * G.mean(axis=0), atol=1e-12)
        # the round lasts exactly theta
        assert orc.round_times(rowptr, col, t, b, kept)[2] == theta
        if (k + 1) % (n - 1) == 0:
            assert sorted(credited) == list(range(n - 1))     # every link of P exactly once
            assert dt.step == 0 and not any(dt.covered)
            assert wl._connected(n, list(epoch_edges))        # Assumption 2 with B = |P|
            credited, epoch_edges = [], set()
    assert np.all((b >= 0) & (b <= deg))


def test_dtur_shorter_rounds_than_full_participation():
    """Corollary 4 (weak sanity): threshold rounds never last longer than waiting for everyone."""
    w = wl.make_workload(1)
    times = wl.arrival_times(w, 100)
    dt = orc.Dtur(w.rowptr, w.col)
    thetas = np.array([dt.update_backups(t)[1] for t in times])
    assert np.all(thetas <= times.max(axis=1))
    assert thetas.mean() < times.max(axis=1).mean()


# ----------------------------------------------------------------------------- gradients

def _independent_loss(x, layers, feats, labels):
    """Mean cross-entropy written sample by sample with explicit loops (no shared code path)."""
    off = 0
    Ws, bs = [], []
    for l in range(len(layers) - 1):
        fin, fout = layers[l], layers[l + 1]
        Ws.append(np.array(x[off:off + fin * fout]).reshape(fout, fin)); off += fin * fout
        bs.append(np.array(x[off:off + fout])); off += fout
    total = 0.0
    for s in range(len(labels)):
        a = np.array(feats[s], dtype=np.float64)
        for l in range(len(Ws)):
            z = np.array([Ws[l][o] @ a + bs[l][o] for o in range(Ws[l].shape[0])])
            a = np.where(z > 0, z, 0.0) if l < len(Ws) - 1 else z
        pz = np.exp(a - a.max())
        pz /= pz.sum()
        total += -np.log(pz[labels[s]])
    return total / len(labels)


@pytest.mark.parametrize("layers", [[6, 3], [5, 4, 3], [4, 6, 5, 3]])
def test_mlp_grad_finite_differences(layers):
    rng = np.random.default_rng(0)
    d = wl.logical_dim(layers)
    x = rng.standard_normal(d) * 0.7
    feats = rng.standard_normal((5, layers[0]))
    labels = rng.integers(0, layers[-1], size=5)
    g, loss = orc.mlp_grad(x, layers, feats, labels)
    assert abs(loss - _independent_loss(x, layers, feats, labels)) < 1e-12
    assert abs(orc.mlp_loss(x, layers, feats, labels) - loss) < 1e-12
    h = 1e-6
    for k in range(d):
        e = np.zeros(d); e[k] = h
        fd = (_independent_loss(x + e, layers, feats, labels) - _independent_loss(x - e, layers, feats, labels)) / (2 * h)
        assert abs(fd - g[k]) <= 1e-6 * max(1.0, abs(g[k])), (k, fd, g[k])


def test_mlp_grad_subgradient_choice_at_the_kink_matches_one_sided_differences():
    """A hidden unit whose pre-activation is exactly zero for one sample: with the unit forced on the gradient is
    the right-hand derivative of the loss in that unit's bias, forced off (the default) the left-hand one; the
    margins report that unit, and only that unit, as sitting on the kink."""
    rng = np.random.default_rng(3)
    layers = [3, 4, 3]
    d = wl.logical_dim(layers)
    x = rng.standard_normal(d) * 0.8
    W0 = x[:12].reshape(4, 3)
    feats = rng.standard_normal((4, 3))
    feats[2] = [1.0, 0.0, 0.0]
    W0[1] = [0.5, 0.25, -2.0]
    x[12 + 1] = -0.5                      # bias of unit 1: z[sample 2][unit 1] = 0.5 - 0.5 = 0 exactly
    labels = rng.integers(0, 3, size=4)
    margins = []
    g_off, loss = orc.mlp_grad(x, layers, feats, labels, margins=margins)
    g_on, loss_on = orc.mlp_grad(x, layers, feats, labels, relu_on={(1, 2, 1): True})
    g_off2, _ = orc.mlp_grad(x, layers, feats, labels, relu_on={(1, 2, 1): False})
    assert loss == loss_on and np.array_equal(g_off, g_off2)
    assert margins[0][2, 1] == 0.0 and (np.delete(margins[0].ravel(), 2 * 4 + 1) > 1e-3).all()
    k = 12 + 1                            # d loss / d bias of unit 1
    h = 1e-7
    e = np.zeros(d); e[k] = h
    right = (_independent_loss(x + e, layers, feats, labels) - loss) / h
    left = (loss - _independent_loss(x - e, layers, feats, labels)) / h
    assert abs(right - g_on[k]) < 1e-6 and abs(left - g_off[k]) < 1e-6
    assert abs(g_on[k] - g_off[k]) > 1e-3  # the two choices really differ here
    # every entry that does not pass through that unit is the same under both choices
    same = np.ones(d, dtype=bool)
    same[3:6] = False                     # row 1 of W0
    same[k] = False
    assert np.allclose(g_on[same], g_off[same], atol=1e-15)


def test_softmax_regression_closed_form():
    rng = np.random.default_rng(1)
    fin, fout, B = 7, 4, 9
    W = rng.standard_normal((fout, fin)); bias = rng.standard_normal(fout)
    A = rng.standard_normal((B, fin)); y = rng.integers(0, fout, size=B)
    g, _ = orc.mlp_grad(np.concatenate([W.ravel(), bias]), [fin, fout], A, y)
    Z = A @ W.T + bias
    S = np.exp(Z) / np.exp(Z).sum(axis=1, keepdims=True)
    Y = np.eye(fout)[y]
    gW = (S - Y).T @ A / B
    gb = (S - Y).mean(axis=0)
    np.testing.assert_allclose(g, np.concatenate([gW.ravel(), gb]), atol=1e-13)


def test_loss_decreases_on_synthetic_task():
    """Weak whole-run trend: config 0 shrunk, 30 rounds, mean loss goes down."""
    w = wl.make_workload(0, samples=200)
    means = wl.class_means(w)
    data = [wl.worker_dataset(w, i, means) for i in range(w.N)]
    X = np.stack([wl.init_params(w, i) for i in range(w.N)]).astype(np.float64)
    times = wl.arrival_times(w, 30)
    b = wl.fixed_backups(w)
    losses = []
    for k in range(30):
        idx = wl.batch_indices(w, k)
        feats = [data[i][0][idx[i]] for i in range(w.N)]
        labels = [data[i][1][idx[i]] for i in range(w.N)]
        r = orc.dbw_round(w.rowptr, w.col, X, times[k], b, 0.5, layers=w.layers, feats=feats, labels=labels)
        X = r["X"]
        losses.append(r["loss"].mean())
    assert losses[-1] < 0.8 * losses[0]


# ----------------------------------------------------------------------------- per-link arrival times

def test_per_link_times_brute_force_and_reduction():
    """With per-link delays the kept set is the p smallest (arrival, index) keys of the worker's own
    links (brute force over subsets); link times equal to the senders' times reproduce the per-worker
    model exactly; T_nbr is the p-th order statistic of the link times; T(k) = max T_j (Section 3.2.2)."""
    rng = np.random.default_rng(21)
    for rowptr, col in _small_graphs() + [wl.random_regular(16, 4, 5)]:
        n = len(rowptr) - 1
        deg = np.diff(rowptr)
        for trial in range(6):
            t = 1.0 + rng.random(n)
            te = np.round(4 * (t[col] + rng.random(len(col)))) / 4          # delays, with ties
            b = rng.integers(0, deg + 1)
            kept = orc.select_fastest(rowptr, col, t, b, t_edge=te)
            T_nbr, T_worker, T_round = orc.round_times(rowptr, col, t, b, kept, t_edge=te)
            waited = np.zeros(n, dtype=bool)
            waited[col[kept == 1]] = True
            for i in range(n):
                es = list(range(rowptr[i], rowptr[i + 1]))
                p = int(deg[i] - b[i])
                best = min(itertools.combinations(es, p), key=lambda s: sorted((te[e], col[e]) for e in s))
                assert sorted(best) == [e for e in es if kept[e]]
                ts = sorted(te[es])
                assert T_nbr[i] == (ts[p - 1] if p >= 1 else 0.0)
                assert T_worker[i] == (max(t[i], T_nbr[i]) if p >= 1 else (t[i] if waited[i] else 0.0))
            part = (deg - b >= 1) | waited
            assert T_round == (T_worker[part].max() if part.any() else 0.0)
            # no extra delay: identical to the per-worker model
            k0 = orc.select_fastest(rowptr, col, t, b)
            assert np.array_equal(k0, orc.select_fastest(rowptr, col, t, b, t_edge=t[col]))
            a0 = orc.round_times(rowptr, col, t, b, k0)
            a1 = orc.round_times(rowptr, col, t, b, k0, t_edge=t[col])
            assert np.array_equal(a0[0], a1[0]) and np.array_equal(a0[1], a1[1]) and a0[2] == a1[2]
            assert a0[2] == (t[(deg - b >= 1) | np.isin(np.arange(n), col[k0 == 1])].max()
                             if ((deg - b >= 1).any() or k0.any()) else 0.0)


def test_non_iid_shards_hold_only_their_classes():
    """Input recipe: with label_skew = k worker i draws labels from classes (i*k + 0..k-1) mod 10 only, and the
    features still are class mean + noise (the label decides the mean)."""
    w = wl.make_workload(5, samples=512, label_skew=2)
    means = wl.class_means(w)
    seen = set()
    for i in range(w.N):
        f, l = wl.worker_dataset(w, i, means)
        own = {(2 * i) % 10, (2 * i + 1) % 10}
        assert set(np.unique(l)) <= own and len(set(np.unique(l))) == 2
        seen |= own
        resid = f - means[l]
        assert abs(float(resid.std()) - w.noise) < 0.05
    assert len(seen) == 10
    f0, l0 = wl.worker_dataset(wl.make_workload(5, samples=512), 0, means)
    assert len(np.unique(l0)) == 10
