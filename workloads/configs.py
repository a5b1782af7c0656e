"""Seeded generators for the five synthetic workloads.

Everything here is input drawing: communication graphs, MNIST-/CIFAR-shaped
Gaussian-mixture data, initial parameters, worker arrival times, backup counts
and mini-batch indices.  Random numbers come from numpy's PCG64; every array is
a pure function of (config, seed, worker / round index), so a single worker's
shard or a single row of a large matrix can be regenerated on its own.

Seeds: the ones the workload statement fixes are used as stated (class means
seed 0 and arrival times seed 1 for config 0, graph seeds 2 and 3 for configs
1 and 2, parameter seed 4 for config 4); every other purpose uses
1000 * (config + 1) + {graph 1, data 2, init 3, times 4, rates 5, batches 6,
backups 7, gradients 8}.
"""
from __future__ import annotations

from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass, field
from typing import List, Optional, Tuple

import numpy as np

_PURPOSE = {"graph": 1, "data": 2, "init": 3, "times": 4, "rates": 5,
            "batches": 6, "backups": 7, "grads": 8}


def _seed(config: int, purpose: str) -> int:
    return 1000 * (config + 1) + _PURPOSE[purpose]


def _rng(*key: int) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64(np.random.SeedSequence(list(key))))


# --------------------------------------------------------------------------
# graphs (undirected, simple, connected) as sorted CSR without self loops
# --------------------------------------------------------------------------

def _csr_from_edges(n: int, edges) -> Tuple[np.ndarray, np.ndarray]:
    adj = [[] for _ in range(n)]
    for u, v in edges:
        adj[u].append(v)
        adj[v].append(u)
    rowptr = np.zeros(n + 1, dtype=np.int32)
    cols = []
    for i in range(n):
        nb = sorted(adj[i])
        rowptr[i + 1] = rowptr[i] + len(nb)
        cols.extend(nb)
    return rowptr, np.asarray(cols, dtype=np.int32)


def _connected(n: int, edges) -> bool:
    adj = [[] for _ in range(n)]
    for u, v in edges:
        adj[u].append(v)
        adj[v].append(u)
    seen = [False] * n
    stack = [0]
    seen[0] = True
    cnt = 1
    while stack:
        u = stack.pop()
        for v in adj[u]:
            if not seen[v]:
                seen[v] = True
                cnt += 1
                stack.append(v)
    return cnt == n


def ring(n: int) -> Tuple[np.ndarray, np.ndarray]:
    """Cycle on n >= 3 nodes (degree 2)."""
    return _csr_from_edges(n, [(i, (i + 1) % n) for i in range(n)])


def complete(n: int) -> Tuple[np.ndarray, np.ndarray]:
    return _csr_from_edges(n, [(i, j) for i in range(n) for j in range(i + 1, n)])


def path(n: int) -> Tuple[np.ndarray, np.ndarray]:
    return _csr_from_edges(n, [(i, i + 1) for i in range(n - 1)])


def random_regular(n: int, k: int, seed: int) -> Tuple[np.ndarray, np.ndarray]:
    """Random k-regular graph.

    A random perfect matching of the n*k half-edges is drawn, then pairs that
    form a self loop or a duplicate edge are repaired by random edge switches
    (each switch keeps every degree); the whole draw is repeated until the
    result is connected.
    """
    assert (n * k) % 2 == 0 and k < n
    rng = _rng(seed)
    while True:
        stubs = np.repeat(np.arange(n), k)
        rng.shuffle(stubs)
        pairs = [[int(stubs[2 * e]), int(stubs[2 * e + 1])] for e in range(n * k // 2)]

        def key(u, v):
            return (u, v) if u < v else (v, u)

        count = {}
        for u, v in pairs:
            count[key(u, v)] = count.get(key(u, v), 0) + 1

        def bad(e):
            u, v = pairs[e]
            return u == v or count[key(u, v)] > 1

        ok = True
        for _sweep in range(100):
            bad_edges = [e for e in range(len(pairs)) if bad(e)]
            if not bad_edges:
                break
            for e in bad_edges:
                for _try in range(100):
                    if not bad(e):
                        break
                    f = int(rng.integers(len(pairs)))
                    if f == e:
                        continue
                    a, b = pairs[e]
                    c, d = pairs[f]
                    # switch (a,b),(c,d) -> (a,c),(b,d) when both new edges are good
                    if a == c or b == d:
                        continue
                    k1, k2 = key(a, c), key(b, d)
                    if count.get(k1, 0) > 0 or count.get(k2, 0) > 0 or k1 == k2:
                        continue
                    count[key(a, b)] -= 1
                    count[key(c, d)] -= 1
                    pairs[e] = [a, c]
                    pairs[f] = [b, d]
                    count[k1] = count.get(k1, 0) + 1
                    count[k2] = count.get(k2, 0) + 1
        else:
            ok = False
        if ok and _connected(n, pairs):
            return _csr_from_edges(n, pairs)


def erdos_renyi_connected(n: int, p: float, seed: int) -> Tuple[np.ndarray, np.ndarray]:
    """G(n, p), resampled (continuing the same stream) until connected."""
    rng = _rng(seed)
    while True:
        u = rng.random((n, n))
        edges = [(i, j) for i in range(n) for j in range(i + 1, n) if u[i, j] < p]
        if _connected(n, edges):
            return _csr_from_edges(n, edges)


# --------------------------------------------------------------------------
# workload descriptors
# --------------------------------------------------------------------------

@dataclass
class Workload:
    index: int
    name: str
    N: int
    graph: str                       # "ring" | "regular" | "er"
    degree: int = 0                  # regular graphs
    er_p: float = 0.0
    graph_seed: int = 0
    layers: Optional[List[int]] = None   # [in, h1, ..., out]; None = mix-only
    d: int = 0                       # logical parameters per worker
    precision: str = "fp32"          # GEMM operand precision: "fp32" | "bf16"
    samples: int = 0                 # samples per worker
    noise: float = 0.0
    clip: bool = False
    means_seed: int = 0
    label_skew: int = 0              # 0: labels uniform over all classes (iid shards); k > 0: worker i only holds k classes
    batch: int = 0
    lr: float = 0.05
    lr_decay: float = 1.0            # eta(k) = lr * lr_decay^k (k = 0 for the first round)
    rounds: int = 0
    backups: str = "fixed"           # "fixed" | "dtur" | "uniform"
    fixed_b: int = 0
    max_b: int = 0
    weight_rule: str = "metropolis"  # "metropolis" | "uniform"
    times: str = "shifted_exp"       # "shifted_exp" | "lognormal"
    shift: float = 1.0
    rate_mode: str = "one"           # "one" | "uniform_0.5_2" | "stragglers" | "round_straggler"
    times_seed: int = 0
    init: str = "he"                 # "he" | "small" | "gaussian"
    init_seed: int = 0
    rowptr: np.ndarray = field(default=None, repr=False)
    col: np.ndarray = field(default=None, repr=False)


def layer_dims(layers: List[int]) -> List[Tuple[int, int]]:
    """(out, in) of every dense layer."""
    return [(layers[l + 1], layers[l]) for l in range(len(layers) - 1)]


def logical_dim(layers: List[int]) -> int:
    return sum(o * i + o for o, i in layer_dims(layers))


CONFIGS = {
    0: dict(name="c0_ring8_softmax", N=8, graph="ring", layers=[784, 10], samples=600,
            noise=0.5, clip=True, means_seed=0, batch=32, rounds=20, backups="fixed", fixed_b=1,
            times_seed=1, init="small"),
    1: dict(name="c1_reg4_n32_mlp200", N=32, graph="regular", degree=4, graph_seed=2,
            layers=[784, 200, 10], samples=2000, noise=0.5, clip=True, means_seed=0, batch=64,
            rounds=200, backups="dtur", rate_mode="uniform_0.5_2"),
    2: dict(name="c2_er64_mlp512_256_bf16", N=64, graph="er", er_p=0.2, graph_seed=3,
            layers=[3072, 512, 256, 10], precision="bf16", samples=5000, noise=0.3, batch=128,
            rounds=100, backups="dtur", rate_mode="stragglers"),
    3: dict(name="c3_reg8_n128_mlp1024_bf16", N=128, graph="regular", degree=8,
            layers=[3072, 1024, 1024, 10], precision="bf16", samples=5000, noise=0.3, batch=256,
            rounds=50, backups="dtur", times="lognormal"),
    # Paper-shaped workloads (Section 5 and Appendix B): 6 workers with logistic regression, 10 workers
    # with the 256-256-10 network, batch 1024, learning rate eta_0 * 0.95^k, at least one straggler per
    # iteration.  The 256-dimensional Gaussian-mixture features stand in for the PCA-reduced images.
    5: dict(name="p0_lrm_6workers", N=6, graph="er", er_p=0.5, layers=[256, 10], samples=4096, noise=0.5,
            batch=1024, lr=0.2, lr_decay=0.95, rounds=60, backups="dtur", rate_mode="round_straggler", init="small"),
    6: dict(name="p1_2nn_10workers", N=10, graph="er", er_p=0.4, layers=[256, 256, 256, 10], samples=6000, noise=0.5,
            batch=1024, lr=1.0, lr_decay=0.95, rounds=60, backups="dtur", rate_mode="round_straggler"),
    4: dict(name="c4_reg32_n1024_mix", N=1024, graph="regular", degree=32, layers=None,
            d=1 << 20, rounds=10, backups="uniform", max_b=8, weight_rule="uniform",
            init="gaussian", init_seed=4),
    # Two more mix-only workloads beyond the five: the paper's own weight rule (Assumption 1) on the graph of
    # workload 4, and a worker count too large for any shared-memory panel of all rows.
    7: dict(name="m0_reg32_n1024_metropolis", N=1024, graph="regular", degree=32, graph_seed=5001, layers=None,
            d=1 << 20, rounds=10, backups="uniform", max_b=8, weight_rule="metropolis", init="gaussian"),
    8: dict(name="m1_reg8_n4096_metropolis", N=4096, graph="regular", degree=8, layers=None,
            d=1 << 16, rounds=10, backups="uniform", max_b=2, weight_rule="metropolis", init="gaussian"),
}


def make_workload(index: int, **overrides) -> Workload:
    """Descriptor of config `index` with its graph built.

    `overrides` may shrink a config for tests (e.g. N, d, samples, rounds);
    the graph is regenerated for the overridden N / degree.
    """
    spec = dict(CONFIGS[index])
    spec.update(overrides)
    w = Workload(index=index, **spec)
    if w.graph_seed == 0:
        w.graph_seed = _seed(index, "graph")
    if w.times_seed == 0:
        w.times_seed = _seed(index, "times")
    if w.init_seed == 0:
        w.init_seed = _seed(index, "init")
    if w.means_seed == 0 and index >= 2:
        w.means_seed = _seed(index, "data")
    if w.layers is not None:
        w.d = logical_dim(w.layers)
    if w.graph == "ring":
        w.rowptr, w.col = ring(w.N)
    elif w.graph == "regular":
        w.rowptr, w.col = random_regular(w.N, w.degree, w.graph_seed)
    elif w.graph == "er":
        w.rowptr, w.col = erdos_renyi_connected(w.N, w.er_p, w.graph_seed)
    else:
        raise ValueError(w.graph)
    return w


# --------------------------------------------------------------------------
# data, parameters, times, backups, batches
# --------------------------------------------------------------------------

def class_means(w: Workload) -> np.ndarray:
    """10 class means, each coordinate N(0,1); float32, shape (classes, in)."""
    rng = _rng(w.means_seed)
    return rng.standard_normal((w.layers[-1], w.layers[0])).astype(np.float32)


def worker_dataset(w: Workload, i: int, means: Optional[np.ndarray] = None):
    """Worker i's shard: features (samples, in) float32, labels (samples,) int32.

    feature = mean[label] + noise * N(0,1), clipped to [0,1] for the
    MNIST-shaped configs; labels uniform over the classes, or, with
    `label_skew` = k > 0, over the k classes (i*k + 0..k-1) mod classes only
    (non-iid shards: every worker sees its own D_j).
    """
    if means is None:
        means = class_means(w)
    rng = _rng(_seed(w.index, "data"), i)
    classes = w.layers[-1]
    if w.label_skew > 0:
        own = (i * w.label_skew + np.arange(w.label_skew)) % classes
        labels = own[rng.integers(0, w.label_skew, size=w.samples)].astype(np.int32)
    else:
        labels = rng.integers(0, classes, size=w.samples).astype(np.int32)
    feats = rng.standard_normal((w.samples, w.layers[0]), dtype=np.float32)
    feats *= np.float32(w.noise)
    feats += means[labels]
    if w.clip:
        np.clip(feats, 0.0, 1.0, out=feats)
    return feats, labels


def init_params(w: Workload, i: int) -> np.ndarray:
    """Worker i's initial logical parameter row (d,) float32.

    Layer order W1, b1, W2, b2, ...; W_l row-major [out][in].  "he": weights
    N(0, 2/in), biases 0.  "small": weights N(0, 0.01^2), biases 0.
    "gaussian" (mix-only): every entry N(0,1).
    """
    rng = _rng(w.init_seed, i)
    if w.init == "gaussian":
        return rng.standard_normal(w.d, dtype=np.float32)
    parts = []
    for out_f, in_f in layer_dims(w.layers):
        std = np.sqrt(2.0 / in_f) if w.init == "he" else 0.01
        parts.append((rng.standard_normal(out_f * in_f, dtype=np.float32) * np.float32(std)))
        parts.append(np.zeros(out_f, dtype=np.float32))
    return np.concatenate(parts)


def gaussian_rows(seed: int, rows, d: int, scale: float = 1.0, threads: int = 8) -> np.ndarray:
    """Rows `rows` of a (., d) float32 N(0, scale^2) matrix; row r depends on (seed, r) only."""
    rows = list(rows)
    out = np.empty((len(rows), d), dtype=np.float32)

    def fill(k):
        r = _rng(seed, rows[k])
        r.standard_normal(d, dtype=np.float32, out=out[k])
        if scale != 1.0:
            out[k] *= np.float32(scale)

    with ThreadPoolExecutor(max_workers=threads) as ex:
        list(ex.map(fill, range(len(rows))))
    return out


def external_gradient_seed(w: Workload) -> int:
    return _seed(w.index, "grads")


def worker_rates(w: Workload) -> np.ndarray:
    """Per-worker exponential rate of the compute-time distribution."""
    rng = _rng(_seed(w.index, "rates"))
    if w.rate_mode in ("one", "round_straggler"):
        return np.ones(w.N)
    if w.rate_mode == "uniform_0.5_2":
        return rng.uniform(0.5, 2.0, size=w.N)
    if w.rate_mode == "stragglers":
        rates = np.ones(w.N)
        n_slow = int(round(0.1 * w.N))
        rates[rng.choice(w.N, size=n_slow, replace=False)] = 0.2
        return rates
    raise ValueError(w.rate_mode)


def arrival_times(w: Workload, rounds: Optional[int] = None) -> np.ndarray:
    """Arrival (compute-finish) times, float64, shape (rounds, N)."""
    rounds = w.rounds if rounds is None else rounds
    rng = _rng(w.times_seed)
    if w.times == "shifted_exp":
        rates = worker_rates(w)
        t = w.shift + rng.exponential(1.0, size=(rounds, w.N)) / rates[None, :]
        if w.rate_mode == "round_straggler":     # every round one random worker takes five times as long
            slow = rng.integers(0, w.N, size=rounds)
            t[np.arange(rounds), slow] *= 5.0
        return t
    if w.times == "lognormal":
        return rng.lognormal(0.0, 1.0, size=(rounds, w.N))
    raise ValueError(w.times)


def learning_rate(w: Workload, k: int) -> float:
    """eta(k) of round k (0-based)."""
    return float(w.lr * w.lr_decay ** k)


def fixed_backups(w: Workload) -> np.ndarray:
    deg = np.diff(w.rowptr)
    return np.minimum(np.full(w.N, w.fixed_b, dtype=np.int32), deg).astype(np.int32)


def uniform_backups(w: Workload, rounds: Optional[int] = None) -> np.ndarray:
    """b_i i.i.d. uniform on {0..max_b} (capped at the degree), shape (rounds, N) int32."""
    rounds = w.rounds if rounds is None else rounds
    rng = _rng(_seed(w.index, "backups"))
    b = rng.integers(0, w.max_b + 1, size=(rounds, w.N)).astype(np.int32)
    return np.minimum(b, np.diff(w.rowptr)[None, :]).astype(np.int32)


def batch_indices(w: Workload, k: int) -> np.ndarray:
    """Mini-batch of round k: (N, batch) int32, uniform without replacement in each shard."""
    rng = _rng(_seed(w.index, "batches"), k)
    out = np.empty((w.N, w.batch), dtype=np.int32)
    for i in range(w.N):
        out[i] = rng.permutation(w.samples)[: w.batch]
    return out
