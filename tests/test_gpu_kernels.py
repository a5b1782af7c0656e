"""GPU parity, kernel by kernel, through the C ABI against the CPU oracle on the same seeded inputs.

Bars: kept masks, T_nbr / T_worker / T_round, b and theta are bit-exact (only comparisons touch
the times); parameters after the fp32 mix agree to 1e-5 per row (max-norm relative), which
leaves two orders of magnitude over the fp32 rounding of a <= 40-term weighted sum.
"""
import numpy as np
import pytest

from oracle import dbw_oracle as orc
from workloads import configs as wl

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")


def _dbw():
    import paper_2102_06280_b200 as p
    return p


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def row_rel_err(got, ref):
    got = np.asarray(got, dtype=np.float64)
    num = np.abs(got - ref).max(axis=1)
    den = np.maximum(np.abs(ref).max(axis=1), 1e-30)
    return float((num / den).max())


GRAPHS = {
    "ring8": lambda: wl.ring(8),
    "path2": lambda: wl.path(2),
    "complete40": lambda: wl.complete(40),          # degree 39 > one warp
    "complete70": lambda: wl.complete(70),          # degree 69: three 32-neighbour chunks
    "reg4_32": lambda: wl.random_regular(32, 4, 2),
    "er64": lambda: wl.erdos_renyi_connected(64, 0.2, 3),
    "reg32_256": lambda: wl.random_regular(256, 32, 11),
    "star_like": lambda: wl._csr_from_edges(6, [(0, 1), (0, 2), (0, 3), (0, 4), (0, 5)]),  # degree-1 leaves
}


def _select_gpu(h, n, nnz, t, b):
    kept = torch.zeros(nnz, dtype=torch.uint8, device="cuda")
    Tw = torch.zeros(n, dtype=torch.float64, device="cuda")
    Tn = torch.zeros(n, dtype=torch.float64, device="cuda")
    Tr = torch.zeros(1, dtype=torch.float64, device="cuda")
    h.select(dev(t), dev(b.astype(np.int32)), kept, Tw, Tn, Tr)
    torch.cuda.synchronize()
    return kept.cpu().numpy(), Tw.cpu().numpy(), Tn.cpu().numpy(), float(Tr.cpu()[0])


@pytest.mark.parametrize("name", list(GRAPHS))
def test_selection_bit_exact(name):
    p = _dbw()
    rowptr, col = GRAPHS[name]()
    n = len(rowptr) - 1
    deg = np.diff(rowptr)
    h = p.Dbw(rowptr, col, d=4)
    rng = np.random.default_rng(5)
    cases = []
    for trial in range(6):
        t = 1.0 + rng.exponential(1.0, size=n)
        if trial % 2:                                  # engineered ties
            t = np.round(t * 2) / 2
        cases.append((t, rng.integers(0, deg + 1)))
    cases.append((1.0 + rng.exponential(1.0, size=n), np.zeros(n, dtype=np.int64)))   # b = 0
    cases.append((1.0 + rng.exponential(1.0, size=n), deg.copy()))                     # b = deg
    cases.append((np.ones(n), rng.integers(0, deg + 1)))                               # all times equal
    for t, b in cases:
        kept, Tw, Tn, Tr = _select_gpu(h, n, len(col), t, b)
        ref = orc.select_fastest(rowptr, col, t, b)
        assert np.array_equal(kept, ref)
        rTn, rTw, rTr = orc.round_times(rowptr, col, t, b, ref)
        assert np.array_equal(Tn, rTn) and np.array_equal(Tw, rTw) and Tr == rTr
    assert h.status() == 0
    h.close()


def test_selection_flags_bad_inputs():
    p = _dbw()
    rowptr, col = wl.ring(8)
    h = p.Dbw(rowptr, col, d=4)
    t = np.arange(8, dtype=np.float64)
    b = np.array([0, 5, 0, -2, 0, 0, 0, 0])
    kept, *_ = _select_gpu(h, 8, len(col), t, b)
    assert h.status() & p.STATUS_BAD_B
    ref = orc.select_fastest(rowptr, col, t, np.clip(b, 0, 2))      # clamped, not trapped
    assert np.array_equal(kept, ref)
    t[3] = np.nan
    kept, *_ = _select_gpu(h, 8, len(col), t, np.ones(8, dtype=np.int64))
    assert h.status() & p.STATUS_NAN_TIME
    t[3] = np.inf                                                    # NaN is ordered last
    assert np.array_equal(kept, orc.select_fastest(rowptr, col, t, np.ones(8, dtype=np.int64)))
    assert h.status() == 0
    h.close()


@pytest.mark.parametrize("name,d", [("ring8", 7850), ("reg4_32", 1000), ("er64", 4100), ("complete40", 260),
                                     ("reg32_256", 3000)])
@pytest.mark.parametrize("rule", ["metropolis", "uniform"])
@pytest.mark.parametrize("order", ["local_then_mix", "mix_then_correct"])
def test_mix_matches_oracle(name, d, rule, order):
    p = _dbw()
    rowptr, col = GRAPHS[name]()
    n = len(rowptr) - 1
    deg = np.diff(rowptr)
    ld = (d + 3) // 4 * 4
    flags = (p.WEIGHT_UNIFORM if rule == "uniform" else 0) | (p.ORDER_MIX_THEN_CORRECT if order == "mix_then_correct" else 0)
    h = p.Dbw(rowptr, col, d=d, ld=ld, flags=flags)
    rng = np.random.default_rng(8)
    X = np.zeros((n, ld), dtype=np.float32)
    G = np.zeros((n, ld), dtype=np.float32)
    X[:, :d] = rng.standard_normal((n, d), dtype=np.float32)
    G[:, :d] = rng.standard_normal((n, d), dtype=np.float32)
    t = 1.0 + rng.exponential(1.0, size=n)
    b = rng.integers(0, deg + 1)
    b[0] = deg[0]                                         # one worker waits for nobody
    kept = orc.select_fastest(rowptr, col, t, b)
    ws, we = orc.mixing_weights(rowptr, col, b, kept, rule)
    ref = orc.mix_update(rowptr, col, X, G, ws, we, 0.05, order)
    Xd, Gd, kd, bd = dev(X), dev(G), dev(kept), dev(b.astype(np.int32))
    for panel in (0, 1, 2, 16, 32, 64, 128, 256, -1):
        h.set_mix_panel(panel)
        out = torch.full_like(Xd, float("nan"))
        h.mix(Xd, Gd, kd, bd, 0.05, out)
        torch.cuda.synchronize()
        got = out.cpu().numpy()
        assert row_rel_err(got, ref) <= 1e-5, panel
        assert not np.any(got[:, d:])                      # padding stays zero
        if panel != -1 and h.mix_in_place_ok():
            inpl = Xd.clone()
            h.mix(inpl, Gd, kd, bd, 0.05, inpl)
            torch.cuda.synchronize()
            assert np.array_equal(inpl.cpu().numpy(), got)  # in place == out of place, bit for bit
    # per-worker learning rates (eta_j of Eq. 4)
    lrw = (0.01 + 0.1 * rng.random(n)).astype(np.float32)
    h.set_mix_panel(0)
    out = torch.empty_like(Xd)
    h.mix(Xd, Gd, kd, bd, 0.0, out, lr_per_worker=dev(lrw))
    torch.cuda.synchronize()
    ref = orc.mix_update(rowptr, col, X, G, ws, we, lrw.astype(np.float64), order)
    assert row_rel_err(out.cpu().numpy(), ref) <= 1e-5
    assert h.status() == 0
    h.close()


@pytest.mark.parametrize("n,deg,d,order", [(320, 16, 1000, "local_then_mix"), (700, 16, 1300, "mix_then_correct"),
                                           (1000, 32, 2052, "local_then_mix"), (512, 8, 516, "local_then_mix"),
                                           (514, 8, 260, "mix_then_correct")])
@pytest.mark.parametrize("panel,kernel", [(2, "mix_tc_kernel"), (3, "mix_sp_kernel")])
def test_mix_tensor_core_kernel_matches_oracle(n, deg, d, order, panel, kernel):
    """The 0/1-selection product on the tensor cores (three exact BF16 pieces per fp32 value), dense and with the
    selection matrix 2:4 structured-sparse in the graph's worker order: worker counts that leave ragged row tiles
    and K chunks, widths that leave a ragged last panel, both update orders, per-worker learning rates, in place
    where one CTA pair owns a panel, run-to-run reproducible."""
    p = _dbw()
    rowptr, col = wl.random_regular(n, deg, 21)
    degs = np.diff(rowptr)
    flags = p.WEIGHT_UNIFORM | (p.ORDER_MIX_THEN_CORRECT if order == "mix_then_correct" else 0)
    h = p.Dbw(rowptr, col, d=d, ld=d, flags=flags)
    h.set_mix_panel(panel)
    assert h.mix_kernel() == kernel
    assert h.mix_in_place_ok() == (n <= 512)
    rng = np.random.default_rng(12)
    X = rng.standard_normal((n, d), dtype=np.float32) * np.float32(3.0)
    X[:, ::7] *= np.float32(1e-4)                          # small and large magnitudes side by side
    G = rng.standard_normal((n, d), dtype=np.float32)
    t = 1.0 + rng.exponential(1.0, size=n)
    b = rng.integers(0, np.minimum(degs, 8) + 1)
    b[0] = degs[0]
    kept = orc.select_fastest(rowptr, col, t, b)
    ws, we = orc.mixing_weights(rowptr, col, b, kept, "uniform")
    lrw = (0.01 + 0.1 * rng.random(n)).astype(np.float32)
    Xd, Gd, kd, bd = dev(X), dev(G), dev(kept), dev(b.astype(np.int32))
    for lr, lr_pw in ((0.05, None), (0.0, lrw)):
        ref = orc.mix_update(rowptr, col, X, G, ws, we, lr if lr_pw is None else lr_pw.astype(np.float64), order)
        out = torch.full_like(Xd, float("nan"))
        h.mix(Xd, Gd, kd, bd, lr, out, lr_per_worker=None if lr_pw is None else dev(lr_pw))
        torch.cuda.synchronize()
        got = out.cpu().numpy()
        assert row_rel_err(got, ref) <= 1e-5
        for _ in range(3):                                   # reproducible: staging buffers are reused between stores
            again = torch.zeros_like(Xd)
            h.mix(Xd, Gd, kd, bd, lr, again, lr_per_worker=None if lr_pw is None else dev(lr_pw))
            torch.cuda.synchronize()
            assert np.array_equal(again.cpu().numpy(), got)
        if h.mix_in_place_ok():
            inpl = Xd.clone()
            h.mix(inpl, Gd, kd, bd, lr, inpl, lr_per_worker=None if lr_pw is None else dev(lr_pw))
            torch.cuda.synchronize()
            assert np.array_equal(inpl.cpu().numpy(), got)
        else:
            with pytest.raises(p.DbwError):
                h.mix(Xd, Gd, kd, bd, lr, Xd)
    assert h.status() == 0
    h.close()


@pytest.mark.parametrize("order", ["local_then_mix", "mix_then_correct"])
def test_mix_staged_kernel_with_metropolis_weights(order):
    """The paper's weight rule (Assumption 1) on a graph with many kept neighbours per worker: the persistent
    tensor-memory staged kernel is selected by itself, carries the weights as 6-bit codes in its neighbour lists,
    and adds in the same order as the shared-memory panel kernel: same bits, same bar against the oracle."""
    p = _dbw()
    n, deg, d = 1000, 32, 2052
    rowptr, col = wl.random_regular(n, deg, 7)
    degs = np.diff(rowptr)
    h = p.Dbw(rowptr, col, d=d, ld=d, flags=p.ORDER_MIX_THEN_CORRECT if order == "mix_then_correct" else 0)
    assert h.mix_kernel() == "mix_staged_kernel" and h.mix_in_place_ok()
    rng = np.random.default_rng(2)
    X = rng.standard_normal((n, d), dtype=np.float32)
    G = rng.standard_normal((n, d), dtype=np.float32)
    t = 1.0 + rng.exponential(1.0, size=n)
    b = rng.integers(0, np.minimum(degs, 9) + 1)
    b[0], b[1] = degs[0], 0
    kept = orc.select_fastest(rowptr, col, t, b)
    ws, we = orc.mixing_weights(rowptr, col, b, kept, "metropolis")
    ref = orc.mix_update(rowptr, col, X, G, ws, we, 0.05, order)
    Xd, Gd, kd, bd = dev(X), dev(G), dev(kept), dev(b.astype(np.int32))
    res = {}
    for panel in (0, 16):
        h.set_mix_panel(panel)
        out = torch.full_like(Xd, float("nan"))
        h.mix(Xd, Gd, kd, bd, 0.05, out)
        torch.cuda.synchronize()
        res[panel] = out.cpu().numpy()
        assert row_rel_err(res[panel], ref) <= 1e-5, panel
    assert h.mix_kernel() == "mix_panel_kernel"
    assert np.array_equal(res[0], res[16])
    h.set_mix_panel(0)
    inpl = Xd.clone()
    h.mix(inpl, Gd, kd, bd, 0.05, inpl)
    torch.cuda.synchronize()
    assert np.array_equal(inpl.cpu().numpy(), res[0])
    assert h.status() == 0
    h.close()


def test_mix_large_worker_count_uses_the_l2_kernel():
    """More workers than a shared-memory panel of even 16 columns can hold: neighbour rows are re-read through L2
    (row-fastest work order inside column panels), out of place only, same bar."""
    p = _dbw()
    n, d = 4200, 1100
    rowptr, col = wl.random_regular(n, 4, 5)
    deg = np.diff(rowptr)
    for rule, order in (("metropolis", "local_then_mix"), ("uniform", "mix_then_correct")):
        flags = (p.WEIGHT_UNIFORM if rule == "uniform" else 0) | (p.ORDER_MIX_THEN_CORRECT if order == "mix_then_correct" else 0)
        h = p.Dbw(rowptr, col, d=d, ld=d, flags=flags)
        assert h.mix_kernel() == "mix_direct_kernel" and not h.mix_in_place_ok()
        rng = np.random.default_rng(3)
        X = rng.standard_normal((n, d), dtype=np.float32)
        G = rng.standard_normal((n, d), dtype=np.float32)
        t = 1.0 + rng.exponential(1.0, size=n)
        b = rng.integers(0, deg + 1)
        kept = orc.select_fastest(rowptr, col, t, b)
        ws, we = orc.mixing_weights(rowptr, col, b, kept, rule)
        ref = orc.mix_update(rowptr, col, X, G, ws, we, 0.05, order)
        Xd = dev(X)
        out = torch.full_like(Xd, float("nan"))
        h.mix(Xd, dev(G), dev(kept), dev(b.astype(np.int32)), 0.05, out)
        torch.cuda.synchronize()
        assert row_rel_err(out.cpu().numpy(), ref) <= 1e-5
        with pytest.raises(p.DbwError):
            h.mix(Xd, dev(G), dev(kept), dev(b.astype(np.int32)), 0.05, Xd)
        assert h.status() == 0
        h.close()


def test_mix_rejects_bad_aliasing():
    p = _dbw()
    rowptr, col = wl.ring(8)
    h = p.Dbw(rowptr, col, d=64)
    X = torch.zeros(8 * 64 + 64, device="cuda")
    G = torch.zeros(8 * 64, device="cuda")
    kept = torch.ones(16, dtype=torch.uint8, device="cuda")
    b = torch.zeros(8, dtype=torch.int32, device="cuda")
    with pytest.raises(p.DbwError):
        h.mix(X[:512], G, kept, b, 0.1, X[32:544])          # partial overlap
    with pytest.raises(p.DbwError):
        h.mix(X[:512], G, kept, b, 0.1, G)                  # output over the gradients
    h.set_mix_panel(-1)
    with pytest.raises(p.DbwError):
        h.mix(X[:512], G, kept, b, 0.1, X[:512])            # direct kernel cannot run in place
    h.close()


@pytest.mark.parametrize("name", ["ring8", "reg4_32", "er64", "complete40"])
def test_update_backups_bit_exact_and_resume(name):
    p = _dbw()
    rowptr, col = GRAPHS[name]()
    n = len(rowptr) - 1
    h = p.Dbw(rowptr, col, d=4)
    assert np.array_equal(h.links(), np.array(orc.spanning_links(rowptr, col)))
    ref = orc.Dtur(rowptr, col)
    rng = np.random.default_rng(3)
    b_d = torch.zeros(n, dtype=torch.int32, device="cuda")
    th_d = torch.zeros(1, dtype=torch.float64, device="cuda")
    rounds = 2 * (n - 1) + 3
    times = 1.0 + rng.exponential(1.0, size=(rounds, n))
    times[1] = np.round(times[1])                            # ties between links
    blob = None
    for k in range(rounds):
        if k == n // 2:
            blob = h.state_export()
            saved = (list(ref.covered), ref.step)
        h.update_backups(dev(times[k]), b_d, th_d)
        torch.cuda.synchronize()
        rb, rtheta = ref.update_backups(times[k])
        assert np.array_equal(b_d.cpu().numpy(), rb) and float(th_d.cpu()[0]) == rtheta
    # resume from the saved state reproduces the same sequence
    h.state_import(blob)
    ref.covered, ref.step = saved
    for k in range(n // 2, n // 2 + 5):
        h.update_backups(dev(times[k]), b_d, th_d)
        rb, rtheta = ref.update_backups(times[k])
        assert np.array_equal(b_d.cpu().numpy(), rb) and float(th_d.cpu()[0]) == rtheta
    h.reset_backups()
    fresh = orc.Dtur(rowptr, col)
    h.update_backups(dev(times[0]), b_d, th_d)
    assert np.array_equal(b_d.cpu().numpy(), fresh.update_backups(times[0])[0])
    with pytest.raises(p.DbwError):
        h.state_import(blob[:-4])
    h.close()


@pytest.mark.parametrize("dims,batch,n", [([784, 10], 32, 8), ([20, 13, 7], 5, 3), ([100, 70, 33, 10], 19, 4),
                                           ([784, 200, 10], 64, 6),
                                           ([64, 48, 24], 12, 3),     # 24 classes: the 32-class instance of the last-layer kernels
                                           ([256, 128], 40, 3),       # one layer of more than 32 classes: GEMM + loss kernel
                                           ([8, 5, 8, 4], 6, 3),      # last layer's weights not 16-byte aligned in the row: GEMM path
                                           ([128, 64, 64, 12], 256, 5)])  # whole tiles of the 128-bit GEMM, 8 x 4 outputs per thread
def test_grad_fp32_matches_oracle(dims, batch, n):
    p = _dbw()
    rowptr, col = wl.ring(max(n, 3)) if n >= 3 else wl.path(n)
    n = len(rowptr) - 1
    m = p.model_layout(dims, batch)
    h = p.Dbw(rowptr, col, d=m.d, model=m)
    rng = np.random.default_rng(0)
    S = 3 * batch
    feat = rng.random((n, S, dims[0]), dtype=np.float32)
    labels = rng.integers(0, dims[-1], size=(n, S)).astype(np.int32)
    Xl = (rng.standard_normal((n, m.d)) * 0.2).astype(np.float32)
    idx = np.stack([rng.permutation(S)[:batch] for _ in range(n)]).astype(np.int32)
    h.set_dataset(dev(feat), dev(labels), S)
    G = torch.zeros(n, m.ld, device="cuda")
    loss = torch.zeros(n, device="cuda")
    h.grad(dev(m.pack(Xl)), dev(idx), G, loss)
    torch.cuda.synchronize()
    got = m.unpack(G.cpu().numpy())
    for i in range(n):
        g, l = orc.mlp_grad(Xl[i], dims, feat[i][idx[i]], labels[i][idx[i]])
        assert np.abs(got[i] - g).max() <= 1e-5 * max(np.abs(g).max(), 1e-30)
        assert abs(float(loss[i]) - l) <= 1e-5 * max(abs(l), 1.0)
    Gp = G.cpu().numpy()
    assert np.count_nonzero(Gp) == np.count_nonzero(got)      # padding untouched
    assert h.status() == 0
    h.close()


@pytest.mark.parametrize("dims,batch,n", [([256, 128, 128, 10], 128, 3),      # whole tiles
                                           ([3072, 512, 256, 10], 128, 2),     # config 2's model
                                           ([72, 200, 136, 10], 40, 3),        # ragged M, N and K tails
                                           ([320, 264, 24], 264, 2),           # two layers, three row tiles
                                           ([256, 256, 256, 10], 1024, 2),     # the paper's 2NN, batch 1024: 16 K-blocks in dW
                                           ([64, 10], 16, 3)])                 # softmax regression: no tensor-core layer
def test_grad_bf16_tensor_cores_match_oracle(dims, batch, n):
    """BF16 operands, fp32 accumulate.  Two references side by side:
    (1) tests/bf16_reference.py: the same gradient in double on operands rounded to bf16 at the points where
        the CUDA path rounds them.  Per layer block: every entry within 5e-3 of the block's max-norm and the
        block's 2-norm error within 1e-3 (measured on these shapes: at most 5e-4 and 4.5e-4); ReLU decisions on
        pre-activations that fp32 accumulation cannot tell from zero are inferred from the GPU's own output
        (see gradient_agrees).  A dropped K block, a wrong bias gradient scale or a wrong ReLU mask on a few
        percent of the entries is orders of magnitude above these bars.
    (2) the double-precision oracle on the fp32 master weights: bf16 rounding (2^-8 per operand, three chained
        GEMM stages for the first layer's dW, ReLU masks that flip where a pre-activation is within rounding
        of zero) is what separates them: 0.15 of each block's max-norm and a cosine above 0.995."""
    from bf16_reference import gradient_agrees
    p = _dbw()
    rowptr, col = wl.ring(n) if n >= 3 else wl.path(n)
    m = p.model_layout(dims, batch)
    h = p.Dbw(rowptr, col, d=m.d, model=m, flags=p.GEMM_BF16)
    rng = np.random.default_rng(1)
    S = 2 * batch
    feat = rng.random((n, S, dims[0]), dtype=np.float32)
    labels = rng.integers(0, dims[-1], size=(n, S)).astype(np.int32)
    parts = []
    for l in range(len(dims) - 1):
        parts.append(rng.standard_normal((n, dims[l] * dims[l + 1])) * np.sqrt(2.0 / dims[l]))
        parts.append(rng.standard_normal((n, dims[l + 1])) * 0.1)
    Xl = np.concatenate(parts, axis=1).astype(np.float32)
    idx = np.stack([rng.permutation(S)[:batch] for _ in range(n)]).astype(np.int32)
    h.set_dataset(dev(feat), dev(labels), S)
    G = torch.zeros(n, m.ld, device="cuda")
    loss = torch.zeros(n, device="cuda")
    Xd = dev(m.pack(Xl))
    for rep in range(2):                                   # second call reuses the rings and tensor memory
        G.zero_()
        h.grad(Xd, dev(idx), G, loss)
        torch.cuda.synchronize()
    got = m.unpack(G.cpu().numpy())
    assert h.status() == 0
    worst = 0.0
    for i in range(n):
        g, l = orc.mlp_grad(Xl[i], dims, feat[i][idx[i]], labels[i][idx[i]])
        # (a ReLU decision on a pre-activation that fp32 accumulation cannot tell from zero may go either way:
        # see gradient_agrees for how those are treated)
        ok, rep = gradient_agrees(got[i].astype(np.float64), Xl[i], dims, feat[i][idx[i]], labels[i][idx[i]])
        worst = max(worst, rep["l2"])
        assert ok, (i, rep)
        le = rep["loss"]
        off = 0
        for lay in range(len(dims) - 1):
            for size in (dims[lay] * dims[lay + 1], dims[lay + 1]):
                a, r = got[i, off:off + size], g[off:off + size]
                assert np.abs(a - r).max() <= 0.15 * np.abs(r).max() + 1e-7, (i, lay, size)
                off += size
        cos = float(got[i] @ g / (np.linalg.norm(got[i]) * np.linalg.norm(g)))
        assert cos > 0.995, cos
        assert abs(float(loss[i]) - le) <= 1e-4 * max(abs(le), 1.0)
        assert abs(float(loss[i]) - l) <= 2e-2 * max(abs(l), 1.0)
    print("bf16 gradient vs bf16-point reference: worst block 2-norm error %.2e" % worst)
    assert np.count_nonzero(G.cpu().numpy()) <= m.d * n     # padding untouched
    h.close()


@pytest.mark.parametrize("flag", [0, 4])
def test_label_out_of_range_is_clamped_and_reported(flag):
    """A label outside [0, classes) must not become an out-of-bounds read: it is clamped, the status word
    says so, and the loss stays finite."""
    p = _dbw()
    rowptr, col = wl.ring(3)
    dims, batch = [64, 32, 10], 16
    m = p.model_layout(dims, batch)
    h = p.Dbw(rowptr, col, d=m.d, model=m, flags=flag)
    rng = np.random.default_rng(2)
    S = 32
    feat = rng.random((3, S, dims[0]), dtype=np.float32)
    labels = rng.integers(0, 10, size=(3, S)).astype(np.int32)
    labels[1, 5] = 1 << 30
    labels[2, 7] = -3
    idx = np.stack([np.arange(batch) for _ in range(3)]).astype(np.int32)
    Xl = (rng.standard_normal((3, m.d)) * 0.1).astype(np.float32)
    h.set_dataset(dev(feat), dev(labels), S)
    G = torch.zeros(3, m.ld, device="cuda")
    loss = torch.zeros(3, device="cuda")
    h.grad(dev(m.pack(Xl)), dev(idx), G, loss)
    torch.cuda.synchronize()
    assert h.status() & p.STATUS_BAD_INDEX
    assert torch.isfinite(loss).all() and torch.isfinite(G).all()
    # the clamped labels are what the gradient was computed with
    fixed = np.clip(labels, 0, 9)
    got = m.unpack(G.cpu().numpy())
    for i in range(3):
        g, _ = orc.mlp_grad(Xl[i], dims, feat[i][idx[i]], fixed[i][idx[i]])
        tol = 1e-5 if flag == 0 else 0.15
        assert np.abs(got[i] - g).max() <= tol * np.abs(g).max()
    h.close()


def test_expired_pipeline_wait_is_reported_and_drains():
    """The bounded wait every tensor-core pipeline uses: a barrier that nothing completes makes the wait give
    up after its poll limit, sets DBW_STATUS_WAIT_TIMEOUT, and every later wait of the thread block returns
    at once instead of spinning its own limit; the context stays usable."""
    import time
    p = _dbw()
    rowptr, col = wl.ring(4)
    h = p.Dbw(rowptr, col, d=4)
    out = torch.zeros(3, dtype=torch.int32, device="cuda")
    torch.cuda.synchronize()
    t0 = time.time()
    h.debug_wait_probe(2000, out)
    torch.cuda.synchronize()
    took = time.time() - t0
    o = out.cpu().numpy()
    assert o[0] == 1 and o[1] == 1
    assert o[2] < 20000                       # the second wait did not poll: a few hundred clocks
    assert took < 5.0
    assert h.status() & p.STATUS_WAIT_TIMEOUT
    assert h.status() == 0                    # cleared by the read; the context still works
    kept, *_ = _select_gpu(h, 4, len(col), np.arange(4.0), np.zeros(4, dtype=np.int64))
    assert kept.all()
    h.close()


@pytest.mark.parametrize("rule", ["uniform", "metropolis"])
def test_mix_with_a_mask_that_disagrees_with_b(rule):
    """dbw_mix on its own takes kept and b from the caller.  With uniform weights the weight is
    1 / (1 + entries set in the row), so rows stay stochastic whatever b says; the mismatch is reported."""
    p = _dbw()
    rowptr, col = GRAPHS["reg4_32"]()
    n, d = 32, 64
    h = p.Dbw(rowptr, col, d=d, flags=p.WEIGHT_UNIFORM if rule == "uniform" else 0)
    rng = np.random.default_rng(3)
    X = rng.standard_normal((n, d)).astype(np.float32)
    G = rng.standard_normal((n, d)).astype(np.float32)
    b = np.ones(n, dtype=np.int32)
    kept = orc.select_fastest(rowptr, col, 1.0 + rng.random(n), b)
    kept2 = kept.copy()
    e0 = int(rowptr[5])
    kept2[e0: e0 + 4] = [1, 0, 0, 0]          # worker 5 keeps one neighbour although b says three
    out = torch.empty(n, d, device="cuda")
    h.mix(dev(X), dev(G), dev(kept2), dev(b), 0.1, out)
    torch.cuda.synchronize()
    assert h.status() & p.STATUS_BAD_B
    got = out.cpu().numpy().astype(np.float64)
    if rule == "uniform":
        b_eff = b.copy()
        b_eff[5] = 3                          # the weights follow the mask
        ws, we = orc.mixing_weights(rowptr, col, b_eff, kept2, orc.UNIFORM)
        assert row_rel_err(got, orc.mix_update(rowptr, col, X, G, ws, we, 0.1)) <= 1e-5
    else:                                     # Assumption 1 on the nominal counts; w_ii = 1 - sum keeps the row stochastic
        ws, we = orc.mixing_weights(rowptr, col, b, kept2, orc.METROPOLIS)
        assert abs(ws[5] + we[e0: e0 + 4].sum() - 1.0) < 1e-12
        assert row_rel_err(got, orc.mix_update(rowptr, col, X, G, ws, we, 0.1)) <= 1e-5
    h.close()


@pytest.mark.parametrize("kernel,graph,panel", [("mix_panel_kernel", "reg4_32", 0), ("mix_staged_kernel", "reg32_256", 1),
                                                ("mix_direct_kernel", "reg4_32", -1), ("mix_tc_kernel", "reg32_256", 2),
                                                ("mix_sp_kernel", "reg32_256", 3)])
@pytest.mark.parametrize("order", ["local_then_mix", "mix_then_correct"])
def test_consensus_only_mix_reads_no_gradient(kernel, graph, panel, order):
    """G == NULL (Section 3.2.1's truncated model: gradients zero after K) gives the bits of a mix with an
    all-zero gradient matrix, in every mix kernel and both update orders."""
    p = _dbw()
    rowptr, col = GRAPHS[graph]()
    n, d = len(rowptr) - 1, 1000
    deg = np.diff(rowptr)
    flags = p.WEIGHT_UNIFORM | (p.ORDER_MIX_THEN_CORRECT if order == "mix_then_correct" else 0)
    h = p.Dbw(rowptr, col, d=d, flags=flags)
    h.set_mix_panel(panel)
    assert h.mix_kernel() == kernel
    rng = np.random.default_rng(4)
    X = dev(rng.standard_normal((n, d)).astype(np.float32))
    t = dev(1.0 + rng.random(n))
    b = dev(rng.integers(0, deg // 2 + 1).astype(np.int32))
    kept = torch.zeros(len(col), dtype=torch.uint8, device="cuda")
    out0, out1 = torch.empty_like(X), torch.empty_like(X)
    h.round(X, t, b, 0.1, out0, kept, G_ext=torch.zeros_like(X))
    h.round(X, t, b, 0.1, out1, kept)                         # neither batches nor gradients: G = 0
    torch.cuda.synchronize()
    assert torch.equal(out0, out1)
    out2 = torch.empty_like(X)
    h.mix(X, None, kept, b, 0.1, out2)
    torch.cuda.synchronize()
    assert torch.equal(out0, out2)
    assert h.status() == 0
    h.close()


def test_consensus_only_rounds_converge_to_the_initial_mean():
    """Corollary 1 / the truncated model of Section 3.2.1 with G = 0 and b = 0 (Metropolis weights doubly
    stochastic): every round agrees with the oracle to 1e-5 (teacher-forced from the GPU's own fp32 state),
    the network mean is preserved and the rows contract geometrically onto it."""
    p = _dbw()
    rowptr, col = GRAPHS["reg4_32"]()
    n, d = 32, 1536
    h = p.Dbw(rowptr, col, d=d)
    rng = np.random.default_rng(6)
    X0 = rng.standard_normal((n, d)).astype(np.float32)
    mean0 = X0.astype(np.float64).mean(axis=0)
    X = dev(X0)
    b = np.zeros(n, dtype=np.int32)
    kept = torch.zeros(len(col), dtype=torch.uint8, device="cuda")
    spread = []
    X_orc = X0.astype(np.float64)
    rounds = 120
    for k in range(rounds):
        t = 1.0 + rng.random(n)
        before = X.cpu().numpy()
        h.round(X, dev(t), dev(b), 0.05, X, kept)             # in place, no gradients
        torch.cuda.synchronize()
        r = orc.dbw_round(rowptr, col, before, t, b, 0.05, G=np.zeros((n, d)))
        assert row_rel_err(X.cpu().numpy(), r["X"]) <= 1e-5, k
        X_orc = orc.dbw_round(rowptr, col, X_orc, t, b, 0.05, G=np.zeros((n, d)))["X"]
        spread.append(float(np.abs(X.cpu().numpy().astype(np.float64) - mean0).max()))
    got = X.cpu().numpy().astype(np.float64)
    assert np.abs(got.mean(axis=0) - mean0).max() <= 1e-5     # mean preserved (fp32 rounding only)
    assert spread[59] < 1e-2 * spread[0] and spread[-1] < 1e-4 * spread[0]
    rate = (spread[59] / spread[9]) ** (1.0 / 50)
    assert rate < 0.95                                        # geometric contraction
    assert np.abs(got - X_orc).max() <= 1e-5
    assert h.status() == 0
    h.close()


def test_degenerate_sizes():
    """One worker (no links), two workers, and a padded leading dimension far above d."""
    p = _dbw()
    # N = 1: no neighbours, the round is a plain SGD step and lasts t_0
    rowptr, col = np.array([0, 0], dtype=np.int32), np.zeros(0, dtype=np.int32)
    h = p.Dbw(rowptr, col, d=10, ld=12)
    X = torch.arange(12, dtype=torch.float32, device="cuda").reshape(1, 12)
    G = torch.ones(1, 12, device="cuda")
    kept = torch.zeros(1, dtype=torch.uint8, device="cuda")
    Tw = torch.zeros(1, dtype=torch.float64, device="cuda")
    Tr = torch.zeros(1, dtype=torch.float64, device="cuda")
    out = torch.empty_like(X)
    t, b = dev(np.array([2.5])), dev(np.zeros(1, dtype=np.int32))
    h.round(X, t, b, 0.5, out, kept, G_ext=G, T_worker=Tw, T_round=Tr)
    torch.cuda.synchronize()
    assert torch.equal(out, X - 0.5 * G)
    assert float(Tw[0]) == 0.0 and float(Tr[0]) == 0.0         # nobody waits for anybody: no participant
    bo = torch.full((1,), 7, dtype=torch.int32, device="cuda")
    th = torch.zeros(1, dtype=torch.float64, device="cuda")
    h.update_backups(t, bo, th)                                   # no links: threshold +inf, b = deg = 0
    torch.cuda.synchronize()
    assert int(bo[0]) == 0 and np.isinf(float(th[0]))
    assert h.status() == 0
    h.close()
    # N = 2, ld much larger than d (the tail is padding and must stay zero)
    rowptr, col = wl.path(2)
    d, ld = 6, 512
    h = p.Dbw(rowptr, col, d=d, ld=ld)
    rng = np.random.default_rng(0)
    Xh = np.zeros((2, ld), dtype=np.float32); Gh = np.zeros((2, ld), dtype=np.float32)
    Xh[:, :d] = rng.standard_normal((2, d)); Gh[:, :d] = rng.standard_normal((2, d))
    Xd = dev(Xh)
    kept = torch.zeros(2, dtype=torch.uint8, device="cuda")
    tt, bb = np.array([1.0, 1.0]), np.zeros(2, dtype=np.int32)
    h.round(Xd, dev(tt), dev(bb), 0.1, Xd, kept, G_ext=dev(Gh))
    torch.cuda.synchronize()
    r = orc.dbw_round(rowptr, col, Xh, tt, bb, 0.1, G=Gh)
    assert row_rel_err(Xd.cpu().numpy()[:, :d], r["X"][:, :d]) <= 1e-5
    assert not np.any(Xd.cpu().numpy()[:, d:])
    assert np.array_equal(kept.cpu().numpy(), r["kept"])
    h.close()


@pytest.mark.parametrize("name", ["ring8", "complete40", "reg4_32", "er64", "reg32_256"])
def test_selection_with_per_link_times_bit_exact(name):
    p = _dbw()
    rowptr, col = GRAPHS[name]()
    n, nnz = len(rowptr) - 1, len(col)
    deg = np.diff(rowptr)
    h = p.Dbw(rowptr, col, d=8)
    rng = np.random.default_rng(31)
    X = rng.standard_normal((n, 8)).astype(np.float32)
    G = rng.standard_normal((n, 8)).astype(np.float32)
    for trial in range(4):
        t = 1.0 + rng.exponential(1.0, size=n)
        te = np.round(4 * (t[col] + rng.random(nnz))) / 4                 # link delays, with ties
        b = rng.integers(0, deg + 1)
        h.set_edge_times(dev(te))
        kept, Tw, Tn, Tr = _select_gpu(h, n, nnz, t, b)
        ref = orc.select_fastest(rowptr, col, t, b, t_edge=te)
        assert np.array_equal(kept, ref)
        rTn, rTw, rTr = orc.round_times(rowptr, col, t, b, ref, t_edge=te)
        assert np.array_equal(Tn, rTn) and np.array_equal(Tw, rTw) and Tr == rTr
        # the whole round follows the link-time selection
        out = torch.empty(n, 8, device="cuda")
        kd = torch.zeros(nnz, dtype=torch.uint8, device="cuda")
        h.round(dev(X), dev(t), dev(b.astype(np.int32)), 0.1, out, kd, G_ext=dev(G))
        torch.cuda.synchronize()
        ws, we = orc.mixing_weights(rowptr, col, b, ref)
        assert np.array_equal(kd.cpu().numpy(), ref)
        assert row_rel_err(out.cpu().numpy(), orc.mix_update(rowptr, col, X, G, ws, we, 0.1)) <= 1e-5
        h.set_edge_times(None)                                            # back to per-worker times
        kept0, *_ = _select_gpu(h, n, nnz, t, b)
        assert np.array_equal(kept0, orc.select_fastest(rowptr, col, t, b))
    assert h.status() == 0
    h.close()
