"""CPU pins of the test-side BF16 reference (tests/bf16_reference.py) that the tensor-core gradient test
compares the GPU against: the rounding itself on values whose bfloat16 neighbours are known, and the
gradient where it must coincide with the double-precision oracle."""
import numpy as np

from bf16_reference import bf16_round, gradient_agrees, mlp_grad_bf16_points
from oracle import dbw_oracle as orc


def test_bf16_round_known_values():
    # bfloat16 keeps 8 significant bits: the spacing in [1, 2) is 2^-7
    assert bf16_round(1.0) == 1.0
    assert bf16_round(1.0 + 2.0 ** -7) == 1.0 + 2.0 ** -7
    assert bf16_round(1.0 + 2.0 ** -8) == 1.0                       # tie: to the even neighbour (1.0)
    assert bf16_round(1.0 + 3 * 2.0 ** -8) == 1.0 + 2.0 ** -6       # tie: to the even neighbour (1 + 2/128)
    assert bf16_round(1.0 + 2.0 ** -8 + 2.0 ** -20) == 1.0 + 2.0 ** -7
    assert bf16_round(-0.3) == -bf16_round(0.3)
    x = np.random.default_rng(0).standard_normal(1000)
    r = bf16_round(x)
    assert np.all(np.abs(r - x) <= np.abs(x) * 2.0 ** -8)           # half a unit in the last place
    assert np.array_equal(bf16_round(r), r)                         # idempotent
    assert np.all((r.astype(np.float32).view(np.uint32) & 0xFFFF) == 0)


def test_single_layer_is_the_oracle_when_features_are_representable():
    """Softmax regression has no tensor-core layer: only A_0 is rounded, so with bf16-representable features the
    reference must be the oracle's gradient exactly."""
    rng = np.random.default_rng(1)
    dims, B = [24, 7], 12
    feats = bf16_round(rng.random((B, 24)))
    labels = rng.integers(0, 7, B)
    x = (rng.standard_normal(24 * 7 + 7) * 0.3).astype(np.float32)
    g, l = mlp_grad_bf16_points(x, dims, feats, labels)
    g0, l0 = orc.mlp_grad(x, dims, feats, labels)
    assert np.abs(g - g0).max() <= 1e-14 and abs(l - l0) <= 1e-14


def test_integer_network_forward_is_exact_and_gradient_is_close():
    """Small integer features and weights: every activation is an integer below 256, hence bf16-exact, so the
    loss and the last layer's gradient equal the oracle's; the hidden layers differ only through the rounding of
    dZ (2^-8 relative)."""
    rng = np.random.default_rng(2)
    dims, B = [8, 6, 5, 4], 10
    feats = rng.integers(0, 4, (B, 8)).astype(np.float64)
    parts = []
    for l in range(3):
        parts.append(rng.integers(-2, 3, dims[l] * dims[l + 1]).astype(np.float64))
        parts.append(rng.integers(-1, 2, dims[l + 1]).astype(np.float64))
    x = np.concatenate(parts).astype(np.float32)
    labels = rng.integers(0, 4, B)
    g, l = mlp_grad_bf16_points(x, dims, feats, labels)
    g0, l0 = orc.mlp_grad(x, dims, feats, labels)
    assert abs(l - l0) <= 1e-13
    last = dims[2] * dims[3] + dims[3]
    assert np.abs(g[-last:] - g0[-last:]).max() <= 1e-13
    assert np.abs(g - g0).max() <= 2.0 ** -7 * np.abs(g0).max()
    assert np.abs(g - g0).max() > 0.0                               # the dZ rounding is really applied


def test_unresolvable_relu_decisions_are_enumerated():
    """A pre-activation that is zero up to fp32 accumulation error may be taken either way by the CUDA path: the
    reference lists it, and best_block_error accepts the gradient of either decision and nothing else."""
    rng = np.random.default_rng(3)
    dims, B = [16, 8, 4], 6
    feats = bf16_round(rng.random((B, 16)))
    x = (rng.standard_normal(16 * 8 + 8 + 8 * 4 + 4) * 0.5).astype(np.float32)
    x[16 * 8: 16 * 8 + 8] = 0.0
    w_row = bf16_round(x[:16])
    # unit 0 of sample 2: make the pre-activation cancel to (nearly) nothing through the fp32 bias
    x[16 * 8] = np.float32(-(feats[2] @ w_row) + 3e-7)
    x[:16] = w_row.astype(np.float32)
    labels = rng.integers(0, 4, B)
    amb = []
    g_on, _ = mlp_grad_bf16_points(x, dims, feats, labels, ambiguous=amb)
    assert amb == [(1, 2, 0)]
    g_off, _ = mlp_grad_bf16_points(x, dims, feats, labels, flips=amb)
    assert np.abs(g_on - g_off).max() > 1e-3 * np.abs(g_on).max()          # the two decisions really differ
    for g in (g_on, g_off):
        ok, rep = gradient_agrees(g, x, dims, feats, labels, tol=1e-9)
        assert ok and rep["max"] <= 1e-12 and rep["ambiguous"] == 1
    assert gradient_agrees(g_off, x, dims, feats, labels, tol=1e-9)[1]["switched"] == 1
    ok, rep = gradient_agrees(0.5 * (g_on + g_off), x, dims, feats, labels, tol=1e-9)
    assert not ok and rep["max"] > 1e-4                                    # anything in between is rejected


def test_strict_gate_rejects_real_defects_even_with_ambiguous_decisions():
    """The defects the gate exists to catch fail it whether or not ambiguous decisions are present: a dropped half
    of the batch in one layer's dW, a bias gradient off by the batch size, a unit masked wrongly."""
    rng = np.random.default_rng(3)
    dims, B = [16, 8, 4], 6
    feats = bf16_round(rng.random((B, 16)))
    x = (rng.standard_normal(16 * 8 + 8 + 8 * 4 + 4) * 0.5).astype(np.float32)
    x[16 * 8: 16 * 8 + 8] = 0.0
    w_row = bf16_round(x[:16])
    x[16 * 8] = np.float32(-(feats[2] @ w_row) + 3e-7)          # one ambiguous decision, as above
    x[:16] = w_row.astype(np.float32)
    labels = rng.integers(0, 4, B)
    g, _ = mlp_grad_bf16_points(x, dims, feats, labels)
    assert gradient_agrees(g * (1 + 1e-5), x, dims, feats, labels)[0]
    half = g.copy(); half[:16 * 8] *= 0.5
    assert not gradient_agrees(half, x, dims, feats, labels)[0]
    bias = g.copy(); bias[16 * 8: 16 * 8 + 8] *= B
    assert not gradient_agrees(bias, x, dims, feats, labels)[0]
    masked = g.copy(); masked[:16 * 8].reshape(8, 16)[3] = 0.0   # a unit that is NOT ambiguous
    assert not gradient_agrees(masked, x, dims, feats, labels)[0]
