"""CPU pins of the test-side BF16 reference (tests/bf16_reference.py) that the tensor-core gradient test
compares the GPU against: the rounding itself on values whose bfloat16 neighbours are known, and the
gradient where it must coincide with the double-precision oracle."""
import numpy as np

from bf16_reference import bf16_round, mlp_grad_bf16_points
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
