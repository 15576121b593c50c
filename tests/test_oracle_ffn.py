"""Pins for the CPU oracle's expert FFN (oracle/ffn.py): a case worked by hand,
limits of SiLU, rounding ties, linearity, and library conversions.  No GPU."""
import numpy as np
import torch

from oracle import ffn
from paper_2601_21198_b200 import inputs


def bits(a):
    return inputs.f32_to_bf16_bits(np.asarray(a, dtype=np.float32))


def test_bf16_conversions_against_torch():
    rng = np.random.default_rng(0)
    x = (rng.standard_normal(20000) * np.exp(rng.uniform(-30, 30, 20000))).astype(np.float32)
    ref = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(ffn.f64_to_bf16(x.astype(np.float64)), ref)
    back = torch.from_numpy(ref.view(np.int16)).view(torch.bfloat16).to(torch.float64).numpy()
    assert np.array_equal(ffn.bf16_to_f64(ref), back)


def test_rounding_ties_go_to_even_and_tiny_values_keep_fixed_spacing():
    one = 1.0
    ulp = 2.0 ** -7
    got = ffn.bf16_to_f64(ffn.f64_to_bf16(np.array([one + ulp / 2, one + 3 * ulp / 2, one + ulp / 2 + 1e-9,
                                                    -(one + ulp / 2), 2.0 ** -133 * 1.5, 2.0 ** -133 * 2.5, 0.0])))
    assert got.tolist() == [1.0, 1.0 + 2 * ulp, 1.0 + ulp, -1.0, 2.0 ** -132, 2.0 ** -132, 0.0]
    assert ffn.f64_to_bf16(np.array([3.4e38, -3.4e38, np.inf])).tolist() == [0x7F80, 0xFF80, 0x7F80]


def test_silu_limits():
    assert ffn.silu(0.0) == 0.0
    assert abs(ffn.silu(40.0) - 40.0) < 1e-12
    assert abs(ffn.silu(-40.0)) < 1e-12
    assert abs(ffn.silu(1.0) - 0.7310585786300049) < 1e-15
    z = np.linspace(-5, 5, 11)
    assert np.allclose(ffn.silu(z) - ffn.silu(-z), z)          # SiLU(z) - SiLU(-z) = z


def test_tiny_expert_worked_by_hand():
    """H = I = 2.  x = (1, -1); W1 = identity, W3 = 2*identity, W2 = [[1,1],[0,1]].
    g = (1,-1), u = (2,-2); SiLU(1)*2 = 1.46211..., SiLU(-1)*(-2) = 0.53788...;
    in bf16 (spacing 2^-7 on [1,2), 2^-8 on [0.5,1)) these are 187/128 = 1.4609375
    and 138/256 = 0.5390625; y = (1.4609375 + 0.5390625, 0.5390625) = (2, 0.5390625)."""
    x = bits([[1.0, -1.0]])
    w1 = {0: bits([[1, 0], [0, 1]])}
    w3 = {0: bits([[2, 0], [0, 2]])}
    w2 = {0: bits([[1, 1], [0, 1]])}
    out, y = ffn.expert_ffn(x, np.array([[0]]), None, w1, w3, w2)
    assert y.tolist() == [[2.0, 0.5390625]]
    assert np.array_equal(out, bits([[2.0, 0.5390625]]))
    # the matrices are [out, in]: swapping W2 for its transpose changes the answer
    out_t, y_t = ffn.expert_ffn(x, np.array([[0]]), None, w1, w3, {0: bits([[1, 0], [1, 1]])})
    assert y_t.tolist() == [[1.4609375, 2.0]]


def test_combine_is_linear_in_the_routing_weights():
    rng = np.random.default_rng(3)
    H, I, E, T = 8, 16, 3, 4
    w1 = {e: bits(rng.standard_normal((I, H)) * 0.3) for e in range(E)}
    w3 = {e: bits(rng.standard_normal((I, H)) * 0.3) for e in range(E)}
    w2 = {e: bits(rng.standard_normal((H, I)) * 0.3) for e in range(E)}
    x = bits(rng.standard_normal((T, H)))
    ids = np.array([[0, 1], [2, 0], [1, 2], [0, 2]])
    _, y_a = ffn.expert_ffn(x, ids[:, :1], None, w1, w3, w2)
    _, y_b = ffn.expert_ffn(x, ids[:, 1:], None, w1, w3, w2)
    wts = rng.random((T, 2))
    _, y = ffn.expert_ffn(x, ids, wts, w1, w3, w2)
    assert np.allclose(y, wts[:, :1] * y_a + wts[:, 1:] * y_b, rtol=1e-13, atol=1e-13)
    _, y_ones = ffn.expert_ffn(x, ids, None, w1, w3, w2)
    assert np.allclose(y_ones, y_a + y_b, rtol=1e-13, atol=1e-13)
    # tokens are independent: token 2 alone gives row 2
    _, y2 = ffn.expert_ffn(x[2:3], ids[2:3], wts[2:3], w1, w3, w2)
    assert np.array_equal(y2[0], y[2])


def test_fp64_and_fp32_accumulation_agree_far_inside_the_tolerance():
    """Bounds the oracle's own error: the same FFN in float32 matmuls differs
    from the fp64 oracle by orders of magnitude less than the 1e-2 tolerance."""
    rng = np.random.default_rng(4)
    H, I = 256, 512
    w1 = bits(rng.standard_normal((I, H)) * 0.02)
    w3 = bits(rng.standard_normal((I, H)) * 0.02)
    w2 = bits(rng.standard_normal((H, I)) * 0.02)
    x = bits(rng.standard_normal((2, H)))
    _, y = ffn.expert_ffn(x, np.array([[0], [0]]), None, {0: w1}, {0: w3}, {0: w2})
    f = inputs.bf16_bits_to_f32
    g, u = f(x) @ f(w1).T, f(x) @ f(w3).T
    h = f(inputs.f32_to_bf16_bits(g / (1 + np.exp(-g)) * u))
    y32 = h @ f(w2).T
    assert np.abs(y32 - y).max() < 1e-4


def test_routing_generator_shapes_and_normalisation():
    ids, w = inputs.routing(64, n_experts=8, k=2, seed=1)
    assert ids.shape == (64, 2) and w.shape == (64, 2)
    assert (ids[:, 0] != ids[:, 1]).all() and ids.min() >= 0 and ids.max() < 8
    assert np.allclose(w.sum(axis=1), 1.0, atol=1e-6)
    counts = np.bincount(inputs.routing(4000, seed=2)[0].ravel(), minlength=8)
    assert counts.max() > 2.5 * counts.min()          # skewed popularity
