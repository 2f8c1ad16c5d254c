"""Pins of the projection oracle: plain loops, the identity weight, linearity in both arguments."""
import numpy as np

from oracle import httm_linear as lin
from oracle import httm_oracle as orc
from paper_2511_21317_b200 import synth


def bits(a):
    return synth.f32_to_bf16_bits(np.asarray(a, dtype=np.float32))


def test_against_plain_loops():
    rng = np.random.default_rng(0)
    x, w = bits(rng.standard_normal((5, 7))), bits(rng.standard_normal((3, 7)))
    xf, wf = orc.bf16_to_double(x), orc.bf16_to_double(w)
    y = lin.linear(x, w)
    for i in range(5):
        for o in range(3):
            assert y[i, o] == sum(xf[i, k] * wf[o, k] for k in range(7)) or abs(y[i, o] - sum(xf[i, k] * wf[o, k] for k in range(7))) < 1e-14


def test_identity_weight_and_transposed_convention():
    rng = np.random.default_rng(1)
    x = bits(rng.standard_normal((4, 6)))
    assert np.array_equal(lin.linear(x, bits(np.eye(6))), orc.bf16_to_double(x))
    w = np.zeros((2, 6))
    w[0, 3] = 1.0          # output 0 picks input channel 3: weights are [out][in]
    w[1, 5] = -2.0
    y = lin.linear(x, bits(w))
    xf = orc.bf16_to_double(x)
    assert np.array_equal(y[:, 0], xf[:, 3]) and np.array_equal(y[:, 1], -2.0 * xf[:, 5])


def test_linearity_and_magnitude_bound():
    rng = np.random.default_rng(2)
    x1, x2 = bits(rng.standard_normal((3, 8))), bits(rng.standard_normal((3, 8)))
    w = bits(rng.standard_normal((5, 8)))
    xs = orc.bf16_to_double(x1) + orc.bf16_to_double(x2)
    assert np.allclose(lin.linear(x1, w) + lin.linear(x2, w), xs @ orc.bf16_to_double(w).T, rtol=1e-13, atol=1e-13)
    assert (np.abs(lin.linear(x1, w)) <= lin.magnitude(x1, w) + 1e-15).all()
