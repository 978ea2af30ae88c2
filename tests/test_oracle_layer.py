"""Pins for the decoder-layer pieces of the oracle: textbook formulas in numpy float64."""
import numpy as np
import torch

from oracle import dcut_oracle as orc


def _bf(x):
    return torch.from_numpy(np.asarray(x, np.float32)).to(torch.bfloat16)


def test_rmsnorm():
    rng = np.random.default_rng(0)
    x, g = _bf(rng.standard_normal((5, 96))), _bf(1 + 0.1 * rng.standard_normal(96))
    xd, gd = x.double().numpy(), g.double().numpy()
    want = xd / np.sqrt((xd ** 2).mean(1, keepdims=True) + 1e-6) * gd
    np.testing.assert_allclose(orc.rmsnorm(x, g, 1e-6), want, rtol=1e-13)
    np.testing.assert_allclose(orc.rmsnorm(_bf(np.full((1, 8), 3.0)), _bf(np.ones(8)), 0.0), np.ones((1, 8)), rtol=1e-15)


def test_linear_is_a_times_w_transposed():
    rng = np.random.default_rng(1)
    a, w = _bf(rng.standard_normal((7, 40))), _bf(rng.standard_normal((11, 40)))
    np.testing.assert_allclose(orc.linear(a, w), a.double().numpy() @ w.double().numpy().T, rtol=1e-13, atol=1e-13)


def test_rope():
    rng = np.random.default_rng(2)
    x = _bf(rng.standard_normal((4, 3, 16)))
    pos = np.array([0, 1, 17, 4000], np.int32)
    y = orc.rope(x, pos, 1.0e6)
    xd = x.double().numpy()
    assert np.array_equal(y[0], xd[0])                                  # position 0 is the identity
    half = 8
    inv = 1.0e6 ** (-np.arange(half) / half)                            # theta^(-2e/Dh)
    for r in range(4):
        ang = pos[r] * inv
        z = (xd[r, :, :half] + 1j * xd[r, :, half:]) * np.exp(1j * ang)  # rotation of the pair (e, e+Dh/2)
        np.testing.assert_allclose(y[r, :, :half], z.real, rtol=1e-12, atol=1e-13)
        np.testing.assert_allclose(y[r, :, half:], z.imag, rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose((y ** 2).sum(-1), (xd ** 2).sum(-1), rtol=1e-12)   # norms preserved


def test_swiglu_and_rounding():
    rng = np.random.default_rng(3)
    g, u = _bf(rng.standard_normal(100) * 3), _bf(rng.standard_normal(100))
    gd, ud = g.double().numpy(), u.double().numpy()
    np.testing.assert_allclose(orc.swiglu(g, u), gd / (1 + np.exp(-gd)) * ud, rtol=1e-13)
    v = rng.standard_normal(1000) * 10
    want = torch.from_numpy(v.astype(np.float32)).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(orc.round_bf16(v), want)                      # round-to-nearest-even
