"""Pins of the oracle's verifier-layer pieces (linear, RMSNorm, rotary embedding,
SwiGLU): scalar loops, closed forms, the invariants that define a rotation, and
torch's CPU routines on small cases."""
import math

import numpy as np
import torch

from oracle import deer_oracle as O


def test_linear_matches_scalar_loops():
    r = np.random.default_rng(0)
    x, w = r.normal(size=(3, 5)), r.normal(size=(4, 5))
    y = O.linear(x, w)
    for m in range(3):
        for n in range(4):
            assert abs(y[m, n] - sum(x[m, c] * w[n, c] for c in range(5))) < 1e-13


def test_rmsnorm_closed_forms():
    # a constant row c: mean square c^2, so y = c / sqrt(c^2 + eps) * gamma
    g = np.array([1.0, 2.0, -3.0, 0.5])
    y = O.rmsnorm(np.full((2, 4), 3.0), g, 1e-6)
    np.testing.assert_allclose(y, np.tile(3.0 / math.sqrt(9.0 + 1e-6) * g, (2, 1)), rtol=1e-14)
    # with gamma = 1 and eps = 0 every row comes out with unit mean square, whatever its scale
    r = np.random.default_rng(1)
    x = r.normal(size=(5, 64)) * r.uniform(0.01, 100.0, size=(5, 1))
    y = O.rmsnorm(x, np.ones(64), 0.0)
    np.testing.assert_allclose((y * y).mean(axis=1), 1.0, rtol=1e-12)
    np.testing.assert_allclose(O.rmsnorm(7.0 * x, np.ones(64), 0.0), y, rtol=1e-12)
    # torch's routine
    t = torch.nn.functional.rms_norm(torch.from_numpy(x), (64,), torch.from_numpy(g.repeat(16)), 1e-5)
    np.testing.assert_allclose(O.rmsnorm(x, g.repeat(16), 1e-5), t.numpy(), rtol=1e-12)


def test_rope_is_a_rotation_with_relative_phase():
    r = np.random.default_rng(2)
    D, theta = 16, 10000.0
    q = r.normal(size=(1, 6, 2, D))
    k = r.normal(size=(1, 6, 2, D))
    pos = np.array([[0, 1, 5, 17, 100, 4097]])
    rq, rk = O.rope(q, pos, theta), O.rope(k, pos, theta)
    np.testing.assert_allclose(rq[0, 0], q[0, 0], atol=1e-15)                       # position 0: identity
    np.testing.assert_allclose((rq ** 2).sum(-1), (q ** 2).sum(-1), rtol=1e-12)      # norms are kept
    # scores depend on the position difference only: shifting both positions changes nothing
    rq2, rk2 = O.rope(q, pos + 1234, theta), O.rope(k, pos + 1234, theta)
    s1 = np.einsum("bthd,bshd->bhts", rq, rk)
    s2 = np.einsum("bthd,bshd->bhts", rq2, rk2)
    np.testing.assert_allclose(s1, s2, atol=1e-9)
    # one pair by hand: dims (d, d + D/2) rotate by pos * theta^(-2d/D)
    d, p = 3, 17
    ang = p * theta ** (-2.0 * d / D)
    a, b = q[0, 3, 1, d], q[0, 3, 1, d + D // 2]
    assert abs(rq[0, 3, 1, d] - (a * math.cos(ang) - b * math.sin(ang))) < 1e-13
    assert abs(rq[0, 3, 1, d + D // 2] - (b * math.cos(ang) + a * math.sin(ang))) < 1e-13


def test_swiglu_values():
    g = np.array([0.0, 1.0, -2.0, 30.0, -30.0])
    u = np.array([5.0, 2.0, 3.0, 1.0, 1.0])
    want = [0.0, 2.0 / (1.0 + math.exp(-1.0)), -6.0 / (1.0 + math.exp(2.0)), 30.0 / (1.0 + math.exp(-30.0)),
            -30.0 / (1.0 + math.exp(30.0))]
    np.testing.assert_allclose(O.swiglu(g, u), want, rtol=1e-14, atol=1e-300)
    t = torch.nn.functional.silu(torch.from_numpy(g)) * torch.from_numpy(u)
    np.testing.assert_allclose(O.swiglu(g, u), t.numpy(), rtol=1e-13)
