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


# ---------------------------------------------------------------- routed mixture of experts

def _moe_case(seed, M=5, hid=6, E=4, inter=3):
    r = np.random.default_rng(seed)
    return (r.normal(size=(M, hid)), r.normal(size=(E, hid)), r.normal(size=(E, 2 * inter, hid)) * 0.5,
            r.normal(size=(E, hid, inter)) * 0.5)


def test_moe_router_against_scalar_loops():
    x, wr, _, _ = _moe_case(0)
    experts, wts = O.moe_route(x, wr, 2)
    for m in range(x.shape[0]):
        logit = [sum(x[m, c] * wr[e, c] for c in range(x.shape[1])) for e in range(4)]
        mx = max(logit)
        ex = [math.exp(v - mx) for v in logit]
        prob = [v / sum(ex) for v in ex]
        order = sorted(range(4), key=lambda e: (-prob[e], e))[:2]
        assert experts[m].tolist() == order
        tot = prob[order[0]] + prob[order[1]]
        np.testing.assert_allclose(wts[m], [prob[order[0]] / tot, prob[order[1]] / tot], atol=1e-14)
    # without renormalisation the weights are the softmax probabilities themselves
    _, raw = O.moe_route(x, wr, 2, renormalise=False)
    assert (raw.sum(axis=1) < 1.0).all()
    # ties go to the lower expert index
    e, w = O.moe_route(np.ones((1, 2)), np.array([[1.0, 0.0], [0.0, 1.0], [0.5, 0.5]]), 2)
    assert e[0].tolist() == [0, 1] and abs(w[0, 0] - 0.5) < 1e-15


def test_moe_mlp_against_scalar_loops_and_special_cases():
    x, wr, wgu, wd = _moe_case(1)
    M, hid = x.shape
    E, twoI, _ = wgu.shape
    inter = twoI // 2
    y = O.moe_mlp(x, wr, wgu, wd, 2)
    experts, wts = O.moe_route(x, wr, 2)
    for m in range(M):
        acc = [0.0] * hid
        for j in range(2):
            e = int(experts[m, j])
            g = [sum(x[m, c] * wgu[e, i, c] for c in range(hid)) for i in range(inter)]
            u = [sum(x[m, c] * wgu[e, inter + i, c] for c in range(hid)) for i in range(inter)]
            a = [g[i] / (1.0 + math.exp(-g[i])) * u[i] for i in range(inter)]
            for o in range(hid):
                acc[o] += wts[m, j] * sum(a[i] * wd[e, o, i] for i in range(inter))
        np.testing.assert_allclose(y[m], acc, atol=1e-12)
    # one expert with weight 1 is the dense gated MLP
    dense = O.linear(O.swiglu(O.linear(x, wgu[2])[:, :inter], O.linear(x, wgu[2])[:, inter:]), wd[2])
    np.testing.assert_allclose(O.moe_mlp(x, wr[2:3], wgu[2:3], wd[2:3], 1), dense, atol=1e-12)
    # identical experts: the routing does not matter, the weights sum to one
    same_gu, same_d = np.repeat(wgu[:1], E, axis=0), np.repeat(wd[:1], E, axis=0)
    dense0 = O.linear(O.swiglu(O.linear(x, wgu[0])[:, :inter], O.linear(x, wgu[0])[:, inter:]), wd[0])
    np.testing.assert_allclose(O.moe_mlp(x, wr, same_gu, same_d, 3), dense0, atol=1e-12)
    # all experts chosen without renormalisation: the full softmax mixture
    full = O.moe_mlp(x, wr, wgu, wd, E, renormalise=False)
    prob = np.exp(x @ wr.T)
    prob /= prob.sum(axis=1, keepdims=True)
    mix = sum(prob[:, e:e + 1] * O.linear(O.swiglu(O.linear(x, wgu[e])[:, :inter], O.linear(x, wgu[e])[:, inter:]), wd[e])
              for e in range(E))
    np.testing.assert_allclose(full, mix, atol=1e-12)
