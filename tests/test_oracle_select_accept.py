"""Pins for the oracle's LM-head selection and acceptance rule."""
import itertools
import math

import numpy as np
import pytest
import torch
from scipy.special import softmax as sp_softmax

from oracle import deer_oracle as O


# ---------------------------------------------------------------- selection

def test_logits_and_argmax_match_scalar_loops():
    r = np.random.default_rng(0)
    h = r.normal(size=(5, 7))
    w = r.normal(size=(11, 7))
    z = O.lm_logits(h, w)
    for m in range(5):
        for v in range(11):
            assert abs(z[m, v] - sum(h[m, c] * w[v, c] for c in range(7))) < 1e-13
    ids = O.select_argmax(z)
    for m in range(5):
        best = max(range(11), key=lambda v: (z[m, v], -v))
        assert ids[m] == best


def test_argmax_takes_lowest_index_among_maxima():
    z = np.array([[0.0, 2.0, 2.0, 1.0], [5.0, 5.0, 5.0, 5.0], [1.0, 0.0, 3.0, 3.0]])
    assert O.select_argmax(z).tolist() == [1, 0, 2]


def test_planted_column_is_found():
    r = np.random.default_rng(1)
    h = r.normal(size=(6, 32))
    w = r.normal(size=(50, 32)) * 0.1
    want = [3, 49, 0, 17, 17, 8]
    for m, v in enumerate(want):
        w_row_boost = h[m] / np.dot(h[m], h[m]) * 100.0
        w2 = w.copy()
        w2[v] += w_row_boost
        assert O.select_argmax(O.lm_logits(h[m:m + 1], w2))[0] == v


@pytest.mark.parametrize("T", [1.0, 0.6, 2.5])
def test_logsumexp_and_max_logprob_match_torch(T):
    r = np.random.default_rng(2)
    z = r.normal(size=(9, 301)) * 4
    ref = torch.logsumexp(torch.from_numpy(z) / T, dim=1).numpy()
    np.testing.assert_allclose(O.logsumexp(z, T), ref, atol=1e-12)
    lp = O.max_logprob(z)
    assert (lp <= 0).all()
    ref_lp = torch.log_softmax(torch.from_numpy(z), dim=1).max(dim=1).values.numpy()
    np.testing.assert_allclose(lp, ref_lp, atol=1e-12)
    # sum of softmax is one
    np.testing.assert_allclose(np.exp(z / T - O.logsumexp(z, T)[:, None]).sum(axis=1), 1.0, atol=1e-12)


def test_top2_gap():
    z = np.array([[1.0, 4.0, 3.5, -2.0], [7.0, 7.0, 0.0, 1.0]])
    np.testing.assert_allclose(O.top2_gap(z), [0.5, 0.0])


# ---------------------------------------------------------------- greedy

def test_greedy_exhaustive_small():
    """All draft/target pairs for V=3, k<=4 against the definition: the accepted
    length is the index of the first mismatch; the emitted tokens are the target
    tokens up to and including that index."""
    for k in range(1, 5):
        for target in itertools.product(range(3), repeat=k):
            drafts = np.array(list(itertools.product(range(3), repeat=k)), dtype=np.int32)
            tgt = np.broadcast_to(np.array(target, dtype=np.int32), drafts.shape)
            a, out, n = O.accept_greedy(drafts, tgt)
            for row in range(drafts.shape[0]):
                mism = [i for i in range(k) if drafts[row, i] != target[i]]
                first = mism[0] if mism else k
                assert a[row] == first
                assert n[row] == min(first + 1, k)
                assert out[row, :n[row]].tolist() == list(target[:n[row]])
                assert (out[row, n[row]:] == -1).all()


def test_greedy_returns_planted_prefix_length():
    from paper_2512_15176_b200 import workload as W
    cfg = W.StepConfig("t", 64, 4, 2, 8, 32, 16, 1000, (8, 8), seed=5)
    target = W.rng(5, "tgt").integers(0, cfg.V, size=(cfg.B, cfg.k)).astype(np.int32)
    L = W.planted_prefix_lengths(cfg)
    assert L.max() <= cfg.k and L.min() >= 0 and len(set(L.tolist())) > 5
    drafts = W.plant_drafts(cfg, target, L)
    a, out, n = O.accept_greedy(drafts, target)
    np.testing.assert_array_equal(a, L)
    np.testing.assert_array_equal(n, np.minimum(L + 1, cfg.k))


def test_greedy_eos_truncates():
    draft = np.array([[4, 9, 2, 7], [4, 9, 2, 7], [4, 9, 2, 7]], dtype=np.int32)
    target = np.array([[4, 9, 2, 7], [4, 9, 5, 7], [4, 8, 2, 7]], dtype=np.int32)
    a, out, n = O.accept_greedy(draft, target, eos_id=9)
    assert a.tolist() == [2, 2, 1] and n.tolist() == [2, 2, 2]
    assert out.tolist() == [[4, 9, -1, -1], [4, 9, -1, -1], [4, 8, -1, -1]]
    a, out, n = O.accept_greedy(draft, target, eos_id=5)
    assert a.tolist() == [4, 2, 1] and n.tolist() == [4, 3, 2]


# ---------------------------------------------------------------- sampling

def _black_box_alpha(zp, zq, T, y):
    """Largest u the oracle still accepts for draft y, by bisection."""
    lo, hi = 0.0, 1.0
    d = np.array([[y]], dtype=np.int32)
    r = np.array([0.5])
    if O.accept_sample(d, zp[None, None], T, zq[None, None], np.array([[1.0]]), r)[0][0] == 1:
        return 1.0
    for _ in range(60):
        mid = 0.5 * (lo + hi)
        acc = O.accept_sample(d, zp[None, None], T, zq[None, None], np.array([[mid]]), r)[0][0]
        lo, hi = (mid, hi) if acc == 1 else (lo, mid)
    return 0.5 * (lo + hi)


def _black_box_residual(zp, zq, T, y_rejected):
    """The law of the oracle's replacement token, recovered from where its
    output changes as r sweeps (0, 1)."""
    V = len(zp)
    d = np.array([[y_rejected]], dtype=np.int32)
    u = np.array([[1.0]])

    def tok(r):
        a, out, n = O.accept_sample(d, zp[None, None], T, zq[None, None], u, np.array([r]))
        assert a[0] == 0 and n[0] == 1
        return int(out[0, 0])

    cdf = np.zeros(V)
    for v in range(V):
        # sup { r : tok(r) <= v }
        if tok(1.0 - 1e-15) <= v:
            cdf[v] = 1.0
            continue
        if tok(1e-300) > v:
            cdf[v] = 0.0
            continue
        lo, hi = 0.0, 1.0
        for _ in range(60):
            mid = 0.5 * (lo + hi)
            lo, hi = (mid, hi) if tok(mid) <= v else (lo, mid)
        cdf[v] = 0.5 * (lo + hi)
    return np.diff(np.concatenate([[0.0], cdf]))


@pytest.mark.parametrize("seed,T", [(0, 1.0), (1, 0.6), (2, 1.7)])
def test_one_step_lossless_identity(seed, T):
    """Appendix lemma: q(a) * alpha(a) + (1 - gamma) * p_res(a) = p(a) for every
    token a, with alpha and p_res measured from the oracle as a black box and
    p, q from scipy's softmax."""
    r = np.random.default_rng(seed)
    V = 7
    zp = r.normal(size=V) * 2
    zq = r.normal(size=V) * 2
    p = sp_softmax(zp / T)
    q = sp_softmax(zq)
    alpha = np.array([_black_box_alpha(zp, zq, T, y) for y in range(V)])
    rejectable = [y for y in range(V) if alpha[y] < 1.0 - 1e-9]
    assert rejectable
    pres = _black_box_residual(zp, zq, T, rejectable[0])
    gamma = float((q * alpha).sum())
    np.testing.assert_allclose(q * alpha + (1.0 - gamma) * pres, p, atol=1e-9)
    np.testing.assert_allclose(gamma, np.minimum(p, q).sum(), atol=1e-9)
    assert abs(pres.sum() - 1.0) < 1e-9
    assert all(pres[v] == 0.0 or p[v] > q[v] for v in range(V))


def test_sampling_monte_carlo_first_token_and_accept_length():
    """Drafts drawn from q, then the rule applied: the first emitted token is
    distributed as p_1 (lossless), and P[accept_len >= i] = prod_{t<=i} gamma_t."""
    rng = np.random.default_rng(123)
    V, k, N = 12, 4, 120000
    zp = rng.normal(size=(k, V)) * 1.5
    zq = zp + rng.normal(size=(k, V)) * 0.8
    T = 0.8
    p = sp_softmax(zp / T, axis=1)
    q = sp_softmax(zq, axis=1)
    drafts = np.stack([rng.choice(V, size=N, p=q[i]) for i in range(k)], axis=1).astype(np.int32)
    u = rng.random((N, k))
    r = rng.random(N)
    a, out, n = O.accept_sample(drafts, np.broadcast_to(zp, (N, k, V)), T, np.broadcast_to(zq, (N, k, V)), u, r)
    first = np.bincount(out[:, 0], minlength=V) / N
    sigma = np.sqrt(p[0] * (1 - p[0]) / N)
    assert (np.abs(first - p[0]) < 4.5 * sigma).all()
    gam = np.minimum(p, q).sum(axis=1)
    for i in range(1, k + 1):
        want = float(np.prod(gam[:i]))
        got = float((a >= i).mean())
        assert abs(got - want) < 4.5 * math.sqrt(want * (1 - want) / N) + 1e-9
    # given exactly i accepted (i < k), the replacement token follows the residual of row i
    for i in range(k):
        sel = (a == i) if i < k else None
        res = np.maximum(0, p[i] - q[i])
        res /= res.sum()
        emp = np.bincount(out[sel, i], minlength=V) / sel.sum()
        sg = np.sqrt(res * (1 - res) / sel.sum())
        assert (np.abs(emp - res) < 4.5 * sg + 1e-9).all()
    assert ((n == np.minimum(a + 1, k))).all()


def test_sampling_special_cases():
    rng = np.random.default_rng(9)
    V, k, B = 9, 5, 200
    z = rng.normal(size=(B, k, V))
    drafts = rng.integers(0, V, size=(B, k)).astype(np.int32)
    u = np.full((B, k), 1.0)            # the hardest uniform to accept
    r = rng.random(B)
    # q == p: alpha = 1 everywhere, everything accepted
    a, out, n = O.accept_sample(drafts, z, 1.0, z, u, r)
    assert (a == k).all() and (n == k).all() and (out == drafts).all()
    # (almost) disjoint supports: drafts live where p is ~0 -> rejected at 0, output ~ p
    zp = np.full((B, k, V), -80.0)
    zq = np.full((B, k, V), -80.0)
    zp[..., :4] = rng.normal(size=(B, k, 4))
    zq[..., 4:] = rng.normal(size=(B, k, 5))
    d2 = rng.integers(4, V, size=(B, k)).astype(np.int32)
    a, out, n = O.accept_sample(d2, zp, 1.0, zq, rng.random((B, k)) * 0.99 + 0.01, r)
    assert (a == 0).all() and (n == 1).all() and (out[:, 0] < 4).all() and (out[:, 1:] == -1).all()
    for b in range(5):
        p0 = sp_softmax(zp[b, 0])
        want = int(np.searchsorted(np.cumsum(p0[:4]) / p0[:4].sum(), r[b]))
        assert out[b, 0] == want
    # small temperature reproduces the greedy rule (drafter one-hot on its own token)
    zt = rng.normal(size=(B, k, V))
    tgt = zt.argmax(axis=2).astype(np.int32)
    d3 = tgt.copy()
    flip = rng.random((B, k)) < 0.3
    d3[flip] = (d3[flip] + 1) % V
    zq3 = np.full((B, k, V), -200.0)
    np.put_along_axis(zq3, d3[..., None].astype(np.int64), 0.0, axis=2)
    a, out, n = O.accept_sample(d3, zt, 1e-3, zq3, rng.random((B, k)) * 0.98 + 0.01, r)
    ag, outg, ng = O.accept_greedy(d3, tgt)
    np.testing.assert_array_equal(a, ag)
    np.testing.assert_array_equal(out, outg)
    np.testing.assert_array_equal(n, ng)


def test_sampling_zero_residual_falls_back_to_target():
    """p == q makes the residual mass zero; a forced rejection then draws from p."""
    z = np.log(np.array([[[0.1, 0.2, 0.3, 0.4]]]))
    for r, want in [(0.05, 0), (0.25, 1), (0.5, 2), (0.95, 3)]:
        a, out, n = O.accept_sample(np.array([[2]], dtype=np.int32), z, 1.0, z, np.array([[1.5]]), np.array([r]))
        assert a[0] == 0 and n[0] == 1 and out[0, 0] == want


def test_sampling_eos():
    z = np.zeros((1, 4, 5))
    d = np.array([[1, 2, 3, 4]], dtype=np.int32)
    a, out, n = O.accept_sample(d, z, 1.0, z, np.full((1, 4), 0.5), np.array([0.5]), eos_id=2)
    assert a[0] == 2 and n[0] == 2 and out[0].tolist() == [1, 2, -1, -1]


# ---------------------------------------------------------------- the extra token after a fully accepted block

def test_greedy_bonus_exhaustive_small():
    """k rows = k-1 drafts + one more row.  By the definition: the emitted tokens are
    the target tokens up to and including the first mismatch among the k-1 drafts,
    or all k target tokens when every draft matches; always accept_len + 1 of them."""
    for k in range(1, 5):
        for target in itertools.product(range(3), repeat=k):
            drafts = np.array(list(itertools.product(range(3), repeat=k)), dtype=np.int32)
            tgt = np.broadcast_to(np.array(target, dtype=np.int32), drafts.shape)
            a, out, n = O.accept_greedy(drafts, tgt, bonus=True)
            for row in range(drafts.shape[0]):
                mism = [i for i in range(k - 1) if drafts[row, i] != target[i]]
                first = mism[0] if mism else k - 1
                assert a[row] == first and n[row] == first + 1
                assert out[row, :n[row]].tolist() == list(target[:n[row]])
                assert (out[row, n[row]:] == -1).all()


def test_sampling_bonus_monte_carlo():
    """With the extra row every block emits accept_len + 1 tokens, each distributed as
    the verifier's own distribution of its row: the first token as p_0 whatever
    happens, and the token after k-1 accepted drafts as p_{k-1} itself.  The mean
    number of emitted tokens is 1 + sum_i prod_{t<=i} gamma_t (a closed form)."""
    rng = np.random.default_rng(321)
    V, k, N = 10, 3, 150000
    zp = rng.normal(size=(k, V)) * 1.2
    zq = zp + rng.normal(size=(k, V)) * 0.6
    T = 0.9
    p = sp_softmax(zp / T, axis=1)
    q = sp_softmax(zq, axis=1)
    drafts = np.stack([rng.choice(V, size=N, p=q[i]) for i in range(k)], axis=1).astype(np.int32)
    u = rng.random((N, k))
    r = rng.random(N)
    a, out, n = O.accept_sample(drafts, np.broadcast_to(zp, (N, k, V)), T, np.broadcast_to(zq, (N, k, V)), u, r, bonus=True)
    assert (n == a + 1).all() and a.max() == k - 1
    first = np.bincount(out[:, 0], minlength=V) / N
    assert (np.abs(first - p[0]) < 4.5 * np.sqrt(p[0] * (1 - p[0]) / N)).all()
    full = a == k - 1
    emp = np.bincount(out[full, k - 1], minlength=V) / full.sum()
    assert (np.abs(emp - p[k - 1]) < 4.5 * np.sqrt(p[k - 1] * (1 - p[k - 1]) / full.sum()) + 1e-9).all()
    gam = np.minimum(p, q).sum(axis=1)
    want = 1.0 + sum(float(np.prod(gam[:i])) for i in range(1, k))
    assert abs(n.mean() - want) < 4.5 * n.std() / math.sqrt(N)
    # the draft in the last column is never looked at
    drafts2 = drafts.copy()
    drafts2[:, k - 1] = (drafts2[:, k - 1] + 1) % V
    a2, out2, n2 = O.accept_sample(drafts2, np.broadcast_to(zp, (N, k, V)), T, np.broadcast_to(zq, (N, k, V)), u, r, bonus=True)
    assert (a2 == a).all() and (out2 == out).all()


def test_sampling_bonus_with_one_row_is_plain_sampling():
    """k = 1: no drafts at all, the block is one ordinary decoding step: the token is
    the inverse CDF of p at r (brute force over the cumulative sums)."""
    rng = np.random.default_rng(5)
    V = 7
    z = rng.normal(size=(4, 1, V))
    r = np.array([0.05, 0.4, 0.77, 0.999])
    a, out, n = O.accept_sample(np.zeros((4, 1), np.int32), z, 1.3, z, np.full((4, 1), 0.5), r, bonus=True)
    assert a.tolist() == [0] * 4 and n.tolist() == [1] * 4
    for b in range(4):
        pb = sp_softmax(z[b, 0] / 1.3)
        acc, want = 0.0, None
        for v in range(V):
            acc += pb[v]
            if acc >= r[b]:
                want = v
                break
        assert out[b, 0] == want


# ---------------------------------------------------------------- two corners

def test_inverse_cdf_when_the_cumulative_sum_falls_short_of_the_target():
    """Hand-built weights whose running sum, rounded term by term, ends below r * total although total is their
    exact sum: the draw is then the last token that carries weight (trailing zero-weight tokens can never be drawn)."""
    big, tiny = 1.0, 2.0 ** -54
    w = np.array([big, tiny, tiny, tiny, tiny, 0.0, 0.0])
    cdf_end = float(np.cumsum(w)[-1])
    assert cdf_end == 1.0                              # each tiny term is below half an ulp of 1 and is lost
    total = math.fsum(w)                               # the exact sum 1 + 2^-52 is representable
    assert total == 1.0 + 2.0 ** -52 and total > cdf_end
    assert O.inverse_cdf(w, total, 1.0) == 4           # r * total > cdf[-1]: last index with weight, not 6
    # the ordinary branch on the same weights
    assert O.inverse_cdf(w, total, 0.5) == 0
    assert O.inverse_cdf(w, total, 0.0) == 0
    # brute force definition on a case without rounding trouble
    w2 = np.array([0.0, 0.25, 0.0, 0.5, 0.25])
    for r, want in [(0.0, 0), (0.1, 1), (0.25, 1), (0.26, 3), (0.75, 3), (0.76, 4), (1.0, 4)]:
        acc, pick = 0.0, None
        for v, x in enumerate(w2):
            acc += x
            if acc >= r * 1.0:
                pick = v
                break
        assert O.inverse_cdf(w2, 1.0, r) == pick == want


def test_sampling_with_the_extra_row_and_an_eos_hand_worked():
    """k = 3 rows = 2 drafts + one more row, vocabulary of 4, worked by hand.
    Row distributions are chosen so that every acceptance probability is 1 or 0:
      sequence 0: both drafts have p = q (alpha = 1) -> accepted; the extra row's p = (0.1, 0.2, 0.3, 0.4) and
                  r = 0.35 picks token 2 (cumulative 0.1, 0.3, 0.6).  Emitted 1, 3, 2.
      sequence 1: draft 0 accepted; draft 1 = token 0 has p(0) = 0 -> rejected whatever u is; residual of
                  p = (0, 0.5, 0.5, 0) against q = (0.5, 0.5, 0, 0) is (0, 0, 0.5, 0) -> token 2.  Emitted 2, 2.
    With eos_id = 3 sequence 0 stops after its second token (the 3): n_out 2, accept_len stays 2; with eos_id = 1
    it stops after the first: n_out 1 and accept_len is cut to 1.  Sequence 1 never emits 3 or 1."""
    lg = lambda p: np.log(np.maximum(np.asarray(p, dtype=np.float64), 1e-300))
    same = [0.25, 0.25, 0.25, 0.25]
    zt = np.stack([
        np.stack([lg(same), lg(same), lg([0.1, 0.2, 0.3, 0.4])]),
        np.stack([lg(same), lg([0.0, 0.5, 0.5, 0.0]), lg(same)]),
    ])
    zq = np.stack([
        np.stack([lg(same), lg(same), lg(same)]),
        np.stack([lg(same), lg([0.5, 0.5, 0.0, 0.0]), lg(same)]),
    ])
    drafts = np.array([[1, 3, 0], [2, 0, 0]], dtype=np.int32)      # column 2 is ignored
    u = np.full((2, 3), 0.999)
    r = np.array([0.35, 0.5])
    a, out, n = O.accept_sample(drafts, zt, 1.0, zq, u, r, eos_id=-1, bonus=True)
    assert a.tolist() == [2, 1] and n.tolist() == [3, 2]
    assert out.tolist() == [[1, 3, 2], [2, 2, -1]]
    a, out, n = O.accept_sample(drafts, zt, 1.0, zq, u, r, eos_id=3, bonus=True)
    assert a.tolist() == [2, 1] and n.tolist() == [2, 2]
    assert out.tolist() == [[1, 3, -1], [2, 2, -1]]
    a, out, n = O.accept_sample(drafts, zt, 1.0, zq, u, r, eos_id=1, bonus=True)
    assert a.tolist() == [1, 1] and n.tolist() == [1, 2]
    assert out.tolist() == [[1, -1, -1], [2, 2, -1]]
    # eos_id = 2: for sequence 0 the extra token itself is the EOS, it is emitted and nothing is cut; sequence 1's
    # first token (an accepted draft) is the EOS, so its correction is dropped and the accepted draft stays counted
    a, out, n = O.accept_sample(drafts, zt, 1.0, zq, u, r, eos_id=2, bonus=True)
    assert a.tolist() == [2, 1] and n.tolist() == [3, 1]
    assert out.tolist() == [[1, 3, 2], [2, -1, -1]]
