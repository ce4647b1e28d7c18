"""Pins for the oracle's top-k / nucleus truncation and for the acceptance rule applied to the truncated
verifier distribution."""
import numpy as np
import pytest
from scipy.special import softmax as sp_softmax

from oracle import deer_oracle as O


def _brute_force(p, top_k, top_p):
    """Sort-based restatement on plain Python lists: tokens ordered by falling probability, tie groups whole."""
    V = len(p)
    order = sorted(range(V), key=lambda v: (-p[v], v))
    keep = set(range(V))
    if top_k and top_k < V:
        kth = p[order[top_k - 1]]
        keep = {v for v in range(V) if p[v] >= kth}
    if top_p < 1.0:
        tot = sum(p[v] for v in keep)
        pk = {v: p[v] / tot for v in keep}
        ordered = [v for v in order if v in keep]
        acc, chosen, i = 0.0, set(), 0
        while i < len(ordered):
            grp = [v for v in ordered[i:] if pk[v] == pk[ordered[i]]]
            chosen.update(grp)
            acc += sum(pk[v] for v in grp)
            i += len(grp)
            if acc >= top_p:
                break
        keep = chosen
    tot = sum(p[v] for v in keep)
    return [p[v] / tot if v in keep else 0.0 for v in range(V)], keep


@pytest.mark.parametrize("seed", range(6))
def test_truncation_matches_sort_based_brute_force(seed):
    r = np.random.default_rng(seed)
    V = 13
    p = sp_softmax(r.normal(size=V) * 1.5)
    if seed % 2:                       # plant ties, one of them at a boundary
        p[3] = p[7]
        p[1] = p[9] = p[11]
        p /= p.sum()
    for top_k in (0, 1, 3, 5, 12, 13, 40):
        for top_p in (1.0, 0.95, 0.7, 0.3, 0.01):
            got, keep = O.truncate_distribution(p, top_k, top_p)
            want, wkeep = _brute_force(list(p), top_k, top_p)
            assert set(np.flatnonzero(keep)) == wkeep, (top_k, top_p)
            np.testing.assert_allclose(got, want, atol=1e-15)


def test_truncation_invariants():
    r = np.random.default_rng(42)
    for _ in range(20):
        V = int(r.integers(2, 60))
        p = sp_softmax(r.normal(size=V) * 2)
        top_k, top_p = int(r.integers(1, V + 1)), float(r.uniform(0.05, 0.999))
        out, keep = O.truncate_distribution(p, top_k, top_p)
        assert abs(out.sum() - 1.0) < 1e-12 and (out[~keep] == 0).all() and (out[keep] > 0).all()
        # an upper level set: everything kept is at least as likely as everything dropped
        assert keep.all() or p[keep].min() > p[~keep].max()
        assert keep.sum() <= top_k                                   # distinct values here: no tie can widen the set
        # the nucleus is minimal: dropping its least likely token leaves less than top_p of the top-k mass
        pk, kk = O.truncate_distribution(p, top_k, 1.0)
        if keep.sum() < kk.sum():
            assert pk[keep].sum() >= top_p - 1e-12
            v_min = np.flatnonzero(keep)[np.argmin(p[keep])]
            assert pk[keep].sum() - pk[v_min] < top_p
        # no truncation asked for: the vector itself
        same, all_kept = O.truncate_distribution(p, 0, 1.0)
        np.testing.assert_array_equal(same, p / p.sum())
        assert all_kept.all()
    # ties travel together
    p = np.array([0.3, 0.2, 0.2, 0.2, 0.1])
    _, keep = O.truncate_distribution(p, 2, 1.0)
    assert keep.tolist() == [True, True, True, True, False]
    _, keep = O.truncate_distribution(p, 0, 0.45)
    assert keep.tolist() == [True, True, True, True, False]
    _, keep = O.truncate_distribution(p, 0, 0.3)
    assert keep.tolist() == [True, False, False, False, False]


def _alpha_and_residual(zp, zq, T, top_k, top_p):
    """alpha(y) for every y and the replacement law, measured from accept_sample as a black box by bisection."""
    V = len(zp)

    def accepted(y, u):
        return O.accept_sample(np.array([[y]], dtype=np.int32), zp[None, None], T, zq[None, None], np.array([[u]]),
                               np.array([0.5]), top_k=top_k, top_p=top_p)[0][0] == 1

    alpha = np.zeros(V)
    for y in range(V):
        if accepted(y, 1.0):
            alpha[y] = 1.0
            continue
        lo, hi = 0.0, 1.0
        for _ in range(60):
            mid = 0.5 * (lo + hi)
            lo, hi = (mid, hi) if accepted(y, mid) else (lo, mid)
        alpha[y] = 0.5 * (lo + hi)
    y_rej = int(np.argmin(alpha))

    def tok(r):
        a, out, n = O.accept_sample(np.array([[y_rej]], dtype=np.int32), zp[None, None], T, zq[None, None],
                                    np.array([[1.0]]), np.array([r]), top_k=top_k, top_p=top_p)
        assert a[0] == 0
        return int(out[0, 0])

    cdf = np.zeros(V)
    for v in range(V):
        if tok(1.0 - 1e-15) <= v:
            cdf[v] = 1.0
            continue
        if tok(1e-300) > v:
            continue
        lo, hi = 0.0, 1.0
        for _ in range(60):
            mid = 0.5 * (lo + hi)
            lo, hi = (mid, hi) if tok(mid) <= v else (lo, mid)
        cdf[v] = 0.5 * (lo + hi)
    return alpha, np.diff(np.concatenate([[0.0], cdf]))


@pytest.mark.parametrize("seed,T,top_k,top_p", [(0, 0.6, 4, 1.0), (1, 0.6, 0, 0.8), (2, 1.0, 5, 0.9), (3, 0.6, 1, 1.0)])
def test_lossless_identity_against_the_truncated_distribution(seed, T, top_k, top_p):
    """The appendix lemma with p replaced by its truncation p': q(a) alpha(a) + (1 - gamma) p_res(a) = p'(a), with
    alpha and p_res measured from the oracle as a black box and p' from the brute force above on scipy's softmax."""
    r = np.random.default_rng(100 + seed)
    V = 8
    zp, zq = r.normal(size=V) * 2, r.normal(size=V) * 2
    p_trunc, keep = _brute_force(list(sp_softmax(zp / T)), top_k, top_p)
    p_trunc = np.array(p_trunc)
    q = sp_softmax(zq)
    alpha, pres = _alpha_and_residual(zp, zq, T, top_k, top_p)
    gamma = float((q * alpha).sum())
    np.testing.assert_allclose(q * alpha + (1.0 - gamma) * pres, p_trunc, atol=1e-9)
    np.testing.assert_allclose(gamma, np.minimum(p_trunc, q).sum(), atol=1e-9)
    assert all(alpha[v] < 1e-15 for v in range(V) if v not in keep)       # a draft outside the kept set never survives
    assert all(pres[v] < 1e-15 for v in range(V) if v not in keep)


def test_top_1_reproduces_the_greedy_rule():
    """Keeping only the most likely token makes p' one-hot at the argmax whatever the temperature: acceptance is
    then the greedy prefix match and the correction the argmax."""
    r = np.random.default_rng(5)
    B, k, V = 40, 6, 11
    zt = r.normal(size=(B, k, V))
    zq = r.normal(size=(B, k, V))
    tgt = zt.argmax(axis=2).astype(np.int32)
    drafts = tgt.copy()
    flip = r.random((B, k)) < 0.25
    drafts[flip] = (drafts[flip] + 1 + r.integers(0, V - 1, size=flip.sum())) % V
    u = r.random((B, k)) * 0.98 + 0.01
    a, out, n = O.accept_sample(drafts, zt, 0.6, zq, u, r.random(B), top_k=1)
    ag, outg, ng = O.accept_greedy(drafts, tgt)
    np.testing.assert_array_equal(a, ag)
    np.testing.assert_array_equal(out, outg)
    np.testing.assert_array_equal(n, ng)


def test_monte_carlo_first_token_follows_the_truncated_distribution():
    rng = np.random.default_rng(77)
    V, k, N, T, top_k, top_p = 10, 3, 80000, 0.6, 6, 0.9
    zp = rng.normal(size=(k, V))
    zq = zp + rng.normal(size=(k, V)) * 0.7
    q = sp_softmax(zq, axis=1)
    p0 = np.array(_brute_force(list(sp_softmax(zp[0] / T)), top_k, top_p)[0])
    drafts = np.stack([rng.choice(V, size=N, p=q[i]) for i in range(k)], axis=1).astype(np.int32)
    a, out, n = O.accept_sample(drafts, np.broadcast_to(zp, (N, k, V)), T, np.broadcast_to(zq, (N, k, V)),
                                rng.random((N, k)), rng.random(N), top_k=top_k, top_p=top_p)
    first = np.bincount(out[:, 0], minlength=V) / N
    sigma = np.sqrt(p0 * (1 - p0) / N)
    assert (np.abs(first - p0) < 4.5 * sigma + 1e-12).all()
    assert (first[p0 == 0] == 0).all()
