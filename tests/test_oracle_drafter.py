"""Pins for the drafter-side additions of the oracle: block attention with row states, the re-fill iteration,
the cache refresh after a verify step."""
import math

import numpy as np
import pytest

from oracle import deer_oracle as O

A, D_, M_ = O.ROW_ABSENT, O.ROW_DECODED, O.ROW_MASKED


def _dense_case(seed, B=2, k=6, Hq=4, Hkv=2, D=8, lens=(5, 19)):
    r = np.random.default_rng(seed)
    page = 16
    max_pages = max(-(-(n + k) // page) for n in lens)
    num_pages = B * max_pages + 3
    k_pool = r.normal(size=(num_pages, Hkv, page, D))
    v_pool = r.normal(size=(num_pages, Hkv, page, D))
    perm = r.permutation(num_pages)
    pt = np.full((B, max_pages), -1, dtype=np.int32)
    top = 0
    for b in range(B):
        for j in range(max_pages):
            pt[b, j] = perm[top]
            top += 1
    q = r.normal(size=(B, k, Hq, D))
    kb = r.normal(size=(B, k, Hkv, D))
    vb = r.normal(size=(B, k, Hkv, D))
    return q, kb, vb, k_pool, v_pool, pt, np.array(lens, dtype=np.int32)


def _scalar_attention(q, kb, vb, k_pool, v_pool, pt, lens, vis, scale):
    """Plain loops with an explicit visibility matrix vis[b][i][j] over the block rows (the prefix is always seen)."""
    B, k, Hq, D = q.shape
    Hkv = kb.shape[2]
    G = Hq // Hkv
    out = np.zeros_like(q)
    for b in range(B):
        n = int(lens[b])
        for i in range(k):
            for h in range(Hq):
                g = h // G
                keys, vals = [], []
                for t in range(n):
                    keys.append(k_pool[pt[b, t // 16], g, t % 16])
                    vals.append(v_pool[pt[b, t // 16], g, t % 16])
                for j in range(k):
                    if vis[b][i][j]:
                        keys.append(kb[b, j, g])
                        vals.append(vb[b, j, g])
                if not keys:
                    continue
                sc = [scale * sum(q[b, i, h, d] * kk[d] for d in range(D)) for kk in keys]
                mx = max(sc)
                w = [math.exp(s - mx) for s in sc]
                tot = sum(w)
                for d in range(D):
                    out[b, i, h, d] = sum(wj * vj[d] for wj, vj in zip(w, vals)) / tot
    return out


def test_all_masked_rows_are_the_plain_bidirectional_fill():
    q, kb, vb, kp, vp, pt, lens = _dense_case(0)
    ids = np.arange(2)
    plain = O.block_attention(q, kb, vb, kp, vp, pt, lens, ids, O.MASK_BIDIR, 0.3)
    st = np.full((2, 6), M_, dtype=np.int32)
    got = O.block_attention(q, kb, vb, kp, vp, pt, lens, ids, O.MASK_BIDIR, 0.3, row_state=st)
    np.testing.assert_array_equal(got, plain)
    # all decoded: they all see each other as well
    st[:] = D_
    np.testing.assert_array_equal(O.block_attention(q, kb, vb, kp, vp, pt, lens, ids, O.MASK_BIDIR, 0.3, row_state=st), plain)


@pytest.mark.parametrize("seed", range(4))
def test_row_states_against_scalar_loops_with_an_explicit_visibility_matrix(seed):
    q, kb, vb, kp, vp, pt, lens = _dense_case(10 + seed, lens=(0, 21) if seed == 3 else (5, 19))
    r = np.random.default_rng(seed)
    st = r.choice([A, D_, M_], size=(2, 6), p=[0.2, 0.4, 0.4]).astype(np.int32)
    st[0, 0], st[0, 1], st[1, 5] = D_, M_, A
    # the rule written out independently: masked sees whatever is there, decoded sees decoded, absent nothing
    vis = [[[(st[b, i] == M_ and st[b, j] != A) or (st[b, i] == D_ and st[b, j] == D_) for j in range(6)]
            for i in range(6)] for b in range(2)]
    want = _scalar_attention(q, kb, vb, kp, vp, pt, lens, vis, 0.35)
    got = O.block_attention(q, kb, vb, kp, vp, pt, lens, np.arange(2), O.MASK_BIDIR, 0.35, row_state=st)
    for b in range(2):
        for i in range(6):
            if st[b, i] == A:
                assert (got[b, i] == 0).all()
            else:
                np.testing.assert_allclose(got[b, i], want[b, i], atol=1e-12)
    with pytest.raises(ValueError):
        O.block_attention(q, kb, vb, kp, vp, pt, lens, np.arange(2), O.MASK_CAUSAL, 0.35, row_state=st)


def test_row_state_invariants():
    q, kb, vb, kp, vp, pt, lens = _dense_case(20)
    ids = np.arange(2)
    st = np.array([[D_, D_, M_, M_, M_, A], [M_, D_, M_, D_, A, A]], dtype=np.int32)
    base = O.block_attention(q, kb, vb, kp, vp, pt, lens, ids, O.MASK_BIDIR, 0.3, row_state=st)
    # (1) permuting the block rows (queries, keys, values and states together) permutes the outputs: no row's
    #     result depends on where in the block the other rows sit
    perm = np.array([4, 2, 0, 5, 1, 3])
    got = O.block_attention(q[:, perm], kb[:, perm], vb[:, perm], kp, vp, pt, lens, ids, O.MASK_BIDIR, 0.3, row_state=st[:, perm])
    np.testing.assert_allclose(got, base[:, perm], atol=1e-12)
    # (2) a decoded row's output does not change when the masked rows' keys and values do (it can be kept as context)
    kb2, vb2 = kb.copy(), vb.copy()
    kb2[st == M_] += 3.0
    vb2[st == M_] -= 2.0
    got = O.block_attention(q, kb2, vb2, kp, vp, pt, lens, ids, O.MASK_BIDIR, 0.3, row_state=st)
    np.testing.assert_allclose(got[st == D_], base[st == D_], atol=1e-12)
    assert np.abs(got[st == M_] - base[st == M_]).max() > 1e-3
    # (3) what sits in an absent row is never read
    kb3, vb3, q3 = kb.copy(), vb.copy(), q.copy()
    kb3[st == A], vb3[st == A], q3[st == A] = 1e6, -1e6, 7.0
    got = O.block_attention(q3, kb3, vb3, kp, vp, pt, lens, ids, O.MASK_BIDIR, 0.3, row_state=st)
    np.testing.assert_array_equal(got, base)
    # (4) the decoded rows alone equal a smaller bidirectional block made of just those rows
    dec = np.flatnonzero(st[0] == D_)
    small = O.block_attention(q[:1, dec], kb[:1, dec], vb[:1, dec], kp, vp, pt, lens, ids[:1], O.MASK_BIDIR, 0.3)
    np.testing.assert_allclose(base[0, dec], small[0], atol=1e-12)


def test_append_with_row_states_writes_the_decoded_rows_only():
    q, kb, vb, kp, vp, pt, lens = _dense_case(30)
    kv = O.PagedKV(kp.copy(), vp.copy(), pt, lens, np.array([2, 2]), np.arange(0), 0)
    st = np.array([[D_, D_, D_, A, A, A], [D_, M_, D_, A, A, A]], dtype=np.int32)
    before_k = kv.k_pool.copy()
    kv.append(np.arange(2), kb, vb, row_state=st)
    for b in range(2):
        for i in range(6):
            t = int(lens[b]) + i
            slot = kv.k_pool[pt[b, t // 16], :, t % 16]
            if st[b, i] == D_:
                np.testing.assert_array_equal(slot, kb[b, i])
            else:
                np.testing.assert_array_equal(slot, before_k[pt[b, t // 16], :, t % 16])


def test_refill_step_hand_worked():
    """Two sequences, k = 5, threshold log 0.5.
    seq 0: rows 0, 1 decoded already (tokens 7, 8); masked rows 2, 3, 4 with confidences 0.9, 0.4, 0.6 -> rows 2 and 4
           are decoded now, row 3 stays masked (1 left).
    seq 1: all masked with confidences 0.1, 0.3, 0.3, 0.2 and row 4 absent -> nobody reaches 0.5, so the most
           confident row is decoded, the lower index of the two at 0.3 (row 1); 3 left."""
    st = np.array([[D_, D_, M_, M_, M_], [M_, M_, M_, M_, A]], dtype=np.int32)
    tok = np.array([[7, 8, -1, -1, -1], [-1, -1, -1, -1, -1]], dtype=np.int32)
    ids = np.array([[50, 51, 52, 53, 54], [60, 61, 62, 63, 64]], dtype=np.int32)
    lp = np.log(np.array([[0.99, 0.99, 0.9, 0.4, 0.6], [0.1, 0.3, 0.3, 0.2, 0.99]]))
    st2, tok2, left = O.refill_step(st, tok, ids, lp, math.log(0.5))
    assert st2.tolist() == [[D_, D_, D_, M_, D_], [M_, D_, M_, M_, A]]
    assert tok2.tolist() == [[7, 8, 52, -1, 54], [-1, 61, -1, -1, -1]]
    assert left.tolist() == [1, 3]
    # the inputs are not modified
    assert st[0, 2] == M_ and tok[0, 2] == -1
    # -inf decodes every masked row at once (the single-step draft); an unreachable threshold one row per
    # iteration, most confident first, so k iterations finish any block
    st3, tok3, left3 = O.refill_step(st, tok, ids, lp, -math.inf)
    assert (st3[st == M_] == D_).all() and left3.tolist() == [0, 0] and tok3[1].tolist() == [60, 61, 62, 63, -1]
    cur, tk, order = st.copy(), tok.copy(), []
    for it in range(5):
        nxt, tk, left = O.refill_step(cur, tk, ids, lp, 1.0)
        order.append([int(i) for i in np.flatnonzero((nxt[1] == D_) & (cur[1] == M_))])
        cur = nxt
    assert order == [[1], [2], [3], [0], []] and left.tolist() == [0, 0]


def test_refresh_rows():
    st = O.refresh_rows(np.array([0, 3, 5]), 5)
    assert st.tolist() == [[A] * 5, [D_, D_, D_, A, A], [D_] * 5]
