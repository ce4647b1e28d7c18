"""Pins for the oracle's block attention: scalar brute force, invariants that
follow from the definition, and torch's CPU SDPA as a third opinion."""
import math

import numpy as np
import pytest
import torch

from oracle import deer_oracle as O


def _case(seed, B, k, Hq, Hkv, D, lens, page=16, sigma=1.0):
    r = np.random.default_rng(seed)
    lens = np.asarray(lens, dtype=np.int32)
    max_pages = max(1, int(-(-int(lens.max() + k) // page)))
    num_pages = B * max_pages + 3
    perm = r.permutation(num_pages)
    pt = np.full((B, max_pages), -1, dtype=np.int32)
    c = 0
    for b in range(B):
        for j in range(-(-int(lens[b]) // page)):
            pt[b, j] = perm[c]
            c += 1
    kp = r.normal(0, sigma, (num_pages, Hkv, page, D))
    vp = r.normal(0, sigma, (num_pages, Hkv, page, D))
    q = r.normal(0, sigma, (B, k, Hq, D))
    kb = r.normal(0, sigma, (B, k, Hkv, D))
    vb = r.normal(0, sigma, (B, k, Hkv, D))
    return q, kb, vb, kp, vp, pt, lens


def _brute(q, kb, vb, kp, vp, pt, lens, mask, scale, page=16):
    """Scalar loops straight from the definition of softmax attention."""
    B, k, Hq, D = q.shape
    Hkv = kb.shape[2]
    G = Hq // Hkv
    out = np.zeros((B, k, Hq, D))
    for b in range(B):
        n = int(lens[b])
        for h in range(Hq):
            g = h // G
            for i in range(k):
                scores, values = [], []
                for t in range(n):
                    pg, sl = pt[b, t // page], t % page
                    scores.append(scale * sum(q[b, i, h, d] * kp[pg, g, sl, d] for d in range(D)))
                    values.append(vp[pg, g, sl])
                for j in range(k):
                    if mask == O.MASK_CAUSAL and j > i:
                        continue
                    scores.append(scale * sum(q[b, i, h, d] * kb[b, j, g, d] for d in range(D)))
                    values.append(vb[b, j, g])
                mx = max(scores)
                w = [math.exp(s - mx) for s in scores]
                den = sum(w)
                for d in range(D):
                    out[b, i, h, d] = sum(wt * v[d] for wt, v in zip(w, values)) / den
    return out


@pytest.mark.parametrize("mask", [O.MASK_CAUSAL, O.MASK_BIDIR])
@pytest.mark.parametrize("B,k,Hq,Hkv,D,lens", [
    (2, 3, 4, 2, 8, [21, 5]),      # ragged, not page multiples
    (1, 1, 2, 2, 4, [16]),         # k = 1, G = 1, exact page
    (2, 4, 2, 1, 4, [0, 33]),      # empty prefix
])
def test_attention_matches_scalar_brute_force(mask, B, k, Hq, Hkv, D, lens):
    q, kb, vb, kp, vp, pt, lens = _case(7, B, k, Hq, Hkv, D, lens)
    scale = 1.0 / math.sqrt(D)
    got = O.block_attention(q, kb, vb, kp, vp, pt, lens, np.arange(B), mask, scale)
    want = _brute(q, kb, vb, kp, vp, pt, lens, mask, scale)
    np.testing.assert_allclose(got, want, rtol=0, atol=1e-12)


@pytest.mark.parametrize("mask", [O.MASK_CAUSAL, O.MASK_BIDIR])
def test_attention_matches_torch_sdpa(mask):
    B, k, Hq, Hkv, D = 2, 8, 8, 2, 64
    q, kb, vb, kp, vp, pt, lens = _case(11, B, k, Hq, Hkv, D, [70, 129])
    scale = 1.0 / math.sqrt(D)
    got = O.block_attention(q, kb, vb, kp, vp, pt, lens, np.arange(B), mask, scale)
    G = Hq // Hkv
    for b in range(B):
        n = int(lens[b])
        dense_k = np.stack([kp[pt[b, t // 16], :, t % 16] for t in range(n)] + [kb[b, j] for j in range(k)])
        dense_v = np.stack([vp[pt[b, t // 16], :, t % 16] for t in range(n)] + [vb[b, j] for j in range(k)])
        K = torch.from_numpy(dense_k).permute(1, 0, 2).repeat_interleave(G, dim=0)   # [Hq, n+k, D]
        Vv = torch.from_numpy(dense_v).permute(1, 0, 2).repeat_interleave(G, dim=0)
        Q = torch.from_numpy(q[b]).permute(1, 0, 2)                                    # [Hq, k, D]
        m = torch.ones(k, n + k, dtype=torch.bool)
        if mask == O.MASK_CAUSAL:
            m[:, n:] = torch.tril(torch.ones(k, k, dtype=torch.bool))
        ref = torch.nn.functional.scaled_dot_product_attention(Q, K, Vv, attn_mask=m, scale=scale)
        np.testing.assert_allclose(got[b], ref.permute(1, 0, 2).numpy(), rtol=0, atol=1e-11)


def test_all_equal_values_give_that_value():
    q, kb, vb, kp, vp, pt, lens = _case(3, 1, 4, 4, 2, 8, [40])
    vp[:] = 0.0
    vb[:] = 0.0
    vp[:, 0, :, :] = np.arange(8) * 0.25
    vb[:, :, 0, :] = np.arange(8) * 0.25
    vp[:, 1, :, :] = -1.5
    vb[:, :, 1, :] = -1.5
    out = O.block_attention(q, kb, vb, kp, vp, pt, lens, [0], O.MASK_CAUSAL, 0.3)
    np.testing.assert_allclose(out[0, :, :2, :], np.broadcast_to(np.arange(8) * 0.25, (4, 2, 8)), atol=1e-13)
    np.testing.assert_allclose(out[0, :, 2:, :], -1.5, atol=1e-13)


def test_one_dominant_key_returns_its_value():
    q, kb, vb, kp, vp, pt, lens = _case(4, 1, 2, 2, 1, 8, [37], sigma=0.1)
    t = 19
    q[:] = 0.0
    q[..., 0] = 1.0
    kp[..., 0] = 0.0
    kb[..., 0] = 0.0
    kp[pt[0, t // 16], 0, t % 16, 0] = 200.0
    out = O.block_attention(q, kb, vb, kp, vp, pt, lens, [0], O.MASK_BIDIR, 1.0)
    np.testing.assert_allclose(out[0, :, :, :], np.broadcast_to(vp[pt[0, t // 16], 0, t % 16], (2, 2, 8)), atol=1e-12)


def test_physical_page_permutation_is_invisible():
    q, kb, vb, kp, vp, pt, lens = _case(5, 2, 4, 4, 2, 8, [50, 23])
    a = O.block_attention(q, kb, vb, kp, vp, pt, lens, [0, 1], O.MASK_CAUSAL, 0.35)
    perm = np.random.default_rng(0).permutation(kp.shape[0])
    inv = np.argsort(perm)
    kp2, vp2 = kp[perm], vp[perm]          # new page p holds old page perm[p]
    pt2 = np.where(pt >= 0, inv[np.maximum(pt, 0)], -1).astype(np.int32)
    b = O.block_attention(q, kb, vb, kp2, vp2, pt2, lens, [0, 1], O.MASK_CAUSAL, 0.35)
    np.testing.assert_array_equal(a, b)


def test_causal_row0_ignores_later_rows_and_bidir_is_permutation_invariant():
    q, kb, vb, kp, vp, pt, lens = _case(6, 1, 5, 2, 2, 8, [18])
    a = O.block_attention(q, kb, vb, kp, vp, pt, lens, [0], O.MASK_CAUSAL, 0.35)
    kb2, vb2 = kb.copy(), vb.copy()
    kb2[:, 1:] += 3.0
    vb2[:, 1:] -= 2.0
    b = O.block_attention(q, kb2, vb2, kp, vp, pt, lens, [0], O.MASK_CAUSAL, 0.35)
    np.testing.assert_array_equal(a[0, 0], b[0, 0])
    assert np.abs(a[0, 1:] - b[0, 1:]).max() > 1e-3
    # the last causal row sees the whole block, exactly like a bidirectional row
    c = O.block_attention(q, kb, vb, kp, vp, pt, lens, [0], O.MASK_BIDIR, 0.35)
    np.testing.assert_allclose(a[0, -1], c[0, -1], atol=1e-14)
    assert np.abs(a[0, 0] - c[0, 0]).max() > 1e-4
    p = np.array([3, 0, 4, 1, 2])
    d = O.block_attention(q, kb[:, p], vb[:, p], kp, vp, pt, lens, [0], O.MASK_BIDIR, 0.35)
    np.testing.assert_allclose(c, d, atol=1e-13)


def test_seq_ids_select_rows_of_the_state():
    q, kb, vb, kp, vp, pt, lens = _case(8, 2, 2, 2, 1, 8, [9, 30])
    a = O.block_attention(q, kb, vb, kp, vp, pt, lens, [0, 1], O.MASK_CAUSAL, 0.35)
    b = O.block_attention(q[::-1], kb[::-1], vb[::-1], kp, vp, pt, lens, [1, 0], O.MASK_CAUSAL, 0.35)
    np.testing.assert_array_equal(a, b[::-1])
