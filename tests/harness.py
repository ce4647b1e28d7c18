"""Shared test harness: draws one step's inputs (workload module), computes the
expected results with the CPU oracle, and -- for the GPU tests -- runs the same
inputs through the C-ABI binding.  Decisions that floating-point reordering
could flip (argmax near-ties, u against alpha, r against a CDF edge) are made
robust here by re-drawing the input until the oracle's own margin is clear."""
from __future__ import annotations

import math
from types import SimpleNamespace

import numpy as np
import torch

from oracle import deer_oracle as O
from paper_2512_15176_b200 import workload as W

ARGMAX_MARGIN = 1e-2      # planted rows are re-drawn until the oracle's top-2 gap exceeds this
ARGMAX_EXEMPT = 1e-3      # a differing id is tolerated only below this oracle top-2 gap
ALPHA_MARGIN = 1e-3       # |log u - log alpha| must exceed this
ATTN_MAX_ABS, ATTN_MEAN_ABS = 2e-2, 2e-3
ATTN_MAX_REL, ATTN_MEAN_REL = 2e-2, 5e-3     # relative to max|ref| / mean|ref|


def f64(t):
    return t.to(torch.float64).numpy() if torch.is_tensor(t) else np.asarray(t, dtype=np.float64)


def draw_state(cfg: W.StepConfig, lengths=None, stress=False):
    """Cache state and pools.  ``stress`` draws Q/K/V ~ N(0,1) so that scores
    are O(1) and the absolute tolerances bite."""
    lengths = W.seq_lengths(cfg) if lengths is None else np.asarray(lengths, dtype=np.int32)
    lay = W.kv_layout(cfg, lengths)
    kp, vp = W.kv_pools(cfg, lay.num_pages, sigma=1.0 if stress else None)
    return SimpleNamespace(cfg=cfg, lengths=lengths, layout=lay, k_pool=kp, v_pool=vp, stress=stress)


def draw_block(cfg, step=0, stress=False):
    q, kb, vb = W.block_qkv(cfg, step, sigma=1.0 if stress else None)
    return q, kb, vb


def oracle_kv(st):
    lay = st.layout
    return O.PagedKV(f64(st.k_pool).astype(np.float32), f64(st.v_pool).astype(np.float32), lay.page_table, lay.seq_len,
                     lay.n_pages, lay.free_stack, lay.free_top)


def oracle_attention(cfg, okv, q, kb, vb):
    return O.block_attention(f64(q), f64(kb), f64(vb), okv.k_pool, okv.v_pool, okv.page_table, okv.seq_len,
                             np.arange(cfg.B), cfg.mask, 1.0 / math.sqrt(cfg.D))


def check_attention(got_bf16, want64, label=""):
    got = f64(got_bf16)
    err = np.abs(got - want64)
    ref_max, ref_mean = np.abs(want64).max(), np.abs(want64).mean()
    assert np.isfinite(got).all(), f"{label}: non-finite attention output"
    assert err.max() <= ATTN_MAX_ABS and err.mean() <= ATTN_MEAN_ABS, f"{label}: abs err max {err.max():.3e} mean {err.mean():.3e}"
    assert err.max() <= ATTN_MAX_REL * ref_max + 1e-30, f"{label}: max err {err.max():.3e} vs max|ref| {ref_max:.3e}"
    assert err.mean() <= ATTN_MEAN_REL * ref_mean + 1e-30, f"{label}: mean err {err.mean():.3e} vs mean|ref| {ref_mean:.3e}"


def draw_hidden_with_margin(cfg, w64, step=0, margin=ARGMAX_MARGIN):
    """Hidden states whose oracle top-2 logit gap exceeds ``margin`` in every
    row; rows that fail are replaced by the same row of the next re-draw.
    Returns (h bf16 [M,hid], z float64 [M,V], redraws)."""
    h = W.hidden(cfg, step, 0).clone()
    z = O.lm_logits(f64(h), w64)
    redraws = 0
    for attempt in range(1, 50):
        bad = np.flatnonzero(O.top2_gap(z) < margin)
        if bad.size == 0:
            break
        h2 = W.hidden(cfg, step, attempt)
        h[torch.from_numpy(bad)] = h2[torch.from_numpy(bad)]
        z[bad] = O.lm_logits(f64(h[torch.from_numpy(bad)]), w64)
        redraws += bad.size
    else:
        raise AssertionError("could not clear argmax margins")
    return h, z, redraws


def check_ids(got, want, z64, label=""):
    got, want = np.asarray(got).reshape(-1), np.asarray(want).reshape(-1)
    diff = np.flatnonzero(got != want)
    if diff.size:
        gaps = O.top2_gap(z64[diff])
        assert (gaps < ARGMAX_EXEMPT).all(), f"{label}: argmax differs at rows {diff[:8]} with oracle top-2 gaps {gaps[:8]}"
        # and the id chosen instead must be the runner-up within the same gap
        for r_, g in zip(diff, got[diff]):
            assert z64[r_].max() - z64[r_, g] < ARGMAX_EXEMPT, f"{label}: row {r_} picked a non-maximal id"


def check_logits(got_f32, z64, label=""):
    err = np.abs(f64(got_f32) - z64)
    assert err.max() <= 2e-2 and err.mean() <= 2e-3, f"{label}: logits err max {err.max():.3e} mean {err.mean():.3e}"
    # fp32 accumulation of exact bf16 products: the error should sit near 1e-5, far inside the stated bar
    assert err.max() <= 1e-3, f"{label}: logits err max {err.max():.3e} (expected ~1e-5)"


R_MARGIN = 1e-4           # r * S keeps this fraction of S away from the edges of the drawn token's cell


def truncated_p(z32_row, T, top_k, top_p):
    p = O.softmax_f64(z32_row, T)
    if top_k or top_p < 1.0:
        p, _ = O.truncate_distribution(p, top_k, top_p)
    return p


def sampling_inputs(cfg, zt32, step=0, r_margin=R_MARGIN, bonus=False, top_k=0, top_p=1.0):
    """Drafter logits, sampled drafts, uniforms with cleared margins.
    ``zt32`` are the target logits (fp32 values, [B,k,V]) the oracle will use.
    bonus: the last row holds no draft; when the k-1 drafts before it are all
    accepted, r is cleared against the edges of that row's own CDF.
    top_k / top_p: the verifier's distribution is truncated first."""
    T = float(np.float32(cfg.temperature))
    ql = W.draft_logits(cfg, step)
    drafts = W.sample_drafts(ql, cfg.seed, step)
    u = W.uniform_open(cfg.seed, f"u{step}", (cfg.B, cfg.k)).numpy()
    r = W.uniform_open(cfg.seed, f"r{step}", (cfg.B,)).numpy()
    gen = W.rng(cfg.seed, f"redraw{step}")
    redraws = 0
    qn = ql.numpy()
    def clear_r(b, wts, tot):
        nonlocal redraws
        cdf = np.cumsum(wts)
        while True:
            t = float(r[b]) * tot
            v = min(int(np.searchsorted(cdf, t, side="left")), cfg.V - 1)
            lo = cdf[v - 1] if v > 0 else 0.0
            if t - lo > r_margin * tot and cdf[v] - t > r_margin * tot:
                return
            r[b] = np.float32((int(gen.integers(0, 1 << 24)) + 0.5) / (1 << 24))
            redraws += 1

    kd = cfg.k - 1 if bonus else cfg.k
    for b in range(cfg.B):
        rejected = False
        for i in range(kd):
            y = int(drafts[b, i])
            zp = zt32[b, i].astype(np.float64) / T
            zq = qn[b, i].astype(np.float64)
            if top_k or top_p < 1.0:
                py = truncated_p(zt32[b, i], T, top_k, top_p)[y]
                logp_y = math.log(py) if py > 0 else -math.inf
            else:
                logp_y = zp[y] - O.logsumexp(zp[None], 1.0)[0]
            la = min(0.0, logp_y - (zq[y] - O.logsumexp(zq[None], 1.0)[0]))
            while abs(math.log(float(u[b, i])) - la) < ALPHA_MARGIN:
                u[b, i] = np.float32((int(gen.integers(0, 1 << 24)) + 0.5) / (1 << 24))
                redraws += 1
            if math.log(float(u[b, i])) > la:          # first rejection: clear r against the residual CDF edges
                p = truncated_p(zt32[b, i], T, top_k, top_p)
                qd = O.softmax_f64(qn[b, i], 1.0)
                res, S = O.residual_distribution(p, qd)
                wts, tot = (res, S) if S > 0 else (p, p.sum())
                clear_r(b, wts, tot)
                rejected = True
                break
        if bonus and not rejected:
            p = truncated_p(zt32[b, kd], T, top_k, top_p)
            clear_r(b, p, p.sum())
    return ql, drafts, torch.from_numpy(u), torch.from_numpy(r), redraws


# ---------------------------------------------------------------- GPU side

def gpu_kv(st, device="cuda"):
    from paper_2512_15176_b200 import binding as L
    return L.KVCache.from_layout(st.layout, st.k_pool, st.v_pool, device)


def kv_state_equal(kv, okv, label=""):
    """Bit-exact comparison of the cache's observable state."""
    np.testing.assert_array_equal(kv.seq_len.cpu().numpy(), okv.seq_len, err_msg=f"{label} seq_len")
    np.testing.assert_array_equal(kv.n_pages.cpu().numpy(), okv.n_pages, err_msg=f"{label} n_pages")
    top = int(kv.free_top.cpu().item())
    assert top == okv.free_top, f"{label} free_top {top} vs {okv.free_top}"
    np.testing.assert_array_equal(kv.free_stack.cpu().numpy()[:top], okv.free_stack[:top], err_msg=f"{label} free stack")
    pt = kv.page_table.cpu().numpy()
    for s in range(pt.shape[0]):
        npg = int(okv.n_pages[s])
        np.testing.assert_array_equal(pt[s, :npg], okv.page_table[s, :npg], err_msg=f"{label} page table row {s}")


def kv_contents_equal(kv, okv, seqs=None, label=""):
    kp = kv.k_pool.cpu().to(torch.float32).numpy()
    vp = kv.v_pool.cpu().to(torch.float32).numpy()
    pt = kv.page_table.cpu().numpy()
    sl = kv.seq_len.cpu().numpy()
    for s in (range(pt.shape[0]) if seqs is None else seqs):
        gk = O.gather_prefix(kp, pt[s], int(sl[s]), 16)
        gv = O.gather_prefix(vp, pt[s], int(sl[s]), 16)
        ok, ov = okv.gather(s)
        np.testing.assert_array_equal(gk, ok, err_msg=f"{label} K contents seq {s}")
        np.testing.assert_array_equal(gv, ov, err_msg=f"{label} V contents seq {s}")


def nucleus_margin_ok(z32, T, top_k, top_p, margin=1e-4):
    """True if, for every row of z32 [M,V], the running mass of the (top-k-renormalised) distribution keeps `margin`
    away from top_p on both sides of the tie group at which it is reached -- so that summation order cannot move
    the nucleus's edge."""
    for row in z32:
        p = O.softmax_f64(row, T)
        if top_k:
            p, _ = O.truncate_distribution(p, top_k, 1.0)
        vals = np.sort(p[p > 0])[::-1]
        cum = np.cumsum(vals)
        i = min(int(np.searchsorted(cum, top_p, side="left")), len(vals) - 1)
        lo = np.flatnonzero(vals == vals[i])
        before = cum[lo[0] - 1] if lo[0] > 0 else 0.0
        incl = cum[lo[-1]]
        if top_p - before < margin or (incl - top_p < margin and lo[-1] < len(vals) - 1):
            return False
    return True


def sampled_oracle_kv(kv, seqs, extra_tokens, page_size=16):
    """An oracle cache holding only the sequences ``seqs`` of the device cache ``kv`` (their pages copied from the
    device pools into a compact pool, page ids renumbered, room for ``extra_tokens`` more tokens each): what the
    oracle needs to follow a few sequences of a batch whose pools are too large to draw or hold on the host.
    Sequence j of the result is sequence seqs[j] of the device cache."""
    pt = kv.page_table.cpu().numpy()
    sl = kv.seq_len.cpu().numpy()
    npg = kv.n_pages.cpu().numpy()
    Hkv, D = kv.k_pool.shape[1], kv.k_pool.shape[3]
    per_seq = [int(npg[s]) + -(-extra_tokens // page_size) + 1 for s in seqs]
    total = sum(per_seq)
    max_pages = max(per_seq)
    k_pool = np.zeros((total, Hkv, page_size, D), dtype=np.float32)
    v_pool = np.zeros((total, Hkv, page_size, D), dtype=np.float32)
    table = np.full((len(seqs), max_pages), -1, dtype=np.int32)
    nxt = 0
    for j, s in enumerate(seqs):
        ids = torch.from_numpy(pt[s, :npg[s]].astype(np.int64)).to(kv.k_pool.device)
        k_pool[nxt:nxt + npg[s]] = kv.k_pool[ids].float().cpu().numpy()
        v_pool[nxt:nxt + npg[s]] = kv.v_pool[ids].float().cpu().numpy()
        table[j, :npg[s]] = np.arange(nxt, nxt + npg[s])
        nxt += int(npg[s])
    free = np.arange(total - 1, nxt - 1, -1, dtype=np.int32)          # the unused pages, popped in ascending order
    stack = np.zeros(total, dtype=np.int32)
    stack[:free.size] = free
    return O.PagedKV(k_pool, v_pool, table, sl[list(seqs)], npg[list(seqs)], stack, free.size)
