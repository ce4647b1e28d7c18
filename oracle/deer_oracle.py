"""CPU oracle for the DEER draft-verify step.  TEST INFRASTRUCTURE ONLY.

A plain, slow, obviously-correct restatement of what the four library calls
compute, written from the paper (Section 3.2 "Inference", Eq. 5, Eq. 6,
Algorithm 1, Appendix "One-step lossless speculative sampling").  Only the
tests, the smoke check and the benchmark's ``cpu_baseline`` / reference arm may
import it; the CUDA path never does, and the two share no code.

All floating point is float64 (inputs are bf16/fp32 values widened exactly by
the caller).  NumPy matmul / exp / cumsum serve as steps; there is no tiling,
fusion or reordering beyond the definitions.

Every function here is pinned by ``tests/test_oracle_*.py`` against brute
force, closed forms or invariants; none is "parity unpinned".
"""
from __future__ import annotations

import numpy as np

MASK_CAUSAL = 0
MASK_BIDIR = 1


# --------------------------------------------------------------------------
# paged cache access
# --------------------------------------------------------------------------

def gather_prefix(pool, page_table_row, n, page_size):
    """Committed tokens 0..n-1 of one sequence as a dense [n, Hkv, D] array.
    Token t lives at pool[page_table_row[t // page_size], :, t % page_size, :]."""
    npg = -(-n // page_size)
    pages = pool[np.asarray(page_table_row[:npg], dtype=np.int64)]      # [npg, Hkv, page, D]
    Hkv, D = pool.shape[1], pool.shape[3]
    return np.transpose(pages, (0, 2, 1, 3)).reshape(npg * page_size, Hkv, D)[:n]


# --------------------------------------------------------------------------
# (1) block attention  -- Section 3.2: the verifier evaluates
#     p_AR(. | x_{1:j+i-1}) for i=1..k in one pass (causal inside the block);
#     the drafter fills all k masked positions jointly from x_{1:j}
#     (bidirectional inside the block).
# --------------------------------------------------------------------------

def block_attention(q, k_blk, v_blk, k_pool, v_pool, page_table, seq_len, seq_ids, mask, scale, page_size=16):
    """q [B,k,Hq,D]; k_blk,v_blk [B,k,Hkv,D]; pools [P,Hkv,page,D] -> [B,k,Hq,D] float64.

    Row i of sequence b attends to its committed prefix (cache tokens
    0..n_b-1) and to block rows j with j <= i (causal) or all j (bidirectional).
    Query head h reads KV head h // (Hq/Hkv)."""
    q = np.asarray(q, dtype=np.float64)
    k_blk = np.asarray(k_blk, dtype=np.float64)
    v_blk = np.asarray(v_blk, dtype=np.float64)
    B, k, Hq, D = q.shape
    Hkv = k_blk.shape[2]
    G = Hq // Hkv
    out = np.zeros((B, k, Hq, D), dtype=np.float64)
    for b in range(B):
        s = int(seq_ids[b])
        n = int(seq_len[s])
        kp = np.asarray(gather_prefix(k_pool, page_table[s], n, page_size), dtype=np.float64)
        vp = np.asarray(gather_prefix(v_pool, page_table[s], n, page_size), dtype=np.float64)
        keys = np.concatenate([kp, k_blk[b]], axis=0)       # [n+k, Hkv, D]
        vals = np.concatenate([vp, v_blk[b]], axis=0)
        allowed = np.ones((k, n + k), dtype=bool)
        if mask == MASK_CAUSAL:
            for i in range(k):
                allowed[i, n + i + 1:] = False
        for h in range(Hq):
            g = h // G
            sc = scale * (q[b, :, h, :] @ keys[:, g, :].T)  # [k, n+k]
            sc = np.where(allowed, sc, -np.inf)
            m = sc.max(axis=1, keepdims=True)
            w = np.exp(sc - m)
            out[b, :, h, :] = (w @ vals[:, g, :]) / w.sum(axis=1, keepdims=True)
    return out


# --------------------------------------------------------------------------
# (2) LM head + selection -- logits z = H W^T give p_AR = softmax(z / T)
#     (Eq. 5's numerator); at temperature 0 the distribution is the one-hot
#     on argmax z.
# --------------------------------------------------------------------------

def lm_logits(h, w):
    """h [M,hid], w [V,hid] -> z [M,V] float64."""
    return np.asarray(h, dtype=np.float64) @ np.asarray(w, dtype=np.float64).T


def select_argmax(z):
    """Per row, the lowest index among the maxima."""
    return np.argmax(np.asarray(z), axis=1).astype(np.int32)


def logsumexp(z, temperature=1.0):
    """Per row log sum_v exp(z[v] / T)."""
    zt = np.asarray(z, dtype=np.float64) / float(temperature)
    m = zt.max(axis=1)
    return m + np.log(np.exp(zt - m[:, None]).sum(axis=1))


def max_logprob(z):
    """Per row log-probability of the argmax token at temperature 1."""
    z = np.asarray(z, dtype=np.float64)
    return z.max(axis=1) - logsumexp(z, 1.0)


def top2_gap(z):
    """Per row difference between the largest and second-largest logit."""
    part = np.partition(np.asarray(z, dtype=np.float64), -2, axis=1)
    return part[:, -1] - part[:, -2]


# --------------------------------------------------------------------------
# (3) acceptance rule -- Eq. 5 (acceptance probability), Eq. 6 / Appendix
#     residual distribution, Algorithm 1's inner loop, stopped at the first
#     rejection because later rows of the parallel pass were conditioned on
#     the rejected draft token.
# --------------------------------------------------------------------------

def _truncate_at_eos(out_row, n_out, accept_len, eos_id):
    """Algorithm 1's EOS break: nothing is emitted after the first EOS."""
    if eos_id < 0:
        return n_out, accept_len
    for i in range(n_out):
        if out_row[i] == eos_id:
            out_row[i + 1:] = -1
            return i + 1, min(accept_len, i + 1)
    return n_out, accept_len


def accept_greedy(draft_ids, target_ids, eos_id=-1, bonus=False):
    """Temperature 0: p_AR is one-hot on the target argmax, so alpha_i is 1 if
    draft == target and 0 otherwise, and the residual is that one-hot.
    Returns (accept_len [B], out_ids [B,k] padded with -1, n_out [B]).

    bonus: the block's k rows hold k-1 drafts (draft_ids[:, k-1] is ignored); row i
    judges draft i, and when all k-1 are accepted the last row, whose input was the
    last draft, gives one more token -- the parallel pass has p_AR(. | all drafts)
    anyway.  Every block then emits accept_len + 1 tokens."""
    draft_ids = np.asarray(draft_ids)
    target_ids = np.asarray(target_ids)
    B, k = draft_ids.shape
    kd = k - 1 if bonus else k                  # drafts under test
    accept_len = np.zeros(B, dtype=np.int32)
    out_ids = np.full((B, k), -1, dtype=np.int32)
    n_out = np.zeros(B, dtype=np.int32)
    for b in range(B):
        a = 0
        while a < kd and draft_ids[b, a] == target_ids[b, a]:
            out_ids[b, a] = draft_ids[b, a]
            a += 1
        n = a
        if a < k:                               # a correction, or (bonus, a == k-1) the extra token
            out_ids[b, a] = target_ids[b, a]
            n = a + 1
        n, a = _truncate_at_eos(out_ids[b], n, a, eos_id)
        accept_len[b] = a
        n_out[b] = n
    return accept_len, out_ids, n_out


def softmax_f64(z, temperature=1.0):
    zt = np.asarray(z, dtype=np.float64) / float(temperature)
    e = np.exp(zt - zt.max())
    return e / e.sum()


def residual_distribution(p, q):
    """Unnormalised residual max(0, p - q) = p - min(p, q) and its mass 1 - gamma."""
    res = np.maximum(0.0, p - q)
    return res, res.sum()


def inverse_cdf(weights, total, r):
    """Smallest index v with sum_{v' <= v} weights[v'] >= r * total."""
    cdf = np.cumsum(weights)
    v = int(np.searchsorted(cdf, r * total, side="left"))
    if v >= len(weights):                       # rounding left cdf[-1] just below r * total
        v = int(np.flatnonzero(np.asarray(weights) > 0)[-1])
    return v


def accept_sample(draft_ids, target_logits, temperature, draft_logits, u, r, eos_id=-1, bonus=False):
    """Speculative rejection sampling over one block per sequence.

    For i = 0..k-1: p = softmax(target_logits[b,i] / T), q = softmax(draft_logits[b,i]);
    alpha_i = min(1, p[y_i] / q[y_i]) (Eq. 5); accept iff u[b,i] <= alpha_i.  At the
    first rejection draw one token from the normalised residual max(0, p - q)
    (Eq. 6) by inverse CDF with r[b] in vocabulary order and stop; if the residual
    mass is exactly zero, draw from p instead.  No extra token is emitted when all
    k drafts are accepted.

    bonus: the k rows hold k-1 drafts (column k-1 of draft_ids, draft_logits and u is
    ignored); when all are accepted one more token is drawn from the last row's p
    itself by the same inverse CDF with r[b] (nothing was proposed there, so there
    is nothing to reject: the residual of p against q = 0 is p)."""
    draft_ids = np.asarray(draft_ids)
    B, k = draft_ids.shape
    kd = k - 1 if bonus else k
    accept_len = np.zeros(B, dtype=np.int32)
    out_ids = np.full((B, k), -1, dtype=np.int32)
    n_out = np.zeros(B, dtype=np.int32)
    for b in range(B):
        a = 0
        n = 0
        for i in range(kd):
            y = int(draft_ids[b, i])
            zp = np.asarray(target_logits[b, i], dtype=np.float64) / float(temperature)
            zq = np.asarray(draft_logits[b, i], dtype=np.float64)
            logp = zp - (zp.max() + np.log(np.exp(zp - zp.max()).sum()))
            logq = zq - (zq.max() + np.log(np.exp(zq - zq.max()).sum()))
            log_alpha = min(0.0, logp[y] - logq[y])
            if np.log(np.float64(u[b, i])) <= log_alpha:
                out_ids[b, i] = y
                a += 1
                n += 1
                continue
            p = np.exp(logp)
            q = np.exp(logq)
            res, S = residual_distribution(p, q)
            if S > 0.0:
                out_ids[b, i] = inverse_cdf(res, S, float(r[b]))
            else:
                out_ids[b, i] = inverse_cdf(p, p.sum(), float(r[b]))
            n += 1
            break
        if bonus and a == kd:
            p = softmax_f64(target_logits[b, kd], temperature)
            out_ids[b, kd] = inverse_cdf(p, p.sum(), float(r[b]))
            n += 1
        n, a = _truncate_at_eos(out_ids[b], n, a, eos_id)
        accept_len[b] = a
        n_out[b] = n
    return accept_len, out_ids, n_out


# --------------------------------------------------------------------------
# (4) KV cache reserve / append / commit -- the chosen tokens join the prefix
#     (Section 3.2, the step after Eq. 6; Algorithm 1's update of j).  Rows of
#     the block beyond the kept length are dropped.
# --------------------------------------------------------------------------

class PagedKV:
    """Paged cache state on plain arrays.  Free pages sit in
    ``free_stack[0:free_top]``; a pop takes the top entry."""

    def __init__(self, k_pool, v_pool, page_table, seq_len, n_pages, free_stack, free_top, page_size=16):
        self.k_pool = k_pool
        self.v_pool = v_pool
        self.page_table = np.array(page_table, dtype=np.int32)
        self.seq_len = np.array(seq_len, dtype=np.int32)
        self.n_pages = np.array(n_pages, dtype=np.int32)
        self.free_stack = np.array(free_stack, dtype=np.int32)
        self.free_top = int(np.asarray(free_top).reshape(-1)[0])
        self.page_size = page_size

    def reserve(self, seq_ids, k):
        """Map enough pages to hold seq_len + k tokens: sequences in the order
        given, logical pages ascending, each popped from the free stack.
        Returns False (state untouched) if the free stack is too small."""
        need_total = 0
        for s in seq_ids:
            need = -(-(int(self.seq_len[s]) + k) // self.page_size)
            need_total += max(0, need - int(self.n_pages[s]))
        if need_total > self.free_top or any(
                -(-(int(self.seq_len[s]) + k) // self.page_size) > self.page_table.shape[1] for s in seq_ids):
            return False
        for s in seq_ids:
            need = -(-(int(self.seq_len[s]) + k) // self.page_size)
            while self.n_pages[s] < need:
                self.free_top -= 1
                self.page_table[s, self.n_pages[s]] = self.free_stack[self.free_top]
                self.n_pages[s] += 1
        return True

    def append(self, seq_ids, k_blk, v_blk):
        """Write block rows at token positions seq_len .. seq_len+k-1 (lengths unchanged)."""
        B, k = k_blk.shape[0], k_blk.shape[1]
        for b in range(B):
            s = int(seq_ids[b])
            for i in range(k):
                t = int(self.seq_len[s]) + i
                pg = self.page_table[s, t // self.page_size]
                self.k_pool[pg, :, t % self.page_size, :] = k_blk[b, i]
                self.v_pool[pg, :, t % self.page_size, :] = v_blk[b, i]

    def commit(self, seq_ids, keep):
        """seq_len += keep; pages wholly beyond the new length go back to the
        free stack: sequences in the order given, logical pages descending."""
        for b, s in enumerate(seq_ids):
            s = int(s)
            self.seq_len[s] += int(keep[b])
            need = -(-int(self.seq_len[s]) // self.page_size)
            while self.n_pages[s] > need:
                self.n_pages[s] -= 1
                self.free_stack[self.free_top] = self.page_table[s, self.n_pages[s]]
                self.page_table[s, self.n_pages[s]] = -1
                self.free_top += 1

    def gather(self, s):
        n = int(self.seq_len[s])
        return (gather_prefix(self.k_pool, self.page_table[s], n, self.page_size),
                gather_prefix(self.v_pool, self.page_table[s], n, self.page_size))


# --------------------------------------------------------------------------
# (5) Algorithm 1's outer loop (it runs until an EOS is emitted; the chosen
#     tokens join the prefix and j is updated to its new length).  One call of
#     emit() is the book-keeping of one pass of that loop for every sequence:
#     what was chosen in this block joins the sequence's output, the sequence
#     ends at an EOS or at a length limit, and only the accepted draft tokens
#     that were really emitted stay in the KV cache.
# --------------------------------------------------------------------------

class DecodeState:
    """Output tokens of every sequence over the passes of the loop."""

    def __init__(self, B, max_new):
        self.max_new = int(max_new)
        self.tokens = np.full((B, max_new), -1, dtype=np.int32)
        self.n_tokens = np.zeros(B, dtype=np.int32)
        self.finished = np.zeros(B, dtype=np.int32)

    def emit(self, accept_len, out_ids, n_out, eos_id=-1, pending=False):
        """Append this block's chosen tokens (``out_ids[b][:n_out[b]]``, already cut
        after an EOS by the acceptance rule).  A sequence that has finished emits
        nothing and keeps nothing.  Returns keep [B]: cache rows to commit.

        pending: row 0 of the block was the token emitted last (its keys and values
        were not in the cache yet) and rows 1.. the drafts, so one more row stays:
        that token's, followed by the accepted drafts'."""
        B = self.tokens.shape[0]
        keep = np.zeros(B, dtype=np.int32)
        for b in range(B):
            if self.finished[b]:
                continue
            room = self.max_new - int(self.n_tokens[b])
            m = min(int(n_out[b]), room)
            for i in range(m):
                self.tokens[b, self.n_tokens[b] + i] = out_ids[b][i]
            self.n_tokens[b] += m
            keep[b] = min(int(accept_len[b]), m) + (1 if pending else 0)
            hit_eos = eos_id >= 0 and any(int(out_ids[b][i]) == eos_id for i in range(m))
            if hit_eos or self.n_tokens[b] >= self.max_new:
                self.finished[b] = 1
        return keep


# --------------------------------------------------------------------------
# (6) The rest of a verifier layer around the block attention.  The paper takes
#     its verifiers (Qwen3) as given; this is the public pre-norm decoder layer of
#     that family written out: RMSNorm, Q/K/V projections, a per-head RMSNorm of
#     q and k, rotary position embedding (half-split pairing), attention, output
#     projection, residual; RMSNorm, gate/up projections, SiLU(gate) * up, down
#     projection, residual.  All in float64; the caller rounds where the device
#     stores bf16.
# --------------------------------------------------------------------------

def linear(x, w):
    """y[m][n] = sum_c x[m][c] * w[n][c]  (weights stored [out][in])."""
    return np.asarray(x, dtype=np.float64) @ np.asarray(w, dtype=np.float64).T


def rmsnorm(x, gamma, eps):
    """y = x / sqrt(mean(x^2) + eps) * gamma over the last axis."""
    x = np.asarray(x, dtype=np.float64)
    ms = (x * x).mean(axis=-1, keepdims=True)
    return x / np.sqrt(ms + eps) * np.asarray(gamma, dtype=np.float64)


def rope(x, positions, theta):
    """Rotary embedding of x [..., T, H, D] at integer positions [..., T]: dimension
    d < D/2 is paired with d + D/2 and the pair is rotated by the angle
    pos * theta^(-2d / D)."""
    x = np.asarray(x, dtype=np.float64)
    D = x.shape[-1]
    half = D // 2
    inv_freq = float(theta) ** (-np.arange(half, dtype=np.float64) * 2.0 / D)
    ang = np.asarray(positions, dtype=np.float64)[..., None, None] * inv_freq          # [..., T, 1, half]
    c, s = np.cos(ang), np.sin(ang)
    a, b = x[..., :half], x[..., half:]
    return np.concatenate([a * c - b * s, b * c + a * s], axis=-1)


def swiglu(gate, up):
    """SiLU(gate) * up with SiLU(g) = g / (1 + exp(-g))."""
    g = np.asarray(gate, dtype=np.float64)
    return g / (1.0 + np.exp(-g)) * np.asarray(up, dtype=np.float64)
