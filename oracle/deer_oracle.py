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

# states of a block row in the drafter's partially filled block (block_attention's row_state)
ROW_ABSENT = -1      # no token there: neither a query nor a key
ROW_DECODED = 0      # a fixed token: context for the rows that are still masked
ROW_MASKED = 1       # still a mask token: to be (re-)filled


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

def block_visibility(k, mask, row_state=None):
    """allowed[i, j]: may block row i see block row j?  Causal: j <= i.  Bidirectional: every j.  Bidirectional
    with row states (the drafter's block while it is being filled over several iterations, Section 4 "Generative
    capabilities"; the drafter-side cache the appendix on the DLLM KV cache looks forward to): a masked row sees
    every row that holds something (decoded or masked -- the joint fill of Section 3.2); a decoded row sees the
    decoded rows only, so that what is computed for it never depends on positions that may still change and can
    be kept as context; an absent row sees nothing and nobody sees it."""
    allowed = np.ones((k, k), dtype=bool)
    if mask == MASK_CAUSAL:
        if row_state is not None:
            raise ValueError("row states belong to the bidirectional (drafter) mask")
        for i in range(k):
            allowed[i, i + 1:] = False
        return allowed
    if row_state is None:
        return allowed
    st = np.asarray(row_state)
    for i in range(k):
        for j in range(k):
            if st[i] == ROW_MASKED:
                allowed[i, j] = st[j] != ROW_ABSENT
            elif st[i] == ROW_DECODED:
                allowed[i, j] = st[j] == ROW_DECODED
            else:
                allowed[i, j] = False
    return allowed


def block_attention(q, k_blk, v_blk, k_pool, v_pool, page_table, seq_len, seq_ids, mask, scale, page_size=16,
                    row_state=None):
    """q [B,k,Hq,D]; k_blk,v_blk [B,k,Hkv,D]; pools [P,Hkv,page,D] -> [B,k,Hq,D] float64.

    Row i of sequence b attends to its committed prefix (cache tokens
    0..n_b-1) and to block rows j with j <= i (causal) or all j (bidirectional).
    Query head h reads KV head h // (Hq/Hkv).
    row_state [B,k] (bidirectional only): see block_visibility; the output rows of
    absent positions are zero."""
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
        allowed[:, n:] = block_visibility(k, mask, None if row_state is None else row_state[b])
        present = np.ones(k, dtype=bool) if row_state is None else np.asarray(row_state[b]) != ROW_ABSENT
        allowed[~present] = True                      # computed like any row, then zeroed: nothing is defined there
        for h in range(Hq):
            g = h // G
            sc = scale * (q[b, :, h, :] @ keys[:, g, :].T)  # [k, n+k]
            sc = np.where(allowed, sc, -np.inf)
            m = sc.max(axis=1, keepdims=True)
            w = np.exp(sc - m)
            o = (w @ vals[:, g, :]) / w.sum(axis=1, keepdims=True)
            out[b, :, h, :] = np.where(present[:, None], o, 0.0)
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


def truncate_distribution(p, top_k=0, top_p=1.0):
    """Top-k / nucleus truncation of a probability vector, as samplers apply it to the verifier's distribution at
    temperature > 0 (the setting of the paper's Table 1 is a temperature; the truncations are the usual
    companions).  Both are upper level sets of p, so that tokens of equal probability are kept or dropped together:
      top_k > 0:  keep {v : p[v] >= the top_k-th largest value of p};
      top_p < 1:  on what is left, renormalised, walk the distinct values downwards, whole tie groups at a time,
                  and stop after the first group with which the accumulated mass reaches top_p.
    Returns (the kept part renormalised to sum 1, the boolean keep mask)."""
    p = np.asarray(p, dtype=np.float64)
    V = p.shape[0]
    keep = np.ones(V, dtype=bool)
    if top_k and 0 < top_k < V:
        kth = np.sort(p)[V - top_k]
        keep &= p >= kth
    if top_p < 1.0:
        pk = np.where(keep, p, 0.0)
        pk = pk / pk.sum()
        order = np.argsort(-pk, kind="stable")
        cum = np.cumsum(pk[order])
        first = int(np.searchsorted(cum, top_p, side="left"))        # first position where the running mass >= top_p
        first = min(first, V - 1)
        keep &= pk >= pk[order[first]]
    out = np.where(keep, p, 0.0)
    return out / out.sum(), keep


def accept_sample(draft_ids, target_logits, temperature, draft_logits, u, r, eos_id=-1, bonus=False, top_k=0, top_p=1.0):
    """Speculative rejection sampling over one block per sequence.

    top_k / top_p: p below is softmax(target_logits / T) after truncate_distribution, so the rule is lossless with
    respect to the truncated verifier distribution; a draft token outside it has alpha = 0.

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
    truncated = bool(top_k) or top_p < 1.0
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
            if truncated:
                p, _ = truncate_distribution(np.exp(logp), top_k, top_p)
                with np.errstate(divide="ignore"):
                    logp = np.log(p)                       # -inf outside the kept set
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
            if truncated:
                p, _ = truncate_distribution(p, top_k, top_p)
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

    def append(self, seq_ids, k_blk, v_blk, row_state=None):
        """Write block rows at token positions seq_len .. seq_len+k-1 (lengths unchanged).  With row states only the
        decoded rows are written (row i still goes to position seq_len + i): a masked or absent position has no
        keys and values worth keeping."""
        B, k = k_blk.shape[0], k_blk.shape[1]
        for b in range(B):
            s = int(seq_ids[b])
            for i in range(k):
                if row_state is not None and row_state[b][i] != ROW_DECODED:
                    continue
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
        self.appended = np.zeros(B, dtype=np.int32)        # tokens that joined each sequence's output in this pass
        for b in range(B):
            if self.finished[b]:
                continue
            room = self.max_new - int(self.n_tokens[b])
            m = min(int(n_out[b]), room)
            for i in range(m):
                self.tokens[b, self.n_tokens[b] + i] = out_ids[b][i]
            self.n_tokens[b] += m
            self.appended[b] = m
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


# --------------------------------------------------------------------------
# (7) The drafter's side of the loop beyond the single-step fill.
#     Section 4 ("Generative capabilities") shows the drafter completing a block
#     over several denoising iterations; the appendix on the DLLM KV cache points
#     to block-wise caches for diffusion models (confidence-gated parallel
#     decoding inside a block, the finished block's keys and values kept as
#     context).  The paper gives neither rule a formula; the ones below are the
#     published block-diffusion decoding rules it points to, reduced to what the
#     attention and cache calls need.
# --------------------------------------------------------------------------

def refill_step(row_state, tokens, ids, logprob, log_threshold):
    """One iteration of a block re-fill.  For each sequence: every row that is still
    masked and whose most likely token (ids) has log-probability (logprob) >=
    log_threshold becomes decoded with that token; if no masked row qualifies, the
    most confident masked row does (lowest row on ties), so each iteration decodes
    at least one row while any is masked.  Decoded and absent rows keep their
    state and token.  Returns (row_state', tokens', masked rows left per sequence).
    log_threshold = -inf decodes everything at once: the single-step block draft."""
    st = np.array(row_state, dtype=np.int32)
    tok = np.array(tokens, dtype=np.int32)
    B, k = st.shape
    left = np.zeros(B, dtype=np.int32)
    for b in range(B):
        masked = [i for i in range(k) if st[b, i] == ROW_MASKED]
        if not masked:
            continue
        chosen = [i for i in masked if logprob[b][i] >= log_threshold]
        if not chosen:
            best = masked[0]
            for i in masked[1:]:
                if logprob[b][i] > logprob[b][best]:
                    best = i
            chosen = [best]
        for i in chosen:
            st[b, i] = ROW_DECODED
            tok[b, i] = ids[b][i]
        left[b] = len(masked) - len(chosen)
    return st, tok, left


def refresh_rows(appended, k):
    """Row states of the pass that brings the drafter's cache up to date after a
    verify step: the `appended[b]` tokens that joined sequence b's output are
    decoded rows (they see each other and the drafter's prefix, and their keys and
    values are written to its cache); the rest of the block is absent."""
    appended = np.asarray(appended)
    st = np.full((appended.shape[0], k), ROW_ABSENT, dtype=np.int32)
    for b in range(appended.shape[0]):
        st[b, :int(appended[b])] = ROW_DECODED
    return st


# --------------------------------------------------------------------------
# (8) Routed mixture-of-experts MLP of a Qwen3-MoE-style verifier layer (the
#     paper's largest verifier, Qwen3-30B-A3B, has one in every layer): a linear
#     router, softmax over the experts, the top_k experts of each row with their
#     probabilities renormalised to sum 1, each expert a SiLU-gated MLP, the
#     weighted sum of their outputs.
# --------------------------------------------------------------------------

def moe_route(x, w_router, top_k, renormalise=True):
    """x [M,hid], w_router [E,hid] -> (experts [M,top_k] int32, weights [M,top_k] float64), each row's experts in
    order of decreasing probability (lower index first among equals)."""
    logits = np.asarray(x, dtype=np.float64) @ np.asarray(w_router, dtype=np.float64).T
    logits = logits - logits.max(axis=1, keepdims=True)
    prob = np.exp(logits)
    prob = prob / prob.sum(axis=1, keepdims=True)
    order = np.argsort(-prob, axis=1, kind="stable")[:, :top_k]
    wts = np.take_along_axis(prob, order, axis=1)
    if renormalise:
        wts = wts / wts.sum(axis=1, keepdims=True)
    return order.astype(np.int32), wts


def moe_mlp(x, w_router, w_gate_up, w_down, top_k, renormalise=True):
    """x [M,hid]; w_router [E,hid]; w_gate_up [E,2I,hid] (gate rows first, then up rows); w_down [E,hid,I]
    -> y [M,hid] = sum_j weight_j * down_e(silu(gate_e(x)) * up_e(x)) over the row's top_k experts e."""
    x = np.asarray(x, dtype=np.float64)
    experts, wts = moe_route(x, w_router, top_k, renormalise)
    E, twoI, hid = np.asarray(w_gate_up).shape
    inter = twoI // 2
    y = np.zeros_like(x)
    for m in range(x.shape[0]):
        for j in range(top_k):
            e = int(experts[m, j])
            gu = linear(x[m:m + 1], w_gate_up[e])[0]
            act = swiglu(gu[:inter], gu[inter:])
            y[m] += wts[m, j] * linear(act[None, :], w_down[e])[0]
    return y
