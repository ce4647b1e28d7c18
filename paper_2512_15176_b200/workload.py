"""Seeded synthetic inputs for the DEER draft-verify step.

This module only *draws inputs*: random tensors, sequence lengths, a page
permutation, planted draft blocks and uniforms.  It holds none of the method's
arithmetic (no attention, no logits, no acceptance rule, no KV commit) and is
the one module that the CUDA path's tests, the benchmark and the CPU oracle's
tests all share.  Everything is a pure function of ``(seed, tag)``.

The shapes follow Qwen3-class verifiers and a ~0.5B GQA drafter (the paper's
Table 1/2 targets and Appendix A drafter); the planted accepted-prefix lengths
follow the decaying-with-a-cap shape of the paper's accept-length histogram
(Appendix B.1).
"""
from __future__ import annotations

import dataclasses
import math
from typing import Optional, Tuple

import numpy as np
import torch

PAGE_SIZE = 16

MASK_CAUSAL = 0
MASK_BIDIR = 1


@dataclasses.dataclass(frozen=True)
class StepConfig:
    """One draft-verify step's shape.  ``ctx`` is a fixed prefix length or an
    inclusive ``(lo, hi)`` range for ragged batches."""

    name: str
    B: int
    Hq: int
    Hkv: int
    D: int
    k: int
    hid: int
    V: int
    ctx: Tuple[int, int]
    mask: int = MASK_CAUSAL
    mode: str = "greedy"            # "greedy" | "argmax_logprob" | "sample"
    temperature: float = 0.0
    sigma_qkv: float = 0.02
    sigma_w: float = 0.02
    sigma_h: float = 1.0
    prefix_law: str = "geometric"   # "geometric" (p=0.1, capped at k) | "uniform"
    seed: int = 1000
    growth: int = 0                 # extra tokens of page capacity per sequence (multi-step soaks)

    @property
    def M(self) -> int:
        return self.B * self.k

    @property
    def G(self) -> int:
        return self.Hq // self.Hkv

    def with_(self, **kw) -> "StepConfig":
        return dataclasses.replace(self, **kw)


def config(index: int) -> StepConfig:
    """The four fixed workloads (index 0..3); the sweep points come from
    :func:`sweep_config`."""
    if index == 0:
        return StepConfig("C1-tiny", 1, 8, 2, 64, 8, 512, 4096, (256, 256),
                          prefix_law="uniform", seed=1000)
    if index == 1:
        return StepConfig("C2-qwen3-8b-verify", 1, 32, 8, 128, 32, 4096, 151936, (4096, 4096), seed=1001)
    if index == 2:
        return StepConfig("C3-dllm-block-fill", 8, 16, 8, 128, 32, 2048, 151936, (8192, 8192),
                          mask=MASK_BIDIR, mode="argmax_logprob", seed=1002)
    if index == 3:
        return StepConfig("C4-qwen3-30b-a3b-T1", 16, 32, 4, 128, 32, 2048, 151936, (2048, 16384),
                          mode="sample", temperature=1.0, seed=1003)
    raise ValueError("config index must be 0..3; use sweep_config for the sweep")


def sweep_config(B: int, ctx: int, k: int, mask: int, steps: int = 64) -> StepConfig:
    """One point of the sweep: ragged lengths UniformInt[ctx/2, ctx], 32q/8kv
    heads, head_dim 128, hidden 4096, vocab 151936, greedy acceptance."""
    return StepConfig(f"C5-B{B}-ctx{ctx}-k{k}-{'causal' if mask == MASK_CAUSAL else 'bidir'}",
                      B, 32, 8, 128, k, 4096, 151936, (ctx // 2, ctx), mask=mask,
                      seed=1004, growth=steps * k)


# --------------------------------------------------------------------------
# seeded streams
# --------------------------------------------------------------------------

def _mix(seed: int, tag: str) -> int:
    """splitmix64-style mix of a seed and a tag into a 63-bit stream seed."""
    x = (seed * 0x9E3779B97F4A7C15) & 0xFFFFFFFFFFFFFFFF
    for ch in tag.encode():
        x ^= ch
        x = (x * 0xBF58476D1CE4E5B9) & 0xFFFFFFFFFFFFFFFF
        x ^= x >> 31
    x = (x * 0x94D049BB133111EB) & 0xFFFFFFFFFFFFFFFF
    x ^= x >> 29
    return x & 0x7FFFFFFFFFFFFFFF


def _gen(seed: int, tag: str, device: str = "cpu") -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(_mix(seed, tag))
    return g


def normal(seed: int, tag: str, shape, sigma: float, dtype=torch.bfloat16, device: str = "cpu") -> torch.Tensor:
    """N(0, sigma) values drawn in fp32 and rounded once to ``dtype``.  With
    ``device='cuda'`` the values come from torch's device generator (used only
    for pools too large to draw on the host; the CPU side then receives a copy
    of those very tensors)."""
    g = _gen(seed, tag, device)
    n = int(np.prod(shape))
    out = torch.empty(n, dtype=dtype, device=device)
    step = 1 << 26
    for s in range(0, n, step):
        e = min(n, s + step)
        out[s:e] = (torch.randn(e - s, generator=g, dtype=torch.float32, device=device) * sigma).to(dtype)
    return out.view(*shape)


def uniform_open(seed: int, tag: str, shape) -> torch.Tensor:
    """fp32 uniforms strictly inside (0, 1): (24 random bits + 0.5) / 2^24."""
    g = _gen(seed, tag)
    bits = torch.randint(0, 1 << 24, tuple(shape), generator=g, dtype=torch.int64)
    return ((bits.to(torch.float64) + 0.5) / float(1 << 24)).to(torch.float32)


def rng(seed: int, tag: str) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(_mix(seed, tag)))


# --------------------------------------------------------------------------
# sequence lengths, pages
# --------------------------------------------------------------------------

def seq_lengths(cfg: StepConfig) -> np.ndarray:
    lo, hi = cfg.ctx
    if lo == hi:
        return np.full(cfg.B, lo, dtype=np.int32)
    return rng(cfg.seed, "seq_len").integers(lo, hi + 1, size=cfg.B).astype(np.int32)


@dataclasses.dataclass
class KVLayout:
    """Integer state of the paged cache, as plain host arrays.  ``free_stack``
    holds the free page ids in ``[0, free_top)``; a pop takes
    ``free_stack[free_top - 1]``."""

    num_pages: int
    max_seqs: int
    max_pages: int
    page_table: np.ndarray   # int32 [max_seqs, max_pages], -1 where unmapped
    seq_len: np.ndarray      # int32 [max_seqs]
    n_pages: np.ndarray      # int32 [max_seqs]   pages mapped per sequence
    free_stack: np.ndarray   # int32 [num_pages]
    free_top: np.ndarray     # int32 [1]


def kv_layout(cfg: StepConfig, lengths: Optional[np.ndarray] = None, slack_pages: int = 8) -> KVLayout:
    """Initial cache state: a seeded permutation of page ids on the free stack,
    then each sequence's prefix mapped by popping pages for sequence 0, 1, ...
    and logical page 0, 1, ... in turn, so physical pages are deliberately
    non-contiguous."""
    if lengths is None:
        lengths = seq_lengths(cfg)
    B = cfg.B
    cap_tokens = lengths.astype(np.int64) + cfg.k + cfg.growth
    max_pages = int(-(-int(cap_tokens.max()) // PAGE_SIZE))
    num_pages = int(sum(-(-int(c) // PAGE_SIZE) for c in cap_tokens)) + slack_pages
    perm = rng(cfg.seed, "page_perm").permutation(num_pages).astype(np.int32)
    page_table = np.full((B, max_pages), -1, dtype=np.int32)
    n_pages = np.zeros(B, dtype=np.int32)
    top = num_pages
    for b in range(B):
        need = -(-int(lengths[b]) // PAGE_SIZE)
        for j in range(need):
            top -= 1
            page_table[b, j] = perm[top]
        n_pages[b] = need
    return KVLayout(num_pages, B, max_pages, page_table, lengths.astype(np.int32).copy(), n_pages,
                    perm.copy(), np.array([top], dtype=np.int32))


# --------------------------------------------------------------------------
# tensors of one step
# --------------------------------------------------------------------------

def kv_pools(cfg: StepConfig, num_pages: int, device: str = "cpu", sigma: Optional[float] = None):
    s = cfg.sigma_qkv if sigma is None else sigma
    shape = (num_pages, cfg.Hkv, PAGE_SIZE, cfg.D)
    return (normal(cfg.seed, "k_pool", shape, s, device=device),
            normal(cfg.seed, "v_pool", shape, s, device=device))


def block_qkv(cfg: StepConfig, step: int = 0, sigma: Optional[float] = None):
    s = cfg.sigma_qkv if sigma is None else sigma
    q = normal(cfg.seed, f"q{step}", (cfg.B, cfg.k, cfg.Hq, cfg.D), s)
    kb = normal(cfg.seed, f"k_blk{step}", (cfg.B, cfg.k, cfg.Hkv, cfg.D), s)
    vb = normal(cfg.seed, f"v_blk{step}", (cfg.B, cfg.k, cfg.Hkv, cfg.D), s)
    return q, kb, vb


def hidden(cfg: StepConfig, step: int = 0, redraw: int = 0) -> torch.Tensor:
    return normal(cfg.seed, f"h{step}.{redraw}", (cfg.M, cfg.hid), cfg.sigma_h)


def lm_head(cfg: StepConfig) -> torch.Tensor:
    return normal(cfg.seed, "w", (cfg.V, cfg.hid), cfg.sigma_w)


def draft_logits(cfg: StepConfig, step: int = 0) -> torch.Tensor:
    """fp32 drafter logits ~N(0,1), [B, k, V] (the drafter distribution q of Eq. 5)."""
    return normal(cfg.seed, f"q_logits{step}", (cfg.B, cfg.k, cfg.V), 1.0, dtype=torch.float32)


# --------------------------------------------------------------------------
# draft blocks
# --------------------------------------------------------------------------

def planted_prefix_lengths(cfg: StepConfig, step: int = 0) -> np.ndarray:
    """Planted matching-prefix length per sequence: Geometric with
    P(L=l)=0.1*0.9^l (l=0,1,...) capped at k, or UniformInt{0..k}."""
    r = rng(cfg.seed, f"prefix_len{step}")
    if cfg.prefix_law == "uniform":
        return r.integers(0, cfg.k + 1, size=cfg.B).astype(np.int32)
    return np.minimum(r.geometric(0.1, size=cfg.B) - 1, cfg.k).astype(np.int32)


def plant_drafts(cfg: StepConfig, target_ids: np.ndarray, L: np.ndarray, step: int = 0) -> np.ndarray:
    """Draft ids [B,k]: equal to ``target_ids`` for the first L[b] positions,
    forced different at position L[b] (if < k), uniform random after it."""
    r = rng(cfg.seed, f"draft_ids{step}")
    tgt = np.asarray(target_ids, dtype=np.int64).reshape(cfg.B, cfg.k)
    out = r.integers(0, cfg.V, size=(cfg.B, cfg.k)).astype(np.int64)
    off = r.integers(0, cfg.V - 1, size=cfg.B).astype(np.int64)
    for b in range(cfg.B):
        l = int(L[b])
        out[b, :l] = tgt[b, :l]
        if l < cfg.k:
            out[b, l] = (tgt[b, l] + 1 + off[b]) % cfg.V
    return out.astype(np.int32)


def sample_drafts(q_logits: torch.Tensor, seed: int, step: int = 0) -> np.ndarray:
    """Draft ids drawn from softmax(q_logits) by inverse CDF in fp64 with an
    own uniform stream (how the drafter's tokens arise at temperature > 0;
    the ids are inputs to both the CUDA path and the oracle)."""
    B, k, V = q_logits.shape
    r = rng(seed, f"draft_sample{step}")
    ids = np.empty((B, k), dtype=np.int32)
    for b in range(B):
        z = q_logits[b].to(torch.float64).numpy()
        p = np.exp(z - z.max(axis=1, keepdims=True))
        cdf = np.cumsum(p, axis=1)
        t = r.random(k) * cdf[:, -1]
        for i in range(k):
            ids[b, i] = min(int(np.searchsorted(cdf[i], t[i], side="left")), V - 1)
    return ids


def algorithmic_bytes(cfg: StepConfig, lengths: np.ndarray) -> dict:
    """Bytes the step must move at least once: each live KV byte, each weight
    byte, each drafter logit, and Q/K/V block rows, hidden states and outputs."""
    tok = int(np.asarray(lengths, dtype=np.int64).sum())
    kv = tok * cfg.Hkv * cfg.D * 2 * 2
    blk = cfg.B * cfg.k * (cfg.Hq * 2 + cfg.Hkv * 2) * cfg.D * 2
    attn = kv + blk
    lm = cfg.V * cfg.hid * 2 + cfg.M * cfg.hid * 2 + cfg.M * 8
    acc = cfg.M * 12
    if cfg.mode == "sample":
        acc += cfg.M * cfg.V * 4
    return {"attn": attn, "lmhead": lm, "accept": acc, "total": attn + lm + acc}


def algorithmic_flops(cfg: StepConfig, lengths: np.ndarray) -> dict:
    tok = int(np.asarray(lengths, dtype=np.int64).sum())
    attn = 4 * cfg.D * cfg.Hq * cfg.k * (tok + cfg.B * cfg.k)
    lm = 2 * cfg.M * cfg.hid * cfg.V
    return {"attn": attn, "lmhead": lm, "total": attn + lm}
