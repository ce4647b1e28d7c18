"""Device buffers and call sequencing for one draft-verify step.

Plumbing only: torch allocates the tensors, the library's kernels do all of
the work.  ``VerifyStep.run()`` issues reserve -> block_attn -> lmhead_select
-> accept -> commit on the current stream without any host synchronisation.
"""
from __future__ import annotations

import math
from typing import Optional

import torch

from . import binding as L
from .workload import MASK_BIDIR, MASK_CAUSAL, StepConfig


def _ws(nbytes: int, device) -> torch.Tensor:
    return torch.empty(max(16, (nbytes + 15) // 16 * 16), dtype=torch.uint8, device=device)


class VerifyStep:
    """Buffers of one step for ``cfg``; ``kv`` is a ``binding.KVCache`` and ``w``
    the device-resident LM-head weight [V, hid] bf16."""

    def __init__(self, cfg: StepConfig, kv: L.KVCache, w: torch.Tensor, max_seq_len: int, device="cuda",
                 store_logits: Optional[bool] = None, overlap_draft_stats: bool = True):
        self.cfg, self.kv, self.w, self.max_seq_len = cfg, kv, w, int(max_seq_len)
        B, k, Hq, Hkv, D, M, V = cfg.B, cfg.k, cfg.Hq, cfg.Hkv, cfg.D, cfg.M, cfg.V
        bf, i32, f32 = torch.bfloat16, torch.int32, torch.float32
        dev = device
        self.seq_ids = torch.arange(B, dtype=i32, device=dev)
        self.q = torch.empty(B, k, Hq, D, dtype=bf, device=dev)
        self.k_blk = torch.empty(B, k, Hkv, D, dtype=bf, device=dev)
        self.v_blk = torch.empty(B, k, Hkv, D, dtype=bf, device=dev)
        self.attn_out = torch.empty(B, k, Hq, D, dtype=bf, device=dev)
        self.h = torch.empty(M, cfg.hid, dtype=bf, device=dev)
        self.draft_ids = torch.zeros(B, k, dtype=i32, device=dev)
        self.target_ids = torch.empty(B, k, dtype=i32, device=dev)
        self.accept_len = torch.empty(B, dtype=i32, device=dev)
        self.out_ids = torch.empty(B, k, dtype=i32, device=dev)
        self.n_out = torch.empty(B, dtype=i32, device=dev)
        self.max_logprob = torch.empty(M, dtype=f32, device=dev) if cfg.mode == "argmax_logprob" else None
        sample = cfg.mode == "sample"
        self.store_logits = sample if store_logits is None else store_logits
        self.lse = torch.empty(M, dtype=f32, device=dev) if sample else None
        self.draft_logit = torch.empty(M, dtype=f32, device=dev) if sample else None
        self.logits = torch.empty(M, V, dtype=f32, device=dev) if self.store_logits else None
        self.q_logits = torch.empty(B, k, V, dtype=f32, device=dev) if sample else None
        self.u = torch.empty(B, k, dtype=f32, device=dev) if sample else None
        self.r = torch.empty(B, dtype=f32, device=dev) if sample else None
        self.attn_ws = _ws(L.deer_block_attn_workspace_bytes(B, k, Hq, Hkv, D, self.max_seq_len), dev)
        self.lm_ws = _ws(L.deer_lmhead_workspace_bytes(M, cfg.hid, V), dev)
        self.acc_ws = _ws(L.deer_accept_workspace_bytes(L.DEER_ACC_SAMPLE if sample else L.DEER_ACC_GREEDY, B, k, V), dev)
        self.scale = 1.0 / math.sqrt(D)
        self.eos_id = -1                # Algorithm 1's EOS break inside a block; < 0 disables
        # Sampling: the pass over the drafter's logits (q of Eq. 5) needs nothing from the verifier, so run() puts it
        # on a second stream at the start of the step and joins before the acceptance.
        self.side = torch.cuda.Stream(device=dev) if (sample and overlap_draft_stats) else None
        self._stats_forked = False
        self.bonus = False              # the k rows are k-1 drafts + one more row (deer_accept's DEER_ACC_BONUS)
        # sampling: top-k / nucleus truncation of the verifier's distribution ahead of the acceptance (0 / 1.0 = off)
        self.top_k, self.top_p = 0, 1.0
        self.tau = torch.empty(M, dtype=f32, device=dev) if sample else None
        self.lse_trunc = torch.empty(M, dtype=f32, device=dev) if sample else None

    # ---- inputs -------------------------------------------------------------
    def load(self, q=None, k_blk=None, v_blk=None, h=None, draft_ids=None, q_logits=None, u=None, r=None):
        for dst, src in ((self.q, q), (self.k_blk, k_blk), (self.v_blk, v_blk), (self.h, h), (self.draft_ids, draft_ids),
                         (self.q_logits, q_logits), (self.u, u), (self.r, r)):
            if src is not None:
                if not torch.is_tensor(src):
                    src = torch.as_tensor(src)
                dst.copy_(src.to(dst.dtype).reshape(dst.shape), non_blocking=True)

    # ---- the four calls -------------------------------------------------------
    def reserve(self):
        L.deer_kv_reserve(self.kv, self.seq_ids, self.cfg.k)

    def attn(self, append: Optional[bool] = None):
        causal = self.cfg.mask == MASK_CAUSAL
        if append is None:
            append = causal
        L.deer_block_attn(self.kv, self.seq_ids, self.q, self.k_blk, self.v_blk, self.attn_out,
                          L.DEER_MASK_CAUSAL if causal else L.DEER_MASK_BIDIR, append, self.scale, self.max_seq_len,
                          self.attn_ws)

    def lmhead(self):
        c = self.cfg
        if c.mode == "greedy":
            L.deer_lmhead_select(self.h, self.w, L.DEER_SEL_ARGMAX, 1.0, None, self.target_ids, None, None, None,
                                 self.logits, self.lm_ws)
        elif c.mode == "argmax_logprob":
            L.deer_lmhead_select(self.h, self.w, L.DEER_SEL_ARGMAX_LOGPROB, 1.0, None, self.target_ids, self.max_logprob,
                                 None, None, self.logits, self.lm_ws)
        else:
            L.deer_lmhead_select(self.h, self.w, L.DEER_SEL_SOFTMAX, c.temperature, self.draft_ids, self.target_ids, None,
                                 self.lse, self.draft_logit, self.logits, self.lm_ws)

    def fork_draft_stats(self):
        """Start the pass over the drafter's logits on the side stream (no-op without one); accept() joins it."""
        if self.side is None:
            return
        c = self.cfg
        self.side.wait_stream(torch.cuda.current_stream())   # after the inputs and the previous step's acceptance
        with torch.cuda.stream(self.side):
            L.deer_draft_stats(c.B, c.k, c.V, self.draft_ids, self.q_logits, self.acc_ws)
        self._stats_forked = True

    def accept(self):
        c = self.cfg
        prestats = self._stats_forked
        if prestats:
            torch.cuda.current_stream().wait_stream(self.side)
            self._stats_forked = False
        extra = L.DEER_ACC_BONUS if self.bonus else 0
        if c.mode == "sample":
            mode = (L.DEER_ACC_SAMPLE_PRESTATS if prestats else L.DEER_ACC_SAMPLE) | extra
            if self.top_k > 0 or self.top_p < 1.0:
                L.deer_truncate(self.logits, self.lse, c.temperature, self.top_k, self.top_p, self.tau, self.lse_trunc)
                L.deer_accept_truncated(mode, c.B, c.k, c.V, self.draft_ids, None, self.logits, self.lse_trunc, self.draft_logit,
                                        self.tau, c.temperature, self.q_logits, self.u, self.r, self.eos_id, self.accept_len,
                                        self.out_ids, self.n_out, self.acc_ws)
            else:
                L.deer_accept(mode, c.B, c.k, c.V, self.draft_ids, None, self.logits, self.lse, self.draft_logit,
                              c.temperature, self.q_logits, self.u, self.r, self.eos_id, self.accept_len, self.out_ids,
                              self.n_out, self.acc_ws)
        else:
            L.deer_accept(L.DEER_ACC_GREEDY | extra, c.B, c.k, c.V, self.draft_ids, self.target_ids, None, None, None, 1.0, None,
                          None, None, self.eos_id, self.accept_len, self.out_ids, self.n_out, None)

    def commit(self):
        L.deer_kv_commit(self.kv, self.seq_ids, self.accept_len, self.cfg.k)

    def accept_commit(self):
        """The end of the step: one launch when the acceptance is greedy, acceptance then commit otherwise."""
        if self.cfg.mode == "sample":
            self.accept()
            self.commit()
            return
        extra = L.DEER_ACC_BONUS if self.bonus else 0
        L.deer_accept_commit(self.kv, self.seq_ids, L.DEER_ACC_GREEDY | extra, self.cfg.k, self.draft_ids, self.target_ids,
                             self.eos_id, self.accept_len, self.out_ids, self.n_out)

    def run(self):
        """One whole step.  The drafter block fill (bidirectional mask) has no
        acceptance and commits nothing."""
        if self.cfg.mask == MASK_BIDIR:
            self.attn(append=False)
            self.lmhead()
            return
        # At the start of the step: it runs beside the attention kernel, which leaves bandwidth and issue slots free.
        self.fork_draft_stats()
        self.reserve()
        self.attn(append=True)
        self.lmhead()
        self.accept_commit()

    #: kernels launched by one run(), by mode (attention + merge, LM head, reserve, acceptance and commit)
    def launches_per_step(self) -> int:
        if self.cfg.mask == MASK_BIDIR:
            return 4
        return 2 + 2 + 1 + (3 if self.cfg.mode == "sample" else 1)


class DecodeLoop:
    """Algorithm 1's outer loop over a batch: every pass runs one verify step
    and then ``deer_emit`` -- the chosen tokens join each sequence's output,
    a sequence ends at an EOS or at ``max_new`` tokens, and the cache keeps only
    the accepted drafts that were emitted.  Nothing synchronises with the host
    between passes; finished sequences stay in the batch and are ignored.

    ``pending``: row 0 of every block is the token emitted last (not in the cache
    yet) and rows 1.. are the drafts; a fully accepted block then yields one more
    token from its last row, and the cache keeps the pending token's row as well."""

    def __init__(self, step: VerifyStep, eos_id: int, max_new: int, pending: bool = False):
        self.vs, self.eos_id, self.pending = step, int(eos_id), bool(pending)
        step.eos_id = int(eos_id)
        step.bonus = self.pending
        B, dev = step.cfg.B, step.q.device
        self.tokens = torch.full((B, max_new), -1, dtype=torch.int32, device=dev)
        self.n_tokens = torch.zeros(B, dtype=torch.int32, device=dev)
        self.finished = torch.zeros(B, dtype=torch.int32, device=dev)
        self.keep = torch.zeros(B, dtype=torch.int32, device=dev)

        self.appended = torch.zeros(B, dtype=torch.int32, device=dev)

    def one_pass(self):
        vs = self.vs
        vs.reserve()
        vs.attn(append=True)
        vs.lmhead()
        vs.accept()
        L.deer_emit(vs.accept_len, vs.out_ids, vs.n_out, self.eos_id, self.tokens, self.n_tokens, self.finished, self.keep,
                    L.DEER_EMIT_PENDING if self.pending else 0, appended=self.appended)
        L.deer_kv_commit(vs.kv, vs.seq_ids, self.keep, vs.cfg.k)


class DrafterBlock:
    """The drafter's side of a pass (Section 3.2's block proposal, Section 4's several
    denoising iterations, and the drafter-side cache the appendix on the DLLM KV cache
    looks forward to) on the library's calls.  ``fill()`` runs iterations of
    bidirectional block attention over the drafter's own paged cache -> LM head
    (argmax + its log-probability) -> ``deer_refill`` until every row is decoded or
    ``max_iters`` is reached, entirely on the device; the decoded tokens are the
    draft block.  ``refresh(appended)`` brings the drafter's cache up to date after
    the verify step: the tokens that joined the output are attended as decoded rows,
    their keys and values appended, and the cache commits ``appended`` rows.
    There is no drafter model here: the per-iteration query/key/value rows and hidden
    states are inputs (``load``)."""

    def __init__(self, cfg: StepConfig, kv: L.KVCache, w: torch.Tensor, max_seq_len: int, device="cuda"):
        self.cfg, self.kv, self.w, self.max_seq_len = cfg, kv, w, int(max_seq_len)
        B, k, Hq, Hkv, D, M = cfg.B, cfg.k, cfg.Hq, cfg.Hkv, cfg.D, cfg.M
        bf, i32, f32 = torch.bfloat16, torch.int32, torch.float32
        self.seq_ids = torch.arange(B, dtype=i32, device=device)
        self.q = torch.empty(B, k, Hq, D, dtype=bf, device=device)
        self.k_blk = torch.empty(B, k, Hkv, D, dtype=bf, device=device)
        self.v_blk = torch.empty(B, k, Hkv, D, dtype=bf, device=device)
        self.attn_out = torch.empty(B, k, Hq, D, dtype=bf, device=device)
        self.h = torch.empty(M, cfg.hid, dtype=bf, device=device)
        self.ids = torch.empty(B, k, dtype=i32, device=device)
        self.logprob = torch.empty(B, k, dtype=f32, device=device)
        self.row_state = torch.ones(B, k, dtype=i32, device=device)
        self.tokens = torch.full((B, k), -1, dtype=i32, device=device)
        self.left = torch.zeros(B, dtype=i32, device=device)
        self.attn_ws = _ws(L.deer_block_attn_workspace_bytes(B, k, Hq, Hkv, D, self.max_seq_len), device)
        self.lm_ws = _ws(L.deer_lmhead_workspace_bytes(M, cfg.hid, cfg.V), device)
        self.scale = 1.0 / math.sqrt(D)

    def load(self, q=None, k_blk=None, v_blk=None, h=None):
        for dst, src in ((self.q, q), (self.k_blk, k_blk), (self.v_blk, v_blk), (self.h, h)):
            if src is not None:
                dst.copy_(src.to(dst.dtype).reshape(dst.shape), non_blocking=True)

    def start_block(self):
        """A fresh block: every row masked, no token yet."""
        self.row_state.fill_(1)
        self.tokens.fill_(-1)

    def iteration(self, log_threshold: float):
        """One denoising iteration on the current row states (inputs as loaded)."""
        L.deer_block_attn_rows(self.kv, self.seq_ids, self.q, self.k_blk, self.v_blk, self.attn_out, self.row_state,
                               L.DEER_MASK_BIDIR, False, self.scale, self.max_seq_len, self.attn_ws)
        L.deer_lmhead_select(self.h, self.w, L.DEER_SEL_ARGMAX_LOGPROB, 1.0, None, self.ids, self.logprob, None, None, None,
                             self.lm_ws)
        L.deer_refill(self.ids, self.logprob, log_threshold, self.row_state, self.tokens, self.left)

    def refresh(self, appended: torch.Tensor):
        """After the verify step: the drafter's keys and values of the tokens that joined the output (inputs as
        loaded: their rows first) go into its cache."""
        k = self.cfg.k
        L.deer_refresh_rows(appended, self.row_state)
        L.deer_kv_reserve(self.kv, self.seq_ids, k)
        L.deer_block_attn_rows(self.kv, self.seq_ids, self.q, self.k_blk, self.v_blk, self.attn_out, self.row_state,
                               L.DEER_MASK_BIDIR, True, self.scale, self.max_seq_len, self.attn_ws)
        L.deer_kv_commit(self.kv, self.seq_ids, appended, k)


class VerifierLayer:
    """One pre-norm decoder layer of a Qwen3-style verifier at the M = B k rows of a
    draft block, on the library's calls: RMSNorm -> Q/K/V projections -> per-head
    RMSNorm of q, k + rotary embedding -> block attention against the paged cache
    (the block's K/V rows are appended) -> output projection + residual -> RMSNorm
    -> MLP + residual.  The MLP is the dense SiLU-gated one (gate/up projection,
    SiLU(gate) * up, down projection) or, with ``moe=(experts, top_k)``, the routed
    mixture of experts.
    Weights are [out][in] bf16 tensors on the device: "wqkv" = the query, key and
    value projections stacked in that order, "wo", "ln1", "ln2", optional "q_norm" /
    "k_norm"; dense: "wgu" (gate rows then up rows), "wd"; routed: "w_router" [E][hid],
    "w_gate_up" [E][2 I][hid], "w_down" [E][hid][I].
    ``fused=False`` issues every step as a call of its own (15 kernels; every
    intermediate is an attribute, so that a test can look at each stage);
    ``fused=True`` uses the calls that take a projection together with the row-wise
    step behind it (9 kernels; the dense gate/up weights are re-laid once as
    (gate, up) row pairs)."""

    def __init__(self, cfg: StepConfig, kv: L.KVCache, weights: dict, max_seq_len: int, inter: int, eps=1e-6,
                 theta=1.0e6, device="cuda", fused=False, moe=None, reserve=True):
        self.cfg, self.kv, self.w, self.max_seq_len = cfg, kv, weights, int(max_seq_len)
        self.inter, self.eps, self.theta = int(inter), float(eps), float(theta)
        self.fused, self.moe, self.reserve = bool(fused), moe, bool(reserve)
        B, k, Hq, Hkv, D, M, hid = cfg.B, cfg.k, cfg.Hq, cfg.Hkv, cfg.D, cfg.M, cfg.hid
        bf = torch.bfloat16
        e = lambda *shape: torch.empty(*shape, dtype=bf, device=device)
        self.seq_ids = torch.arange(B, dtype=torch.int32, device=device)
        self.xn, self.q, self.k_blk, self.v_blk = e(M, hid), e(B, k, Hq, D), e(B, k, Hkv, D), e(B, k, Hkv, D)
        self.qkv = e(M, (Hq + 2 * Hkv) * D)
        self.attn_out, self.x1, self.xn2 = e(B, k, Hq, D), e(M, hid), e(M, hid)
        self.act, self.x2, self.xn_next = e(M, self.inter), e(M, hid), e(M, hid)
        self.gu = e(M, 2 * self.inter) if not (fused or moe) else None
        self.attn_ws = _ws(L.deer_block_attn_workspace_bytes(B, k, Hq, Hkv, D, self.max_seq_len), device)
        n_qkv = (Hq + 2 * Hkv) * D
        self.lin_ws = _ws(max(L.deer_layer_workspace_bytes(M, hid, n) for n in (n_qkv, 2 * self.inter, hid)) or 16, device)
        self.scale = 1.0 / math.sqrt(D)
        if moe:
            E, self.top_k = int(moe[0]), int(moe[1])
            self.moe_ws = _ws(L.deer_moe_workspace_bytes(M, hid, E, self.inter, self.top_k), device)
        elif fused:
            wgu = weights["wgu"]
            self.wgu_pairs = torch.stack([wgu[:self.inter], wgu[self.inter:]], dim=1).reshape(2 * self.inter, hid).contiguous()

    def forward(self, x: torch.Tensor, xn: Optional[torch.Tensor] = None, next_ln: Optional[torch.Tensor] = None) -> torch.Tensor:
        """x [M, hid]: the layer's input.  xn: RMSNorm(x) * ln1 if the caller already has it (the previous layer's
        fused tail).  next_ln: the next layer's first RMSNorm weights; with them (fused, dense MLP) the layer also
        leaves RMSNorm(output) in ``xn_next``."""
        c, w = self.cfg, self.w
        M = c.M
        if xn is None:
            L.deer_rmsnorm(x, w["ln1"], self.xn, self.eps)
            xn = self.xn
        if self.fused:
            L.deer_linear_qkv_rope(self.kv, self.seq_ids, xn, w["wqkv"], self.q, self.k_blk, self.v_blk, w.get("q_norm"),
                                   w.get("k_norm"), self.eps, self.theta, self.lin_ws)
        else:
            L.deer_linear(xn, w["wqkv"], self.qkv, workspace=self.lin_ws)
            L.deer_qkv_split_norm_rope(self.kv, self.seq_ids, self.qkv, self.q, self.k_blk, self.v_blk, w.get("q_norm"),
                                       w.get("k_norm"), self.eps, self.theta)
        if self.reserve:
            L.deer_kv_reserve(self.kv, self.seq_ids, c.k)
        L.deer_block_attn(self.kv, self.seq_ids, self.q, self.k_blk, self.v_blk, self.attn_out, L.DEER_MASK_CAUSAL, True,
                          self.scale, self.max_seq_len, self.attn_ws)
        if self.fused:
            L.deer_linear_residual_norm(self.attn_out.view(M, -1), w["wo"], self.x1, residual=x, gamma=w["ln2"], y_norm=self.xn2,
                                        eps=self.eps, workspace=self.lin_ws)
        else:
            L.deer_linear(self.attn_out.view(M, -1), w["wo"], self.x1, residual=x, workspace=self.lin_ws)
            L.deer_rmsnorm(self.x1, w["ln2"], self.xn2, self.eps)
        if self.moe:
            L.deer_moe_mlp(self.xn2, w["w_router"], w["w_gate_up"], w["w_down"], self.x2, self.top_k, self.moe_ws, residual=self.x1)
            if next_ln is not None:
                L.deer_rmsnorm(self.x2, next_ln, self.xn_next, self.eps)
        elif self.fused:
            L.deer_linear_swiglu(self.xn2, self.wgu_pairs, self.act)
            L.deer_linear_residual_norm(self.act, w["wd"], self.x2, residual=self.x1, gamma=next_ln,
                                        y_norm=self.xn_next if next_ln is not None else None, eps=self.eps, workspace=self.lin_ws)
        else:
            L.deer_linear(self.xn2, w["wgu"], self.gu, workspace=self.lin_ws)
            L.deer_swiglu(self.gu, self.act)
            L.deer_linear(self.act, w["wd"], self.x2, residual=self.x1, workspace=self.lin_ws)
            if next_ln is not None:
                L.deer_rmsnorm(self.x2, next_ln, self.xn_next, self.eps)
        return self.x2


class VerifierStack:
    """``layers`` decoder layers in a row over one paged cache layout: every layer has key / value pools of its own,
    all of them indexed by the same page table, lengths and free stack (``kvs[l]`` = a ``binding.KVCache`` built
    on layer l's pools and the shared integer state).  One ``deer_kv_reserve`` per step serves all layers; the
    caller commits once after the acceptance (through any of the handles)."""

    def __init__(self, cfg: StepConfig, kvs, weights, max_seq_len: int, inter: int, eps=1e-6, theta=1.0e6, device="cuda",
                 fused=True, moe=None):
        assert len(kvs) == len(weights)
        self.cfg, self.kvs, self.eps = cfg, kvs, eps
        self.layers = [VerifierLayer(cfg, kv, w, max_seq_len, inter, eps, theta, device, fused=fused, moe=moe, reserve=False)
                       for kv, w in zip(kvs, weights)]
        self.seq_ids = self.layers[0].seq_ids

    def forward(self, x: torch.Tensor) -> torch.Tensor:
        L.deer_kv_reserve(self.kvs[0], self.seq_ids, self.cfg.k)
        xn = None
        for i, layer in enumerate(self.layers):
            nxt = self.layers[i + 1].w["ln1"] if i + 1 < len(self.layers) else None
            x = layer.forward(x, xn=xn, next_ln=nxt)
            xn = layer.xn_next if nxt is not None else None
        return x
