"""ctypes binding of ``libdeer.so``: the same entry points as ``include/deer.h``
with torch tensors in place of raw pointers.  Argument marshalling only --
every step of the path runs in the library's CUDA kernels; there is no CPU or
PyTorch fallback, and a missing library is a hard error.
"""
from __future__ import annotations

import ctypes
import os
from ctypes import POINTER, Structure, c_char_p, c_float, c_int, c_int32, c_size_t, c_void_p
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libdeer.so")

DEER_OK = 0
DEER_ERR_INVALID_ARG, DEER_ERR_UNSUPPORTED, DEER_ERR_NO_PAGES, DEER_ERR_CUDA, DEER_ERR_WORKSPACE, DEER_ERR_BAD_PAGE = 1, 2, 3, 4, 5, 6
DEER_ERR_TIMEOUT = 7
DEER_MASK_CAUSAL, DEER_MASK_BIDIR = 0, 1
DEER_SEL_ARGMAX, DEER_SEL_ARGMAX_LOGPROB, DEER_SEL_SOFTMAX = 0, 1, 2
DEER_ACC_GREEDY, DEER_ACC_SAMPLE, DEER_ACC_SAMPLE_PRESTATS, DEER_ACC_BONUS = 0, 1, 2, 4
DEER_EMIT_PENDING = 1

EXPORTS = [
    "deer_last_error", "deer_kv_create", "deer_kv_destroy", "deer_kv_reserve", "deer_kv_commit", "deer_accept_commit", "deer_kv_status", "deer_selftest_bounded_wait",
    "deer_block_attn_workspace_bytes", "deer_block_attn", "deer_lmhead_workspace_bytes", "deer_lmhead_select",
    "deer_accept_workspace_bytes", "deer_accept", "deer_verify_step_host",
    "deer_lmhead_static_max_rows", "deer_lmhead_select_static", "deer_emit", "deer_draft_stats",
    "deer_linear_workspace_bytes", "deer_linear", "deer_rmsnorm", "deer_qk_norm_rope", "deer_qkv_split_norm_rope", "deer_swiglu",
    "deer_truncate", "deer_accept_truncated", "deer_block_attn_rows", "deer_refill", "deer_refresh_rows",
    "deer_moe_workspace_bytes", "deer_moe_route", "deer_moe_mlp",
    "deer_layer_workspace_bytes", "deer_linear_qkv_rope", "deer_linear_residual_norm", "deer_linear_swiglu",
]


class DeerError(RuntimeError):
    def __init__(self, code: int, text: str):
        super().__init__(f"libdeer status {code}: {text}")
        self.code = code


class deer_kv_desc(Structure):
    _fields_ = [("k_pool", c_void_p), ("v_pool", c_void_p), ("page_table", c_void_p), ("seq_len", c_void_p),
                ("n_pages", c_void_p), ("free_stack", c_void_p), ("free_top", c_void_p), ("status", c_void_p),
                ("num_pages", c_int32), ("n_kv_heads", c_int32), ("head_dim", c_int32), ("page_size", c_int32),
                ("max_seqs", c_int32), ("max_pages", c_int32)]


class deer_step_dev(Structure):
    _fields_ = [("q", c_void_p), ("k_blk", c_void_p), ("v_blk", c_void_p), ("attn_out", c_void_p), ("h", c_void_p),
                ("seq_ids", c_void_p), ("draft_ids", c_void_p), ("target_ids", c_void_p), ("accept_len", c_void_p),
                ("out_ids", c_void_p), ("n_out", c_void_p), ("attn_ws", c_void_p), ("attn_ws_bytes", c_size_t),
                ("lm_ws", c_void_p), ("lm_ws_bytes", c_size_t)]


_lib = None


def lib() -> ctypes.CDLL:
    """Load the C-ABI library (once).  Raises if it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2512_15176_b200.build` "
                           "(there is no fallback path)")
    L = ctypes.CDLL(LIB_PATH)
    L.deer_last_error.restype = c_char_p
    L.deer_last_error.argtypes = []
    L.deer_kv_create.argtypes = [POINTER(c_void_p), POINTER(deer_kv_desc)]
    L.deer_kv_destroy.argtypes = [c_void_p]
    L.deer_kv_reserve.argtypes = [c_void_p, c_void_p, c_int, c_int, c_void_p]
    L.deer_kv_commit.argtypes = [c_void_p, c_void_p, c_void_p, c_int, c_int, c_void_p]
    L.deer_accept_commit.argtypes = [c_void_p, c_void_p, c_int, c_int, c_int, c_void_p, c_void_p, c_int32, c_void_p, c_void_p,
                                     c_void_p, c_void_p]
    L.deer_kv_status.argtypes = [c_void_p, POINTER(c_int32), c_void_p]
    L.deer_selftest_bounded_wait.argtypes = [c_void_p, c_void_p]
    L.deer_block_attn_workspace_bytes.restype = c_size_t
    L.deer_block_attn_workspace_bytes.argtypes = [c_int] * 6
    L.deer_block_attn.argtypes = [c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_int, c_int, c_int, c_int,
                                  c_int, c_float, c_int, c_void_p, c_size_t, c_void_p]
    L.deer_lmhead_workspace_bytes.restype = c_size_t
    L.deer_lmhead_workspace_bytes.argtypes = [c_int] * 3
    L.deer_lmhead_select.argtypes = [c_void_p, c_void_p, c_int, c_int, c_int, c_int, c_float, c_void_p, c_void_p, c_void_p,
                                     c_void_p, c_void_p, c_void_p, c_void_p, c_size_t, c_void_p]
    L.deer_lmhead_static_max_rows.restype = c_size_t
    L.deer_lmhead_static_max_rows.argtypes = []
    L.deer_lmhead_select_static.argtypes = [c_void_p, c_void_p, c_int, c_int, c_int, c_int, c_float, c_void_p, c_void_p,
                                            c_void_p, c_void_p, c_void_p, c_void_p, c_void_p]
    L.deer_accept_workspace_bytes.restype = c_size_t
    L.deer_accept_workspace_bytes.argtypes = [c_int] * 4
    L.deer_accept.argtypes = [c_int, c_int, c_int, c_int, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_float,
                              c_void_p, c_void_p, c_void_p, c_int32, c_void_p, c_void_p, c_void_p, c_void_p, c_size_t,
                              c_void_p]
    L.deer_accept_truncated.argtypes = [c_int, c_int, c_int, c_int, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p,
                                        c_float, c_void_p, c_void_p, c_void_p, c_int32, c_void_p, c_void_p, c_void_p, c_void_p,
                                        c_size_t, c_void_p]
    L.deer_truncate.argtypes = [c_int, c_int, c_void_p, c_void_p, c_float, c_int, c_float, c_void_p, c_void_p, c_void_p]
    L.deer_linear_workspace_bytes.restype = c_size_t
    L.deer_linear_workspace_bytes.argtypes = [c_int] * 3
    L.deer_linear.argtypes = [c_void_p, c_void_p, c_void_p, c_void_p, c_int, c_int, c_int, c_void_p, c_size_t, c_void_p]
    L.deer_rmsnorm.argtypes = [c_void_p, c_void_p, c_void_p, c_int, c_int, c_float, c_void_p]
    L.deer_qk_norm_rope.argtypes = [c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_int, c_int, c_int, c_float,
                                    c_float, c_void_p]
    L.deer_qkv_split_norm_rope.argtypes = [c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_int,
                                           c_int, c_int, c_float, c_float, c_void_p]
    L.deer_swiglu.argtypes = [c_void_p, c_void_p, c_int, c_int, c_void_p]
    L.deer_draft_stats.argtypes = [c_int, c_int, c_int, c_void_p, c_void_p, c_void_p, c_size_t, c_void_p]
    L.deer_emit.argtypes = [c_int, c_int, c_void_p, c_void_p, c_void_p, c_int32, c_int32, c_void_p, c_void_p, c_void_p, c_void_p,
                            c_void_p, c_int, c_void_p]
    L.deer_block_attn_rows.argtypes = [c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_int, c_int, c_int,
                                       c_int, c_int, c_float, c_int, c_void_p, c_size_t, c_void_p]
    L.deer_refill.argtypes = [c_int, c_int, c_void_p, c_void_p, c_float, c_void_p, c_void_p, c_void_p, c_void_p]
    L.deer_refresh_rows.argtypes = [c_int, c_int, c_void_p, c_void_p, c_void_p]
    L.deer_layer_workspace_bytes.restype = c_size_t
    L.deer_layer_workspace_bytes.argtypes = [c_int] * 3
    L.deer_linear_qkv_rope.argtypes = [c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p,
                                       c_int, c_int, c_int, c_int, c_float, c_float, c_void_p, c_size_t, c_void_p]
    L.deer_linear_residual_norm.argtypes = [c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_int, c_int, c_int,
                                            c_float, c_void_p, c_size_t, c_void_p]
    L.deer_linear_swiglu.argtypes = [c_void_p, c_void_p, c_void_p, c_int, c_int, c_int, c_void_p]
    L.deer_moe_workspace_bytes.restype = c_size_t
    L.deer_moe_workspace_bytes.argtypes = [c_int] * 5
    L.deer_moe_route.argtypes = [c_void_p, c_void_p, c_int, c_int, c_int, c_int, c_int, c_void_p, c_void_p, c_void_p, c_size_t,
                                 c_void_p]
    L.deer_moe_mlp.argtypes = [c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_int, c_int, c_int, c_int, c_int,
                               c_void_p, c_size_t, c_void_p]
    L.deer_verify_step_host.argtypes = [c_void_p, POINTER(deer_step_dev), c_void_p, c_void_p, c_void_p, c_void_p, c_void_p,
                                        c_void_p, c_int, c_int, c_int, c_int, c_int, c_float, c_int, c_void_p, c_void_p,
                                        c_void_p, c_void_p]
    for name in EXPORTS:
        getattr(L, name)          # every declared entry point must be exported
    _lib = L
    return L


def _check(rc: int) -> None:
    if rc != DEER_OK:
        raise DeerError(rc, lib().deer_last_error().decode())


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    if t is None:
        return None
    assert t.is_contiguous(), "tensors passed to libdeer must be contiguous"
    return t.data_ptr()


def _stream(stream) -> Optional[int]:
    if stream is None:
        return torch.cuda.current_stream().cuda_stream or None
    if isinstance(stream, torch.cuda.Stream):
        return stream.cuda_stream or None
    return stream or None


class KVCache:
    """Device tensors of one paged cache plus the library handle over them."""

    def __init__(self, k_pool, v_pool, page_table, seq_len, n_pages, free_stack, free_top):
        self.k_pool, self.v_pool = k_pool, v_pool
        self.page_table, self.seq_len, self.n_pages = page_table, seq_len, n_pages
        self.free_stack, self.free_top = free_stack, free_top
        self.status = torch.zeros(1, dtype=torch.int32, device=k_pool.device)
        num_pages, Hkv, page, D = k_pool.shape
        self.desc = deer_kv_desc(_ptr(k_pool), _ptr(v_pool), _ptr(page_table), _ptr(seq_len), _ptr(n_pages),
                                 _ptr(free_stack), _ptr(free_top), _ptr(self.status),
                                 num_pages, Hkv, D, page, page_table.shape[0], page_table.shape[1])
        self.handle = c_void_p()
        _check(lib().deer_kv_create(ctypes.byref(self.handle), ctypes.byref(self.desc)))

    @classmethod
    def from_layout(cls, layout, k_pool, v_pool, device="cuda"):
        """``layout`` is a ``workload.KVLayout`` (host arrays); pools are bf16 tensors."""
        i32 = lambda a: torch.from_numpy(a.copy()).to(device=device, dtype=torch.int32).contiguous()
        return cls(k_pool.to(device).contiguous(), v_pool.to(device).contiguous(), i32(layout.page_table),
                   i32(layout.seq_len), i32(layout.n_pages), i32(layout.free_stack), i32(layout.free_top))

    @property
    def n_kv_heads(self):
        return self.k_pool.shape[1]

    @property
    def head_dim(self):
        return self.k_pool.shape[3]

    def close(self):
        if self.handle:
            lib().deer_kv_destroy(self.handle)
            self.handle = c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def deer_kv_reserve(kv: KVCache, seq_ids: torch.Tensor, k: int, stream=None) -> None:
    _check(lib().deer_kv_reserve(kv.handle, _ptr(seq_ids), seq_ids.numel(), k, _stream(stream)))


def deer_selftest_bounded_wait(kv: KVCache, stream=None) -> None:
    _check(lib().deer_selftest_bounded_wait(kv.handle, _stream(stream)))


def deer_kv_commit(kv: KVCache, seq_ids: torch.Tensor, keep: torch.Tensor, k: int, stream=None) -> None:
    _check(lib().deer_kv_commit(kv.handle, _ptr(seq_ids), _ptr(keep), seq_ids.numel(), k, _stream(stream)))


def deer_kv_status(kv: KVCache, stream=None) -> int:
    code = c_int32(0)
    _check(lib().deer_kv_status(kv.handle, ctypes.byref(code), _stream(stream)))
    return code.value


def deer_block_attn_workspace_bytes(B, k, Hq, Hkv, D, max_seq_len) -> int:
    return lib().deer_block_attn_workspace_bytes(B, k, Hq, Hkv, D, max_seq_len)


def deer_block_attn(kv: KVCache, seq_ids, q, k_blk, v_blk, out, mask, append, scale, max_seq_len, workspace, stream=None):
    B, k, Hq, D = q.shape
    _check(lib().deer_block_attn(kv.handle, _ptr(seq_ids), _ptr(q), _ptr(k_blk), _ptr(v_blk), _ptr(out), B, k, Hq,
                                 int(mask), int(append), float(scale), int(max_seq_len), _ptr(workspace),
                                 workspace.numel() * workspace.element_size() if workspace is not None else 0,
                                 _stream(stream)))


def deer_lmhead_workspace_bytes(M, hid, V) -> int:
    return lib().deer_lmhead_workspace_bytes(M, hid, V)


def deer_lmhead_select(h, w, mode, temperature, draft_ids, out_ids, out_max_logprob, out_lse, out_draft_logit, out_logits,
                       workspace, stream=None):
    M, hid = h.shape
    V = w.shape[0]
    _check(lib().deer_lmhead_select(_ptr(h), _ptr(w), M, hid, V, int(mode), float(temperature), _ptr(draft_ids),
                                    _ptr(out_ids), _ptr(out_max_logprob), _ptr(out_lse), _ptr(out_draft_logit),
                                    _ptr(out_logits), _ptr(workspace),
                                    workspace.numel() * workspace.element_size() if workspace is not None else 0,
                                    _stream(stream)))


def deer_lmhead_static_max_rows() -> int:
    return lib().deer_lmhead_static_max_rows()


def deer_lmhead_select_static(h, w, mode, temperature, draft_ids, out_ids, out_max_logprob, out_lse, out_draft_logit,
                              out_logits, stream=None):
    """deer_lmhead_select for callers that cannot supply (or allocate) a workspace:
    the scratch is a fixed array inside the library, so M is limited to
    deer_lmhead_static_max_rows() and calls on one GPU must not overlap."""
    M, hid = h.shape
    V = w.shape[0]
    _check(lib().deer_lmhead_select_static(_ptr(h), _ptr(w), M, hid, V, int(mode), float(temperature), _ptr(draft_ids),
                                           _ptr(out_ids), _ptr(out_max_logprob), _ptr(out_lse), _ptr(out_draft_logit),
                                           _ptr(out_logits), _stream(stream)))


def deer_accept_workspace_bytes(mode, B, k, V) -> int:
    return lib().deer_accept_workspace_bytes(mode, B, k, V)


def deer_accept(mode, B, k, V, draft_ids, target_ids, target_logits, target_lse, target_draft_logit, temperature,
                draft_logits, u, r, eos_id, accept_len, out_ids, n_out, workspace, stream=None):
    _check(lib().deer_accept(int(mode), B, k, V, _ptr(draft_ids), _ptr(target_ids), _ptr(target_logits), _ptr(target_lse),
                             _ptr(target_draft_logit), float(temperature), _ptr(draft_logits), _ptr(u), _ptr(r), int(eos_id),
                             _ptr(accept_len), _ptr(out_ids), _ptr(n_out), _ptr(workspace),
                             workspace.numel() * workspace.element_size() if workspace is not None else 0,
                             _stream(stream)))


def deer_accept_commit(kv: KVCache, seq_ids, mode, k, draft_ids, target_ids, eos_id, accept_len, out_ids, n_out, stream=None):
    _check(lib().deer_accept_commit(kv.handle, _ptr(seq_ids), int(mode), seq_ids.numel(), k, _ptr(draft_ids), _ptr(target_ids),
                                    int(eos_id), _ptr(accept_len), _ptr(out_ids), _ptr(n_out), _stream(stream)))


def deer_truncate(target_logits, target_lse, temperature, top_k, top_p, tau, lse_trunc, stream=None):
    V = target_logits.shape[-1]
    M = target_logits.numel() // V
    _check(lib().deer_truncate(M, V, _ptr(target_logits), _ptr(target_lse), float(temperature), int(top_k), float(top_p),
                               _ptr(tau), _ptr(lse_trunc), _stream(stream)))


def deer_accept_truncated(mode, B, k, V, draft_ids, target_ids, target_logits, target_lse, target_draft_logit, target_tau,
                          temperature, draft_logits, u, r, eos_id, accept_len, out_ids, n_out, workspace, stream=None):
    _check(lib().deer_accept_truncated(int(mode), B, k, V, _ptr(draft_ids), _ptr(target_ids), _ptr(target_logits),
                                       _ptr(target_lse), _ptr(target_draft_logit), _ptr(target_tau), float(temperature),
                                       _ptr(draft_logits), _ptr(u), _ptr(r), int(eos_id), _ptr(accept_len), _ptr(out_ids),
                                       _ptr(n_out), _ptr(workspace),
                                       workspace.numel() * workspace.element_size() if workspace is not None else 0,
                                       _stream(stream)))


def deer_linear_workspace_bytes(M, K, N) -> int:
    return lib().deer_linear_workspace_bytes(M, K, N)


def deer_linear(x, w, y, residual=None, workspace=None, stream=None):
    M, K = x.shape
    N = w.shape[0]
    _check(lib().deer_linear(_ptr(x), _ptr(w), _ptr(residual), _ptr(y), M, K, N, _ptr(workspace),
                             workspace.numel() * workspace.element_size() if workspace is not None else 0, _stream(stream)))


def deer_rmsnorm(x, gamma, y, eps, stream=None):
    M, hid = x.shape
    _check(lib().deer_rmsnorm(_ptr(x), _ptr(gamma), _ptr(y), M, hid, float(eps), _stream(stream)))


def deer_qk_norm_rope(kv: "KVCache", seq_ids, q, k_blk, q_gamma, k_gamma, eps, theta, stream=None):
    B, k, Hq, _ = q.shape
    _check(lib().deer_qk_norm_rope(kv.handle, _ptr(seq_ids), _ptr(q), _ptr(k_blk), _ptr(q_gamma), _ptr(k_gamma), B, k, Hq,
                                   float(eps), float(theta), _stream(stream)))


def deer_qkv_split_norm_rope(kv: "KVCache", seq_ids, qkv, q, k_blk, v_blk, q_gamma, k_gamma, eps, theta, stream=None):
    B, k, Hq, _ = q.shape
    _check(lib().deer_qkv_split_norm_rope(kv.handle, _ptr(seq_ids), _ptr(qkv), _ptr(q), _ptr(k_blk), _ptr(v_blk), _ptr(q_gamma),
                                          _ptr(k_gamma), B, k, Hq, float(eps), float(theta), _stream(stream)))


def deer_swiglu(gate_up, y, stream=None):
    M, I = y.shape
    _check(lib().deer_swiglu(_ptr(gate_up), _ptr(y), M, I, _stream(stream)))


def deer_layer_workspace_bytes(M, K, N) -> int:
    return lib().deer_layer_workspace_bytes(M, K, N)


def deer_linear_qkv_rope(kv: "KVCache", seq_ids, x, w_qkv, q, k_blk, v_blk, q_gamma, k_gamma, eps, theta, workspace, stream=None):
    B, k, Hq, _ = q.shape
    _check(lib().deer_linear_qkv_rope(kv.handle, _ptr(seq_ids), _ptr(x), _ptr(w_qkv), _ptr(q), _ptr(k_blk), _ptr(v_blk), _ptr(q_gamma),
                                      _ptr(k_gamma), B, k, Hq, x.shape[1], float(eps), float(theta), _ptr(workspace),
                                      workspace.numel() * workspace.element_size(), _stream(stream)))


def deer_linear_residual_norm(x, w, y, residual=None, gamma=None, y_norm=None, eps=1e-6, workspace=None, stream=None):
    M, K = x.shape
    _check(lib().deer_linear_residual_norm(_ptr(x), _ptr(w), _ptr(residual), _ptr(gamma), _ptr(y), _ptr(y_norm), M, K, w.shape[0],
                                           float(eps), _ptr(workspace),
                                           workspace.numel() * workspace.element_size() if workspace is not None else 0,
                                           _stream(stream)))


def deer_linear_swiglu(x, w_pairs, y, stream=None):
    M, K = x.shape
    _check(lib().deer_linear_swiglu(_ptr(x), _ptr(w_pairs), _ptr(y), M, K, y.shape[1], _stream(stream)))


def deer_moe_workspace_bytes(M, hid, E, I, top_k) -> int:
    return lib().deer_moe_workspace_bytes(M, hid, E, I, top_k)


def deer_moe_route(x, w_router, top_k, experts, weights, renormalise=True, workspace=None, stream=None):
    M, hid = x.shape
    E = w_router.shape[0]
    if workspace is None:                      # plumbing: room for the M x E fp32 logits
        workspace = torch.empty(max(16, M * E * 4), dtype=torch.uint8, device=x.device)
    _check(lib().deer_moe_route(_ptr(x), _ptr(w_router), M, hid, E, int(top_k), 1 if renormalise else 0,
                                _ptr(experts), _ptr(weights), _ptr(workspace), workspace.numel() * workspace.element_size(),
                                _stream(stream)))


def deer_moe_mlp(x, w_router, w_gate_up, w_down, y, top_k, workspace, residual=None, stream=None):
    M, hid = x.shape
    E, two_i, _ = w_gate_up.shape
    _check(lib().deer_moe_mlp(_ptr(x), _ptr(w_router), _ptr(w_gate_up), _ptr(w_down), _ptr(residual), _ptr(y), M, hid, E, two_i // 2,
                              int(top_k), _ptr(workspace), workspace.numel() * workspace.element_size(), _stream(stream)))


def deer_draft_stats(B, k, V, draft_ids, draft_logits, workspace, stream=None):
    _check(lib().deer_draft_stats(B, k, V, _ptr(draft_ids), _ptr(draft_logits), _ptr(workspace),
                                  workspace.numel() * workspace.element_size(), _stream(stream)))


def deer_emit(accept_len, out_ids, n_out, eos_id, tokens, n_tokens, finished, keep, flags=0, stream=None, appended=None):
    B, k = out_ids.shape
    _check(lib().deer_emit(B, k, _ptr(accept_len), _ptr(out_ids), _ptr(n_out), int(eos_id), tokens.shape[1], _ptr(tokens),
                           _ptr(n_tokens), _ptr(finished), _ptr(keep), _ptr(appended), int(flags), _stream(stream)))


def deer_block_attn_rows(kv: KVCache, seq_ids, q, k_blk, v_blk, out, row_state, mask, append, scale, max_seq_len, workspace,
                         stream=None):
    B, k, Hq, D = q.shape
    _check(lib().deer_block_attn_rows(kv.handle, _ptr(seq_ids), _ptr(q), _ptr(k_blk), _ptr(v_blk), _ptr(out), _ptr(row_state),
                                      B, k, Hq, int(mask), int(append), float(scale), int(max_seq_len), _ptr(workspace),
                                      workspace.numel() * workspace.element_size() if workspace is not None else 0,
                                      _stream(stream)))


def deer_refill(ids, logprob, log_threshold, row_state, tokens, left=None, stream=None):
    B, k = row_state.shape
    _check(lib().deer_refill(B, k, _ptr(ids), _ptr(logprob), float(log_threshold), _ptr(row_state), _ptr(tokens), _ptr(left),
                             _stream(stream)))


def deer_refresh_rows(appended, row_state, stream=None):
    B, k = row_state.shape
    _check(lib().deer_refresh_rows(B, k, _ptr(appended), _ptr(row_state), _stream(stream)))


def deer_verify_step_host(kv: KVCache, dev: deer_step_dev, w, q_host, k_blk_host, v_blk_host, h_host, draft_ids_host,
                          B, k, Hq, hid, V, scale, max_seq_len, accept_len_host, out_ids_host, n_out_host, stream=None):
    _check(lib().deer_verify_step_host(kv.handle, ctypes.byref(dev), _ptr(w), _ptr(q_host), _ptr(k_blk_host),
                                       _ptr(v_blk_host), _ptr(h_host), _ptr(draft_ids_host), B, k, Hq, hid, V, float(scale),
                                       int(max_seq_len), _ptr(accept_len_host), _ptr(out_ids_host), _ptr(n_out_host),
                                       _stream(stream)))
