"""Run one library call a few times on a chosen shape -- the small, self-ending
program that profiler captures are taken from.

    python profile_case.py lmhead --M 32 --hid 4096 --V 32768 --iters 3
    python profile_case.py attn --B 8 --Hq 32 --Hkv 8 --k 32 --ctx 8192 --iters 3
    python profile_case.py qstats --B 4 --k 32 --V 151936 --iters 3
    python profile_case.py layer --B 1 --k 32 --ctx 4096 --hid 4096 --inter 12288 --iters 20
    python profile_case.py trunc --M 512 --V 151936 --top-k-trunc 50 --top-p 0.9 --iters 3
    python profile_case.py moe --M 32 --hid 2048 --experts 128 --inter 768 --top-k 8 --iters 3

Prints the average CUDA-event time per call and the achieved GB/s over the
call's algorithmic bytes.

With --probes (attn, lmhead) the calls run on the library built with timing probes
(`python -m paper_2512_15176_b200.build --probes`): the attention kernel records SM clock values at the hand-overs of
its pipeline for 64 tiles of one thread block, the block-pair LM head what its MMA-issuing thread's time goes to, and
the tables are printed after the timing line (times with probes are a little longer than without).
"""
from __future__ import annotations

import argparse
import math

import numpy as np
import torch

import os
import sys

sys.path.insert(0, os.path.dirname(os.path.abspath(__file__)))

from paper_2512_15176_b200 import binding as L  # noqa: E402
from paper_2512_15176_b200 import workload as W  # noqa: E402


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("what", choices=["lmhead", "attn", "qstats", "layer", "trunc", "moe"])
    ap.add_argument("--top-p", type=float, default=0.9)
    ap.add_argument("--top-k-trunc", type=int, default=50)
    ap.add_argument("--peaked", action="store_true", help="trunc: rows with a language model's rank-frequency shape")
    ap.add_argument("--inter", type=int, default=12288)
    ap.add_argument("--separate", action="store_true", help="layer: every step as a call of its own instead of the fused calls")
    ap.add_argument("--experts", type=int, default=0, help="layer: routed MLP with this many experts (0 = dense)")
    ap.add_argument("--top-k", type=int, default=8)
    ap.add_argument("--M", type=int, default=32)
    ap.add_argument("--hid", type=int, default=4096)
    ap.add_argument("--V", type=int, default=32768)
    ap.add_argument("--B", type=int, default=8)
    ap.add_argument("--Hq", type=int, default=32)
    ap.add_argument("--Hkv", type=int, default=8)
    ap.add_argument("--D", type=int, default=128)
    ap.add_argument("--k", type=int, default=32)
    ap.add_argument("--ctx", type=int, default=8192)
    ap.add_argument("--mode", default="argmax", choices=["argmax", "logprob", "softmax"])
    ap.add_argument("--logits", action="store_true")
    ap.add_argument("--bidir", action="store_true")
    ap.add_argument("--iters", type=int, default=3)
    ap.add_argument("--warmup", type=int, default=1)
    ap.add_argument("--probes", action="store_true", help="attn, lmhead: run on the library built with timing probes and print them")
    a = ap.parse_args()
    if a.probes:
        from paper_2512_15176_b200 import build as B_
        L.LIB_PATH = B_.build(probes=True)
    dev = "cuda"
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    flush_rd = torch.zeros(64 << 20, dtype=torch.int32, device=dev)
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(a.iters)]

    if a.what == "lmhead":
        cfg = W.StepConfig("prof", 1, 1, 1, 64, 1, a.hid, a.V, (0, 0), seed=31).with_(B=a.M)
        w = W.normal(31, "w", (a.V, a.hid), 0.02, device=dev)
        h = W.hidden(cfg).to(dev)
        ids = torch.empty(a.M, dtype=torch.int32, device=dev)
        f = lambda: torch.empty(a.M, dtype=torch.float32, device=dev)
        mlp, lse, dl = f(), f(), f()
        Z = torch.empty(a.M, a.V, dtype=torch.float32, device=dev) if a.logits else None
        drafts = torch.zeros(a.M, dtype=torch.int32, device=dev)
        ws = torch.empty(L.deer_lmhead_workspace_bytes(a.M, a.hid, a.V), dtype=torch.uint8, device=dev)
        mode = {"argmax": L.DEER_SEL_ARGMAX, "logprob": L.DEER_SEL_ARGMAX_LOGPROB, "softmax": L.DEER_SEL_SOFTMAX}[a.mode]
        call = lambda: L.deer_lmhead_select(h, w, mode, 1.0, drafts, ids, mlp, lse, dl, Z, ws)
        nbytes = a.V * a.hid * 2 + a.M * a.hid * 2 + a.M * 8 + (a.M * a.V * 4 if a.logits else 0)
        flops = 2.0 * a.M * a.hid * a.V
    elif a.what == "attn":
        cfg = W.StepConfig("prof", a.B, a.Hq, a.Hkv, a.D, a.k, 64, 64, (a.ctx, a.ctx),
                           mask=W.MASK_BIDIR if a.bidir else W.MASK_CAUSAL, seed=32)
        lengths = W.seq_lengths(cfg)
        lay = W.kv_layout(cfg, lengths)
        kp, vp = W.kv_pools(cfg, lay.num_pages, device=dev, sigma=1.0)
        kv = L.KVCache.from_layout(lay, kp, vp, dev)
        q, kb, vb = (t.to(dev) for t in W.block_qkv(cfg, sigma=1.0))
        out = torch.empty_like(q)
        seq_ids = torch.arange(a.B, dtype=torch.int32, device=dev)
        ws = torch.empty(L.deer_block_attn_workspace_bytes(a.B, a.k, a.Hq, a.Hkv, a.D, a.ctx), dtype=torch.uint8, device=dev)
        call = lambda: L.deer_block_attn(kv, seq_ids, q, kb, vb, out, cfg.mask, 0, 1.0 / math.sqrt(a.D), a.ctx, ws)
        nbytes = W.algorithmic_bytes(cfg, lengths)["attn"]
        flops = float(W.algorithmic_flops(cfg, lengths)["attn"])
    elif a.what == "layer":
        # one verifier layer (Qwen3-8B shape by default) at M = B k rows, replayed from a CUDA graph
        from paper_2512_15176_b200.runner import VerifierLayer
        cfg = W.StepConfig("prof", a.B, a.Hq, a.Hkv, a.D, a.k, a.hid, 64, (a.ctx, a.ctx), seed=34, growth=a.k)
        lengths = W.seq_lengths(cfg)
        lay = W.kv_layout(cfg, lengths)
        kp, vp = W.kv_pools(cfg, lay.num_pages, device=dev, sigma=1.0)
        kv = L.KVCache.from_layout(lay, kp, vp, dev)
        hid, QD, KD = a.hid, a.Hq * a.D, a.Hkv * a.D
        mk = lambda n, shape, sig: W.normal(34, n, shape, sig, device=dev)
        w = {"ln1": mk("ln1", (hid,), 1.0), "ln2": mk("ln2", (hid,), 1.0), "q_norm": mk("qn", (a.D,), 1.0),
             "k_norm": mk("kn", (a.D,), 1.0), "wqkv": mk("wqkv", (QD + 2 * KD, hid), hid ** -0.5),
             "wo": mk("wo", (hid, QD), QD ** -0.5)}
        if a.experts:
            w.update({"w_router": mk("wr", (a.experts, hid), hid ** -0.5 * 3.0),
                      "w_gate_up": mk("wgue", (a.experts, 2 * a.inter, hid), hid ** -0.5),
                      "w_down": mk("wde", (a.experts, hid, a.inter), a.inter ** -0.5)})
        else:
            w.update({"wgu": mk("wgu", (2 * a.inter, hid), hid ** -0.5), "wd": mk("wd", (hid, a.inter), a.inter ** -0.5)})
        x = mk("x", (cfg.M, hid), 1.0)
        layer = VerifierLayer(cfg, kv, w, a.ctx + a.k, a.inter, fused=not a.separate,
                              moe=(a.experts, a.top_k) if a.experts else None)
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())       # the weights and pools were drawn on the current stream
        with torch.cuda.stream(side):
            for _ in range(3):
                layer.forward(x)
            side.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=side):
                layer.forward(x)
        torch.cuda.synchronize()
        call = g.replay
        dense = sum(t.numel() * 2 for n, t in w.items() if n not in ("w_gate_up", "w_down"))
        if a.experts:
            e_ids = torch.empty(cfg.M, a.top_k, dtype=torch.int32, device=dev)
            e_w = torch.empty(cfg.M, a.top_k, dtype=torch.float32, device=dev)
            L.deer_moe_route(layer.xn2, w["w_router"], a.top_k, e_ids, e_w)
            torch.cuda.synchronize()
            dense += int(torch.unique(e_ids).numel()) * 3 * a.inter * hid * 2      # the experts the rows really chose
        nbytes = dense + W.algorithmic_bytes(cfg, lengths)["attn"]
        flops = 2.0 * cfg.M * (dense / 2 if not a.experts else sum(t.numel() for n, t in w.items() if n in ("wqkv", "wo"))
                               + a.top_k * 3 * a.inter * hid)
    elif a.what == "trunc":
        # top-k / nucleus threshold per row of fp32 logits (the sampling setting's truncation ahead of the acceptance)
        z = W.normal(35, "z", (a.M, a.V), 1.3, dtype=torch.float32, device=dev)
        if a.peaked:        # a language model's shape: -1.1 log(rank) under a permutation per row, plus noise
            base = -1.1 * torch.log(torch.arange(1, a.V + 1, device=dev, dtype=torch.float32))
            perm = torch.argsort(torch.rand(a.M, a.V, device=dev, generator=torch.Generator(dev).manual_seed(35)), dim=1)
            z = z * 0.25 + base[perm]
        lse = torch.logsumexp(z / 0.6, dim=1).contiguous()
        tau = torch.empty(a.M, dtype=torch.float32, device=dev)
        lse_t = torch.empty(a.M, dtype=torch.float32, device=dev)
        call = lambda: L.deer_truncate(z, lse, 0.6, a.top_k_trunc, a.top_p, tau, lse_t)
        nbytes = a.M * a.V * 4
        flops = 0.0
    elif a.what == "moe":
        # the routed MLP alone at M rows
        E, I, hid = a.experts or 128, a.inter, a.hid
        mk = lambda n, shape, sig: W.normal(36, n, shape, sig, device=dev)
        x = mk("x", (a.M, hid), 1.0)
        wr, wgu, wd = mk("wr", (E, hid), hid ** -0.5 * 3.0), mk("wgu", (E, 2 * I, hid), hid ** -0.5), mk("wd", (E, hid, I), I ** -0.5)
        y = torch.empty(a.M, hid, dtype=torch.bfloat16, device=dev)
        ws = torch.empty(L.deer_moe_workspace_bytes(a.M, hid, E, I, a.top_k), dtype=torch.uint8, device=dev)
        e_ids = torch.empty(a.M, a.top_k, dtype=torch.int32, device=dev)
        e_w = torch.empty(a.M, a.top_k, dtype=torch.float32, device=dev)
        L.deer_moe_route(x, wr, a.top_k, e_ids, e_w)
        torch.cuda.synchronize()
        call = lambda: L.deer_moe_mlp(x, wr, wgu, wd, y, a.top_k, ws)
        nbytes = int(torch.unique(e_ids).numel()) * 3 * I * hid * 2 + E * hid * 2       # the chosen experts' matrices + the router
        flops = 2.0 * a.M * a.top_k * 3 * I * hid
    else:
        M = a.B * a.k
        ql = W.normal(33, "ql", (a.B, a.k, a.V), 1.0, dtype=torch.float32, device=dev)
        zt = W.normal(33, "zt", (a.B, a.k, a.V), 1.0, dtype=torch.float32, device=dev)
        drafts = torch.zeros(a.B, a.k, dtype=torch.int32, device=dev)
        lse = torch.logsumexp(zt, dim=2).contiguous()
        zd = zt[:, :, 0].contiguous()
        u = torch.full((a.B, a.k), 0.5, device=dev)
        r = torch.full((a.B,), 0.5, device=dev)
        al = torch.empty(a.B, dtype=torch.int32, device=dev)
        oi = torch.empty(a.B, a.k, dtype=torch.int32, device=dev)
        no = torch.empty(a.B, dtype=torch.int32, device=dev)
        ws = torch.empty(L.deer_accept_workspace_bytes(L.DEER_ACC_SAMPLE, a.B, a.k, a.V), dtype=torch.uint8, device=dev)
        call = lambda: L.deer_accept(L.DEER_ACC_SAMPLE, a.B, a.k, a.V, drafts, None, zt, lse, zd, 1.0, ql, u, r, -1, al, oi, no, ws)
        nbytes = M * a.V * 4
        flops = 0.0

    for _ in range(a.warmup):
        call()
    torch.cuda.synchronize()
    for e0, e1 in ev:
        flush.zero_()
        flush_rd.max()          # read pass: leaves L2 full of clean lines
        e0.record()
        call()
        e1.record()
    torch.cuda.synchronize()
    ms = float(np.mean([e0.elapsed_time(e1) for e0, e1 in ev]))
    print(f"{a.what}: {ms * 1e3:.1f} us/call, {nbytes / ms / 1e6:.1f} GB/s over {nbytes} algorithmic bytes, "
          f"{flops / ms / 1e9:.1f} TFLOP/s")
    if a.probes:
        print_probes(a.what)


def print_probes(what: str) -> None:
    """The probe tables of the last call (library built with DEER_TIMING_PROBES)."""
    import ctypes
    lib = L.lib()
    buf = (ctypes.c_longlong * (64 * 8))()
    if what == "attn":
        lib.deer_attn_probe_read.argtypes = [ctypes.c_void_p]
        lib.deer_attn_probe_read(buf)
        d = np.array(buf[:], dtype=np.int64).reshape(64, 8)
        d = d[(d[:, :7] > 0).all(axis=1)]
        if len(d) < 8:
            print("probes: the probed block had too few tiles")
            return
        names = ["slot free seen", "K landed seen", "S committed", "S complete seen", "P handed over", "P+V seen", "O committed"]
        print(f"probes: {len(d)} tiles of one block; tile period {np.median(np.diff(d[:, 0])):.0f} cycles (median)")
        for j in range(6):
            print(f"  {names[j]:16s} -> {names[j + 1]:16s} {np.median(d[:, j + 1] - d[:, j]):7.0f} cycles")
        print(f"  {names[6]:16s} -> {names[0]:16s} {np.median(d[4:, 0] - d[:-4, 6]):7.0f} cycles (four tiles on: the ring's depth)")
    elif what == "lmhead":
        lib.deer_lmhead_probe_read.argtypes = [ctypes.c_void_p]
        lib.deer_lmhead_probe_read(buf)
        d = np.array(buf[:], dtype=np.int64).reshape(64, 8)
        d = d[d[:, 3] > 0]
        if len(d) == 0:
            print("probes: the block-pair kernel did not run (M <= 128)")
            return
        print(f"probes: {len(d)} leader blocks; {d[:, 3].mean():.0f} MMAs each, {(d[:, 0] / d[:, 3]).mean():.1f} cycles per MMA; "
              f"waiting for operands {100 * (d[:, 1] / d[:, 0]).mean():.1f} %, for an accumulator {100 * (d[:, 2] / d[:, 0]).mean():.1f} %, "
              f"issuing {100 * (1 - (d[:, 1] + d[:, 2]) / d[:, 0]).mean():.1f} %")


if __name__ == "__main__":
    main()
