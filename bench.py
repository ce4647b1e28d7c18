#!/usr/bin/env python
"""Benchmark of the DEER draft-verify step on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config 1] [--impl ours|reference]

A "step" is one pass of the whole hot path -- kv_reserve, block attention
(append), LM head + argmax, acceptance, kv_commit -- over one batch of seeded
synthetic input shaped like a Qwen3-8B verify step (workload index 1: batch 1,
32q/8kv heads, head_dim 128, context 4096, block 32, hidden 4096, vocab
151936).  Prints ONE JSON line.  With N > 1 (under torchrun) every rank runs an
independent replica on its own GPU; there is no data-path collective.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2512_15176_b200 import workload as W  # noqa: E402

METRIC = "verified draft tokens/s per verify step"
UNIT = "tokens/s"

# DRAM bytes (read + write) of one lmhead_umma_kernel launch from ncu, per workload name; absent = not captured for
# the kernel as it stands.  Captured at full size (M = 32, hidden 4096, V = 151936: 1 246 011 392 read + 5 147 392
# written, dram__bytes_{read,write}.sum alone, one launch), 1.005 x the algorithmic bytes.
LMHEAD_TRAFFIC = {"C2-qwen3-8b-verify": 1246011392 + 5147392}


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {"hbm_gbs": float(d["hbm_gbs"]), "bf16_tflops": float(d["bf16_tflops"]),
                "bf16_tflops_sustained": float(d.get("bf16_tflops_sustained", d["bf16_tflops"])), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples SM clock and throttle reasons through NVML (read-only queries) in
    a thread while the timed region runs."""

    REASONS = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown", 0x4: "sw_power_cap"}

    def __init__(self, gpu_index: int, period_s: float = 0.002):
        self.gpu, self.period = gpu_index, period_s
        self.sm, self.bits, self.max_mhz, self.power = [], 0, None, []
        self.stop_flag = threading.Event()
        self.thread = None
        self.err = None

    def start(self):
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            idx = self.gpu
            vis = os.environ.get("CUDA_VISIBLE_DEVICES")
            if vis:
                try:
                    idx = int(vis.split(",")[self.gpu])
                except Exception:
                    idx = self.gpu
            self.h = pynvml.nvmlDeviceGetHandleByIndex(idx)
            self.max_mhz = float(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
        except Exception as e:          # NVML missing: report it rather than guess
            self.err = repr(e)
            return
        self.thread = threading.Thread(target=self._loop, daemon=True)
        self.thread.start()

    def _loop(self):
        nv = self.nv
        while not self.stop_flag.is_set():
            try:
                self.sm.append(float(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)))
                self.bits |= int(nv.nvmlDeviceGetCurrentClocksEventReasons(self.h))
                self.power.append(nv.nvmlDeviceGetPowerUsage(self.h) / 1000.0)
            except Exception as e:
                self.err = repr(e)
                return
            time.sleep(self.period)

    def stop(self):
        if self.thread is None:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": ["clock sampling unavailable: %s" % self.err]}
        self.stop_flag.set()
        self.thread.join(timeout=2)
        reasons = sorted(name for bit, name in self.REASONS.items() if self.bits & bit)
        return {"sm_mhz": float(np.median(self.sm)) if self.sm else None, "sm_max_mhz": self.max_mhz, "reasons": reasons,
                "samples": len(self.sm), "power_w_max": max(self.power) if self.power else None}


def max_over_ranks(values, device, world):
    """Element-wise maximum of ``values`` over all ranks (the replicas are independent, so the job's time is the
    slowest rank's); with one rank the values themselves."""
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if world > 1:
        import torch.distributed as dist
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t]


def dist_env():
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    return rank, world, local


# ---------------------------------------------------------------------------
# oracle arm: the CPU oracle as it stands, on the host cores
# ---------------------------------------------------------------------------

def oracle_step_seconds(cfg, repeat=1):
    """One whole step of ``cfg`` through the oracle (attention, logits, argmax,
    greedy acceptance, KV append + commit).  Returns (seconds per step, tokens
    per step, description of the sample)."""
    import math
    from oracle import deer_oracle as O
    lengths = W.seq_lengths(cfg)
    lay = W.kv_layout(cfg, lengths)
    kp, vp = W.kv_pools(cfg, lay.num_pages)
    f32 = lambda t: t.to(torch.float32).numpy()
    kv = O.PagedKV(f32(kp), f32(vp), lay.page_table, lay.seq_len, lay.n_pages, lay.free_stack, lay.free_top)
    w = f32(W.lm_head(cfg))
    q, kb, vb = (f32(t) for t in W.block_qkv(cfg))
    h = f32(W.hidden(cfg))
    ids = np.arange(cfg.B)
    times = []
    snap = (kv.page_table.copy(), kv.seq_len.copy(), kv.n_pages.copy(), kv.free_stack.copy(), kv.free_top)
    for it in range(repeat):
        kv.page_table, kv.seq_len, kv.n_pages, kv.free_stack = (a.copy() for a in snap[:4])
        kv.free_top = snap[4]           # every repeat sees the same prefix
        t0 = time.perf_counter()
        kv.reserve(ids, cfg.k)
        O.block_attention(q, kb, vb, kv.k_pool, kv.v_pool, kv.page_table, kv.seq_len, ids, cfg.mask, 1.0 / math.sqrt(cfg.D))
        kv.append(ids, kb, vb)
        z = O.lm_logits(h, w)
        target = O.select_argmax(z).reshape(cfg.B, cfg.k)
        drafts = W.plant_drafts(cfg, target, W.planted_prefix_lengths(cfg, it), it)
        a, out, n = O.accept_greedy(drafts, target)
        kv.commit(ids, a)
        times.append(time.perf_counter() - t0)
    return float(np.mean(times)), cfg.M, f"whole step of {cfg.name} (all {cfg.M} block rows, full vocabulary), {repeat} run(s)"


def run_reference(args, cfg):
    rank, world, _ = dist_env()
    if rank != 0:
        return
    cores = len(os.sched_getaffinity(0))
    for _ in range(max(0, min(args.warmup, 1))):
        oracle_step_seconds(cfg, 1)
    reps = max(1, min(args.steps, 3))
    sec, toks, sample = oracle_step_seconds(cfg, reps)
    val = toks / sec
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": reps,
            "warmup": min(args.warmup, 1), "ms_per_step": sec * 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": cfg.name, "B": cfg.B, "k": cfg.k, "ctx": list(cfg.ctx), "hid": cfg.hid, "V": cfg.V},
            "cpu_baseline": {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# ---------------------------------------------------------------------------
# CUDA arm
# ---------------------------------------------------------------------------

def run_ours(args, cfg):
    rank, world, local = dist_env()
    if world > 1:
        import torch.distributed as dist
        torch.cuda.set_device(local)
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    from paper_2512_15176_b200 import binding as L
    from paper_2512_15176_b200.runner import VerifyStep
    L.lib()          # fail loudly if the library has not been built

    peaks = load_peaks()
    greedy = cfg.mode == "greedy"
    lengths = W.seq_lengths(cfg)
    lay = W.kv_layout(cfg, lengths)
    # pools of the larger workloads are drawn on the device (hundreds of MB); the values only feed the timing
    kp, vp = W.kv_pools(cfg, lay.num_pages, device="cpu" if lay.num_pages * cfg.Hkv * cfg.D < (1 << 22) else str(dev))
    kv = L.KVCache.from_layout(lay, kp, vp, dev)
    saved = [t.clone() for t in (kv.page_table, kv.seq_len, kv.n_pages, kv.free_stack, kv.free_top)]
    w = W.lm_head(cfg).to(dev)
    vs = VerifyStep(cfg, kv, w, int(lengths.max()), device=dev, store_logits=None if cfg.mode == "sample" else False)
    q, kb, vb = W.block_qkv(cfg)
    h = W.hidden(cfg)
    vs.load(q, kb, vb, h)

    def restore():
        for dst, src in zip((kv.page_table, kv.seq_len, kv.n_pages, kv.free_stack, kv.free_top), saved):
            dst.copy_(src)

    # drafts planted against the head's own argmax (an untimed pre-pass; only the
    # timing inputs come from it, never an expected value of a test)
    if cfg.mode == "sample":
        ql = W.draft_logits(cfg)
        drafts = W.sample_drafts(ql, cfg.seed)
        vs.load(draft_ids=drafts, q_logits=ql, u=W.uniform_open(cfg.seed, "u", (cfg.B, cfg.k)),
                r=W.uniform_open(cfg.seed, "r", (cfg.B,)))
        del ql
    else:
        vs.lmhead()
        torch.cuda.synchronize()
        target = vs.target_ids.cpu().numpy()
        drafts = W.plant_drafts(cfg, target, W.planted_prefix_lengths(cfg))
        vs.load(draft_ids=drafts)
    bidir = cfg.mask == W.MASK_BIDIR
    flush = torch.empty(512 << 20, dtype=torch.uint8, device=dev)
    flush_rd = torch.zeros(64 << 20, dtype=torch.int32, device=dev)      # 256 MiB

    def flush_l2():
        """Evict L2 between steps: a 512 MiB write, then a 256 MiB read so that the
        write's dirty lines are back in HBM before the timed step starts."""
        flush.zero_()
        flush_rd.max()

    def phase_attn():
        if not bidir:
            vs.fork_draft_stats()          # sampling: the drafter-logit pass starts on a second stream (joined by accept)
            vs.reserve()
        vs.attn(append=not bidir)

    def phase_accept():
        if not bidir:              # the drafter's block fill proposes; nothing is accepted or committed
            vs.accept()
            vs.commit()

    phases = [phase_attn, vs.lmhead, phase_accept]

    def one_step(events=None):
        restore()
        flush_l2()
        for i, ph in enumerate(phases):
            if events is not None:
                events[i].record()
            ph()
        if events is not None:
            events[3].record()

    for _ in range(max(args.warmup, 3)):
        one_step()
    torch.cuda.synchronize()
    graph, gev = None, None
    if not args.no_graph:
        # The whole step is replayed from one CUDA graph, with timing events recorded inside it between the phases:
        # the host's launch work no longer paces the GPU.  The calls and their arguments are exactly the ones above.
        gev = [torch.cuda.Event(enable_timing=True, external=True) for _ in range(4)]
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            for i, ph in enumerate(phases):
                gev[i].record()
                ph()
            gev[3].record()
        for _ in range(3):
            restore()
            flush_l2()
            graph.replay()
        torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(args.steps)]
    marks = []          # per step: ms from the step's start to the end of each phase
    torch.cuda.synchronize()
    wall0 = time.perf_counter()
    for s in range(args.steps):
        if graph is None:
            one_step(evs[s])
        else:
            restore()
            flush_l2()
            graph.replay()
            torch.cuda.synchronize()          # the graph's events are re-recorded by the next replay: read them now
            marks.append([gev[0].elapsed_time(gev[i]) for i in (1, 2, 3)])
    torch.cuda.synchronize()
    wall = time.perf_counter() - wall0
    if world > 1:
        dist.barrier()
    clocks = sampler.stop() if rank == 0 else None
    if graph is None:
        marks = [[e[0].elapsed_time(e[i]) for i in (1, 2, 3)] for e in evs]
    step_ms = [m[2] for m in marks]
    attn_ms = [m[0] for m in marks]
    lm_ms = [m[1] - m[0] for m in marks]
    total_ms = float(sum(step_ms))
    status = L.deer_kv_status(kv)
    accepted = int(vs.accept_len.sum().item())

    # ---- end to end: host buffers in, verdict out, every step (the greedy verify step has such a call) ----
    e2e_s, h2d, d2h = 0.0, 0, 0
    if greedy:
        pin = lambda t: t.contiguous().pin_memory()
        hq, hkb, hvb, hh = pin(q), pin(kb), pin(vb), pin(h)
        hd = pin(torch.from_numpy(drafts))
        ha = torch.empty(cfg.B, dtype=torch.int32).pin_memory()
        ho = torch.empty(cfg.B, cfg.k, dtype=torch.int32).pin_memory()
        hn = torch.empty(cfg.B, dtype=torch.int32).pin_memory()
        sd = L.deer_step_dev(vs.q.data_ptr(), vs.k_blk.data_ptr(), vs.v_blk.data_ptr(), vs.attn_out.data_ptr(), vs.h.data_ptr(),
                             vs.seq_ids.data_ptr(), vs.draft_ids.data_ptr(), vs.target_ids.data_ptr(), vs.accept_len.data_ptr(),
                             vs.out_ids.data_ptr(), vs.n_out.data_ptr(), vs.attn_ws.data_ptr(), vs.attn_ws.numel(),
                             vs.lm_ws.data_ptr(), vs.lm_ws.numel())
        h2d = sum(t.numel() * t.element_size() for t in (hq, hkb, hvb, hh, hd))
        d2h = sum(t.numel() * t.element_size() for t in (ha, ho, hn))
        es = torch.cuda.Stream()          # a stream of its own: the call replays its copies and kernels as one graph there
        for s in range(3 + args.steps):
            restore()
            flush_l2()
            torch.cuda.synchronize()
            t0 = time.perf_counter()
            L.deer_verify_step_host(kv, sd, w, hq, hkb, hvb, hh, hd, cfg.B, cfg.k, cfg.Hq, cfg.hid, cfg.V, vs.scale,
                                    int(lengths.max()), ha, ho, hn, stream=es)
            dt = time.perf_counter() - t0
            if s >= 3:
                e2e_s += dt
    total_s, e2e_total = max_over_ranks([total_ms / 1e3, e2e_s], dev, world)
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    tokens = cfg.M * args.steps * world
    value = tokens / total_s
    ab = W.algorithmic_bytes(cfg, lengths)
    fl = W.algorithmic_flops(cfg, lengths)
    hbm, tens = peaks["hbm_gbs"] * 1e9, peaks["bf16_tflops_sustained"] * 1e12
    attn_s, lm_s = float(np.mean(attn_ms)) / 1e3, float(np.mean(lm_ms)) / 1e3
    step_s = total_s / args.steps
    # the dominant kernel is the LM head; it is HBM-bound below about hbm-ridge rows and tensor-bound above
    lm_tensor_bound = fl["lmhead"] / tens > ab["lmhead"] / hbm
    if lm_tensor_bound:
        achieved, peak, unit, bound = fl["lmhead"] / lm_s / 1e12, peaks["bf16_tflops_sustained"], "TFLOP/s", "tensor"
    else:
        achieved, peak, unit, bound = ab["lmhead"] / lm_s / 1e9, peaks["hbm_gbs"], "GB/s", "hbm"
    floor_s = (max(ab["attn"] / hbm, fl["attn"] / tens) + max(ab["lmhead"] / hbm, fl["lmhead"] / tens) + ab["accept"] / hbm)
    accept_text = {"greedy": "greedy, planted Geometric(0.1) prefix capped at k",
                   "argmax_logprob": "none (drafter block fill: argmax + max log-probability per position)",
                   "sample": "rejection sampling at temperature %.2g with residual resampling" % cfg.temperature}[cfg.mode]
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
        "ms_per_step": step_s * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": {"workload": cfg.name, "B": cfg.B, "k": cfg.k, "Hq": cfg.Hq, "Hkv": cfg.Hkv, "D": cfg.D,
                   "ctx": [int(lengths.min()), int(lengths.max())], "hid": cfg.hid, "V": cfg.V,
                   "mask": "bidirectional" if bidir else "causal", "accept": accept_text, "parallelism": f"replicas x{world}",
                   "launch": "host launches" if args.no_graph else "one CUDA graph per step, timing events recorded inside it",
                   "l2": "flushed between steps by a 512 MiB write followed by a 256 MiB read; the weight stream exceeds L2 by itself"},
        "roofline": {"bound": bound, "kernel": "deer_lmhead_select", "achieved": achieved, "peak": peak,
                     "unit": unit, "frac": achieved / peak, "traffic": LMHEAD_TRAFFIC.get(cfg.name), "peak_source": peaks["source"],
                     "bytes_per_launch": ab["lmhead"], "flops_per_launch": fl["lmhead"], "avg_launch_ms": lm_s * 1e3,
                     "step_frac_of_roofline_floor": floor_s / step_s, "step_floor_ms": floor_s * 1e3},
        "phases": {"attn_ms": attn_s * 1e3, "attn_gbs": ab["attn"] / attn_s / 1e9, "attn_frac_of_hbm": ab["attn"] / attn_s / hbm,
                   "attn_tflops": fl["attn"] / attn_s / 1e12, "lmhead_ms": lm_s * 1e3, "lmhead_gbs": ab["lmhead"] / lm_s / 1e9,
                   "lmhead_tflops": fl["lmhead"] / lm_s / 1e12, "accept_commit_ms": (step_s - attn_s - lm_s) * 1e3},
        "e2e": ({"value": cfg.M * args.steps * world / e2e_total, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                 "ms_per_step": e2e_total * 1e3 / args.steps} if greedy else
                {"value": None, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0,
                 "note": "the host-buffer entry point covers the greedy verify step only"}),
        "gpu_launches": args.steps * vs.launches_per_step(),
        "clocks": clocks,
        "kv_status": status, "accepted_tokens_last_step": accepted, "wall_s_timed_loop": wall,
        "flops_per_step": fl["total"],
    }
    if world == 1 and greedy and not args.no_cpu_baseline:
        sec, toks, sample = oracle_step_seconds(cfg, 1)
        line["cpu_baseline"] = {"value": toks / sec, "unit": UNIT, "cores": len(os.sched_getaffinity(0)), "kind": "oracle",
                                "sample": sample}
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--config", type=int, default=1, help="workload index 0..3 (1 = Qwen3-8B-shaped verify step)")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-graph", action="store_true", help="launch every call from the host instead of replaying CUDA graphs")
    ap.add_argument("--sweep-point", default=None, metavar="B,CTX,K,MASK",
                    help="time one point of the sweep instead of a fixed workload: batch, context (ragged lengths in "
                         "[CTX/2, CTX]), block size, causal|bidir")
    args = ap.parse_args()
    if args.sweep_point:
        b, ctx, k, mask = args.sweep_point.split(",")
        cfg = W.sweep_config(int(b), int(ctx), int(k), W.MASK_BIDIR if mask == "bidir" else W.MASK_CAUSAL, steps=1)
        if mask == "bidir":
            cfg = cfg.with_(mode="argmax_logprob")
        args.no_cpu_baseline = True
    else:
        cfg = W.config(args.config)
    if args.impl == "reference" and cfg.mode != "greedy":
        raise SystemExit("the oracle arm times the greedy verify step (workload 0 or 1)")
    if args.impl == "reference":
        run_reference(args, cfg)
    else:
        run_ours(args, cfg)


if __name__ == "__main__":
    main()
