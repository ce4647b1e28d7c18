#!/usr/bin/env python
"""Benchmark of the DEER draft-verify step on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config 1] [--impl ours|reference]
    python bench.py --sweep [--steps K]          # every point of the sweep -> profiles/sweep.md

A "step" is one pass of the whole hot path -- kv_reserve, block attention
(append), LM head + argmax, acceptance, kv_commit -- over one batch of seeded
synthetic input.  The headline workload is the Qwen3-8B-shaped verify step
(workload index 1: batch 1, 32q/8kv heads, head_dim 128, context 4096, block
32, hidden 4096, vocab 151936); the same JSON line carries, under
``workloads``, the drafter block fill, the Qwen3-30B-A3B-shaped sampling step
and one large sweep point, each timed the same way.  Prints ONE JSON line.
With N > 1 (under torchrun) every rank runs an independent replica on its own
GPU; there is no data-path collective.
"""
from __future__ import annotations

import argparse
import hashlib
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
TRAFFIC_FILE = os.path.join(ROOT, "profiles", "dram_traffic.json")
KERNEL_SOURCES = {"lmhead_umma_kernel": ["paper_2512_15176_b200/csrc/lmhead_umma.cu", "paper_2512_15176_b200/csrc/sm100.cuh",
                                         "paper_2512_15176_b200/csrc/lmhead.cuh"]}


def kernel_source_hash(kernel: str) -> str:
    h = hashlib.sha256()
    for rel in KERNEL_SOURCES[kernel]:
        with open(os.path.join(ROOT, rel), "rb") as f:
            h.update(f.read())
    return h.hexdigest()[:16]


def recorded_traffic(kernel: str, workload: str):
    """DRAM bytes (read + write) of one launch of ``kernel`` on ``workload`` as a profiler counted them, from the
    tracked file beside the profile summaries -- or None when nothing was recorded for this workload, or when the
    kernel's sources have changed since (the record carries their hash)."""
    try:
        with open(TRAFFIC_FILE) as f:
            rec = json.load(f).get(kernel, {}).get(workload)
    except (OSError, ValueError):
        return None
    if not rec or rec.get("source_sha16") != kernel_source_hash(kernel):
        return None
    return int(rec["dram_bytes_read"]) + int(rec["dram_bytes_write"])


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {"hbm_gbs": float(d["hbm_gbs"]), "bf16_tflops": float(d["bf16_tflops"]),
                "bf16_tflops_sustained": float(d.get("bf16_tflops_sustained", d["bf16_tflops"])), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples SM clock and throttle reasons through NVML (read-only queries) in
    a thread, back to back (a query takes a fraction of a millisecond), from the
    warm-up replays to the end of the timed region."""

    REASONS = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown", 0x4: "sw_power_cap"}

    def __init__(self, gpu_index: int, period_s: float = 0.0002):
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
        n = 0
        while not self.stop_flag.is_set():
            try:
                self.sm.append(float(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)))
                self.bits |= int(nv.nvmlDeviceGetCurrentClocksEventReasons(self.h))
                if n % 16 == 0:
                    self.power.append(nv.nvmlDeviceGetPowerUsage(self.h) / 1000.0)
            except Exception as e:
                self.err = repr(e)
                return
            n += 1
            time.sleep(self.period)

    def stop(self):
        if self.thread is None:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": ["clock sampling unavailable: %s" % self.err]}
        self.stop_flag.set()
        self.thread.join(timeout=2)
        reasons = sorted(name for bit, name in self.REASONS.items() if self.bits & bit)
        return {"sm_mhz": float(np.median(self.sm)) if self.sm else None, "sm_min_mhz": float(min(self.sm)) if self.sm else None,
                "sm_max_mhz": self.max_mhz, "reasons": reasons, "samples": len(self.sm),
                "power_w_max": max(self.power) if self.power else None}


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


def config_dict(cfg, world):
    """What both arms print as ``config``: the workload, and how the CUDA arm is launched and keeps L2 cold."""
    lengths = W.seq_lengths(cfg)
    bidir = cfg.mask == W.MASK_BIDIR
    accept_text = {"greedy": "greedy, planted Geometric(0.1) prefix capped at k",
                   "argmax_logprob": "none (drafter block fill: argmax + max log-probability per position)",
                   "sample": "rejection sampling at temperature %.2g with residual resampling" % cfg.temperature}[cfg.mode]
    return {"workload": cfg.name, "B": cfg.B, "k": cfg.k, "Hq": cfg.Hq, "Hkv": cfg.Hkv, "D": cfg.D,
            "ctx": [int(lengths.min()), int(lengths.max())], "hid": cfg.hid, "V": cfg.V,
            "mask": "bidirectional" if bidir else "causal", "accept": accept_text, "parallelism": f"replicas x{world}",
            "launch": "CUDA arm: one CUDA graph per step, timed by events at its two ends",
            "l2": "CUDA arm: flushed between steps by a 512 MiB write followed by a 256 MiB read; the weight stream "
                  "exceeds L2 by itself"}


# ---------------------------------------------------------------------------
# oracle arm: the CPU oracle as it stands, on the host cores
# ---------------------------------------------------------------------------

class OracleStep:
    """One whole step of ``cfg`` through the oracle (attention, logits, argmax, greedy acceptance, KV append +
    commit).  ``vocab_rows`` < V bounds the sample: the logits are then taken against the first vocab_rows rows of
    the head only (everything else is done in full)."""

    def __init__(self, cfg, vocab_rows=None):
        from oracle import deer_oracle as O
        self.O, self.cfg = O, cfg
        lengths = W.seq_lengths(cfg)
        lay = W.kv_layout(cfg, lengths)
        kp, vp = W.kv_pools(cfg, lay.num_pages)
        f32 = lambda t: t.to(torch.float32).numpy()
        self.kv = O.PagedKV(f32(kp), f32(vp), lay.page_table, lay.seq_len, lay.n_pages, lay.free_stack, lay.free_top)
        self.w = f32(W.lm_head(cfg))
        self.vocab_rows = cfg.V if vocab_rows is None else int(vocab_rows)
        self.q, self.kb, self.vb = (f32(t) for t in W.block_qkv(cfg))
        self.h = f32(W.hidden(cfg))
        kv = self.kv
        self.snap = (kv.page_table.copy(), kv.seq_len.copy(), kv.n_pages.copy(), kv.free_stack.copy(), kv.free_top)

    def run(self, it=0) -> float:
        import math
        O, cfg, kv = self.O, self.cfg, self.kv
        kv.page_table, kv.seq_len, kv.n_pages, kv.free_stack = (a.copy() for a in self.snap[:4])
        kv.free_top = self.snap[4]           # every run sees the same prefix
        ids = np.arange(cfg.B)
        t0 = time.perf_counter()
        kv.reserve(ids, cfg.k)
        O.block_attention(self.q, self.kb, self.vb, kv.k_pool, kv.v_pool, kv.page_table, kv.seq_len, ids, cfg.mask,
                          1.0 / math.sqrt(cfg.D))
        kv.append(ids, self.kb, self.vb)
        z = O.lm_logits(self.h, self.w[:self.vocab_rows])
        target = O.select_argmax(z).reshape(cfg.B, cfg.k)
        drafts = W.plant_drafts(cfg, target, W.planted_prefix_lengths(cfg, it), it)
        a, out, n = O.accept_greedy(drafts, target)
        kv.commit(ids, a)
        return time.perf_counter() - t0

    def sample_text(self, runs):
        cfg = self.cfg
        if self.vocab_rows == cfg.V:
            return f"whole step of {cfg.name} (all {cfg.M} block rows, full vocabulary), {runs} timed run(s) after a warm-up run"
        return (f"step of {cfg.name} with the logits taken against the first {self.vocab_rows} of {cfg.V} vocabulary rows "
                f"(all {cfg.M} block rows, attention and acceptance in full); tokens/s scaled by {self.vocab_rows}/{cfg.V}; "
                f"{runs} timed run(s) after a warm-up run")


def run_reference(args, cfg):
    rank, world, _ = dist_env()
    if rank != 0:
        return
    cores = len(os.sched_getaffinity(0))
    budget_s = 150.0
    st = OracleStep(cfg)
    t_full = st.run()                                   # untimed: pages the inputs in, and sizes the sample
    n_runs = args.steps + max(0, args.warmup - 1)
    if n_runs * t_full > budget_s:
        rows = max(1024, int(cfg.V * budget_s / (n_runs * t_full)) // 1024 * 1024)
        st = OracleStep(cfg, vocab_rows=min(rows, cfg.V))
    for _ in range(max(0, args.warmup - 1)):
        st.run()
    secs = [st.run(it) for it in range(args.steps)]
    sec = float(np.mean(secs))
    val = cfg.M * (st.vocab_rows / cfg.V) / sec
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": sec * 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": config_dict(cfg, world),
            "cpu_baseline": {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": st.sample_text(args.steps)},
            "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# ---------------------------------------------------------------------------
# CUDA arm
# ---------------------------------------------------------------------------

_W_CACHE = {}


def head_weights(cfg, dev, on_device):
    """The LM-head weights of ``cfg`` on ``dev`` (the last one is kept: sweep points share theirs).  ``on_device``
    draws them with the device generator -- other values than the host draw the tests use, which is fine where they
    only feed a timing."""
    key = (cfg.seed, cfg.V, cfg.hid, cfg.sigma_w, bool(on_device), str(dev))
    if key not in _W_CACHE:
        _W_CACHE.clear()
        torch.cuda.empty_cache()
        _W_CACHE[key] = (W.normal(cfg.seed, "w", (cfg.V, cfg.hid), cfg.sigma_w, device=str(dev)) if on_device
                         else W.lm_head(cfg).to(dev))
    return _W_CACHE[key]


class Flusher:
    def __init__(self, dev):
        self.wr = torch.empty(512 << 20, dtype=torch.uint8, device=dev)
        self.rd = torch.zeros(64 << 20, dtype=torch.int32, device=dev)      # 256 MiB

    def __call__(self):
        """Evict L2 between steps: a 512 MiB write, then a 256 MiB read so that the
        write's dirty lines are back in HBM before the timed step starts."""
        self.wr.zero_()
        self.rd.max()


def measure(cfg, steps, warmup, dev, peaks, flush, world=1, rank=0, with_e2e=False, clock_sampler=None, device_weights=False,
            consecutive=False):
    """Times ``steps`` steps of ``cfg`` on the current device.  Returns a dict with the step time (events at the two
    ends of the step's graph), the phase split (a second graph with events between the phases), the roofline of the
    LM-head call and of the whole step.  ``consecutive``: the timed steps follow one another on the same cache --
    every step commits what it accepted, the contexts grow, and each step gets freshly planted drafts -- instead of
    starting from the same state each time."""
    from paper_2512_15176_b200 import binding as L
    from paper_2512_15176_b200.runner import VerifyStep
    import torch.distributed as dist

    greedy = cfg.mode == "greedy"
    lengths = W.seq_lengths(cfg)
    lay = W.kv_layout(cfg, lengths)
    # pools of the larger workloads are drawn on the device (hundreds of MB); the values only feed the timing
    kp, vp = W.kv_pools(cfg, lay.num_pages, device="cpu" if lay.num_pages * cfg.Hkv * cfg.D < (1 << 22) else str(dev))
    kv = L.KVCache.from_layout(lay, kp, vp, dev)
    del kp, vp
    saved = [t.clone() for t in (kv.page_table, kv.seq_len, kv.n_pages, kv.free_stack, kv.free_top)]
    w = head_weights(cfg, dev, device_weights)
    max_seq_len = int(lengths.max()) + cfg.growth           # consecutive steps grow the contexts
    vs = VerifyStep(cfg, kv, w, max_seq_len, device=dev, store_logits=None if cfg.mode == "sample" else False)
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
    step_drafts = None
    if consecutive and greedy and not bidir:
        # the hidden states stay, so the targets do; every step gets its own planted prefix lengths
        step_drafts = torch.stack([torch.from_numpy(W.plant_drafts(cfg, target, W.planted_prefix_lengths(cfg, s), s))
                                   for s in range(steps)]).to(dev)

    def phase_attn():
        if not bidir:
            vs.fork_draft_stats()          # sampling: the drafter-logit pass starts on a second stream (joined by accept)
            vs.reserve()
        vs.attn(append=not bidir)

    def phase_accept():
        if not bidir:              # the drafter's block fill proposes; nothing is accepted or committed
            vs.accept_commit()

    phases = [phase_attn, vs.lmhead, phase_accept]

    def eager_step():
        restore()
        flush()
        for ph in phases:
            ph()

    if clock_sampler is not None:
        clock_sampler.start()
    for _ in range(max(warmup, 3)):
        eager_step()
    torch.cuda.synchronize()
    # The whole step is replayed from one CUDA graph: the host's launch work does not pace the GPU.  Graph A carries
    # timing events at its two ends only (the step time); graph B also between the phases (the split).
    def capture(inner):
        ev = [torch.cuda.Event(enable_timing=True, external=True) for _ in range(4)]
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            ev[0].record()
            for i, ph in enumerate(phases):
                if inner and i > 0:
                    ev[i].record()
                ph()
            ev[3].record()
        return g, ev

    g_step, ev_step = capture(False)
    g_ph, ev_ph = capture(True)

    def replay(g):
        restore()
        flush()
        g.replay()
        torch.cuda.synchronize()          # the graph's events are re-recorded by the next replay: read them now

    for g in (g_step, g_ph):
        for _ in range(3):
            replay(g)
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    wall0 = time.perf_counter()
    step_ms = []
    if step_drafts is not None:
        restore()
    for s_i in range(steps):
        if step_drafts is not None:
            vs.draft_ids.copy_(step_drafts[s_i])
            flush()
            g_step.replay()
            torch.cuda.synchronize()
        else:
            replay(g_step)
        step_ms.append(ev_step[0].elapsed_time(ev_step[3]))
    torch.cuda.synchronize()
    wall = time.perf_counter() - wall0
    if world > 1:
        dist.barrier()
    marks = []
    for _ in range(min(steps, 50)):
        replay(g_ph)
        marks.append([ev_ph[0].elapsed_time(ev_ph[i]) for i in (1, 2, 3)])
    status = L.deer_kv_status(kv)
    accepted = int(vs.accept_len.sum().item()) if not bidir else None
    # The drafts were planted against the head's own argmax, so the accepted lengths of the timed steps must be the
    # planted prefix lengths: what was timed did the work.
    planted_ok = None
    if greedy and not bidir:
        last = steps - 1 if step_drafts is not None else 0
        want = W.planted_prefix_lengths(cfg, last) if step_drafts is not None else W.planted_prefix_lengths(cfg)
        planted_ok = bool((vs.accept_len.cpu().numpy() == want).all())
        if not planted_ok:
            raise RuntimeError(f"{cfg.name}: accepted lengths differ from the planted prefix lengths")

    # ---- end to end: host buffers in, results out, every step (the greedy verify step has such a call) ----
    e2e_s, h2d, d2h = 0.0, 0, 0
    if greedy and with_e2e:
        pin = lambda t: t.contiguous().pin_memory()
        # q, k_blk, v_blk side by side in one pinned buffer and one device buffer, the three results likewise: the call
        # then moves each group with one copy
        nq, nk = q.numel(), kb.numel()
        hin = torch.empty(nq + 2 * nk, dtype=torch.bfloat16).pin_memory()
        hq, hkb, hvb = hin[:nq].view_as(q), hin[nq:nq + nk].view_as(kb), hin[nq + nk:].view_as(vb)
        hq.copy_(q), hkb.copy_(kb), hvb.copy_(vb)
        hh = pin(h)
        hd = pin(torch.from_numpy(drafts))
        hout = torch.empty(2 * cfg.B + cfg.M, dtype=torch.int32).pin_memory()
        ha, ho, hn = hout[:cfg.B], hout[cfg.B:cfg.B + cfg.M].view(cfg.B, cfg.k), hout[cfg.B + cfg.M:]
        din = torch.empty(nq + 2 * nk, dtype=torch.bfloat16, device=dev)
        dout = torch.empty(2 * cfg.B + cfg.M, dtype=torch.int32, device=dev)
        sd = L.deer_step_dev(din.data_ptr(), din[nq:].data_ptr(), din[nq + nk:].data_ptr(), vs.attn_out.data_ptr(), vs.h.data_ptr(),
                             vs.seq_ids.data_ptr(), vs.draft_ids.data_ptr(), vs.target_ids.data_ptr(), dout.data_ptr(),
                             dout[cfg.B:].data_ptr(), dout[cfg.B + cfg.M:].data_ptr(), vs.attn_ws.data_ptr(), vs.attn_ws.numel(),
                             vs.lm_ws.data_ptr(), vs.lm_ws.numel())
        h2d = sum(t.numel() * t.element_size() for t in (hq, hkb, hvb, hh, hd))
        d2h = sum(t.numel() * t.element_size() for t in (ha, ho, hn))
        es = torch.cuda.Stream()          # a stream of its own: the call replays its copies and kernels as one graph there
        for s in range(3 + steps):
            restore()
            flush()
            torch.cuda.synchronize()
            t0 = time.perf_counter()
            L.deer_verify_step_host(kv, sd, w, hq, hkb, hvb, hh, hd, cfg.B, cfg.k, cfg.Hq, cfg.hid, cfg.V, vs.scale,
                                    max_seq_len, ha, ho, hn, stream=es)
            dt = time.perf_counter() - t0
            if s >= 3:
                e2e_s += dt
        if not (ha.numpy() == W.planted_prefix_lengths(cfg)).all():
            raise RuntimeError(f"{cfg.name}: the host-buffer step's accepted lengths differ from the planted prefix lengths")
    clocks = clock_sampler.stop() if clock_sampler is not None else None
    total_s, e2e_total = max_over_ranks([float(sum(step_ms)) / 1e3, e2e_s], dev, world)

    ab = W.algorithmic_bytes(cfg, lengths)
    fl = W.algorithmic_flops(cfg, lengths)
    hbm, tens = peaks["hbm_gbs"] * 1e9, peaks["bf16_tflops_sustained"] * 1e12
    m = np.asarray(marks, dtype=np.float64)
    attn_s, lm_s, acc_s = float(m[:, 0].mean()) / 1e3, float((m[:, 1] - m[:, 0]).mean()) / 1e3, float((m[:, 2] - m[:, 1]).mean()) / 1e3
    step_s = total_s / steps
    # the dominant kernel is the LM head; it is HBM-bound below about hbm-ridge rows and tensor-bound above
    if fl["lmhead"] / tens > ab["lmhead"] / hbm:
        achieved, peak, unit, bound = fl["lmhead"] / lm_s / 1e12, peaks["bf16_tflops_sustained"], "TFLOP/s", "tensor"
    else:
        achieved, peak, unit, bound = ab["lmhead"] / lm_s / 1e9, peaks["hbm_gbs"], "GB/s", "hbm"
    attn_floor = max(ab["attn"] / hbm, fl["attn"] / tens)
    lm_floor = max(ab["lmhead"] / hbm, fl["lmhead"] / tens)
    floor_s = attn_floor + lm_floor + ab["accept"] / hbm
    out = {
        "config": config_dict(cfg, world),
        "ms_per_step": step_s * 1e3,
        "value": cfg.M * steps * world / total_s,
        "steps": steps,
        "roofline": {"bound": bound, "kernel": "lmhead_umma_kernel" if cfg.M <= 128 else "lmhead_umma_pair_kernel",
                     "achieved": achieved, "peak": peak, "unit": unit, "frac": achieved / peak,
                     "traffic": recorded_traffic("lmhead_umma_kernel", cfg.name) if cfg.M <= 128 else None,
                     "peak_source": peaks["source"] + (" (sustained)" if bound == "tensor" else ""),
                     "bytes_per_launch": ab["lmhead"], "flops_per_launch": fl["lmhead"], "avg_launch_ms": lm_s * 1e3,
                     "step_frac_of_roofline_floor": floor_s / step_s, "step_floor_ms": floor_s * 1e3,
                     "attn_plus_lmhead_frac_of_floor": (attn_floor + lm_floor) / (attn_s + lm_s)},
        "phases": {"attn_ms": attn_s * 1e3, "attn_gbs": ab["attn"] / attn_s / 1e9, "attn_frac_of_hbm": ab["attn"] / attn_s / hbm,
                   "attn_tflops": fl["attn"] / attn_s / 1e12, "attn_frac_of_floor": attn_floor / attn_s,
                   "lmhead_ms": lm_s * 1e3, "lmhead_gbs": ab["lmhead"] / lm_s / 1e9, "lmhead_tflops": fl["lmhead"] / lm_s / 1e12,
                   "accept_commit_ms": acc_s * 1e3, "step_ms_with_phase_events": float(m[:, 2].mean())},
        "gpu_launches": steps * vs.launches_per_step(),
        "kv_status": status, "accepted_tokens_last_step": accepted, "accepted_equals_planted": planted_ok,
        "wall_s_timed_loop": wall,
        "consecutive_steps": bool(step_drafts is not None),
        "flops_per_step": fl["total"], "clocks": clocks,
    }
    if greedy and with_e2e:
        out["e2e"] = {"value": cfg.M * steps * world / e2e_total, "unit": UNIT, "h2d_bytes_per_step": h2d,
                      "d2h_bytes_per_step": d2h, "ms_per_step": e2e_total * 1e3 / steps}
    del vs, kv, w
    torch.cuda.empty_cache()
    return out


def measure_layer(name, dev, peaks, flush, B, k, ctx, hid, Hq, Hkv, D, inter, moe=None, layers=1, steps=20):
    """One verifier layer (or a short stack) around the block attention at the M = B k rows of a draft block, on the
    fused calls, replayed from a CUDA graph with L2 flushed between replays.  The floor is the time the weights
    (for a routed MLP: the experts the rows really chose) and the live KV take at the measured HBM peak."""
    from paper_2512_15176_b200 import binding as L
    from paper_2512_15176_b200.runner import VerifierStack
    cfg = W.StepConfig(name, B, Hq, Hkv, D, k, hid, 64, (ctx, ctx), seed=34, growth=k)
    lengths = W.seq_lengths(cfg)
    lay = W.kv_layout(cfg, lengths)
    i32 = lambda a: torch.from_numpy(a.copy()).to(device=dev, dtype=torch.int32).contiguous()
    shared = [i32(a) for a in (lay.page_table, lay.seq_len, lay.n_pages, lay.free_stack, lay.free_top)]
    mk = lambda n, shape, sig: W.normal(34, n, shape, sig, device=str(dev))
    QD, KD = Hq * D, Hkv * D
    kvs, weights, w_bytes = [], [], 0
    for l in range(layers):
        kp, vp = W.kv_pools(cfg.with_(seed=34 + l), lay.num_pages, device=str(dev), sigma=1.0)
        kvs.append(L.KVCache(kp, vp, *shared))
        w = {"ln1": mk(f"ln1{l}", (hid,), 1.0), "ln2": mk(f"ln2{l}", (hid,), 1.0), "q_norm": mk(f"qn{l}", (D,), 1.0),
             "k_norm": mk(f"kn{l}", (D,), 1.0), "wqkv": mk(f"wqkv{l}", (QD + 2 * KD, hid), hid ** -0.5),
             "wo": mk(f"wo{l}", (hid, QD), QD ** -0.5)}
        if moe:
            E, top_k = moe
            w.update({"w_router": mk(f"wr{l}", (E, hid), hid ** -0.5 * 3.0), "w_gate_up": mk(f"wgue{l}", (E, 2 * inter, hid), hid ** -0.5),
                      "w_down": mk(f"wde{l}", (E, hid, inter), inter ** -0.5)})
        else:
            w.update({"wgu": mk(f"wgu{l}", (2 * inter, hid), hid ** -0.5), "wd": mk(f"wd{l}", (hid, inter), inter ** -0.5)})
        weights.append(w)
    x = mk("x", (cfg.M, hid), 1.0)
    stack = VerifierStack(cfg, kvs, weights, ctx + k, inter, fused=True, moe=moe)
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())           # the weights and pools were drawn on the current stream
    with torch.cuda.stream(side):
        for _ in range(3):
            stack.forward(x)
        side.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=side):
            stack.forward(x)
    torch.cuda.synchronize()
    # bytes the layers must move: dense weights once, the chosen experts' matrices once, the live KV once
    for l, w in enumerate(weights):
        w_bytes += sum(t.numel() * 2 for n, t in w.items() if n in ("wqkv", "wo", "wgu", "wd", "w_router"))
        if moe:
            e_ids = torch.empty(cfg.M, moe[1], dtype=torch.int32, device=dev)
            e_w = torch.empty(cfg.M, moe[1], dtype=torch.float32, device=dev)
            L.deer_moe_route(stack.layers[l].xn2, w["w_router"], moe[1], e_ids, e_w)
            torch.cuda.synchronize()
            w_bytes += int(torch.unique(e_ids).numel()) * 3 * inter * hid * 2
    kv_bytes = layers * W.algorithmic_bytes(cfg, lengths)["attn"]
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    for e0, e1 in ev:
        flush()
        e0.record()
        g.replay()
        e1.record()
    torch.cuda.synchronize()
    ms = float(np.mean([e0.elapsed_time(e1) for e0, e1 in ev]))
    floor_ms = (w_bytes + kv_bytes) / (peaks["hbm_gbs"] * 1e9) * 1e3
    status = [L.deer_kv_status(kv) for kv in kvs]
    del stack, kvs, weights
    torch.cuda.empty_cache()
    return {"config": {"workload": name, "B": B, "k": k, "ctx": ctx, "hid": hid, "Hq": Hq, "Hkv": Hkv, "D": D, "inter": inter,
                       "experts": list(moe) if moe else None, "layers": layers, "calls": "fused"},
            "ms_per_layer": ms / layers, "bytes_per_layer": (w_bytes + kv_bytes) / layers,
            "gbs": (w_bytes + kv_bytes) / ms / 1e6, "frac_of_hbm_floor": floor_ms / ms, "kv_status": max(status)}


def run_ours(args, cfg):
    rank, world, local = dist_env()
    if world > 1:
        import torch.distributed as dist
        torch.cuda.set_device(local)
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    from paper_2512_15176_b200 import binding as L
    L.lib()          # fail loudly if the library has not been built

    peaks = load_peaks()
    flush = Flusher(dev)
    sampler = ClockSampler(local) if rank == 0 else None
    head = measure(cfg, args.steps, args.warmup, dev, peaks, flush, world, rank, with_e2e=True, clock_sampler=sampler)

    # the other named workloads, one GPU's worth each (rank 0 of a multi-rank job skips them: the job's line is the
    # headline's replicas)
    others = {}
    if world == 1 and not args.no_workloads and not args.sweep_point and args.config == 1:
        extra_steps = min(args.steps, 20)
        for name, c in (("C3", W.config(2)), ("C4", W.config(3)),
                        ("C5-B64-ctx32768-k32-causal", W.sweep_config(64, 32768, 32, W.MASK_CAUSAL, steps=1))):
            r = measure(c, extra_steps, 3, dev, peaks, flush, clock_sampler=ClockSampler(local), device_weights=True)
            r.pop("flops_per_step", None)
            others[name] = r
        # the rest of a verifier layer around the attention, per layer: Qwen3-8B's dense layer and Qwen3-30B-A3B's
        # routed one, at one sequence's block and at sixteen
        others["layer-qwen3-8b-B1"] = measure_layer("layer-qwen3-8b", dev, peaks, flush, 1, 32, 4096, 4096, 32, 8, 128, 12288, layers=2)
        others["layer-qwen3-30b-a3b-B1"] = measure_layer("layer-qwen3-30b-a3b", dev, peaks, flush, 1, 32, 4096, 2048, 32, 4, 128, 768,
                                                         moe=(128, 8), layers=2)
        others["layer-qwen3-30b-a3b-B16"] = measure_layer("layer-qwen3-30b-a3b", dev, peaks, flush, 16, 32, 4096, 2048, 32, 4, 128, 768,
                                                          moe=(128, 8), layers=1)
    if rank != 0:
        if world > 1:
            import torch.distributed as dist
            dist.destroy_process_group()
        return

    line = {
        "metric": METRIC, "value": head["value"], "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
        "ms_per_step": head["ms_per_step"], "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic", "config": head["config"], "roofline": head["roofline"], "phases": head["phases"],
        "e2e": head.get("e2e", {"value": None, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0,
                                "note": "the host-buffer entry point covers the greedy verify step only"}),
        "gpu_launches": head["gpu_launches"], "clocks": head["clocks"], "kv_status": head["kv_status"],
        "accepted_tokens_last_step": head["accepted_tokens_last_step"], "accepted_equals_planted": head["accepted_equals_planted"],
        "wall_s_timed_loop": head["wall_s_timed_loop"],
        "flops_per_step": head["flops_per_step"],
    }
    if others:
        line["workloads"] = others
    if world == 1 and cfg.mode == "greedy" and not args.no_cpu_baseline:
        st = OracleStep(cfg)
        st.run()                        # warm-up: the first run pages the 1.2 GB of weights in
        sec = st.run()
        line["cpu_baseline"] = {"value": cfg.M / sec, "unit": UNIT, "cores": len(os.sched_getaffinity(0)), "kind": "oracle",
                                "sample": st.sample_text(1)}
    print(json.dumps(line), flush=True)
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


# ---------------------------------------------------------------------------
# the sweep: every point, one table
# ---------------------------------------------------------------------------

def run_sweep(args):
    """All 96 points (batch x context x block size x mask).  A causal point runs ``--steps`` (default here: 64)
    consecutive verify steps on one cache, committing every step; a bidirectional point the drafter's block fill
    that many times (it commits nothing).  Writes the table to --sweep-out and prints one JSON line with its rows."""
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    from paper_2512_15176_b200 import binding as L
    L.lib()
    peaks = load_peaks()
    flush = Flusher(dev)
    rows = []
    for mask, mname in ((W.MASK_CAUSAL, "causal"), (W.MASK_BIDIR, "bidir")):
        for B in (1, 4, 16, 64):
            for ctx in (1024, 4096, 16384, 32768):
                for k in (8, 16, 32):
                    cfg = W.sweep_config(B, ctx, k, mask, steps=args.steps + 8)
                    if mask == W.MASK_BIDIR:
                        cfg = cfg.with_(mode="argmax_logprob")
                    r = measure(cfg, args.steps, 3, dev, peaks, flush, device_weights=True, consecutive=True)
                    rows.append({"B": B, "ctx": ctx, "k": k, "mask": mname, "ms_per_step": r["ms_per_step"],
                                 "tokens_per_s": r["value"], "attn_ms": r["phases"]["attn_ms"],
                                 "attn_frac_of_floor": r["phases"]["attn_frac_of_floor"], "lmhead_ms": r["phases"]["lmhead_ms"],
                                 "lmhead_bound": r["roofline"]["bound"], "lmhead_frac": r["roofline"]["frac"],
                                 "accept_commit_ms": r["phases"]["accept_commit_ms"],
                                 "step_frac_of_floor": r["roofline"]["step_frac_of_roofline_floor"], "kv_status": r["kv_status"]})
    path = os.path.join(ROOT, args.sweep_out)
    with open(path, "w") as f:
        f.write("# Sweep: batch x context x block size x mask (32q/8kv heads, head_dim 128, hidden 4096, vocabulary 151936)\n\n")
        f.write(f"`python bench.py --sweep --steps {args.steps}` on one B200; ragged lengths in [ctx/2, ctx]; causal points: "
                f"{args.steps} consecutive verify steps on one cache (greedy acceptance, geometric planted prefixes drawn anew "
                "every step, every step commits, the contexts grow); bidirectional points: the drafter's block fill (argmax + "
                "max log-probability; commits nothing); one CUDA graph per step, L2 flushed between steps; times are means "
                "over the steps.  Peaks: HBM %.1f GB/s, bf16 %.1f TFLOP/s sustained (%s).  `of floor` = time "
                "the algorithmic bytes / flops take at those peaks over the measured time.\n\n" %
                (peaks["hbm_gbs"], peaks["bf16_tflops_sustained"], peaks["source"]))
        f.write("| mask | B | ctx | k | step us | verified tok/s | attention us | attn of floor | LM head us | LM head of peak | accept+commit us | step of floor |\n")
        f.write("|---|---|---|---|---|---|---|---|---|---|---|---|\n")
        for r in rows:
            f.write("| %s | %d | %d | %d | %.1f | %.0f | %.1f | %.2f | %.1f | %.2f (%s) | %.1f | %.2f |\n" %
                    (r["mask"], r["B"], r["ctx"], r["k"], r["ms_per_step"] * 1e3, r["tokens_per_s"], r["attn_ms"] * 1e3,
                     r["attn_frac_of_floor"], r["lmhead_ms"] * 1e3, r["lmhead_frac"], r["lmhead_bound"],
                     r["accept_commit_ms"] * 1e3, r["step_frac_of_floor"]))
    print(json.dumps({"sweep": rows, "table": args.sweep_out}), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None, help="timed steps (default 200; 64 with --sweep)")
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--config", type=int, default=1, help="workload index 0..3 (1 = Qwen3-8B-shaped verify step)")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-workloads", action="store_true", help="time the headline workload only")
    ap.add_argument("--sweep-point", default=None, metavar="B,CTX,K,MASK",
                    help="time one point of the sweep instead of a fixed workload: batch, context (ragged lengths in "
                         "[CTX/2, CTX]), block size, causal|bidir")
    ap.add_argument("--sweep", action="store_true", help="time every point of the sweep and write the table")
    ap.add_argument("--sweep-out", default="profiles/sweep.md")
    args = ap.parse_args()
    if args.steps is None:
        args.steps = 64 if args.sweep else 200
    if args.sweep:
        run_sweep(args)
        return
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
