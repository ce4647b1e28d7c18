"""The verifier-layer calls (deer_linear, deer_rmsnorm, deer_qk_norm_rope, deer_swiglu)
and their composition with the block attention (runner.VerifierLayer) against the
oracle.  Every stage is compared with the oracle applied to the DEVICE's own input
of that stage (so that a stage's bf16 rounding is not blamed on the next one);
the layer's output is also compared end to end."""
import math

import numpy as np
import pytest
import torch

from oracle import deer_oracle as O
from paper_2512_15176_b200 import workload as W
from tests import harness as Hn

pytestmark = pytest.mark.gpu

BF16_EPS = 2.0 ** -8          # half an ulp of bf16 is 2^-9 relative; one rounding per stored value


def _close(got_bf16, want64, label, extra=0.0, roundings=1.0):
    """|got - want| <= bf16 rounding of want + a little fp32 accumulation noise.  roundings: how many bf16 roundings
    lie between the stage's input and its output (a stage that rounds its operands before combining them has more
    than the one of its store)."""
    got = Hn.f64(got_bf16.cpu())
    err = np.abs(got - want64)
    tol = roundings * BF16_EPS * np.abs(want64) + 2e-3 * np.abs(want64).max() * (1.0 + extra) / 4
    assert np.isfinite(got).all(), label
    assert (err <= tol).all(), f"{label}: max err {err.max():.3e} at tolerance {tol.flat[err.argmax()]:.3e}"


@pytest.mark.parametrize("M,K,N,res,ws", [(8, 512, 1536, False, True), (32, 4096, 1024, True, True), (32, 4096, 1024, True, False),
                                          (33, 128, 1000, True, True), (32, 12288, 4096, True, True), (100, 1024, 24576, False, True),
                                          (200, 256, 520, False, True), (300, 192, 4096, True, False)])
def test_linear(M, K, N, res, ws):
    """ws: with the workspace that lets the call cut the contraction into ranges (few output columns, M <= 128)."""
    from paper_2512_15176_b200 import binding as L
    x = W.normal(11, "x", (M, K), 1.0)
    w = W.normal(11, "w", (N, K), 1.0 / math.sqrt(K))
    r = W.normal(11, "r", (M, N), 1.0) if res else None
    y = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device="cuda")
    work = torch.empty(max(L.deer_linear_workspace_bytes(M, K, N), 16), dtype=torch.uint8, device="cuda") if ws else None
    L.deer_linear(x.cuda(), w.cuda(), y, residual=r.cuda() if res else None, workspace=work)
    torch.cuda.synchronize()
    want = O.linear(Hn.f64(x), Hn.f64(w)) + (Hn.f64(r) if res else 0.0)
    _close(y, want, f"linear {M}x{K}x{N}")


def test_rmsnorm_and_swiglu():
    from paper_2512_15176_b200 import binding as L
    x = W.normal(12, "x", (37, 4096), 1.7)
    g = W.normal(12, "g", (4096,), 1.0)
    y = torch.empty_like(x, device="cuda")
    L.deer_rmsnorm(x.cuda(), g.cuda(), y, 1e-6)
    _close(y, O.rmsnorm(Hn.f64(x), Hn.f64(g), 1e-6), "rmsnorm")
    gu = W.normal(12, "gu", (37, 2 * 1536), 2.0)
    act = torch.empty(37, 1536, dtype=torch.bfloat16, device="cuda")
    L.deer_swiglu(gu.cuda(), act)
    g64 = Hn.f64(gu)
    _close(act, O.swiglu(g64[:, :1536], g64[:, 1536:]), "swiglu")


@pytest.mark.parametrize("qk_norm", [False, True])
def test_qk_norm_rope(qk_norm):
    """Positions are the sequences' committed lengths (ragged, up to ~30 000) plus the block row."""
    from paper_2512_15176_b200 import binding as L
    cfg = W.StepConfig("rope", 3, 8, 2, 128, 8, 256, 512, (0, 0), seed=77)
    lengths = np.array([0, 4097, 29990], dtype=np.int32)
    st = Hn.draw_state(cfg.with_(ctx=(0, 0)), np.zeros(3, dtype=np.int32), True)
    kv = Hn.gpu_kv(st)
    kv.seq_len.copy_(torch.from_numpy(lengths))
    q, kb, _ = Hn.draw_block(cfg, 0, True)
    qg = W.normal(77, "qg", (cfg.D,), 1.0) if qk_norm else None
    kg = W.normal(77, "kg", (cfg.D,), 1.0) if qk_norm else None
    qd, kd = q.cuda(), kb.cuda()
    ids = torch.arange(3, dtype=torch.int32, device="cuda")
    L.deer_qk_norm_rope(kv, ids, qd, kd, qg.cuda() if qk_norm else None, kg.cuda() if qk_norm else None, 1e-6, 1.0e6)
    pos = lengths[:, None] + np.arange(cfg.k)[None, :]
    for got, src, gam in ((qd, q, qg), (kd, kb, kg)):
        v = Hn.f64(src)
        if qk_norm:
            v = Hn.f64(torch.from_numpy(O.rmsnorm(v, Hn.f64(gam), 1e-6)).to(torch.bfloat16))     # the device rounds here too
        _close(got, O.rope(v, pos, 1.0e6), "rope", extra=1.0)


def test_verifier_layer_matches_oracle():
    """A small Qwen3-shaped layer (hidden 512, 8 query / 2 KV heads of 128, intermediate 1536) over a ragged paged
    cache: every stage against the oracle on the device's own stage input, the cache state after the append, and
    the layer output end to end."""
    from paper_2512_15176_b200 import binding as L
    from paper_2512_15176_b200.runner import VerifierLayer
    cfg = W.StepConfig("layer", 4, 8, 2, 128, 8, 512, 512, (40, 700), seed=78, growth=8)
    inter, eps, theta = 1536, 1e-6, 1.0e6
    st = Hn.draw_state(cfg, None, True)
    okv, kv = Hn.oracle_kv(st), Hn.gpu_kv(st)
    hid, Hq, Hkv, D, M = cfg.hid, cfg.Hq, cfg.Hkv, cfg.D, cfg.M
    mk = lambda name, shape, sig: W.normal(78, name, shape, sig)
    w = {"ln1": mk("ln1", (hid,), 1.0), "ln2": mk("ln2", (hid,), 1.0), "q_norm": mk("qn", (D,), 1.0), "k_norm": mk("kn", (D,), 1.0),
         "wq": mk("wq", (Hq * D, hid), hid ** -0.5), "wk": mk("wk", (Hkv * D, hid), hid ** -0.5),
         "wv": mk("wv", (Hkv * D, hid), hid ** -0.5), "wo": mk("wo", (hid, Hq * D), (Hq * D) ** -0.5),
         "wgu": mk("wgu", (2 * inter, hid), hid ** -0.5), "wd": mk("wd", (hid, inter), inter ** -0.5)}
    wd = {n: t.cuda() for n, t in w.items()}
    wd["wqkv"] = torch.cat([w["wq"], w["wk"], w["wv"]], dim=0).contiguous().cuda()
    w64 = {n: Hn.f64(t) for n, t in w.items()}
    x = mk("x", (M, hid), 1.0)
    layer = VerifierLayer(cfg, kv, wd, int(st.lengths.max()) + cfg.k, inter, eps, theta)
    out = layer.forward(x.cuda())
    torch.cuda.synchronize()
    assert L.deer_kv_status(kv) == 0
    dev = lambda t: Hn.f64(t.cpu())
    rb = lambda a: Hn.f64(torch.from_numpy(np.asarray(a)).to(torch.bfloat16))            # what a bf16 store keeps
    x64 = Hn.f64(x)
    _close(layer.xn, O.rmsnorm(x64, w64["ln1"], eps), "ln1")
    xn = dev(layer.xn)
    pos = st.lengths[:, None] + np.arange(cfg.k)[None, :]
    for name, got, wt, gam, H in (("q", layer.q, "wq", "q_norm", Hq), ("k", layer.k_blk, "wk", "k_norm", Hkv)):
        proj = rb(O.linear(xn, w64[wt])).reshape(cfg.B, cfg.k, H, D)
        normed = rb(O.rmsnorm(proj, w64[gam], eps))
        _close(got, O.rope(normed, pos, theta), name + " after norm and rope", extra=2.0)
    _close(layer.v_blk, O.linear(xn, w64["wv"]).reshape(cfg.B, cfg.k, Hkv, D), "v")
    # attention on the device's own q / k / v
    ids = np.arange(cfg.B)
    assert okv.reserve(ids, cfg.k)
    want_attn = O.block_attention(dev(layer.q), dev(layer.k_blk), dev(layer.v_blk), okv.k_pool, okv.v_pool, okv.page_table,
                                  okv.seq_len, ids, O.MASK_CAUSAL, 1.0 / math.sqrt(D))
    Hn.check_attention(layer.attn_out.cpu(), want_attn, "layer attention")
    okv.append(ids, dev(layer.k_blk).astype(np.float32), dev(layer.v_blk).astype(np.float32))
    Hn.kv_state_equal(kv, okv, "layer")
    _close(layer.x1, O.linear(dev(layer.attn_out).reshape(M, -1), w64["wo"]) + x64, "o_proj + residual")
    x1 = dev(layer.x1)
    _close(layer.xn2, O.rmsnorm(x1, w64["ln2"], eps), "ln2")
    _close(layer.gu, O.linear(dev(layer.xn2), w64["wgu"]), "gate/up")
    gu = dev(layer.gu)
    _close(layer.act, O.swiglu(gu[:, :inter], gu[:, inter:]), "swiglu")
    _close(out, O.linear(dev(layer.act), w64["wd"]) + x1, "down + residual")
    # end to end in float64 with a bf16 rounding wherever the device stores one
    e_xn = rb(O.rmsnorm(x64, w64["ln1"], eps))
    e_q = rb(O.rope(rb(O.rmsnorm(rb(O.linear(e_xn, w64["wq"])).reshape(cfg.B, cfg.k, Hq, D), w64["q_norm"], eps)), pos, theta))
    e_k = rb(O.rope(rb(O.rmsnorm(rb(O.linear(e_xn, w64["wk"])).reshape(cfg.B, cfg.k, Hkv, D), w64["k_norm"], eps)), pos, theta))
    e_v = rb(O.linear(e_xn, w64["wv"])).reshape(cfg.B, cfg.k, Hkv, D)
    okv2 = Hn.oracle_kv(st)
    assert okv2.reserve(ids, cfg.k)
    e_at = rb(O.block_attention(e_q, e_k, e_v, okv2.k_pool, okv2.v_pool, okv2.page_table, okv2.seq_len, ids, O.MASK_CAUSAL,
                                1.0 / math.sqrt(D)))
    e_x1 = rb(O.linear(e_at.reshape(M, -1), w64["wo"]) + x64)
    e_gu = rb(O.linear(rb(O.rmsnorm(e_x1, w64["ln2"], eps)), w64["wgu"]))
    e_out = O.linear(rb(O.swiglu(e_gu[:, :inter], e_gu[:, inter:])), w64["wd"]) + e_x1
    err = np.abs(dev(out) - e_out)
    assert err.max() <= 5e-2 * np.abs(e_out).max() and err.mean() <= 5e-3 * np.abs(e_out).mean() + 1e-3, (err.max(), err.mean())


def _layer_weights(seed, hid, Hq, Hkv, D, inter):
    mk = lambda name, shape, sig: W.normal(seed, name, shape, sig)
    w = {"ln1": mk("ln1", (hid,), 1.0), "ln2": mk("ln2", (hid,), 1.0), "q_norm": mk("qn", (D,), 1.0), "k_norm": mk("kn", (D,), 1.0),
         "wq": mk("wq", (Hq * D, hid), hid ** -0.5), "wk": mk("wk", (Hkv * D, hid), hid ** -0.5),
         "wv": mk("wv", (Hkv * D, hid), hid ** -0.5), "wo": mk("wo", (hid, Hq * D), (Hq * D) ** -0.5),
         "wgu": mk("wgu", (2 * inter, hid), hid ** -0.5), "wd": mk("wd", (hid, inter), inter ** -0.5)}
    dev = {n: t.cuda() for n, t in w.items()}
    dev["wqkv"] = torch.cat([w["wq"], w["wk"], w["wv"]], dim=0).contiguous().cuda()
    return w, dev


def _check_layer_stages(layer, st, okv, w64, x, cfg, inter, eps, theta, out, label):
    """Every stage the layer object exposes, against the oracle on the device's own input of that stage."""
    hid, Hq, Hkv, D, M = cfg.hid, cfg.Hq, cfg.Hkv, cfg.D, cfg.M
    dev = lambda t: Hn.f64(t.cpu())
    rb = lambda a: Hn.f64(torch.from_numpy(np.asarray(a)).to(torch.bfloat16))
    x64 = Hn.f64(x)
    xn = dev(layer.xn)
    _close(layer.xn, O.rmsnorm(x64, w64["ln1"], eps), label + " ln1")
    pos = st.lengths[:, None] + np.arange(cfg.k)[None, :]
    for name, got, wt, gam, H in (("q", layer.q, "wq", "q_norm", Hq), ("k", layer.k_blk, "wk", "k_norm", Hkv)):
        proj = rb(O.linear(xn, w64[wt])).reshape(cfg.B, cfg.k, H, D)
        normed = rb(O.rmsnorm(proj, w64[gam], eps))
        _close(got, O.rope(normed, pos, theta), f"{label} {name} after norm and rope", extra=2.0)
    _close(layer.v_blk, O.linear(xn, w64["wv"]).reshape(cfg.B, cfg.k, Hkv, D), label + " v")
    ids = np.arange(cfg.B)
    assert okv.reserve(ids, cfg.k)
    want_attn = O.block_attention(dev(layer.q), dev(layer.k_blk), dev(layer.v_blk), okv.k_pool, okv.v_pool, okv.page_table,
                                  okv.seq_len, ids, O.MASK_CAUSAL, 1.0 / math.sqrt(D))
    Hn.check_attention(layer.attn_out.cpu(), want_attn, label + " attention")
    _close(layer.x1, O.linear(dev(layer.attn_out).reshape(M, -1), w64["wo"]) + x64, label + " o_proj + residual")
    x1 = dev(layer.x1)
    _close(layer.xn2, O.rmsnorm(x1, w64["ln2"], eps), label + " ln2")
    # gate and up are rounded to bf16 before the gate; where the device's fp32 sum and the oracle's fp64 one fall on
    # different sides of a rounding boundary the operands differ by an ulp each, on top of the output's own rounding
    gu = rb(O.linear(dev(layer.xn2), w64["wgu"]))
    _close(layer.act, O.swiglu(gu[:, :inter], gu[:, inter:]), label + " gated activation", roundings=4.0)
    _close(out, O.linear(dev(layer.act), w64["wd"]) + x1, label + " down + residual")


def test_fused_layer_at_the_qwen3_8b_shape():
    """Hidden 4096, 32 query / 8 KV heads of 128, intermediate 12288, one sequence's block of 32: the layer on the
    fused calls (projection + rotary tail, projection + residual + RMSNorm tail, gate/up with the SiLU gate in the
    epilogue), every stage against the oracle, and against the same layer on the separate calls."""
    from paper_2512_15176_b200 import binding as L
    from paper_2512_15176_b200.runner import VerifierLayer
    cfg = W.StepConfig("layer8b", 1, 32, 8, 128, 32, 4096, 512, (700, 700), seed=79, growth=32)
    inter, eps, theta = 12288, 1e-6, 1.0e6
    w, wdev = _layer_weights(79, cfg.hid, cfg.Hq, cfg.Hkv, cfg.D, inter)
    w64 = {n: Hn.f64(t) for n, t in w.items()}
    x = W.normal(79, "x", (cfg.M, cfg.hid), 1.0)
    nxt = W.normal(79, "ln_next", (cfg.hid,), 1.0)
    outs = {}
    for fused in (True, False):
        st = Hn.draw_state(cfg, None, True)
        okv, kv = Hn.oracle_kv(st), Hn.gpu_kv(st)
        layer = VerifierLayer(cfg, kv, wdev, int(st.lengths.max()) + cfg.k, inter, eps, theta, fused=fused)
        out = layer.forward(x.cuda(), next_ln=nxt.cuda())
        torch.cuda.synchronize()
        assert L.deer_kv_status(kv) == 0
        _check_layer_stages(layer, st, okv, w64, x, cfg, inter, eps, theta, out, "fused" if fused else "separate")
        _close(layer.xn_next, O.rmsnorm(Hn.f64(out.cpu()), Hn.f64(nxt), eps), "next layer's ln1")
        outs[fused] = (out.cpu().clone(), layer.xn_next.cpu().clone(), layer.act.cpu().clone())
    # same arithmetic, same roundings; only the order in which a row's squares are summed differs between the fused
    # tail and the separate normalisation, so a value may land on the other side of a bf16 rounding here and there
    for a, b, name in zip(outs[True], outs[False], ("output", "normalised output", "activations")):
        fa, fb = Hn.f64(a), Hn.f64(b)
        d = np.abs(fa - fb)
        assert (d <= 2.0 ** -6 * np.abs(fb) + 1e-3 * np.abs(fb).max()).all() and (d > 0).mean() < 0.05, \
            f"fused and separate calls differ in the {name}: max {d.max():.3e}, {100 * (d > 0).mean():.2f} % of the values"


def test_layer_stack_and_moe_layer():
    """Three layers over one shared page table (each with pools of its own): the stack on the fused calls equals the
    layers run one by one on the separate calls, bit for bit, and all layers' caches hold the appended rows.  Then
    one layer with a routed MLP against the oracle."""
    from paper_2512_15176_b200 import binding as L
    from paper_2512_15176_b200.runner import VerifierLayer, VerifierStack
    cfg = W.StepConfig("stack", 3, 8, 2, 128, 8, 512, 512, (40, 500), seed=80, growth=8)
    inter, eps, theta, n_layers = 1024, 1e-6, 1.0e6, 3
    st = Hn.draw_state(cfg, None, True)
    lay = st.layout
    i32 = lambda a: torch.from_numpy(a.copy()).to(device="cuda", dtype=torch.int32).contiguous()
    x = W.normal(80, "x", (cfg.M, cfg.hid), 1.0)
    msl = int(st.lengths.max()) + cfg.k
    results = []
    for fused in (True, False):
        shared = [i32(a) for a in (lay.page_table, lay.seq_len, lay.n_pages, lay.free_stack, lay.free_top)]
        kvs, weights = [], []
        for l in range(n_layers):
            kp, vp = W.kv_pools(cfg.with_(seed=80 + 10 * l), lay.num_pages, sigma=1.0)
            kvs.append(L.KVCache(kp.cuda(), vp.cuda(), *shared))
            weights.append(_layer_weights(80 + l, cfg.hid, cfg.Hq, cfg.Hkv, cfg.D, inter)[1])
        if fused:
            out = VerifierStack(cfg, kvs, weights, msl, inter, eps, theta, fused=True).forward(x.cuda())
        else:
            L.deer_kv_reserve(kvs[0], torch.arange(cfg.B, dtype=torch.int32, device="cuda"), cfg.k)
            cur = x.cuda()
            for l in range(n_layers):
                cur = VerifierLayer(cfg, kvs[l], weights[l], msl, inter, eps, theta, fused=False, reserve=False).forward(cur).clone()
            out = cur
        keep = torch.full((cfg.B,), cfg.k, dtype=torch.int32, device="cuda")
        L.deer_kv_commit(kvs[0], torch.arange(cfg.B, dtype=torch.int32, device="cuda"), keep, cfg.k)
        torch.cuda.synchronize()
        assert all(L.deer_kv_status(kv) == 0 for kv in kvs)
        assert np.isfinite(Hn.f64(out.cpu())).all()
        results.append((out.cpu().clone(), [kv.k_pool.cpu().clone() for kv in kvs], shared[1].cpu().clone()))
    # The two paths cut the gate/up contraction differently at this width (the separate call splits it into ranges,
    # the gated epilogue does not), so their sums differ in the last fp32 bits and a bf16 rounding flips here and
    # there: equal up to a few bf16 ulps after three layers, not bit for bit (at widths where neither splits they
    # are: see the test above).
    fa, fb = Hn.f64(results[0][0]), Hn.f64(results[1][0])
    d = np.abs(fa - fb)
    assert d.max() <= 3e-2 * np.abs(fb).max() and d.mean() <= 2e-3 * np.abs(fb).mean(), (d.max(), d.mean())
    for l, (a, b) in enumerate(zip(results[0][1], results[1][1])):
        da = np.abs(Hn.f64(a) - Hn.f64(b))                           # every layer appended (nearly) the same rows
        assert da.max() <= 3e-2 * np.abs(Hn.f64(b)).max() and (l > 0 or da.max() == 0.0), (l, da.max())
    assert (results[0][2].numpy() == st.lengths + cfg.k).all()

    # one layer with a routed MLP (8 experts, 2 per row)
    E, top_k, mi = 8, 2, 256
    st = Hn.draw_state(cfg, None, True)
    okv, kv = Hn.oracle_kv(st), Hn.gpu_kv(st)
    w, wdev = _layer_weights(81, cfg.hid, cfg.Hq, cfg.Hkv, cfg.D, mi)
    moe_w = {"w_router": W.normal(81, "wr", (E, cfg.hid), cfg.hid ** -0.5 * 3.0), "w_gate_up": W.normal(81, "wgu_e", (E, 2 * mi, cfg.hid), cfg.hid ** -0.5),
             "w_down": W.normal(81, "wd_e", (E, cfg.hid, mi), mi ** -0.5)}
    wdev.update({n: t.cuda() for n, t in moe_w.items()})
    layer = VerifierLayer(cfg, kv, wdev, msl, mi, eps, theta, fused=True, moe=(E, top_k))
    out = layer.forward(x.cuda())
    torch.cuda.synchronize()
    assert L.deer_kv_status(kv) == 0
    xn2, x1 = Hn.f64(layer.xn2.cpu()), Hn.f64(layer.x1.cpu())
    logits = np.sort(xn2 @ Hn.f64(moe_w["w_router"]).T, axis=1)[:, ::-1]
    clear = (logits[:, top_k - 1] - logits[:, top_k]) > 2e-3          # rows whose routing is clear of rounding
    assert clear.mean() > 0.8
    want = O.moe_mlp(xn2, Hn.f64(moe_w["w_router"]), Hn.f64(moe_w["w_gate_up"]), Hn.f64(moe_w["w_down"]), top_k) + x1
    err = np.abs(Hn.f64(out.cpu()) - want)[clear]
    assert err.max() <= 2.5e-2 * np.abs(want).max() and err.mean() <= 4e-3 * np.abs(want).mean(), (err.max(), err.mean())
