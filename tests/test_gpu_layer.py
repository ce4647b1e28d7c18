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


def _close(got_bf16, want64, label, extra=0.0):
    """|got - want| <= bf16 rounding of want + a little fp32 accumulation noise."""
    got = Hn.f64(got_bf16.cpu())
    err = np.abs(got - want64)
    tol = BF16_EPS * np.abs(want64) + 2e-3 * np.abs(want64).max() * (1.0 + extra) / 4
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
