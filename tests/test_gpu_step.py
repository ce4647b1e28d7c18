"""Whole-step parity at the full sizes of the fixed workloads, in the launch
configuration the benchmark times: reserve -> block_attn -> lmhead_select ->
accept -> commit through the C-ABI, against the oracle on the same inputs."""
import math

import numpy as np
import pytest
import torch

from oracle import deer_oracle as O
from paper_2512_15176_b200 import workload as W
from tests import harness as Hn

pytestmark = pytest.mark.gpu


def _greedy_step(cfg, stress=False, steps=1, lengths=None):
    from paper_2512_15176_b200 import binding as L
    from paper_2512_15176_b200.runner import VerifyStep
    cfg = cfg.with_(growth=max(cfg.growth, steps * cfg.k))
    st = Hn.draw_state(cfg, lengths, stress)
    okv = Hn.oracle_kv(st)
    kv = Hn.gpu_kv(st)
    w = W.lm_head(cfg)
    w64 = Hn.f64(w)
    vs = VerifyStep(cfg, kv, w.cuda(), int(st.lengths.max()) + steps * cfg.k, store_logits=False)
    ids = np.arange(cfg.B)
    for step in range(steps):
        q, kb, vb = Hn.draw_block(cfg, step, stress)
        h, z, _ = Hn.draw_hidden_with_margin(cfg, w64, step)
        target = O.select_argmax(z).reshape(cfg.B, cfg.k)
        Lp = W.planted_prefix_lengths(cfg, step)
        drafts = W.plant_drafts(cfg, target, Lp, step)
        # oracle
        assert okv.reserve(ids, cfg.k)
        want_attn = Hn.oracle_attention(cfg, okv, q, kb, vb)
        okv.append(ids, Hn.f64(kb).astype(np.float32), Hn.f64(vb).astype(np.float32))
        a, out, n = O.accept_greedy(drafts, target)
        np.testing.assert_array_equal(a, Lp)
        okv.commit(ids, a)
        # GPU
        vs.load(q, kb, vb, h, drafts)
        vs.run()
        torch.cuda.synchronize()
        assert L.deer_kv_status(kv) == 0
        Hn.check_attention(vs.attn_out.cpu(), want_attn, f"{cfg.name} step {step}")
        Hn.check_ids(vs.target_ids.cpu().numpy(), target, z, f"{cfg.name} step {step}")
        np.testing.assert_array_equal(vs.accept_len.cpu().numpy(), a)
        np.testing.assert_array_equal(vs.out_ids.cpu().numpy(), out)
        np.testing.assert_array_equal(vs.n_out.cpu().numpy(), n)
        Hn.kv_state_equal(kv, okv, f"{cfg.name} step {step}")
    Hn.kv_contents_equal(kv, okv, label=cfg.name)


@pytest.mark.parametrize("stress", [False, True])
def test_c1_tiny_verify_step(stress):
    _greedy_step(W.config(0), stress, steps=4)


@pytest.mark.parametrize("stress", [False, True])
def test_c2_qwen3_8b_verify_step(stress):
    _greedy_step(W.config(1), stress, steps=1)


def test_c3_dllm_block_fill():
    """Bidirectional block fill: ids and fp32 max-logprob for all 32 positions of
    8 sequences in one pass; nothing is appended or committed."""
    from paper_2512_15176_b200 import binding as L
    from paper_2512_15176_b200.runner import VerifyStep
    cfg = W.config(2)
    for stress in (False, True):
        st = Hn.draw_state(cfg, None, stress)
        okv = Hn.oracle_kv(st)
        kv = Hn.gpu_kv(st)
        w = W.lm_head(cfg)
        w64 = Hn.f64(w)
        q, kb, vb = Hn.draw_block(cfg, 0, stress)
        h, z, _ = Hn.draw_hidden_with_margin(cfg, w64)
        vs = VerifyStep(cfg, kv, w.cuda(), int(st.lengths.max()))
        vs.load(q, kb, vb, h)
        vs.run()
        torch.cuda.synchronize()
        assert L.deer_kv_status(kv) == 0
        Hn.check_attention(vs.attn_out.cpu(), Hn.oracle_attention(cfg, okv, q, kb, vb), cfg.name)
        Hn.check_ids(vs.target_ids.cpu().numpy(), O.select_argmax(z), z, cfg.name)
        np.testing.assert_allclose(vs.max_logprob.cpu().numpy(), O.max_logprob(z), atol=2e-4, rtol=0)
        Hn.kv_state_equal(kv, okv, cfg.name)       # untouched
        del vs, kv
        torch.cuda.empty_cache()


def test_c4_qwen3_30b_a3b_sampling_step():
    """Temperature-1 verify step with ragged contexts.  Accept lengths must match
    the oracle exactly (margins cleared on u); the residual draw is checked for
    validity against the oracle's CDF because the GPU's own fp32 logits differ
    from the oracle's by rounding."""
    from paper_2512_15176_b200 import binding as L
    from paper_2512_15176_b200.runner import VerifyStep
    cfg = W.config(3)
    st = Hn.draw_state(cfg)
    okv = Hn.oracle_kv(st)
    kv = Hn.gpu_kv(st)
    w = W.lm_head(cfg)
    w64 = Hn.f64(w)
    q, kb, vb = Hn.draw_block(cfg)
    h, z, _ = Hn.draw_hidden_with_margin(cfg, w64)
    zt = z.reshape(cfg.B, cfg.k, cfg.V)
    T = float(np.float32(cfg.temperature))
    ql, drafts, u, r, _ = Hn.sampling_inputs(cfg, zt.astype(np.float32), r_margin=1e-12)
    ids = np.arange(cfg.B)
    assert okv.reserve(ids, cfg.k)
    want_attn = Hn.oracle_attention(cfg, okv, q, kb, vb)
    okv.append(ids, Hn.f64(kb).astype(np.float32), Hn.f64(vb).astype(np.float32))
    a, out, n = O.accept_sample(drafts, zt, T, ql.numpy(), u.numpy(), r.numpy())
    okv.commit(ids, a)

    vs = VerifyStep(cfg, kv, w.cuda(), int(st.lengths.max()) + cfg.k)
    vs.load(q, kb, vb, h, drafts, ql, u, r)
    vs.run()
    torch.cuda.synchronize()
    assert L.deer_kv_status(kv) == 0
    Hn.check_attention(vs.attn_out.cpu(), want_attn, cfg.name)
    Hn.check_ids(vs.target_ids.cpu().numpy(), O.select_argmax(z), z, cfg.name)
    np.testing.assert_allclose(vs.lse.cpu().numpy(), O.logsumexp(z, T), atol=3e-4, rtol=0)
    Hn.check_logits(vs.logits.cpu(), z, cfg.name)
    np.testing.assert_array_equal(vs.accept_len.cpu().numpy(), a)
    np.testing.assert_array_equal(vs.n_out.cpu().numpy(), n)
    got = vs.out_ids.cpu().numpy()
    for b in range(cfg.B):
        i = int(a[b])
        np.testing.assert_array_equal(got[b, :i], out[b, :i])
        assert (got[b, n[b]:] == -1).all()
        if i < cfg.k and got[b, i] != out[b, i]:
            # valid if r*S lies within the token's CDF cell widened by the rounding of fp32 logits
            p = O.softmax_f64(zt[b, i], T)
            qd = O.softmax_f64(ql[b, i].numpy(), 1.0)
            res, S = O.residual_distribution(p, qd)
            cdf = np.cumsum(res)
            v = int(got[b, i])
            t = float(r[b]) * S
            assert res[v] > 0 and (cdf[v - 1] if v else 0.0) - 1e-5 * S <= t <= cdf[v] + 1e-5 * S, f"seq {b}: invalid residual draw {v}"
    Hn.kv_state_equal(kv, okv, cfg.name)
    Hn.kv_contents_equal(kv, okv, seqs=[0, 7, 15], label=cfg.name)


@pytest.mark.parametrize("B,ctx,k,mask", [
    (4, 1024, 8, W.MASK_CAUSAL),
    (16, 4096, 16, W.MASK_CAUSAL),
    (4, 16384, 32, W.MASK_BIDIR),
    (64, 1024, 32, W.MASK_CAUSAL),
])
def test_c5_sweep_points(B, ctx, k, mask):
    """Sweep points with ragged lengths; the vocabulary is cut to 8192 rows here
    so that the oracle's logits stay cheap (the full head is covered by the C2-C4
    tests); attention, acceptance and the KV cycle run at the point's real shape."""
    cfg = W.sweep_config(B, ctx, k, mask, steps=3).with_(V=8192)
    if mask == W.MASK_BIDIR:
        from paper_2512_15176_b200 import binding as L
        from paper_2512_15176_b200.runner import VerifyStep
        cfg = cfg.with_(mode="argmax_logprob")
        st = Hn.draw_state(cfg, None, True)
        okv, kv = Hn.oracle_kv(st), Hn.gpu_kv(st)
        w = W.lm_head(cfg)
        q, kb, vb = Hn.draw_block(cfg, 0, True)
        h, z, _ = Hn.draw_hidden_with_margin(cfg, Hn.f64(w))
        vs = VerifyStep(cfg, kv, w.cuda(), int(st.lengths.max()))
        vs.load(q, kb, vb, h)
        vs.run()
        torch.cuda.synchronize()
        assert L.deer_kv_status(kv) == 0
        Hn.check_attention(vs.attn_out.cpu(), Hn.oracle_attention(cfg, okv, q, kb, vb), cfg.name)
        Hn.check_ids(vs.target_ids.cpu().numpy(), O.select_argmax(z), z, cfg.name)
    else:
        _greedy_step(cfg, stress=True, steps=3)


@pytest.mark.parametrize("own_stream,adjacent", [(False, False), (True, False), (True, True), (False, True)])
def test_host_buffer_step_matches_oracle(own_stream, adjacent):
    """deer_verify_step_host, four consecutive steps from pinned host buffers that are refilled in place: on the legacy
    default stream every call enqueues its copies and kernels one by one; on a stream of its own the first call
    captures them into a graph and the later ones replay it.  With `adjacent`, q / k_blk / v_blk and the three results
    are slices of one buffer on each side (the call then moves each group with one copy).  Results and cache state
    against the oracle."""
    from paper_2512_15176_b200 import binding as L
    from paper_2512_15176_b200.runner import VerifyStep
    steps = 4
    cfg = W.config(0).with_(growth=steps * W.config(0).k)
    st = Hn.draw_state(cfg, None, True)
    okv, kv = Hn.oracle_kv(st), Hn.gpu_kv(st)
    w = W.lm_head(cfg)
    w64 = Hn.f64(w)
    w_dev = w.cuda()
    vs = VerifyStep(cfg, kv, w_dev, int(st.lengths.max()) + steps * cfg.k, store_logits=False)
    ids = np.arange(cfg.B)
    pin = lambda t: t.contiguous().pin_memory()
    q0, kb0, vb0 = Hn.draw_block(cfg, 0, True)
    hh = pin(torch.empty(cfg.M, cfg.hid, dtype=torch.bfloat16))
    hd = pin(torch.empty(cfg.B, cfg.k, dtype=torch.int32))
    if adjacent:
        nq, nk = q0.numel(), kb0.numel()
        hin = torch.empty(nq + 2 * nk, dtype=torch.bfloat16).pin_memory()
        hq, hkb, hvb = hin[:nq].view_as(q0), hin[nq:nq + nk].view_as(kb0), hin[nq + nk:].view_as(vb0)
        hout = torch.full((2 * cfg.B + cfg.M,), -7, dtype=torch.int32).pin_memory()
        ha, ho, hn = hout[:cfg.B], hout[cfg.B:cfg.B + cfg.M].view(cfg.B, cfg.k), hout[cfg.B + cfg.M:]
        din = torch.empty(nq + 2 * nk, dtype=torch.bfloat16, device="cuda")
        dout = torch.empty(2 * cfg.B + cfg.M, dtype=torch.int32, device="cuda")
        dq, dk, dv = din, din[nq:], din[nq + nk:]
        da, do, dn = dout, dout[cfg.B:], dout[cfg.B + cfg.M:]
    else:
        hq, hkb, hvb = pin(q0), pin(kb0), pin(vb0)
        ha = torch.empty(cfg.B, dtype=torch.int32).pin_memory()
        ho = torch.empty(cfg.B, cfg.k, dtype=torch.int32).pin_memory()
        hn = torch.empty(cfg.B, dtype=torch.int32).pin_memory()
        dq, dk, dv, da, do, dn = vs.q, vs.k_blk, vs.v_blk, vs.accept_len, vs.out_ids, vs.n_out
    sd = L.deer_step_dev(dq.data_ptr(), dk.data_ptr(), dv.data_ptr(), vs.attn_out.data_ptr(), vs.h.data_ptr(),
                         vs.seq_ids.data_ptr(), vs.draft_ids.data_ptr(), vs.target_ids.data_ptr(), da.data_ptr(),
                         do.data_ptr(), dn.data_ptr(), vs.attn_ws.data_ptr(), vs.attn_ws.numel(),
                         vs.lm_ws.data_ptr(), vs.lm_ws.numel())
    stream = torch.cuda.Stream() if own_stream else None
    torch.cuda.synchronize()
    for step in range(steps):
        q, kb, vb = Hn.draw_block(cfg, step, True)
        h, z, _ = Hn.draw_hidden_with_margin(cfg, w64, step)
        target = O.select_argmax(z).reshape(cfg.B, cfg.k)
        drafts = W.plant_drafts(cfg, target, W.planted_prefix_lengths(cfg, step), step)
        for dst, src in ((hq, q), (hkb, kb), (hvb, vb), (hh, h), (hd, torch.from_numpy(drafts))):
            dst.copy_(src.reshape(dst.shape))
        assert okv.reserve(ids, cfg.k)
        okv.append(ids, Hn.f64(kb).astype(np.float32), Hn.f64(vb).astype(np.float32))
        a, out, n = O.accept_greedy(drafts, target)
        okv.commit(ids, a)
        L.deer_verify_step_host(kv, sd, w_dev, hq, hkb, hvb, hh, hd, cfg.B, cfg.k, cfg.Hq, cfg.hid, cfg.V, vs.scale,
                                int(st.lengths.max()) + steps * cfg.k, ha, ho, hn, stream=stream)
        np.testing.assert_array_equal(ha.numpy(), a)
        np.testing.assert_array_equal(ho.numpy(), out)
        np.testing.assert_array_equal(hn.numpy(), n)
        assert L.deer_kv_status(kv) == 0
        Hn.kv_state_equal(kv, okv, f"host step {step}")
    Hn.kv_contents_equal(kv, okv, label="host steps")


def test_host_buffer_step_notices_a_swapped_device_buffer():
    """The recorded graph holds every device pointer by value, so a call that differs from the recorded one in a
    single staging buffer (here the hidden states, then the result arrays) must not replay the old graph: the step
    has to read the new hidden states and write the new result arrays."""
    from paper_2512_15176_b200 import binding as L
    from paper_2512_15176_b200.runner import VerifyStep
    cfg = W.config(0).with_(growth=64)
    st = Hn.draw_state(cfg, None, True)
    kv = Hn.gpu_kv(st)
    saved = [t.clone() for t in (kv.page_table, kv.seq_len, kv.n_pages, kv.free_stack, kv.free_top)]
    w = W.lm_head(cfg)
    w64 = Hn.f64(w)
    w_dev = w.cuda()
    msl = int(st.lengths.max()) + 64
    vs = VerifyStep(cfg, kv, w_dev, msl, store_logits=False)
    pin = lambda t: t.contiguous().pin_memory()
    q, kb, vb = Hn.draw_block(cfg, 0, True)
    hq, hkb, hvb = pin(q), pin(kb), pin(vb)
    h0, z0, _ = Hn.draw_hidden_with_margin(cfg, w64, 0)
    h1, z1, _ = Hn.draw_hidden_with_margin(cfg, w64, 1)
    t0, t1 = (O.select_argmax(z).reshape(cfg.B, cfg.k) for z in (z0, z1))
    assert (t0 != t1).any()
    drafts = t0.copy()                       # every row of h0 is accepted in full; against h1 almost nothing is
    hh, hd = pin(h0), pin(torch.from_numpy(drafts))
    ha = torch.empty(cfg.B, dtype=torch.int32).pin_memory()
    ho = torch.empty(cfg.B, cfg.k, dtype=torch.int32).pin_memory()
    hn = torch.empty(cfg.B, dtype=torch.int32).pin_memory()
    stream = torch.cuda.Stream()

    def run(h_dev, out_ids_dev):
        for dst, src in zip((kv.page_table, kv.seq_len, kv.n_pages, kv.free_stack, kv.free_top), saved):
            dst.copy_(src)
        torch.cuda.synchronize()
        sd = L.deer_step_dev(vs.q.data_ptr(), vs.k_blk.data_ptr(), vs.v_blk.data_ptr(), vs.attn_out.data_ptr(), h_dev.data_ptr(),
                             vs.seq_ids.data_ptr(), vs.draft_ids.data_ptr(), vs.target_ids.data_ptr(), vs.accept_len.data_ptr(),
                             out_ids_dev.data_ptr(), vs.n_out.data_ptr(), vs.attn_ws.data_ptr(), vs.attn_ws.numel(),
                             vs.lm_ws.data_ptr(), vs.lm_ws.numel())
        L.deer_verify_step_host(kv, sd, w_dev, hq, hkb, hvb, hh, hd, cfg.B, cfg.k, cfg.Hq, cfg.hid, cfg.V, vs.scale, msl,
                                ha, ho, hn, stream=stream)
        return ha.numpy().copy(), ho.numpy().copy()

    a, out = run(vs.h, vs.out_ids)                      # records a graph
    want_a, want_out, _ = O.accept_greedy(drafts, t0)
    np.testing.assert_array_equal(a, want_a)
    np.testing.assert_array_equal(out, want_out)
    # same call, other device buffer for the result ids: the old one must stay as it was
    other_out = torch.full_like(vs.out_ids, -77)
    vs.out_ids.fill_(-55)
    torch.cuda.synchronize()
    a, out = run(vs.h, other_out)
    np.testing.assert_array_equal(out, want_out)
    assert (vs.out_ids.cpu().numpy() == -55).all()
    # same call, other device buffer for the hidden states, new host content
    hh.copy_(h1)
    other_h = torch.zeros_like(vs.h)
    a, out = run(other_h, vs.out_ids)
    want_a, want_out, _ = O.accept_greedy(drafts, t1)
    np.testing.assert_array_equal(a, want_a)
    np.testing.assert_array_equal(out, want_out)
    assert torch.equal(other_h.cpu(), h1)


@pytest.mark.parametrize("B,ctx,k,V,steps", [
    (4, 32768, 32, 8192, 64),          # the longest context, every sequence followed by the oracle
    (64, 16384, 16, 8192, 64),         # the largest batch with a long context: four sampled sequences
    (64, 32768, 8, 151936, 1),         # the largest batch and context at the full vocabulary, one step
])
def test_c5_sweep_corners(B, ctx, k, V, steps):
    """Sweep corners at their real sizes.  The pools are drawn on the device (gigabytes); the oracle follows a seeded
    sample of four sequences (their pages copied out) for the attention values and the cache contents, and every
    sequence for the integer cache state, over all consecutive steps, each with freshly planted drafts and a commit.
    Attention is compared at the first, a middle and the last step."""
    from paper_2512_15176_b200 import binding as L
    from paper_2512_15176_b200.runner import VerifyStep
    cfg = W.sweep_config(B, ctx, k, W.MASK_CAUSAL, steps=steps).with_(V=V)
    lengths = W.seq_lengths(cfg)
    lay = W.kv_layout(cfg, lengths)
    kp, vp = W.kv_pools(cfg, lay.num_pages, device="cuda", sigma=1.0)
    kv = L.KVCache.from_layout(lay, kp, vp, "cuda")
    del kp, vp
    sample = sorted(W.rng(cfg.seed, "sample").choice(B, size=min(4, B), replace=False).tolist())
    okv_s = Hn.sampled_oracle_kv(kv, sample, steps * k)
    okv_all = O.PagedKV(np.zeros((1, 1, 16, 1), np.float32), np.zeros((1, 1, 16, 1), np.float32), lay.page_table, lay.seq_len,
                        lay.n_pages, lay.free_stack, lay.free_top)
    w = W.lm_head(cfg)
    w64 = Hn.f64(w)
    msl = int(lengths.max()) + steps * k
    vs = VerifyStep(cfg, kv, w.cuda(), msl, store_logits=False)
    ids_all, ids_s = np.arange(B), np.arange(len(sample))
    check_at = {0, steps // 2, steps - 1}
    # the hidden states (and so the targets) stay; every step plants a new prefix and draws new block rows
    h, z, _ = Hn.draw_hidden_with_margin(cfg, w64, 0)
    target = O.select_argmax(z).reshape(B, k)
    vs.load(h=h)
    for step in range(steps):
        q, kb, vb = Hn.draw_block(cfg, step, True)
        Lp = W.planted_prefix_lengths(cfg, step)
        drafts = W.plant_drafts(cfg, target, Lp, step)
        a, out, n = O.accept_greedy(drafts, target)
        np.testing.assert_array_equal(a, Lp)
        assert okv_all.reserve(ids_all, k) and okv_s.reserve(ids_s, k)
        qs, kbs, vbs = (Hn.f64(t[sample]) for t in (q, kb, vb))
        if step in check_at:
            want = O.block_attention(qs, kbs, vbs, okv_s.k_pool, okv_s.v_pool, okv_s.page_table, okv_s.seq_len, ids_s,
                                     cfg.mask, 1.0 / math.sqrt(cfg.D))
        okv_s.append(ids_s, kbs.astype(np.float32), vbs.astype(np.float32))
        okv_all.commit(ids_all, a)
        okv_s.commit(ids_s, a[sample])
        vs.load(q, kb, vb, None, drafts)
        vs.run()
        if step in check_at:
            torch.cuda.synchronize()
            assert L.deer_kv_status(kv) == 0
            Hn.check_attention(vs.attn_out.cpu()[sample], want, f"{cfg.name} step {step}")
            if step == 0:
                Hn.check_ids(vs.target_ids.cpu().numpy(), target, z, cfg.name)
            np.testing.assert_array_equal(vs.accept_len.cpu().numpy(), a)
            np.testing.assert_array_equal(vs.out_ids.cpu().numpy(), out)
            Hn.kv_state_equal(kv, okv_all, f"{cfg.name} step {step}")
    torch.cuda.synchronize()
    assert L.deer_kv_status(kv) == 0
    Hn.kv_state_equal(kv, okv_all, cfg.name)
    # contents of the sampled sequences: each side gathers through its own page table
    pt, sl = kv.page_table.cpu().numpy(), kv.seq_len.cpu().numpy()
    for j, s in enumerate(sample):
        npg = -(-int(sl[s]) // 16)
        pages = torch.from_numpy(pt[s, :npg].astype(np.int64)).cuda()
        for pool, opool in ((kv.k_pool, okv_s.k_pool), (kv.v_pool, okv_s.v_pool)):
            got = pool[pages].float().cpu().numpy().transpose(0, 2, 1, 3).reshape(npg * 16, cfg.Hkv, cfg.D)[:int(sl[s])]
            want_c = O.gather_prefix(opool, okv_s.page_table[j], int(okv_s.seq_len[j]), 16)
            np.testing.assert_array_equal(got, want_c, err_msg=f"{cfg.name} contents of sequence {s}")
