"""GPU parity of the drafter-side calls: block attention with row states, the re-fill decision, the cache refresh,
and one whole pass of Algorithm 1's loop body -- draft (several iterations), verify, accept, emit, commit, refresh --
chained on the device, against the oracle."""
import math

import numpy as np
import pytest
import torch

from oracle import deer_oracle as O
from paper_2512_15176_b200 import workload as W
from tests import harness as Hn

pytestmark = pytest.mark.gpu


def _states(cfg, seed, p_absent=0.2, p_decoded=0.4):
    r = W.rng(seed, "row_state")
    st = r.choice([-1, 0, 1], size=(cfg.B, cfg.k), p=[p_absent, p_decoded, 1 - p_absent - p_decoded]).astype(np.int32)
    return st


@pytest.mark.parametrize("B,k,Hq,Hkv,D,lens", [
    (3, 8, 8, 2, 64, [0, 1, 255]),
    (2, 32, 32, 8, 128, [1500, 777]),
    (2, 32, 32, 4, 128, [300, 1031]),          # two row tiles per KV head
    (2, 7, 6, 2, 128, [130, 0]),
    (4, 16, 16, 8, 128, [64, 65, 63, 2000]),
])
def test_attention_with_row_states(B, k, Hq, Hkv, D, lens):
    from paper_2512_15176_b200 import binding as L
    cfg = W.StepConfig("rows", B, Hq, Hkv, D, k, 64, 64, (0, 0), mask=W.MASK_BIDIR, seed=1500 + B * k)
    st = Hn.draw_state(cfg, lens, True)
    q, kb, vb = Hn.draw_block(cfg, 0, True)
    okv, kv = Hn.oracle_kv(st), Hn.gpu_kv(st)
    seq_ids = torch.arange(B, dtype=torch.int32, device="cuda")
    msl = int(max(lens))
    ws = torch.empty(max(16, L.deer_block_attn_workspace_bytes(B, k, Hq, Hkv, D, msl)), dtype=torch.uint8, device="cuda")
    for case, rs in enumerate([np.ones((B, k), np.int32), np.zeros((B, k), np.int32), _states(cfg, 1), _states(cfg, 2, 0.5, 0.3)]):
        if case >= 2:
            rs[0, 0] = 1                       # at least one of each of the live kinds
            rs[-1, -1] = 0
        # what sits in absent rows must not matter: poison it on the device side only
        qd, kd, vd = q.clone(), kb.clone(), vb.clone()
        absent = torch.from_numpy(rs == -1)
        qd[absent], kd[absent], vd[absent] = 3.0e4, -3.0e4, float("inf")
        want = O.block_attention(Hn.f64(q), Hn.f64(kb), Hn.f64(vb), okv.k_pool, okv.v_pool, okv.page_table, okv.seq_len,
                                 np.arange(B), cfg.mask, 1.0 / math.sqrt(D), row_state=rs)
        out = torch.full((B, k, Hq, D), float("nan"), dtype=torch.bfloat16, device="cuda")
        L.deer_block_attn_rows(kv, seq_ids, qd.cuda(), kd.cuda(), vd.cuda(), out, torch.from_numpy(rs).cuda(), L.DEER_MASK_BIDIR, 0,
                               1.0 / math.sqrt(D), msl, ws)
        torch.cuda.synchronize()
        assert L.deer_kv_status(kv) == 0
        live = rs != -1
        got = out.cpu()
        Hn.check_attention(got[torch.from_numpy(live)], want[live], f"row states case {case}")
    # the states belong to the bidirectional mask
    with pytest.raises(L.DeerError):
        L.deer_block_attn_rows(kv, seq_ids, q.cuda(), kb.cuda(), vb.cuda(), out, torch.from_numpy(rs).cuda(), L.DEER_MASK_CAUSAL, 0,
                               1.0 / math.sqrt(D), msl, ws)


@pytest.mark.parametrize("D", [64, 128])
def test_refresh_pass_appends_the_decoded_rows(D):
    """Ragged numbers of tokens per sequence join the drafter's cache: rows 0..appended-1 decoded, the rest absent;
    attention output of the live rows, cache state and contents against the oracle, over three rounds."""
    from paper_2512_15176_b200 import binding as L
    B, k, Hkv = 5, 8, 2
    cfg = W.StepConfig("refresh", B, 4, Hkv, D, k, 64, 64, (3, 90), mask=W.MASK_BIDIR, seed=1600 + D, growth=3 * k)
    st = Hn.draw_state(cfg, None, True)
    okv, kv = Hn.oracle_kv(st), Hn.gpu_kv(st)
    ids = np.arange(B)
    seq_ids = torch.arange(B, dtype=torch.int32, device="cuda")
    msl = int(st.lengths.max()) + 3 * k
    ws = torch.empty(L.deer_block_attn_workspace_bytes(B, k, cfg.Hq, Hkv, D, msl), dtype=torch.uint8, device="cuda")
    out = torch.empty(B, k, cfg.Hq, D, dtype=torch.bfloat16, device="cuda")
    rs_dev = torch.empty(B, k, dtype=torch.int32, device="cuda")
    gen = W.rng(cfg.seed, "appended")
    for rnd in range(3):
        appended = gen.integers(0, k + 1, size=B).astype(np.int32)
        appended[rnd % B] = 0 if rnd == 0 else k
        q, kb, vb = Hn.draw_block(cfg, rnd, True)
        rs = O.refresh_rows(appended, k)
        assert okv.reserve(ids, k)
        want = O.block_attention(Hn.f64(q), Hn.f64(kb), Hn.f64(vb), okv.k_pool, okv.v_pool, okv.page_table, okv.seq_len, ids,
                                 cfg.mask, 1.0 / math.sqrt(D), row_state=rs)
        okv.append(ids, Hn.f64(kb).astype(np.float32), Hn.f64(vb).astype(np.float32), row_state=rs)
        okv.commit(ids, appended)
        app_dev = torch.from_numpy(appended).cuda()
        L.deer_refresh_rows(app_dev, rs_dev)
        L.deer_kv_reserve(kv, seq_ids, k)
        L.deer_block_attn_rows(kv, seq_ids, q.cuda(), kb.cuda(), vb.cuda(), out, rs_dev, L.DEER_MASK_BIDIR, 1, 1.0 / math.sqrt(D),
                               msl, ws)
        L.deer_kv_commit(kv, seq_ids, app_dev, k)
        torch.cuda.synchronize()
        assert L.deer_kv_status(kv) == 0
        np.testing.assert_array_equal(rs_dev.cpu().numpy(), rs)
        live = rs != -1
        if live.any():
            Hn.check_attention(out.cpu()[torch.from_numpy(live)], want[live], f"refresh round {rnd}")
        Hn.kv_state_equal(kv, okv, f"refresh round {rnd}")
        Hn.kv_contents_equal(kv, okv, label=f"refresh round {rnd}")


@pytest.mark.parametrize("B,k", [(1, 1), (7, 8), (300, 32)])
def test_refill_decision_bit_exact(B, k):
    from paper_2512_15176_b200 import binding as L
    r = W.rng(1700 + B, "refill")
    st = r.choice([-1, 0, 1], size=(B, k), p=[0.1, 0.3, 0.6]).astype(np.int32)
    tok = np.where(st == 0, r.integers(0, 1000, size=(B, k)), -1).astype(np.int32)
    st_d, tok_d = torch.from_numpy(st).cuda(), torch.from_numpy(tok).cuda()
    left_d = torch.full((B,), -9, dtype=torch.int32, device="cuda")
    thr = math.log(0.5)
    for it in range(k + 1):
        ids = r.integers(0, 1000, size=(B, k)).astype(np.int32)
        lp = np.log(r.random((B, k))).astype(np.float32)
        lp[:, : k // 2] = np.round(lp[:, : k // 2])            # ties among the most confident rows
        st, tok, left = O.refill_step(st, tok, ids, lp, thr if it % 2 == 0 else 1.0)
        L.deer_refill(torch.from_numpy(ids).cuda(), torch.from_numpy(lp).cuda(), thr if it % 2 == 0 else 1.0, st_d, tok_d, left_d)
        torch.cuda.synchronize()
        np.testing.assert_array_equal(st_d.cpu().numpy(), st)
        np.testing.assert_array_equal(tok_d.cpu().numpy(), tok)
        np.testing.assert_array_equal(left_d.cpu().numpy(), left)
    assert (st != 1).all()                                      # k + 1 iterations finish any block


def test_whole_loop_body_on_the_device():
    """Algorithm 1's loop body with both models' hot paths chained on the device and no host round trip inside a
    pass: the drafter fills a block over up to three iterations (its own paged cache, bidirectional attention with
    row states, LM head with log-probabilities, re-fill decisions), the drafts go to the verifier's greedy step,
    deer_emit appends, both caches commit -- the drafter's through the refresh pass.  Four passes; drafts, outputs
    and both caches against the oracle.  The drafter's hidden states are planted so that its tokens match the
    verifier's for a prefix of each block (so some blocks are accepted in part, some in full)."""
    from paper_2512_15176_b200 import binding as L
    from paper_2512_15176_b200.runner import DecodeLoop, DrafterBlock, VerifyStep
    passes, iters, max_new = 4, 3, 40
    vcfg = W.StepConfig("loop-v", 3, 8, 2, 128, 8, 256, 2048, (40, 300), seed=1800, growth=passes * 8)
    dcfg = W.StepConfig("loop-d", 3, 4, 2, 64, 8, 128, 2048, (40, 300), mask=W.MASK_BIDIR, seed=1801, growth=passes * 8)
    B, k = vcfg.B, vcfg.k
    vst, dst = Hn.draw_state(vcfg, None, True), Hn.draw_state(dcfg, W.seq_lengths(vcfg), True)
    vokv, vkv = Hn.oracle_kv(vst), Hn.gpu_kv(vst)
    dokv, dkv = Hn.oracle_kv(dst), Hn.gpu_kv(dst)
    wv, wd = W.lm_head(vcfg), W.lm_head(dcfg)
    wv64, wd64 = Hn.f64(wv), Hn.f64(wd)
    msl = int(vst.lengths.max()) + passes * k
    vs = VerifyStep(vcfg, vkv, wv.cuda(), msl, store_logits=False)
    loop = DecodeLoop(vs, -1, max_new)
    db = DrafterBlock(dcfg, dkv, wd.cuda(), msl)
    ost = O.DecodeState(B, max_new)
    ids = np.arange(B)
    thr = math.log(0.02)
    kept_total = np.zeros(B, dtype=np.int64)
    for ps in range(passes):
        # ---- verifier inputs of this pass and its targets (known in advance: the hidden states are inputs) ----
        vq, vkb, vvb = Hn.draw_block(vcfg, ps, True)
        vh, vz, _ = Hn.draw_hidden_with_margin(vcfg, wv64, ps)
        target = O.select_argmax(vz).reshape(B, k)
        # ---- the drafter fills its block ----
        db.start_block()
        st = np.ones((B, k), np.int32)
        tok = np.full((B, k), -1, np.int32)
        for it in range(iters):
            dq, dkb, dvb = Hn.draw_block(dcfg, 10 * ps + it, True)
            dh, dz, _ = Hn.draw_hidden_with_margin(dcfg, wd64, 10 * ps + it)
            # plant: the drafter's hidden state of row i is replaced so that its argmax is the verifier's target on a
            # prefix of the block (a large multiple of that token's weight row)
            plant = W.planted_prefix_lengths(dcfg.with_(prefix_law="uniform"), 10 * ps + it)
            dh = dh.clone()
            for b in range(B):
                for i in range(int(plant[b])):
                    dh[b * k + i] = (wd[int(target[b, i])].float() * 40.0).to(torch.bfloat16)
            dz = O.lm_logits(Hn.f64(dh), wd64)
            assert (O.top2_gap(dz) > 1e-2).all()
            want_attn = O.block_attention(Hn.f64(dq), Hn.f64(dkb), Hn.f64(dvb), dokv.k_pool, dokv.v_pool, dokv.page_table,
                                          dokv.seq_len, ids, W.MASK_BIDIR, 1.0 / math.sqrt(dcfg.D), row_state=st)
            live = st != -1
            lp = O.max_logprob(dz).reshape(B, k)
            # keep the decisions clear of the threshold and of ties in confidence
            assert (np.abs(lp - thr) > 1e-3).all()
            st_before = st
            st, tok, left = O.refill_step(st, tok, O.select_argmax(dz).reshape(B, k), lp, thr if it < iters - 1 else -math.inf)
            db.load(dq, dkb, dvb, dh)
            db.iteration(thr if it < iters - 1 else -math.inf)
            torch.cuda.synchronize()
            Hn.check_attention(db.attn_out.cpu()[torch.from_numpy(live)], want_attn[live], f"pass {ps} iteration {it}")
            np.testing.assert_array_equal(db.row_state.cpu().numpy(), st)
            np.testing.assert_array_equal(db.tokens.cpu().numpy(), tok)
            assert (st_before != st).any() or (st_before != 1).all()
        assert (st == 0).all()
        drafts = tok
        # ---- verify, accept, emit, commit: on the device without a host round trip ----
        assert vokv.reserve(ids, k)
        vokv.append(ids, Hn.f64(vkb).astype(np.float32), Hn.f64(vvb).astype(np.float32))
        a, out, n = O.accept_greedy(drafts, target)
        keep = ost.emit(a, out, n, -1)
        kept_total = kept_total + keep
        vokv.commit(ids, keep)
        vs.load(vq, vkb, vvb, vh)
        vs.draft_ids.copy_(db.tokens)                           # the drafter's block, device to device
        loop.one_pass()
        # ---- the drafter's cache takes in what joined the output ----
        rq, rkb, rvb = Hn.draw_block(dcfg, 10 * ps + 9, True)
        rs = O.refresh_rows(ost.appended, k)
        assert dokv.reserve(ids, k)
        dokv.append(ids, Hn.f64(rkb).astype(np.float32), Hn.f64(rvb).astype(np.float32), row_state=rs)
        dokv.commit(ids, ost.appended)
        db.load(rq, rkb, rvb)
        db.refresh(loop.appended)
    torch.cuda.synchronize()
    assert L.deer_kv_status(vkv) == 0 and L.deer_kv_status(dkv) == 0
    np.testing.assert_array_equal(loop.tokens.cpu().numpy(), ost.tokens)
    np.testing.assert_array_equal(loop.n_tokens.cpu().numpy(), ost.n_tokens)
    np.testing.assert_array_equal(loop.finished.cpu().numpy(), ost.finished)
    assert (ost.n_tokens > passes).any()                        # some drafts were accepted
    for kv, okv, name in ((vkv, vokv, "verifier cache"), (dkv, dokv, "drafter cache")):
        Hn.kv_state_equal(kv, okv, name)
        Hn.kv_contents_equal(kv, okv, label=name)
    # the drafter's cache holds the prompt plus everything that was emitted; the verifier's the prompt plus the accepted
    # drafts (a correction was never a block row, so its keys and values are not there in this alignment)
    np.testing.assert_array_equal(dokv.seq_len, vst.lengths + ost.n_tokens)
    np.testing.assert_array_equal(vokv.seq_len, vst.lengths + kept_total)
