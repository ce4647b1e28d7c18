"""GPU parity of deer_accept (stage-isolated, bit-exact) and of the paged-KV
reserve / append / commit cycle against the oracle."""
import math

import numpy as np
import pytest
import torch

from oracle import deer_oracle as O
from paper_2512_15176_b200 import workload as W
from tests import harness as Hn

pytestmark = pytest.mark.gpu


def _greedy(draft, target, eos=-1, bonus=False):
    from paper_2512_15176_b200 import binding as L
    B, k = draft.shape
    dev = "cuda"
    a = torch.full((B,), -9, dtype=torch.int32, device=dev)
    o = torch.full((B, k), -9, dtype=torch.int32, device=dev)
    n = torch.full((B,), -9, dtype=torch.int32, device=dev)
    L.deer_accept(L.DEER_ACC_GREEDY | (L.DEER_ACC_BONUS if bonus else 0), B, k, 100, torch.as_tensor(draft, device=dev),
                  torch.as_tensor(target, device=dev),
                  None, None, None, 1.0, None, None, None, eos, a, o, n, None)
    torch.cuda.synchronize()
    return a.cpu().numpy(), o.cpu().numpy(), n.cpu().numpy()


@pytest.mark.parametrize("B,k", [(1, 8), (64, 32), (300, 5), (7, 1)])
def test_greedy_bit_exact(B, k):
    cfg = W.StepConfig("g", B, 4, 2, 64, k, 64, 5000, (0, 0), seed=600 + B)
    target = W.rng(cfg.seed, "t").integers(0, cfg.V, size=(B, k)).astype(np.int32)
    Lp = W.planted_prefix_lengths(cfg)
    draft = W.plant_drafts(cfg, target, Lp)
    for eos in (-1, int(target[0, min(1, k - 1)])):
        got = _greedy(draft, target, eos)
        want = O.accept_greedy(draft, target, eos)
        for g, w_ in zip(got, want):
            np.testing.assert_array_equal(g, w_)
        if eos < 0:
            np.testing.assert_array_equal(got[0], Lp)      # the planted-prefix invariant
        # k-1 drafts and one more row: always accept_len + 1 tokens
        got = _greedy(draft, target, eos, bonus=True)
        want = O.accept_greedy(draft, target, eos, bonus=True)
        for g, w_ in zip(got, want):
            np.testing.assert_array_equal(g, w_)


def _sample(cfg, zt32, ql, drafts, u, r, eos=-1, split=False, bonus=False):
    """split: the drafter statistics come from deer_draft_stats on a second stream, joined before the acceptance."""
    from paper_2512_15176_b200 import binding as L
    B, k, V = cfg.B, cfg.k, cfg.V
    dev = "cuda"
    T = float(np.float32(cfg.temperature))
    lse = torch.from_numpy(O.logsumexp(zt32.reshape(B * k, V), T).astype(np.float32)).to(dev)
    zd = torch.from_numpy(np.take_along_axis(zt32, drafts[..., None].astype(np.int64), axis=2)[..., 0].astype(np.float32)).to(dev)
    a = torch.full((B,), -9, dtype=torch.int32, device=dev)
    o = torch.full((B, k), -9, dtype=torch.int32, device=dev)
    n = torch.full((B,), -9, dtype=torch.int32, device=dev)
    ws = torch.empty(L.deer_accept_workspace_bytes(L.DEER_ACC_SAMPLE, B, k, V), dtype=torch.uint8, device=dev)
    d_dev, ql_dev = torch.as_tensor(drafts, device=dev), ql.to(dev)
    mode = L.DEER_ACC_SAMPLE
    if split:
        mode = L.DEER_ACC_SAMPLE_PRESTATS
        side, main = torch.cuda.Stream(), torch.cuda.current_stream()
        side.wait_stream(main)
        with torch.cuda.stream(side):
            L.deer_draft_stats(B, k, V, d_dev, ql_dev, ws)
        main.wait_stream(side)
    L.deer_accept(mode | (L.DEER_ACC_BONUS if bonus else 0), B, k, V, d_dev, None, torch.from_numpy(zt32).to(dev), lse, zd,
                  cfg.temperature, ql_dev, u.to(dev), r.to(dev), eos, a, o, n, ws)
    torch.cuda.synchronize()
    return a.cpu().numpy(), o.cpu().numpy(), n.cpu().numpy()


@pytest.mark.parametrize("B,k,V,T", [(4, 8, 1000, 1.0), (16, 32, 4099, 0.6), (3, 5, 151936, 1.0), (33, 4, 37, 1.7)])
def test_sampling_bit_exact_on_identical_logits(B, k, V, T):
    """Both sides receive the same fp32 target logits, drafter logits, uniforms;
    accepted lengths and every emitted id (incl. the residual draw) must agree."""
    cfg = W.StepConfig("s", B, 4, 2, 64, k, 64, V, (0, 0), mode="sample", temperature=T, seed=700 + V)
    ql0 = W.draft_logits(cfg)
    # target logits close enough to the drafter's that accept lengths spread over 0..k
    zt32 = (ql0 + W.normal(cfg.seed, "zt", (B, k, V), 0.5, dtype=torch.float32)).numpy() * np.float32(T)
    ql, drafts, u, r, _ = Hn.sampling_inputs(cfg, zt32)
    got = _sample(cfg, zt32, ql, drafts, u, r)
    want = O.accept_sample(drafts, zt32, float(np.float32(T)), ql.numpy(), u.numpy(), r.numpy())
    for g, w_, name in zip(got, want, ("accept_len", "out_ids", "n_out")):
        np.testing.assert_array_equal(g, w_, err_msg=name)
    assert len(set(want[0].tolist())) > 1 or B < 4
    # the drafter statistics computed ahead of time on another stream: same result
    got = _sample(cfg, zt32, ql, drafts, u, r, split=True)
    for g, w_, name in zip(got, want, ("accept_len", "out_ids", "n_out")):
        np.testing.assert_array_equal(g, w_, err_msg=name + " (deer_draft_stats)")
    # EOS: cut at a token that the oracle emitted
    eos = int(want[1][0, 0])
    got = _sample(cfg, zt32, ql, drafts, u, r, eos)
    want = O.accept_sample(drafts, zt32, float(np.float32(T)), ql.numpy(), u.numpy(), r.numpy(), eos)
    for g, w_ in zip(got, want):
        np.testing.assert_array_equal(g, w_)


@pytest.mark.parametrize("B,k,V,T", [(6, 4, 1000, 1.0), (16, 8, 4099, 0.8), (5, 1, 300, 1.0)])
def test_sampling_with_the_extra_row(B, k, V, T):
    """k-1 drafts and one more row.  Target logits close to the drafter's, so that many
    blocks are accepted in full and draw their last token from p of the extra row; r is
    cleared against that row's CDF edges too."""
    cfg = W.StepConfig("sb", B, 4, 2, 64, k, 64, V, (0, 0), mode="sample", temperature=T, seed=760 + V)
    ql0 = W.draft_logits(cfg)
    zt32 = (ql0 + W.normal(cfg.seed, "zt", (B, k, V), 0.15, dtype=torch.float32)).numpy() * np.float32(T)
    ql, drafts, u, r, _ = Hn.sampling_inputs(cfg, zt32, bonus=True)
    want = O.accept_sample(drafts, zt32, float(np.float32(T)), ql.numpy(), u.numpy(), r.numpy(), bonus=True)
    assert (want[2] == want[0] + 1).all()
    assert (want[0] == k - 1).any()                      # the extra row is exercised
    for split in (False, True):
        got = _sample(cfg, zt32, ql, drafts, u, r, split=split, bonus=True)
        for g, w_, name in zip(got, want, ("accept_len", "out_ids", "n_out")):
            np.testing.assert_array_equal(g, w_, err_msg=name)


@pytest.mark.parametrize("rv", [0.0, float(np.nextafter(np.float32(1.0), np.float32(0.0)))])
def test_residual_draw_at_the_ends_of_the_unit_interval(rv):
    """r = 0 selects the first token of the vocabulary (the smallest v whose cumulative residual is >= 0) and the
    largest fp32 below 1 the last token that carries residual mass or one next to it; every sequence is made to
    reject at row 0 (u next to 1 against an alpha far below 1)."""
    B, k, V = 5, 3, 777
    cfg = W.StepConfig("r", B, 4, 2, 64, k, 64, V, (0, 0), mode="sample", temperature=1.0, seed=820)
    ql = W.draft_logits(cfg)
    zt32 = W.normal(cfg.seed, "zt", (B, k, V), 1.0, dtype=torch.float32).numpy()
    p0 = np.stack([O.softmax_f64(zt32[b, 0], 1.0) for b in range(B)])
    q0 = np.stack([O.softmax_f64(ql[b, 0].numpy(), 1.0) for b in range(B)])
    drafts = np.zeros((B, k), dtype=np.int32)
    drafts[:, 0] = np.argmax(q0 / p0, axis=1)           # alpha = p/q is smallest there
    u = torch.full((B, k), 0.999)
    r = torch.full((B,), rv, dtype=torch.float32)
    want = O.accept_sample(drafts, zt32, 1.0, ql.numpy(), u.numpy(), r.numpy())
    assert (want[0] == 0).all()
    got = _sample(cfg, zt32, ql, drafts, u, r)
    np.testing.assert_array_equal(got[0], want[0])
    np.testing.assert_array_equal(got[2], want[2])
    if rv == 0.0:
        np.testing.assert_array_equal(got[1], want[1])
        assert (got[1][:, 0] == 0).all()
    else:
        for b in range(B):
            res, S = O.residual_distribution(p0[b], q0[b])
            cdf = np.cumsum(res)
            v = int(got[1][b, 0])
            assert res[v] > 0 and cdf[v] >= float(np.float32(rv)) * S * (1 - 1e-6), (b, v)


def test_sampling_identical_distributions_accept_everything():
    """p == q gives alpha = 1 at every position, so even u next to 1 accepts."""
    cfg = W.StepConfig("z", 2, 4, 2, 64, 2, 64, 500, (0, 0), mode="sample", temperature=1.0, seed=800)
    ql = W.draft_logits(cfg)
    zt32 = ql.numpy().copy()
    drafts = np.zeros((2, 2), dtype=np.int32)
    u = torch.full((2, 2), 0.999999)
    r = torch.tensor([0.3, 0.9])
    # identical distributions: alpha = 1, everything accepted whatever u is
    got = _sample(cfg, zt32, ql, drafts, u, r)
    want = O.accept_sample(drafts, zt32, 1.0, ql.numpy(), u.numpy(), r.numpy())
    for g, w_ in zip(got, want):
        np.testing.assert_array_equal(g, w_)
    assert (got[0] == 2).all()


# ---------------------------------------------------------------- KV cycle

@pytest.mark.parametrize("B,k,Hkv,D", [(4, 8, 2, 64), (64, 32, 8, 128), (5, 1, 1, 128)])
def test_kv_soak_64_steps(B, k, Hkv, D):
    """reserve -> append (through deer_block_attn) -> commit(keep) repeated 64
    times with random keeps, state and contents compared bit for bit each step."""
    from paper_2512_15176_b200 import binding as L
    steps = 64
    cfg = W.StepConfig("kv", B, Hkv * 2, Hkv, D, k, 64, 64, (0, 300), seed=900 + B, growth=steps * k)
    st = Hn.draw_state(cfg, stress=True)
    okv = Hn.oracle_kv(st)
    kv = Hn.gpu_kv(st)
    ids = np.arange(B)
    seq_ids = torch.arange(B, dtype=torch.int32, device="cuda")
    msl = int(st.lengths.max()) + steps * k
    ws = torch.empty(L.deer_block_attn_workspace_bytes(B, k, cfg.Hq, Hkv, D, msl), dtype=torch.uint8, device="cuda")
    out = torch.empty(B, k, cfg.Hq, D, dtype=torch.bfloat16, device="cuda")
    gen = W.rng(cfg.seed, "keep")
    for step in range(steps):
        q, kb, vb = Hn.draw_block(cfg, step, True)
        keep = gen.integers(0, k + 1, size=B).astype(np.int32)
        L.deer_kv_reserve(kv, seq_ids, k)
        L.deer_block_attn(kv, seq_ids, q.cuda(), kb.cuda(), vb.cuda(), out, L.DEER_MASK_CAUSAL, 1, 1.0 / math.sqrt(D), msl, ws)
        L.deer_kv_commit(kv, seq_ids, torch.from_numpy(keep).cuda(), k)
        assert okv.reserve(ids, k)
        okv.append(ids, Hn.f64(kb).astype(np.float32), Hn.f64(vb).astype(np.float32))
        okv.commit(ids, keep)
        if step % 8 == 7 or step < 3:
            torch.cuda.synchronize()
            Hn.kv_state_equal(kv, okv, f"step {step}")
            Hn.kv_contents_equal(kv, okv, label=f"step {step}")
    assert L.deer_kv_status(kv) == 0
    # attention over the grown cache still matches (the appended rows are really there)
    q, kb, vb = Hn.draw_block(cfg, steps, True)
    want = Hn.oracle_attention(cfg, okv, q, kb, vb)
    L.deer_block_attn(kv, seq_ids, q.cuda(), kb.cuda(), vb.cuda(), out, L.DEER_MASK_CAUSAL, 0, 1.0 / math.sqrt(D), msl, ws)
    torch.cuda.synchronize()
    Hn.check_attention(out.cpu(), want, "after soak")


@pytest.mark.parametrize("B,k,bonus,with_eos", [(1, 32, False, False), (64, 32, False, True), (300, 5, True, False), (7, 1, False, True)])
def test_accept_commit_in_one_launch(B, k, bonus, with_eos):
    """deer_accept_commit against the oracle's greedy acceptance followed by its commit: the acceptance outputs and
    the whole cache state (lengths, page counts, page table, free stack), bit for bit."""
    from paper_2512_15176_b200 import binding as L
    cfg = W.StepConfig("ac", B, 4, 2, 64, k, 64, 5000, (0, 200), seed=960 + B)
    st = Hn.draw_state(cfg, stress=True)
    okv = Hn.oracle_kv(st)
    kv = Hn.gpu_kv(st)
    ids = np.arange(B)
    seq_ids = torch.arange(B, dtype=torch.int32, device="cuda")
    target = W.rng(cfg.seed, "t").integers(0, cfg.V, size=(B, k)).astype(np.int32)
    draft = W.plant_drafts(cfg, target, W.planted_prefix_lengths(cfg))
    eos = int(target[0, min(1, k - 1)]) if with_eos else -1
    a = torch.full((B,), -9, dtype=torch.int32, device="cuda")
    o = torch.full((B, k), -9, dtype=torch.int32, device="cuda")
    n = torch.full((B,), -9, dtype=torch.int32, device="cuda")
    L.deer_kv_reserve(kv, seq_ids, k)
    L.deer_accept_commit(kv, seq_ids, L.DEER_ACC_GREEDY | (L.DEER_ACC_BONUS if bonus else 0), k, torch.as_tensor(draft, device="cuda"),
                         torch.as_tensor(target, device="cuda"), eos, a, o, n)
    torch.cuda.synchronize()
    want = O.accept_greedy(draft, target, eos, bonus=bonus)
    for g, w_ in zip((a.cpu().numpy(), o.cpu().numpy(), n.cpu().numpy()), want):
        np.testing.assert_array_equal(g, w_)
    assert okv.reserve(ids, k)
    okv.commit(ids, want[0])
    Hn.kv_state_equal(kv, okv, "after accept + commit")
    assert L.deer_kv_status(kv) == 0
    # sampling is not this call's business
    with pytest.raises(L.DeerError):
        L.deer_accept_commit(kv, seq_ids, L.DEER_ACC_SAMPLE, k, torch.as_tensor(draft, device="cuda"),
                             torch.as_tensor(target, device="cuda"), eos, a, o, n)


def test_reserve_without_pages_reports_and_changes_nothing():
    from paper_2512_15176_b200 import binding as L
    cfg = W.StepConfig("np", 3, 4, 2, 64, 32, 64, 64, (16, 16), seed=950)
    st = Hn.draw_state(cfg)
    st.layout.free_top[0] = 2            # three sequences need two pages each
    kv = Hn.gpu_kv(st)
    before = (kv.page_table.clone(), kv.n_pages.clone(), kv.free_top.clone())
    L.deer_kv_reserve(kv, torch.arange(3, dtype=torch.int32, device="cuda"), 32)
    assert L.deer_kv_status(kv) == L.DEER_ERR_NO_PAGES
    assert torch.equal(kv.page_table, before[0]) and torch.equal(kv.n_pages, before[1]) and torch.equal(kv.free_top, before[2])


def test_bounded_wait_gives_up_and_reports():
    """The wait every tensor-core kernel uses, on a barrier nothing arrives on: it gives up after its limit (about a
    second), the status word says so, and the context goes on working."""
    import time
    from paper_2512_15176_b200 import binding as L
    cfg = W.StepConfig("bw", 2, 4, 2, 64, 4, 64, 64, (8, 8), seed=990)
    st = Hn.draw_state(cfg)
    kv = Hn.gpu_kv(st)
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    L.deer_selftest_bounded_wait(kv)
    torch.cuda.synchronize()
    dt = time.perf_counter() - t0
    assert 0.2 < dt < 10.0, dt
    assert L.deer_kv_status(kv) == L.DEER_ERR_TIMEOUT
    assert L.deer_kv_status(kv) == 0
    L.deer_kv_reserve(kv, torch.arange(2, dtype=torch.int32, device="cuda"), 4)
    torch.cuda.synchronize()
    assert L.deer_kv_status(kv) == 0
