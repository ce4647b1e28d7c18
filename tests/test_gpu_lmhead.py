"""GPU parity of deer_lmhead_select against the oracle."""
import numpy as np
import pytest
import torch

from oracle import deer_oracle as O
from paper_2512_15176_b200 import workload as W
from tests import harness as Hn

pytestmark = pytest.mark.gpu


def _select(h, w, mode, T=1.0, drafts=None, logits=False):
    from paper_2512_15176_b200 import binding as L
    M, hid = h.shape
    V = w.shape[0]
    dev = "cuda"
    ids = torch.full((M,), -7, dtype=torch.int32, device=dev)
    mlp = torch.full((M,), float("nan"), device=dev) if mode == L.DEER_SEL_ARGMAX_LOGPROB else None
    lse = torch.full((M,), float("nan"), device=dev) if mode == L.DEER_SEL_SOFTMAX else None
    dl = torch.full((M,), float("nan"), device=dev) if drafts is not None else None
    Z = torch.full((M, V), float("nan"), device=dev) if logits else None
    ws = torch.empty(L.deer_lmhead_workspace_bytes(M, hid, V), dtype=torch.uint8, device=dev)
    d = torch.as_tensor(drafts, dtype=torch.int32, device=dev) if drafts is not None else None
    L.deer_lmhead_select(h.cuda(), w.cuda() if not w.is_cuda else w, mode, T, d, ids, mlp, lse, dl, Z, ws)
    torch.cuda.synchronize()
    return ids.cpu().numpy(), mlp, lse, dl, Z


@pytest.mark.parametrize("M,hid,V", [
    (8, 512, 4096),        # the tiny config's head
    (1, 64, 16),           # smallest legal shapes
    (33, 128, 1000),       # ragged rows, V not a multiple of 16 or 128
    (64, 256, 5003),       # odd V (scalar logits store)
    (100, 192, 3000),      # 128-row tile with a ragged tail
    (256, 128, 2048),      # two 128-row tiles
    (300, 64, 777),
    (384, 128, 4000),      # three 128-row tiles: the second block pair's peer has no rows at all
    (520, 256, 9000),      # three block pairs, the last with 8 rows
])
def test_all_outputs_small(M, hid, V):
    from paper_2512_15176_b200 import binding as L
    cfg = W.StepConfig("lm", 1, 1, 1, 64, 1, hid, V, (0, 0), seed=500 + M).with_(B=M)
    w = W.lm_head(cfg.with_(sigma_w=0.05))
    w64 = Hn.f64(w)
    h, z, _ = Hn.draw_hidden_with_margin(cfg, w64, margin=1e-3)
    drafts = W.rng(cfg.seed, "d").integers(0, V, size=M).astype(np.int32)
    # argmax only
    ids, *_ = _select(h, w, L.DEER_SEL_ARGMAX)
    Hn.check_ids(ids, O.select_argmax(z), z, "argmax")
    # argmax + log-probability, with the logits stored
    ids, mlp, _, _, Z = _select(h, w, L.DEER_SEL_ARGMAX_LOGPROB, logits=True)
    Hn.check_ids(ids, O.select_argmax(z), z, "argmax_logprob")
    np.testing.assert_allclose(mlp.cpu().numpy(), O.max_logprob(z), atol=2e-4, rtol=0)
    Hn.check_logits(Z.cpu(), z, "logits")
    # softmax statistics at a temperature
    for T in (1.0, 0.6):
        T32 = float(np.float32(T))
        ids, _, lse, dl, Z = _select(h, w, L.DEER_SEL_SOFTMAX, T=T, drafts=drafts, logits=True)
        Hn.check_ids(ids, O.select_argmax(z), z, "softmax")
        np.testing.assert_allclose(lse.cpu().numpy(), O.logsumexp(z, T32), atol=3e-4, rtol=0)
        np.testing.assert_allclose(dl.cpu().numpy(), z[np.arange(M), drafts], atol=1e-3, rtol=0)
        Hn.check_logits(Z.cpu(), z, "logits")


def test_ties_resolve_to_the_lowest_index():
    from paper_2512_15176_b200 import binding as L
    hid, V, M = 64, 1024, 16
    h = torch.zeros(M, hid, dtype=torch.bfloat16)
    h[:, 0] = 1.0
    w = torch.zeros(V, hid, dtype=torch.bfloat16)
    w[:, 0] = -1.0
    for v in (3, 130, 131, 700, 1023):       # equal maxima in different warps, tiles and parts
        w[v, 0] = 2.0
    ids, *_ = _select(h, w, L.DEER_SEL_ARGMAX)
    assert (ids == 3).all()
    w[3, 0] = -1.0
    ids, *_ = _select(h, w, L.DEER_SEL_ARGMAX)
    assert (ids == 130).all()


@pytest.fixture(scope="module")
def qwen_head():
    cfg = W.config(1)
    w = W.lm_head(cfg)
    return cfg, w, w.cuda()


def test_qwen3_8b_head_full_size(qwen_head):
    """The 4096 x 151936 head at M = 32 in the launch configuration the benchmark
    times: every id against the oracle, logits on every row."""
    from paper_2512_15176_b200 import binding as L
    cfg, w, w_dev = qwen_head
    w64 = Hn.f64(w)
    h, z, redraws = Hn.draw_hidden_with_margin(cfg, w64)
    assert redraws < cfg.M
    ids, _, _, _, Z = _select(h, w_dev, L.DEER_SEL_ARGMAX, logits=True)
    Hn.check_ids(ids, O.select_argmax(z), z, "C2 argmax")
    Hn.check_logits(Z.cpu(), z, "C2 logits")
    ids2, mlp, *_ = _select(h, w_dev, L.DEER_SEL_ARGMAX_LOGPROB)
    np.testing.assert_array_equal(ids, ids2)
    np.testing.assert_allclose(mlp.cpu().numpy(), O.max_logprob(z), atol=2e-4, rtol=0)


def test_large_m_full_vocab(qwen_head):
    """M = 256 rows (a batch of 8 blocks) against the full vocabulary; hidden 4096."""
    from paper_2512_15176_b200 import binding as L
    cfg, w, w_dev = qwen_head
    cfg = cfg.with_(B=8, seed=1501)
    w64 = Hn.f64(w)
    h, z, _ = Hn.draw_hidden_with_margin(cfg, w64)
    drafts = W.rng(cfg.seed, "d").integers(0, cfg.V, size=cfg.M).astype(np.int32)
    ids, _, lse, dl, _ = _select(h, w_dev, L.DEER_SEL_SOFTMAX, T=0.6, drafts=drafts)
    Hn.check_ids(ids, O.select_argmax(z), z, "M256")
    np.testing.assert_allclose(lse.cpu().numpy(), O.logsumexp(z, float(np.float32(0.6))), atol=3e-4, rtol=0)
    np.testing.assert_allclose(dl.cpu().numpy(), z[np.arange(cfg.M), drafts], atol=1e-3, rtol=0)
