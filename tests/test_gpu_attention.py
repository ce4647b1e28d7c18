"""GPU parity of deer_block_attn against the oracle, element by element."""
import math

import numpy as np
import pytest
import torch

from paper_2512_15176_b200 import workload as W
from tests import harness as Hn

pytestmark = pytest.mark.gpu


def _run(cfg, lengths=None, stress=False, append=False, max_seq_len=None):
    from paper_2512_15176_b200 import binding as L
    st = Hn.draw_state(cfg, lengths, stress)
    q, kb, vb = Hn.draw_block(cfg, 0, stress)
    okv = Hn.oracle_kv(st)
    want = Hn.oracle_attention(cfg, okv, q, kb, vb)
    kv = Hn.gpu_kv(st)
    seq_ids = torch.arange(cfg.B, dtype=torch.int32, device="cuda")
    msl = int(st.lengths.max()) if max_seq_len is None else max_seq_len
    ws = torch.empty(max(16, L.deer_block_attn_workspace_bytes(cfg.B, cfg.k, cfg.Hq, cfg.Hkv, cfg.D, msl)), dtype=torch.uint8, device="cuda")
    out = torch.full((cfg.B, cfg.k, cfg.Hq, cfg.D), float("nan"), dtype=torch.bfloat16, device="cuda")
    if append:
        L.deer_kv_reserve(kv, seq_ids, cfg.k)
        assert okv.reserve(np.arange(cfg.B), cfg.k)
        okv.append(np.arange(cfg.B), Hn.f64(kb).astype(np.float32), Hn.f64(vb).astype(np.float32))
    L.deer_block_attn(kv, seq_ids, q.cuda(), kb.cuda(), vb.cuda(), out, cfg.mask, append, 1.0 / math.sqrt(cfg.D), msl, ws)
    torch.cuda.synchronize()
    assert L.deer_kv_status(kv) == 0
    Hn.check_attention(out.cpu(), want, cfg.name)
    if append:
        # rows written at n .. n+k-1: make them visible by committing all k on both sides
        keep = torch.full((cfg.B,), cfg.k, dtype=torch.int32, device="cuda")
        L.deer_kv_commit(kv, seq_ids, keep, cfg.k)
        okv.commit(np.arange(cfg.B), [cfg.k] * cfg.B)
        torch.cuda.synchronize()
        Hn.kv_state_equal(kv, okv, cfg.name)
        Hn.kv_contents_equal(kv, okv, label=cfg.name)
    return out


@pytest.mark.parametrize("stress", [False, True])
def test_tiny_config(stress):
    _run(W.config(0), stress=stress, append=True)


@pytest.mark.parametrize("mask", [W.MASK_CAUSAL, W.MASK_BIDIR])
@pytest.mark.parametrize("B,k,Hq,Hkv,D,lens", [
    (3, 8, 8, 2, 64, [0, 1, 255]),            # empty prefix, single token, ragged tail
    (2, 1, 4, 4, 128, [16, 700]),             # k = 1, G = 1
    (2, 32, 32, 8, 128, [1500, 777]),         # several chunks, 128 rows per KV head
    (2, 32, 32, 4, 128, [300, 1031]),         # 256 rows per KV head -> two row tiles
    (1, 5, 6, 2, 64, [97]),                   # odd k, G = 3
    (4, 16, 16, 8, 128, [64, 65, 63, 4096]),  # page/tile boundaries
    (2, 7, 6, 2, 128, [130, 1]),              # G = 3: 21 rows on the 128 lanes
    (2, 32, 20, 4, 128, [200, 999]),          # G = 5: 25 block rows per row tile, two row tiles
    (3, 32, 32, 4, 128, [5000, 64, 700]),     # G = 8, very unequal lengths: shares cross unit and sequence boundaries
])
def test_shapes_and_edges(mask, B, k, Hq, Hkv, D, lens):
    cfg = W.StepConfig("edge", B, Hq, Hkv, D, k, 64, 64, (min(lens), max(lens)), mask=mask, seed=77)
    _run(cfg, lengths=lens, stress=True, append=(mask == W.MASK_CAUSAL))


def test_many_short_sequences():
    """Hundreds of sequences of 0..150 tokens (many of them empty): every thread
    block's share of the work holds dozens of (sequence, KV head) pieces, more
    than its piece list takes at once."""
    B = 900
    lens = W.rng(81, "lens").integers(0, 3, size=B) * W.rng(81, "lens2").integers(0, 76, size=B)
    cfg = W.StepConfig("short", B, 8, 8, 128, 2, 64, 64, (int(lens.min()), int(lens.max())), seed=81)
    _run(cfg, lengths=lens.tolist(), stress=True, append=True)


def test_one_unusable_sequence_does_not_disturb_the_others():
    """A sequence longer than max_seq_len is skipped and reported; its
    neighbours in the batch still get their exact results."""
    from paper_2512_15176_b200 import binding as L
    lens = [300, 900, 40]
    cfg = W.StepConfig("skip", 3, 8, 2, 128, 8, 64, 64, (40, 900), seed=82)
    st = Hn.draw_state(cfg, lens, True)
    q, kb, vb = Hn.draw_block(cfg, 0, True)
    want = Hn.oracle_attention(cfg, Hn.oracle_kv(st), q, kb, vb)
    kv = Hn.gpu_kv(st)
    seq_ids = torch.arange(3, dtype=torch.int32, device="cuda")
    ws = torch.empty(L.deer_block_attn_workspace_bytes(3, 8, 8, 2, 128, 512), dtype=torch.uint8, device="cuda")
    out = torch.zeros(3, 8, 8, 128, dtype=torch.bfloat16, device="cuda")
    L.deer_block_attn(kv, seq_ids, q.cuda(), kb.cuda(), vb.cuda(), out, 0, 0, 1.0 / math.sqrt(128), 512, ws)
    assert L.deer_kv_status(kv) == L.DEER_ERR_INVALID_ARG
    got = out.cpu()
    Hn.check_attention(got[[0, 2]], want[[0, 2]], "neighbours of a skipped sequence")


def test_split_is_invisible():
    """The same inputs with different context splits (steered by max_seq_len)
    give the same result within rounding."""
    cfg = W.StepConfig("split", 1, 8, 2, 128, 8, 64, 64, (3000, 3000), seed=78)
    a = _run(cfg, stress=True, max_seq_len=3000)
    b = _run(cfg, stress=True, max_seq_len=60000)
    assert (a.float() - b.float()).abs().max() < 1e-2


def test_sequence_longer_than_bound_is_reported():
    from paper_2512_15176_b200 import binding as L
    cfg = W.StepConfig("bound", 1, 4, 2, 64, 4, 64, 64, (100, 100), seed=79)
    st = Hn.draw_state(cfg)
    q, kb, vb = Hn.draw_block(cfg)
    kv = Hn.gpu_kv(st)
    seq_ids = torch.zeros(1, dtype=torch.int32, device="cuda")
    ws = torch.empty(L.deer_block_attn_workspace_bytes(1, 4, 4, 2, 64, 50), dtype=torch.uint8, device="cuda")
    out = torch.zeros(1, 4, 4, 64, dtype=torch.bfloat16, device="cuda")
    L.deer_block_attn(kv, seq_ids, q.cuda(), kb.cuda(), vb.cuda(), out, 0, 0, 0.125, 50, ws)
    assert L.deer_kv_status(kv) == L.DEER_ERR_INVALID_ARG
    assert L.deer_kv_status(kv) == 0          # reading clears it


@pytest.mark.parametrize("gain", [8.0, 40.0])
def test_dominant_keys_far_above_the_first_tile(gain):
    """Keys planted late in the context whose scores lie hundreds of octaves above everything seen before them: the
    exponentials of a segment are taken against its first tile's maximum, so such a tile must raise the reference
    point (at gain 8 the exponentials are huge but finite, at gain 40 they overflow) and the output must still be
    the softmax by definition -- essentially the planted key's value row."""
    from paper_2512_15176_b200 import binding as L
    cfg = W.StepConfig("dominant", 2, 8, 2, 128, 8, 64, 64, (0, 0), seed=83)
    lens = [900, 3000]
    st = Hn.draw_state(cfg, lens, True)
    q, kb, vb = Hn.draw_block(cfg, 0, True)
    G = cfg.Hq // cfg.Hkv
    planted = [(0, 700, 3, 5), (1, 150, 0, 0), (1, 2999, 7, 6), (1, 1600, 2, 3)]     # (sequence, token, block row, query head)
    for b, t, i, h in planted:
        pg = int(st.layout.page_table[b, t // 16])
        st.k_pool[pg, h // G, t % 16] = (q[b, i, h].float() * gain).to(torch.bfloat16)
    okv = Hn.oracle_kv(st)
    want = Hn.oracle_attention(cfg, okv, q, kb, vb)
    kv = Hn.gpu_kv(st)
    seq_ids = torch.arange(cfg.B, dtype=torch.int32, device="cuda")
    msl = max(lens)
    ws = torch.empty(L.deer_block_attn_workspace_bytes(cfg.B, cfg.k, cfg.Hq, cfg.Hkv, cfg.D, msl), dtype=torch.uint8, device="cuda")
    out = torch.full((cfg.B, cfg.k, cfg.Hq, cfg.D), float("nan"), dtype=torch.bfloat16, device="cuda")
    L.deer_block_attn(kv, seq_ids, q.cuda(), kb.cuda(), vb.cuda(), out, cfg.mask, 0, 1.0 / math.sqrt(cfg.D), msl, ws)
    torch.cuda.synchronize()
    assert L.deer_kv_status(kv) == 0
    Hn.check_attention(out.cpu(), want, f"dominant keys, gain {gain}")
    for b, t, i, h in planted:
        pg = int(st.layout.page_table[b, t // 16])
        v_row = st.v_pool[pg, h // G, t % 16].float()
        assert (out[b, i, h].cpu().float() - v_row).abs().max() < 2e-2          # that row's output is the planted key's value
