"""Algorithm 1's outer loop on the GPU (verify step + deer_emit + commit, several
passes without a host round trip) against the oracle's loop on the same
seeded inputs: output tokens, their counts, the finished flags and the whole
KV state, bit for bit."""
import numpy as np
import pytest
import torch

from oracle import deer_oracle as O
from paper_2512_15176_b200 import workload as W
from tests import harness as Hn

pytestmark = pytest.mark.gpu


def _emit_only(B, k, max_new, eos_id, passes, seed, pending=False):
    """deer_emit alone on random accept results."""
    from paper_2512_15176_b200 import binding as L
    rng = W.rng(seed, "emit")
    st = O.DecodeState(B, max_new)
    dev = "cuda"
    tokens = torch.full((B, max_new), -1, dtype=torch.int32, device=dev)
    n_tokens = torch.zeros(B, dtype=torch.int32, device=dev)
    finished = torch.zeros(B, dtype=torch.int32, device=dev)
    keep = torch.full((B,), -9, dtype=torch.int32, device=dev)
    for _ in range(passes):
        target = rng.integers(0, 12, size=(B, k)).astype(np.int32)
        draft = np.where(rng.random((B, k)) < 0.7, target, (target + 1) % 12).astype(np.int32)
        a, out, n = O.accept_greedy(draft, target, eos_id, bonus=pending)
        want_keep = st.emit(a, out, n, eos_id, pending=pending)
        L.deer_emit(torch.from_numpy(a).to(dev), torch.from_numpy(out).to(dev), torch.from_numpy(n).to(dev), eos_id, tokens,
                    n_tokens, finished, keep, L.DEER_EMIT_PENDING if pending else 0)
        torch.cuda.synchronize()
        np.testing.assert_array_equal(keep.cpu().numpy(), want_keep)
        np.testing.assert_array_equal(tokens.cpu().numpy(), st.tokens)
        np.testing.assert_array_equal(n_tokens.cpu().numpy(), st.n_tokens)
        np.testing.assert_array_equal(finished.cpu().numpy(), st.finished)
    return st


@pytest.mark.parametrize("B,k,max_new,eos_id", [(1, 1, 3, -1), (7, 8, 20, 3), (300, 32, 50, 5), (5, 4, 0, -1)])
def test_emit_bit_exact(B, k, max_new, eos_id):
    st = _emit_only(B, k, max_new, eos_id, passes=8, seed=900 + B)
    if max_new > 0 and eos_id < 0:
        assert st.finished.all()                 # 8 passes of >= 1 token fill 3 new tokens


@pytest.mark.parametrize("B,k,max_new,eos_id", [(1, 1, 3, -1), (9, 8, 20, 3), (200, 32, 64, 5)])
def test_emit_pending_bit_exact(B, k, max_new, eos_id):
    _emit_only(B, k, max_new, eos_id, passes=8, seed=950 + B, pending=True)


@pytest.mark.parametrize("pending", [False, True])
def test_greedy_decode_loop_matches_oracle(pending):
    """Six passes of the tiny verifier shape, four ragged sequences: one runs into
    the length limit, the planted EOS ends others early, the rest keep going.
    pending: k-1 drafts behind the pending token, one more token from the last row,
    the pending token's row kept in the cache."""
    from paper_2512_15176_b200 import binding as L
    from paper_2512_15176_b200.runner import DecodeLoop, VerifyStep
    passes, max_new = 6, 28                 # sequences 0 and 3 fill up, 2 meets the EOS, 1 keeps going
    cfg = W.StepConfig("loop", 4, 8, 2, 128, 8, 256, 2048, (40, 300), seed=910, growth=passes * 8)
    st = Hn.draw_state(cfg, None, True)
    okv, kv = Hn.oracle_kv(st), Hn.gpu_kv(st)
    w = W.lm_head(cfg)
    w64 = Hn.f64(w)
    vs = VerifyStep(cfg, kv, w.cuda(), int(st.lengths.max()) + passes * cfg.k, store_logits=False)
    ids = np.arange(cfg.B)
    ost = None
    inputs = []
    # the EOS id is chosen from the first pass's targets so that it really occurs
    for step in range(passes):
        q, kb, vb = Hn.draw_block(cfg, step, True)
        h, z, _ = Hn.draw_hidden_with_margin(cfg, w64, step)
        target = O.select_argmax(z).reshape(cfg.B, cfg.k)
        drafts = W.plant_drafts(cfg, target, W.planted_prefix_lengths(cfg.with_(prefix_law="uniform"), step), step)
        inputs.append((q, kb, vb, h, target, drafts))
    eos_id = int(inputs[1][4][2, 0])             # sequence 2 emits it in the second pass at the latest
    ost = O.DecodeState(cfg.B, max_new)
    loop = DecodeLoop(vs, eos_id, max_new, pending=pending)
    for step, (q, kb, vb, h, target, drafts) in enumerate(inputs):
        assert okv.reserve(ids, cfg.k)
        okv.append(ids, Hn.f64(kb).astype(np.float32), Hn.f64(vb).astype(np.float32))
        a, out, n = O.accept_greedy(drafts, target, eos_id, bonus=pending)
        okv.commit(ids, ost.emit(a, out, n, eos_id, pending=pending))
        vs.load(q, kb, vb, h, drafts)
        loop.one_pass()                          # no synchronisation between the passes
    torch.cuda.synchronize()
    assert L.deer_kv_status(kv) == 0
    np.testing.assert_array_equal(loop.tokens.cpu().numpy(), ost.tokens)
    np.testing.assert_array_equal(loop.n_tokens.cpu().numpy(), ost.n_tokens)
    np.testing.assert_array_equal(loop.finished.cpu().numpy(), ost.finished)
    assert ost.finished.any() and not ost.finished.all()      # the case exercises both outcomes
    Hn.kv_state_equal(kv, okv, "decode loop")
    Hn.kv_contents_equal(kv, okv, label="decode loop")
