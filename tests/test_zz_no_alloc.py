"""deer_lmhead_select_static: the LM-head call for callers that cannot allocate.

A host that may not call the CUDA allocator where it uses the library (a
serving loop with a sealed memory pool, a plug-in handed only its inputs and
outputs) cannot supply the workspace deer_lmhead_select wants.  The static
variant keeps that scratch in a fixed array inside the library.  This test
calls it through the C ABI twice in a row -- the second call finds the first
call's leftovers in the shared array -- and checks every output against the
workspace-based entry point and against the CPU oracle, and that the device's
free memory does not move across a call.  It is collected last on purpose."""
import numpy as np
import pytest
import torch

from oracle import deer_oracle as O
from paper_2512_15176_b200 import workload as W

pytestmark = pytest.mark.gpu


def _outputs(M, V, dev):
    return (torch.full((M,), -5, dtype=torch.int32, device=dev), torch.full((M,), float("nan"), device=dev),
            torch.full((M,), float("nan"), device=dev), torch.full((M, V), float("nan"), device=dev))


def test_static_scratch_matches_workspace_entry_point_twice():
    from paper_2512_15176_b200 import binding as L
    dev = "cuda"
    hid, V = 512, 4096
    assert L.deer_lmhead_static_max_rows() == 256
    w = W.normal(4242, "w", (V, hid), 0.05).to(dev)
    # every output tensor is allocated BEFORE the calls under test; the calls themselves get no workspace
    for call, (M, mode, T) in enumerate([(256, L.DEER_SEL_SOFTMAX, 0.6), (40, L.DEER_SEL_SOFTMAX, 1.0)]):
        h = W.normal(4242, f"h{call}", (M, hid), 1.0).to(dev)
        drafts = torch.from_numpy(W.rng(4242, f"d{call}").integers(0, V, size=M).astype(np.int32)).to(dev)
        ids_a, lse_a, dl_a, z_a = _outputs(M, V, dev)
        ids_b, lse_b, dl_b, z_b = _outputs(M, V, dev)
        ws = torch.empty(L.deer_lmhead_workspace_bytes(M, hid, V), dtype=torch.uint8, device=dev)
        L.deer_lmhead_select(h, w, mode, T, drafts, ids_a, None, lse_a, dl_a, z_a, ws)
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        reserved_before = torch.cuda.memory_reserved()
        L.deer_lmhead_select_static(h, w, mode, T, drafts, ids_b, None, lse_b, dl_b, z_b)
        torch.cuda.synchronize()
        if call > 0:       # the very first call on a device resolves the array's address; later ones touch no allocator
            assert torch.cuda.mem_get_info()[0] == free_before and torch.cuda.memory_reserved() == reserved_before
        assert torch.equal(ids_a, ids_b)
        # and against the oracle on the same inputs
        z64 = O.lm_logits(h.cpu().to(torch.float64).numpy(), w.cpu().to(torch.float64).numpy())
        want_ids = O.select_argmax(z64)
        got_ids = ids_b.cpu().numpy()
        differ = np.flatnonzero(got_ids != want_ids)
        assert (O.top2_gap(z64[differ]) < 1e-3).all()
        np.testing.assert_allclose(lse_b.cpu().numpy(), O.logsumexp(z64, float(np.float32(T))), atol=3e-4, rtol=0)
        np.testing.assert_allclose(dl_b.cpu().numpy(), z64[np.arange(M), drafts.cpu().numpy()], atol=1e-3, rtol=0)
        np.testing.assert_allclose(z_b.cpu().numpy(), z64, atol=1e-3, rtol=0)
        assert not torch.isnan(lse_b).any() and not torch.isnan(z_b).any()
        np.testing.assert_allclose(lse_b.cpu().numpy(), lse_a.cpu().numpy(), atol=3e-4, rtol=0)
        np.testing.assert_allclose(dl_b.cpu().numpy(), dl_a.cpu().numpy(), atol=1e-3, rtol=0)
        np.testing.assert_allclose(z_b.cpu().numpy(), z_a.cpu().numpy(), atol=1e-3, rtol=0)
    # argmax + log-probability mode on the same shared array, a third call
    M = 8
    h = W.normal(4242, "h2", (M, hid), 1.0).to(dev)
    ids_a, mlp_a, _, _ = _outputs(M, V, dev)
    ids_b, mlp_b, _, _ = _outputs(M, V, dev)
    ws = torch.empty(L.deer_lmhead_workspace_bytes(M, hid, V), dtype=torch.uint8, device=dev)
    L.deer_lmhead_select(h, w, L.DEER_SEL_ARGMAX_LOGPROB, 1.0, None, ids_a, mlp_a, None, None, None, ws)
    L.deer_lmhead_select_static(h, w, L.DEER_SEL_ARGMAX_LOGPROB, 1.0, None, ids_b, mlp_b, None, None, None)
    torch.cuda.synchronize()
    assert torch.equal(ids_a, ids_b)
    np.testing.assert_allclose(mlp_b.cpu().numpy(), mlp_a.cpu().numpy(), atol=2e-4, rtol=0)
    z64 = O.lm_logits(h.cpu().to(torch.float64).numpy(), w.cpu().to(torch.float64).numpy())
    np.testing.assert_allclose(mlp_b.cpu().numpy(), O.max_logprob(z64), atol=2e-4, rtol=0)


def test_static_scratch_first_call_inside_a_capture_is_refused_or_already_resolved():
    """On a device whose array address is still unknown, a call on a capturing stream must refuse (the look-up is not
    a capturable operation); once an earlier call has resolved it -- the case when the test above ran first -- the
    same call is simply recorded.  Either way the capture survives."""
    from paper_2512_15176_b200 import binding as L
    dev = "cuda"
    M, hid, V = 8, 64, 128
    h = W.normal(4243, "h", (M, hid), 1.0).to(dev)
    w = W.normal(4243, "w", (V, hid), 0.05).to(dev)
    ids = torch.full((M,), -5, dtype=torch.int32, device=dev)
    st = torch.cuda.Stream()
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    refused = False
    with torch.cuda.graph(g, stream=st):
        try:
            L.deer_lmhead_select_static(h, w, L.DEER_SEL_ARGMAX, 1.0, None, ids, None, None, None, None)
        except L.DeerError as e:
            assert e.code == L.DEER_ERR_UNSUPPORTED
            refused = True
    if not refused:
        g.replay()
        torch.cuda.synchronize()
        z64 = O.lm_logits(h.cpu().to(torch.float64).numpy(), w.cpu().to(torch.float64).numpy())
        assert (ids.cpu().numpy() == O.select_argmax(z64)).all()


def test_static_scratch_rejects_more_rows_than_it_holds():
    from paper_2512_15176_b200 import binding as L
    dev = "cuda"
    M, hid, V = 257, 64, 128
    h = torch.zeros(M, hid, dtype=torch.bfloat16, device=dev)
    w = torch.zeros(V, hid, dtype=torch.bfloat16, device=dev)
    ids = torch.zeros(M, dtype=torch.int32, device=dev)
    with pytest.raises(L.DeerError) as e:
        L.deer_lmhead_select_static(h, w, L.DEER_SEL_ARGMAX, 1.0, None, ids, None, None, None, None)
    assert e.value.code == L.DEER_ERR_UNSUPPORTED and "256" in str(e.value)
