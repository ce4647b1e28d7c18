"""GPU parity of the routed mixture-of-experts MLP (router, regrouping by expert, grouped gate/up + SiLU gate, grouped
down projection, weighted sum) against the oracle."""
import numpy as np
import pytest
import torch

from oracle import deer_oracle as O
from paper_2512_15176_b200 import workload as W
from tests import harness as Hn

pytestmark = pytest.mark.gpu


def _case(seed, M, hid, E, inter, top_k, margin=2e-3):
    """Inputs whose routing is clear of rounding: rows whose top_k-th and (top_k + 1)-th router logits are closer
    than `margin` are re-drawn."""
    wr = W.normal(seed, "wr", (E, hid), hid ** -0.5 * 3.0)
    wgu = W.normal(seed, "wgu", (E, 2 * inter, hid), hid ** -0.5)
    wd = W.normal(seed, "wd", (E, hid, inter), inter ** -0.5)
    x = W.normal(seed, "x0", (M, hid), 1.0)
    for attempt in range(1, 30):
        lg = np.sort(Hn.f64(x) @ Hn.f64(wr).T, axis=1)[:, ::-1]
        gaps = lg[:, :-1] - lg[:, 1:]
        bad = np.flatnonzero(gaps[:, : min(top_k, E - 1)].min(axis=1) < margin)
        if bad.size == 0:
            break
        x2 = W.normal(seed, f"x{attempt}", (M, hid), 1.0)
        x[torch.from_numpy(bad)] = x2[torch.from_numpy(bad)]
    else:
        raise AssertionError("could not clear the routing margins")
    return x, wr, wgu, wd


@pytest.mark.parametrize("M,hid,E,top_k", [(5, 128, 8, 2), (32, 2048, 128, 8), (130, 256, 16, 4), (8, 512, 200, 1)])
def test_router_matches_oracle(M, hid, E, top_k):
    from paper_2512_15176_b200 import binding as L
    x, wr, _, _ = _case(2000 + M, M, hid, E, 64, top_k)
    want_e, want_w = O.moe_route(Hn.f64(x), Hn.f64(wr), top_k)
    e = torch.full((M, top_k), -9, dtype=torch.int32, device="cuda")
    w = torch.full((M, top_k), float("nan"), device="cuda")
    L.deer_moe_route(x.cuda(), wr.cuda(), top_k, e, w)
    torch.cuda.synchronize()
    np.testing.assert_array_equal(e.cpu().numpy(), want_e)
    np.testing.assert_allclose(w.cpu().numpy(), want_w, atol=2e-6, rtol=1e-5)
    _, raw = O.moe_route(Hn.f64(x), Hn.f64(wr), top_k, renormalise=False)
    L.deer_moe_route(x.cuda(), wr.cuda(), top_k, e, w, renormalise=False)
    torch.cuda.synchronize()
    np.testing.assert_allclose(w.cpu().numpy(), raw, atol=2e-6, rtol=1e-5)


@pytest.mark.parametrize("M,hid,E,inter,top_k", [
    (5, 128, 8, 64, 2),            # tiny
    (32, 512, 16, 192, 4),         # a channel tile that is only half full
    (150, 256, 4, 128, 2),         # more than 128 rows for one expert: two row tiles
    (32, 2048, 128, 768, 8),       # the Qwen3-30B-A3B layer's MLP at one sequence's block
    (7, 256, 12, 64, 12),          # every expert chosen by every row
])
def test_moe_mlp_matches_oracle(M, hid, E, inter, top_k):
    from paper_2512_15176_b200 import binding as L
    x, wr, wgu, wd = _case(2100 + M + E, M, hid, E, inter, top_k)
    res = W.normal(2100, "res", (M, hid), 1.0)
    want = O.moe_mlp(Hn.f64(x), Hn.f64(wr), Hn.f64(wgu), Hn.f64(wd), top_k)
    ws = torch.empty(L.deer_moe_workspace_bytes(M, hid, E, inter, top_k), dtype=torch.uint8, device="cuda")
    y = torch.full((M, hid), float("nan"), dtype=torch.bfloat16, device="cuda")
    args = (x.cuda(), wr.cuda(), wgu.cuda(), wd.cuda())
    for residual in (None, res):
        ref = want + (Hn.f64(residual) if residual is not None else 0.0)
        L.deer_moe_mlp(*args, y, top_k, ws, residual=None if residual is None else residual.cuda())
        torch.cuda.synchronize()
        got = Hn.f64(y.cpu())
        assert np.isfinite(got).all()
        err = np.abs(got - ref)
        # three bf16 roundings on the way (activations, expert outputs, result): a few 2^-9 of the values' size
        assert err.max() <= 2.5e-2 * np.abs(ref).max() and err.mean() <= 4e-3 * np.abs(ref).mean(), (err.max(), err.mean())
    # same inputs, same workspace, again: the call leaves nothing behind that the next one trips over
    L.deer_moe_mlp(*args, y, top_k, ws, residual=res.cuda())
    torch.cuda.synchronize()
    assert np.array_equal(Hn.f64(y.cpu()), got)
    # one expert with weight 1 is the dense gated MLP
    if E >= 2:
        y1 = torch.empty_like(y)
        L.deer_moe_mlp(x.cuda(), wr[:1].cuda(), wgu[:1].cuda(), wd[:1].cuda(), y1, 1, ws)
        torch.cuda.synchronize()
        g = O.linear(Hn.f64(x), Hn.f64(wgu[0]))
        dense = O.linear(O.swiglu(g[:, :inter], g[:, inter:]), Hn.f64(wd[0]))
        e1 = np.abs(Hn.f64(y1.cpu()) - dense)
        assert e1.max() <= 2.5e-2 * np.abs(dense).max() and e1.mean() <= 4e-3 * np.abs(dense).mean()
