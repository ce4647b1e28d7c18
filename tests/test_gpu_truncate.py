"""GPU parity of deer_truncate (one threshold and one log-sum-exp per row) and of the acceptance rule on the
truncated verifier distribution, against the oracle."""
import numpy as np
import pytest
import torch

from oracle import deer_oracle as O
from paper_2512_15176_b200 import workload as W
from tests import harness as Hn

pytestmark = pytest.mark.gpu


MASS_TOL = 2e-6      # the kernel sums fp32 probabilities (2 ulp exp2, fp32 bin sums): its running mass is good to ~3e-7


def _pick_top_p(z32, T, top_k, top_p):
    """A top_p near the requested one whose nucleus edge is clear of rounding in every row, if there is one (with
    150 000 tokens a single token's mass is as small as the tolerance, so there may be none)."""
    for step in range(40):
        cand = top_p + step * 3.1e-4
        if cand >= 1.0 or Hn.nucleus_margin_ok(z32, T, top_k, cand, margin=MASS_TOL):
            return cand, True
    return top_p, False


def _check_level_set(row, T, top_k, top_p, tau_got, label):
    """The threshold is right if the set it keeps is an upper level set that satisfies the definition up to the
    mass tolerance: (top-k) it is the top-k set cut further only by the nucleus; (nucleus) its mass reaches top_p
    and would not without its least likely tie group."""
    p = O.softmax_f64(row, T)
    keep = row >= tau_got
    assert keep.any(), label
    pk, kk = O.truncate_distribution(p, top_k, 1.0)             # after top-k, renormalised
    assert not (keep & ~kk).any(), f"{label}: keeps tokens outside the top-k set"
    if top_p >= 1.0:
        assert (keep == kk).all(), f"{label}: top-k set differs"
        return
    mass = pk[keep].sum()
    least = pk[keep].min()
    without = mass - pk[keep & (pk == least)].sum()
    assert mass >= top_p - MASS_TOL, f"{label}: kept mass {mass} below top_p {top_p}"
    assert without < top_p + MASS_TOL, f"{label}: the set is not minimal ({without} already reaches {top_p})"


def _expected(z32, T, top_k, top_p):
    tau, lse_t = [], []
    for row in z32:
        p = O.softmax_f64(row, T)
        _, keep = O.truncate_distribution(p, top_k, top_p)
        tau.append(row[keep].min() if not keep.all() else -np.inf)
        zt = row[keep].astype(np.float64) / T
        lse_t.append(zt.max() + np.log(np.exp(zt - zt.max()).sum()))
    return np.array(tau, dtype=np.float32), np.array(lse_t)


def _run_truncate(z32, T, top_k, top_p):
    from paper_2512_15176_b200 import binding as L
    M, V = z32.shape
    dev = "cuda"
    lse = torch.from_numpy(O.logsumexp(z32.astype(np.float64), T).astype(np.float32)).to(dev)
    tau = torch.full((M,), float("nan"), device=dev)
    lse_t = torch.full((M,), float("nan"), device=dev)
    L.deer_truncate(torch.from_numpy(z32).to(dev), lse, T, top_k, top_p, tau, lse_t)
    torch.cuda.synchronize()
    return tau.cpu().numpy(), lse_t.cpu().numpy()


@pytest.mark.parametrize("M,V", [(8, 1000), (16, 4099), (5, 151936), (300, 2048)])
@pytest.mark.parametrize("top_k,top_p", [(50, 1.0), (0, 0.9), (20, 0.8), (1, 1.0), (0, 0.35), (700, 0.97)])
def test_truncate_matches_oracle(M, V, top_k, top_p):
    T = float(np.float32(0.6))
    z32 = W.normal(1200 + V, "z", (M, V), 1.3, dtype=torch.float32).numpy()
    top_p, clear = _pick_top_p(z32, T, top_k, top_p)
    want_tau, want_lse = _expected(z32, T, top_k, top_p)
    got_tau, got_lse = _run_truncate(z32, T, top_k, top_p)
    for m in range(M):
        _check_level_set(z32[m], T, top_k, top_p, got_tau[m], f"row {m}")
        zt = z32[m][z32[m] >= got_tau[m]].astype(np.float64) / T
        assert abs(got_lse[m] - (zt.max() + np.log(np.exp(zt - zt.max()).sum()))) < 3e-4
    if clear:
        # with the nucleus edge clear of rounding (always so for top-k alone) the threshold is the oracle's, bit for bit
        np.testing.assert_array_equal(got_tau, want_tau)
        np.testing.assert_allclose(got_lse, want_lse, atol=3e-4, rtol=0)


def test_truncate_with_heavy_ties():
    """Logits on a grid of a few dozen values: thousands of tokens per tie group, more than the exact stage holds at
    once, so the bins are refined by bit pattern; whole tie groups must stay or go."""
    T = float(np.float32(1.0))
    M, V = 6, 20000
    z = W.normal(1300, "z", (M, V), 1.5, dtype=torch.float32).numpy()
    z32 = (np.round(z * 4) / 4).astype(np.float32)
    z32[2] = 0.5                                            # one single value in the whole row
    z32[3, :] = np.where(np.arange(V) % 2 == 0, -0.0, 0.0)  # both zeros: one tie group
    for top_k, top_p in [(100, 1.0), (0, 0.6), (5000, 0.9)]:
        if top_p < 1.0:
            top_p, clear = _pick_top_p(z32[[0, 1, 4, 5]], T, top_k, top_p)
            assert clear                                        # tie groups of thousands of tokens: wide margins exist
        want_tau, want_lse = _expected(z32, T, top_k, top_p)
        got_tau, got_lse = _run_truncate(z32, T, top_k, top_p)
        for m in range(M):
            kept = z32[m] >= want_tau[m]
            assert ((z32[m] >= got_tau[m]) == kept).all(), (top_k, top_p, m, got_tau[m], want_tau[m])
        np.testing.assert_allclose(got_lse, want_lse, atol=3e-4, rtol=0)


def _peaked_rows(seed, M, V, slope):
    """Rows shaped like a language model's: logit = -slope * log(rank) under a random permutation, plus noise."""
    g = np.random.default_rng(seed)
    z = np.empty((M, V), dtype=np.float32)
    base = (-slope * np.log(np.arange(1, V + 1))).astype(np.float32)
    for m in range(M):
        z[m, g.permutation(V)] = base
    return z + W.normal(seed, "noise", (M, V), 0.3, dtype=torch.float32).numpy()


def test_truncate_peaked_rows():
    """Peaked rows of full vocabulary length: the nucleus is a few tokens to a few hundred (and, at 0.9999, far more
    than any short candidate list holds)."""
    T = float(np.float32(0.8))
    z32 = _peaked_rows(1360, 6, 151936, 1.1)
    for top_k, top_p in [(0, 0.9), (0, 0.5), (40, 0.95), (0, 0.9999), (100, 1.0)]:
        clear = True
        if top_p < 1.0:
            top_p, clear = _pick_top_p(z32, T, top_k, top_p)
        want_tau, want_lse = _expected(z32, T, top_k, top_p)
        got_tau, got_lse = _run_truncate(z32, T, top_k, top_p)
        for m in range(z32.shape[0]):
            _check_level_set(z32[m], T, top_k, top_p, got_tau[m], f"row {m} top_k {top_k} top_p {top_p}")
        if clear:
            np.testing.assert_array_equal(got_tau, want_tau)
            np.testing.assert_allclose(got_lse, want_lse, atol=3e-4, rtol=0)


def test_truncate_on_rows_that_mislead_a_sample():
    """Long rows whose largest logits sit exactly on, or exactly off, a regular stride of positions, or fill a tie
    group larger than any candidate list: a cut placed from a strided sample of the row is then far too high or
    far too low, and the result must still be the oracle's (the kernel may use a sample only to place a cut)."""
    T = float(np.float32(0.8))
    V = 151936
    base = W.normal(1350, "z", (7, V), 1.0, dtype=torch.float32).numpy() - np.float32(6.0)
    pos = np.arange(V)
    rows = []
    for stride4 in (9, 8, 37):                                  # float4 strides a sampler might use
        on = (pos // 4) % stride4 == 0
        z = base[len(rows)].copy()                              # high values exactly on the stride
        z[on] += np.float32(9.0)
        rows.append(z)
    z = base[3].copy()                                          # 40 high values on the stride 9, nothing else near
    z[(np.arange(40) * 9 * 4 * 50)] = np.float32(8.0) + np.arange(40, dtype=np.float32) / 64
    rows.append(z)
    z = base[4].copy()                                          # 3000 high values, all off the stride 9
    off = pos[(pos // 4) % 9 == 4][:3000]
    z[off] = np.float32(7.0) + (np.arange(3000) % 17).astype(np.float32) / 32
    rows.append(z)
    z = base[5].copy()                                          # a tie group of 5000 at the top
    z[:5000] = np.float32(6.5)
    rows.append(z)
    z = base[6].copy()                                          # high values in 128-byte runs, 512 runs per row
    z[(pos // 4) % (V // 4 // 512) < 8] += np.float32(9.0)
    rows.append(z)
    z32 = np.stack(rows).astype(np.float32)
    for top_k, top_p in [(50, 1.0), (20, 0.9), (300, 0.5), (1, 1.0)]:
        clear = True
        if top_p < 1.0:
            top_p, clear = _pick_top_p(z32, T, top_k, top_p)
        want_tau, want_lse = _expected(z32, T, top_k, top_p)
        got_tau, got_lse = _run_truncate(z32, T, top_k, top_p)
        for m in range(len(rows)):
            _check_level_set(z32[m], T, top_k, top_p, got_tau[m], f"row {m} top_k {top_k} top_p {top_p}")
        if clear:
            np.testing.assert_array_equal(got_tau, want_tau)
            np.testing.assert_allclose(got_lse, want_lse, atol=3e-4, rtol=0)


def _sample_truncated(cfg, zt32, ql, drafts, u, r, top_k, top_p, from_oracle, eos=-1, bonus=False, tau_out=None):
    """deer_accept_truncated on given fp32 logits.  from_oracle: the thresholds and truncated log-sum-exps come from the
    oracle (the acceptance in isolation); otherwise from deer_truncate (the two calls chained; tau_out receives its
    thresholds)."""
    from paper_2512_15176_b200 import binding as L
    B, k, V = cfg.B, cfg.k, cfg.V
    dev = "cuda"
    T = float(np.float32(cfg.temperature))
    flat = zt32.reshape(B * k, V)
    zt_dev = torch.from_numpy(zt32).to(dev)
    if from_oracle:
        tau_np, lse_np = _expected(flat, T, top_k, top_p)
        tau = torch.from_numpy(tau_np).to(dev)
        lse_t = torch.from_numpy(lse_np.astype(np.float32)).to(dev)
    else:
        lse = torch.from_numpy(O.logsumexp(flat.astype(np.float64), T).astype(np.float32)).to(dev)
        tau = torch.empty(B * k, device=dev)
        lse_t = torch.empty(B * k, device=dev)
        L.deer_truncate(zt_dev, lse, T, top_k, top_p, tau, lse_t)
        if tau_out is not None:
            torch.cuda.synchronize()
            tau_out.append(tau.cpu().numpy().reshape(B, k))
    zd = torch.from_numpy(np.take_along_axis(zt32, drafts[..., None].astype(np.int64), axis=2)[..., 0].astype(np.float32)).to(dev)
    a = torch.full((B,), -9, dtype=torch.int32, device=dev)
    o = torch.full((B, k), -9, dtype=torch.int32, device=dev)
    n = torch.full((B,), -9, dtype=torch.int32, device=dev)
    ws = torch.empty(L.deer_accept_workspace_bytes(L.DEER_ACC_SAMPLE, B, k, V), dtype=torch.uint8, device=dev)
    L.deer_accept_truncated(L.DEER_ACC_SAMPLE | (L.DEER_ACC_BONUS if bonus else 0), B, k, V, torch.as_tensor(drafts, device=dev),
                            None, zt_dev, lse_t, zd, tau, cfg.temperature, ql.to(dev), u.to(dev), r.to(dev), eos, a, o, n, ws)
    torch.cuda.synchronize()
    return a.cpu().numpy(), o.cpu().numpy(), n.cpu().numpy()


@pytest.mark.parametrize("B,k,V,T,top_k,top_p", [(6, 8, 1000, 0.6, 40, 1.0), (16, 16, 4099, 0.6, 0, 0.9),
                                                  (3, 5, 151936, 0.6, 64, 0.95), (12, 4, 300, 1.0, 1, 1.0)])
def test_sampling_on_the_truncated_distribution_bit_exact(B, k, V, T, top_k, top_p):
    cfg = W.StepConfig("st", B, 4, 2, 64, k, 64, V, (0, 0), mode="sample", temperature=T, seed=1400 + V)
    ql0 = W.draft_logits(cfg)
    zt32 = (ql0 + W.normal(cfg.seed, "zt", (B, k, V), 0.5, dtype=torch.float32)).numpy() * np.float32(T)
    Tf = float(np.float32(T))
    top_p, clear = _pick_top_p(zt32.reshape(B * k, V), Tf, top_k, top_p)
    ql, drafts, u, r, _ = Hn.sampling_inputs(cfg, zt32, top_k=top_k, top_p=top_p)
    want = O.accept_sample(drafts, zt32, Tf, ql.numpy(), u.numpy(), r.numpy(), top_k=top_k, top_p=top_p)
    # (1) the acceptance alone, thresholds from the oracle: bit-exact
    got = _sample_truncated(cfg, zt32, ql, drafts, u, r, top_k, top_p, True)
    for g, w_, name in zip(got, want, ("accept_len", "out_ids", "n_out")):
        np.testing.assert_array_equal(g, w_, err_msg=f"{name} (thresholds from the oracle)")
    # (2) chained behind deer_truncate: its thresholds are valid level sets (checked row by row), and the result is
    #     the oracle's on exactly the sets they keep (the oracle sees the dropped logits as -1e30) -- the same as (1)
    #     whenever the nucleus edges are clear of rounding
    taus = []
    got = _sample_truncated(cfg, zt32, ql, drafts, u, r, top_k, top_p, False, tau_out=taus)
    tau = taus[0]
    for b in range(B):
        for i in range(k):
            _check_level_set(zt32[b, i], Tf, top_k, top_p, tau[b, i], f"row {b},{i}")
    z_cut = np.where(zt32 >= tau[..., None], zt32, np.float32(-1e30))
    if clear:
        want2 = want
    else:
        ql, drafts, u, r, _ = Hn.sampling_inputs(cfg, z_cut)
        want2 = O.accept_sample(drafts, z_cut, Tf, ql.numpy(), u.numpy(), r.numpy())
        got = _sample_truncated(cfg, zt32, ql, drafts, u, r, top_k, top_p, False)
    for g, w_, name in zip(got, want2, ("accept_len", "out_ids", "n_out")):
        np.testing.assert_array_equal(g, w_, err_msg=f"{name} (thresholds from the library)")
    # every emitted correction lies inside the kept set
    for b in range(B):
        i = int(want[0][b])
        if i < k:
            _, keep = O.truncate_distribution(O.softmax_f64(zt32[b, i], Tf), top_k, top_p)
            assert keep[want[1][b, i]]
    if top_k == 1:
        # one-hot p': the greedy rule
        tgt = zt32.argmax(axis=2).astype(np.int32)
        ag, og, ng = O.accept_greedy(drafts, tgt)
        np.testing.assert_array_equal(want[0], ag)
        np.testing.assert_array_equal(want[1], og)
    # with the extra row and an EOS (thresholds from the oracle)
    ql, drafts, u, r, _ = Hn.sampling_inputs(cfg, zt32, bonus=True, top_k=top_k, top_p=top_p)
    eos = int(want[1][0, 0])
    want = O.accept_sample(drafts, zt32, Tf, ql.numpy(), u.numpy(), r.numpy(), eos, True, top_k, top_p)
    got = _sample_truncated(cfg, zt32, ql, drafts, u, r, top_k, top_p, True, eos, True)
    for g, w_, name in zip(got, want, ("accept_len", "out_ids", "n_out")):
        np.testing.assert_array_equal(g, w_, err_msg=name + " (extra row, EOS)")
