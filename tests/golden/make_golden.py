"""Writes tests/golden/oracle_tiny.json: the oracle's outputs on one tiny seeded
case.  It calls nothing but ``oracle/`` (inputs come from numpy's own seeded
generator), so the stored values can only ever be the oracle's.  The file is a
drift guard -- a later edit of the oracle that changes any value shows up in
``tests/test_oracle_golden.py`` -- not a pin: the independent pins are the
brute-force, closed-form and invariant tests in ``tests/test_oracle_*.py``.

    python tests/golden/make_golden.py
"""
import json
import os
import sys

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, os.path.dirname(os.path.dirname(HERE)))

from oracle import deer_oracle as O  # noqa: E402


def tiny_case():
    """Inputs of the tiny case: 2 sequences (13 and 0 cached tokens), 2 KV heads x 2 query heads each, head dim 4,
    block of 3 rows, vocabulary 11."""
    g = np.random.Generator(np.random.PCG64(20251215))
    B, k, Hq, Hkv, D, V, hid, P = 2, 3, 4, 2, 4, 11, 6, 4
    seq_len = np.array([13, 0], dtype=np.int32)
    num_pages, max_pages = 8, 5
    page_table = np.full((B, max_pages), -1, dtype=np.int32)
    page_table[0, :4] = [5, 2, 7, 0]
    k_pool = g.standard_normal((num_pages, Hkv, P, D))
    v_pool = g.standard_normal((num_pages, Hkv, P, D))
    q = g.standard_normal((B, k, Hq, D))
    kb = g.standard_normal((B, k, Hkv, D))
    vb = g.standard_normal((B, k, Hkv, D))
    h = g.standard_normal((B * k, hid))
    w = g.standard_normal((V, hid))
    ql = g.standard_normal((B, k, V))
    u = g.uniform(0.05, 0.95, size=(B, k))
    r = g.uniform(0.05, 0.95, size=B)
    drafts = g.integers(0, V, size=(B, k)).astype(np.int32)
    return dict(B=B, k=k, V=V, P=P, seq_len=seq_len, page_table=page_table, k_pool=k_pool, v_pool=v_pool, q=q, kb=kb,
                vb=vb, h=h, w=w, ql=ql, u=u, r=r, drafts=drafts)


def oracle_outputs(c):
    out = {}
    ids = np.arange(c["B"])
    for name, mask in (("attn_causal", 0), ("attn_bidir", 1)):
        out[name] = O.block_attention(c["q"], c["kb"], c["vb"], c["k_pool"], c["v_pool"], c["page_table"], c["seq_len"],
                                      ids, mask, 0.5, page_size=c["P"]).tolist()
    z = O.lm_logits(c["h"], c["w"])
    out["argmax"] = O.select_argmax(z).tolist()
    out["lse_T0.6"] = O.logsumexp(z, 0.6).tolist()
    out["max_logprob"] = O.max_logprob(z).tolist()
    target = O.select_argmax(z).reshape(c["B"], c["k"])
    a, o, n = O.accept_greedy(c["drafts"], target)
    out["greedy"] = [a.tolist(), o.tolist(), n.tolist()]
    a, o, n = O.accept_sample(c["drafts"], z.reshape(c["B"], c["k"], c["V"]), 0.6, c["ql"], c["u"], c["r"])
    out["sample"] = [a.tolist(), o.tolist(), n.tolist()]
    return out


if __name__ == "__main__":
    path = os.path.join(HERE, "oracle_tiny.json")
    with open(path, "w") as f:
        json.dump(oracle_outputs(tiny_case()), f, indent=1)
    print("wrote", path)
