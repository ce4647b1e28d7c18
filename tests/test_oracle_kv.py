"""Pins for the oracle's paged-KV manager: a dense shadow cache, page
conservation, and exact reversibility of reserve/commit."""
import numpy as np

from oracle import deer_oracle as O
from paper_2512_15176_b200 import workload as W


def _state(cfg, lengths):
    lay = W.kv_layout(cfg, lengths)
    r = np.random.default_rng(1)
    kp = r.normal(size=(lay.num_pages, cfg.Hkv, 16, cfg.D)).astype(np.float32)
    vp = r.normal(size=(lay.num_pages, cfg.Hkv, 16, cfg.D)).astype(np.float32)
    kv = O.PagedKV(kp, vp, lay.page_table, lay.seq_len, lay.n_pages, lay.free_stack, lay.free_top)
    return lay, kv


def _check_conservation(kv, num_pages):
    live = []
    for s in range(kv.page_table.shape[0]):
        row = kv.page_table[s]
        assert (row[:kv.n_pages[s]] >= 0).all() and (row[kv.n_pages[s]:] == -1).all()
        assert kv.n_pages[s] >= -(-int(kv.seq_len[s]) // 16)
        live += row[:kv.n_pages[s]].tolist()
    free = kv.free_stack[:kv.free_top].tolist()
    assert len(live) + len(free) == num_pages
    assert sorted(live + free) == list(range(num_pages))


def test_layout_is_a_permutation_and_non_contiguous():
    cfg = W.StepConfig("t", 3, 4, 2, 8, 8, 16, 100, (20, 90), seed=3, growth=64)
    lay = W.kv_layout(cfg)
    live = [p for b in range(3) for p in lay.page_table[b, :lay.n_pages[b]]]
    assert len(set(live)) == len(live)
    assert sorted(live + lay.free_stack[:lay.free_top[0]].tolist()) == list(range(lay.num_pages))
    assert any(abs(int(a) - int(b)) != 1 for a, b in zip(live[:-1], live[1:]))


def test_soak_against_dense_shadow_cache():
    cfg = W.StepConfig("t", 4, 4, 2, 8, 8, 16, 100, (0, 70), seed=4, growth=40 * 8)
    lengths = np.array([0, 15, 16, 70], dtype=np.int32)
    lay, kv = _state(cfg, lengths)
    shadow_k = [O.gather_prefix(kv.k_pool, kv.page_table[s], int(lengths[s]), 16).copy() for s in range(4)]
    shadow_v = [O.gather_prefix(kv.v_pool, kv.page_table[s], int(lengths[s]), 16).copy() for s in range(4)]
    r = np.random.default_rng(2)
    ids = np.arange(4)
    for step in range(40):
        kb = r.normal(size=(4, 8, 2, 8)).astype(np.float32)
        vb = r.normal(size=(4, 8, 2, 8)).astype(np.float32)
        keep = r.integers(0, 9, size=4)
        assert kv.reserve(ids, 8)
        _check_conservation(kv, lay.num_pages)
        kv.append(ids, kb, vb)
        kv.commit(ids, keep)
        _check_conservation(kv, lay.num_pages)
        for s in range(4):
            shadow_k[s] = np.concatenate([shadow_k[s], kb[s, :keep[s]]])
            shadow_v[s] = np.concatenate([shadow_v[s], vb[s, :keep[s]]])
            gk, gv = kv.gather(s)
            np.testing.assert_array_equal(gk, shadow_k[s])
            np.testing.assert_array_equal(gv, shadow_v[s])
            assert kv.n_pages[s] == -(-int(kv.seq_len[s]) // 16)


def test_commit_zero_then_reserve_restores_state():
    cfg = W.StepConfig("t", 3, 4, 2, 8, 8, 16, 100, (5, 40), seed=5, growth=64)
    lay, kv = _state(cfg, np.array([5, 16, 40], dtype=np.int32))
    ids = np.arange(3)
    assert kv.reserve(ids, 8)
    snap = (kv.page_table.copy(), kv.seq_len.copy(), kv.n_pages.copy(), kv.free_stack[:kv.free_top].copy())
    kv.commit(ids, [0, 0, 0])
    assert kv.seq_len.tolist() == [5, 16, 40]
    assert kv.reserve(ids, 8)
    np.testing.assert_array_equal(kv.seq_len, snap[1])
    np.testing.assert_array_equal(kv.n_pages, snap[2])
    # the same set of pages is mapped again (order inside a sequence may differ
    # only if it took more than one page; here each takes at most one or two)
    for s in range(3):
        assert sorted(kv.page_table[s, :kv.n_pages[s]].tolist()) == sorted(snap[0][s, :snap[2][s]].tolist())
    assert sorted(kv.free_stack[:kv.free_top].tolist()) == sorted(snap[3].tolist())


def test_reserve_fails_cleanly_when_out_of_pages():
    cfg = W.StepConfig("t", 2, 4, 2, 8, 8, 16, 100, (16, 16), seed=6)
    lay, kv = _state(cfg, np.array([16, 16], dtype=np.int32))
    kv.free_top = 1
    before = (kv.page_table.copy(), kv.n_pages.copy(), kv.free_top)
    assert not kv.reserve([0, 1], 8)
    np.testing.assert_array_equal(kv.page_table, before[0])
    np.testing.assert_array_equal(kv.n_pages, before[1])
    assert kv.free_top == before[2]


def test_full_page_rollback_frees_exactly_the_tail_pages():
    cfg = W.StepConfig("t", 1, 4, 2, 8, 32, 16, 100, (30, 30), seed=7)
    lay, kv = _state(cfg, np.array([30], dtype=np.int32))
    top0 = kv.free_top
    assert kv.reserve([0], 32)                 # 62 tokens -> 4 pages (2 new)
    assert kv.n_pages[0] == 4 and kv.free_top == top0 - 2
    newp = kv.page_table[0, 2:4].copy()
    kv.commit([0], [2])                        # 32 tokens -> exactly 2 pages
    assert kv.seq_len[0] == 32 and kv.n_pages[0] == 2 and kv.free_top == top0
    # pushed back highest logical page first
    assert kv.free_stack[top0 - 2:top0].tolist() == [newp[1], newp[0]]
