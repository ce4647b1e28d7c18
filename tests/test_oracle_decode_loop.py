"""Pins of the oracle's Algorithm-1 loop book-keeping (DecodeState.emit):
expected outputs are written out by hand or follow from counting, never from
the function itself."""
import numpy as np

from oracle import deer_oracle as O


def test_hand_worked_trace():
    """Two sequences, k = 3, EOS = 9, at most 5 new tokens.  By hand:
    pass 1: seq0 accepts 2 drafts + correction -> [4,5,6]; seq1 rejects at once -> [7]
    pass 2: seq0 has room for 2 of [1,2,3] -> [4,5,6,1,2], full, keeps min(3,2)=2 rows;
            seq1 emits [8,9] (EOS cut by the acceptance rule) -> finished, keeps 1
    pass 3: both finished: nothing changes, nothing kept."""
    st = O.DecodeState(2, 5)
    keep = st.emit(np.array([2, 0]), np.array([[4, 5, 6], [7, -1, -1]]), np.array([3, 1]), eos_id=9)
    assert keep.tolist() == [2, 0] and st.n_tokens.tolist() == [3, 1] and st.finished.tolist() == [0, 0]
    keep = st.emit(np.array([3, 1]), np.array([[1, 2, 3], [8, 9, -1]]), np.array([3, 2]), eos_id=9)
    assert keep.tolist() == [2, 1]
    assert st.tokens.tolist() == [[4, 5, 6, 1, 2], [7, 8, 9, -1, -1]]
    assert st.n_tokens.tolist() == [5, 3] and st.finished.tolist() == [1, 1]
    before = st.tokens.copy()
    keep = st.emit(np.array([3, 3]), np.array([[1, 1, 1], [1, 1, 1]]), np.array([3, 3]), eos_id=9)
    assert keep.tolist() == [0, 0] and (st.tokens == before).all() and st.n_tokens.tolist() == [5, 3]


def test_counts_follow_from_planted_lengths():
    """Greedy passes with planted matching-prefix lengths L and no EOS: each pass
    emits L+1 tokens (L if L = k), so after S passes a sequence holds
    min(max_new, sum) tokens and the kept rows are the accepted drafts."""
    rng = np.random.default_rng(5)
    B, k, S, V, max_new = 6, 4, 5, 50, 14
    st = O.DecodeState(B, max_new)
    total = np.zeros(B, dtype=np.int64)
    for step in range(S):
        L = rng.integers(0, k + 1, size=B)
        target = rng.integers(0, V, size=(B, k))
        draft = target.copy()
        for b in range(B):
            if L[b] < k:
                draft[b, L[b]] = (target[b, L[b]] + 1) % V
        a, out, n = O.accept_greedy(draft, target)
        was_done = st.finished.copy()
        had = st.n_tokens.copy()
        keep = st.emit(a, out, n)
        for b in range(B):
            if was_done[b]:
                assert keep[b] == 0 and st.n_tokens[b] == had[b]
                continue
            emitted = L[b] + (1 if L[b] < k else 0)
            total[b] += emitted
            assert st.n_tokens[b] == min(max_new, had[b] + emitted)
            assert keep[b] == min(L[b], max_new - had[b])
    assert ((st.n_tokens == max_new) == (st.finished == 1)).all()
    assert (st.n_tokens == np.minimum(total, max_new)).all()


def test_eos_ends_a_sequence_and_later_passes_are_ignored():
    st = O.DecodeState(1, 100)
    a, out, n = O.accept_greedy(np.array([[3, 7, 5, 5]]), np.array([[3, 7, 5, 6]]), eos_id=7)
    assert n.tolist() == [2] and a.tolist() == [2]          # the EOS itself was an accepted draft
    keep = st.emit(a, out, n, eos_id=7)
    assert keep.tolist() == [2] and st.finished.tolist() == [1] and st.tokens[0, :3].tolist() == [3, 7, -1]
    keep = st.emit(np.array([4]), np.array([[1, 2, 3, 4]]), np.array([4]), eos_id=7)
    assert keep.tolist() == [0] and st.n_tokens.tolist() == [2]


def test_pending_token_alignment_hand_worked():
    """Row 0 of a block is the token emitted last, rows 1.. the drafts (k = 4 rows,
    3 drafts, every block emits accept_len + 1 tokens).  By hand:
    pass 1: seq0 accepts 2 drafts + correction [4,5,6] -> keeps the pending token's
            row and the 2 drafts' rows = 3; seq1 accepts all 3 + the extra token
            [1,2,3,7] -> keeps 4 rows
    pass 2: seq0 has room for 1 of [8,9] (max 4 new tokens) -> keeps 1 + min(1, 1) = 2,
            finished; seq1 was full after pass 1 -> finished there, keeps nothing now."""
    st = O.DecodeState(2, 4)
    keep = st.emit(np.array([2, 3]), np.array([[4, 5, 6, -1], [1, 2, 3, 7]]), np.array([3, 4]), pending=True)
    assert keep.tolist() == [3, 4] and st.n_tokens.tolist() == [3, 4] and st.finished.tolist() == [0, 1]
    keep = st.emit(np.array([1, 0]), np.array([[8, 9, -1, -1], [5, -1, -1, -1]]), np.array([2, 1]), pending=True)
    assert keep.tolist() == [2, 0]
    assert st.tokens.tolist() == [[4, 5, 6, 8], [1, 2, 3, 7]] and st.finished.tolist() == [1, 1]
