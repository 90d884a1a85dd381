"""Pins of the CPU checker's tri-gram store: brute-force window counts (the numerator of
Eq. 1), a full sort for top-k, and the step list of Algorithm 2 on hand cases."""
from collections import Counter

from oracle.trigram import TrigramStore
from paper_2407_12021_b200 import inputs as gen


def _windows(tokens):
    return Counter((tokens[i - 2], tokens[i - 1], tokens[i]) for i in range(2, len(tokens)))


def test_update_equals_brute_force_window_count():
    toks = gen.zipf_tokens(5000, 50, 11, 1).tolist()
    st = TrigramStore()
    st.update(toks)
    want = _windows(toks)
    assert st.entries() == dict(want)
    assert sum(want.values()) == len(toks) - 2


def test_probability_is_eq1_ratio():
    toks = gen.zipf_tokens(3000, 20, 12, 1).tolist()
    st = TrigramStore()
    st.update(toks)
    tri = _windows(toks)
    bi = Counter((toks[i - 1], toks[i]) for i in range(1, len(toks) - 1))   # bigrams that have a successor
    for (a, b, c), n in list(tri.items())[:200]:
        assert st.total(a, b) == bi[(a, b)]
        assert st.prob(a, b, c) == n / bi[(a, b)]


def test_hand_case_algorithm2():
    st = TrigramStore()
    st.update([1, 2, 3, 1, 2, 3, 1, 2, 4])
    assert st.count(1, 2, 3) == 2 and st.count(1, 2, 4) == 1
    assert st.count(2, 3, 1) == 2 and st.count(3, 1, 2) == 2
    assert len(st.entries()) == 4
    st.update([7, 8])          # shorter than a tri-gram: nothing happens
    st.update([])
    assert len(st.entries()) == 4
    st.update([1, 2, 4])       # exactly one window
    assert st.count(1, 2, 4) == 2


def test_saturation_and_split_calls():
    st = TrigramStore(cap=3)
    st.update([5] * 10)                      # eight windows (5,5,5)
    assert st.count(5, 5, 5) == 3
    # feeding a stream piecewise, each piece carrying the two tokens before it, counts every
    # window exactly once
    toks = gen.zipf_tokens(400, 9, 13, 1).tolist()
    whole, parts = TrigramStore(), TrigramStore()
    whole.update(toks)
    cuts = [0, 3, 4, 50, 51, 52, 200, 400]
    for lo, hi in zip(cuts[:-1], cuts[1:]):
        parts.update(toks[max(lo - 2, 0):hi])
    assert whole.entries() == parts.entries()


def test_topk_equals_full_sort_with_tie_rule():
    toks = gen.zipf_tokens(20000, 12, 14, 1).tolist()
    st = TrigramStore()
    st.update(toks)
    tri = _windows(toks)
    for a in range(12):
        for b in range(12):
            row = sorted(((c, n) for (x, y, c), n in tri.items() if (x, y) == (a, b)),
                         key=lambda cn: (-cn[1], cn[0]))
            for k in (1, 4, 16):
                t, n = st.topk(a, b, k)
                want_t = [c for c, _ in row[:k]] + [-1] * max(0, k - len(row))
                want_n = [m for _, m in row[:k]] + [0] * max(0, k - len(row))
                assert (t, n) == (want_t, want_n)
    # ties: equal counts come out in ascending token order
    st = TrigramStore()
    st.update([1, 1, 9, 1, 1, 3, 1, 1, 7])
    assert st.topk(1, 1, 4)[0][:3] == [3, 7, 9]
    assert st.topk(4, 4, 2) == ([-1, -1], [0, 0])     # unknown context
    # the count filter drops rare continuations
    st.update([1, 1, 7])
    assert st.topk(1, 1, 4, min_count=2) == ([7, -1, -1, -1], [2, 0, 0, 0])


def test_prune_and_merge_by_hand():
    from oracle.trigram import TrigramStore
    s = TrigramStore(cap=10)
    s.update([1, 2, 3, 1, 2, 3, 1, 2, 4])          # (1,2,3) x2, (2,3,1) x2, (3,1,2) x2, (1,2,4) x1
    assert s.entries() == {(1, 2, 3): 2, (2, 3, 1): 2, (3, 1, 2): 2, (1, 2, 4): 1}
    s.prune(2)
    assert s.entries() == {(1, 2, 3): 2, (2, 3, 1): 2, (3, 1, 2): 2}
    assert s.topk(1, 2, 3) == ([3, -1, -1], [2, 0, 0])
    s.merge({(1, 2, 3): 9, (7, 7, 7): 4})
    assert s.entries() == {(1, 2, 3): 10, (2, 3, 1): 2, (3, 1, 2): 2, (7, 7, 7): 4}      # 2 + 9 saturates at the cap
    s.prune(11)
    assert s.entries() == {} and s.table == {}
