"""Property tests of the CPU checker's integer parts (hypothesis): statements that hold for any input
and that a dropped term, a wrong index or a swapped argument would break."""
import numpy as np
from hypothesis import given, settings, strategies as st

from oracle import draft as od
from oracle import sample as osmp
from oracle.trigram import TrigramStore

tokens = st.lists(st.integers(0, 7), min_size=0, max_size=60)


@settings(max_examples=60, deadline=None)
@given(tokens, st.integers(0, 59))
def test_counts_are_window_multiplicities_and_splits_add_up(text, cut):
    s = TrigramStore()
    s.update(text)
    want = {}
    for i in range(2, len(text)):
        key = (text[i - 2], text[i - 1], text[i])
        want[key] = want.get(key, 0) + 1
    assert s.entries() == want
    # counting a stream piecewise, each piece with the two tokens before it, gives the same table
    cut = min(cut, len(text))
    two = TrigramStore()
    two.update(text[:cut])
    two.update(text[max(cut - 2, 0):])
    assert two.entries() == want
    for (a, b), row in s.table.items():
        assert s.total(a, b) == sum(row.values())
        toks, cnts = s.topk(a, b, 3)
        valid = [(t, c) for t, c in zip(toks, cnts) if t >= 0]
        assert valid == sorted(((t, c) for t, c in row.items()), key=lambda tc: (-tc[1], tc[0]))[:3]


@settings(max_examples=60, deadline=None)
@given(tokens, st.integers(1, 5))
def test_prune_then_merge_of_the_removed_part_restores_the_table(text, t):
    s = TrigramStore()
    s.update(text)
    before = s.entries()
    s.prune(t)
    kept = s.entries()
    assert kept == {k: n for k, n in before.items() if n >= t}
    s.merge({k: n for k, n in before.items() if n < t})
    assert s.entries() == before


@settings(max_examples=40, deadline=None)
@given(tokens, st.integers(1, 20), st.integers(0, 4), st.integers(1, 4))
def test_draft_tree_is_a_prefix_of_the_larger_budget_tree(text, n, depth, k):
    s = TrigramStore()
    s.update(text)
    prev, root = (text[0], text[1]) if len(text) >= 2 else (0, 1)
    small = od.draft_tree(s, prev, root, n, depth, k)
    large = od.draft_tree(s, prev, root, n + 7, depth, k)
    assert large[0][:len(small[0])] == small[0] and large[1][:len(small[1])] == small[1]
    assert len(small[0]) == min(n, len(large[0])) or len(large[0]) == len(small[0])
    deeper = od.draft_tree(s, prev, root, 10 ** 6, depth + 1, k)
    unbounded = od.draft_tree(s, prev, root, 10 ** 6, depth, k)
    assert deeper[0][:len(unbounded[0])] == unbounded[0]        # breadth first: a deeper limit only appends levels


@settings(max_examples=60, deadline=None)
@given(st.lists(st.floats(-8, 8, width=32), min_size=1, max_size=12), st.floats(0.0625, 4.0, width=32),
       st.floats(2.0 ** -10, 1.0, width=32), st.floats(0, 1, exclude_max=True, width=32), st.floats(0, 1, exclude_max=True, width=32))
def test_draw_is_in_the_nucleus_and_monotone_in_u(logits, temp, top_p, u1, u2):
    l = np.array(logits, dtype=np.float32)
    q = osmp.weights(l, temp)
    members = sorted(osmp.nucleus(q, top_p))
    assert int(np.argmax(q)) in members and all(q[v] > 0 for v in members)
    # everything outside is no heavier than anything inside
    outside = [v for v in range(len(l)) if v not in members]
    assert not outside or max(int(q[v]) for v in outside) <= min(int(q[v]) for v in members)
    lo, hi = sorted((u1, u2))
    a, b = osmp.sample(l, temp, top_p, lo), osmp.sample(l, temp, top_p, hi)
    assert a in members and b in members and a <= b
