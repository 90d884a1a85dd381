"""Pins of the CPU checker's draft-tree retrieval against hand-worked trees and an independent
statement of the same tree (all root-to-node rank paths, sorted)."""
import itertools

import pytest

from oracle import draft as od
from oracle.trigram import TrigramStore
from paper_2407_12021_b200 import inputs as gen


def _store(rows):
    s = TrigramStore()
    for (a, b), cont in rows.items():
        for c, n in cont.items():
            for _ in range(n):
                s.update([a, b, c])
    return s


def test_hand_worked_tree():
    # context (1,2): 4 and 3 tie at 5 -> token order 3, 4; then 7.  (2,3) -> 9.  (2,4) -> 3, 8.  (3,9) -> 1.
    s = _store({(1, 2): {3: 5, 4: 5, 7: 2}, (2, 3): {9: 1}, (2, 4): {8: 1, 3: 4}, (3, 9): {1: 2}, (2, 7): {}})
    tok, par, real = od.draft_tree(s, 1, 2, 16, 3, 2)
    #   0:2 -> 1:3, 2:4 (k = 2 drops 7);  1:3 ctx (2,3) -> 3:9;  2:4 ctx (2,4) -> 4:3, 5:8;
    #   3:9 ctx (3,9) -> 6:1;  4:3 ctx (4,3) none; 5:8 none; depth limit 3 stops below node 6
    assert tok == [2, 3, 4, 9, 3, 8, 1]
    assert par == [-1, 0, 0, 1, 2, 2, 3]
    assert real == 7
    # node budget cuts in the middle of a sibling list
    tok, par, real = od.draft_tree(s, 1, 2, 5, 3, 3)
    assert tok == [2, 3, 4, 7, 9] and par == [-1, 0, 0, 0, 1] and real == 5
    # depth limit 1: only the root is expanded
    tok, par, _ = od.draft_tree(s, 1, 2, 16, 1, 3)
    assert tok == [2, 3, 4, 7] and par == [-1, 0, 0, 0]
    # depth limit 0 / unknown context: the root alone
    assert od.draft_tree(s, 1, 2, 16, 0, 3) == ([2], [-1], 1)
    assert od.draft_tree(s, 5, 5, 16, 3, 3) == ([5], [-1], 1)


def test_hand_worked_filler():
    empty = TrigramStore()
    tok, par, real = od.draft_tree(empty, 0, 1, 6, 2, 2, filler=[5, 5, 6, 7, 8, 9, 10])
    assert (tok, par, real) == ([1, 5, 5, 6, 7, 8], [-1, 0, 1, 0, 1, 3], 1)
    # clashing filler tokens are passed over and stay consumed
    tok, par, real = od.draft_tree(empty, 0, 1, 4, 1, 3, filler=[5, 5, 5, 6, 7])
    assert (tok, par, real) == ([1, 5, 6, 7], [-1, 0, 0, 0], 1)
    with pytest.raises(ValueError):
        od.draft_tree(empty, 0, 1, 4, 1, 3, filler=[5, 5, 5, 6])       # runs out
    with pytest.raises(ValueError):
        od.draft_tree(empty, 0, 1, 6, 1, 2, filler=list(range(10, 40)))   # a root with two children is full
    # without a filler the tree stays short
    assert od.draft_tree(empty, 0, 1, 4, 1, 3) == ([1], [-1], 1)


def _all_rank_paths(store, prev, root, max_depth, k):
    """Every node of the unbounded tree as (rank path, token path), by recursion."""
    out = []

    def rec(u, w, ranks, toks):
        out.append((tuple(ranks), tuple(toks)))
        if len(ranks) == max_depth:
            return
        ranked, _ = store.topk(u, w, k)
        for r, t in enumerate(ranked):
            if t >= 0:
                rec(w, t, ranks + [r], toks + [t])

    rec(prev, root, [], [root])
    return out


@pytest.mark.parametrize("seed,n_nodes,max_depth,k", [(1, 64, 6, 4), (2, 24, 3, 3), (3, 128, 4, 8), (4, 7, 5, 2)])
def test_equals_sorted_rank_paths_on_random_tables(seed, n_nodes, max_depth, k):
    vocab = 12
    s = TrigramStore()
    s.update(gen.zipf_tokens(600, vocab, seed, 3).tolist())
    text = gen.zipf_tokens(2, vocab, seed, 4).tolist()
    tok, par, real = od.draft_tree(s, text[0], text[1], n_nodes, max_depth, k)
    # breadth-first numbering = nodes sorted by depth, then by the rank path, cut at the budget
    want = sorted(_all_rank_paths(s, text[0], text[1], max_depth, k), key=lambda rt: (len(rt[0]), rt[0]))[:n_nodes]
    got = []
    for i in range(len(tok)):
        path, j = [], i
        while j >= 0:
            path.append(tok[j])
            j = par[j]
        got.append(tuple(reversed(path)))
    assert got == [t for _, t in want]
    assert real == len(tok) == len(want)


@pytest.mark.parametrize("seed", range(6))
def test_filled_tree_invariants(seed):
    vocab, n_nodes, max_depth, k = 40, 64, 6, 4
    s = TrigramStore()
    s.update(gen.zipf_tokens(300, vocab, seed, 3).tolist())
    text = gen.zipf_tokens(2, vocab, seed, 4).tolist()
    filler = gen.zipf_tokens(4 * n_nodes, vocab, seed, 9).tolist()
    tok, par, real = od.draft_tree(s, text[0], text[1], n_nodes, max_depth, k, filler=filler)
    bare = od.draft_tree(s, text[0], text[1], n_nodes, max_depth, k)
    assert len(tok) == n_nodes and (tok[:real], par[:real], real) == bare
    depth = [0] * n_nodes
    for i in range(1, n_nodes):
        assert 0 <= par[i] < i
        depth[i] = depth[par[i]] + 1
        assert depth[i] <= max_depth
    for p in range(n_nodes):
        kids = [tok[i] for i in range(1, n_nodes) if par[i] == p]
        assert len(kids) == len(set(kids)) and len(kids) <= k
    # filler tokens are used in list order
    it = iter(filler)
    assert all(any(t == f for f in it) for t in tok[real:])


def test_decode_context():
    assert od.decode_context(7, 8, [9]) == (8, 9)
    assert od.decode_context(7, 8, [9, 10, 11]) == (10, 11)
    for prev, root, acc in itertools.product([1], [2], [[3], [3, 4]]):
        assert od.decode_context(prev, root, acc) == tuple(([prev, root] + acc)[-2:])
