"""Pins of the CPU checker's draft maker (Monte Carlo tree search): the score formula at hand-computed
points, hand-worked searches on tables small enough to follow, and invariants of the result."""
import math

import pytest

from oracle import mcts as om
from oracle.trigram import TrigramStore
from paper_2407_12021_b200 import inputs as gen


def _store(rows):
    s = TrigramStore()
    for (a, b), cont in rows.items():
        for c, n in cont.items():
            for _ in range(n):
                s.update([a, b, c])
    return s


def test_puct_formula_at_known_points():
    # no visits anywhere: the exploration term vanishes with sqrt(0)
    assert om.puct(0.0, 0.7, 0, 0, 32.0, 8.0) == 0.0
    # sum N = 8, c2 = 8: E = c1 + ln(17/8);  PUCT = Q + E P sqrt(8) / (1 + N)
    want = 1.5 + (32.0 + math.log(17.0 / 8.0)) * 0.25 * math.sqrt(8.0) / 3.0
    assert om.puct(1.5, 0.25, 8, 2, 32.0, 8.0) == pytest.approx(want, rel=1e-15)
    # the other constant the paper uses
    want = (2.414 + math.log(10.0 / 8.0)) * 1.0 * 1.0 / 1.0
    assert om.puct(0.0, 1.0, 1, 0, 2.414, 8.0) == pytest.approx(want, rel=1e-15)
    # more visits of the child lower its score, a larger prior raises it
    assert om.puct(1.0, 0.5, 10, 1, 32.0, 8.0) > om.puct(1.0, 0.5, 10, 4, 32.0, 8.0)
    assert om.puct(1.0, 0.6, 10, 1, 32.0, 8.0) > om.puct(1.0, 0.5, 10, 1, 32.0, 8.0)


def test_single_chain_by_hand():
    # one continuation everywhere: 1 2 -> 3 -> 4 -> 5 -> 6, all probabilities 1
    s = _store({(1, 2): {3: 2}, (2, 3): {4: 1}, (3, 4): {5: 3}, (4, 5): {6: 1}, (5, 6): {7: 1}})
    u = [[0.5] * 4 for _ in range(10)]
    tok, par, sent = om.mcts_draft(s, 1, 2, 10, 3, 4, 4, u)
    # iteration 1 expands the root (child 3) and simulates 4, 5: state 2 3 4 5, score 1 + 3; every later
    # iteration descends one level further until the sentence is 3 tokens long, score always 4
    assert tok == [2, 3, 4, 5] and par == [-1, 0, 1, 2]
    assert sent == [([3, 4, 5], 4.0)]
    # length 1: only the root is ever expanded
    tok, par, sent = om.mcts_draft(s, 1, 2, 5, 1, 4, 4, u)
    assert (tok, par) == ([2, 3], [-1, 0]) and sent == [([3], 2.0)]
    # unknown context: nothing to propose
    assert om.mcts_draft(s, 9, 9, 5, 3, 4, 4, u) == ([9], [-1], [])


def test_two_branches_by_hand():
    # root context (1,2): 3 (count 3) and 4 (count 1); below 3 nothing, below 4: 5 with certainty
    s = _store({(1, 2): {3: 3, 4: 1}, (2, 4): {5: 2}})
    u = [[0.0] * 2 for _ in range(3)]
    tok, par, sent = om.mcts_draft(s, 1, 2, 3, 2, 8, 4, u, c1=32.0, c2=8.0)
    # it 1: expand root -> children 3 (P .75), 4 (P .25); continue with the LAST child 4; simulate 5 (P 1):
    #       state 2 4 5, score 1 + .25 + 1 = 2.25 -> node 4 and root: N 1, W 2.25
    # it 2: select among root's children, sum N = 1, E = 32 + ln(10/8):
    #       child 3: 0 + E .75 / 1,  child 4: 2.25 + E .25 / 2  -> child 3 (about 24.2 against 6.3);
    #       3 is not expanded: expand, no candidates; state 2 3, score 1.75 -> node 3: N 1, W 1.75
    # it 3: sum N = 2: child 3: 1.75 + E' .75 sqrt2 / 2, child 4: 2.25 + E' .25 sqrt2 / 2 -> child 3 again;
    #       expanded without children: stop; score 1.75 -> node 3: N 2, W 3.5
    # node 5 was only simulated, never created: the search tree is the root and its two children
    assert tok == [2, 3, 4] and par == [-1, 0, 0]
    assert sent == [([4], 2.25), ([3], 1.75)]
    # one more iteration: child 3 again (1.75 + E'' .75 sqrt3 / 3 against 2.25 + E'' .25 sqrt3 / 2), W 5.25 / N 3
    tok, par, sent = om.mcts_draft(s, 1, 2, 4, 2, 8, 4, [[0.0] * 2 for _ in range(4)])
    assert tok == [2, 3, 4] and sent == [([4], 2.25), ([3], 1.75)]


@pytest.mark.parametrize("seed", range(4))
def test_invariants_on_random_tables(seed):
    vocab, iters, length, n, k = 30, 60, 4, 24, 4
    s = TrigramStore()
    text = gen.zipf_tokens(1500, vocab, seed, 3).tolist()
    s.update(text)
    u = gen.uniform01(iters * length, seed, 5).reshape(iters, length).tolist()
    tok, par, sent = om.mcts_draft(s, text[10], text[11], iters, length, n, k, u)
    assert tok[0] == text[11] and par[0] == -1 and len(tok) <= 1 + n * length
    depth = [0] * len(tok)
    for i in range(1, len(tok)):
        assert 0 <= par[i] < i and par[i] >= par[i - 1]                  # breadth-first numbering
        depth[i] = depth[par[i]] + 1
        assert depth[i] <= length
        u_, w_ = (text[10], tok[0]) if par[i] == 0 else (tok[par[par[i]]], tok[par[i]])
        assert tok[i] in s.topk(u_, w_, k)[0]                             # every edge is a stored continuation
    for p in range(len(tok)):
        kids = [tok[i] for i in range(1, len(tok)) if par[i] == p]
        assert len(kids) == len(set(kids))
    assert 1 <= len(sent) <= n
    scores = [sc for _, sc in sent]
    assert scores == sorted(scores, reverse=True)
    paths = set()
    for i in range(len(tok)):
        path, j = [], i
        while j > 0:
            path.append(tok[j]); j = par[j]
        paths.add(tuple(reversed(path)))
    assert all(tuple(t) in paths for t, _ in sent)
    # the same numbers give the same search
    assert om.mcts_draft(s, text[10], text[11], iters, length, n, k, u) == (tok, par, sent)
