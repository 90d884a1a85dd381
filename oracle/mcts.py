"""Plain CPU statement of the draft maker: Monte Carlo tree search over tri-gram continuations
(Eq. 2-3, Algorithm 1; "Draft Maker and Self-Improvement").  Test infrastructure.

Algorithm 1 is followed phase by phase -- selection by the PUCT score, expansion of every candidate
word of the reached node, simulation by drawing continuations from the tri-gram statistics, back
propagation of a score built from the tri-gram probabilities, ranking of the found sentences -- with
these readings where the listing or the text leave a choice:

  * a node stands for a token; its context is (token of its parent, its token), the root's context is
    the last two tokens of the text; its candidate words are the top-k list of that context (rank order);
  * a sentence holds at most `length` tokens after the root ("length of each retrieved continuation
    candidate");
  * selection descends while the node has been expanded and has children, taking the child with the
    largest PUCT (Eq. 2) -- Q = score / visits (0 for an unvisited child), P = Eq. 1 probability of the
    child's token in the node's context, sums over the node's children, E by Eq. 3 -- the first such
    child on ties;
  * expansion creates one child per candidate word at once and continues with the last one created,
    as the listing does;
  * simulation extends the state token by token, drawing from the top-k list of the last two tokens in
    proportion to the counts with a uniform number supplied by the caller (inverse CDF in rank order,
    integer arithmetic: first entry whose running count exceeds floor(sum * floor(u 2^24) / 2^24));
  * the score of an iteration is 1.0 plus, for every token of the state after the first, its Eq. 1
    probability given its two predecessors, added in order; it is added to the reached node and all
    its ancestors together with one visit;
  * the sentences are the root-to-leaf paths of the search tree (leaf = node without children, depth
    >= 1), ranked by the leaf's mean score (score / visits, 0 if never visited), earlier-created
    leaves first on ties; the best `n_candidates` are merged into one prefix tree, numbered breadth
    first, children in creation (rank) order.
All floating-point work is IEEE double, one rounded operation at a time, in the order written.

What is the algorithm's and what is this module's: the order of the four phases inside an iteration, the
rule that expansion creates every candidate at once and goes on with the last one, the score of 1.0 plus
tri-gram probabilities, and back propagation to every ancestor are Algorithm 1's definition of the search --
an iteration reads the visit counts and scores the previous one left, so any other order is a different
search and a different draft.  They are restated here from that definition.  The data structures (parallel
lists indexed by node number, contexts kept per node), the selection rule's tie break, the integer inverse
CDF of the simulation, the ranking and the prefix-tree merge are this module's own, as listed above.
"""
from __future__ import annotations

import math
from typing import List, Sequence, Tuple

from .trigram import TrigramStore


def _prob(store: TrigramStore, a: int, b: int, c: int) -> float:
    tot = store.total(a, b)
    return store.count(a, b, c) / tot if tot else 0.0


def puct(q: float, p: float, n_sum: int, n_a: int, c1: float, c2: float) -> float:
    """Eq. 2 with the exploration factor of Eq. 3."""
    e = c1 + math.log((n_sum + c2 + 1.0) / c2)
    return q + ((e * p) * math.sqrt(float(n_sum))) / (1.0 + n_a)


def mcts_draft(store: TrigramStore, prev_token: int, root_token: int, iterations: int, length: int, n_candidates: int,
               k: int, u: Sequence[Sequence[float]], c1: float = 32.0, c2: float = 8.0):
    """Returns (tokens, parents, sentences): the merged prefix tree (node 0 = root) and the ranked
    sentences [(tokens after the root, mean score)].  u[it][j] is the uniform number of the j-th
    simulation draw of iteration it."""
    tok = [int(root_token)]
    par = [-1]
    depth = [0]
    kids: List[List[int]] = [[]]
    expanded = [False]
    visits = [0]
    score = [0.0]

    def context(i: int) -> Tuple[int, int]:
        return (int(prev_token) if i == 0 else tok[par[i]], tok[i])

    for it in range(iterations):
        node = 0
        state = [tok[0]]
        end = False
        # selection
        while expanded[node] and kids[node] and not end:
            a, b = context(node)
            n_sum = sum(visits[c] for c in kids[node])
            best, best_s = -1, 0.0
            for c in kids[node]:
                q = score[c] / visits[c] if visits[c] else 0.0
                s = puct(q, _prob(store, a, b, tok[c]), n_sum, visits[c], c1, c2)
                if best < 0 or s > best_s:
                    best, best_s = c, s
            node = best
            state.append(tok[node])
            if len(state) == length + 1:
                end = True
        # expansion
        if not expanded[node] and not end:
            a, b = context(node)
            words = [w for w in store.topk(a, b, k)[0] if w >= 0]
            expanded[node] = True
            for w in words:
                tok.append(int(w)); par.append(node); depth.append(depth[node] + 1)
                kids.append([]); expanded.append(False); visits.append(0); score.append(0.0)
                kids[node].append(len(tok) - 1)
            if words:
                node = kids[node][-1]
                state.append(tok[node])
        # simulation
        draws = 0
        while len(state) < length + 1:
            a = state[-2] if len(state) >= 2 else int(prev_token)
            b = state[-1]
            words, counts = store.topk(a, b, k)
            words = [w for w in words if w >= 0]
            if not words:
                break
            total = sum(counts[:len(words)])
            u24 = int(math.floor(float(u[it][draws]) * 2.0 ** 24))
            target = (total * u24) >> 24
            run = 0
            for w, cnt in zip(words, counts):
                run += cnt
                if run > target:
                    state.append(int(w))
                    break
            draws += 1
        # back propagation
        s = 1.0
        for i in range(1, len(state)):
            a = state[i - 2] if i >= 2 else int(prev_token)
            s = s + _prob(store, a, state[i - 1], state[i])
        cur = node
        while cur >= 0:
            visits[cur] += 1
            score[cur] = score[cur] + s
            cur = par[cur]

    # ranking of the sentences and their prefix tree
    leaves = [i for i in range(1, len(tok)) if not kids[i]]
    mean = lambda i: score[i] / visits[i] if visits[i] else 0.0
    leaves.sort(key=lambda i: (-mean(i), i))
    chosen = leaves[:n_candidates]
    sentences = []
    keep = {0}
    for i in chosen:
        path, j = [], i
        while j > 0:
            path.append(tok[j]); keep.add(j); j = par[j]
        sentences.append((list(reversed(path)), mean(i)))
    order = [0]
    head = 0
    while head < len(order):
        order += [c for c in kids[order[head]] if c in keep]
        head += 1
    index = {old: new for new, old in enumerate(order)}
    tokens = [tok[i] for i in order]
    parents = [-1] + [index[par[i]] for i in order[1:]]
    return tokens, parents, sentences
