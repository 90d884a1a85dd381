"""Plain CPU statement of draft-tree retrieval from the tri-gram store (test infrastructure).

The method retrieves candidate continuations of the text from the tri-gram statistics, starting
from the last two tokens of the input, keeps the best-ranked ones and hands them to the model as
one pseudo-sequence in which a common prefix appears once (Figure 1; "Draft Construction and
Verification").  The retrieval stated here is the exhaustive one the verification step of this
repository is fed with: every node of the tree is expanded by the k most probable continuations of
its own two-token context (Eq. 1 ranks them), breadth first, until the node budget or the depth
limit is reached.  The paper's own ranking of candidates is a tree search (Eq. 2-3, Algorithm 1);
that search is not part of this function.

A verification step of fixed shape needs exactly `n_nodes` nodes.  When the table runs dry the rest
of the tree is filled from a caller-supplied list of tokens (random numbers are inputs here, never
drawn inside): the paper has no counterpart of the filler, it only keeps the launch shape constant.
"""
from __future__ import annotations

from typing import List, Optional, Sequence, Tuple

from .trigram import TrigramStore


def draft_tree(store: TrigramStore, prev_token: int, root_token: int, n_nodes: int, max_depth: int, k: int,
               filler: Optional[Sequence[int]] = None) -> Tuple[List[int], List[int], int]:
    """Returns (tokens, parents, nodes_from_table).

    Node 0 holds `root_token` (the last committed token); its context is (prev_token, root_token).
    A node holding token w whose parent holds u has context (u, w).  Nodes are visited in index
    order; a visited node of depth < max_depth gets one child per entry of store.topk(u, w, k), in
    rank order, appended at the end, until the tree has n_nodes nodes.  So siblings are distinct,
    parents[i] < i, and node indices are breadth-first.

    With `filler` given and fewer than n_nodes nodes found, nodes are visited round-robin (0, 1, ...,
    wrapping over the tree as it stands); a visited node with depth < max_depth and fewer than k
    children gets ONE more child: the next filler token that none of its children holds (tokens
    passed over are consumed).  ValueError when the filler runs out or no node has room.
    """
    if n_nodes < 1 or max_depth < 0 or k < 1:
        raise ValueError("n_nodes >= 1, max_depth >= 0, k >= 1")
    tokens = [int(root_token)]
    parents = [-1]
    depth = [0]
    head = 0
    while head < len(tokens) and len(tokens) < n_nodes:
        if depth[head] < max_depth:
            u = int(prev_token) if head == 0 else tokens[parents[head]]
            ranked, _ = store.topk(u, tokens[head], k)
            for t in ranked:
                if t < 0 or len(tokens) >= n_nodes:
                    break
                tokens.append(int(t))
                parents.append(head)
                depth.append(depth[head] + 1)
        head += 1
    from_table = len(tokens)
    if filler is not None:
        tokens, parents = fill_tree(tokens, parents, n_nodes, max_depth, k, filler)
    return tokens, parents, from_table


def fill_tree(tokens: Sequence[int], parents: Sequence[int], n_nodes: int, max_depth: int, k: int,
              filler: Sequence[int]) -> Tuple[List[int], List[int]]:
    """Completes a draft tree (parents[i] < i) to exactly n_nodes nodes with caller-supplied tokens, by the
    rule of draft_tree's docstring: nodes are visited round-robin; a visited node with depth < max_depth
    and fewer than k children gets the next filler token that none of its children holds.  A tree that
    already has n_nodes nodes or more is returned unchanged."""
    tokens = [int(t) for t in tokens]
    parents = [int(p) for p in parents]
    depth = [0] * len(tokens)
    for i in range(1, len(tokens)):
        depth[i] = depth[parents[i]] + 1
    pos = 0
    p = 0
    idle = 0
    while len(tokens) < n_nodes:
        kids = [tokens[i] for i in range(1, len(tokens)) if parents[i] == p]
        if depth[p] < max_depth and len(kids) < k:
            while pos < len(filler) and int(filler[pos]) in kids:
                pos += 1
            if pos >= len(filler):
                raise ValueError("filler exhausted")
            tokens.append(int(filler[pos]))
            pos += 1
            parents.append(p)
            depth.append(depth[p] + 1)
            idle = 0
        else:
            idle += 1
            if idle > len(tokens):
                raise ValueError("no node has room for a filler child")
        p = (p + 1) % len(tokens)
    return tokens, parents


def decode_context(prev_token: int, root_token: int, accepted: Sequence[int]) -> Tuple[int, int]:
    """Last two tokens of the text after a step that emitted `accepted` (at least one token):
    the context the next step's retrieval starts from."""
    chain = [int(prev_token), int(root_token)] + [int(t) for t in accepted]
    return chain[-2], chain[-1]
