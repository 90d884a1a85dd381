"""Plain CPU statement of the tri-gram store (test infrastructure, see package header).

Eq. 1 defines P(w_i | w_{i-2}, w_{i-1}) = C(w_{i-2}, w_{i-1}, w_i) / C(w_{i-2}, w_{i-1}).
The store keeps the numerators as integer counts; within one context (w_{i-2}, w_{i-1}) the
denominator is shared, so ranking continuations by count is ranking them by probability.
Algorithm 2 ("Dynamic Adjustment of tri-gram Probabilities") raises the entry of every
tri-gram of a recent token span by an increment, up to a maximum, inserting absent ones.
"""
from __future__ import annotations

from typing import Dict, List, Sequence, Tuple


class TrigramStore:
    def __init__(self, cap: int = 2 ** 31 - 1, increment: int = 1):
        self.table: Dict[Tuple[int, int], Dict[int, int]] = {}
        self.cap = cap            # Algorithm 2's "maxProb", on the count scale
        self.increment = increment

    def update(self, tokens: Sequence[int]) -> None:
        """Algorithm 2 over the given span: every window (t[i-2], t[i-1], t[i]), i = 2..n-1,
        is raised once; a span shorter than three tokens changes nothing.  (The caller picks the
        span, which is the role of the algorithm's maxLength.)"""
        for i in range(2, len(tokens)):
            ctx = (int(tokens[i - 2]), int(tokens[i - 1]))
            row = self.table.setdefault(ctx, {})
            c = int(tokens[i])
            if c in row:
                row[c] = min(row[c] + self.increment, self.cap)
            else:
                row[c] = min(self.increment, self.cap)

    def count(self, a: int, b: int, c: int) -> int:
        return self.table.get((int(a), int(b)), {}).get(int(c), 0)

    def total(self, a: int, b: int) -> int:
        """Sum of the context's tri-gram counts: the denominator of Eq. 1."""
        return sum(self.table.get((int(a), int(b)), {}).values())

    def prob(self, a: int, b: int, c: int) -> float:
        tot = self.total(a, b)
        return self.count(a, b, c) / tot if tot else 0.0

    def topk(self, a: int, b: int, k: int, min_count: int = 0) -> Tuple[List[int], List[int]]:
        """The k most probable continuations of (a, b): count descending, token id ascending
        among equals; entries with count < min_count are skipped; short lists are padded with
        token -1, count 0."""
        row = self.table.get((int(a), int(b)), {})
        items = sorted(((c, n) for c, n in row.items() if n >= min_count),
                       key=lambda cn: (-cn[1], cn[0]))[:k]
        toks = [c for c, _ in items] + [-1] * (k - len(items))
        cnts = [n for _, n in items] + [0] * (k - len(items))
        return toks, cnts

    def prune(self, min_count: int) -> None:
        """Removes every tri-gram whose count is below min_count (the "threshold for the elimination of
        tri-gram probability" of the experimental settings, on the count scale); contexts left without a
        continuation disappear."""
        self.table = {ctx: kept for ctx, kept in
                      ((ctx, {c: n for c, n in row.items() if n >= min_count}) for ctx, row in self.table.items()) if kept}

    def merge(self, entries: Dict[Tuple[int, int, int], int]) -> None:
        """Adds stored entries (as returned by entries()) to the table: counts add up, saturating at the cap."""
        for (a, b, c), n in entries.items():
            row = self.table.setdefault((int(a), int(b)), {})
            row[int(c)] = min(row.get(int(c), 0) + int(n), self.cap)

    def entries(self) -> Dict[Tuple[int, int, int], int]:
        return {(a, b, c): n for (a, b), row in self.table.items() for c, n in row.items()}
