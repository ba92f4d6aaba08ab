"""High-precision, definition-level references used to pin the CPU oracle.

Nothing here follows the oracle's step-by-step arithmetic.  The references are
the *sequence-level* definitions of the paper, evaluated with 60-digit decimals
on the exactly widened stored logits:

  * the codebook of Sec. 4.1: in dictionary order every sequence owns the
    interval [lo, lo + P(sequence)); a code decodes to the sequence whose
    interval contains it (enumerated by brute force);
  * top-k and nucleus membership stated by counting ("how many tokens rank
    strictly before this one", "how much mass ranks strictly before it"),
    not by sorting.
"""
from __future__ import annotations

from decimal import Decimal, getcontext
from typing import Dict, List, Sequence, Tuple

getcontext().prec = 60


def D(x) -> Decimal:
    return Decimal(float(x))  # float -> Decimal is exact


def conditional(logits: Sequence[float], temp: float = 1.0, top_k: int = 0,
                top_p: float = 1.0, typical_p: float = 1.0) -> List[Decimal]:
    """Modified next-token distribution, membership defined by counting."""
    V = len(logits)
    neg_inf = float("-inf")
    alive = [l > neg_inf for l in logits]

    def before(i, j):  # does token i rank strictly before token j?
        return logits[i] > logits[j] or (logits[i] == logits[j] and i < j)

    if 0 < top_k < sum(alive):
        alive = [alive[j] and sum(1 for i in range(V) if alive[i] and before(i, j)) < top_k
                 for j in range(V)]
    tau = D(temp)
    xs = [D(logits[j]) / tau if alive[j] else None for j in range(V)]
    m = max(x for x in xs if x is not None)
    w = [(x - m).exp() if x is not None else Decimal(0) for x in xs]
    if 0.0 < typical_p < 1.0:
        # locally typical set by counting: token j stays iff the mass of the tokens whose
        # |-ln p - H| is smaller (or equal, with a lower index) has not reached the target
        total = sum(w)
        pr = [x / total for x in w]
        H = -sum(q * q.ln() for q in pr if q > 0)
        dist = [abs(-q.ln() - H) if q > 0 else None for q in pr]

        def closer(i, j):
            return dist[i] < dist[j] or (dist[i] == dist[j] and i < j)
        target = D(typical_p) * total
        alive = [alive[j] and dist[j] is not None and
                 sum(w[i] for i in range(V) if alive[i] and dist[i] is not None and closer(i, j)) < target
                 for j in range(V)]
        w = [w[j] if alive[j] else Decimal(0) for j in range(V)]
    if 0.0 < top_p < 1.0:
        total = sum(w)
        target = D(top_p) * total
        # token j stays iff the mass ranked strictly before it has not reached the target
        alive2 = []
        for j in range(V):
            if not alive[j]:
                alive2.append(False)
                continue
            mass_before = sum(w[i] for i in range(V) if alive[i] and before(i, j))
            alive2.append(mass_before < target)
        alive = alive2
        w = [w[j] if alive[j] else Decimal(0) for j in range(V)]
    total = sum(w)
    return [x / total for x in w]


def enumerate_codebook(row_probs, start: int, T: int, eos: int = -1
                       ) -> List[Tuple[Tuple[int, ...], Decimal, Decimal]]:
    """All complete sequences of a bigram model in dictionary order with their
    intervals: [(sequence, lo, width)].  row_probs(prev) -> list of Decimal."""
    out = []

    def rec(prefix, prev, lo, width):
        if len(prefix) == T or (prefix and prefix[-1] == eos):
            out.append((tuple(prefix), lo, width))
            return
        p = row_probs(prev)
        acc = lo
        for tok, pt in enumerate(p):
            if pt > 0:
                rec(prefix + [tok], tok, acc, width * pt)
            acc += width * pt

    rec([], start, Decimal(0), Decimal(1))
    return out


def locate(book, c: float):
    """(sequence, lo, width, distance of c to the nearest end of its interval)."""
    cd = D(c)
    for seq, lo, width in book:
        if lo <= cd < lo + width:
            return seq, lo, width, min(cd - lo, lo + width - cd)
    return book[-1][0], book[-1][1], book[-1][2], Decimal(0)


def expectation(book, f) -> Decimal:
    return sum(width * Decimal(f(seq)) for seq, _, width in book)
