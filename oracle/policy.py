"""CPU oracle of the greedy marginal-utility policy — TEST INFRASTRUCTURE ONLY.

Follows the paper's Design section step by step, in exact rational arithmetic where it decides
anything:

  Utility(i) = Freq(i) * (alpha * Quality(i, M_i, R_i) - size(i, M_i, R_i) / Bandwidth)

(the printed formula has an unbalanced parenthesis; this is the reading with the parenthesis
closed after the delay term), the problem is a multiple-choice knapsack, and the greedy step picks,
among all entries, the move (compress further, or evict) with the smallest

  marginal utility drop = (Utility(i, m) - Utility(i, n)) / (size(i) * (m - n)),

i.e. utility lost per byte saved, until the tier's capacity holds everything that is left.  The
textbook greedy the paper cites works on each entry's LP-undominated options (the upper convex
hull of its (size, utility) points, eviction = (0, 0) included), which is what makes the result
optimal for the linear relaxation.

An option is (size in bytes, quality); options of all entries are concatenated and
option_begin[i] .. option_begin[i+1] delimit entry i's.  A choice is an index into the entry's own
options, or -1 for eviction.
"""
from __future__ import annotations

from fractions import Fraction


def utility(freq, alpha, bandwidth, size, quality) -> Fraction:
    """The utility definition, exactly."""
    return Fraction(freq) * (Fraction(alpha) * Fraction(quality) - Fraction(size) / Fraction(bandwidth))


def hull_of_entry(points: list[tuple[int, Fraction, int]]) -> list[tuple[int, Fraction, int]]:
    """LP-undominated choices of one entry, from its best one down to eviction.

    points: (size, utility, option index) of every option.  Returns the chain the greedy walks:
    first the point of largest utility (the smallest such point on ties; eviction if nothing has
    positive utility), then points of strictly smaller size with strictly growing utility lost per
    byte saved, ending with eviction (0, 0, -1)."""
    pts = [(0, Fraction(0), -1)] + sorted(points, key=lambda p: (p[0], -p[1], p[2]))
    best = max(pts, key=lambda p: (p[1], -p[0]))
    # candidates strictly smaller than the best point; on equal size keep the higher utility
    lower = {}
    for s, u, k in pts:
        if s < best[0] and (s not in lower or u > lower[s][1]):
            lower[s] = (s, u, k)
    chain = [best]
    cur = best
    while cur[0] > 0:
        # the next vertex of the upper hull: the smaller point with the least utility lost per byte
        # saved; among equals the smallest one (the points between lie on the same edge)
        nxt = min((p for p in lower.values() if p[0] < cur[0]),
                  key=lambda p: ((cur[1] - p[1]) / (cur[0] - p[0]), p[0]))
        chain.append(nxt)
        cur = nxt
    return chain


def assign_tier(freq, options, option_begin, alpha, bandwidth, capacity, candidates=None):
    """Greedy assignment of one storage tier.  Returns (choice per entry, bytes used, total utility);
    entries outside `candidates` are not considered and get choice -1."""
    n = len(freq)
    cand = range(n) if candidates is None else candidates
    chains, pos = {}, {}
    for i in cand:
        pts = [(int(options[k][0]), utility(freq[i], alpha, bandwidth, options[k][0], options[k][1]),
                k - option_begin[i]) for k in range(option_begin[i], option_begin[i + 1])]
        chains[i] = hull_of_entry(pts)
        pos[i] = 0
    used = sum(chains[i][0][0] for i in chains)
    while used > capacity:
        # the move with the smallest marginal utility drop; the lowest entry index on ties
        best = None
        for i in sorted(chains):
            ch, p = chains[i], pos[i]
            if p + 1 < len(ch):
                drop = (ch[p][1] - ch[p + 1][1]) / (ch[p][0] - ch[p + 1][0])
                if best is None or drop < best[0]:
                    best = (drop, i)
        _, i = best
        used -= chains[i][pos[i]][0] - chains[i][pos[i] + 1][0]
        pos[i] += 1
    choice = [-1] * n
    total = Fraction(0)
    for i in chains:
        choice[i] = chains[i][pos[i]][2]
        total += chains[i][pos[i]][1]
    return choice, used, total


def assign_tiers(freq, options, option_begin, tiers):
    """Tiers in order (fastest first): what a tier evicts is offered to the next one.  tiers:
    (alpha, bandwidth, capacity) each.  Returns (tier per entry or -1, choice per entry or -1)."""
    n = len(freq)
    tier_of, choice_of = [-1] * n, [-1] * n
    left = list(range(n))
    for t, (alpha, bandwidth, capacity) in enumerate(tiers):
        choice, _, _ = assign_tier(freq, options, option_begin, alpha, bandwidth, capacity, candidates=left)
        nxt = []
        for i in left:
            if choice[i] >= 0:
                tier_of[i], choice_of[i] = t, choice[i]
            else:
                nxt.append(i)
        left = nxt
    return tier_of, choice_of
