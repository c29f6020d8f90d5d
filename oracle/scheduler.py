"""Oracle of the load-driven DCP scheduler (Section 5.1): closed-form targets and Algorithm 1.

TEST INFRASTRUCTURE ONLY: a plain, slow, direct implementation (every search is a linear scan over all
open groups, every comparison is exact integer arithmetic) against which the heap-accelerated library
routine is checked placement by placement. Nothing in the product path imports this module.

What follows the paper literally
  W = sum s_i^2                                   (Table "Notation")
  Lambda* = s_max^2 / C                           (Eq. load-target)
  M* = ceil(C W / (G s_max^2))                    (Eq. mstar)
  C^* = s_max^2 sqrt((pp-1) theta G / (c W))      (Eq. cstar-cont)
  C_mem = ceil2(s_max / B), C* = min{G, ceil2(max{C_mem, C^*})}      (Eq. cstar)
  cp(s) = min{C*, ceil2(max{s^2 / Lambda*, s / B})}                   (Eq. cp)
  group g is feasible for s iff load(g) + s^2/|g| <= Lambda* and tokens(g) + s/|g| <= B
  Algorithm 1: longest first; a new cp(s)-sized group while enough ranks are free, else the smallest
  feasible open group of size >= cp(s), ties by load; otherwise the micro-batch is closed; idle ranks
  are backfilled; next micro-batch.
ceil2(x) is the smallest power of two that is at least x.

Readings where the paper only sketches (the library takes the same ones):
  R1  Ties after (size, load) go to the group opened first; equal lengths keep their input order.
  R2  The early-close test at the end of Algorithm 1's inner loop (degree shrunk, micro-batch balanced): after a
      placement, if the next document's degree is smaller than the degree just used, every rank is busy, and the least-loaded group carries at least 3/4 of the
      per-rank load of the most loaded one, the micro-batch is closed.
  R3  Backfill: while the smallest open group (ties: higher per-rank load first, then opened first) is
      no larger than the number of idle ranks, it is doubled (its documents run at twice the degree).
  R4  Ranks: at close, groups sorted by size (descending, ties by opening order) take consecutive rank
      blocks from rank 0, which makes every block aligned to its own size.
  R5  G and C must be powers of two and C >= C_mem (otherwise the longest document cannot be placed).
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from fractions import Fraction
from typing import List, Sequence


def ceil2(x) -> int:
    """Smallest power of two >= x (x a positive int, Fraction or float)."""
    t = 1
    while t < x:
        t *= 2
    return t


@dataclass
class Targets:
    W: int
    s_max: int
    C_mem: int
    C_hat: float
    C_star: int
    Lambda_star: Fraction
    M_star: int


def targets(lengths: Sequence[int], G: int, B: int, pp: int, theta_over_c: float) -> Targets:
    W = sum(int(s) * int(s) for s in lengths)
    s_max = max(int(s) for s in lengths)
    C_mem = ceil2(Fraction(s_max, B))
    C_hat = s_max * s_max * math.sqrt((pp - 1) * theta_over_c * G / W)
    C_star = min(G, ceil2(max(C_mem, C_hat)))
    lam = Fraction(s_max * s_max, C_star)
    M_star = -((-C_star * W) // (G * s_max * s_max))
    return Targets(W, s_max, C_mem, C_hat, C_star, lam, M_star)


def cp_degree(s: int, s_max: int, C: int, B: int) -> int:
    lam = Fraction(s_max * s_max, C)
    return min(C, ceil2(max(Fraction(s * s) / lam, Fraction(s, B))))


@dataclass
class Group:
    size: int
    opened: int                 # order of opening inside the micro-batch
    load_n: int = 0             # sum of s^2 of its documents (per-rank load = load_n / size)
    tok_n: int = 0              # sum of s (per-rank tokens = tok_n / size)
    docs: List[int] = field(default_factory=list)


@dataclass
class Placement:
    mb: List[int]               # micro-batch of every document (input order)
    rank0: List[int]            # first rank of its group
    cp: List[int]               # size of its group (after backfill)
    n_mb: int


def pack(lengths: Sequence[int], G: int, B: int, C: int) -> Placement:
    s = [int(x) for x in lengths]
    n = len(s)
    assert G >= 1 and G & (G - 1) == 0 and C >= 1 and C & (C - 1) == 0 and C <= G
    s_max = max(s)
    assert C * B >= s_max, "C below C_mem"
    order = sorted(range(n), key=lambda i: (-s[i], i))
    mb_of, rank0_of, cp_of = [0] * n, [0] * n, [0] * n
    pos, m = 0, 0
    while pos < n:
        groups: List[Group] = []
        free = G
        while pos < n:
            i = order[pos]
            k = cp_degree(s[i], s_max, C, B)
            if free >= k:
                g = Group(k, len(groups))
                groups.append(g)
                free -= k
            else:
                best = None
                for cand in groups:                        # the direct scan of every open group
                    if cand.size < k:
                        continue
                    if (cand.load_n + s[i] * s[i]) * C > s_max * s_max * cand.size:
                        continue
                    if cand.tok_n + s[i] > B * cand.size:
                        continue
                    key = (cand.size, cand.load_n, cand.opened)
                    if best is None or key < best[0]:
                        best = (key, cand)
                if best is None:
                    break
                g = best[1]
            g.docs.append(i)
            g.load_n += s[i] * s[i]
            g.tok_n += s[i]
            pos += 1
            if pos < n and cp_degree(s[order[pos]], s_max, C, B) < k and free == 0:
                lo = min(Fraction(x.load_n, x.size) for x in groups)
                hi = max(Fraction(x.load_n, x.size) for x in groups)
                if 4 * lo >= 3 * hi:
                    break
        # backfill idle ranks by doubling the smallest group
        while groups:
            gmin = min(groups, key=lambda x: (x.size, -Fraction(x.load_n, x.size), x.opened))
            if gmin.size > free:
                break
            free -= gmin.size
            gmin.size *= 2
        # ranks: largest groups first, consecutive blocks
        at = 0
        for g in sorted(groups, key=lambda x: (-x.size, x.opened)):
            for i in g.docs:
                mb_of[i], rank0_of[i], cp_of[i] = m, at, g.size
            at += g.size
        m += 1
    return Placement(mb_of, rank0_of, cp_of, m)
