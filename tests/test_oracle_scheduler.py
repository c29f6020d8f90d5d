"""Pins of the scheduler oracle (oracle/scheduler.py) to what the paper and arithmetic fix.

* the four-rank, 4K-budget example of Section 2.3 (a 16K sequence spans all four ranks, an 8K one two,
  a 4K one a single rank; the same ranks serve as one group of four, two of two, four of one in
  successive micro-batches);
* the cap that Eq. (cstar-cont) gives is the minimiser of the cost model of Eq. (capcost), evaluated
  here from the model's definition, not from the closed form;
* M* counts work: M* G Lambda* >= W > (M* - 1) G Lambda*  (Eq. mstar);
* cp(s) is the smallest power of two that meets both requirements of Eq. (cp), found by search;
* Algorithm 1's invariants on random batches: every document placed once, micro-batches are
  contiguous runs of the longest-first order, groups are powers of two on aligned disjoint rank
  blocks, token budget and load target hold for every group as packed, and every piggyback choice is
  the one an exhaustive search over the open groups would make.
"""
import math
from fractions import Fraction

import numpy as np
import pytest

from oracle import scheduler as S


def test_four_rank_example_of_the_paper():
    lengths = [16384, 8192, 8192, 4096, 4096, 4096, 4096]
    t = S.targets(lengths, G=4, B=4096, pp=1, theta_over_c=1.0)
    assert (t.C_mem, t.C_star) == (4, 4) and t.Lambda_star == 16384 ** 2 // 4
    assert [S.cp_degree(s, t.s_max, t.C_star, 4096) for s in (16384, 8192, 4096)] == [4, 2, 1]
    p = S.pack(lengths, G=4, B=4096, C=4)
    assert p.n_mb == 3
    assert p.mb == [0, 1, 1, 2, 2, 2, 2]
    assert p.cp == [4, 2, 2, 1, 1, 1, 1]
    assert p.rank0 == [0, 0, 2, 0, 1, 2, 3]


def test_cap_minimises_the_cost_model():
    rng = np.random.default_rng(0)
    for _ in range(20):
        lengths = [int(x) for x in rng.integers(256, 200000, size=200)]
        G, pp, theta, c = 512, int(rng.integers(2, 12)), 1e-9, float(rng.uniform(1e-4, 1e-1))
        t = S.targets(lengths, G, B=8192, pp=pp, theta_over_c=theta / c)
        W, smax = t.W, t.s_max

        def cost(C):                                        # Eq. (capcost), from its definition
            lam = smax * smax / C
            M = C * W / (G * smax * smax)
            return theta * W / G + (pp - 1) * theta * lam + c * M

        assert cost(t.C_hat) <= cost(t.C_hat * 1.01) and cost(t.C_hat) <= cost(t.C_hat * 0.99)
        assert t.C_star == min(G, S.ceil2(max(t.C_mem, t.C_hat)))
        assert t.C_star >= t.C_mem or t.C_star == G


def test_target_micro_batch_count_conserves_work():
    rng = np.random.default_rng(1)
    for _ in range(50):
        lengths = [int(x) for x in rng.integers(64, 100000, size=int(rng.integers(1, 400)))]
        G = 2 ** int(rng.integers(0, 11))
        t = S.targets(lengths, G, B=4096, pp=4, theta_over_c=1e-6)
        cap = G * t.Lambda_star
        assert t.M_star * cap >= t.W > (t.M_star - 1) * cap


def test_degree_is_the_smallest_power_of_two_that_meets_both_requirements():
    rng = np.random.default_rng(2)
    for _ in range(300):
        smax = int(rng.integers(1000, 300000))
        s = int(rng.integers(1, smax + 1))
        B = int(rng.integers(512, 16384))
        C = 2 ** int(rng.integers(0, 10))
        lam = Fraction(smax * smax, C)
        want = next((k for k in (2 ** j for j in range(40)) if Fraction(s * s, k) <= lam and Fraction(s, k) <= B), None)
        assert S.cp_degree(s, smax, C, B) == min(C, want)


def _replay(lengths, G, B, C):
    """Re-derives, from the placement alone, what every group held when each document arrived."""
    p = S.pack(lengths, G, B, C)
    n = len(lengths)
    smax = max(lengths)
    order = sorted(range(n), key=lambda i: (-lengths[i], i))
    assert sorted(p.mb) == [p.mb[i] for i in order]          # contiguous runs of the sorted order
    assert set(p.mb) == set(range(p.n_mb))
    for m in range(p.n_mb):
        docs = [i for i in order if p.mb[i] == m]
        blocks = {}
        for i in docs:
            blocks.setdefault(p.rank0[i], []).append(i)
        used = 0
        for r0, members in blocks.items():
            size = p.cp[members[0]]
            assert all(p.cp[i] == size for i in members)
            assert size & (size - 1) == 0 and size <= G and r0 % size == 0 and r0 + size <= G
            used += size
            tok = sum(lengths[i] for i in members)
            load = sum(lengths[i] ** 2 for i in members)
            # as packed the group was at most as large as now (backfill only doubles), so these hold a fortiori
            assert tok <= B * size and load * C <= smax * smax * size
        assert used <= G
        spans = sorted((r0, r0 + p.cp[m_[0]]) for r0, m_ in blocks.items())
        assert all(a[1] <= b[0] for a, b in zip(spans, spans[1:]))
    return p


@pytest.mark.parametrize("seed", range(12))
def test_packing_invariants_on_random_batches(seed):
    rng = np.random.default_rng(100 + seed)
    G = 2 ** int(rng.integers(2, 8))
    B = int(rng.choice([4096, 8192]))
    n = int(rng.integers(1, 300))
    lengths = [int(min(B * G, max(16, round(math.exp(rng.normal(math.log(2048), 1.3)))))) for _ in range(n)]
    C = min(G, S.ceil2(max(S.ceil2(Fraction(max(lengths), B)), 2 ** int(rng.integers(0, 6)))))
    _replay(lengths, G, B, C)


def test_piggyback_takes_the_smallest_then_least_loaded_feasible_group():
    # G = 4, B = 16384, C = 2, Lambda* = 16000^2 / 2 = 1.28e8.
    # 16000 opens a group of 2 (its load alone reaches Lambda*), 7000 and 6000 groups of 1; no rank is
    # free any more, and the group of 2 is full by load, so the shorter documents piggyback on the
    # groups of 1, each on the less loaded of the two at that moment (loads are sums of s^2).
    lengths = [16000, 7000, 6000, 4000, 3000, 2500]
    p = S.pack(lengths, G=4, B=16384, C=2)
    assert p.n_mb == 1 and p.cp == [2, 1, 1, 1, 1, 1]
    g7000, g6000 = p.rank0[1], p.rank0[2]
    assert g7000 != g6000
    assert p.rank0[3] == g6000          # 4000 arrives first (longest first): 3.6e7 < 4.9e7
    assert p.rank0[4] == g7000          # 3000: 6000+4000 = 5.2e7 > 4.9e7
    assert p.rank0[5] == g6000          # 2500: 7000+3000 = 5.8e7 > 5.2e7


def test_idle_ranks_are_backfilled_by_doubling_the_smallest_group():
    p = S.pack([5000, 1000], G=8, B=8192, C=1)
    # two groups of one on eight ranks: 1000 (smallest, tie on size broken by load: 5000 first) ...
    assert p.n_mb == 1 and sum(sorted(set(zip(p.rank0, p.cp)), key=lambda x: x[0])[i][1] for i in range(2)) == 8
    assert sorted(p.cp) == [4, 4]
