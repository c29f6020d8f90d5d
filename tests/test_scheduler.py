"""The library's scheduler (heap-accelerated, C ABI in include/hydra_sched.h) against the oracle's
direct scans: same targets, same degrees, and the same placement of every document (Section 5.1.3:
the heaps must reproduce the linear search's least-loaded placement and tie-breaking exactly)."""
import math
import time
from fractions import Fraction

import numpy as np
import pytest

import paper_2609_34318_b200 as P
from oracle import scheduler as S


def lognormal_batch(rng, n, median, sigma, lo, hi):
    return [int(min(hi, max(lo, round(math.exp(rng.normal(math.log(median), sigma)))))) for _ in range(n)]


@pytest.mark.parametrize("seed", range(10))
def test_targets_and_degrees_match_the_oracle(seed):
    rng = np.random.default_rng(seed)
    n = int(rng.integers(1, 500))
    lengths = lognormal_batch(rng, n, 2048, 1.4, 16, 262144)
    G = 2 ** int(rng.integers(0, 12))
    B = int(rng.choice([2048, 4096, 8192]))
    pp = int(rng.integers(1, 10))
    ratio = float(10 ** rng.uniform(-12, -6))
    want = S.targets(lengths, G, B, pp, ratio)
    got = P.hydra_sched_targets(lengths, G, B, pp, ratio)
    assert (got.s_max, got.C_mem, got.C_star, got.M_star) == (want.s_max, want.C_mem, want.C_star, want.M_star)
    assert got.W == float(want.W) and got.C_hat == pytest.approx(want.C_hat, rel=1e-12)
    assert got.Lambda_star == pytest.approx(float(want.Lambda_star), rel=1e-15)
    C = max(want.C_star, want.C_mem)
    for s in rng.choice(lengths, size=min(50, n)):
        assert P.hydra_sched_cp(int(s), want.s_max, C, B) == S.cp_degree(int(s), want.s_max, C, B)


@pytest.mark.parametrize("seed", range(40))
def test_every_placement_matches_the_direct_scan(seed):
    rng = np.random.default_rng(1000 + seed)
    G = 2 ** int(rng.integers(0, 9))
    B = int(rng.choice([1024, 4096, 8192]))
    n = int(rng.integers(1, 600))
    sigma = float(rng.choice([0.3, 1.0, 1.6]))
    lengths = lognormal_batch(rng, n, int(rng.choice([256, 2048, 16384])), sigma, 1, B * G)
    if seed % 5 == 0:                                     # many equal lengths: ties everywhere
        lengths = [min(int(x), B * G) for x in rng.choice([512, 1024, 4096], size=n)]
    C_mem = S.ceil2(Fraction(max(lengths), B))
    C = min(G, max(C_mem, 2 ** int(rng.integers(0, 9))))
    want = S.pack(lengths, G, B, C)
    mb, rank0, cp, n_mb = P.hydra_sched_pack(lengths, G, B, C)
    assert n_mb == want.n_mb
    assert mb.tolist() == want.mb and rank0.tolist() == want.rank0 and cp.tolist() == want.cp


def test_invalid_arguments_are_refused():
    assert P.hydra_sched_pack([100, 200], 6, 4096, 2, check=False) == P.HYDRA_ERR_INVALID_ARG      # G not 2^j
    assert P.hydra_sched_pack([100, 200], 8, 4096, 16, check=False) == P.HYDRA_ERR_INVALID_ARG     # C > G
    assert P.hydra_sched_pack([100000], 8, 4096, 2, check=False) == P.HYDRA_ERR_INVALID_ARG        # C < C_mem
    assert P.hydra_sched_pack([0, 5], 8, 4096, 2, check=False) == P.HYDRA_ERR_INVALID_ARG
    assert P.hydra_sched_cp(5, 4, 2, 4096) == 0


def test_degrees_feed_the_chunk_cutter():
    # scheduler -> Eq. (usp) -> zigzag pairs: a 256K document at degree 256 with 64 heads runs on an
    # inner Ulysses group of 64 and an outer ring of 4, i.e. 8 chunks and 36 causal pairs
    lengths = [262144] + [4096] * 64
    mb, rank0, cp, n_mb = P.hydra_sched_pack(lengths, 256, 8192, 256)
    assert cp[0] == 256
    cp_u, cp_r = P.hydra_usp_factor(int(cp[0]), 64)
    assert (cp_u, cp_r) == (64, 4)
    pairs, _, _, _ = P.hydra_zigzag_pairs(np.array([0, 262144], dtype=np.int32), cp_r)
    assert len(pairs) == 36


def test_heaps_scale_better_than_the_scan():
    # not a benchmark: the library must place a production-sized batch in well under a second
    rng = np.random.default_rng(7)
    lengths = lognormal_batch(rng, 200000, 1024, 1.4, 64, 262144)
    t0 = time.perf_counter()
    mb, rank0, cp, n_mb = P.hydra_sched_pack(lengths, 2048, 8192, 64)
    dt = time.perf_counter() - t0
    assert n_mb > 0 and dt < 5.0
