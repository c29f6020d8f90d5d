"""Pins of the oracle's integer bookkeeping (zigzag chunks, causal pairs, Eq. (usp))."""
import os

import numpy as np
import pytest

import hydra_workloads as hw
import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def test_usp_factor_matches_values_printed_in_the_paper():
    with open(os.path.join(GOLDEN, "usp_examples.txt")) as f:
        rows = [l.split("#")[0].split() for l in f if l.split("#")[0].strip()]
    assert len(rows) >= 3
    for p, h, cp_u, cp_r in rows:
        assert oracle.usp_factor(int(p), int(h)) == (int(cp_u), int(cp_r))


def test_usp_factor_of_the_benchmark_shape():
    # 128 heads with an inner Ulysses group of 8 leave 16 heads per rank; degree 32 at 256K context
    # with 8 heads' worth of Ulysses is Ulysses 8 x ring 4.
    assert oracle.usp_factor(32, 8) == (8, 4)


@pytest.mark.parametrize("cp_r", [1, 2, 4, 8])
def test_zigzag_ownership_is_balanced(cp_r):
    n_c = 2 * cp_r
    owners = [oracle.zigzag_rank(c, cp_r) for c in range(n_c)]
    for r in range(cp_r):
        assert sorted(c for c in range(n_c) if owners[c] == r) == [r, n_c - 1 - r]


def test_ring_of_four_pair_counts_and_schedule():
    L = 262144
    pairs = oracle.causal_pairs([0, L], 4)
    assert len(pairs) == 36 and sum(p["diagonal"] for p in pairs) == 8
    assert all(p["q_len"] == 32768 and p["k_len"] == 32768 for p in pairs)
    # brute force: the pairs tile the causal triangle exactly once
    total = sum(p["q_len"] * (p["q_len"] + 1) // 2 if p["diagonal"] else p["q_len"] * p["k_len"]
                for p in pairs)
    assert total == L * (L + 1) // 2 == 34359869440
    for rank in range(4):
        mine = [p for p in pairs if p["rank"] == rank]
        assert len(mine) == 9
        for step in range(4):
            work = sum(0.5 if p["diagonal"] else 1.0 for p in mine if p["step"] == step)
            assert work == 2.0
    r0 = {(p["step"], p["qc"], p["kc"]) for p in pairs if p["rank"] == 0}
    assert r0 == {(0, 0, 0), (0, 7, 0), (0, 7, 7), (1, 7, 3), (1, 7, 4), (2, 7, 2), (2, 7, 5),
                  (3, 7, 1), (3, 7, 6)}


@pytest.mark.parametrize("L", [1, 2, 3, 7, 8, 9, 300, 301, 1023])
@pytest.mark.parametrize("cp_r", [0, 1, 2, 4])
def test_pairs_cover_every_causal_cell_exactly_once(L, cp_r):
    pairs = oracle.causal_pairs([0, L], cp_r)
    cover = np.zeros((L, L), dtype=np.int32)
    for p in pairs:
        for i in range(p["q_start"], p["q_start"] + p["q_len"]):
            hi = min(i, p["k_start"] + p["k_len"] - 1)
            if hi >= p["k_start"]:
                cover[i, p["k_start"]:hi + 1] += 1
    assert np.array_equal(cover, np.tril(np.ones((L, L), dtype=np.int32)))
    chunks = oracle.zigzag_chunks(L, cp_r)
    assert sum(l for _, l in chunks) == L
    assert max(l for _, l in chunks) - min(l for _, l in chunks) <= 1
    groups = [p["group"] for p in pairs]
    assert groups == sorted(groups)


def test_tiny_split_is_150_150():
    assert oracle.zigzag_chunks(300, 1) == [(0, 150), (150, 150)]
    pairs = oracle.causal_pairs([0, 300], 1)
    assert [(p["qc"], p["kc"], p["diagonal"]) for p in pairs] == [(0, 0, 1), (1, 0, 0), (1, 1, 1)]


def test_workload_lengths_are_the_recorded_lists():
    assert hw.lengths_sha1(hw.lengths_lognormal()).startswith("9c011f49f53b")
    assert hw.lengths_sha1(hw.lengths_skewed()).startswith("fc61255c3e90")
    assert hw.lengths_sha1(hw.lengths_uniform()).startswith("2c267829c285")
    assert hw.workload("packed32k").causal_pairs_total == 48922862
    assert hw.workload("skewed128k").causal_pairs_total == 4848284685
    assert hw.workload("short64k").causal_pairs_total == 11355655


def test_bf16_round_trip_is_round_to_nearest_even():
    torch = pytest.importorskip("torch")
    rng = np.random.default_rng(0)
    x = np.concatenate([rng.standard_normal(4096).astype(np.float32) * 10,
                        np.array([0.0, -0.0, 1.0, 1.00390625, 1.01171875, 3.3895e38, 1e-40],
                                 dtype=np.float32)])
    want = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(hw.f32_to_bf16_bits(x), want)
    assert np.array_equal(hw.bf16_bits_to_f32(want),
                          torch.from_numpy(want.view(np.int16)).view(torch.bfloat16).float().numpy())
