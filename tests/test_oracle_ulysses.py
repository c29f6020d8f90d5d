"""Pins of the Ulysses pack / unpack oracle to what Section 3.5 fixes: after the all-to-all every rank
holds all tokens of the group for its own h / P heads, the way back restores the token split, and the
volume is Eq. (ulysses)'s. None of these re-evaluates the oracle's own index formula."""
import os

import numpy as np
import pytest

import oracle

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "ulysses_pack_2x4.txt")


def tagged(S, h, d):
    """Element (t, a, c) carries its own coordinates: 16-bit tag = t * 64 + a * 4 + c (small cases)."""
    t, a, c = np.meshgrid(np.arange(S), np.arange(h), np.arange(d), indexing="ij")
    v = t * 64 + a * 4 + c
    assert v.max() < 65536 and h <= 16 and d <= 4
    return v.astype(np.uint16)


@pytest.mark.parametrize("world,n,h,d", [(2, 3, 4, 2), (4, 5, 8, 3), (1, 4, 3, 2), (8, 2, 8, 1), (2, 1, 16, 4)])
def test_after_the_exchange_every_rank_holds_all_tokens_of_its_own_heads(world, n, h, d):
    """Section 3.5: the transposes partition the heads across the ranks. The expected result is a slice
    of the global tensor, taken with numpy indexing, not with the oracle's loops."""
    X = tagged(world * n, h, d)                                     # the group's sequence, [S, h, d]
    local = [X[r * n:(r + 1) * n] for r in range(world)]            # token split
    recv = oracle.all_to_all([oracle.ulysses_pack(x, world) for x in local])
    hg = h // world
    for r in range(world):
        assert np.array_equal(recv[r].reshape(world * n, hg, d), X[:, r * hg:(r + 1) * hg, :])


@pytest.mark.parametrize("world,n,h,d", [(2, 3, 4, 2), (4, 5, 8, 3), (8, 2, 8, 1)])
def test_the_way_back_restores_the_token_split(world, n, h, d):
    """After attention a rank holds [S, h / P, d] for its heads; it splits it by owner of the tokens
    (contiguous blocks), the exchange runs again, and unpack must give every rank its own rows with all
    heads."""
    X = tagged(world * n, h, d)
    hg = h // world
    head_split = [X[:, r * hg:(r + 1) * hg, :] for r in range(world)]
    send = [hs.reshape(world, n, hg, d) for hs in head_split]        # block i = the tokens rank i owns
    recv = oracle.all_to_all(send)
    for r in range(world):
        assert np.array_equal(oracle.ulysses_unpack(recv[r]), X[r * n:(r + 1) * n])


def test_pack_and_unpack_are_inverse_permutations():
    rng = np.random.default_rng(5)
    x = rng.integers(0, 65536, size=(7, 12, 5), dtype=np.uint16)
    for cp_u in (1, 2, 3, 4, 6, 12):
        y = oracle.ulysses_pack(x, cp_u)
        assert y.shape == (cp_u, 7, 12 // cp_u, 5)
        assert sorted(y.ravel().tolist()) == sorted(x.ravel().tolist())      # a permutation
        assert np.array_equal(oracle.ulysses_unpack(y), x)
    assert np.array_equal(oracle.ulysses_pack(x, 1)[0], x)                   # degree 1: nothing moves
    with pytest.raises(ValueError):
        oracle.ulysses_pack(x, 5)


def test_volume_is_eq_ulysses():
    """Eq. (ulysses): about 4 S h / P elements per rank (q, k, v on the way in, the output on the way
    back), per unit of head dimension."""
    S, h, P, d = 64, 8, 4, 1
    n = S // P
    x = np.zeros((n, h, d), dtype=np.uint16)
    per_tensor = oracle.ulysses_pack(x, P).size
    assert 4 * per_tensor == 4 * S * h // P


def test_worked_example_by_hand():
    """2 ranks, 2 local tokens, 4 heads, d = 1, written out by hand in the fixture: rows are
    'block token head-in-block value'."""
    x = np.array([[[10], [11], [12], [13]], [[20], [21], [22], [23]]], dtype=np.uint16)   # x[t, a] = 10 (t+1) + a
    y = oracle.ulysses_pack(x, 2)
    with open(GOLDEN) as f:
        rows = [tuple(int(v) for v in line.split()) for line in f if line.strip() and not line.startswith("#")]
    assert len(rows) == y.size
    for j, t, b, v in rows:
        assert int(y[j, t, b, 0]) == v
