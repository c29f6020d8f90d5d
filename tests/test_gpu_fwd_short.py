"""The short-sequence forward kernel and the routing between the two forward kernels.

Section 2.2 of the paper: most sequences of a training batch are short. Pairs whose q and kv ranges are at most
`hydra_set_fwd_short_len` tokens long go to a kernel of their own (one CTA per SM, two independent 128-row q
tiles in flight, steps of 64 keys); the others stay on the CTA-pair kernel; a call whose short pairs carry less
than a quarter of its work uses the CTA-pair kernel alone. Every case here is checked against the fp64 oracle
(the small parity cases of the other test files run on both kernels as well: fixture `both_forward_kernels`).
"""
import numpy as np
import pytest
import torch

import hydra_workloads as hw
from conftest import FWD_SHORT_LEN_DEFAULT
from gpu_util import TOL_LSE, TOL_REL, check, pairs_for, run_gpu, run_oracle

pytestmark = pytest.mark.gpu
DQK, DV = hw.D_QK, hw.D_V


def rand_inputs(seed, T, h):
    rng = np.random.default_rng(seed)
    f = lambda d: hw.f32_to_bf16_bits(rng.standard_normal((T, h, d)).astype(np.float32))
    return dict(q=f(DQK), k=f(DQK), v=f(DV), do=f(DV))


def forward_launches(fn):
    """Launches of the library's kernels made by fn()."""
    import paper_2609_34318_b200 as P
    before = P.hydra_launch_count()
    fn()
    return P.hydra_launch_count() - before


@pytest.fixture(autouse=True)
def default_routing():
    import paper_2609_34318_b200 as P
    P.hydra_set_fwd_short_len(FWD_SHORT_LEN_DEFAULT)
    yield
    P.hydra_set_fwd_short_len(FWD_SHORT_LEN_DEFAULT)


@pytest.mark.parametrize("lengths", [
    [7, 33, 128, 300],            # a tile with 7 rows, one of exactly 128, one sequence of three tiles
    [1, 1, 1, 2],                 # work items of a single row and a single key
    [63, 65, 64],                 # one key more and one key less than a step
    [129, 257, 64, 500, 127],     # one row more than a tile, one more than two
    [2048],                       # the longest sequence the default routing sends here: 16 tiles, up to 32 steps
    [200] * 40,                   # more work items than the two slots of every SM hold at once
])
def test_short_sequences_against_the_oracle(lengths):
    h = 3
    cu = hw.cu_seqlens(lengths)
    x = rand_inputs(sum(lengths), int(cu[-1]), h)
    got = run_gpu(x, cu, h)
    ref = run_oracle(x, cu)
    check(got, ref, label=f"{lengths[:5]} ")


def test_random_length_mixes_and_both_kernels_agree():
    import paper_2609_34318_b200 as P
    rng = np.random.default_rng(11)
    for trial in range(4):
        lengths = [int(v) for v in rng.integers(1, 700, size=int(rng.integers(3, 12)))]
        h = int(rng.integers(1, 5))
        cu = hw.cu_seqlens(lengths)
        x = rand_inputs(100 + trial, int(cu[-1]), h)
        ref = run_oracle(x, cu, backward=False)
        res = {}
        for name, limit in (("short", 1 << 20), ("pair", 0)):
            P.hydra_set_fwd_short_len(limit)
            res[name] = run_gpu(x, cu, h, backward=False)
            check(res[name], ref, names=("out", "lse"), label=f"trial {trial} {name} ")
        # two summation orders of the same sums: a few bf16 roundings of O apart, never more
        assert np.abs(res["short"]["out"] - res["pair"]["out"]).max() <= TOL_REL * np.abs(ref["out"]).max()
        assert np.abs(res["short"]["lse"] - res["pair"]["lse"]).max() <= TOL_LSE


def test_one_call_uses_both_kernels_when_short_pairs_carry_enough_work():
    """A long sequence and many short ones: the long pair runs on CTA pairs, the short ones on the other kernel,
    in the same call (two launches); with few short ones the call stays on one kernel (one launch)."""
    import paper_2609_34318_b200 as P
    from paper_2609_34318_b200.runner import AttnStep, bits_to_tensor
    h = 2
    for lengths, launches in (([3000] + [300] * 60, 2), ([3000, 300, 300], 1), ([300] * 8, 1)):
        cu = hw.cu_seqlens(lengths)
        x = rand_inputs(len(lengths), int(cu[-1]), h)
        step = AttnStep(cu, h)
        q, k, v = (bits_to_tensor(x[n]) for n in ("q", "k", "v"))
        assert forward_launches(lambda: step.forward(q, k, v)) == launches, lengths[:3]
        got = run_gpu(x, cu, h, backward=False)
        check(got, run_oracle(x, cu, backward=False), names=("out", "lse"), label=f"{lengths[:3]} ")


def test_chunked_short_pairs_write_partials_and_merge():
    """Short sequences cut into zigzag chunks: diagonal and full pairs with offsets, partial outputs, the merge."""
    h = 2
    lengths = [300, 77, 512, 130]
    cu = hw.cu_seqlens(lengths)
    x = rand_inputs(5, int(cu[-1]), h)
    lib_pairs, rows, ora_pairs = pairs_for(cu, [1, 0, 2, 1])
    got = run_gpu(x, cu, h, lib_pairs, rows)
    check(got, run_oracle(x, cu, pairs=ora_pairs), label="chunked short ")


def test_non_causal_short_pairs():
    h = 2
    lengths = [100, 65, 257]
    cu = hw.cu_seqlens(lengths)
    x = rand_inputs(6, int(cu[-1]), h)
    got = run_gpu(x, cu, h, causal=False)
    check(got, run_oracle(x, cu, causal=False), label="non-causal short ")


@pytest.mark.parametrize("short_len", [FWD_SHORT_LEN_DEFAULT, 0])
def test_output_that_is_16_but_not_32_byte_aligned(short_len):
    """The interface asks for 16-byte alignment; both forward kernels store 32 bytes at a time only when the
    address allows it."""
    import paper_2609_34318_b200 as P
    P.hydra_set_fwd_short_len(short_len)
    from paper_2609_34318_b200.runner import AttnStep, bits_to_tensor
    h = 2
    lengths = [70, 300]
    cu = hw.cu_seqlens(lengths)
    T = int(cu[-1])
    x = rand_inputs(7, T, h)
    step = AttnStep(cu, h)
    raw = torch.zeros(T * h * DV * 2 + 64, dtype=torch.uint8, device="cuda")
    off = (16 - raw.data_ptr() % 32) % 32                # an address that is 16 modulo 32
    out = raw[off:off + T * h * DV * 2].view(torch.bfloat16).view(T, h, DV)
    assert out.data_ptr() % 32 == 16
    q, k, v = (bits_to_tensor(x[n]) for n in ("q", "k", "v"))
    P.hydra_attn_fwd(q, k, v, cu, h, None, True, step.scale, out, step.lse, None, None, 0, step.workspace)
    assert step.poll()[0] == 0
    ref = run_oracle(x, cu, backward=False)
    got = out.float().cpu().numpy().astype(np.float64)
    assert np.abs(got - ref["out"]).max() <= TOL_REL * np.abs(ref["out"]).max()
    assert bool((raw[:off] == 0).all()) and bool((raw[off + T * h * DV * 2:] == 0).all())


@pytest.mark.parametrize("short_len", [1 << 20, 0])
@pytest.mark.parametrize("q_start,q_len,k_start,k_len", [
    (0, 300, 200, 100),       # the first 200 q rows come before every key: a whole tile without keys, one with some
    (10, 140, 149, 60),       # only the last q row sees a key (its own position)
    (0, 130, 200, 90),        # no q row sees any key
    (50, 200, 0, 0),          # an empty kv range
    (255, 5, 0, 260),         # five rows at the end of a long kv range
])
def test_partials_of_hand_made_pairs_with_rows_that_see_no_key(short_len, q_start, q_len, k_start, k_len):
    """Rows of a pair that see no key get O = 0 and LSE = -inf (their weight in a merge is then 0): on both
    forward kernels, for whole tiles without keys, for single rows, and for pairs with no visible key at all."""
    import oracle
    import paper_2609_34318_b200 as P
    from paper_2609_34318_b200.runner import AttnStep, bits_to_tensor
    P.hydra_set_fwd_short_len(short_len)
    lengths, h = [31, 300, 64], 2
    cu = hw.cu_seqlens(lengths)
    T = int(cu[-1])
    x = rand_inputs(q_start + k_len, T, h)
    pair = dict(seq=1, q_start=q_start, q_len=q_len, k_start=k_start, k_len=k_len, part_row=3, group=0)
    step = AttnStep(cu, h, [pair], q_len + 5)
    step.o_part.fill_(float("nan"))
    step.lse_part.fill_(float("nan"))
    q, k, v = (bits_to_tensor(x[n]) for n in ("q", "k", "v"))
    P.hydra_attn_fwd(q, k, v, cu, h, step.pairs, True, step.scale, step.out, step.lse, step.o_part, step.lse_part,
                     q_len + 5, step.workspace)
    assert step.poll()[0] == 0
    ref_o, ref_l = oracle.attn_partial(x["q"], x["k"], x["v"], cu, pair, True, np.float32(step.scale))
    got_o = step.o_part.float().cpu().numpy().astype(np.float64)
    got_l = step.lse_part.cpu().numpy().astype(np.float64)
    assert np.isnan(got_l[:, :3]).all() and np.isnan(got_l[:, 3 + q_len:]).all(), "rows outside the pair were written"
    o, l = got_o[3:3 + q_len], got_l[:, 3:3 + q_len]
    assert np.array_equal(np.isneginf(l), np.isneginf(ref_l)), "which rows see no key"
    fin = np.isfinite(ref_l)
    if fin.any():
        assert np.abs(l[fin] - ref_l[fin]).max() <= TOL_LSE
    assert np.abs(o - ref_o).max() <= TOL_REL * max(np.abs(ref_o).max(), 1e-30) + 0.0
    assert (o[np.isneginf(ref_l).T] == 0).all()
