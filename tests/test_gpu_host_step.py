"""The whole step through the C ABI with HOST buffers (`hydra_attn_fwd_bwd_host`) against the oracle.

The entry point pipelines groups over two internal copy streams: runs of whole sequences when every sequence is
small against the step, ranges of heads over all sequences otherwise. The cases cover a head count that splits
into full groups plus a remainder, a single group, a step of many short sequences (groups of sequences, one of
them empty), chunked pairs through the merge in both forms, and two calls in a row on the same arena (the
internal streams and events are reused).
"""
import numpy as np
import pytest

import hydra_workloads as hw
from gpu_util import check, pairs_for, run_oracle

pytestmark = pytest.mark.gpu
DQK, DV = hw.D_QK, hw.D_V


def rand_inputs(rng, T, h):
    f = lambda d: hw.f32_to_bf16_bits(rng.standard_normal((T, h, d)).astype(np.float32))
    return dict(q=f(DQK), k=f(DQK), v=f(DV), do=f(DV))


def host_step(x, cu, h, lib_pairs, calls=1):
    import torch
    import paper_2609_34318_b200 as P
    from paper_2609_34318_b200.runner import bits_to_tensor
    T = int(cu[-1])
    host = {n: bits_to_tensor(x[n]).cpu().pin_memory() for n in ("q", "k", "v", "do")}
    nan16 = lambda d: torch.full((T, h, d), float("nan"), dtype=torch.bfloat16).pin_memory()
    ho = dict(out=nan16(DV), lse=torch.full((h, T), float("nan"), dtype=torch.float32).pin_memory(),
              dq=nan16(DQK), dk=nan16(DQK), dv=nan16(DV))
    arena = torch.empty(P.hydra_host_step_arena_bytes(cu, h, lib_pairs) + 256, dtype=torch.uint8, device="cuda")
    off = (-arena.data_ptr()) % 256
    scale = float(np.float32(1.0 / np.sqrt(np.float32(DQK))))
    for _ in range(calls):
        P.hydra_attn_fwd_bwd_host(host["q"], host["k"], host["v"], host["do"], cu, h, lib_pairs, True, scale,
                                  ho["out"], ho["lse"], ho["dq"], ho["dk"], ho["dv"],
                                  arena.data_ptr() + off, arena.numel() - off)
    torch.cuda.synchronize()
    return {n: t.float().numpy().astype(np.float64) for n, t in ho.items()}


@pytest.mark.parametrize("h,cp_r", [(9, 0), (3, 0), (8, 1), (6, 2)])
def test_host_step_matches_the_oracle(h, cp_r):
    lengths = [130, 257, 64, 1, 300]
    cu = hw.cu_seqlens(lengths)
    x = rand_inputs(np.random.default_rng(100 + h), int(cu[-1]), h)
    lib_pairs, _, ora_pairs = pairs_for(cu, cp_r) if cp_r else (None, 0, None)
    got = host_step(x, cu, h, lib_pairs)
    ref = run_oracle(x, cu, True, pairs=ora_pairs)
    check(got, ref, label=f"host step h={h} cp_r={cp_r}: ")


@pytest.mark.parametrize("h,cp_r", [(8, 0), (6, 1), (5, 0)])
def test_host_step_in_groups_of_sequences(h, cp_r):
    """Many short sequences, none over a group's share of the step: runs of sequences travel as contiguous token
    ranges with all heads (about 16 groups here); a sequence without tokens sits inside one of them."""
    lengths = [5] * 60 + [0] + [17, 40, 3] * 12 + [90] * 6
    cu = hw.cu_seqlens(lengths)
    x = rand_inputs(np.random.default_rng(300 + h), int(cu[-1]), h)
    lib_pairs, _, ora_pairs = pairs_for(cu, cp_r) if cp_r else (None, 0, None)
    got = host_step(x, cu, h, lib_pairs)
    ref = run_oracle(x, cu, True, pairs=ora_pairs)
    check(got, ref, label=f"host step in groups of sequences h={h} cp_r={cp_r}: ")


@pytest.mark.parametrize("seed", range(10))
def test_random_host_steps(seed):
    """Seeded mixes: many short sequences (groups of sequences), short ones around a long one and a few long ones
    (groups of heads), 1 to 12 heads, some sequences cut into zigzag chunks."""
    rng = np.random.default_rng(5000 + seed)
    style = ["many_short", "mixed", "few"][seed % 3]
    if style == "many_short":
        lengths = [int(v) for v in rng.integers(0, 120, size=int(rng.integers(20, 120)))]
    elif style == "mixed":
        lengths = [int(v) for v in rng.integers(1, 200, size=int(rng.integers(5, 40)))] + [int(rng.integers(300, 1500))]
        lengths = [lengths[i] for i in rng.permutation(len(lengths))]
    else:
        lengths = [int(v) for v in rng.integers(1, 900, size=int(rng.integers(1, 4)))]
    if sum(lengths) == 0:
        lengths.append(3)
    h = int(rng.integers(1, 13))
    cp_r = [int(v) for v in rng.choice([0, 0, 0, 1, 2], size=len(lengths))]
    cu = hw.cu_seqlens(lengths)
    x = rand_inputs(rng, int(cu[-1]), h)
    lib_pairs, _, ora_pairs = pairs_for(cu, cp_r) if any(cp_r) else (None, 0, None)
    got = host_step(x, cu, h, lib_pairs)
    check(got, run_oracle(x, cu, True, pairs=ora_pairs), label=f"host step seed {seed} ({style}, h={h}): ")


def test_two_host_steps_in_a_row_give_the_same_bits():
    cu = hw.cu_seqlens([200, 513])
    x = rand_inputs(np.random.default_rng(7), int(cu[-1]), 12)
    once = host_step(x, cu, 12, None, calls=1)
    twice = host_step(x, cu, 12, None, calls=2)
    for n in once:
        assert np.array_equal(once[n], twice[n], equal_nan=True), n
