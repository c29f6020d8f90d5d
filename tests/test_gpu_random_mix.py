"""Seeded random problems across the entry points, checked against the fp64 oracle.

Each seed draws a path (heads of 192 / 128 per head, the same grouped, heads of 128 / 128), a mix of sequence
lengths (tiny, short, mixed, long, or sitting on tile edges; empty sequences included), a ring degree per sequence
(Section 5.2: 0 = not cut, else 2 * cp_r zigzag chunks and the merge), the backward form (dS hand-off, recomputing,
banded) and the routing between the two forward kernels. The fixed cases of the other files pin the known corners;
this one guards the combinations nobody thought of.
"""
import numpy as np
import pytest

import hydra_workloads as hw
import oracle
import test_gpu_gqa as grouped
import test_gpu_head_dims as d128
from conftest import FWD_SHORT_LEN_DEFAULT
from gpu_util import check, pairs_for, run_gpu, run_oracle

pytestmark = pytest.mark.gpu


@pytest.fixture
def settings():
    import paper_2609_34318_b200 as P
    yield P
    P.hydra_set_bwd_scratch_limit(4 << 30)
    P.hydra_set_bwd_band_scratch(P.HYDRA_BAND_AUTO)
    P.hydra_set_fwd_short_len(FWD_SHORT_LEN_DEFAULT)


def draw_lengths(rng):
    style = rng.choice(["tiny", "short", "mixed", "long"])
    top = {"tiny": 40, "short": 300, "mixed": 900, "long": 2600}[style]
    n = int(rng.integers(1, 4 if style == "long" else 9))
    lengths = [int(v) for v in rng.integers(0 if rng.random() < 0.3 else 1, top, size=n)]
    if rng.random() < 0.3:
        lengths = [int(rng.choice([63, 64, 65, 127, 128, 129, 255, 256, 257, 511, 512, 513])) for _ in lengths]
    if sum(lengths) == 0:
        lengths.append(5)
    return lengths


@pytest.mark.parametrize("seed", range(48))
def test_random_problem_matches_the_oracle(settings, seed):
    P = settings
    rng = np.random.default_rng(77000 + seed)
    kind = rng.choice(["per_head_192", "grouped_192", "heads_of_128"])
    lengths = draw_lengths(rng)
    cp_r = [int(v) for v in rng.choice([0, 0, 1, 2, 3, 4], size=len(lengths))]
    form = rng.choice(["hand_off", "recompute", "banded"])
    short_len = int(rng.choice([FWD_SHORT_LEN_DEFAULT, 0, 1 << 20, 256]))
    P.hydra_set_fwd_short_len(short_len)
    if form == "recompute":
        P.hydra_set_bwd_scratch_limit(0)
    elif form == "banded":
        P.hydra_set_bwd_scratch_limit(1 << 20)
        P.hydra_set_bwd_band_scratch(1 << 20)
    cu = hw.cu_seqlens(lengths)
    T = int(cu[-1])
    lib_pairs, rows, ora_pairs = pairs_for(cu, cp_r) if any(cp_r) else (None, 0, None)
    label = f"seed {seed} {kind} {lengths} ring {cp_r} {form} short_len {short_len}: "
    if kind == "per_head_192":
        h = int(rng.integers(1, 5))
        f = lambda d: hw.f32_to_bf16_bits(rng.standard_normal((T, h, d)).astype(np.float32))
        x = dict(q=f(hw.D_QK), k=f(hw.D_QK), v=f(hw.D_V), do=f(hw.D_V))
        got = run_gpu(x, cu, h, lib_pairs, rows, True)
        ref = run_oracle(x, cu, True, pairs=ora_pairs)
    else:
        h_kv = int(rng.integers(1, 3))
        h = h_kv * int(rng.choice([1, 2, 4]))
        if kind == "grouped_192":
            x = grouped.inputs(rng, T, h, h_kv)
            got = grouped.run_gpu_gqa(x, cu, h, h_kv, lib_pairs, rows)
            scale = np.float32(1.0 / np.sqrt(np.float32(hw.D_QK)))
            out, lse = oracle.attn_fwd_gqa(x["q"], x["k"], x["v"], cu, True, scale)
            if ora_pairs is None:
                dq, dk, dv = oracle.attn_bwd_gqa(x["q"], x["k"], x["v"], x["do"], cu, True, scale, out, lse)
            else:
                dq, dk, dv = oracle.attn_bwd_pairs_gqa(x["q"], x["k"], x["v"], x["do"], cu, ora_pairs, True, scale, lse,
                                                       oracle.bwd_prep(x["do"], out))
            ref = dict(out=out, lse=lse, dq=dq, dk=dk, dv=dv)
        else:
            x = d128.inputs(rng, T, h, h_kv)
            got = d128.run_d128(x, cu, h, h_kv, lib_pairs, rows, accumulate=bool(rng.random() < 0.5))
            ref = d128.reference(x, cu, ora_pairs)
    check(got, ref, label=label)
