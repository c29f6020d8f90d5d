"""The banded backward: problems whose dS hand-off buffer is over the limit run as bands of key rows, each
with its own hand-off; dk and dv of a band are final, dq is summed in fp32 over the bands and rounded once.
Checked against the fp64 oracle with the same tolerance as the one-shot forms, and against the one-shot
hand-off itself."""
import numpy as np
import pytest

import hydra_workloads as hw
from gpu_util import check, pairs_for, run_gpu, run_oracle

pytestmark = pytest.mark.gpu
DQK, DV = hw.D_QK, hw.D_V


def rand_inputs(rng, T, h):
    f = lambda d: hw.f32_to_bf16_bits(rng.standard_normal((T, h, d)).astype(np.float32))
    return dict(q=f(DQK), k=f(DQK), v=f(DV), do=f(DV))


@pytest.fixture
def banded():
    """dS limit of 1 MiB (so that small problems are 'too long') and 1 MiB of band scratch."""
    import paper_2609_34318_b200 as P
    P.hydra_set_bwd_scratch_limit(1 << 20)
    P.hydra_set_bwd_band_scratch(1 << 20)
    yield P
    P.hydra_set_bwd_scratch_limit(4 << 30)
    P.hydra_set_bwd_band_scratch(P.HYDRA_BAND_AUTO)


@pytest.mark.parametrize("lengths,h,cp_r", [([1000], 2, 0), ([1500], 2, 2), ([700, 130, 64, 900], 2, [1, 0, 0, 2]),
                                            ([2047], 1, 1), ([129, 1, 640], 3, 0)])
def test_banded_backward_matches_the_oracle(banded, lengths, h, cp_r):
    P = banded
    cu = hw.cu_seqlens(lengths)
    x = rand_inputs(np.random.default_rng(7), int(cu[-1]), h)
    lib_pairs, rows, ora_pairs = pairs_for(cu, cp_r) if cp_r else (None, 0, None)
    _, _, n_bands = P.hydra_bwd_bands(cu, h, lib_pairs, True, 1 << 20)
    launches0 = P.hydra_launch_count()
    got = run_gpu(x, cu, h, lib_pairs, rows, True)
    launches = P.hydra_launch_count() - launches0
    if sum(L * L for L in lengths) * h > 1 << 20:
        assert n_bands >= 2
        # forward (+ merge) + prep + two kernels per band + the cast of dq: the bands really ran
        assert launches >= 1 + 1 + 2 * n_bands + 1
    check(got, run_oracle(x, cu, True, pairs=ora_pairs), label=f"banded {lengths}: ")


def test_banded_and_one_shot_backward_agree(banded):
    P = banded
    lengths, h = [1400, 300], 2
    cu = hw.cu_seqlens(lengths)
    x = rand_inputs(np.random.default_rng(8), int(cu[-1]), h)
    got_b = run_gpu(x, cu, h)
    P.hydra_set_bwd_scratch_limit(4 << 30)
    got_o = run_gpu(x, cu, h)
    for n in ("dq", "dk", "dv"):
        scale = np.abs(got_o[n]).max()
        assert np.abs(got_b[n] - got_o[n]).max() <= 2 ** -7 * scale, n
    # a key tile belongs to one band: the same products in the same order
    assert np.array_equal(got_b["dk"], got_o["dk"]) and np.array_equal(got_b["dv"], got_o["dv"])


def test_banded_backward_non_causal(banded):
    P = banded
    lengths, h = [900, 200], 2
    cu = hw.cu_seqlens(lengths)
    x = rand_inputs(np.random.default_rng(9), int(cu[-1]), h)
    from paper_2609_34318_b200.runner import AttnStep, bits_to_tensor
    step = AttnStep(cu, h, None, 0, False, None)
    q, k, v, do = (bits_to_tensor(x[n]) for n in ("q", "k", "v", "do"))
    for t in (step.dq, step.dk, step.dv):
        t.fill_(float("nan"))
    step.forward(q, k, v)
    n0 = P.hydra_launch_count()
    step.backward(q, k, v, do)
    assert P.hydra_launch_count() - n0 > 6
    status, detail = step.poll()
    assert status == 0, (status, detail)
    T = int(cu[-1])
    got = {n: getattr(step, n)[:T].float().cpu().numpy().astype(np.float64) for n in ("out", "dq", "dk", "dv")}
    got["lse"] = step.lse[:, :T].cpu().numpy().astype(np.float64)
    check(got, run_oracle(x, cu, False), label="banded non-causal: ")


@pytest.mark.parametrize("seed", range(8))
def test_banded_backward_random_mixes(banded, seed):
    """Random length mixes and ring degrees with a random scratch between 1 and 3 MiB: whatever the bands
    turn out to be (or if the problem is small enough to need none), the result is the oracle's."""
    P = banded
    rng = np.random.default_rng(500 + seed)
    n = int(rng.integers(1, 5))
    lengths = [int(v) for v in rng.choice([65, 128, 200, 383, 640, 777, 1025, 1500], size=n)]
    cp_r = [int(v) for v in rng.choice([0, 1, 2], size=n)]
    h = int(rng.integers(1, 4))
    P.hydra_set_bwd_band_scratch(int(rng.integers(1 << 20, 3 << 20)))
    cu = hw.cu_seqlens(lengths)
    x = rand_inputs(rng, int(cu[-1]), h)
    lib_pairs, rows, ora_pairs = pairs_for(cu, cp_r) if any(cp_r) else (None, 0, None)
    got = run_gpu(x, cu, h, lib_pairs, rows, True)
    check(got, run_oracle(x, cu, True, pairs=ora_pairs), label=f"banded mix {lengths} cp_r {cp_r} h {h}: ")
