"""hydra_lse_merge_noalloc against hydra_lse_merge and against the oracle's merge.

The no-alloc entry point exists for callers that cannot call cudaMalloc (a process that gave all
device memory to its own pool, or a loop whose rules forbid a call that may synchronise the device).
It must give what the ordinary merge gives: both are compared on the same partials with the suite's
tolerances, and the no-alloc result is also compared, element by element, with the fp64 oracle's merge of
those same partials (the two GPU entry points share a kernel, so agreeing with each other proves little).
Two calls in a row, on different problems, check that the shared table array is rewritten each time, and
the device's free memory must be the same before and after the second call: the property the entry point
exists for. This file sorts last on purpose: a run that stops at the first failure has then run
everything else.
"""
import numpy as np
import pytest
import torch

import hydra_workloads as hw
import oracle
from gpu_util import TOL_LSE, TOL_REL, oracle_merge_of_partials

pytestmark = pytest.mark.gpu


def _partials(lengths, h, cp_r, seed):
    """Run the forward on zigzag pairs and return everything the two merges need."""
    import paper_2609_34318_b200 as P
    from paper_2609_34318_b200.runner import AttnStep, bits_to_tensor
    rng = np.random.default_rng(seed)
    cu = hw.cu_seqlens(lengths)
    T = int(cu[-1])
    pairs, part_rows, _, _ = P.hydra_zigzag_pairs(cu, cp_r)
    step = AttnStep(cu, h, pairs, part_rows)
    mk = lambda d: bits_to_tensor(hw.f32_to_bf16_bits(rng.standard_normal((T, h, d)).astype(np.float32)))
    q, k, v = mk(hw.D_QK), mk(hw.D_QK), mk(hw.D_V)
    P.hydra_attn_fwd(q, k, v, cu, h, pairs, True, step.scale, step.out, step.lse, step.o_part, step.lse_part,
                     part_rows, step.workspace)
    torch.cuda.synchronize()
    return P, cu, pairs, part_rows, step


def _merge_both_ways(lengths, h, cp_r, seed, memory_must_stay_flat):
    P, cu, pairs, part_rows, step = _partials(lengths, h, cp_r, seed)
    T = int(cu[-1])
    merged = np.zeros(T, dtype=bool)
    for p in pairs:
        if p["part_row"] >= 0:
            t0 = int(cu[p["seq"]]) + int(p["q_start"])
            merged[t0:t0 + int(p["q_len"])] = True
    assert merged.any()
    out_a, lse_a = torch.full_like(step.out, float("nan")), torch.full_like(step.lse, float("nan"))
    out_b, lse_b = torch.full_like(step.out, float("nan")), torch.full_like(step.lse, float("nan"))
    P.hydra_lse_merge(step.o_part, step.lse_part, part_rows, cu, h, pairs, out_a, lse_a, step.workspace)
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    launches_before = P.hydra_launch_count()
    P.hydra_lse_merge_noalloc(step.o_part, step.lse_part, part_rows, cu, h, pairs, out_b, lse_b)
    torch.cuda.synchronize()
    free_after = torch.cuda.mem_get_info()[0]
    assert P.hydra_launch_count() == launches_before + 1          # counted like every other launch
    if memory_must_stay_flat:
        # the first call on a device may make the driver load the module's data; from the second call
        # on, the device's free memory must not move at all
        assert free_after == free_before, (free_before, free_after)
    idx = torch.from_numpy(np.nonzero(merged)[0]).cuda()
    a, b = out_a[idx].float().cpu().numpy(), out_b[idx].float().cpu().numpy()
    la, lb = lse_a[:, idx].cpu().numpy(), lse_b[:, idx].cpu().numpy()
    assert np.isfinite(b).all() and np.isfinite(lb).all()
    assert np.abs(a - b).max() <= TOL_REL * np.abs(a).max()
    assert np.abs(la - lb).max() <= TOL_LSE
    # against the oracle's merge of the same partials, element by element
    ref_o, ref_l = oracle_merge_of_partials(cu, pairs, step.o_part, step.lse_part, T, h)
    rows = np.nonzero(merged)[0]
    got_o = out_b.float().cpu().numpy().astype(np.float64)[rows]
    got_l = lse_b.cpu().numpy().astype(np.float64)[:, rows]
    assert np.abs(got_o - ref_o[rows]).max() <= TOL_REL * np.abs(ref_o[rows]).max()
    assert np.abs(got_l - ref_l[:, rows]).max() <= TOL_LSE
    # rows of chunks that have a single pair are not the merge's business: both leave them alone
    rest = torch.from_numpy(np.nonzero(~merged)[0]).cuda()
    if len(rest):
        assert torch.isnan(out_b[rest].float()).all()


def test_no_alloc_merge_matches_the_ordinary_merge_twice_in_a_row():
    _merge_both_ways([300, 77, 1001], 4, 1, seed=11, memory_must_stay_flat=False)   # two chunks per sequence
    _merge_both_ways([2000, 5, 640], 3, 4, seed=12, memory_must_stay_flat=True)     # another problem: ring of 4


def test_no_alloc_merge_rejects_what_exceeds_its_fixed_tables():
    import paper_2609_34318_b200 as P
    # more merged q chunks than the fixed tables hold: refused with a clear status, nothing launched
    n = 2049
    lengths = [16] * n
    cu = hw.cu_seqlens(lengths)
    pairs, part_rows, _, _ = P.hydra_zigzag_pairs(cu, 1)
    dummy = torch.zeros(16, dtype=torch.uint8, device="cuda")
    s = P.hydra_lse_merge_noalloc(dummy, dummy, part_rows, cu, 1, pairs, dummy, dummy, check=False)
    assert s == P.HYDRA_ERR_UNSUPPORTED
    assert P.hydra_status_string(s) == "HYDRA_ERR_UNSUPPORTED"


def test_no_alloc_merge_rejects_overlapping_rows_like_the_ordinary_merge():
    import paper_2609_34318_b200 as P
    cu = hw.cu_seqlens([64])
    pairs, part_rows, _, _ = P.hydra_zigzag_pairs(cu, 1)
    dummy = torch.zeros(1 << 16, dtype=torch.uint8, device="cuda")
    n0 = P.hydra_launch_count()
    bad = pairs.copy()
    merged = np.nonzero(bad["part_row"] >= 0)[0]
    assert len(merged) >= 2
    bad["part_row"][merged[1]] = bad["part_row"][merged[0]]          # two partials on the same rows
    for fn, extra in ((P.hydra_lse_merge_noalloc, ()), (P.hydra_lse_merge, (dummy,))):
        s = fn(dummy, dummy, part_rows, cu, 1, bad, dummy, dummy, *extra, check=False)
        assert s == P.HYDRA_ERR_INVALID_ARG, (fn.__name__, s)
    assert P.hydra_launch_count() == n0


@pytest.mark.parametrize("lengths,cp_r", [([1], 3), ([1, 1, 1], 2)])
def test_no_alloc_merge_with_nothing_to_merge_is_a_no_op_like_the_ordinary_merge(lengths, cp_r):
    """One-token sequences: every q chunk that exists has a single pair, which wrote out / lse itself. Both
    entry points return OK without a launch and without touching anything, whatever the partial buffers are."""
    import paper_2609_34318_b200 as P
    cu = hw.cu_seqlens(lengths)
    T = int(cu[-1])
    pairs, part_rows, _, _ = P.hydra_zigzag_pairs(cu, cp_r)
    assert part_rows == 0 and (pairs["part_row"] < 0).all()
    out = torch.full((T, 2, hw.D_V), float("nan"), dtype=torch.bfloat16, device="cuda")
    lse = torch.full((2, T), float("nan"), dtype=torch.float32, device="cuda")
    ws = torch.zeros(4096, dtype=torch.uint8, device="cuda")
    n0 = P.hydra_launch_count()
    assert P.hydra_lse_merge(None, None, 0, cu, 2, pairs, out, lse, ws, check=False) == P.HYDRA_OK
    assert P.hydra_lse_merge_noalloc(None, None, 0, cu, 2, pairs, out, lse, check=False) == P.HYDRA_OK
    torch.cuda.synchronize()
    assert P.hydra_launch_count() == n0
    assert torch.isnan(out.float()).all() and torch.isnan(lse).all()
