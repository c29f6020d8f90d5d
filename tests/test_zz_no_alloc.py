"""hydra_lse_merge_noalloc against hydra_lse_merge.

The no-alloc entry point exists for callers that cannot call cudaMalloc (a process that gave all
device memory to its own pool, or a loop whose rules forbid a call that may synchronise the device).
It must give what the ordinary merge gives. Both run the same kernel on the same partials, so the
results are expected to agree to the bit; the comparison still uses the suite's tolerances.
Two calls in a row, on different problems, check that the shared table array is rewritten each time.
This file sorts last on purpose: a run that stops at the first failure has then run everything else.
"""
import numpy as np
import pytest
import torch

import hydra_workloads as hw
from gpu_util import TOL_LSE, TOL_REL

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


def _merge_both_ways(lengths, h, cp_r, seed):
    P, cu, pairs, part_rows, step = _partials(lengths, h, cp_r, seed)
    merged = np.zeros(int(cu[-1]), dtype=bool)
    for p in pairs:
        if p["part_row"] >= 0:
            t0 = int(cu[p["seq"]]) + int(p["q_start"])
            merged[t0:t0 + int(p["q_len"])] = True
    assert merged.any()
    out_a, lse_a = torch.full_like(step.out, float("nan")), torch.full_like(step.lse, float("nan"))
    out_b, lse_b = torch.full_like(step.out, float("nan")), torch.full_like(step.lse, float("nan"))
    P.hydra_lse_merge(step.o_part, step.lse_part, part_rows, cu, h, pairs, out_a, lse_a, step.workspace)
    P.hydra_lse_merge_noalloc(step.o_part, step.lse_part, part_rows, cu, h, pairs, out_b, lse_b)
    torch.cuda.synchronize()
    idx = torch.from_numpy(np.nonzero(merged)[0]).cuda()
    a, b = out_a[idx].float().cpu().numpy(), out_b[idx].float().cpu().numpy()
    la, lb = lse_a[:, idx].cpu().numpy(), lse_b[:, idx].cpu().numpy()
    assert np.isfinite(b).all() and np.isfinite(lb).all()
    assert np.abs(a - b).max() <= TOL_REL * np.abs(a).max()
    assert np.abs(la - lb).max() <= TOL_LSE
    # rows of chunks that have a single pair are not the merge's business: both leave them alone
    rest = torch.from_numpy(np.nonzero(~merged)[0]).cuda()
    if len(rest):
        assert torch.isnan(out_b[rest].float()).all()


def test_no_alloc_merge_matches_the_ordinary_merge_twice_in_a_row():
    _merge_both_ways([300, 77, 1001], 4, 1, seed=11)        # three chunked sequences, two chunks each
    _merge_both_ways([2000, 5, 640], 3, 4, seed=12)         # a different problem: ring of four


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
