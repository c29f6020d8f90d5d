"""The streaming form of the merge (`hydra_lse_merge_accumulate`): a ring engine folds the partials of
every ring step into the running (out, lse). Emulated on one GPU: the pairs of a zigzag ring are
processed step by step (all ranks' pairs of a step in one call), and the result must equal the
unchunked attention of the oracle (chunking and merging is an exact identity up to rounding).
"""
import numpy as np
import pytest

import hydra_workloads as hw
from gpu_util import TOL_LSE, TOL_REL, check, run_oracle

pytestmark = pytest.mark.gpu
DQK, DV = hw.D_QK, hw.D_V


def rand_inputs(rng, T, h):
    f = lambda d: hw.f32_to_bf16_bits(rng.standard_normal((T, h, d)).astype(np.float32))
    return dict(q=f(DQK), k=f(DQK), v=f(DV), do=f(DV))


@pytest.mark.parametrize("lengths,cp_r,h", [([1024, 300], 2, 3), ([2048], 4, 2), ([257, 64, 513], 1, 4)])
def test_ring_steps_accumulate_to_the_unchunked_result(lengths, cp_r, h):
    import torch
    import paper_2609_34318_b200 as P
    from paper_2609_34318_b200.runner import bits_to_tensor

    cu = hw.cu_seqlens(lengths)
    T = int(cu[-1])
    x = rand_inputs(np.random.default_rng(11 + cp_r), T, h)
    q, k, v = (bits_to_tensor(x[n]) for n in ("q", "k", "v"))
    pairs, _, rank, step = P.hydra_zigzag_pairs(cu, cp_r)
    scale = float(np.float32(1.0 / np.sqrt(np.float32(DQK))))
    out = torch.full((T, h, DV), float("nan"), dtype=torch.bfloat16, device="cuda")
    lse = torch.full((h, T), float("nan"), dtype=torch.float32, device="cuda")
    n_steps = int(step.max()) + 1
    assert n_steps == max(cp_r, 1)
    for t in range(n_steps):
        sel = pairs[step == t].copy()
        assert len(sel) > 0
        rows = 0
        for p in sel:                                   # every pair of the step writes a partial
            p["part_row"] = rows
            rows += int(p["q_len"])
        o_part = torch.full((rows, h, DV), float("nan"), dtype=torch.bfloat16, device="cuda")
        lse_part = torch.full((h, rows), float("nan"), dtype=torch.float32, device="cuda")
        ws = torch.empty(max(P.hydra_workspace_bytes(P.HYDRA_WS_FWD, cu, h, sel), 256), dtype=torch.uint8, device="cuda")
        P.hydra_attn_fwd(q, k, v, cu, h, sel, True, scale, out, lse, o_part, lse_part, rows, ws)
        if t == 0:
            P.hydra_lse_merge(o_part, lse_part, rows, cu, h, sel, out, lse, ws)
        else:
            P.hydra_lse_merge_accumulate(o_part, lse_part, rows, cu, h, sel, out, lse, ws)
    torch.cuda.synchronize()
    got = dict(out=out.float().cpu().numpy().astype(np.float64), lse=lse.cpu().numpy().astype(np.float64))
    ref = run_oracle(x, cu, True, backward=False)
    # every step rounds the running out to bf16 once more than the one-shot merge does
    check(got, ref, names=("out", "lse"), tol_rel=TOL_REL, tol_lse=TOL_LSE, label=f"ring steps cp_r={cp_r}: ")


def test_accumulate_leaves_other_rows_alone_and_matches_the_one_shot_merge():
    import torch
    import paper_2609_34318_b200 as P
    from paper_2609_34318_b200.runner import AttnStep, bits_to_tensor

    lengths, cp_r, h = [600, 200], 2, 2
    cu = hw.cu_seqlens(lengths)
    T = int(cu[-1])
    x = rand_inputs(np.random.default_rng(5), T, h)
    q, k, v = (bits_to_tensor(x[n]) for n in ("q", "k", "v"))
    pairs, part_rows, _, step = P.hydra_zigzag_pairs(cu, cp_r)
    one = AttnStep(cu, h, pairs, part_rows, True, None)
    one.forward(q, k, v)                                 # all pairs at once, one-shot merge
    scale = float(np.float32(1.0 / np.sqrt(np.float32(DQK))))
    # only the pairs of sequence 0, two steps; sequence 1's rows must keep their sentinel
    out = torch.full((T, h, DV), 7.0, dtype=torch.bfloat16, device="cuda")
    lse = torch.full((h, T), 7.0, dtype=torch.float32, device="cuda")
    for t in range(cp_r):
        sel = pairs[(step == t) & (pairs["seq"] == 0)].copy()
        rows = 0
        for p in sel:
            p["part_row"] = rows
            rows += int(p["q_len"])
        o_part = torch.empty((rows, h, DV), dtype=torch.bfloat16, device="cuda")
        lse_part = torch.empty((h, rows), dtype=torch.float32, device="cuda")
        ws = torch.empty(max(P.hydra_workspace_bytes(P.HYDRA_WS_FWD, cu, h, sel), 256), dtype=torch.uint8, device="cuda")
        P.hydra_attn_fwd(q, k, v, cu, h, sel, True, scale, out, lse, o_part, lse_part, rows, ws)
        (P.hydra_lse_merge if t == 0 else P.hydra_lse_merge_accumulate)(o_part, lse_part, rows, cu, h, sel, out, lse, ws)
    torch.cuda.synchronize()
    L0 = lengths[0]
    assert torch.all(out[L0:] == 7.0) and torch.all(lse[:, L0:] == 7.0)
    a, b = out[:L0].float(), one.out[:L0].float()
    assert (a - b).abs().max().item() <= 2 ** -7 * b.abs().max().item()      # one extra bf16 rounding
    assert (lse[:, :L0] - one.lse[:, :L0]).abs().max().item() <= 1e-5


# ------------------------------------------------------------------------------------------------
# backward, one ring step at a time: hydra_attn_bwd_accumulate + hydra_grad_cast
# ------------------------------------------------------------------------------------------------
def _bwd_by_steps(P, torch, x, cu, h, pairs, groups, one):
    """Runs the backward of `pairs` in the listed groups (boolean masks), accumulating in fp32."""
    from paper_2609_34318_b200.runner import bits_to_tensor
    T = int(cu[-1])
    q, k, v, do = (bits_to_tensor(x[n]) for n in ("q", "k", "v", "do"))
    scale = float(np.float32(1.0 / np.sqrt(np.float32(DQK))))
    acc = [torch.zeros((T, h, d), dtype=torch.float32, device="cuda") for d in (DQK, DQK, DV)]
    ws = torch.empty(P.hydra_workspace_bytes(P.HYDRA_WS_BWD, cu, h, pairs), dtype=torch.uint8, device="cuda")
    for mask in groups:
        sel = pairs[mask].copy()
        assert len(sel) > 0
        P.hydra_attn_bwd_accumulate(q, k, v, one.out, one.lse, do, cu, h, sel, True, scale, acc[0], acc[1],
                                    acc[2], ws)
        status, detail = P.hydra_poll_status(ws)
        assert status == 0, (status, detail)
    grads = [torch.full(a.shape, float("nan"), dtype=torch.bfloat16, device="cuda") for a in acc]
    for a, g in zip(acc, grads):
        P.hydra_grad_cast(a, g)
    torch.cuda.synchronize()
    return acc, grads


@pytest.mark.parametrize("lengths,cp_r,h", [([1024, 300], 2, 3), ([2048], 4, 2), ([257, 64, 513], 1, 4)])
def test_backward_ring_steps_accumulate_to_the_unchunked_gradients(lengths, cp_r, h):
    import torch
    import paper_2609_34318_b200 as P
    from paper_2609_34318_b200.runner import AttnStep, bits_to_tensor

    cu = hw.cu_seqlens(lengths)
    x = rand_inputs(np.random.default_rng(23 + cp_r), int(cu[-1]), h)
    pairs, part_rows, rank, step = P.hydra_zigzag_pairs(cu, cp_r)
    one = AttnStep(cu, h, pairs, part_rows, True, None)
    q, k, v, do = (bits_to_tensor(x[n]) for n in ("q", "k", "v", "do"))
    one.forward(q, k, v)                                 # merged out / lse of all pairs
    one.backward(q, k, v, do)                            # one-shot backward, for comparison
    n_ranks, n_steps = int(rank.max()) + 1, int(step.max()) + 1
    # one call per (rank, step): what a ring engine issues
    groups = [(rank == r) & (step == t) for t in range(n_steps) for r in range(n_ranks)]
    groups = [g for g in groups if g.any()]
    assert sum(int(g.sum()) for g in groups) == len(pairs)
    acc, grads = _bwd_by_steps(P, torch, x, cu, h, pairs, groups, one)
    got = {n: g.float().cpu().numpy().astype(np.float64) for n, g in zip(("dq", "dk", "dv"), grads)}
    ref = run_oracle(x, cu, True, backward=True)
    check(got, ref, names=("dq", "dk", "dv"), tol_rel=TOL_REL, label=f"bwd ring steps cp_r={cp_r}: ")
    # against the one-shot backward: same products, summed in fp32 in a different order, rounded once
    for name, g, o in zip(("dq", "dk", "dv"), grads, (one.dq, one.dk, one.dv)):
        g, o = g.float(), o[: g.shape[0]].float()
        assert (g - o).abs().max().item() <= 2 ** -6 * o.abs().max().item(), name
    # the cast is exactly round-to-nearest-even of the accumulator
    for a, g in zip(acc, grads):
        assert torch.equal(a.to(torch.bfloat16), g)


def test_backward_accumulate_adds_and_leaves_other_rows_alone():
    import torch
    import paper_2609_34318_b200 as P
    from paper_2609_34318_b200.runner import AttnStep, bits_to_tensor

    lengths, cp_r, h = [600, 200], 2, 2
    cu = hw.cu_seqlens(lengths)
    T = int(cu[-1])
    x = rand_inputs(np.random.default_rng(7), T, h)
    pairs, part_rows, _, _ = P.hydra_zigzag_pairs(cu, cp_r)
    one = AttnStep(cu, h, pairs, part_rows, True, None)
    q, k, v, do = (bits_to_tensor(x[n]) for n in ("q", "k", "v", "do"))
    one.forward(q, k, v)
    one.backward(q, k, v, do)
    scale = float(np.float32(1.0 / np.sqrt(np.float32(DQK))))
    sel = pairs[pairs["seq"] == 0].copy()                # sequence 0 only; accumulators preloaded with 3
    acc = [torch.full((T, h, d), 3.0, dtype=torch.float32, device="cuda") for d in (DQK, DQK, DV)]
    ws = torch.empty(P.hydra_workspace_bytes(P.HYDRA_WS_BWD, cu, h, sel), dtype=torch.uint8, device="cuda")
    P.hydra_attn_bwd_accumulate(q, k, v, one.out, one.lse, do, cu, h, sel, True, scale, acc[0], acc[1], acc[2], ws)
    torch.cuda.synchronize()
    L0 = lengths[0]
    for a, o in zip(acc, (one.dq, one.dk, one.dv)):
        assert torch.all(a[L0:] == 3.0)                  # rows of sequence 1 untouched
        d = (a[:L0] - 3.0) - o[:L0].float()              # what was added = the one-shot gradient (bf16-rounded there)
        assert d.abs().max().item() <= 2 ** -7 * o[:L0].float().abs().max().item() + 1e-5


def test_grad_cast_ragged_sizes_and_arguments():
    import torch
    import paper_2609_34318_b200 as P

    g = torch.Generator(device="cuda"); g.manual_seed(3)
    for n in (0, 1, 7, 8, 9, 4099, 1 << 20):
        a = torch.randn(n + 8, device="cuda", generator=g) * 100
        out = torch.full((n + 8,), 5.0, dtype=torch.bfloat16, device="cuda")
        P.hydra_grad_cast(a, out, n)
        torch.cuda.synchronize()
        assert torch.equal(out[:n], a[:n].to(torch.bfloat16))
        assert torch.all(out[n:] == 5.0)
    a = torch.zeros(16, device="cuda")
    assert P.hydra_grad_cast(a, a, -1, check=False) == P.HYDRA_ERR_INVALID_ARG
    assert P.hydra_grad_cast(0, a, 8, check=False) == P.HYDRA_ERR_INVALID_ARG


def test_clock_probe_reports_a_plausible_sm_clock():
    import torch
    import paper_2609_34318_b200 as P
    from paper_2609_34318_b200.runner import AttnStep, bits_to_tensor

    cu = hw.cu_seqlens([2048, 700])
    x = rand_inputs(np.random.default_rng(1), int(cu[-1]), 2)
    q, k, v, do = (bits_to_tensor(x[n]) for n in ("q", "k", "v", "do"))
    step = AttnStep(cu, 2, None, 0, True, None)
    step.forward(q, k, v)
    fwd = P.hydra_poll_clocks(step.workspace)
    step.backward(q, k, v, do)
    bwd = P.hydra_poll_clocks(step.workspace)
    assert 300.0 < fwd[0] < 2500.0 and fwd[1] == 0.0 and fwd[2] == 0.0
    assert bwd[0] == 0.0 and 300.0 < bwd[1] < 2500.0 and 300.0 < bwd[2] < 2500.0
