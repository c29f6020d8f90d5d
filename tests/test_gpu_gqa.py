"""Grouped-query attention (shared KV heads) on the GPU against the oracle: forward, merge of cut sequences,
and the accumulating backward whose dk / dv rows sum over the query heads of a group. Same tolerances as the
per-head path."""
import numpy as np
import pytest

import hydra_workloads as hw
import oracle
from gpu_util import check, pairs_for

pytestmark = [pytest.mark.gpu, pytest.mark.usefixtures("both_forward_kernels")]
DQK, DV = hw.D_QK, hw.D_V


@pytest.fixture(params=["hand_off", "recompute"])
def backward_form(request):
    import paper_2609_34318_b200 as P
    P.hydra_set_bwd_scratch_limit(0 if request.param == "recompute" else 4 << 30)
    yield request.param
    P.hydra_set_bwd_scratch_limit(4 << 30)


def inputs(rng, T, h, h_kv):
    f = lambda heads, d: hw.f32_to_bf16_bits(rng.standard_normal((T, heads, d)).astype(np.float32))
    return dict(q=f(h, DQK), k=f(h_kv, DQK), v=f(h_kv, DV), do=f(h, DV))


def run_gpu_gqa(x, cu, h, h_kv, lib_pairs, part_rows, causal=True):
    import torch
    import paper_2609_34318_b200 as P
    from paper_2609_34318_b200.runner import bits_to_tensor
    T = int(cu[-1])
    scale = float(np.float32(1.0 / np.sqrt(np.float32(DQK))))
    q, k, v, do = (bits_to_tensor(x[n]) for n in ("q", "k", "v", "do"))
    bf, f32 = torch.bfloat16, torch.float32
    out = torch.full((T, h, DV), float("nan"), dtype=bf, device="cuda")
    lse = torch.full((h, T), float("nan"), dtype=f32, device="cuda")
    o_part = torch.full((max(part_rows, 1), h, DV), float("nan"), dtype=bf, device="cuda")
    lse_part = torch.full((h, max(part_rows, 1)), float("nan"), dtype=f32, device="cuda")
    ws = torch.empty(max(P.hydra_workspace_bytes(w, cu, h, lib_pairs) for w in (P.HYDRA_WS_FWD, P.HYDRA_WS_BWD)),
                     dtype=torch.uint8, device="cuda")
    has_parts = lib_pairs is not None and bool((lib_pairs["part_row"] >= 0).any())
    P.hydra_attn_fwd_gqa(q, k, v, cu, h, h_kv, lib_pairs, causal, scale, out, lse,
                         o_part if has_parts else None, lse_part if has_parts else None, part_rows, ws)
    if has_parts:
        P.hydra_lse_merge(o_part, lse_part, part_rows, cu, h, lib_pairs, out, lse, ws)
    acc = [torch.zeros((T, heads, d), dtype=f32, device="cuda") for heads, d in ((h, DQK), (h_kv, DQK), (h_kv, DV))]
    P.hydra_attn_bwd_accumulate_gqa(q, k, v, out, lse, do, cu, h, h_kv, lib_pairs, causal, scale, acc[0], acc[1],
                                    acc[2], ws)
    grads = [torch.empty(a.shape, dtype=bf, device="cuda") for a in acc]
    for a, g in zip(acc, grads):
        P.hydra_grad_cast(a, g)
    status, detail = P.hydra_poll_status(ws)
    assert status == 0, (status, detail)
    f64 = lambda t: t.float().cpu().numpy().astype(np.float64)
    return dict(out=f64(out), lse=f64(lse), dq=f64(grads[0]), dk=f64(grads[1]), dv=f64(grads[2]))


@pytest.mark.parametrize("lengths,h,h_kv,cp_r", [
    ([300, 129, 64], 4, 2, 0), ([700], 6, 1, 0), ([640, 200], 8, 2, 2), ([257], 4, 4, 0), ([1, 130, 513], 8, 4, 1)])
def test_gqa_forward_and_backward_match_the_oracle(backward_form, lengths, h, h_kv, cp_r):
    cu = hw.cu_seqlens(lengths)
    x = inputs(np.random.default_rng(11 + h + h_kv), int(cu[-1]), h, h_kv)
    lib_pairs, rows, ora_pairs = pairs_for(cu, cp_r) if cp_r else (None, 0, None)
    got = run_gpu_gqa(x, cu, h, h_kv, lib_pairs, rows)
    scale = np.float32(1.0 / np.sqrt(np.float32(DQK)))
    out, lse = oracle.attn_fwd_gqa(x["q"], x["k"], x["v"], cu, True, scale)
    if ora_pairs is None:
        dq, dk, dv = oracle.attn_bwd_gqa(x["q"], x["k"], x["v"], x["do"], cu, True, scale, out, lse)
    else:
        d = oracle.bwd_prep(x["do"], out)
        dq, dk, dv = oracle.attn_bwd_pairs_gqa(x["q"], x["k"], x["v"], x["do"], cu, ora_pairs, True, scale, lse, d)
    check(got, dict(out=out, lse=lse, dq=dq, dk=dk, dv=dv), label=f"gqa {lengths} h={h}/{h_kv}: ")


@pytest.mark.parametrize("lengths,h,h_kv,cp_r", [([300, 129, 64], 4, 2, 0), ([640, 200], 8, 1, 2)])
def test_gqa_one_shot_backward_matches_the_oracle(backward_form, lengths, h, h_kv, cp_r):
    import torch
    import paper_2609_34318_b200 as P
    from paper_2609_34318_b200.runner import bits_to_tensor
    cu = hw.cu_seqlens(lengths)
    T = int(cu[-1])
    x = inputs(np.random.default_rng(23), T, h, h_kv)
    lib_pairs, rows, ora_pairs = pairs_for(cu, cp_r) if cp_r else (None, 0, None)
    scale = float(np.float32(1.0 / np.sqrt(np.float32(DQK))))
    q, k, v, do = (bits_to_tensor(x[n]) for n in ("q", "k", "v", "do"))
    bf = torch.bfloat16
    out = torch.empty((T, h, DV), dtype=bf, device="cuda")
    lse = torch.empty((h, T), dtype=torch.float32, device="cuda")
    o_part = torch.empty((max(rows, 1), h, DV), dtype=bf, device="cuda")
    lse_part = torch.empty((h, max(rows, 1)), dtype=torch.float32, device="cuda")
    need = P.hydra_workspace_bytes_gqa(P.HYDRA_WS_BWD, cu, h, h_kv, lib_pairs)
    assert need >= P.hydra_workspace_bytes(P.HYDRA_WS_BWD, cu, h, lib_pairs) + T * h_kv * (DQK + DV) * 4
    ws = torch.empty(need, dtype=torch.uint8, device="cuda")
    has_parts = rows > 0
    P.hydra_attn_fwd_gqa(q, k, v, cu, h, h_kv, lib_pairs, True, scale, out, lse, o_part if has_parts else None,
                         lse_part if has_parts else None, rows, ws)
    if has_parts:
        P.hydra_lse_merge(o_part, lse_part, rows, cu, h, lib_pairs, out, lse, ws)
    dq = torch.full((T, h, DQK), float("nan"), dtype=bf, device="cuda")
    dk = torch.full((T, h_kv, DQK), float("nan"), dtype=bf, device="cuda")
    dv = torch.full((T, h_kv, DV), float("nan"), dtype=bf, device="cuda")
    small = P.hydra_attn_bwd_gqa(q, k, v, out, lse, do, cu, h, h_kv, lib_pairs, True, scale, dq, dk, dv, ws,
                                 workspace_bytes=P.hydra_workspace_bytes(P.HYDRA_WS_FWD, cu, h) + T * h * 4 + 4096,
                                 check=False)
    assert small == P.HYDRA_ERR_WORKSPACE_TOO_SMALL
    P.hydra_attn_bwd_gqa(q, k, v, out, lse, do, cu, h, h_kv, lib_pairs, True, scale, dq, dk, dv, ws)
    status, detail = P.hydra_poll_status(ws)
    assert status == 0, (status, detail)
    f64 = lambda t: t.float().cpu().numpy().astype(np.float64)
    o_ref, l_ref = oracle.attn_fwd_gqa(x["q"], x["k"], x["v"], cu, True, np.float32(scale))
    if ora_pairs is None:
        ref = oracle.attn_bwd_gqa(x["q"], x["k"], x["v"], x["do"], cu, True, np.float32(scale), o_ref, l_ref)
    else:
        d = oracle.bwd_prep(x["do"], o_ref)
        ref = oracle.attn_bwd_pairs_gqa(x["q"], x["k"], x["v"], x["do"], cu, ora_pairs, True, np.float32(scale), l_ref, d)
    check(dict(out=f64(out), lse=f64(lse), dq=f64(dq), dk=f64(dk), dv=f64(dv)),
          dict(out=o_ref, lse=l_ref, dq=ref[0], dk=ref[1], dv=ref[2]), label=f"gqa one-shot {lengths}: ")


def test_gqa_entry_points_reject_bad_head_counts():
    import torch
    import paper_2609_34318_b200 as P
    cu = hw.cu_seqlens([64])
    t = torch.zeros(64 * 4 * DQK, dtype=torch.bfloat16, device="cuda")
    ws = torch.empty(1 << 16, dtype=torch.uint8, device="cuda")
    s = P.hydra_attn_fwd_gqa(t, t, t, cu, 4, 3, None, True, 0.07, t, t, None, None, 0, ws, check=False)
    assert s == P.HYDRA_ERR_INVALID_ARG                                       # 3 does not divide 4
    s = P.hydra_attn_bwd_accumulate_gqa(t, t, t, t, t, t, cu, 4, 0, None, True, 0.07, t, t, t, ws, check=False)
    assert s == P.HYDRA_ERR_INVALID_ARG


@pytest.mark.parametrize("seed", range(6))
def test_gqa_random_mixes(backward_form, seed):
    rng = np.random.default_rng(900 + seed)
    n = int(rng.integers(1, 5))
    lengths = [int(v) for v in rng.choice([1, 64, 129, 200, 383, 640, 777], size=n)]
    cp_r = [int(v) for v in rng.choice([0, 1, 2, 3], size=n)]
    h_kv = int(rng.integers(1, 3))
    h = h_kv * int(rng.choice([1, 2, 4]))
    cu = hw.cu_seqlens(lengths)
    x = inputs(rng, int(cu[-1]), h, h_kv)
    lib_pairs, rows, ora_pairs = pairs_for(cu, cp_r) if any(cp_r) else (None, 0, None)
    got = run_gpu_gqa(x, cu, h, h_kv, lib_pairs, rows)
    scale = np.float32(1.0 / np.sqrt(np.float32(DQK)))
    out, lse = oracle.attn_fwd_gqa(x["q"], x["k"], x["v"], cu, True, scale)
    if ora_pairs is None:
        dq, dk, dv = oracle.attn_bwd_gqa(x["q"], x["k"], x["v"], x["do"], cu, True, scale, out, lse)
    else:
        d = oracle.bwd_prep(x["do"], out)
        dq, dk, dv = oracle.attn_bwd_pairs_gqa(x["q"], x["k"], x["v"], x["do"], cu, ora_pairs, True, scale, lse, d)
    check(got, dict(out=out, lse=lse, dq=dq, dk=dk, dv=dv), label=f"gqa mix {lengths} {cp_r} h={h}/{h_kv}: ")
