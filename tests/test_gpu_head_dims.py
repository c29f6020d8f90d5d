"""Heads of d_qk = d_v = 128 (the grouped-query model of the paper's scale-out simulation, Section 6) through
the entry points that take the head dimensions, against the fp64 oracle: forward, merge of cut sequences,
both forms of the one-shot backward, the banded backward, the accumulating grouped-query backward, and the
refusal of any other pair of dimensions. Same tolerances as for 192 / 128."""
import numpy as np
import pytest
import torch

import hydra_workloads as hw
import oracle
from gpu_util import check, guard, pairs_for

pytestmark = [pytest.mark.gpu, pytest.mark.usefixtures("both_forward_kernels")]
D = 128


@pytest.fixture(params=["hand_off", "recompute"])
def backward_form(request):
    import paper_2609_34318_b200 as P
    P.hydra_set_bwd_scratch_limit(0 if request.param == "recompute" else 4 << 30)
    yield request.param
    P.hydra_set_bwd_scratch_limit(4 << 30)


def inputs(rng, T, h, h_kv, q_scale=1.0):
    f = lambda heads, s=1.0: hw.f32_to_bf16_bits((s * rng.standard_normal((T, heads, D))).astype(np.float32))
    return dict(q=f(h, q_scale), k=f(h_kv), v=f(h_kv), do=f(h))


class Buffers:
    """Outputs and workspace of one d = 128 problem (NaN-filled, between guard bands)."""
    def __init__(self, P, cu, h, h_kv, lib_pairs, part_rows):
        T = int(cu[-1])
        bf, f32 = torch.bfloat16, torch.float32
        nan = float("nan")
        self.out = torch.full((T, h, D), nan, dtype=bf, device="cuda")
        self.lse = torch.full((h, T), nan, dtype=f32, device="cuda")
        self.o_part = torch.full((max(part_rows, 1), h, D), nan, dtype=bf, device="cuda")
        self.lse_part = torch.full((h, max(part_rows, 1)), nan, dtype=f32, device="cuda")
        self.dq = torch.full((T, h, D), nan, dtype=bf, device="cuda")
        self.dk = torch.full((T, h_kv, D), nan, dtype=bf, device="cuda")
        self.dv = torch.full((T, h_kv, D), nan, dtype=bf, device="cuda")
        need = max(P.hydra_workspace_bytes_dims(w, cu, h, h_kv, D, D, lib_pairs)
                   for w in (P.HYDRA_WS_FWD, P.HYDRA_WS_MERGE, P.HYDRA_WS_BWD))
        assert need > 0
        self.workspace = torch.empty(need, dtype=torch.uint8, device="cuda")
        self.verify = guard(self)


def run_d128(x, cu, h, h_kv, lib_pairs, part_rows, accumulate=False):
    import paper_2609_34318_b200 as P
    from paper_2609_34318_b200.runner import bits_to_tensor
    T = int(cu[-1])
    scale = float(np.float32(1.0 / np.sqrt(np.float32(D))))
    q, k, v, do = (bits_to_tensor(x[n]) for n in ("q", "k", "v", "do"))
    b = Buffers(P, cu, h, h_kv, lib_pairs, part_rows)
    has_parts = lib_pairs is not None and bool((lib_pairs["part_row"] >= 0).any())
    P.hydra_attn_fwd_dims(q, k, v, cu, h, h_kv, D, D, lib_pairs, True, scale, b.out, b.lse,
                          b.o_part if has_parts else None, b.lse_part if has_parts else None, part_rows, b.workspace)
    if has_parts:
        P.hydra_lse_merge(b.o_part, b.lse_part, part_rows, cu, h, lib_pairs, b.out, b.lse, b.workspace)
    if accumulate:
        acc = [torch.zeros((T, heads, D), dtype=torch.float32, device="cuda") for heads in (h, h_kv, h_kv)]
        P.hydra_attn_bwd_accumulate_dims(q, k, v, b.out, b.lse, do, cu, h, h_kv, D, D, lib_pairs, True, scale,
                                         acc[0], acc[1], acc[2], b.workspace)
        for a, g in zip(acc, (b.dq, b.dk, b.dv)):
            P.hydra_grad_cast(a, g)
    else:
        P.hydra_attn_bwd_dims(q, k, v, b.out, b.lse, do, cu, h, h_kv, D, D, lib_pairs, True, scale, b.dq, b.dk, b.dv,
                              b.workspace)
    status, detail = P.hydra_poll_status(b.workspace)
    assert status == 0, (status, detail)
    torch.cuda.synchronize()
    b.verify("d128: ")
    f64 = lambda t: t.float().cpu().numpy().astype(np.float64)
    return dict(out=f64(b.out), lse=f64(b.lse), dq=f64(b.dq), dk=f64(b.dk), dv=f64(b.dv))


def reference(x, cu, ora_pairs):
    scale = np.float32(1.0 / np.sqrt(np.float32(D)))
    out, lse = oracle.attn_fwd_gqa(x["q"], x["k"], x["v"], cu, True, scale)
    if ora_pairs is None:
        dq, dk, dv = oracle.attn_bwd_gqa(x["q"], x["k"], x["v"], x["do"], cu, True, scale, out, lse)
    else:
        d = oracle.bwd_prep(x["do"], out)
        dq, dk, dv = oracle.attn_bwd_pairs_gqa(x["q"], x["k"], x["v"], x["do"], cu, ora_pairs, True, scale, lse, d)
    return dict(out=out, lse=lse, dq=dq, dk=dk, dv=dv)


@pytest.mark.parametrize("lengths,h,cp_r", [
    ([7, 33, 128, 300], 4, 0), ([300], 4, 1), ([1, 127, 129, 255, 257], 2, 0), ([1500, 700, 90], 3, 0),
    ([2047], 2, 2), ([640, 200, 65], 2, [4, 1, 0])])
def test_per_head_forward_and_backward_at_128(backward_form, lengths, h, cp_r):
    cu = hw.cu_seqlens(lengths)
    x = inputs(np.random.default_rng(31 + h), int(cu[-1]), h, h)
    lib_pairs, rows, ora_pairs = pairs_for(cu, cp_r) if cp_r else (None, 0, None)
    got = run_d128(x, cu, h, h, lib_pairs, rows)
    check(got, reference(x, cu, ora_pairs), label=f"d128 {lengths} h={h} ring {cp_r}: ")


@pytest.mark.parametrize("lengths,h,h_kv,cp_r", [([300, 129, 64], 8, 1, 0), ([700], 8, 2, 0), ([640, 200], 16, 2, 2)])
def test_grouped_query_at_128(backward_form, lengths, h, h_kv, cp_r):
    """The shape of the paper's grouped-query model: several query heads per KV head, heads of 128."""
    cu = hw.cu_seqlens(lengths)
    x = inputs(np.random.default_rng(37 + h_kv), int(cu[-1]), h, h_kv)
    lib_pairs, rows, ora_pairs = pairs_for(cu, cp_r) if cp_r else (None, 0, None)
    ref = reference(x, cu, ora_pairs)
    check(run_d128(x, cu, h, h_kv, lib_pairs, rows, accumulate=True), ref, label=f"d128 gqa acc {lengths} {h}/{h_kv}: ")
    check(run_d128(x, cu, h, h_kv, lib_pairs, rows, accumulate=False), ref, label=f"d128 gqa {lengths} {h}/{h_kv}: ")


def test_banded_backward_at_128():
    import paper_2609_34318_b200 as P
    P.hydra_set_bwd_scratch_limit(1 << 20)
    P.hydra_set_bwd_band_scratch(1 << 20)
    try:
        lengths, h = [1500, 300], 2
        cu = hw.cu_seqlens(lengths)
        x = inputs(np.random.default_rng(41), int(cu[-1]), h, h)
        n0 = P.hydra_launch_count()
        got = run_d128(x, cu, h, h, None, 0)
        assert P.hydra_launch_count() - n0 >= 1 + 1 + 2 * 2 + 1          # forward, prep, two bands at least, cast
        check(got, reference(x, cu, None), label="d128 banded: ")
    finally:
        P.hydra_set_bwd_scratch_limit(4 << 30)
        P.hydra_set_bwd_band_scratch(P.HYDRA_BAND_AUTO)


def test_large_scores_at_128():
    cu = hw.cu_seqlens([520])
    x = inputs(np.random.default_rng(43), 520, 2, 2, q_scale=8.0)
    check(run_d128(x, cu, 2, 2, None, 0), reference(x, cu, None), label="d128 large scores: ")


def test_other_head_dimensions_are_refused():
    import paper_2609_34318_b200 as P
    cu = hw.cu_seqlens([64])
    dummy = torch.zeros(1 << 20, dtype=torch.uint8, device="cuda")
    n0 = P.hydra_launch_count()
    for d_qk, d_v in ((64, 64), (192, 192), (128, 64), (256, 128)):
        assert P.hydra_workspace_bytes_dims(P.HYDRA_WS_BWD, cu, 2, 2, d_qk, d_v) == 0
        s = P.hydra_attn_fwd_dims(dummy, dummy, dummy, cu, 2, 2, d_qk, d_v, None, True, 0.1, dummy, dummy, None, None,
                                  0, dummy, check=False)
        assert s == P.HYDRA_ERR_UNSUPPORTED, (d_qk, d_v, s)
        s = P.hydra_attn_bwd_dims(dummy, dummy, dummy, dummy, dummy, dummy, cu, 2, 2, d_qk, d_v, None, True, 0.1,
                                  dummy, dummy, dummy, dummy, check=False)
        assert s == P.HYDRA_ERR_UNSUPPORTED, (d_qk, d_v, s)
    assert P.hydra_launch_count() == n0
