"""The elementwise steps of the gated MLA block on the GPU against their fp64 oracle, element by element.
Inputs are bf16; the kernels compute in fp32 and round every output once, so the bound is bf16's half unit
in the last place on the output's magnitude (2^-8 relative, plus the same on the largest input for the
rotations, whose outputs may cancel) - far inside the 2e-2 of the attention tensors."""
import numpy as np
import pytest
import torch

import hydra_workloads as hw
from oracle import mla_ops as M

pytestmark = pytest.mark.gpu
THETA = 10000.0


def bits(rng, shape, scale=1.0):
    return hw.f32_to_bf16_bits((scale * rng.standard_normal(shape)).astype(np.float32))


def dev(b):
    from paper_2609_34318_b200.runner import bits_to_tensor
    return bits_to_tensor(b)


def f64(t):
    return t.float().cpu().numpy().astype(np.float64)


def close(got, ref, scale, label):
    """Every element within one bf16 rounding of the reference (half a unit in the last place: 2^-8 of its
    magnitude) plus fp32 arithmetic noise on the inputs' scale."""
    bound = 2.0 ** -8 * 1.01 * np.abs(ref) + 1e-5 * scale
    worst = (np.abs(got - ref) - bound).max()
    assert worst <= 0.0, (label, float(worst), float(np.abs(got - ref).max()), scale)


def positions_for(lengths):
    return np.concatenate([np.arange(L, dtype=np.int32) for L in lengths])


@pytest.mark.parametrize("lengths,h,in_place", [([7, 33, 128, 300], 4, False), ([1000, 64], 16, True),
                                                ([262143 - 5, 0], 1, False)])
def test_query_rotary_embedding_and_its_inverse(lengths, h, in_place):
    import paper_2609_34318_b200 as P
    rng = np.random.default_rng(51)
    if lengths[0] > 100000:                      # a handful of tokens at the far end of a 256K sequence
        pos = np.arange(lengths[0], lengths[0] + 5, dtype=np.int32)
    else:
        pos = positions_for(lengths)
    T = len(pos)
    xb = bits(rng, (T, h, 192))
    x = hw.bf16_bits_to_f64(xb)
    ref = M.rope(x, pos, 128, 64, THETA)
    xd, pd = dev(xb), torch.from_numpy(pos).cuda()
    yd = xd if in_place else torch.full_like(xd, float("nan"))
    keep = xd.clone()
    P.hydra_mla_rope(xd, pd, T, h, 192, 128, 64, THETA, False, yd)
    torch.cuda.synchronize()
    got = f64(yd)
    assert np.array_equal(got[..., :128], x[..., :128])             # the position-free columns pass through
    close(got[..., 128:], ref[..., 128:], np.abs(x).max(), f"rope {lengths}")
    # the backward of the step: rotating a gradient by the opposite angle undoes the rotation of the same data
    back = torch.full_like(xd, float("nan"))
    P.hydra_mla_rope(yd, pd, T, h, 192, 128, 64, THETA, True, back)
    torch.cuda.synchronize()
    close(f64(back), M.rope(got, pos, 128, 64, THETA, inverse=True), np.abs(x).max(), f"rope inverse {lengths}")
    assert np.abs(f64(back) - f64(keep)).max() <= 2.0 ** -6 * np.abs(x).max()        # two roundings from the original


@pytest.mark.parametrize("lengths,h", [([5, 130], 3), ([700, 300, 24], 16)])
def test_key_value_assembly_forward_and_backward(lengths, h):
    import paper_2609_34318_b200 as P
    rng = np.random.default_rng(52)
    pos = positions_for(lengths)
    T = len(pos)
    up_b, pe_b = bits(rng, (T, h, 256)), bits(rng, (T, 64))
    k_ref, v_ref = M.kv_assemble(hw.bf16_bits_to_f64(up_b), hw.bf16_bits_to_f64(pe_b), pos, 128, 64, 128, THETA)
    pd = torch.from_numpy(pos).cuda()
    k = torch.full((T, h, 192), float("nan"), dtype=torch.bfloat16, device="cuda")
    v = torch.full((T, h, 128), float("nan"), dtype=torch.bfloat16, device="cuda")
    P.hydra_mla_kv_assemble(dev(up_b), dev(pe_b), pd, T, h, 128, 64, 128, THETA, k, v)
    torch.cuda.synchronize()
    gk, gv = f64(k), f64(v)
    assert np.array_equal(gk[..., :128], k_ref[..., :128]) and np.array_equal(gv, v_ref)     # pure copies
    close(gk[..., 128:], k_ref[..., 128:], np.abs(hw.bf16_bits_to_f64(pe_b)).max(), "assembled key, rotary part")
    # backward
    dk_b, dv_b = bits(rng, (T, h, 192)), bits(rng, (T, h, 128))
    up_ref, pe_ref = M.kv_assemble_bwd(hw.bf16_bits_to_f64(dk_b), hw.bf16_bits_to_f64(dv_b), pos, 128, 64, 128, THETA)
    dup = torch.full((T, h, 256), float("nan"), dtype=torch.bfloat16, device="cuda")
    dpe = torch.full((T, 64), float("nan"), dtype=torch.bfloat16, device="cuda")
    P.hydra_mla_kv_assemble_bwd(dev(dk_b), dev(dv_b), pd, T, h, 128, 64, 128, THETA, dup, dpe)
    torch.cuda.synchronize()
    assert np.array_equal(f64(dup), up_ref)
    close(f64(dpe), pe_ref, np.abs(pe_ref).max(), "rotary key gradient (summed over heads)")


def test_gate_forward_and_backward():
    import paper_2609_34318_b200 as P
    rng = np.random.default_rng(53)
    shape = (777, 4, 128)
    ob, gb, db = bits(rng, shape), bits(rng, shape, 3.0), bits(rng, shape)
    o, g, d = (hw.bf16_bits_to_f64(b) for b in (ob, gb, db))
    y = torch.full(shape, float("nan"), dtype=torch.bfloat16, device="cuda")
    n = int(np.prod(shape))
    P.hydra_gate_apply(dev(ob), dev(gb), n, y)
    d_out = torch.full_like(y, float("nan"))
    d_gate = torch.full_like(y, float("nan"))
    P.hydra_gate_apply_bwd(dev(db), dev(ob), dev(gb), n, d_out, d_gate)
    torch.cuda.synchronize()
    ref_o, ref_g = M.gate_apply_bwd(d, o, g)
    for got, ref, name in ((f64(y), M.gate_apply(o, g), "gate"), (f64(d_out), ref_o, "d_out"), (f64(d_gate), ref_g, "d_gate")):
        # __expf in the sigmoid: a few fp32 units on top of the output's rounding
        assert (np.abs(got - ref) <= 2.0 ** -8 * 1.05 * np.abs(ref) + 1e-5 * np.abs(ref).max()).all(), name


def test_bad_arguments_are_refused():
    import paper_2609_34318_b200 as P
    z = torch.zeros(4096, dtype=torch.uint8, device="cuda")
    n0 = P.hydra_launch_count()
    assert P.hydra_mla_rope(z, z, 4, 2, 192, 129, 64, THETA, False, z, check=False) == P.HYDRA_ERR_INVALID_ARG
    assert P.hydra_mla_rope(z, z, 4, 2, 192, 160, 64, THETA, False, z, check=False) == P.HYDRA_ERR_INVALID_ARG
    assert P.hydra_mla_rope(z, z, 4, 2, 192, 128, 64, 1.0, False, z, check=False) == P.HYDRA_ERR_INVALID_ARG
    assert P.hydra_gate_apply(z, z, 12, z, check=False) == P.HYDRA_ERR_INVALID_ARG
    assert P.hydra_mla_kv_assemble(z, z, z, 4, 2, 128, 63, 128, THETA, z, z, check=False) == P.HYDRA_ERR_INVALID_ARG
    assert P.hydra_launch_count() == n0


@pytest.mark.parametrize("in_place", [False, True])
def test_dimensions_that_are_not_multiples_of_eight_take_the_four_byte_kernels(in_place):
    """The kernels move 16 bytes per access where every dimension is a multiple of 8 elements; other (even)
    dimensions fall back to one rotary pair per access. Heads of 20 with rotary columns [4, 16); an up-projection of
    12 + 10 columns with a rotary key of 4."""
    import paper_2609_34318_b200 as P
    rng = np.random.default_rng(54)
    lengths, h = [9, 70], 3
    pos = positions_for(lengths)
    T = len(pos)
    pd = torch.from_numpy(pos).cuda()
    xb = bits(rng, (T, h, 20))
    x = hw.bf16_bits_to_f64(xb)
    ref = M.rope(x, pos, 4, 12, THETA)
    xd = dev(xb)
    yd = xd if in_place else torch.full_like(xd, float("nan"))
    P.hydra_mla_rope(xd, pd, T, h, 20, 4, 12, THETA, False, yd)
    torch.cuda.synchronize()
    got = f64(yd)
    assert np.array_equal(got[..., :4], x[..., :4]) and np.array_equal(got[..., 16:], x[..., 16:])
    close(got[..., 4:16], ref[..., 4:16], np.abs(x).max(), "rope, odd dimensions")
    up_b, pe_b = bits(rng, (T, h, 22)), bits(rng, (T, 4))
    k_ref, v_ref = M.kv_assemble(hw.bf16_bits_to_f64(up_b), hw.bf16_bits_to_f64(pe_b), pos, 12, 4, 10, THETA)
    k = torch.full((T, h, 16), float("nan"), dtype=torch.bfloat16, device="cuda")
    v = torch.full((T, h, 10), float("nan"), dtype=torch.bfloat16, device="cuda")
    P.hydra_mla_kv_assemble(dev(up_b), dev(pe_b), pd, T, h, 12, 4, 10, THETA, k, v)
    torch.cuda.synchronize()
    gk, gv = f64(k), f64(v)
    assert np.array_equal(gk[..., :12], k_ref[..., :12]) and np.array_equal(gv, v_ref)
    close(gk[..., 12:], k_ref[..., 12:], np.abs(hw.bf16_bits_to_f64(pe_b)).max(), "assembled key, odd dimensions")
    dk_b, dv_b = bits(rng, (T, h, 16)), bits(rng, (T, h, 10))
    up_ref, pe_ref = M.kv_assemble_bwd(hw.bf16_bits_to_f64(dk_b), hw.bf16_bits_to_f64(dv_b), pos, 12, 4, 10, THETA)
    dup = torch.full((T, h, 22), float("nan"), dtype=torch.bfloat16, device="cuda")
    dpe = torch.full((T, 4), float("nan"), dtype=torch.bfloat16, device="cuda")
    P.hydra_mla_kv_assemble_bwd(dev(dk_b), dev(dv_b), pd, T, h, 12, 4, 10, THETA, dup, dpe)
    torch.cuda.synchronize()
    assert np.array_equal(f64(dup), up_ref)
    close(f64(dpe), pe_ref, np.abs(pe_ref).max(), "rotary key gradient, odd dimensions")
