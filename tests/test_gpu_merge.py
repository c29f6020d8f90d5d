"""The LSE merge kernel on hand-made partials (Section 5.2: the partial results of the ring steps are merged with
their log-sum-exp), against the oracle's merge of the same buffers.

The forward-driven tests feed the merge well-behaved partials. Here the partial buffers are filled directly:
2 to 10 partials per chunk (the kernel takes them in batches of two or four), partials that saw no key
(LSE = -inf) whose O rows hold NaN and must count for nothing, rows all of whose partials saw no key
(O = 0, LSE = -inf), LSEs hundreds of units apart, and the streaming form in which the current (out, lse)
rows are one more input.
"""
import numpy as np
import pytest
import torch

import hydra_workloads as hw
from gpu_util import TOL_LSE, oracle_merge_of_partials

pytestmark = pytest.mark.gpu
DV = hw.D_V


def _fill(rng, part_rows, h, none_frac, spread):
    o = torch.from_numpy(rng.standard_normal((part_rows, h, DV)).astype(np.float32)).to(torch.bfloat16)
    l = (spread * rng.standard_normal((h, part_rows))).astype(np.float32)
    none = rng.random((h, part_rows)) < none_frac            # partials that saw no key
    l[none] = -np.inf
    o_f = o.float()
    o_f[torch.from_numpy(none.T.copy())] = float("nan")      # their O rows are garbage
    return o_f.to(torch.bfloat16).cuda(), torch.from_numpy(l).cuda(), none


def _compare(out, lse, ref_out, ref_lse, label):
    got_o = out.float().cpu().numpy().astype(np.float64)
    got_l = lse.cpu().numpy().astype(np.float64)
    rows = ~np.isnan(ref_lse)                                # rows of merged chunks
    assert rows.any()
    assert np.array_equal(np.isneginf(got_l[rows]), np.isneginf(ref_lse[rows])), f"{label}: -inf pattern of LSE"
    fin = rows & np.isfinite(ref_lse)
    if fin.any():
        assert np.abs(got_l[fin] - ref_lse[fin]).max() <= TOL_LSE, label
    sel = rows.T                                             # [T, h]
    assert np.isfinite(got_o[sel]).all(), f"{label}: a partial without keys leaked into O"
    # one rounding of the fp32 result to bf16, plus the approximate exponentials of the weights
    err = np.abs(got_o[sel] - ref_out[sel])
    assert (err <= 2.0 ** -8 * np.abs(ref_out[sel]) + 2e-3).all(), (label, err.max())
    dead = rows & np.isneginf(ref_lse)
    if dead.any():
        assert (got_o[dead.T] == 0).all(), f"{label}: rows without any key must be 0"


@pytest.mark.parametrize("cp_r,lengths,h", [(1, [300, 64, 9], 3), (2, [517, 130], 2), (4, [400, 90], 2), (5, [1000, 37], 1)])
@pytest.mark.parametrize("none_frac,spread", [(0.0, 3.0), (0.3, 3.0), (0.7, 200.0)])
def test_merge_of_hand_made_partials(cp_r, lengths, h, none_frac, spread):
    import paper_2609_34318_b200 as P
    rng = np.random.default_rng(cp_r * 100 + int(none_frac * 10))
    cu = hw.cu_seqlens(lengths)
    T = int(cu[-1])
    pairs, part_rows, _, _ = P.hydra_zigzag_pairs(cu, cp_r)
    counts = {}
    for p in pairs:
        if p["part_row"] >= 0:
            counts[int(p["group"])] = counts.get(int(p["group"]), 0) + 1
    assert max(counts.values()) == 2 * cp_r                   # the last chunk sees every chunk
    o_part, lse_part, _ = _fill(rng, part_rows, h, none_frac, spread)
    out = torch.full((T, h, DV), float("nan"), dtype=torch.bfloat16, device="cuda")
    lse = torch.full((h, T), float("nan"), dtype=torch.float32, device="cuda")
    ws = torch.empty(4096, dtype=torch.uint8, device="cuda")
    P.hydra_lse_merge(o_part, lse_part, part_rows, cu, h, pairs, out, lse, ws)
    torch.cuda.synchronize()
    ref_out, ref_lse = oracle_merge_of_partials(cu, pairs, o_part, lse_part, T, h)
    _compare(out, lse, ref_out, ref_lse, f"cp_r {cp_r} none {none_frac}")
    # rows of chunks with a single pair are not the merge's to write
    untouched = np.isnan(ref_lse)
    assert torch.isnan(lse).cpu().numpy()[untouched].all()


@pytest.mark.parametrize("cp_r", [1, 3])
def test_streaming_merge_takes_the_current_rows_as_one_more_input(cp_r):
    import paper_2609_34318_b200 as P
    rng = np.random.default_rng(7 + cp_r)
    lengths, h = [260, 75], 2
    cu = hw.cu_seqlens(lengths)
    T = int(cu[-1])
    pairs, part_rows, _, _ = P.hydra_zigzag_pairs(cu, cp_r)
    o_part, lse_part, _ = _fill(rng, part_rows, h, 0.3, 5.0)
    out0, lse0, _ = _fill(rng, T, h, 0.3, 5.0)                # what (out, lse) hold so far; some rows nothing yet
    out, lse = out0.clone(), lse0.clone()
    ws = torch.empty(4096, dtype=torch.uint8, device="cuda")
    P.hydra_lse_merge_accumulate(o_part, lse_part, part_rows, cu, h, pairs, out, lse, ws)
    torch.cuda.synchronize()
    ref_out, ref_lse = oracle_merge_of_partials(cu, pairs, o_part, lse_part, T, h,
                                                out_cur=out0.float().cpu().numpy().astype(np.float64),
                                                lse_cur=lse0.cpu().numpy().astype(np.float64))
    _compare(out, lse, ref_out, ref_lse, f"streaming cp_r {cp_r}")


def test_buffers_that_are_16_but_not_32_byte_aligned_take_the_16_byte_kernel():
    """The interface asks for 16-byte alignment; the merge moves 32 bytes per lane only when both the partial
    buffer and out allow it."""
    import paper_2609_34318_b200 as P
    rng = np.random.default_rng(3)
    lengths, h, cp_r = [333, 70], 2, 2
    cu = hw.cu_seqlens(lengths)
    T = int(cu[-1])
    pairs, part_rows, _, _ = P.hydra_zigzag_pairs(cu, cp_r)
    o_al, lse_part, _ = _fill(rng, part_rows, h, 0.2, 4.0)

    def shifted(t):                                          # the same values at an address that is 16 modulo 32
        raw = torch.zeros(t.numel() * t.element_size() + 64, dtype=torch.uint8, device="cuda")
        off = (16 - raw.data_ptr() % 32) % 32
        view = raw[off:off + t.numel() * t.element_size()].view(t.dtype).view(t.shape)
        view.copy_(t)
        assert view.data_ptr() % 32 == 16
        return view
    o_part = shifted(o_al)
    out = shifted(torch.full((T, h, DV), float("nan"), dtype=torch.bfloat16, device="cuda"))
    lse = torch.full((h, T), float("nan"), dtype=torch.float32, device="cuda")
    ws = torch.empty(4096, dtype=torch.uint8, device="cuda")
    P.hydra_lse_merge(o_part, lse_part, part_rows, cu, h, pairs, out, lse, ws)
    torch.cuda.synchronize()
    ref_out, ref_lse = oracle_merge_of_partials(cu, pairs, o_part, lse_part, T, h)
    _compare(out, lse, ref_out, ref_lse, "16-byte aligned buffers")
