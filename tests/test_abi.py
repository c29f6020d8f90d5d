"""CPU-side checks of the C ABI: the library loads, exports what include/hydra_attn.h declares,
its host-only entry points agree bit for bit with the oracle's integer bookkeeping, and argument
validation returns the documented codes. No kernel runs here."""
import ctypes
import os
import re

import numpy as np
import pytest

import oracle
import paper_2609_34318_b200 as P

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    names = set()
    for header in sorted(os.listdir(os.path.join(ROOT, "include"))):
        if not header.endswith(".h"):
            continue
        with open(os.path.join(ROOT, "include", header)) as f:
            text = re.sub(r"/\*.*?\*/", "", f.read(), flags=re.S)
        names |= set(re.findall(r"\b(hydra_[a-z0-9_]+)\s*\(", text))
    return sorted(names)


def test_library_exports_every_declared_symbol():
    names = declared_symbols()
    assert {"hydra_attn_fwd", "hydra_attn_bwd", "hydra_lse_merge"} <= set(names)
    lib = ctypes.CDLL(P.LIBRARY_PATH)
    for n in names:
        assert hasattr(lib, n), f"{n} is declared in the header but not exported"
    assert set(n for n in P.EXPORTS) <= set(names)


def test_binding_has_the_same_names():
    for n in declared_symbols():
        assert hasattr(P, n), f"binding lacks {n}"


def test_version_and_status_strings():
    assert P.hydra_version() >= 1
    assert P.hydra_status_string(0) == "HYDRA_OK"
    assert P.hydra_status_string(5) == "HYDRA_ERR_DEVICE_TIMEOUT"
    assert P.hydra_status_string(99) == "HYDRA_ERR_UNKNOWN"


def test_usp_factor_matches_oracle_and_paper_values():
    assert P.hydra_usp_factor(256, 64) == (64, 4)         # Section 5.2: ring of four at P=256, h=64
    for degree, heads in [(1, 1), (8, 64), (64, 64), (128, 64), (32, 8), (16, 16), (2, 3)]:
        assert P.hydra_usp_factor(degree, heads) == oracle.usp_factor(degree, heads)
    with pytest.raises(P.HydraError):
        P.hydra_usp_factor(0, 4)
    with pytest.raises(P.HydraError):
        P.hydra_usp_factor(12, 8)                         # 8 does not divide 12


@pytest.mark.parametrize("lengths,cp_r", [([300], 1), ([262144], 4), ([7, 33, 128, 300], 0),
                                          ([5, 0, 3, 1000, 1], 2), ([1, 2, 3], 4), ([100, 200], [0, 2])])
def test_zigzag_pairs_match_the_oracle_bit_for_bit(lengths, cp_r):
    cu = np.concatenate([[0], np.cumsum(lengths)]).astype(np.int32)
    pairs, part_rows, rank, step = P.hydra_zigzag_pairs(cu, cp_r)
    ref = oracle.causal_pairs(cu, cp_r)
    assert len(pairs) == len(ref)
    rows = 0
    by_group = {}
    for p in ref:
        by_group.setdefault(p["group"], []).append(p)
    for i, r in enumerate(ref):
        for name in ("seq", "q_start", "q_len", "k_start", "k_len", "group"):
            assert int(pairs[i][name]) == r[name], (i, name)
        assert int(rank[i]) == r["rank"] and int(step[i]) == r["step"]
        if len(by_group[r["group"]]) > 1:
            assert int(pairs[i]["part_row"]) == rows
            rows += r["q_len"]
        else:
            assert int(pairs[i]["part_row"]) == -1
    assert part_rows == rows


def test_zigzag_pairs_rejects_bad_input():
    with pytest.raises(P.HydraError):
        P.hydra_zigzag_pairs([0, 10, 5], 1)      # decreasing cu_seqlens
    with pytest.raises(P.HydraError):
        P.hydra_zigzag_pairs([1, 10], 1)         # does not start at 0
    with pytest.raises(P.HydraError):
        P.hydra_zigzag_pairs([0, 10], -1)


def test_workspace_bytes():
    cu = [0, 100, 300]
    assert P.hydra_workspace_bytes(P.HYDRA_WS_FWD, cu, 4) >= 16
    small = P.hydra_workspace_bytes(P.HYDRA_WS_BWD, cu, 4)
    big = P.hydra_workspace_bytes(P.HYDRA_WS_BWD, [0, 100, 3000], 4)
    assert small >= 300 * 4 * 4 and big > small               # holds D [h, T] fp32; monotone in T
    assert P.hydra_workspace_bytes(P.HYDRA_WS_BWD, [0, 100, 50], 4) == 0     # invalid input
    assert P.hydra_workspace_bytes(7, cu, 4) == 0


def _call_fwd(cu, h, pairs, ws=0x1000, ws_bytes=4096, q=0x1000, out=0x1000, part=0x1000, part_rows=0,
              scale=0.07):
    return P.hydra_attn_fwd(q, q, q, cu, h, pairs, True, scale, out, out, part, part, part_rows, ws,
                            ws_bytes, stream=0, check=False)


def test_forward_validation_codes_without_a_gpu():
    cu = [0, 64, 200]
    ok_pair = dict(seq=1, q_start=0, q_len=136, k_start=0, k_len=136, group=0)
    assert _call_fwd([0, 64, 32], 2, None) == P.HYDRA_ERR_INVALID_ARG                 # non-monotone
    assert _call_fwd(cu, 0, None) == P.HYDRA_ERR_INVALID_ARG                          # no heads
    assert _call_fwd(cu, 2, None, scale=0.0) == P.HYDRA_ERR_INVALID_ARG
    assert _call_fwd(cu, 2, None, ws=0x1004) == P.HYDRA_ERR_INVALID_ARG               # misaligned
    assert _call_fwd(cu, 2, None, ws_bytes=8) == P.HYDRA_ERR_WORKSPACE_TOO_SMALL
    assert _call_fwd(cu, 2, None, q=0) == P.HYDRA_ERR_INVALID_ARG                     # null tensor
    bad = dict(ok_pair, q_len=137)
    assert _call_fwd(cu, 2, [bad]) == P.HYDRA_ERR_INVALID_ARG                         # pair leaves its sequence
    assert _call_fwd(cu, 2, [dict(ok_pair, seq=2)]) == P.HYDRA_ERR_INVALID_ARG
    assert _call_fwd(cu, 2, [dict(ok_pair, flags=1)]) == P.HYDRA_ERR_INVALID_ARG
    two = [dict(ok_pair, k_len=60, part_row=0), dict(ok_pair, k_start=60, k_len=76, part_row=100)]
    assert _call_fwd(cu, 2, two, part_rows=300) == P.HYDRA_ERR_INVALID_ARG            # partial rows overlap
    assert _call_fwd(cu, 2, two[:1] + [dict(two[1], part_row=136)], part_rows=200) == P.HYDRA_ERR_INVALID_ARG
    differing = [dict(ok_pair, part_row=0), dict(ok_pair, q_len=100, part_row=136)]
    assert _call_fwd(cu, 2, differing, part_rows=400) == P.HYDRA_ERR_INVALID_ARG      # group with two q ranges
    unordered = [dict(ok_pair, group=1), dict(ok_pair, seq=0, q_len=64, k_len=64, group=0)]
    assert _call_fwd(cu, 2, unordered) == P.HYDRA_ERR_INVALID_ARG


def test_backward_requires_identical_or_disjoint_chunks():
    cu = [0, 256]
    overlapping = [dict(seq=0, q_start=0, q_len=128, k_start=0, k_len=128, group=0),
                   dict(seq=0, q_start=64, q_len=128, k_start=0, k_len=128, group=1)]
    s = P.hydra_attn_bwd(0x1000, 0x1000, 0x1000, 0x1000, 0x1000, 0x1000, cu, 2, overlapping, True, 0.07,
                         0x1000, 0x1000, 0x1000, 0x1000, 1 << 20, stream=0, check=False)
    assert s == P.HYDRA_ERR_INVALID_ARG
    s = P.hydra_attn_bwd(0x1000, 0x1000, 0x1000, 0x1000, 0x1000, 0x1000, cu, 2, None, True, 0.07,
                         0x1000, 0x1000, 0x1000, 0x1000, 64, stream=0, check=False)
    assert s == P.HYDRA_ERR_WORKSPACE_TOO_SMALL


def test_accumulating_backward_and_cast_validate_like_the_plain_calls():
    cu = [0, 256]
    overlapping = [dict(seq=0, q_start=0, q_len=128, k_start=0, k_len=128, group=0),
                   dict(seq=0, q_start=64, q_len=128, k_start=0, k_len=128, group=1)]
    s = P.hydra_attn_bwd_accumulate(0x1000, 0x1000, 0x1000, 0x1000, 0x1000, 0x1000, cu, 2, overlapping, True,
                                    0.07, 0x1000, 0x1000, 0x1000, 0x1000, 1 << 20, stream=0, check=False)
    assert s == P.HYDRA_ERR_INVALID_ARG
    s = P.hydra_attn_bwd_accumulate(0x1000, 0x1000, 0x1000, 0x1000, 0x1000, 0x1000, cu, 2, None, True, 0.07,
                                    0x1000, 0x1004, 0x1000, 0x1000, 1 << 20, stream=0, check=False)
    assert s == P.HYDRA_ERR_INVALID_ARG                                               # misaligned accumulator
    assert P.hydra_grad_cast(0x1000, 0x1000, -1, stream=0, check=False) == P.HYDRA_ERR_INVALID_ARG
    assert P.hydra_grad_cast(0x1000, 0x1000, 0, stream=0, check=False) == P.HYDRA_OK   # nothing to do
    assert P.hydra_grad_cast(0, 0x1000, 8, stream=0, check=False) == P.HYDRA_ERR_INVALID_ARG
    assert P.hydra_grad_cast(0x1000, 0x1008, 8, stream=0, check=False) == P.HYDRA_ERR_INVALID_ARG


def test_no_cpu_fallback():
    """With valid arguments and no usable device the call fails loudly instead of computing."""
    torch = pytest.importorskip("torch")
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    s = _call_fwd([0, 64, 200], 2, None)
    assert s in (P.HYDRA_ERR_CUDA, P.HYDRA_ERR_NOT_SM100)


def test_product_does_not_import_the_oracle():
    pkg = os.path.join(ROOT, "paper_2609_34318_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                with open(os.path.join(dirpath, f)) as fh:
                    text = fh.read()
                assert "import oracle" not in text and "from oracle" not in text, f
                assert "hydra_oracle" not in text, f


def _visible(p, causal):
    """Boolean [q_len, k_len] mask of the positions a pair computes."""
    qi = p["q_start"] + np.arange(p["q_len"])[:, None]
    kj = p["k_start"] + np.arange(p["k_len"])[None, :]
    return (kj <= qi) if causal else np.ones((p["q_len"], p["k_len"]), bool)


@pytest.mark.parametrize("lengths,cp_r,causal,scratch", [
    ([1000], 0, True, 1 << 20), ([1000], 0, False, 1 << 20), ([1500], 2, True, 1 << 20),
    ([700, 130, 64, 900], [1, 0, 0, 2], True, 1 << 20), ([2048], 1, True, 3 << 19), ([300, 5], 0, True, 1 << 30)])
def test_bands_cover_every_visible_position_once_and_fit_their_scratch(lengths, cp_r, causal, scratch):
    h = 2
    cu = np.concatenate([[0], np.cumsum(lengths)]).astype(np.int32)
    pairs = P.hydra_zigzag_pairs(cu, cp_r)[0] if cp_r else None
    whole = pairs if pairs is not None else np.array(
        [(b, 0, L, 0, L, -1, b, 0) for b, L in enumerate(lengths)], dtype=P.PAIR_DTYPE)
    out, band, n_bands = P.hydra_bwd_bands(cu, h, pairs, causal, scratch)
    assert n_bands >= 1 and len(out) == len(band) and list(band) == sorted(band)
    cover = [np.zeros((L, L), np.int32) for L in lengths]
    for p in out:
        assert p["q_len"] > 0 and p["k_len"] > 0 and p["part_row"] == -1
        assert p["q_start"] + p["q_len"] <= lengths[p["seq"]] and p["k_start"] + p["k_len"] <= lengths[p["seq"]]
        cover[p["seq"]][p["q_start"]:p["q_start"] + p["q_len"], p["k_start"]:p["k_start"] + p["k_len"]] += \
            _visible(p, causal)
    want = [np.zeros((L, L), np.int32) for L in lengths]
    for p in whole:
        want[p["seq"]][p["q_start"]:p["q_start"] + p["q_len"], p["k_start"]:p["k_start"] + p["k_len"]] += \
            _visible(p, causal)
    for c, w in zip(cover, want):
        assert np.array_equal(c, w)
    # a band's dS buffer (16 KB per visible 64 x 128 block and head, plus one spare block) fits the scratch
    for b in range(n_bands):
        blocks = 1
        for p in out[band == b]:
            for jk in range(0, p["k_len"], 128):
                first_q = max(0, p["k_start"] + jk - p["q_start"]) if causal else 0
                if first_q < p["q_len"]:
                    blocks += (p["q_len"] + 63) // 64 - first_q // 64
        assert blocks * 16384 * h <= scratch + 4 * 16384 * h * len(out[band == b]), (b, blocks)
    if scratch >= 1 << 30:
        assert n_bands == 1
    elif sum(L * L for L in lengths) > 1 << 20:
        assert n_bands > 1


def test_bands_refuse_a_scratch_smaller_than_one_tile_column():
    out, band, n_bands = P.hydra_bwd_bands([0, 4096], 4, None, True, 1 << 16)
    assert n_bands == 0 and len(out) == 0


def test_ulysses_pack_validation_without_a_gpu():
    args = dict(stream=0, check=False)
    assert P.hydra_ulysses_pack(0x1000, 8, 6, 8, 4, 0x2000, **args) == P.HYDRA_ERR_INVALID_ARG     # 4 does not divide 6
    assert P.hydra_ulysses_pack(0x1000, 8, 3, 4, 3, 0x2000, **args) == P.HYDRA_ERR_UNSUPPORTED     # 8-byte chunks
    assert P.hydra_ulysses_pack(0x1000, 0, 4, 8, 2, 0x2000, **args) == P.HYDRA_OK                  # nothing to move
    assert P.hydra_ulysses_pack(0x1000, 8, 4, 8, 2, 0x1000, **args) == P.HYDRA_ERR_INVALID_ARG     # in place
    assert P.hydra_ulysses_unpack(0x1008, 8, 4, 8, 2, 0x2000, **args) == P.HYDRA_ERR_INVALID_ARG   # misaligned
    assert P.hydra_ulysses_unpack(0, 8, 4, 8, 2, 0x2000, **args) == P.HYDRA_ERR_INVALID_ARG
    assert P.hydra_ulysses_pack(0x1000, 1 << 34, 64, 192, 4, 0x2000, **args) == P.HYDRA_ERR_UNSUPPORTED
    assert P.hydra_ulysses_pack(0x1000, -1, 4, 8, 2, 0x2000, **args) == P.HYDRA_ERR_INVALID_ARG


def test_workspace_bytes_with_the_band_scratch():
    """Over the dS limit the backward asks for the base size alone, or, with the bands switched on, for the
    base size + an fp32 dq + the scratch (capped by the full dS buffer)."""
    cu, h = [0, 20000], 4
    try:
        P.hydra_set_bwd_scratch_limit(1 << 30)
        P.hydra_set_bwd_band_scratch(0)
        base = P.hydra_workspace_bytes(P.HYDRA_WS_BWD, cu, h)
        assert 20000 * h * 4 <= base < 20000 * h * 4 + (1 << 16)          # D only: dS (1.6 GB) is over the limit
        P.hydra_set_bwd_band_scratch(256 << 20)
        banded = P.hydra_workspace_bytes(P.HYDRA_WS_BWD, cu, h)
        acc = 20000 * h * 192 * 4
        assert base + acc + (256 << 20) <= banded <= base + acc + (256 << 20) + 4096
        P.hydra_set_bwd_band_scratch(64 << 30)                            # more than the whole buffer: capped
        capped = P.hydra_workspace_bytes(P.HYDRA_WS_BWD, cu, h)
        full = 20000 * 20000 // 2 * 2 * h
        assert base + acc + full <= capped <= base + acc + int(full * 1.05) + (1 << 20)
        # the default: as much scratch as the dS limit while the whole buffer is at most 16 times the limit
        P.hydra_set_bwd_band_scratch(P.HYDRA_BAND_AUTO)
        P.hydra_set_bwd_scratch_limit(256 << 20)                          # 1.6 GB of dS: 7 bands
        assert P.hydra_workspace_bytes(P.HYDRA_WS_BWD, cu, h) == banded
        P.hydra_set_bwd_scratch_limit(64 << 20)                           # 25 bands: too many, recompute instead
        assert P.hydra_workspace_bytes(P.HYDRA_WS_BWD, cu, h) == base
        P.hydra_set_bwd_scratch_limit(4 << 30)                            # under the limit: the bands play no part
        assert P.hydra_workspace_bytes(P.HYDRA_WS_BWD, cu, h) <= base + int(full * 1.05) + (1 << 20)
        # grouped-query form: fp32 dk, dv of the KV heads on top
        g = P.hydra_workspace_bytes_gqa(P.HYDRA_WS_BWD, cu, h, 2)
        assert g >= P.hydra_workspace_bytes(P.HYDRA_WS_BWD, cu, h) + 20000 * 2 * (192 + 128) * 4
        assert P.hydra_workspace_bytes_gqa(P.HYDRA_WS_BWD, cu, h, 3) == 0  # 3 does not divide 4
    finally:
        P.hydra_set_bwd_scratch_limit(4 << 30)
        P.hydra_set_bwd_band_scratch(P.HYDRA_BAND_AUTO)


@pytest.mark.parametrize("seed", range(12))
def test_bands_cover_random_problems_exactly_once(seed):
    rng = np.random.default_rng(7000 + seed)
    n = int(rng.integers(1, 5))
    lengths = [int(v) for v in rng.choice([1, 65, 128, 200, 383, 640, 777, 1025, 1500], size=n)]
    cp_r = [int(v) for v in rng.choice([0, 1, 2, 3], size=n)]
    causal = bool(rng.integers(0, 2))
    h = int(rng.integers(1, 4))
    scratch = int(rng.integers(1 << 20, 4 << 20))
    cu = np.concatenate([[0], np.cumsum(lengths)]).astype(np.int32)
    pairs = P.hydra_zigzag_pairs(cu, cp_r)[0] if any(cp_r) else None
    whole = pairs if pairs is not None else np.array(
        [(b, 0, L, 0, L, -1, b, 0) for b, L in enumerate(lengths)], dtype=P.PAIR_DTYPE)
    out, band, n_bands = P.hydra_bwd_bands(cu, h, pairs, causal, scratch)
    if n_bands == 0:                       # a single tile column over the scratch: the caller recomputes
        assert max(lengths) * 128 * 2 * h * 2 > scratch // 2
        return
    cover = [np.zeros((L, L), np.int32) for L in lengths]
    for p in out:
        cover[p["seq"]][p["q_start"]:p["q_start"] + p["q_len"], p["k_start"]:p["k_start"] + p["k_len"]] += \
            _visible(p, causal)
    want = [np.zeros((L, L), np.int32) for L in lengths]
    for p in whole:
        if p["q_len"] > 0 and p["k_len"] > 0:
            want[p["seq"]][p["q_start"]:p["q_start"] + p["q_len"], p["k_start"]:p["k_start"] + p["k_len"]] += \
                _visible(p, causal)
    for c, w in zip(cover, want):
        assert np.array_equal(c, w)
    # a key tile of a chunk lies in one band only (dk, dv of a band are final)
    owner = {}
    for p, b in zip(out, band):
        for k0 in range(p["k_start"], p["k_start"] + p["k_len"], 128):
            assert owner.setdefault((int(p["seq"]), int(k0)), int(b)) == int(b)


def test_plan_build_timer_is_host_only_and_bounded():
    """The work tables of a call are built on the host; the timer needs no GPU. A new cu_seqlens must not cost
    more than the kernels it feeds: the many-short batch (690 chunk pairs, 32 heads, 22 000 forward items)
    builds each of its three tables in well under ten milliseconds even on a slow host."""
    import hydra_workloads as hw
    w = hw.workload("short64k_split")
    cu = w.cu()
    pairs, _, _, _ = P.hydra_zigzag_pairs(cu, w.cp_r)
    for kind in (P.HYDRA_WS_FWD, P.HYDRA_WS_MERGE, P.HYDRA_WS_BWD):
        t = min(P.hydra_plan_build_seconds(kind, cu, w.n_heads, pairs) for _ in range(3))
        assert 0.0 <= t < 10e-3, (kind, t)
    assert P.hydra_plan_build_seconds(7, cu, w.n_heads, pairs) < 0
