"""Parity at the full sizes of the five benchmark configurations, in the launch configuration the
benchmark times.  The oracle is quadratic, so: the 32K and 64K configurations are checked in full on
a subset of heads (heads are independent and generated from independent streams); the 128K and 256K
configurations are checked on sampled query rows (O, LSE, dQ: cost linear in the row's position),
on sampled key rows near the end of the long sequence (dK, dV) and through gradient identities that
hold at any size."""
import numpy as np
import pytest
import torch

import hydra_workloads as hw
import oracle
from gpu_util import TOL_LSE, TOL_REL, check, pairs_for

pytestmark = pytest.mark.gpu
DQK, DV = hw.D_QK, hw.D_V


_INPUT_CACHE = {}


def device_inputs(w):
    """bf16 tensors of the whole workload on the GPU, generated one head at a time (kept for the next test
    of the same workload; a different workload takes the cache over)."""
    from paper_2609_34318_b200.runner import bits_to_tensor
    if w.name in _INPUT_CACHE:
        return _INPUT_CACHE[w.name]
    _INPUT_CACHE.clear()
    T, h = w.total, w.n_heads
    t = {n: torch.empty((T, h, DV if n in ("v", "do") else DQK), dtype=torch.bfloat16, device="cuda")
         for n in ("q", "k", "v", "do")}
    for a in range(h):
        for n in t:
            t[n][:, a, :] = bits_to_tensor(hw.tensor_bits(n, T, [a]))[:, 0, :]
    _INPUT_CACHE[w.name] = t
    return t


def run_workload(w, dout_rows=None):
    """Forward and backward of the whole workload. With `dout_rows` the upstream gradient is zeroed outside
    those tokens (a new tensor: the generated one is left as it is)."""
    from paper_2609_34318_b200.runner import AttnStep
    cu = w.cu()
    lib_pairs, rows, ora_pairs = pairs_for(cu, w.cp_r) if w.cp_r else (None, 0, None)
    t = device_inputs(w)
    if dout_rows is not None:
        keep = torch.zeros(w.total, dtype=torch.bool, device="cuda")
        keep[torch.as_tensor(np.asarray(dout_rows, dtype=np.int64), device="cuda")] = True
        t = dict(t)
        t["do"] = t["do"] * keep[:, None, None]
    step = AttnStep(cu, w.n_heads, lib_pairs, rows, True, float(w.scale))
    for buf in (step.out, step.lse, step.dq, step.dk, step.dv):
        buf.fill_(float("nan"))
    step.forward(t["q"], t["k"], t["v"])
    step.backward(t["q"], t["k"], t["v"], t["do"])
    status, detail = step.poll()
    assert status == 0, (status, detail)
    torch.cuda.synchronize()
    return step, t, ora_pairs


def head_subset_check(w, heads, step, ora_pairs):
    """Full oracle on a few heads against the same heads of the GPU result."""
    cu = w.cu()
    x = w.tensors(heads)
    out, lse = oracle.attn_fwd(x["q"], x["k"], x["v"], cu, True, w.scale)
    if ora_pairs is None:
        dq, dk, dv = oracle.attn_bwd(x["q"], x["k"], x["v"], x["do"], cu, True, w.scale, out, lse)
    else:
        d = oracle.bwd_prep(x["do"], out)
        dq, dk, dv = oracle.attn_bwd_pairs(x["q"], x["k"], x["v"], x["do"], cu, ora_pairs, True, w.scale, lse, d)
    ref = dict(out=out, lse=lse, dq=dq, dk=dk, dv=dv)
    hsel = torch.tensor(heads, device="cuda")
    got = dict(out=step.out.index_select(1, hsel), lse=step.lse.index_select(0, hsel),
               dq=step.dq.index_select(1, hsel), dk=step.dk.index_select(1, hsel),
               dv=step.dv.index_select(1, hsel))
    got = {n: v.float().cpu().numpy().astype(np.float64) for n, v in got.items()}
    return check(got, ref, label=f"{w.name} heads {heads} ")


def test_packed_32k_full_oracle_on_two_heads():
    w = hw.workload("packed32k")
    step, _, ora_pairs = run_workload(w)
    assert torch.isfinite(step.out.float()).all() and torch.isfinite(step.dq.float()).all()
    head_subset_check(w, [0, w.n_heads - 1], step, ora_pairs)


def test_many_short_64k_full_oracle_on_two_heads():
    w = hw.workload("short64k")
    step, _, ora_pairs = run_workload(w)
    assert torch.isfinite(step.dk.float()).all() and torch.isfinite(step.dv.float()).all()
    head_subset_check(w, [0, w.n_heads - 1], step, ora_pairs)


def test_many_short_64k_every_sequence_split_and_merged():
    w = hw.workload("short64k_split")
    step, _, ora_pairs = run_workload(w)
    assert len(ora_pairs) == 3 * len(w.lengths)
    head_subset_check(w, [5], step, ora_pairs)


def sampled_check(w, step, t, q_tokens, k_tokens, heads):
    """Sampled query rows and key rows of the unchunked problem (chunking is an exact identity)."""
    cu = w.cu()
    x = w.tensors(heads)
    for slot, a in enumerate(heads):
        tok = np.asarray(q_tokens, dtype=np.int64)
        hd = np.full(len(tok), slot, dtype=np.int32)
        o, l, _, dq = oracle.sample_rows(x["q"], x["k"], x["v"], x["do"], cu, True, w.scale, tok, hd)
        idx = torch.from_numpy(tok).cuda()
        g_o = step.out[idx, a].float().cpu().numpy().astype(np.float64)
        g_l = step.lse[a, idx].cpu().numpy().astype(np.float64)
        g_dq = step.dq[idx, a].float().cpu().numpy().astype(np.float64)
        assert np.abs(g_l - l).max() <= TOL_LSE, (w.name, a, np.abs(g_l - l).max())
        # the contract's max norm over the sampled rows, plus a per-row relative bound on late rows:
        # with near-flat softmax rows the max norm alone would not notice a late row that lost a
        # whole kv chunk, a 5 % row-relative bound does
        seq_of = np.searchsorted(cu, tok, side="right") - 1
        late = (tok - cu[seq_of]) >= 1024
        for name, g, r in (("out", g_o, o), ("dq", g_dq, dq)):
            assert np.abs(g - r).max() <= TOL_REL * np.abs(r).max(), (w.name, name, a)
            if late.any():
                rel = np.linalg.norm(g[late] - r[late], axis=1) / np.linalg.norm(r[late], axis=1)
                assert rel.max() <= 5e-2, (w.name, name, a, float(rel.max()))
        if len(k_tokens):
            tk = np.asarray(k_tokens, dtype=np.int64)
            hk = np.full(len(tk), slot, dtype=np.int32)
            dk, dv = oracle.sample_keys(x["q"], x["k"], x["v"], x["do"], cu, True, w.scale, tk, hk)
            idk = torch.from_numpy(tk).cuda()
            g_dk = step.dk[idk, a].float().cpu().numpy().astype(np.float64)
            g_dv = step.dv[idk, a].float().cpu().numpy().astype(np.float64)
            for name, g, r in (("dk", g_dk, dk), ("dv", g_dv, dv)):
                assert np.abs(g - r).max() <= TOL_REL * np.abs(r).max(), (w.name, name, a)


def gradient_identities(w, step, t):
    """Hold for any input: per (sequence, head) sum_j dV_j = sum_i dO_i and sum_j dK_j = 0, and
    sum_i <q_i, dQ_i> = sum_j <k_j, dK_j>. Checked in fp32 on the device for every head."""
    cu = w.cu()
    for b in range(len(w.lengths)):
        s = slice(int(cu[b]), int(cu[b + 1]))
        dv_sum = step.dv[s].float().sum(0)
        do_sum = t["do"][s].float().sum(0)
        scale = t["do"][s].float().abs().sum(0).clamp_min(1.0)
        assert ((dv_sum - do_sum).abs() / scale).max().item() < 1e-2, (w.name, b, "sum dV != sum dO")
        dk_sum = step.dk[s].float().sum(0).abs()
        dk_abs = step.dk[s].float().abs().sum(0).clamp_min(1e-3)
        assert (dk_sum / dk_abs).max().item() < 2e-2, (w.name, b, "sum dK != 0")
        qdq = (t["q"][s].float() * step.dq[s].float()).sum((0, 2))
        kdk = (t["k"][s].float() * step.dk[s].float()).sum((0, 2))
        mag = (t["k"][s].float() * step.dk[s].float()).abs().sum((0, 2)).clamp_min(1e-3)
        assert ((qdq - kdk).abs() / mag).max().item() < 2e-2, (w.name, b, "<q,dQ> != <k,dK>")


@pytest.fixture(params=["bands_off", "banded_48gb"])
def long_backward_form(request):
    """The two forms of the backward on the long configurations: dq recomputing S and dP (the dS buffer of
    the whole problem is over the limit), and the form bench.py times: bands of key rows with 48 GB of dS
    scratch."""
    import paper_2609_34318_b200 as P
    P.hydra_set_bwd_band_scratch((48 << 30) if request.param == "banded_48gb" else 0)
    yield request.param
    P.hydra_set_bwd_band_scratch(P.HYDRA_BAND_AUTO)


def bands_ran(w, form, launches):
    """The banded form launches the two backward kernels once per band."""
    import paper_2609_34318_b200 as P
    if form != "banded_48gb":
        assert launches <= 6
        return
    cu = w.cu()
    lib_pairs = pairs_for(cu, w.cp_r)[0] if w.cp_r else None
    n_bands = P.hydra_bwd_bands(cu, w.n_heads, lib_pairs, True, 48 << 30)[2]
    assert n_bands >= 2 and launches >= 2 * n_bands + 2, (n_bands, launches)


def test_skewed_128k_sampled_rows_and_identities(long_backward_form):
    import paper_2609_34318_b200 as P
    w = hw.workload("skewed128k")
    n0 = P.hydra_launch_count()
    step, t, _ = run_workload(w)
    bands_ran(w, long_backward_form, P.hydra_launch_count() - n0)
    cu = w.cu()
    b_long = int(np.argmax(w.lengths))
    lo, hi = int(cu[b_long]), int(cu[b_long + 1])
    rng = np.random.default_rng(1)
    q_tokens = sorted(set([lo, lo + 1, lo + 127, lo + 128, lo + 129, hi - 1, hi - 129, 0, int(cu[1]) - 1,
                           int(cu[-1]) - 1] + [int(v) for v in rng.integers(0, w.total, 40)]))
    k_tokens = [hi - 1, hi - 130, int(cu[-1]) - 1, 5]
    sampled_check(w, step, t, q_tokens, k_tokens, [0, w.n_heads - 1])
    gradient_identities(w, step, t)
    assert torch.isfinite(step.out.float()).all()


def test_ring_256k_sampled_rows_and_identities(long_backward_form):
    import paper_2609_34318_b200 as P
    w = hw.workload("ring256k")
    n0 = P.hydra_launch_count()
    step, t, ora_pairs = run_workload(w)
    bands_ran(w, long_backward_form, P.hydra_launch_count() - n0)
    assert len(ora_pairs) == 36
    L = w.total
    rng = np.random.default_rng(2)
    edges = [c * L // 8 for c in range(1, 8)]
    q_tokens = sorted(set([0, 1, 127, 128, L - 1] + [e + d for e in edges for d in (-1, 0, 1)] +
                          [int(v) for v in rng.integers(0, L, 24)]))
    k_tokens = [L - 1, L - 200]
    sampled_check(w, step, t, q_tokens, k_tokens, [0, w.n_heads - 1])
    gradient_identities(w, step, t)
    assert torch.isfinite(step.out.float()).all() and torch.isfinite(step.dq.float()).all()


# ------------------------------------------------------------------------------------------------
# every key row at full size: upstream gradient on a few query rows only
# ------------------------------------------------------------------------------------------------
def spike_rows(cu, lengths, n_chunks, rng):
    """Query rows that carry dO: first and last row of every chunk of the longest sequence, rows at 64- and
    128-row phase offsets inside chunks, rows of other sequences, and a few random ones."""
    b = int(np.argmax(lengths))
    lo, L = int(cu[b]), int(lengths[b])
    edges = [c * L // n_chunks for c in range(n_chunks + 1)]
    rows = []
    for c in range(n_chunks):
        rows += [lo + edges[c], lo + edges[c + 1] - 1]
        mid = edges[c] + (edges[c + 1] - edges[c]) // 2
        rows += [lo + mid - 1 - 64 * (c % 2), lo + mid + 63 + 128 * (c % 3)]
        rows += [lo + int(v) for v in rng.integers(edges[c], edges[c + 1], 3)]
    T = int(cu[-1])
    rows += [0, T - 1] + [int(v) for v in rng.integers(0, T, 6)]
    return sorted(set(r for r in rows if 0 <= r < T))


def spike_check(w, n_chunks, seed):
    """dO is non-zero on ~60 query rows, so the oracle gives dK and dV of EVERY key row (and dQ of those rows)
    in O(rows x L x d). Compared element by element on two heads: the contract's max norm per tensor, and the
    same 2e-2 inside every block of 128 key rows against that block's own largest reference value (the share
    of a late spike row in a late key block is ~1/position of the tensor's largest entry: only a per-block
    norm notices a block whose dS or P tile went wrong). dQ must be exactly zero off the spike rows."""
    cu = w.cu()
    rng = np.random.default_rng(seed)
    rows = spike_rows(cu, w.lengths, n_chunks, rng)
    step, t, _ = run_workload(w, dout_rows=rows)
    heads = [0, w.n_heads - 1]
    x = w.tensors(heads)
    keep = np.zeros(w.total, dtype=bool)
    keep[rows] = True
    x["do"][~keep] = 0
    dq_ref, dk_ref, dv_ref = oracle.spike_bwd(x["q"], x["k"], x["v"], x["do"], cu, True, w.scale, np.asarray(rows))
    hsel = torch.tensor(heads, device="cuda")
    worst = {}
    for name, got_t, ref in (("dk", step.dk, dk_ref), ("dv", step.dv, dv_ref)):
        got = got_t.index_select(1, hsel).float().cpu().numpy().astype(np.float64)
        assert np.isfinite(got).all(), (w.name, name)
        err = np.abs(got - ref)
        assert err.max() <= TOL_REL * np.abs(ref).max(), (w.name, name, err.max(), np.abs(ref).max())
        T = w.total
        nb = (T + 127) // 128
        pad = nb * 128 - T
        e_blk = np.pad(err, ((0, pad), (0, 0), (0, 0))).reshape(nb, -1).max(1)
        r_blk = np.pad(np.abs(ref), ((0, pad), (0, 0), (0, 0))).reshape(nb, -1).max(1)
        live = r_blk > 0
        ratio = e_blk[live] / r_blk[live]
        worst[name] = float(ratio.max())
        bad = np.nonzero(live)[0][ratio > TOL_REL]
        assert len(bad) == 0, (w.name, name, "key blocks over 2e-2 of their own maximum", bad[:8], ratio.max())
        # blocks whose reference is identically zero: no spike row sees them, or only the first row of a
        # sequence does (one key: dP = D exactly, which fp32 reproduces to ~1e-8)
        assert e_blk[~live].max(initial=0.0) <= 1e-6 * np.abs(ref).max(), \
            (w.name, name, "gradient where the reference is identically zero", e_blk[~live].max(initial=0.0))
    idx = torch.as_tensor(np.asarray(rows, dtype=np.int64), device="cuda")
    g_dq = step.dq.index_select(0, idx).index_select(1, hsel).float().cpu().numpy().astype(np.float64)
    assert np.abs(g_dq - dq_ref).max() <= TOL_REL * np.abs(dq_ref).max(), (w.name, "dq")
    # per spike row, relative to the row's own norm (row 0 of a sequence has dQ = 0 exactly: one key, dP = D)
    r_norm = np.linalg.norm(dq_ref.reshape(len(rows) * 2, -1), axis=1)
    e_norm = np.linalg.norm((g_dq - dq_ref).reshape(len(rows) * 2, -1), axis=1)
    live = r_norm > 1e-9 * r_norm.max()
    assert e_norm[~live].max(initial=0.0) <= 1e-5 * r_norm.max(), (w.name, "dq rows with zero reference")
    rel = e_norm[live] / r_norm[live]
    worst["dq_row"] = float(rel.max())
    assert rel.max() <= TOL_REL, (w.name, "dq rows", float(rel.max()))
    off = torch.ones(w.total, dtype=torch.bool, device="cuda")
    off[idx] = False
    assert step.dq[off].float().abs().max().item() == 0.0, (w.name, "dq off the spike rows")
    print(f"{w.name} spike dO on {len(rows)} rows: worst per-block dk {worst['dk']:.2e} dv {worst['dv']:.2e}, "
          f"dq row {worst['dq_row']:.2e}")


def test_ring_256k_every_key_row_with_spike_dout(long_backward_form):
    spike_check(hw.workload("ring256k"), 8, seed=3)


def test_skewed_128k_every_key_row_with_spike_dout(long_backward_form):
    spike_check(hw.workload("skewed128k"), 8, seed=4)
