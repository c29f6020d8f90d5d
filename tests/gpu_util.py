"""Helpers of the GPU parity tests: run a problem through the C ABI and through the oracle."""
from __future__ import annotations

import numpy as np

import hydra_workloads as hw
import oracle

TOL_REL = 2e-2      # max |gpu - ref| <= TOL_REL * max |ref| on O, dQ, dK, dV
TOL_LSE = 1e-3      # absolute, on LSE
TOL_ABS = 1e-5      # applied ONLY to tensors whose reference is identically zero (dQ, dK of a length-1
                    # sequence): fp32 rounding of exp2(s - LSE) leaves ~1e-7 where the exact value is 0


def pairs_for(cu, cp_r):
    """(library pairs, part_rows, oracle pairs) for a uniform outer-ring degree (0 = not cut)."""
    import paper_2609_34318_b200 as P
    lib_pairs, part_rows, _, _ = P.hydra_zigzag_pairs(cu, cp_r)
    return lib_pairs, part_rows, oracle.causal_pairs(cu, cp_r)


GUARD_BYTES = 4096          # sentinel band before and after every output and the workspace
GUARD_FILL = 0xA5


def guard(step, names=("out", "lse", "o_part", "lse_part", "dq", "dk", "dv", "workspace")):
    """Re-homes the listed buffers of an AttnStep inside larger allocations whose margins hold a sentinel
    byte, and returns the function that checks the margins (compute-sanitizer is not available: a write
    before the first or past the last byte of a buffer shows here instead)."""
    import torch
    bands = []
    for n in names:
        old = getattr(step, n)
        nbytes = old.numel() * old.element_size()
        room = (nbytes + 255) // 256 * 256
        raw = torch.full((room + 2 * GUARD_BYTES,), GUARD_FILL, dtype=torch.uint8, device=old.device)
        assert raw.data_ptr() % 256 == 0
        new = raw[GUARD_BYTES:GUARD_BYTES + nbytes].view(old.dtype).view(old.shape)
        new.copy_(old)
        setattr(step, n, new)
        bands.append((n, raw, nbytes))

    def verify(where=""):
        for n, raw, nbytes in bands:
            lo = raw[:GUARD_BYTES]
            hi = raw[GUARD_BYTES + nbytes:]
            assert bool((lo == GUARD_FILL).all()), f"{where}{n}: bytes written before the buffer"
            assert bool((hi == GUARD_FILL).all()), f"{where}{n}: bytes written past the buffer"
    return verify


def run_gpu(x, cu, h, pairs=None, part_rows=0, causal=True, scale=None, backward=True, poison=True):
    """x: dict of uint16 bit arrays q, k, v, do. Returns dict of float64 numpy results. Every output and the
    workspace sit between sentinel bands that are checked after the calls."""
    import torch
    from paper_2609_34318_b200.runner import AttnStep, bits_to_tensor
    step = AttnStep(cu, h, pairs, part_rows, causal, scale)
    verify_guards = guard(step)
    if poison:
        for t in (step.out, step.lse, step.dq, step.dk, step.dv, step.o_part, step.lse_part):
            t.fill_(float("nan"))
    q, k, v, do = (bits_to_tensor(x[n]) for n in ("q", "k", "v", "do"))
    step.forward(q, k, v)
    res = {}
    if backward:
        step.backward(q, k, v, do)
    status, detail = step.poll()
    assert status == 0, f"device status {status} (item {detail})"
    torch.cuda.synchronize()
    verify_guards()
    T = int(cu[-1])
    res["out"] = step.out[:T].float().cpu().numpy().astype(np.float64)
    res["lse"] = step.lse[:, :T].cpu().numpy().astype(np.float64)
    if backward:
        res["dq"] = step.dq[:T].float().cpu().numpy().astype(np.float64)
        res["dk"] = step.dk[:T].float().cpu().numpy().astype(np.float64)
        res["dv"] = step.dv[:T].float().cpu().numpy().astype(np.float64)
    res["_step"] = step
    return res


def run_oracle(x, cu, causal=True, scale=None, pairs=None, backward=True):
    """Unchunked oracle forward; backward over `pairs` (oracle pair dicts) or unchunked."""
    scale = np.float32(1.0 / np.sqrt(np.float32(hw.D_QK))) if scale is None else np.float32(scale)
    out, lse = oracle.attn_fwd(x["q"], x["k"], x["v"], cu, causal, scale)
    res = dict(out=out, lse=lse)
    if backward:
        if pairs is None:
            dq, dk, dv = oracle.attn_bwd(x["q"], x["k"], x["v"], x["do"], cu, causal, scale, out, lse)
        else:
            d = oracle.bwd_prep(x["do"], out)
            dq, dk, dv = oracle.attn_bwd_pairs(x["q"], x["k"], x["v"], x["do"], cu, pairs, causal, scale,
                                               lse, d)
        res.update(dq=dq, dk=dk, dv=dv)
    return res


def check(got, ref, names=("out", "lse", "dq", "dk", "dv"), tol_rel=TOL_REL, tol_lse=TOL_LSE, label=""):
    report = {}
    for n in names:
        if n not in ref:
            continue
        g, r = got[n], ref[n]
        assert g.shape == r.shape, (n, g.shape, r.shape)
        assert np.isfinite(g[np.isfinite(r)]).all(), f"{label}{n}: non-finite values (unwritten rows?)"
        if n == "lse":
            fin = np.isfinite(r)
            err = np.abs(g[fin] - r[fin]).max() if fin.any() else 0.0
            assert np.array_equal(np.isneginf(g), np.isneginf(r)), f"{label}lse: -inf pattern differs"
            report[n] = err
            assert err <= tol_lse, f"{label}lse: max abs err {err:.3e} > {tol_lse}"
        else:
            err = np.abs(g - r).max()
            ref_max = np.abs(r).max()
            report[n] = err / max(ref_max, 1e-30)
            bound = tol_rel * ref_max if ref_max > 0 else TOL_ABS
            assert err <= bound, \
                f"{label}{n}: max abs err {err:.3e} > {tol_rel} * max|ref| = {tol_rel * ref_max:.3e}"
    return report


def row_rel_err(got, ref):
    """Per-row relative L2 error (rows = all leading axes), max over rows with a non-zero reference."""
    g = got.reshape(-1, got.shape[-1]); r = ref.reshape(-1, ref.shape[-1])
    nr = np.linalg.norm(r, axis=1)
    ok = nr > 0
    return float((np.linalg.norm(g - r, axis=1)[ok] / nr[ok]).max()) if ok.any() else 0.0


def oracle_merge_of_partials(cu, pairs, o_part, lse_part, T, h, out_cur=None, lse_cur=None):
    """fp64 merge (the oracle's) of partial buffers as they stand on the GPU, per merged q chunk; NaN elsewhere.
    With out_cur / lse_cur (numpy, [T,h,dv] / [h,T]) the current rows are one more input (streaming form)."""
    o_np = o_part.float().cpu().numpy().astype(np.float64)
    l_np = lse_part.cpu().numpy().astype(np.float64)
    out = np.full((T, h, hw.D_V), np.nan)
    lse = np.full((h, T), np.nan)
    i = 0
    while i < len(pairs):
        j = i
        while j < len(pairs) and pairs[j]["group"] == pairs[i]["group"]:
            j += 1
        p = pairs[i]
        if p["part_row"] >= 0 and p["q_len"] > 0:
            n = int(p["q_len"])
            os_ = [o_np[int(pairs[t]["part_row"]):int(pairs[t]["part_row"]) + n] for t in range(i, j)]
            ls_ = [l_np[:, int(pairs[t]["part_row"]):int(pairs[t]["part_row"]) + n] for t in range(i, j)]
            t0 = int(cu[p["seq"]]) + int(p["q_start"])
            if out_cur is not None:
                os_ = [out_cur[t0:t0 + n]] + os_
                ls_ = [lse_cur[:, t0:t0 + n]] + ls_
            mo, ml = oracle.lse_merge(os_, ls_)
            out[t0:t0 + n] = mo
            lse[:, t0:t0 + n] = ml
        i = j
    return out, lse
