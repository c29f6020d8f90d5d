"""ctypes front-end of the fp64 oracle, plus the oracle's own chunk cutter.

TEST INFRASTRUCTURE: imported only by tests, the smoke check and the benchmark's CPU legs.

The attention arithmetic is in ``hydra_oracle.c``; this file marshals numpy arrays and implements,
independently of the CUDA library, the integer bookkeeping of the outer ring (Section 5.2,
Eq. (usp): a degree P is factored into an inner Ulysses group cp_u and an outer ring cp_r; a ring
of cp_r ranks cuts a sequence into 2*cp_r zigzag chunks so that rank r owns chunks r and
2*cp_r-1-r, and every causal (q-chunk, kv-chunk) pair is one partial attention problem).
"""
from __future__ import annotations

import ctypes
import hashlib
import os
import subprocess
from typing import Dict, List, Sequence, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "hydra_oracle.c")
_LIB = None


def _host_tag() -> str:
    """The library is compiled for the CPU it runs on; a copy built elsewhere is not reused."""
    flags = ""
    try:
        with open("/proc/cpuinfo") as f:
            for line in f:
                if line.startswith("flags"):
                    flags = line
                    break
    except OSError:
        pass
    with open(_SRC, "rb") as f:
        src = f.read()
    return hashlib.sha1(flags.encode() + src).hexdigest()[:12]


def build() -> str:
    """Compile hydra_oracle.c with gcc + OpenMP (no fast-math) and return the .so path."""
    so = os.path.join(_HERE, f"libhydra_oracle.{_host_tag()}.so")
    if not os.path.exists(so):
        tmp = so + f".tmp{os.getpid()}"
        cmd = ["gcc", "-O3", "-march=native", "-fno-fast-math", "-ffp-contract=off", "-fopenmp",
               "-fvisibility=hidden", "-shared", "-fPIC", "-o", tmp, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
        os.replace(tmp, so)
    return so


def _lib():
    global _LIB
    if _LIB is None:
        _LIB = ctypes.CDLL(build())
        _LIB.oracle_p_row.restype = ctypes.c_int64
    return _LIB


def n_threads() -> int:
    """Threads the OpenMP loops use (OMP_NUM_THREADS if set, else all cores)."""
    env = os.environ.get("OMP_NUM_THREADS")
    if env:
        return int(env.split(",")[0])
    return os.cpu_count() or 1


# ------------------------------------------------------------------------------------------------
# integer helpers (the oracle's own; the CUDA library has an independent implementation)
# ------------------------------------------------------------------------------------------------
def zigzag_chunks(length: int, cp_r: int) -> List[Tuple[int, int]]:
    """(start, len) of the 2*cp_r contiguous chunks of a sequence; boundaries floor(c*L/n_c).

    cp_r == 0 means "not cut": one chunk holding the whole sequence.  Empty chunks are kept in
    the list (len 0) so that chunk indices keep their meaning; pair enumeration drops them.
    """
    n_c = 1 if cp_r == 0 else 2 * cp_r
    edges = [(c * length) // n_c for c in range(n_c + 1)]
    return [(edges[c], edges[c + 1] - edges[c]) for c in range(n_c)]


def zigzag_rank(chunk: int, cp_r: int) -> int:
    """Ring rank that owns a chunk: r for the first cp_r chunks, mirrored for the rest."""
    if cp_r == 0:
        return 0
    return chunk if chunk < cp_r else 2 * cp_r - 1 - chunk


def causal_pairs(cu_seqlens: Sequence[int], cp_r: Sequence[int] | int) -> List[Dict[str, int]]:
    """All causal (q-chunk, kv-chunk) pairs of a packed batch, kv chunk not later than q chunk.

    Each entry: seq, q_start, q_len, k_start, k_len, qc, kc, rank (owner of the q chunk),
    step ((rank(qc) - rank(kc)) mod cp_r: the ring step at which that K/V block visits),
    group (running index of the q chunk; pairs of a group are merged), diagonal (0/1).
    """
    n = len(cu_seqlens) - 1
    degs = [cp_r] * n if isinstance(cp_r, int) else list(cp_r)
    pairs: List[Dict[str, int]] = []
    group = 0
    for b in range(n):
        length = int(cu_seqlens[b + 1]) - int(cu_seqlens[b])
        chunks = zigzag_chunks(length, degs[b])
        for qc, (qs, ql) in enumerate(chunks):
            if ql == 0:
                continue
            for kc in range(qc + 1):
                ks, kl = chunks[kc]
                if kl == 0:
                    continue
                ring = max(degs[b], 1)
                pairs.append(dict(seq=b, q_start=qs, q_len=ql, k_start=ks, k_len=kl, qc=qc, kc=kc,
                                  rank=zigzag_rank(qc, degs[b]),
                                  step=(zigzag_rank(qc, degs[b]) - zigzag_rank(kc, degs[b])) % ring,
                                  group=group, diagonal=int(qc == kc)))
            group += 1
    return pairs


# ------------------------------------------------------------------------------------------------
# marshalling
# ------------------------------------------------------------------------------------------------
_F64_INPUTS = False


class f64_inputs:
    """Context manager: q, k, v, dO are float64 arrays instead of bf16 bit patterns.

    Exists for the finite-difference pin only (steps far below bf16 resolution)."""

    def __enter__(self):
        global _F64_INPUTS
        _F64_INPUTS = True
        _lib().oracle_set_inputs_f64(ctypes.c_int(1))

    def __exit__(self, *exc):
        global _F64_INPUTS
        _F64_INPUTS = False
        _lib().oracle_set_inputs_f64(ctypes.c_int(0))


def _u16(x: np.ndarray) -> np.ndarray:
    x = np.ascontiguousarray(x)
    want = np.float64 if _F64_INPUTS else np.uint16
    if x.dtype != want:
        raise TypeError(f"oracle inputs must be {want.__name__} here (bf16 bit patterns by default)")
    return x


def usp_factor(degree: int, heads: int) -> Tuple[int, int]:
    """Eq. (usp): P = cp_u * cp_r with cp_u = min(P, h), cp_r = P / cp_u."""
    cp_u = min(degree, heads)
    if degree % cp_u:
        raise ValueError("degree is not a multiple of its Ulysses factor")
    return cp_u, degree // cp_u


def _p(a: np.ndarray):
    return a.ctypes.data_as(ctypes.c_void_p)


def _cu(cu_seqlens) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(cu_seqlens, dtype=np.int32))


def attn_fwd(q, k, v, cu_seqlens, causal: bool, scale: float):
    """Unchunked attention of a packed batch. q,k [T,h,dqk], v [T,h,dv] (uint16 bf16 bits).

    Returns out [T,h,dv] float64 and lse [h,T] float64.  ``scale`` is widened from float32.
    """
    q, k, v, cu = _u16(q), _u16(k), _u16(v), _cu(cu_seqlens)
    T, h, dqk = q.shape
    dv = v.shape[2]
    out = np.zeros((T, h, dv), dtype=np.float64)
    lse = np.full((h, T), -np.inf, dtype=np.float64)
    _lib().oracle_attn_fwd(_p(q), _p(k), _p(v), _p(cu), ctypes.c_int(len(cu) - 1), ctypes.c_int(h),
                           ctypes.c_int(dqk), ctypes.c_int(dv), ctypes.c_int(int(causal)),
                           ctypes.c_double(float(np.float32(scale))), _p(out), _p(lse))
    return out, lse


def attn_partial(q, k, v, cu_seqlens, pair: Dict[str, int], causal: bool, scale: float):
    """Partial (O [q_len,h,dv], LSE [h,q_len]) of one (q-chunk, kv-chunk) pair."""
    q, k, v, cu = _u16(q), _u16(k), _u16(v), _cu(cu_seqlens)
    _, h, dqk = q.shape
    dv = v.shape[2]
    ql = int(pair["q_len"])
    o = np.zeros((ql, h, dv), dtype=np.float64)
    l = np.full((h, ql), -np.inf, dtype=np.float64)
    _lib().oracle_attn_partial(_p(q), _p(k), _p(v), _p(cu), ctypes.c_int(int(pair["seq"])),
                               ctypes.c_int(h), ctypes.c_int(dqk), ctypes.c_int(dv),
                               ctypes.c_int(int(pair["q_start"])), ctypes.c_int(ql),
                               ctypes.c_int(int(pair["k_start"])), ctypes.c_int(int(pair["k_len"])),
                               ctypes.c_int(int(causal)), ctypes.c_double(float(np.float32(scale))),
                               _p(o), _p(l))
    return o, l


def lse_merge(o_parts: Sequence[np.ndarray], lse_parts: Sequence[np.ndarray]):
    """One-shot n-way merge of partials that cover the same rows."""
    n = len(o_parts)
    o_parts = [np.ascontiguousarray(o, dtype=np.float64) for o in o_parts]
    lse_parts = [np.ascontiguousarray(l, dtype=np.float64) for l in lse_parts]
    rows, h, dv = o_parts[0].shape
    out = np.zeros((rows, h, dv), dtype=np.float64)
    lse = np.zeros((h, rows), dtype=np.float64)
    op = (ctypes.c_void_p * n)(*[o.ctypes.data for o in o_parts])
    lp = (ctypes.c_void_p * n)(*[l.ctypes.data for l in lse_parts])
    _lib().oracle_lse_merge(ctypes.c_int(n), op, lp, ctypes.c_int64(rows), ctypes.c_int(h),
                            ctypes.c_int(dv), _p(out), _p(lse))
    return out, lse


def bwd_prep(dout, out: np.ndarray) -> np.ndarray:
    """D [h,T] = rowsum(dO * O) with the fp64 O."""
    dout = _u16(dout)
    out = np.ascontiguousarray(out, dtype=np.float64)
    T, h, dv = dout.shape
    d = np.zeros((h, T), dtype=np.float64)
    _lib().oracle_bwd_prep(_p(dout), _p(out), ctypes.c_int64(T), ctypes.c_int(h), ctypes.c_int(dv),
                           _p(d))
    return d


def attn_bwd(q, k, v, dout, cu_seqlens, causal: bool, scale: float, out, lse):
    """Unchunked backward; returns dq, dk [T,h,dqk] and dv [T,h,dv] in float64."""
    q, k, v, dout, cu = _u16(q), _u16(k), _u16(v), _u16(dout), _cu(cu_seqlens)
    T, h, dqk = q.shape
    dv = v.shape[2]
    out = np.ascontiguousarray(out, dtype=np.float64)
    lse = np.ascontiguousarray(lse, dtype=np.float64)
    dq = np.zeros((T, h, dqk)); dk = np.zeros((T, h, dqk)); dvv = np.zeros((T, h, dv))
    _lib().oracle_attn_bwd(_p(q), _p(k), _p(v), _p(dout), _p(cu), ctypes.c_int(len(cu) - 1),
                           ctypes.c_int(h), ctypes.c_int(dqk), ctypes.c_int(dv),
                           ctypes.c_int(int(causal)), ctypes.c_double(float(np.float32(scale))),
                           _p(out), _p(lse), _p(dq), _p(dk), _p(dvv))
    return dq, dk, dvv


def attn_bwd_pairs(q, k, v, dout, cu_seqlens, pairs: Sequence[Dict[str, int]], causal: bool,
                   scale: float, lse, d):
    """Backward summed over the listed pairs, each using the merged LSE and D (both [h,T])."""
    q, k, v, dout, cu = _u16(q), _u16(k), _u16(v), _u16(dout), _cu(cu_seqlens)
    T, h, dqk = q.shape
    dv = v.shape[2]
    lse = np.ascontiguousarray(lse, dtype=np.float64)
    d = np.ascontiguousarray(d, dtype=np.float64)
    dq = np.zeros((T, h, dqk)); dk = np.zeros((T, h, dqk)); dvv = np.zeros((T, h, dv))
    for p in pairs:
        _lib().oracle_attn_bwd_pair(_p(q), _p(k), _p(v), _p(dout), _p(cu),
                                    ctypes.c_int(len(cu) - 1), ctypes.c_int(int(p["seq"])),
                                    ctypes.c_int(h), ctypes.c_int(dqk), ctypes.c_int(dv),
                                    ctypes.c_int(int(p["q_start"])), ctypes.c_int(int(p["q_len"])),
                                    ctypes.c_int(int(p["k_start"])), ctypes.c_int(int(p["k_len"])),
                                    ctypes.c_int(int(causal)),
                                    ctypes.c_double(float(np.float32(scale))), _p(lse), _p(d),
                                    _p(dq), _p(dk), _p(dvv))
    return dq, dk, dvv


def p_row(q, k, cu_seqlens, seq: int, head: int, i: int, causal: bool, scale: float) -> np.ndarray:
    """Softmax probabilities of query row i of one sequence and head."""
    q, k, cu = _u16(q), _u16(k), _cu(cu_seqlens)
    _, h, dqk = q.shape
    length = int(cu[seq + 1] - cu[seq])
    buf = np.zeros(max(length, 1), dtype=np.float64)
    nk = _lib().oracle_p_row(_p(q), _p(k), _p(cu), ctypes.c_int(seq), ctypes.c_int(h),
                             ctypes.c_int(head), ctypes.c_int(dqk), ctypes.c_int64(i),
                             ctypes.c_int(int(causal)), ctypes.c_double(float(np.float32(scale))),
                             _p(buf))
    return buf[:nk]


def sample_rows(q, k, v, dout, cu_seqlens, causal: bool, scale: float, tok, head):
    """O, LSE, D, dQ of sampled (token, head) query rows of the unchunked problem."""
    q, k, v, dout, cu = _u16(q), _u16(k), _u16(v), _u16(dout), _cu(cu_seqlens)
    _, h, dqk = q.shape
    dv = v.shape[2]
    tok = np.ascontiguousarray(tok, dtype=np.int64)
    head = np.ascontiguousarray(head, dtype=np.int32)
    n = len(tok)
    o = np.zeros((n, dv)); lse = np.zeros(n); dsum = np.zeros(n); dq = np.zeros((n, dqk))
    _lib().oracle_sample_rows(_p(q), _p(k), _p(v), _p(dout), _p(cu), ctypes.c_int(len(cu) - 1),
                              ctypes.c_int(h), ctypes.c_int(dqk), ctypes.c_int(dv),
                              ctypes.c_int(int(causal)), ctypes.c_double(float(np.float32(scale))),
                              ctypes.c_int64(n), _p(tok), _p(head), _p(o), _p(lse), _p(dsum), _p(dq))
    return o, lse, dsum, dq


def sample_keys(q, k, v, dout, cu_seqlens, causal: bool, scale: float, tok, head):
    """dK, dV of sampled (token, head) key rows of the unchunked problem."""
    q, k, v, dout, cu = _u16(q), _u16(k), _u16(v), _u16(dout), _cu(cu_seqlens)
    _, h, dqk = q.shape
    dv = v.shape[2]
    tok = np.ascontiguousarray(tok, dtype=np.int64)
    head = np.ascontiguousarray(head, dtype=np.int32)
    n = len(tok)
    dk = np.zeros((n, dqk)); dvv = np.zeros((n, dv))
    _lib().oracle_sample_keys(_p(q), _p(k), _p(v), _p(dout), _p(cu), ctypes.c_int(len(cu) - 1),
                              ctypes.c_int(h), ctypes.c_int(dqk), ctypes.c_int(dv),
                              ctypes.c_int(int(causal)), ctypes.c_double(float(np.float32(scale))),
                              ctypes.c_int64(n), _p(tok), _p(head), _p(dk), _p(dvv))
    return dk, dvv


def spike_bwd(q, k, v, dout, cu_seqlens, causal: bool, scale: float, tok):
    """Backward when dO is zero outside the query rows `tok` (all heads of each): returns dQ of those rows
    [n, h, dqk] and dK [T, h, dqk], dV [T, h, dv] of every key row. The caller passes a dO that is zero
    elsewhere; only the listed rows are read."""
    q, k, v, dout, cu = _u16(q), _u16(k), _u16(v), _u16(dout), _cu(cu_seqlens)
    T, h, dqk = q.shape
    dv = v.shape[2]
    assert dqk <= 512 and dv <= 512
    tok = np.ascontiguousarray(tok, dtype=np.int64)
    n = len(tok)
    dq = np.zeros((n, h, dqk)); dk = np.zeros((T, h, dqk)); dvv = np.zeros((T, h, dv))
    _lib().oracle_spike_bwd(_p(q), _p(k), _p(v), _p(dout), _p(cu), ctypes.c_int(len(cu) - 1), ctypes.c_int(h),
                            ctypes.c_int(dqk), ctypes.c_int(dv), ctypes.c_int(int(causal)),
                            ctypes.c_double(float(np.float32(scale))), ctypes.c_int64(n), _p(tok), _p(dq), _p(dk),
                            _p(dvv))
    return dq, dk, dvv
