"""Oracle of grouped-query attention (Table "Notation": h query heads and h_kv KV heads per rank, h_kv << h
for the GQA model of Section 6, which shares eight KV heads).

TEST INFRASTRUCTURE ONLY. Nothing in the product path imports this module.

Definition used (the paper names the head counts only; this is the usual grouping, taken as a reading):
with g = h / h_kv, query head a attends to KV head a // g. So the forward is the
per-head attention of the plain oracle on K, V with every KV head written out g times, and the gradient of
a KV head is the SUM of the per-head gradients of the g query heads that read it. The two steps are written
exactly like that: expand, call the plain oracle, sum.
"""
import numpy as np

from . import attention as A


def expand_kv(x: np.ndarray, h: int) -> np.ndarray:
    """[T, h_kv, d] -> [T, h, d]: query head a reads KV head a // (h / h_kv)."""
    T, h_kv, d = x.shape
    if h_kv < 1 or h % h_kv:
        raise ValueError("the number of KV heads must divide the number of query heads")
    g = h // h_kv
    out = np.empty((T, h, d), dtype=x.dtype)
    for a in range(h):
        out[:, a, :] = x[:, a // g, :]
    return out


def reduce_kv(dx: np.ndarray, h_kv: int) -> np.ndarray:
    """[T, h, d] per-query-head gradients -> [T, h_kv, d]: the sum over the heads of each group."""
    T, h, d = dx.shape
    g = h // h_kv
    out = np.zeros((T, h_kv, d), dtype=np.float64)
    for a in range(h):
        out[:, a // g, :] += dx[:, a, :]
    return out


def attn_fwd_gqa(q, k, v, cu_seqlens, causal: bool, scale: float):
    h = q.shape[1]
    return A.attn_fwd(q, expand_kv(k, h), expand_kv(v, h), cu_seqlens, causal, scale)


def attn_bwd_gqa(q, k, v, dout, cu_seqlens, causal: bool, scale: float, out, lse):
    """Returns dq [T,h,dqk], dk [T,h_kv,dqk], dv [T,h_kv,dv] in float64."""
    h, h_kv = q.shape[1], k.shape[1]
    dq, dk, dv = A.attn_bwd(q, expand_kv(k, h), expand_kv(v, h), dout, cu_seqlens, causal, scale, out, lse)
    return dq, reduce_kv(dk, h_kv), reduce_kv(dv, h_kv)


def attn_bwd_pairs_gqa(q, k, v, dout, cu_seqlens, pairs, causal: bool, scale: float, lse, d):
    """The same over a list of chunk pairs, each using the merged LSE and D."""
    h, h_kv = q.shape[1], k.shape[1]
    dq, dk, dv = A.attn_bwd_pairs(q, expand_kv(k, h), expand_kv(v, h), dout, cu_seqlens, pairs, causal, scale,
                                  lse, d)
    return dq, reduce_kv(dk, h_kv), reduce_kv(dv, h_kv)
