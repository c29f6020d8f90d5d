"""Oracle of the elementwise steps of a gated multi-head-latent attention block around the attention kernel
(Section 5.2, "Exposed All-to-All Overlap": query rotary embedding; the KV up-projection's output split into
the value and the key's position-free part; the key's rotary embedding and concatenation; the gate), forward
and backward. TEST INFRASTRUCTURE: fp64 numpy written from the definitions, shares nothing with the CUDA
library. The paper names the steps, not their formulas; the readings are those stated with the entry points
in include/hydra_attn.h (rotary pairs (2i, 2i+1), angle = position * theta^(-2i/rope_dim); one rotary key
vector per token shared by all heads; up-projection rows [key part | value]; gate = sigmoid).

Pins (tests/test_oracle_mla_ops.py): a rotation written out by hand, position 0 = identity, norms kept,
rope(p1) after rope(p2) = rope(p1 + p2), scores of rotated q and k depend on the position difference only,
inverse after forward = identity; the backward of every step is the adjoint of its forward (<f(x), g> =
<x, f_bwd(g)>) and, for the gate, agrees with central differences.
"""
from __future__ import annotations

import numpy as np


def rope(x: np.ndarray, positions, rope_offset: int, rope_dim: int, theta: float, inverse: bool = False) -> np.ndarray:
    """x [T, h, d] float64. Rotates the pairs (2i, 2i+1) of columns [rope_offset, rope_offset + rope_dim)."""
    x = np.asarray(x, dtype=np.float64)
    y = x.copy()
    T = x.shape[0]
    for t in range(T):
        for i in range(rope_dim // 2):
            ang = float(positions[t]) * float(theta) ** (-2.0 * i / rope_dim)
            if inverse:
                ang = -ang
            c, s = np.cos(ang), np.sin(ang)
            a, b = x[t, :, rope_offset + 2 * i], x[t, :, rope_offset + 2 * i + 1]
            y[t, :, rope_offset + 2 * i] = a * c - b * s
            y[t, :, rope_offset + 2 * i + 1] = a * s + b * c
    return y


def kv_assemble(kv_up: np.ndarray, k_pe: np.ndarray, positions, d_nope: int, d_rope: int, d_v: int, theta: float):
    """kv_up [T, h, d_nope + d_v], k_pe [T, d_rope] -> k [T, h, d_nope + d_rope], v [T, h, d_v]."""
    kv_up = np.asarray(kv_up, dtype=np.float64)
    T, h, _ = kv_up.shape
    pe = rope(np.asarray(k_pe, dtype=np.float64)[:, None, :], positions, 0, d_rope, theta)[:, 0, :]
    k = np.zeros((T, h, d_nope + d_rope))
    v = np.zeros((T, h, d_v))
    for t in range(T):
        for a in range(h):
            k[t, a, :d_nope] = kv_up[t, a, :d_nope]
            k[t, a, d_nope:] = pe[t]
            v[t, a] = kv_up[t, a, d_nope:]
    return k, v


def kv_assemble_bwd(dk: np.ndarray, dv: np.ndarray, positions, d_nope: int, d_rope: int, d_v: int, theta: float):
    """The adjoint of kv_assemble: dkv_up [T, h, d_nope + d_v], dk_pe [T, d_rope]."""
    dk, dv = np.asarray(dk, dtype=np.float64), np.asarray(dv, dtype=np.float64)
    T, h, _ = dk.shape
    dkv_up = np.zeros((T, h, d_nope + d_v))
    summed = np.zeros((T, 1, d_rope))
    for t in range(T):
        for a in range(h):
            dkv_up[t, a, :d_nope] = dk[t, a, :d_nope]
            dkv_up[t, a, d_nope:] = dv[t, a]
            summed[t, 0] += dk[t, a, d_nope:]
    dk_pe = rope(summed, positions, 0, d_rope, theta, inverse=True)[:, 0, :]
    return dkv_up, dk_pe


def gate_apply(out: np.ndarray, gate: np.ndarray) -> np.ndarray:
    out, gate = np.asarray(out, dtype=np.float64), np.asarray(gate, dtype=np.float64)
    return out / (1.0 + np.exp(-gate))


def gate_apply_bwd(dy: np.ndarray, out: np.ndarray, gate: np.ndarray):
    dy, out, gate = (np.asarray(a, dtype=np.float64) for a in (dy, out, gate))
    s = 1.0 / (1.0 + np.exp(-gate))
    return dy * s, dy * out * s * (1.0 - s)
