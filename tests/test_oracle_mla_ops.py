"""Pins of the oracle of the gated-MLA elementwise steps (oracle/mla_ops.py) to what the mathematics fixes."""
import numpy as np

from oracle import mla_ops as M

THETA = 10000.0


def test_rotation_written_out_by_hand():
    # one token at position 3, one head, four rotary columns after two untouched ones
    x = np.array([[[5.0, -7.0, 1.0, 0.0, 0.0, 2.0]]])
    y = M.rope(x, [3], 2, 4, THETA)
    a0, a1 = 3.0, 3.0 * THETA ** (-0.5)                 # angles of pairs 0 and 1
    want = [5.0, -7.0, np.cos(a0), np.sin(a0), -2.0 * np.sin(a1), 2.0 * np.cos(a1)]
    np.testing.assert_allclose(y[0, 0], want, rtol=1e-14, atol=1e-15)


def test_rotation_properties():
    rng = np.random.default_rng(1)
    T, h, d, off, rd = 9, 3, 24, 8, 16
    x = rng.standard_normal((T, h, d))
    pos = rng.integers(0, 5000, T)
    y = M.rope(x, pos, off, rd, THETA)
    # columns outside the rotary range are untouched; norms of rotated pairs are kept
    assert np.array_equal(y[..., :off], x[..., :off])
    np.testing.assert_allclose((y[..., off:] ** 2).reshape(T, h, rd // 2, 2).sum(-1),
                               (x[..., off:] ** 2).reshape(T, h, rd // 2, 2).sum(-1), rtol=1e-12)
    # position 0 is the identity; inverse undoes forward; rotations compose by adding positions
    np.testing.assert_allclose(M.rope(x, np.zeros(T, dtype=int), off, rd, THETA), x, rtol=0, atol=0)
    np.testing.assert_allclose(M.rope(y, pos, off, rd, THETA, inverse=True), x, rtol=1e-11, atol=1e-12)
    p2 = rng.integers(0, 300, T)
    np.testing.assert_allclose(M.rope(M.rope(x, pos, off, rd, THETA), p2, off, rd, THETA),
                               M.rope(x, pos + p2, off, rd, THETA), rtol=1e-9, atol=1e-10)


def test_scores_depend_on_the_position_difference_only():
    rng = np.random.default_rng(2)
    q, k = rng.standard_normal((1, 1, 64)), rng.standard_normal((1, 1, 64))
    s = lambda m, n: float((M.rope(q, [m], 0, 64, THETA) * M.rope(k, [n], 0, 64, THETA)).sum())
    np.testing.assert_allclose(s(100, 40), s(1060, 1000), rtol=1e-9)
    np.testing.assert_allclose(s(7, 7), float((q * k).sum()), rtol=1e-12)
    assert abs(s(100, 40) - s(100, 41)) > 1e-3


def test_rotation_backward_is_its_adjoint():
    rng = np.random.default_rng(3)
    x, g = rng.standard_normal((6, 2, 20)), rng.standard_normal((6, 2, 20))
    pos = rng.integers(0, 1000, 6)
    lhs = (M.rope(x, pos, 4, 16, THETA) * g).sum()
    rhs = (x * M.rope(g, pos, 4, 16, THETA, inverse=True)).sum()
    np.testing.assert_allclose(lhs, rhs, rtol=1e-11)


def test_key_value_assembly_and_its_adjoint():
    rng = np.random.default_rng(4)
    T, h, dn, dr, dv = 5, 3, 8, 6, 4
    kv_up, k_pe = rng.standard_normal((T, h, dn + dv)), rng.standard_normal((T, dr))
    pos = rng.integers(0, 700, T)
    k, v = M.kv_assemble(kv_up, k_pe, pos, dn, dr, dv, THETA)
    assert k.shape == (T, h, dn + dr) and v.shape == (T, h, dv)
    assert np.array_equal(k[..., :dn], kv_up[..., :dn]) and np.array_equal(v, kv_up[..., dn:])
    pe = M.rope(k_pe[:, None, :], pos, 0, dr, THETA)[:, 0]
    for a in range(h):                                   # every head carries the same rotated vector
        np.testing.assert_allclose(k[:, a, dn:], pe, rtol=0, atol=0)
    gk, gv = rng.standard_normal(k.shape), rng.standard_normal(v.shape)
    dkv_up, dk_pe = M.kv_assemble_bwd(gk, gv, pos, dn, dr, dv, THETA)
    np.testing.assert_allclose((k * gk).sum() + (v * gv).sum(), (kv_up * dkv_up).sum() + (k_pe * dk_pe).sum(), rtol=1e-11)


def test_gate_and_its_backward():
    rng = np.random.default_rng(5)
    out, gate, dy = (rng.standard_normal((4, 2, 8)) for _ in range(3))
    y = M.gate_apply(out, gate)
    np.testing.assert_allclose(M.gate_apply(out, np.zeros_like(gate)), 0.5 * out, rtol=1e-15)
    np.testing.assert_allclose(M.gate_apply(out, np.full_like(gate, 40.0)), out, rtol=1e-15)
    d_out, d_gate = M.gate_apply_bwd(dy, out, gate)
    eps = 1e-6
    for idx in [(0, 0, 0), (3, 1, 7), (2, 0, 5)]:
        for which, grad in ((0, d_out), (1, d_gate)):
            args = [out.copy(), gate.copy()]
            args[which][idx] += eps
            up = (M.gate_apply(*args) * dy).sum()
            args[which][idx] -= 2 * eps
            dn = (M.gate_apply(*args) * dy).sum()
            np.testing.assert_allclose((up - dn) / (2 * eps), grad[idx], rtol=1e-7, atol=1e-9)
    assert y.shape == out.shape
