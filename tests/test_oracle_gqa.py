"""Pins of the grouped-query oracle: it reduces to the plain oracle at h_kv = h, it agrees with a dense
numpy evaluation written for shared KV heads directly (no head is copied there), and its dK / dV are the
derivatives of the forward with respect to the SHARED tensors (central differences in float64), which a
missing or mis-grouped sum over the query heads of a group would break."""
import numpy as np
import pytest

import hydra_workloads as hw
import oracle


def dense_gqa(q, k, v, causal, scale):
    """One sequence, float64, softmax written out; query head a reads k[:, a // g]."""
    T, h, _ = q.shape
    g = h // k.shape[1]
    out = np.zeros((T, h, v.shape[2]))
    lse = np.zeros((h, T))
    for a in range(h):
        s = scale * (q[:, a, :] @ k[:, a // g, :].T)
        if causal:
            s = np.where(np.tril(np.ones((T, T), bool)), s, -np.inf)
        m = s.max(axis=1, keepdims=True)
        e = np.exp(s - m)
        z = e.sum(axis=1, keepdims=True)
        out[:, a, :] = (e / z) @ v[:, a // g, :]
        lse[a] = (m + np.log(z))[:, 0]
    return out, lse


def small(rng, T, h, h_kv, dqk=8, dv=4):
    f = lambda *s: rng.standard_normal(s)
    return f(T, h, dqk), f(T, h_kv, dqk), f(T, h_kv, dv), f(T, h, dv)


@pytest.mark.parametrize("h,h_kv,causal", [(4, 2, True), (6, 1, True), (4, 4, False), (8, 2, False)])
def test_forward_matches_a_dense_evaluation_with_shared_heads(h, h_kv, causal):
    rng = np.random.default_rng(h * 10 + h_kv)
    T = 19
    q, k, v, _ = small(rng, T, h, h_kv)
    scale = 0.3
    with oracle.f64_inputs():
        out, lse = oracle.attn_fwd_gqa(q, k, v, [0, T], causal, scale)
    ref_out, ref_lse = dense_gqa(q, k, v, causal, float(np.float32(scale)))
    assert np.abs(out - ref_out).max() < 1e-12 and np.abs(lse - ref_lse).max() < 1e-12


def test_equal_head_counts_reduce_to_the_plain_oracle():
    rng = np.random.default_rng(1)
    T, h = 40, 3
    x = {n: hw.f32_to_bf16_bits(rng.standard_normal((T, h, d)).astype(np.float32))
         for n, d in (("q", 16), ("k", 16), ("v", 8), ("do", 8))}
    cu = [0, 25, 40]
    out, lse = oracle.attn_fwd(x["q"], x["k"], x["v"], cu, True, 0.25)
    out_g, lse_g = oracle.attn_fwd_gqa(x["q"], x["k"], x["v"], cu, True, 0.25)
    assert np.array_equal(out, out_g) and np.array_equal(lse, lse_g)
    ref = oracle.attn_bwd(x["q"], x["k"], x["v"], x["do"], cu, True, 0.25, out, lse)
    got = oracle.attn_bwd_gqa(x["q"], x["k"], x["v"], x["do"], cu, True, 0.25, out, lse)
    for a, b in zip(ref, got):
        assert np.array_equal(a, b)


@pytest.mark.parametrize("h,h_kv", [(4, 2), (6, 1), (6, 3)])
def test_dk_dv_are_derivatives_with_respect_to_the_shared_tensors(h, h_kv):
    rng = np.random.default_rng(7 + h + h_kv)
    T = 11
    q, k, v, do = small(rng, T, h, h_kv)
    cu, scale, eps = [0, 6, T], 0.4, 1e-6

    def loss(kk, vv):
        with oracle.f64_inputs():
            o, _ = oracle.attn_fwd_gqa(q, kk, vv, cu, True, scale)
        return float((o * do).sum())

    with oracle.f64_inputs():
        out, lse = oracle.attn_fwd_gqa(q, k, v, cu, True, scale)
        dq, dk, dv = oracle.attn_bwd_gqa(q, k, v, do, cu, True, scale, out, lse)
    assert dk.shape == k.shape and dv.shape == v.shape and dq.shape == q.shape
    for _ in range(12):
        t, a, c = int(rng.integers(T)), int(rng.integers(h_kv)), int(rng.integers(k.shape[2]))
        kp, km = k.copy(), k.copy()
        kp[t, a, c] += eps
        km[t, a, c] -= eps
        fd = (loss(kp, v) - loss(km, v)) / (2 * eps)
        assert abs(fd - dk[t, a, c]) < 1e-6 * max(1.0, abs(fd)), ("dk", t, a, c, fd, dk[t, a, c])
        c = int(rng.integers(v.shape[2]))
        vp, vm = v.copy(), v.copy()
        vp[t, a, c] += eps
        vm[t, a, c] -= eps
        fd = (loss(k, vp) - loss(k, vm)) / (2 * eps)
        assert abs(fd - dv[t, a, c]) < 1e-6 * max(1.0, abs(fd)), ("dv", t, a, c, fd, dv[t, a, c])


def test_the_group_sum_is_over_consecutive_query_heads():
    dx = np.arange(2 * 6 * 1, dtype=np.float64).reshape(2, 6, 1)
    r = oracle.reduce_kv(dx, 3)
    assert r[:, :, 0].tolist() == [[0 + 1, 2 + 3, 4 + 5], [6 + 7, 8 + 9, 10 + 11]]
    e = oracle.expand_kv(np.array([[[1.0], [2.0]]]), 6)
    assert e[0, :, 0].tolist() == [1, 1, 1, 2, 2, 2]
    with pytest.raises(ValueError):
        oracle.expand_kv(np.zeros((1, 4, 1)), 6)
