"""Pins of the recurrent-state oracle (no GPU): plain-Python loops and the recurrence's closed forms.
The paper does not define the operator, so these pin the declared reading, not a paper value."""
import numpy as np
import pytest

from oracle import linear_attn as la


def rand_case(rng, B, Hk, Hv, dk, dv, slots=None):
    slots = slots or B
    state = rng.standard_normal((slots, Hv, dk, dv))
    q = rng.standard_normal((B, Hk, dk))
    k = rng.standard_normal((B, Hk, dk))
    k /= np.linalg.norm(k, axis=-1, keepdims=True)
    v = rng.standard_normal((B, Hv, dv))
    a = rng.uniform(0.5, 1.0, (B, Hv))
    beta = rng.uniform(0.0, 1.0, (B, Hv))
    return state, q, k, v, a, beta


def loops(state, slot, q, k, v, a, beta, scale):
    B, Hk, dk = len(q), len(q[0]), len(q[0][0])
    Hv, dv = len(v[0]), len(v[0][0])
    out = [[[0.0] * dv for _ in range(Hv)] for _ in range(B)]
    st = state.tolist()
    for b in range(B):
        s = slot[b]
        if s < 0:
            continue
        for h in range(Hv):
            hk = h // (Hv // Hk)
            S = st[s][h]
            for i in range(dk):
                for j in range(dv):
                    S[i][j] *= a[b][h]
            u = [v[b][h][j] - sum(S[i][j] * k[b][hk][i] for i in range(dk)) for j in range(dv)]
            for i in range(dk):
                for j in range(dv):
                    S[i][j] += beta[b][h] * k[b][hk][i] * u[j]
            for j in range(dv):
                out[b][h][j] = scale * sum(S[i][j] * q[b][hk][i] for i in range(dk))
    return np.array(out), np.array(st)


def test_matches_plain_python_loops():
    rng = np.random.default_rng(1)
    state, q, k, v, a, beta = rand_case(rng, 3, 2, 4, 8, 6, slots=5)
    slot = [4, -1, 1]
    ref_out, ref_state = loops(state.copy(), slot, q.tolist(), k.tolist(), v.tolist(), a.tolist(), beta.tolist(), 0.3)
    got_state = state.copy()
    out = la.decode_step(got_state, slot, q, k, v, a, beta, scale=0.3)
    np.testing.assert_allclose(out, ref_out, atol=1e-13)
    np.testing.assert_allclose(got_state, ref_state, atol=1e-13)
    assert (got_state[[0, 2, 3]] == state[[0, 2, 3]]).all()            # untouched slots


def test_beta_zero_is_pure_decay():
    rng = np.random.default_rng(2)
    state, q, k, v, a, beta = rand_case(rng, 2, 2, 2, 16, 8)
    beta[:] = 0.0
    s0 = state.copy()
    out = la.decode_step(state, [0, 1], q, k, v, a, beta)
    for b in range(2):
        for h in range(2):
            np.testing.assert_allclose(state[b, h], a[b, h] * s0[b, h], atol=1e-15)
            np.testing.assert_allclose(out[b, h], a[b, h] * s0[b, h].T @ q[b, h] / 4.0, atol=1e-13)


def test_empty_state_stores_the_outer_product():
    rng = np.random.default_rng(3)
    state, q, k, v, a, beta = rand_case(rng, 1, 1, 2, 16, 8)
    state[:] = 0.0
    out = la.decode_step(state, [0], q, k, v, a, beta, scale=1.0)
    for h in range(2):
        np.testing.assert_allclose(state[0, h], beta[0, h] * np.outer(k[0, 0], v[0, h]), atol=1e-15)
        np.testing.assert_allclose(out[0, h], beta[0, h] * (k[0, 0] @ q[0, 0]) * v[0, h], atol=1e-13)


def test_delta_rule_retrieval_with_unit_key_and_full_write():
    """a = beta = 1, |k| = 1: the new state returns v for key k and acts as before on k's complement."""
    rng = np.random.default_rng(4)
    state, q, k, v, a, beta = rand_case(rng, 2, 1, 1, 32, 16)
    a[:] = 1.0
    beta[:] = 1.0
    s0 = state.copy()
    la.decode_step(state, [0, 1], q, k, v, a, beta)
    for b in range(2):
        np.testing.assert_allclose(state[b, 0].T @ k[b, 0], v[b, 0], atol=1e-12)
        w = rng.standard_normal(32)
        w -= (w @ k[b, 0]) * k[b, 0]                                   # orthogonal to k
        np.testing.assert_allclose(state[b, 0].T @ w, s0[b, 0].T @ w, atol=1e-12)


def test_value_heads_share_the_key_head_in_contiguous_groups():
    rng = np.random.default_rng(5)
    state, q, k, v, a, beta = rand_case(rng, 1, 2, 4, 8, 4)
    state[:] = 0.0
    beta[:] = 1.0
    la.decode_step(state, [0], q, k, v, a, beta)
    for h in range(4):
        np.testing.assert_allclose(state[0, h], np.outer(k[0, h // 2], v[0, h]), atol=1e-15)
