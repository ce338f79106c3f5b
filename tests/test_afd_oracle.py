"""Pins of the attention-module oracle's rotary encoding and projections (no GPU)."""
import math

import numpy as np

from oracle import afd


def test_rope_position_zero_is_the_identity_and_norms_are_preserved():
    rng = np.random.default_rng(1)
    x = rng.standard_normal((3, 4, 64))
    assert (afd.rope(x, [0, 0, 0], 10000.0) == x).all()
    y = afd.rope(x, [5, 1234, 65000], 10000.0)
    np.testing.assert_allclose(np.linalg.norm(y, axis=-1), np.linalg.norm(x, axis=-1), rtol=1e-12)


def test_rope_scores_depend_on_the_position_difference_only():
    rng = np.random.default_rng(2)
    q = rng.standard_normal((1, 1, 128))
    k = rng.standard_normal((1, 1, 128))
    def score(m, n):
        return float(afd.rope(q, [m], 1e4)[0, 0] @ afd.rope(k, [n], 1e4)[0, 0])
    assert abs(score(100, 90) - score(5010, 5000)) < 1e-9
    assert abs(score(7, 7) - float(q[0, 0] @ k[0, 0])) < 1e-12
    assert abs(score(100, 90) - score(100, 91)) > 1e-6


def test_rope_matches_a_plain_python_restatement():
    rng = np.random.default_rng(3)
    D, pos, theta = 8, 37, 100.0
    x = rng.standard_normal((1, 1, D))
    y = afd.rope(x, [pos], theta)[0, 0]
    for i in range(D // 2):
        ang = pos * theta ** (-2 * i / D)
        a, b = x[0, 0, i], x[0, 0, i + D // 2]
        assert abs(y[i] - (a * math.cos(ang) - b * math.sin(ang))) < 1e-14
        assert abs(y[i + D // 2] - (b * math.cos(ang) + a * math.sin(ang))) < 1e-14


def test_projection_layout_rows_are_q_heads_then_k_then_v():
    Hq, Hkv, D, hidden = 4, 2, 8, 16
    w = np.zeros(((Hq + 2 * Hkv) * D, hidden))
    w[0, 0] = 1.0                       # q head 0, dim 0 reads x[0]
    w[Hq * D + D + 3, 1] = 2.0          # k head 1, dim 3 reads 2*x[1]
    w[(Hq + Hkv) * D + 5, 2] = -1.0     # v head 0, dim 5 reads -x[2]
    x = np.zeros((1, hidden)); x[0, :3] = [1.0, 0.5, 4.0]
    q, k, v = afd.project_qkv(x, w, [0], Hq, Hkv, D, 1e4)
    assert q[0, 0, 0] == 1.0 and k[0, 1, 3] == 1.0 and v[0, 0, 5] == -4.0
    assert np.count_nonzero(q) == 1 and np.count_nonzero(k) == 1 and np.count_nonzero(v) == 1
