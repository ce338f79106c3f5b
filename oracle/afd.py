"""CPU oracle of the complete attention module (the AFD partition) -- TEST INFRASTRUCTURE.

Only tests and the benchmark's CPU leg import this; it shares nothing with the CUDA path.
The paper says what the module contains (Section 4: AFD "separates complete attention modules
from FFN or MoE operators", i.e. the projections around core attention) and prints no formulas;
the module below is the textbook one, step by step in fp64:

    qkv = x W_qkv^T ; rotary encoding of q and k heads ; append k, v ; softmax attention ; y = out W_o^T

The rotary convention (rotate-half: the pair (x_i, x_{i+D/2}) turns by position * theta^(-2i/D))
is a declared reading, so parity against the paper is UNPINNED for it; it is pinned to its own
mathematics instead (tests/test_afd_oracle.py): position 0 is the identity, norms are preserved,
<rope(q, m), rope(k, n)> depends on m - n only, and a plain-Python restatement.
The only roundings are at the module's declared bf16 interfaces: q, k_new and v_new as they are
handed to core attention and stored in the cache (the activation interface of Appendix B.3:
tensors of a stated shape and byte size cross between operators), and the attention output handed
to the output projection.  Everything between two interfaces is fp64: the projection is not
rounded before the rotation, and y is returned unrounded.
"""
from __future__ import annotations

import numpy as np

import oracle


def round_bf16(x: np.ndarray) -> np.ndarray:
    """fp64 -> nearest-even bf16 -> fp64."""
    return oracle.bf16_bits_to_f64(oracle.f32_to_bf16_bits(x.astype(np.float32)))


def rope(x: np.ndarray, positions, theta: float) -> np.ndarray:
    """x: [B, H, D] float64; rotate-half rotary encoding at positions[b]."""
    B, H, D = x.shape
    half = D // 2
    out = np.empty_like(x)
    for b in range(B):
        for i in range(half):
            ang = float(positions[b]) * theta ** (-2.0 * i / D)
            c, s = np.cos(ang), np.sin(ang)
            out[b, :, i] = x[b, :, i] * c - x[b, :, i + half] * s
            out[b, :, i + half] = x[b, :, i + half] * c + x[b, :, i] * s
    return out


def project_qkv(x, w_qkv, positions, Hq, Hkv, D, theta):
    """Returns bf16-rounded (q [B,Hq,D], k [B,Hkv,D], v [B,Hkv,D]) as float64 arrays."""
    B = x.shape[0]
    qkv = x @ w_qkv.T                                          # fp64, not rounded: no interface here
    q = qkv[:, :Hq * D].reshape(B, Hq, D)
    k = qkv[:, Hq * D:(Hq + Hkv) * D].reshape(B, Hkv, D)
    v = qkv[:, (Hq + Hkv) * D:].reshape(B, Hkv, D)
    pos = np.maximum(np.asarray(positions), 0)
    return round_bf16(rope(q, pos, theta)), round_bf16(rope(k, pos, theta)), round_bf16(v)


def module_step(pool, x, w_qkv, w_o, positions, page_table, Hq, Hkv, D, theta, window=0, P=16):
    """One decode step on `pool` (uint16, updated in place).  x: [B, hidden], weights fp64.
    Returns (y [B, hidden] float64, q, k, v as float64 bf16-valued arrays)."""
    q, k, v = project_qkv(x, w_qkv, positions, Hq, Hkv, D, theta)
    to_bits = lambda a: oracle.f32_to_bf16_bits(a.astype(np.float32))      # noqa: E731  (exact: values are bf16)
    pos = np.asarray(positions, np.int32)
    assert oracle.kv_append(pool, Hkv, D, P, to_bits(k), to_bits(v), pos, page_table) == 0
    lens = np.where(pos >= 0, pos + 1, 0).astype(np.int32)
    out, _, rc = oracle.decode_attention(pool, Hq, Hkv, D, P, to_bits(q), lens, page_table, window=window)
    assert rc == 0
    out = round_bf16(out).reshape(x.shape[0], Hq * D)
    return out @ w_o.T, q, k, v
