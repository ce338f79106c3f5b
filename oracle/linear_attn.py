"""CPU oracle of the recurrent-state ("linear attention") decode step -- TEST INFRASTRUCTURE.

Only the tests and the benchmark's CPU-baseline leg import this module; it shares nothing with
the CUDA path.  The paper names the operator class (Section 3.4: layers that keep a "compact
recurrent state") but prints no definition, so parity against the paper is UNPINNED: the
recurrence below is a declared reading, the gated delta rule as published for gated delta
networks, written out step by step in fp64:

    S1 = a * S                      decay
    u  = v - S1^T k                 what the state mispredicts for key k
    S' = S1 + beta * k u^T          rank-one correction
    o  = scale * S'^T q             read-out with the updated state

What pins it instead (tests/test_linear_oracle.py): plain-Python loops on tiny inputs, and the
closed forms the recurrence has -- beta = 0 is pure decay, an empty state stores beta * k v^T,
with a = beta = 1 and a unit key the updated state returns v exactly for that key (the delta
rule's defining retrieval property) and leaves directions orthogonal to k untouched.
"""
from __future__ import annotations

import numpy as np


def bf16_to_f64(u16: np.ndarray) -> np.ndarray:
    return (u16.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def decode_step(state: np.ndarray, slot, q, k, v, a, beta, scale=None):
    """state: float64 [slots, Hv, dk, dv], updated in place.  q, k: [B, Hk, dk]; v: [B, Hv, dv];
    a, beta: [B, Hv] (all float64).  Returns out [B, Hv, dv] float64."""
    B, Hk, dk = q.shape
    Hv, dv = v.shape[1], v.shape[2]
    rep = Hv // Hk
    if scale is None:
        scale = 1.0 / np.sqrt(np.float64(dk))
    out = np.zeros((B, Hv, dv), dtype=np.float64)
    for b in range(B):
        s = int(slot[b])
        if s < 0 or s >= state.shape[0]:
            continue
        for h in range(Hv):
            hk = h // rep
            S1 = a[b, h] * state[s, h]                         # [dk, dv]
            u = v[b, h] - S1.T @ k[b, hk]                      # [dv]
            S2 = S1 + beta[b, h] * np.outer(k[b, hk], u)
            state[s, h] = S2
            out[b, h] = scale * (S2.T @ q[b, hk])
    return out
