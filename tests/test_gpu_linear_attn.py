"""GPU parity of the recurrent-state decode step against its fp64 oracle, through the C ABI.
State: fp32 on the GPU, compared to the fp64 oracle within 2e-5 * (1 + |ref|) (a dk-term fp32 dot
product and two fused multiply-adds per element); output: bf16, within 2^-8 |ref| + 2e-3."""
import numpy as np
import pytest
import torch

import oracle
from oracle import linear_attn as la
from paper_2609_14237_b200 import binding as B

pytestmark = pytest.mark.gpu


def bits_to_bf16(x):
    return torch.from_numpy(oracle.f32_to_bf16_bits(x.astype(np.float32)).view(np.int16)).view(torch.bfloat16)


def run_case(seed, Bn, Hk, Hv, dk, dv, slots, steps=3, inactive=()):
    B.build()
    rng = np.random.default_rng(seed)
    state = rng.standard_normal((slots, Hv, dk, dv)).astype(np.float32)
    slot = rng.permutation(slots)[:Bn].astype(np.int32)
    for i in inactive:
        slot[i] = -1
    d_state = torch.from_numpy(state.copy()).cuda()
    ref_state = state.astype(np.float64)
    d_slot = torch.from_numpy(slot).cuda()
    for _ in range(steps):
        q = rng.standard_normal((Bn, Hk, dk))
        k = rng.standard_normal((Bn, Hk, dk))
        k /= np.linalg.norm(k, axis=-1, keepdims=True)
        v = rng.standard_normal((Bn, Hv, dv))
        a = rng.uniform(0.8, 1.0, (Bn, Hv)).astype(np.float32)
        beta = rng.uniform(0.0, 1.0, (Bn, Hv)).astype(np.float32)
        tq, tk, tv = bits_to_bf16(q), bits_to_bf16(k), bits_to_bf16(v)
        f = lambda t: oracle.bf16_bits_to_f64(t.view(torch.int16).numpy().view(np.uint16))   # noqa: E731
        out = torch.full((Bn, Hv, dv), float("nan"), dtype=torch.bfloat16, device="cuda")
        dq, dk_, dv_, da, db = tq.cuda(), tk.cuda(), tv.cuda(), torch.from_numpy(a).cuda(), torch.from_numpy(beta).cuda()
        B.opw_linear_attn_decode_step(batch=Bn, num_k_heads=Hk, num_v_heads=Hv, dk=dk, dv=dv, state=d_state.data_ptr(),
                                      num_slots=slots, slot=d_slot.data_ptr(), q=dq.data_ptr(), k=dk_.data_ptr(),
                                      v=dv_.data_ptr(), a=da.data_ptr(), beta=db.data_ptr(), out=out.data_ptr(),
                                      stream=torch.cuda.current_stream().cuda_stream)
        torch.cuda.synchronize()
        ref_out = la.decode_step(ref_state, slot, f(tq), f(tk), f(tv), a.astype(np.float64), beta.astype(np.float64))
        got_state = d_state.cpu().numpy().astype(np.float64)
        assert (np.abs(got_state - ref_state) <= 2e-5 * (1 + np.abs(ref_state))).all()
        got = oracle.bf16_bits_to_f64(out.cpu().view(torch.int16).numpy().view(np.uint16))
        assert np.isfinite(got).all()
        assert (np.abs(got - ref_out) <= 2.0 ** -8 * np.abs(ref_out) + 2e-3).all(), np.abs(got - ref_out).max()
        for i in inactive:
            assert (got[i] == 0).all()
        ref_state = got_state.copy()            # continue from the GPU's fp32 state: errors must not compound in the check
    untouched = sorted(set(range(slots)) - set(int(s) for s in slot if s >= 0))
    assert (d_state.cpu().numpy()[untouched] == state[untouched]).all()


@pytest.mark.parametrize("Hk,Hv,dk,dv", [(2, 4, 128, 128), (1, 1, 64, 64), (2, 2, 128, 256), (4, 8, 64, 128)])
def test_matches_the_oracle_over_several_steps(Hk, Hv, dk, dv):
    run_case(7 + dk + dv, 5, Hk, Hv, dk, dv, slots=9, inactive=(3,))


def test_qwen3_next_like_layer_batch_64():
    run_case(99, 64, 16, 32, 128, 128, slots=70, steps=2)


def test_argument_checks():
    B.build()
    L = B.lib()
    x = torch.zeros(1 << 14, dtype=torch.float32, device="cuda").data_ptr()
    args = lambda Hk, Hv, dk, dv, b=1: (b, Hk, Hv, dk, dv, x, 1, x, x, x, x, x, x, 0.0, x, None)   # noqa: E731
    assert L.opw_linear_attn_decode_step(*args(1, 1, 96, 64)) == B.OPW_ERR_UNSUPPORTED
    assert L.opw_linear_attn_decode_step(*args(2, 3, 64, 64)) == B.OPW_ERR_INVALID_ARG
    assert L.opw_linear_attn_decode_step(*args(1, 1, 64, 64, b=0)) == B.OPW_OK
    assert B.opw_linear_attn_state_bytes(32, 128, 128, 10) == 10 * 32 * 128 * 128 * 4
