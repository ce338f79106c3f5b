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


@pytest.mark.parametrize("flags", [0, B.OPW_PLAN_GRAPH | B.OPW_PLAN_ADVANCE])
def test_mixed_plan_runs_a_hybrid_stack_in_one_submission(flags):
    """linear, full attention (fused append), linear -- two decode steps, one native call each."""
    import sys, os
    sys.path.insert(0, os.path.dirname(__file__))
    from helpers import P
    from paper_2609_14237_b200 import synth

    B.build()
    rng = np.random.default_rng(5)
    Bn, Hk, Hv, dk, dv = 4, 2, 4, 128, 128
    wl = synth.Workload("mix", Bn, 16, 2, 128, [0], "uniform_1024_4096", 81)
    inp = synth.make_inputs(wl, device="cpu", growth=2, steps=2, lengths=np.array([40, 700, 1500, 16], np.int32))
    pool = inp.pools[0].cuda()
    ref_pool = oracle.as_u16(inp.pools[0]).copy()
    st = B.Stage(pools=[pool], layer_window=[0], num_q_heads=16, num_kv_heads=2, head_dim=128, max_batch=Bn,
                 max_pages_per_seq=inp.max_pages_per_seq)
    states = [rng.standard_normal((Bn, Hv, dk, dv)).astype(np.float32) for _ in range(2)]
    d_states = [torch.from_numpy(x.copy()).cuda() for x in states]
    ref_states = [x.astype(np.float64) for x in states]
    slot = torch.arange(Bn, dtype=torch.int32, device="cuda")
    # static buffers
    lq = [torch.empty(Bn, Hk, dk, dtype=torch.bfloat16, device="cuda") for _ in range(2)]
    lk = [torch.empty_like(t) for t in lq]
    lv = [torch.empty(Bn, Hv, dv, dtype=torch.bfloat16, device="cuda") for _ in range(2)]
    la_ = [torch.empty(Bn, Hv, dtype=torch.float32, device="cuda") for _ in range(2)]
    lb = [torch.empty_like(t) for t in la_]
    lo = [torch.empty(Bn, Hv, dv, dtype=torch.bfloat16, device="cuda") for _ in range(2)]
    aq = torch.empty(Bn, 16, 128, dtype=torch.bfloat16, device="cuda")
    ak = torch.empty(Bn, 2, 128, dtype=torch.bfloat16, device="cuda")
    av = torch.empty_like(ak)
    ao = torch.empty_like(aq)
    pos = torch.from_numpy(inp.positions(0)).cuda()
    tab = inp.page_tables[0].cuda()

    def lin(i):
        return dict(kind="linear", batch=Bn, num_k_heads=Hk, num_v_heads=Hv, dk=dk, dv=dv, state=d_states[i].data_ptr(),
                    num_slots=Bn, slot=slot.data_ptr(), q=lq[i].data_ptr(), k=lk[i].data_ptr(), v=lv[i].data_ptr(),
                    a=la_[i].data_ptr(), beta=lb[i].data_ptr(), out=lo[i].data_ptr())

    ops = [lin(0), dict(kind="attention", layer=0, batch=Bn, q=aq.data_ptr(), k_new=ak.data_ptr(), v_new=av.data_ptr(),
                        positions=pos.data_ptr(), page_table=tab.data_ptr(), out=ao.data_ptr()), lin(1)]
    plan = B.opw_attn_plan_create_mixed(st.handle, ops, flags)
    f = lambda t: oracle.bf16_bits_to_f64(t.cpu().view(torch.int16).numpy().view(np.uint16))   # noqa: E731
    for step in range(2):
        host = []
        for i in range(2):
            q = rng.standard_normal((Bn, Hk, dk)); k = rng.standard_normal((Bn, Hk, dk))
            k /= np.linalg.norm(k, axis=-1, keepdims=True)
            v = rng.standard_normal((Bn, Hv, dv))
            a = rng.uniform(0.8, 1.0, (Bn, Hv)).astype(np.float32); beta = rng.uniform(0, 1, (Bn, Hv)).astype(np.float32)
            lq[i].copy_(bits_to_bf16(q)); lk[i].copy_(bits_to_bf16(k)); lv[i].copy_(bits_to_bf16(v))
            la_[i].copy_(torch.from_numpy(a)); lb[i].copy_(torch.from_numpy(beta))
            host.append((a, beta))
        aq.copy_(inp.q[step, 0]); ak.copy_(inp.k_new[step, 0]); av.copy_(inp.v_new[step, 0])
        if not flags & B.OPW_PLAN_ADVANCE:
            pos.copy_(torch.from_numpy(inp.positions(step)))
        B.opw_attn_plan_submit(plan, torch.cuda.current_stream().cuda_stream)
        assert st.poll_error() == B.OPW_OK
        for i in range(2):
            a, beta = host[i]
            ref = la.decode_step(ref_states[i], np.arange(Bn), f(lq[i]), f(lk[i]), f(lv[i]), a.astype(np.float64),
                                 beta.astype(np.float64))
            got = f(lo[i])
            assert (np.abs(got - ref) <= 2.0 ** -8 * np.abs(ref) + 2e-3).all()
            gs = d_states[i].cpu().numpy().astype(np.float64)
            assert (np.abs(gs - ref_states[i]) <= 2e-5 * (1 + np.abs(ref_states[i]))).all()
            ref_states[i] = gs
        assert oracle.kv_append(ref_pool, 2, 128, P, inp.k_new[step, 0], inp.v_new[step, 0], inp.positions(step),
                                inp.page_tables[0]) == 0
        assert (pool.cpu().view(torch.int16).numpy().view(np.uint16) == ref_pool).all()
        ref, _, _ = oracle.decode_attention(ref_pool, 16, 2, 128, P, inp.q[step, 0], inp.kv_lens(step), inp.page_tables[0])
        assert np.abs(f(ao) - ref).max() <= 1e-2
    B.opw_attn_plan_destroy(plan)
    st.close()


def test_argument_checks():
    B.build()
    L = B.lib()
    x = torch.zeros(1 << 14, dtype=torch.float32, device="cuda").data_ptr()
    args = lambda Hk, Hv, dk, dv, b=1: (b, Hk, Hv, dk, dv, x, 1, x, x, x, x, x, x, 0.0, x, None)   # noqa: E731
    assert L.opw_linear_attn_decode_step(*args(1, 1, 96, 64)) == B.OPW_ERR_UNSUPPORTED
    assert L.opw_linear_attn_decode_step(*args(2, 3, 64, 64)) == B.OPW_ERR_INVALID_ARG
    assert L.opw_linear_attn_decode_step(*args(1, 1, 64, 64, b=0)) == B.OPW_OK
    assert B.opw_linear_attn_state_bytes(32, 128, 128, 10) == 10 * 32 * 128 * 128 * 4
