"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle on the
same seeded inputs.  Append and page indexing must be bit-exact; attention output must
satisfy max |err| <= 1e-2 and mean |err| <= 1e-3 (bf16 in, fp32 accumulate, bf16 out),
plus the tighter checks below (error relative to the output's rms, log-sum-exp)."""
import time

import numpy as np
import pytest
import torch

import oracle
from helpers import MAX_ABS, P, bits, check_close, make_case, out_to_f64, rand_bits
from paper_2609_14237_b200 import binding as B
from paper_2609_14237_b200 import synth

pytestmark = pytest.mark.gpu

@pytest.fixture(scope="module", autouse=True)
def built():
    B.build()
    assert torch.cuda.is_available()


def dev(a, dtype=None):
    t = torch.from_numpy(np.ascontiguousarray(a))
    if dtype is torch.bfloat16:
        t = t.view(torch.int16).view(torch.bfloat16)
    return t.cuda()


def gpu_attention(pool_np, tab, q_bits, lens, Hq, Hkv, D, window=0, scale=0.0, want_lse=True, **tune):
    pool = dev(pool_np, torch.bfloat16)
    st = B.Stage(pools=[pool], layer_window=[window], num_q_heads=Hq, num_kv_heads=Hkv, head_dim=D,
                 max_batch=len(lens), max_pages_per_seq=tab.shape[1], softmax_scale=scale, **tune)
    q = dev(q_bits, torch.bfloat16)
    kv = dev(np.asarray(lens, np.int32))
    tb = dev(tab.astype(np.int32))
    out = torch.full((len(lens), Hq, D), float("nan"), dtype=torch.bfloat16, device="cuda")
    lse = torch.full((len(lens), Hq), float("nan"), dtype=torch.float32, device="cuda") if want_lse else None
    st.decode_attention(0, q, kv, tb, out, lse)
    rc = st.poll_error()
    launches = st.launch_count()
    st.close()
    return out, (lse.cpu().numpy().astype(np.float64) if want_lse else None), rc, launches


# ------------------------------------------------------------------ append ---

def test_append_is_bit_exact_over_the_whole_pool():
    rng = np.random.default_rng(31)
    Hkv, D = 2, 64
    lens = [0, 15, 16, 255, 100, 17, 64]
    pool_np, tab, _, _, _ = make_case(rng, [n + 1 for n in lens], 8, Hkv, D)
    k_new, v_new = rand_bits(rng, (len(lens), Hkv, D)), rand_bits(rng, (len(lens), Hkv, D))
    pos = np.array(lens, np.int32)
    pos[5] = -1                                                        # an inactive slot
    pool = dev(pool_np, torch.bfloat16)
    st = B.Stage(pools=[pool], layer_window=[0], num_q_heads=8, num_kv_heads=Hkv, head_dim=D,
                 max_batch=len(lens), max_pages_per_seq=tab.shape[1])
    st.kv_append(0, dev(k_new, torch.bfloat16), dev(v_new, torch.bfloat16), dev(pos), dev(tab))
    assert st.poll_error() == B.OPW_OK and st.launch_count() == 1
    ref = pool_np.copy()
    assert oracle.kv_append(ref, Hkv, D, P, k_new, v_new, pos, tab) == 0
    got = pool.cpu().view(torch.int16).numpy().view(np.uint16)
    assert (got == ref).all()
    assert (got != pool_np).sum() > 0
    st.close()


def test_append_reports_bad_pages_without_writing():
    rng = np.random.default_rng(32)
    Hkv, D = 8, 128
    pool_np, tab, _, _, _ = make_case(rng, [20, 20, 20], 32, Hkv, D)
    bad = tab.copy()
    bad[0, 1] = -1
    bad[1, 1] = 1 << 20
    k_new, v_new = rand_bits(rng, (3, Hkv, D)), rand_bits(rng, (3, Hkv, D))
    pool = dev(pool_np, torch.bfloat16)
    st = B.Stage(pools=[pool], layer_window=[0], num_q_heads=32, num_kv_heads=Hkv, head_dim=D, max_batch=3,
                 max_pages_per_seq=tab.shape[1])
    st.kv_append(0, dev(k_new, torch.bfloat16), dev(v_new, torch.bfloat16), dev(np.array([19, 19, 19], np.int32)), dev(bad))
    assert st.poll_error() == B.OPW_ERR_BAD_PAGE
    assert st.poll_error() == B.OPW_OK                                   # cleared by the poll
    ref = pool_np.copy()
    oracle.kv_append(ref, Hkv, D, P, k_new, v_new, np.array([-1, -1, 19], np.int32), tab)
    assert (pool.cpu().view(torch.int16).numpy().view(np.uint16) == ref).all()
    st.close()


# --------------------------------------------------------------- attention ---

@pytest.mark.parametrize("Hq,Hkv,D", [(8, 2, 64), (32, 8, 128), (8, 8, 64), (64, 8, 128), (16, 1, 128), (24, 2, 64), (5, 1, 64),
                                      (16, 2, 256), (4, 2, 256)])
@pytest.mark.parametrize("window", [0, 40])
def test_attention_small_shapes_match_the_oracle(Hq, Hkv, D, window):
    rng = np.random.default_rng(40 + Hq + D)
    lens = [1, 2, 15, 16, 17, 33, 100, 256, 777]
    pool, tab, q, _, _ = make_case(rng, lens, Hq, Hkv, D)
    ref, ref_lse, rc = oracle.decode_attention(pool, Hq, Hkv, D, P, q, lens, tab, window=window)
    assert rc == 0
    out, lse, rc, launches = gpu_attention(pool, tab, q, lens, Hq, Hkv, D, window=window)
    assert rc == B.OPW_OK and launches == 2
    check_close(out_to_f64(out), ref, lse, ref_lse)


def test_config1_tiny_step_append_then_attention():
    wl = synth.WORKLOADS["c1_tiny"]
    inp = synth.make_inputs(wl, device="cpu", growth=3, steps=3)
    pool_ref = oracle.as_u16(inp.pools[0]).copy()
    pool = inp.pools[0].cuda()
    st = B.Stage(pools=[pool], layer_window=[0], num_q_heads=wl.num_q_heads, num_kv_heads=wl.num_kv_heads,
                 head_dim=wl.head_dim, max_batch=wl.batch, max_pages_per_seq=inp.max_pages_per_seq)
    tab = inp.page_tables[0]
    for step in range(3):
        pos, n = inp.positions(step), inp.kv_lens(step)
        q, k, v = inp.q[step, 0], inp.k_new[step, 0], inp.v_new[step, 0]
        out = torch.empty(wl.batch, wl.num_q_heads, wl.head_dim, dtype=torch.bfloat16, device="cuda")
        lse = torch.empty(wl.batch, wl.num_q_heads, dtype=torch.float32, device="cuda")
        st.kv_append(0, k.cuda(), v.cuda(), dev(pos), tab.cuda())
        st.decode_attention(0, q.cuda(), dev(n), tab.cuda(), out, lse)
        assert st.poll_error() == B.OPW_OK
        assert oracle.kv_append(pool_ref, wl.num_kv_heads, wl.head_dim, P, k, v, pos, tab) == 0
        assert (pool.cpu().view(torch.int16).numpy().view(np.uint16) == pool_ref).all()     # bit-exact cache
        ref, ref_lse, _ = oracle.decode_attention(pool_ref, wl.num_q_heads, wl.num_kv_heads, wl.head_dim, P, q, n, tab)
        check_close(out_to_f64(out), ref, lse.cpu().numpy().astype(np.float64), ref_lse)
    st.close()


@pytest.mark.parametrize("Hq,Hkv,D", [(8, 2, 64), (32, 8, 128), (24, 2, 64), (16, 2, 256)])
def test_fused_step_appends_bit_exactly_and_attends_over_the_new_key(Hq, Hkv, D):
    """opw_decode_step == opw_kv_append + opw_decode_attention: same pool bytes, same output."""
    wl = synth.Workload("f", 9, Hq, Hkv, D, [0, 40], "tiny", 79)
    lens = np.array([0, 15, 16, 255, 100, 17, 64, 2000, 31], np.int32)
    inp = synth.make_inputs(wl, device="cpu", growth=3, steps=3, lengths=lens)
    pools = [p.cuda() for p in inp.pools]
    refs = [oracle.as_u16(p).copy() for p in inp.pools]
    st = B.Stage(pools=pools, layer_window=wl.layer_window, num_q_heads=Hq, num_kv_heads=Hkv, head_dim=D,
                 max_batch=9, max_pages_per_seq=inp.max_pages_per_seq)
    for step in range(3):
        pos = inp.positions(step).copy()
        pos[5] = -1                                                   # an inactive slot every step
        n = np.where(pos >= 0, pos + 1, 0).astype(np.int32)
        for layer in range(2):
            q, k, v = inp.q[step, layer], inp.k_new[step, layer], inp.v_new[step, layer]
            out = torch.full((9, Hq, D), float("nan"), dtype=torch.bfloat16, device="cuda")
            lse = torch.full((9, Hq), float("nan"), dtype=torch.float32, device="cuda")
            before = st.launch_count()
            st.decode_step(layer, q.cuda(), k.cuda(), v.cuda(), dev(pos), inp.page_tables[layer].cuda(), out, lse)
            assert st.poll_error() == B.OPW_OK and st.launch_count() - before == 2
            assert oracle.kv_append(refs[layer], Hkv, D, P, k, v, pos, inp.page_tables[layer]) == 0
            assert (pools[layer].cpu().view(torch.int16).numpy().view(np.uint16) == refs[layer]).all()
            ref, ref_lse, _ = oracle.decode_attention(refs[layer], Hq, Hkv, D, P, q, n, inp.page_tables[layer],
                                                      window=wl.layer_window[layer])
            check_close(out_to_f64(out), ref, lse.cpu().numpy().astype(np.float64), ref_lse)
    st.close()


def test_fused_step_with_a_position_beyond_the_table_appends_nothing_for_that_row():
    rng = np.random.default_rng(64)
    Hq, Hkv, D = 8, 2, 64
    pool_np, tab, q, _, _ = make_case(rng, [33, 48], Hq, Hkv, D)          # tables of 3 pages: 48 positions
    k_new, v_new = rand_bits(rng, (2, Hkv, D)), rand_bits(rng, (2, Hkv, D))
    pool = dev(pool_np, torch.bfloat16)
    st = B.Stage(pools=[pool], layer_window=[0], num_q_heads=Hq, num_kv_heads=Hkv, head_dim=D, max_batch=2,
                 max_pages_per_seq=tab.shape[1])
    out = torch.empty(2, Hq, D, dtype=torch.bfloat16, device="cuda")
    pos = np.array([32, 48], np.int32)                                    # row 1 points past its table
    st.decode_step(0, dev(q, torch.bfloat16), dev(k_new, torch.bfloat16), dev(v_new, torch.bfloat16), dev(pos),
                   dev(tab), out)
    assert st.poll_error() == B.OPW_ERR_BAD_PAGE
    ref = pool_np.copy()
    oracle.kv_append(ref, Hkv, D, P, k_new, v_new, np.array([32, -1], np.int32), tab)
    assert (pool.cpu().view(torch.int16).numpy().view(np.uint16) == ref).all()
    st.close()


@pytest.mark.parametrize("fused", [True, False])
def test_programmatic_dependent_launch_keeps_back_to_back_steps_ordered(fused):
    """By default every kernel may start while its predecessor finishes; eight steps enqueued
    without a host synchronisation in between must still leave the exact pool and the right outputs."""
    wl = synth.Workload("pdl", 8, 32, 8, 128, [0, 200], "uniform_1024_4096", 80)
    inp = synth.make_inputs(wl, device="cpu", growth=4, steps=4)
    pools = [p.cuda() for p in inp.pools]
    refs = [oracle.as_u16(p).copy() for p in inp.pools]
    st = B.Stage(pools=pools, layer_window=wl.layer_window, num_q_heads=32, num_kv_heads=8, head_dim=128,
                 max_batch=8, max_pages_per_seq=inp.max_pages_per_seq)
    tabs = [t.cuda() for t in inp.page_tables]
    dq, dk, dv = inp.q.cuda(), inp.k_new.cuda(), inp.v_new.cuda()
    pos = [dev(inp.positions(s)) for s in range(4)]
    lens = [dev(inp.kv_lens(s)) for s in range(4)]
    outs = torch.empty(4, 2, 8, 32, 128, dtype=torch.bfloat16, device="cuda")
    for step in range(4):
        for layer in range(2):
            if fused:
                st.decode_step(layer, dq[step, layer], dk[step, layer], dv[step, layer], pos[step], tabs[layer], outs[step, layer])
            else:
                st.kv_append(layer, dk[step, layer], dv[step, layer], pos[step], tabs[layer])
                st.decode_attention(layer, dq[step, layer], lens[step], tabs[layer], outs[step, layer])
    assert st.poll_error() == B.OPW_OK
    for step in range(4):
        for layer in range(2):
            assert oracle.kv_append(refs[layer], 8, 128, P, inp.k_new[step, layer], inp.v_new[step, layer],
                                    inp.positions(step), inp.page_tables[layer]) == 0
            ref, _, _ = oracle.decode_attention(refs[layer], 32, 8, 128, P, inp.q[step, layer], inp.kv_lens(step),
                                                inp.page_tables[layer], window=wl.layer_window[layer])
            check_close(out_to_f64(outs[step, layer]), ref)
    for layer in range(2):
        assert (pools[layer].cpu().view(torch.int16).numpy().view(np.uint16) == refs[layer]).all()
    st.close()


@pytest.mark.parametrize("fused", [True, False])
def test_programmatic_dependent_launch_with_an_all_inactive_step_between_two_live_ones(fused):
    """A grid with nothing to do must still pass its dependency wait before it completes, or the kernels
    behind it could overtake the step in front of it: live step, all-inactive step, live step, enqueued
    back to back on one stream (programmatic dependent launch is the default), repeated over two layers; every output and the whole
    pool against the oracle."""
    wl = synth.Workload("pdl0", 8, 32, 8, 128, [0, 200], "uniform_1024_4096", 81)
    inp = synth.make_inputs(wl, device="cpu", growth=3, steps=3)
    pools = [p.cuda() for p in inp.pools]
    refs = [oracle.as_u16(p).copy() for p in inp.pools]
    st = B.Stage(pools=pools, layer_window=wl.layer_window, num_q_heads=32, num_kv_heads=8, head_dim=128,
                 max_batch=8, max_pages_per_seq=inp.max_pages_per_seq)
    tabs = [t.cuda() for t in inp.page_tables]
    dq, dk, dv = inp.q.cuda(), inp.k_new.cuda(), inp.v_new.cuda()
    # step 1 is the empty one: every slot inactive; the live steps are decode steps 0 and 1 of the sequences
    pos_np = [inp.positions(0), np.full(8, -1, np.int32), inp.positions(1)]
    len_np = [np.where(p >= 0, p + 1, 0).astype(np.int32) for p in pos_np]
    pos, lens = [dev(p) for p in pos_np], [dev(n) for n in len_np]
    outs = torch.full((3, 2, 8, 32, 128), float("nan"), dtype=torch.bfloat16, device="cuda")
    lses = torch.full((3, 2, 8, 32), float("nan"), dtype=torch.float32, device="cuda")
    for rep in range(3):                                   # the same three steps enqueued three times over:
        for step in range(3):                              # later repetitions rewrite the same slots with the same rows
            for layer in range(2):
                if fused:
                    st.decode_step(layer, dq[step, layer], dk[step, layer], dv[step, layer], pos[step], tabs[layer],
                                   outs[step, layer], lses[step, layer])
                else:
                    st.kv_append(layer, dk[step, layer], dv[step, layer], pos[step], tabs[layer])
                    st.decode_attention(layer, dq[step, layer], lens[step], tabs[layer], outs[step, layer], lses[step, layer])
    assert st.poll_error() == B.OPW_OK
    for step in range(3):
        for layer in range(2):
            assert oracle.kv_append(refs[layer], 8, 128, P, inp.k_new[step, layer], inp.v_new[step, layer],
                                    pos_np[step], inp.page_tables[layer]) == 0
    for step in range(3):
        for layer in range(2):
            # (the live steps of every repetition saw the pool with both new rows already in place or being
            # rewritten with identical bytes; attention reads only rows below its own length)
            ref, ref_lse, _ = oracle.decode_attention(refs[layer], 32, 8, 128, P, inp.q[step, layer], len_np[step],
                                                      inp.page_tables[layer], window=wl.layer_window[layer])
            check_close(out_to_f64(outs[step, layer]), ref, lses[step, layer].cpu().numpy().astype(np.float64), ref_lse)
    assert (out_to_f64(outs[1]) == 0).all() and np.isneginf(lses[1].cpu().numpy()).all()
    for layer in range(2):
        assert (pools[layer].cpu().view(torch.int16).numpy().view(np.uint16) == refs[layer]).all()
    st.close()


def test_a_smaller_stage_created_later_leaves_an_earlier_larger_stage_working():
    """The kernels' shared-memory limit belongs to the device, not to a stage: creating a stage with a
    small static batch after one with a large static batch must not lower it under the first one."""
    rng = np.random.default_rng(67)
    Hq, Hkv, D = 8, 2, 64
    lens = rng.integers(1, 60, size=4096).astype(np.int32)
    lens[::7] = 0
    pool_np, tab, q, _, _ = make_case(rng, [max(int(n), 1) for n in lens], Hq, Hkv, D)
    pool = dev(pool_np, torch.bfloat16)
    big = B.Stage(pools=[pool], layer_window=[0], num_q_heads=Hq, num_kv_heads=Hkv, head_dim=D, max_batch=4096,
                  max_pages_per_seq=tab.shape[1], tune_warps=12, tune_stages=4)
    small = B.Stage(pools=[pool], layer_window=[0], num_q_heads=Hq, num_kv_heads=Hkv, head_dim=D, max_batch=2,
                    max_pages_per_seq=tab.shape[1], tune_warps=2, tune_stages=2)
    out = torch.full((4096, Hq, D), float("nan"), dtype=torch.bfloat16, device="cuda")
    lse = torch.full((4096, Hq), float("nan"), dtype=torch.float32, device="cuda")
    big.decode_attention(0, dev(q, torch.bfloat16), dev(lens), dev(tab), out, lse)     # raises OpwError if the launch is refused
    assert big.poll_error() == B.OPW_OK
    ref, ref_lse, rc = oracle.decode_attention(pool_np, Hq, Hkv, D, P, q, lens, tab)
    assert rc == 0
    check_close(out_to_f64(out), ref, lse.cpu().numpy().astype(np.float64), ref_lse,
                max_abs=2.0 ** -8 * float(np.abs(ref).max()) + 1e-3)
    out2 = torch.empty(2, Hq, D, dtype=torch.bfloat16, device="cuda")
    small.decode_attention(0, dev(q[:2], torch.bfloat16), dev(lens[:2]), dev(tab[:2]), out2)
    assert small.poll_error() == B.OPW_OK
    check_close(out_to_f64(out2), ref[:2], max_abs=2.0 ** -8 * float(np.abs(ref).max()) + 1e-3)
    small.close()
    big.close()


def test_single_key_returns_v_bit_exactly():
    rng = np.random.default_rng(51)
    Hq, Hkv, D = 8, 2, 64
    pool, tab, q, ks, vs = make_case(rng, [1, 1, 1], Hq, Hkv, D)
    out, lse, rc, _ = gpu_attention(pool, tab, q, [1, 1, 1], Hq, Hkv, D)
    got = out.cpu().view(torch.int16).numpy().view(np.uint16)
    for b in range(3):
        for h in range(Hq):
            assert (got[b, h] == vs[b][0, h // 4]).all()


def test_garbage_in_unwritten_slots_cannot_leak_into_the_result():
    """Slots after the last key (and before the window) may hold NaN/Inf bit patterns."""
    rng = np.random.default_rng(58)
    Hq, Hkv, D = 32, 8, 128
    lens = [1, 17, 100, 250]
    W = 60
    pool, tab, q, ks, vs = make_case(rng, lens, Hq, Hkv, D)
    ref, ref_lse, _ = oracle.decode_attention(pool, Hq, Hkv, D, P, q, lens, tab, window=W)
    poisoned = np.full_like(pool, 0x7FC0)                            # bf16 NaN everywhere
    for b, n in enumerate(lens):
        lo = max(0, n - W)
        k = np.full((n, Hkv, D), 0x7F80, np.uint16)                  # +Inf before the window
        v = np.full((n, Hkv, D), 0x7FC0, np.uint16)
        k[lo:], v[lo:] = ks[b][lo:], vs[b][lo:]
        oracle.scatter_logical(poisoned, Hkv, P, D, tab[b], k, v)
    out, lse, rc, _ = gpu_attention(poisoned, tab, q, lens, Hq, Hkv, D, window=W)
    assert rc == B.OPW_OK
    check_close(out_to_f64(out), ref, lse, ref_lse)


def test_q_zero_probes_every_key_counted_once_long_and_windowed():
    rng = np.random.default_rng(52)
    Hq, Hkv, D = 8, 2, 64
    lens = [1, 16, 17, 4000, 9000, 33000]
    one = bits(np.float32(1.0))
    for window in (0, 1, 17, 4096):
        pool, tab, q, ks, vs = make_case(rng, lens, Hq, Hkv, D)
        q[:] = 0
        marks = [0, 15, 16, 3999, 8999, 20000]
        for b, n in enumerate(lens):
            lo = max(0, n - window) if window else 0
            v = np.zeros((n, Hkv, D), np.uint16)
            v[:, :, 0] = one
            for c, j0 in enumerate(marks):
                if j0 < n:
                    v[j0, :, 1 + c] = one
            v[:lo, :, 10] = one
            oracle.scatter_logical(pool, Hkv, P, D, tab[b], ks[b], v)
        out, lse, rc, _ = gpu_attention(pool, tab, q, lens, Hq, Hkv, D, window=window)
        got = out_to_f64(out)
        for b, n in enumerate(lens):
            lo = max(0, n - window) if window else 0
            n_eff = n - lo
            np.testing.assert_allclose(got[b, :, 0], 1.0, rtol=2 ** -7)
            for c, j0 in enumerate(marks):
                want = 1.0 / n_eff if lo <= j0 < n else 0.0
                np.testing.assert_allclose(got[b, :, 1 + c], want, rtol=2 ** -7, atol=0)
            assert (got[b, :, 10] == 0).all()
            np.testing.assert_allclose(lse[b], np.log(n_eff), atol=1e-4)


def test_page_permutation_is_bitwise_invisible():
    rng = np.random.default_rng(53)
    Hq, Hkv, D = 32, 8, 128
    lens = [100, 2000, 5000, 257]
    pool, tab, q, _, _ = make_case(rng, lens, Hq, Hkv, D)
    out1, lse1, _, _ = gpu_attention(pool, tab, q, lens, Hq, Hkv, D)
    total = pool.size // (Hkv * 2 * P * D)
    perm = rng.permutation(total)
    pe = Hkv * 2 * P * D
    pool2 = np.empty_like(pool)
    pool2.reshape(total, pe)[perm] = pool.reshape(total, pe)
    tab2 = np.where(tab >= 0, perm[np.maximum(tab, 0)], -1).astype(np.int32)
    out2, lse2, _, _ = gpu_attention(pool2, tab2, q, lens, Hq, Hkv, D)
    assert torch.equal(out1.view(torch.int16), out2.view(torch.int16))
    assert (lse1 == lse2).all()


def test_window_poisoned_entries_and_inactive_rows():
    rng = np.random.default_rng(54)
    Hq, Hkv, D = 32, 8, 128
    lens = [18, 650, 1010, 2560]
    W = 400
    pool, tab, q, _, _ = make_case(rng, lens, Hq, Hkv, D)
    ref, ref_lse, _ = oracle.decode_attention(pool, Hq, Hkv, D, P, q, lens, tab, window=W)
    poisoned = tab.copy()
    for b, n in enumerate(lens):
        poisoned[b, :max(0, n - W) // P] = -1
        poisoned[b, (n + P - 1) // P:] = -1
    out, lse, rc, _ = gpu_attention(pool, poisoned, q, lens, Hq, Hkv, D, window=W)
    assert rc == B.OPW_OK
    check_close(out_to_f64(out), ref, lse, ref_lse)
    # inactive rows: zeros and -inf
    lens2 = [18, 0, 1010, -5]
    ref2, ref_lse2, _ = oracle.decode_attention(pool, Hq, Hkv, D, P, q, lens2, tab)
    out2, lse2, rc2, _ = gpu_attention(pool, tab, q, lens2, Hq, Hkv, D)
    assert rc2 == B.OPW_OK
    check_close(out_to_f64(out2), ref2, lse2, ref_lse2)
    assert (out_to_f64(out2)[1] == 0).all() and np.isneginf(lse2[3]).all()


def test_bad_page_ids_are_masked_and_reported_not_dereferenced():
    rng = np.random.default_rng(55)
    Hq, Hkv, D = 8, 2, 64
    lens = [100, 200]
    pool, tab, q, ks, vs = make_case(rng, lens, Hq, Hkv, D)
    bad = tab.copy()
    bad[1, 3] = -1
    bad[1, 7] = 1 << 24
    out, lse, rc, _ = gpu_attention(pool, bad, q, lens, Hq, Hkv, D)
    assert rc == B.OPW_ERR_BAD_PAGE
    # row 0 is unaffected; row 1 equals attention with the two bad pages' keys removed
    ref, _, _ = oracle.decode_attention(pool, Hq, Hkv, D, P, q, lens, tab)
    got = out_to_f64(out)
    assert np.abs(got[0] - ref[0]).max() <= MAX_ABS
    keep = [j for j in range(200) if j // P not in (3, 7)]
    pool2, tab2, _, _, _ = make_case(rng, [len(keep)], Hq, Hkv, D)
    oracle.scatter_logical(pool2, Hkv, P, D, tab2[0], ks[1][keep], vs[1][keep])
    ref1, _, _ = oracle.decode_attention(pool2, Hq, Hkv, D, P, q[1:2], [len(keep)], tab2)
    assert np.abs(got[1] - ref1[0]).max() <= MAX_ABS


@pytest.mark.parametrize("tune", [dict(tune_warps=1, tune_stages=2), dict(tune_warps=4, tune_stages=6),
                                  dict(tune_warps=4, tune_stages=3, tune_ctas_per_sm=2), dict(tune_warps=8, tune_stages=3),
                                  dict(tune_warps=3, tune_stages=8), dict(flags=B.OPW_FLAG_NO_PDL),
                                  dict(tune_warps=5, tune_stages=3, flags=B.OPW_FLAG_NO_PDL)])
def test_result_does_not_depend_on_the_split(tune):
    """The log-sum-exp merge is exact in real arithmetic: any split agrees within rounding."""
    rng = np.random.default_rng(56)
    Hq, Hkv, D = 32, 8, 128
    lens = [5000, 33, 12000, 1]
    pool, tab, q, _, _ = make_case(rng, lens, Hq, Hkv, D)
    ref, ref_lse, _ = oracle.decode_attention(pool, Hq, Hkv, D, P, q, lens, tab)
    out, lse, rc, _ = gpu_attention(pool, tab, q, lens, Hq, Hkv, D, **tune)
    assert rc == B.OPW_OK
    check_close(out_to_f64(out), ref, lse, ref_lse)


def test_custom_scale_and_no_lse_buffer():
    rng = np.random.default_rng(57)
    Hq, Hkv, D = 16, 2, 128
    lens = [300, 45]
    pool, tab, q, _, _ = make_case(rng, lens, Hq, Hkv, D)
    ref, _, _ = oracle.decode_attention(pool, Hq, Hkv, D, P, q, lens, tab, scale=0.25)
    out, _, rc, _ = gpu_attention(pool, tab, q, lens, Hq, Hkv, D, scale=0.25, want_lse=False)
    assert rc == B.OPW_OK
    check_close(out_to_f64(out), ref)


def test_host_buffer_step_matches_the_device_step():
    wl = synth.Workload("h", 6, 32, 8, 128, [0, 64], "uniform_1024_4096", 77)
    inp = synth.make_inputs(wl, device="cpu", growth=2, steps=2, lengths=np.array([5, 200, 1023, 64, 15, 4097], np.int32))
    pools = [p.cuda() for p in inp.pools]
    refs = [oracle.as_u16(p).copy() for p in inp.pools]
    st = B.Stage(pools=pools, layer_window=wl.layer_window, num_q_heads=32, num_kv_heads=8, head_dim=128,
                 max_batch=6, max_pages_per_seq=inp.max_pages_per_seq)
    for step in range(2):
        for layer in range(2):
            if layer == 0:                                # separate host buffers: four copies
                q = inp.q[step, layer].pin_memory()
                k = inp.k_new[step, layer].pin_memory()
                v = inp.v_new[step, layer].pin_memory()
                pos = torch.from_numpy(inp.positions(step)).pin_memory()
            else:                                         # one packed host buffer: a single copy
                _, q, k, v, pos = st.packed_host_buffers(6)
                q.copy_(inp.q[step, layer])
                k.copy_(inp.k_new[step, layer])
                v.copy_(inp.v_new[step, layer])
                pos.copy_(torch.from_numpy(inp.positions(step)))
            tab = inp.page_tables[layer].pin_memory()
            out = torch.empty(6, 32, 128, dtype=torch.bfloat16).pin_memory()
            lse = torch.empty(6, 32, dtype=torch.float32).pin_memory()
            st.decode_step_host(layer, q, k, v, pos, tab if step == 0 else None, out, lse)
            assert st.poll_error() == B.OPW_OK
            assert oracle.kv_append(refs[layer], 8, 128, P, k, v, pos, tab) == 0
            assert (pools[layer].cpu().view(torch.int16).numpy().view(np.uint16) == refs[layer]).all()
            ref, ref_lse, _ = oracle.decode_attention(refs[layer], 32, 8, 128, P, q, inp.kv_lens(step), tab,
                                                      window=wl.layer_window[layer])
            check_close(out_to_f64(out), ref, lse.numpy().astype(np.float64), ref_lse)
    assert st.launch_count() == 2 * 2 * 2
    st.close()


def test_two_stages_with_copy_streams_take_turns_on_one_compute_stream():
    """Two microbatches, a stage handle each (OPW_FLAG_COPY_STREAMS), both enqueuing on one compute stream: copies in
    and out run on the stages' own streams.  Twelve steps without waiting for anything but each stage's previous
    output; pools and every output against the oracle."""
    steps = 12
    wl = synth.Workload("cs", 6, 32, 8, 128, [0, 64], "uniform_1024_4096", 85)
    inp = synth.make_inputs(wl, device="cpu", growth=steps, steps=steps, lengths=np.array([5, 200, 1023, 64, 15, 3000], np.int32))
    pools = [p.cuda() for p in inp.pools]
    refs = [oracle.as_u16(p).copy() for p in inp.pools]
    stages = [B.Stage(pools=pools, layer_window=wl.layer_window, num_q_heads=32, num_kv_heads=8, head_dim=128, max_batch=6,
                      max_pages_per_seq=inp.max_pages_per_seq, flags=B.OPW_FLAG_COPY_STREAMS) for _ in range(2)]
    compute = torch.cuda.Stream()
    packs = [[stages[l].packed_host_buffers(6) for _ in range(2)] for l in range(2)]     # [layer = microbatch][double buffer]
    outs = torch.empty(steps, 2, 6, 32, 128, dtype=torch.bfloat16).pin_memory()
    lses = torch.empty(steps, 2, 6, 32, dtype=torch.float32).pin_memory()
    tabs = [t.pin_memory() for t in inp.page_tables]
    for step in range(steps):
        for layer in range(2):                               # microbatch `layer` owns layer `layer` and stage `layer`
            st = stages[layer]
            st.wait_host_output()
            _, q, k, v, pos = packs[layer][step & 1]
            q.copy_(inp.q[step, layer]); k.copy_(inp.k_new[step, layer]); v.copy_(inp.v_new[step, layer])
            pos.copy_(torch.from_numpy(inp.positions(step)))
            with torch.cuda.stream(compute):
                st.decode_step_host(layer, q, k, v, pos, tabs[layer] if step == 0 else None, outs[step, layer], lses[step, layer])
    for st in stages:
        st.wait_host_output()
    torch.cuda.synchronize()
    assert all(st.poll_error() == B.OPW_OK for st in stages)
    for step in range(steps):
        for layer in range(2):
            assert oracle.kv_append(refs[layer], 8, 128, P, inp.k_new[step, layer], inp.v_new[step, layer],
                                    inp.positions(step), inp.page_tables[layer]) == 0
            ref, ref_lse, _ = oracle.decode_attention(refs[layer], 32, 8, 128, P, inp.q[step, layer], inp.kv_lens(step),
                                                      inp.page_tables[layer], window=wl.layer_window[layer])
            check_close(out_to_f64(outs[step, layer]), ref, lses[step, layer].numpy().astype(np.float64), ref_lse)
    for layer in range(2):
        assert (pools[layer].cpu().view(torch.int16).numpy().view(np.uint16) == refs[layer]).all()
    for st in stages:
        st.close()


def test_host_steps_with_page_table_deltas_equal_steps_with_the_table_resent_in_full():
    """Forty decode steps from host buffers, twice: once re-sending the whole page table every step, once sending it
    in full at the first step only (with the pages of later steps still unmapped) and from then on just the
    (row, logical page, physical page) triple of every sequence that crosses into a new page.  Pools and outputs
    must agree bit for bit, and with the oracle at the end."""
    steps = 40
    wl = synth.Workload("pd", 5, 32, 8, 128, [0, 64], "uniform_1024_4096", 84)
    lens = np.array([5, 200, 1023, 64, 15], np.int32)
    inp = synth.make_inputs(wl, device="cpu", growth=steps, steps=steps, lengths=lens)
    results = []
    for use_delta in (False, True):
        pools = [p.clone().cuda() for p in inp.pools]
        st = B.Stage(pools=pools, layer_window=wl.layer_window, num_q_heads=32, num_kv_heads=8, head_dim=128,
                     max_batch=5, max_pages_per_seq=inp.max_pages_per_seq)
        outs = torch.empty(steps, 2, 5, 32, 128, dtype=torch.bfloat16).pin_memory()
        tri = torch.empty(steps, 2, 5, 3, dtype=torch.int32).pin_memory()
        sent = 0
        for step in range(steps):
            pos_np = inp.positions(step)
            for layer in range(2):
                _, q, k, v, pos = st.packed_host_buffers(5)
                q.copy_(inp.q[step, layer]); k.copy_(inp.k_new[step, layer]); v.copy_(inp.v_new[step, layer])
                pos.copy_(torch.from_numpy(pos_np))
                full = inp.page_tables[layer]
                if not use_delta:
                    tab = full.clone().pin_memory()
                elif step == 0:                                  # the table as a server holds it at admission: nothing
                    tab = full.clone()                            # mapped beyond the page the first token goes to
                    for b in range(5):
                        tab[b, int(pos_np[b]) // P + 1:] = -1
                    tab = tab.pin_memory()
                else:
                    tab = None
                    rows = [b for b in range(5) if int(pos_np[b]) % P == 0]       # this step's token opens a new page
                    for i, b in enumerate(rows):
                        lp = int(pos_np[b]) // P
                        tri[step, layer, i] = torch.tensor([b, lp, int(full[b, lp])], dtype=torch.int32)
                    st.page_table_delta_host(layer, tri[step, layer, :len(rows)])
                    sent += len(rows)
                st.decode_step_host(layer, q, k, v, pos, tab, outs[step, layer])
                assert st.poll_error() == B.OPW_OK
        results.append((outs.clone(), [p.cpu() for p in pools]))
        if use_delta:
            assert sent == 2 * sum((int(n) + steps - 1) // P - int(n) // P for n in lens)      # one triple per page opened
            with pytest.raises(B.OpwError) as e:
                B.opw_attn_stage_page_table_delta_host(st.handle, 0, tri.data_ptr(), 4 * 5 + 1)
            assert e.value.status == B.OPW_ERR_CAPACITY
            bad = torch.tensor([[7, 0, 0], [0, 10 ** 6, 0]], dtype=torch.int32).pin_memory()     # row / logical page outside the table
            st.page_table_delta_host(0, bad)
            assert st.poll_error() == B.OPW_ERR_BAD_PAGE
        st.close()
    assert torch.equal(results[0][0].view(torch.int16), results[1][0].view(torch.int16))
    for a, b in zip(results[0][1], results[1][1]):
        assert torch.equal(a.view(torch.int16), b.view(torch.int16))
    refs = [oracle.as_u16(p).copy() for p in inp.pools]
    for step in range(steps):
        for layer in range(2):
            assert oracle.kv_append(refs[layer], 8, 128, P, inp.k_new[step, layer], inp.v_new[step, layer],
                                    inp.positions(step), inp.page_tables[layer]) == 0
    for layer in range(2):
        assert (oracle.as_u16(results[1][1][layer]) == refs[layer]).all()
        ref, _, _ = oracle.decode_attention(refs[layer], 32, 8, 128, P, inp.q[steps - 1, layer], inp.kv_lens(steps - 1),
                                            inp.page_tables[layer], window=wl.layer_window[layer])
        check_close(out_to_f64(results[1][0][steps - 1, layer]), ref)


@pytest.mark.parametrize("fused", [False, True])
@pytest.mark.parametrize("flags", [0, B.OPW_PLAN_GRAPH, B.OPW_PLAN_GRAPH | B.OPW_PLAN_ADVANCE, B.OPW_PLAN_ADVANCE,
                                   B.OPW_PLAN_OVERLAP, B.OPW_PLAN_GRAPH | B.OPW_PLAN_ADVANCE | B.OPW_PLAN_OVERLAP])
def test_plan_submits_a_multi_layer_multi_microbatch_step_in_one_call(flags, fused):
    """Two layers (one windowed) x two microbatches, three decode steps, one native call per step."""
    wl = synth.Workload("p", 6, 32, 8, 128, [0, 48], "uniform_1024_4096", 78)
    lens = np.array([5, 200, 1023, 64, 15, 3000], np.int32)
    inp = synth.make_inputs(wl, device="cpu", growth=3, steps=3, lengths=lens)
    pools = [p.cuda() for p in inp.pools]
    refs = [oracle.as_u16(p).copy() for p in inp.pools]
    st = B.Stage(pools=pools, layer_window=wl.layer_window, num_q_heads=32, num_kv_heads=8, head_dim=128,
                 max_batch=4, max_pages_per_seq=inp.max_pages_per_seq)
    mbs = [slice(0, 4), slice(4, 6)]                              # microbatches of 4 and 2 sequences
    # static device buffers, bound once
    q = [[torch.empty(mb.stop - mb.start, 32, 128, dtype=torch.bfloat16, device="cuda") for mb in mbs] for _ in range(2)]
    k = [[torch.empty(mb.stop - mb.start, 8, 128, dtype=torch.bfloat16, device="cuda") for mb in mbs] for _ in range(2)]
    v = [[torch.empty_like(t) for t in row] for row in k]
    out = [[torch.empty_like(t) for t in row] for row in q]
    lse = [[torch.empty(mb.stop - mb.start, 32, dtype=torch.float32, device="cuda") for mb in mbs] for _ in range(2)]
    pos = [dev(lens[mb]) for mb in mbs]
    kvl = [dev(lens[mb] + 1) for mb in mbs]
    tabs = [[inp.page_tables[l][mb].contiguous().cuda() for mb in mbs] for l in range(2)]
    items = []
    for m, mb in enumerate(mbs):
        for l in range(2):
            items.append(dict(layer=l, batch=mb.stop - mb.start, q=q[l][m].data_ptr(), k_new=k[l][m].data_ptr(),
                              v_new=v[l][m].data_ptr(), positions=pos[m].data_ptr(),
                              kv_lens=None if fused else kvl[m].data_ptr(),
                              page_table=tabs[l][m].data_ptr(), out=out[l][m].data_ptr(), lse=lse[l][m].data_ptr()))
    plan = B.opw_attn_plan_create(st.handle, items, flags)
    stream = torch.cuda.current_stream().cuda_stream
    for step in range(3):
        for m, mb in enumerate(mbs):
            for l in range(2):
                q[l][m].copy_(inp.q[step, l][mb])
                k[l][m].copy_(inp.k_new[step, l][mb])
                v[l][m].copy_(inp.v_new[step, l][mb])
            if not flags & B.OPW_PLAN_ADVANCE:                    # the caller moves the metadata itself
                pos[m].copy_(torch.from_numpy(inp.positions(step)[mb]))
                kvl[m].copy_(torch.from_numpy(inp.kv_lens(step)[mb]))
        before = st.launch_count()
        B.opw_attn_plan_submit(plan, stream)
        assert st.poll_error() == B.OPW_OK
        assert st.launch_count() - before == 4 * (2 if fused else 3) + (2 if flags & B.OPW_PLAN_ADVANCE else 0)
        for l in range(2):
            assert oracle.kv_append(refs[l], 8, 128, P, inp.k_new[step, l], inp.v_new[step, l], inp.positions(step),
                                    inp.page_tables[l]) == 0
            assert (pools[l].cpu().view(torch.int16).numpy().view(np.uint16) == refs[l]).all()
            ref, ref_lse, _ = oracle.decode_attention(refs[l], 32, 8, 128, P, inp.q[step, l], inp.kv_lens(step),
                                                      inp.page_tables[l], window=wl.layer_window[l])
            got = torch.cat([out[l][m] for m in range(2)])
            got_lse = torch.cat([lse[l][m] for m in range(2)])
            check_close(out_to_f64(got), ref, got_lse.cpu().numpy().astype(np.float64), ref_lse)
    if flags & B.OPW_PLAN_ADVANCE:
        assert (pos[0].cpu().numpy() == lens[mbs[0]] + 3).all()
        assert fused or (kvl[1].cpu().numpy() == lens[mbs[1]] + 4).all()
    B.opw_attn_plan_destroy(plan)
    st.close()


@pytest.mark.parametrize("flags", [B.OPW_PLAN_OVERLAP, B.OPW_PLAN_OVERLAP | B.OPW_PLAN_GRAPH])
def test_overlapped_plan_with_an_empty_item_between_live_ones(flags):
    """An item with batch 0 enqueues nothing and records no event; the items around it must still be
    ordered through the workspace set they share (as a captured graph too)."""
    wl = synth.Workload("pe", 4, 32, 8, 128, [0, 48, 0, 48], "uniform_1024_4096", 83)
    inp = synth.make_inputs(wl, device="cpu", growth=1, steps=1, lengths=np.array([700, 33, 2500, 16], np.int32))
    pools = [p.cuda() for p in inp.pools]
    refs = [oracle.as_u16(p).copy() for p in inp.pools]
    st = B.Stage(pools=pools, layer_window=wl.layer_window, num_q_heads=32, num_kv_heads=8, head_dim=128,
                 max_batch=4, max_pages_per_seq=inp.max_pages_per_seq)
    dq, dk, dv = inp.q.cuda(), inp.k_new.cuda(), inp.v_new.cuda()
    pos = dev(inp.positions(0))
    tabs = [t.cuda() for t in inp.page_tables]
    outs = [torch.full((4, 32, 128), float("nan"), dtype=torch.bfloat16, device="cuda") for _ in range(4)]
    items = []
    for l in range(4):
        items.append(dict(layer=l, batch=0 if l == 1 else 4, q=dq[0, l].data_ptr(), k_new=dk[0, l].data_ptr(),
                          v_new=dv[0, l].data_ptr(), positions=pos.data_ptr(), page_table=tabs[l].data_ptr(),
                          out=outs[l].data_ptr()))
    plan = B.opw_attn_plan_create(st.handle, items, flags)
    B.opw_attn_plan_submit(plan, torch.cuda.current_stream().cuda_stream)
    assert st.poll_error() == B.OPW_OK
    for l in (0, 2, 3):
        assert oracle.kv_append(refs[l], 8, 128, P, inp.k_new[0, l], inp.v_new[0, l], inp.positions(0), inp.page_tables[l]) == 0
        ref, _, _ = oracle.decode_attention(refs[l], 32, 8, 128, P, inp.q[0, l], inp.kv_lens(0), inp.page_tables[l],
                                            window=wl.layer_window[l])
        check_close(out_to_f64(outs[l]), ref)
    for l in range(4):                                      # layer 1's pool is untouched
        assert (pools[l].cpu().view(torch.int16).numpy().view(np.uint16) == refs[l]).all()
    B.opw_attn_plan_destroy(plan)
    st.close()


@pytest.mark.parametrize("flags", [0, B.OPW_PLAN_OVERLAP | B.OPW_PLAN_GRAPH])
def test_plan_of_fused_steps_with_very_many_rows(flags):
    """512 sequences x 8 kv heads = 4096 rows: list mode in every item of a plan (with the overlap flag the
    combine of one item runs beside the next item's attention, each on its own list)."""
    wl = synth.Workload("pl", 512, 16, 8, 64, [0, 40, 0], "uniform_1_200", 84)
    inp = synth.make_inputs(wl, device="cpu", growth=1, steps=1)
    pools = [p.cuda() for p in inp.pools]
    refs = [oracle.as_u16(p).copy() for p in inp.pools]
    st = B.Stage(pools=pools, layer_window=wl.layer_window, num_q_heads=16, num_kv_heads=8, head_dim=64,
                 max_batch=512, max_pages_per_seq=inp.max_pages_per_seq)
    dq, dk, dv = inp.q.cuda(), inp.k_new.cuda(), inp.v_new.cuda()
    pos = dev(inp.positions(0))
    tabs = [t.cuda() for t in inp.page_tables]
    outs = [torch.full((512, 16, 64), float("nan"), dtype=torch.bfloat16, device="cuda") for _ in range(3)]
    items = [dict(layer=l, batch=512, q=dq[0, l].data_ptr(), k_new=dk[0, l].data_ptr(), v_new=dv[0, l].data_ptr(),
                  positions=pos.data_ptr(), page_table=tabs[l].data_ptr(), out=outs[l].data_ptr()) for l in range(3)]
    plan = B.opw_attn_plan_create(st.handle, items, flags)
    B.opw_attn_plan_submit(plan, torch.cuda.current_stream().cuda_stream)
    assert st.poll_error() == B.OPW_OK
    for l in range(3):
        assert oracle.kv_append(refs[l], 8, 64, P, inp.k_new[0, l], inp.v_new[0, l], inp.positions(0), inp.page_tables[l]) == 0
        ref, _, _ = oracle.decode_attention(refs[l], 16, 8, 64, P, inp.q[0, l], inp.kv_lens(0), inp.page_tables[l],
                                            window=wl.layer_window[l])
        check_close(out_to_f64(outs[l]), ref, max_abs=2.0 ** -8 * float(np.abs(ref).max()) + 1e-3)
        assert (pools[l].cpu().view(torch.int16).numpy().view(np.uint16) == refs[l]).all()
    B.opw_attn_plan_destroy(plan)
    st.close()


def test_overlapped_plan_needs_distinct_outputs_for_consecutive_items():
    pool = torch.zeros(4 * 2 * 2 * 16 * 64, dtype=torch.bfloat16, device="cuda")
    st = B.Stage(pools=[pool], layer_window=[0], num_q_heads=8, num_kv_heads=2, head_dim=64, max_batch=2, max_pages_per_seq=2)
    x = pool.data_ptr()
    item = dict(layer=0, batch=1, q=x, k_new=x, v_new=x, positions=x, page_table=x, out=x)
    with pytest.raises(B.OpwError) as ei:
        B.opw_attn_plan_create(st.handle, [item, dict(item)], B.OPW_PLAN_OVERLAP)
    assert ei.value.status == B.OPW_ERR_INVALID_ARG
    plan = B.opw_attn_plan_create(st.handle, [item, dict(item, out=x + 4096)], B.OPW_PLAN_OVERLAP)
    B.opw_attn_plan_destroy(plan)
    st.close()


def test_a_wait_that_runs_out_is_reported_and_the_stage_keeps_working():
    """The bounded wait gives up after 0.1 s on a barrier nothing completes; no fault, no hang."""
    rng = np.random.default_rng(65)
    Hq, Hkv, D = 8, 2, 64
    lens = [100, 3000]
    pool_np, tab, q, _, _ = make_case(rng, lens, Hq, Hkv, D)
    pool = dev(pool_np, torch.bfloat16)
    st = B.Stage(pools=[pool], layer_window=[0], num_q_heads=Hq, num_kv_heads=Hkv, head_dim=D, max_batch=2,
                 max_pages_per_seq=tab.shape[1])
    t0 = time.perf_counter()
    B.opw_attn_stage_probe_timeout(st.handle, torch.cuda.current_stream().cuda_stream)
    assert st.poll_error() == B.OPW_ERR_TIMEOUT
    assert 0.05 < time.perf_counter() - t0 < 5.0
    assert st.poll_error() == B.OPW_OK                                   # cleared
    out = torch.empty(2, Hq, D, dtype=torch.bfloat16, device="cuda")
    st.decode_attention(0, dev(q, torch.bfloat16), dev(np.asarray(lens, np.int32)), dev(tab), out)
    assert st.poll_error() == B.OPW_OK
    ref, _, _ = oracle.decode_attention(pool_np, Hq, Hkv, D, P, q, lens, tab)
    check_close(out_to_f64(out), ref)
    st.close()


def test_step_calls_validate_arguments_on_the_host():
    pool = torch.zeros(4 * 2 * 2 * 16 * 64, dtype=torch.bfloat16, device="cuda")
    st = B.Stage(pools=[pool], layer_window=[0], num_q_heads=8, num_kv_heads=2, head_dim=64, max_batch=2, max_pages_per_seq=2)
    L, h = B.lib(), st.handle
    x = pool.data_ptr()
    assert L.opw_kv_append(h, 1, 1, x, x, x, x, None) == B.OPW_ERR_INVALID_ARG          # layer out of range
    assert L.opw_kv_append(h, 0, 3, x, x, x, x, None) == B.OPW_ERR_CAPACITY             # batch > max_batch
    assert L.opw_kv_append(h, 0, 1, None, x, x, x, None) == B.OPW_ERR_INVALID_ARG
    assert L.opw_kv_append(h, 0, 1, x + 2, x, x, x, None) == B.OPW_ERR_INVALID_ARG       # misaligned
    assert L.opw_decode_attention(h, 0, 1, x, x, x, None, None, None) == B.OPW_ERR_INVALID_ARG
    assert L.opw_decode_attention(h, 0, 0, x, x, x, x, None, None) == B.OPW_OK           # empty batch: nothing to do
    assert st.launch_count() == 0
    st.close()


def test_read_sharing_rows_with_the_same_pages_and_query_agree():
    """Two batch rows may read the same pages (a shared prefix): same table, same q, same result."""
    rng = np.random.default_rng(66)
    Hq, Hkv, D = 32, 8, 128
    lens = [3000, 3000, 50, 3000]
    pool, tab, q, _, _ = make_case(rng, lens, Hq, Hkv, D)
    tab[1] = tab[0]
    tab[3] = tab[0]
    q[1] = q[0]
    q[3] = q[0]
    ref, ref_lse, _ = oracle.decode_attention(pool, Hq, Hkv, D, P, q, lens, tab)
    out, lse, rc, _ = gpu_attention(pool, tab, q, lens, Hq, Hkv, D)
    assert rc == B.OPW_OK
    got = out_to_f64(out)
    check_close(got, ref, lse, ref_lse)
    # the rows are split at different places, so they agree to rounding, not bit for bit
    assert np.abs(got[0] - got[1]).max() <= 2.0 ** -7 and np.abs(got[0] - got[3]).max() <= 2.0 ** -7


def test_all_rows_inactive_and_one_key_batches():
    rng = np.random.default_rng(60)
    Hq, Hkv, D = 32, 8, 128
    pool, tab, q, _, _ = make_case(rng, [5, 9, 1], Hq, Hkv, D)
    out, lse, rc, launches = gpu_attention(pool, tab, q, [0, -3, 0], Hq, Hkv, D)
    assert rc == B.OPW_OK and launches == 2
    assert (out_to_f64(out) == 0).all() and np.isneginf(lse).all()
    ref, ref_lse, _ = oracle.decode_attention(pool, Hq, Hkv, D, P, q, [1, 1, 1], tab)
    out, lse, rc, _ = gpu_attention(pool, tab, q, [1, 1, 1], Hq, Hkv, D)
    check_close(out_to_f64(out), ref, lse, ref_lse)


def test_many_short_sequences_fill_the_static_batch():
    """4096 slots, lengths 1..40, some inactive: rows far outnumber workers, every row is complete."""
    rng = np.random.default_rng(61)
    Hq, Hkv, D = 8, 2, 64
    lens = rng.integers(0, 41, size=4096).astype(np.int32)
    total = int(((np.maximum(lens, 1) + P - 1) // P).sum()) + 2
    maxp = 3
    tab = np.full((4096, maxp), -1, np.int32)
    order = rng.permutation(total).astype(np.int32)
    off = 0
    for b, n in enumerate(lens):
        c = (max(int(n), 1) + P - 1) // P
        tab[b, :c] = order[off:off + c]
        off += c
    pool = rand_bits(rng, oracle.pool_elems(total, Hkv, P, D))
    q = rand_bits(rng, (4096, Hq, D))
    ref, ref_lse, rc = oracle.decode_attention(pool, Hq, Hkv, D, P, q, lens, tab)
    assert rc == 0
    out, lse, rc, _ = gpu_attention(pool, tab, q, lens.tolist(), Hq, Hkv, D)
    assert rc == B.OPW_OK
    # With one or two keys the output is (nearly) a raw N(0,1) value: among 2 M of them some exceed 4,
    # where half a bf16 ulp is already 1.6e-2.  The absolute bound is stated for the benchmark
    # configurations; here the bound relative to the value (2^-8 |ref|, in check_close) is the binding one.
    check_close(out_to_f64(out), ref, lse, ref_lse, max_abs=2.0 ** -8 * float(np.abs(ref).max()) + 1e-3)


@pytest.mark.parametrize("flags", [0, B.OPW_FLAG_NO_PDL])
@pytest.mark.parametrize("window", [0, 48])
def test_very_many_rows_list_mode_split_rows_complete_rows_and_inactive_slots(flags, window):
    """batch x kv heads >= 4096: the attention kernel lists the rows it leaves as partials and the combine walks
    that list; complete rows are final as the attention kernel wrote them, inactive slots are zeroed by the
    combine.  Lengths 0..300 give all three kinds; two launches in a row check that the list's counters return
    to zero."""
    rng = np.random.default_rng(163)
    Hq, Hkv, D = 16, 8, 64
    lens = rng.integers(0, 301, size=640).astype(np.int32)
    lens[rng.integers(0, 640, size=40)] = 0
    lens = lens.tolist()
    pool_np, tab, q_bits, _, _ = make_case(rng, [max(n, 1) for n in lens], Hq, Hkv, D)
    ref, ref_lse, rc = oracle.decode_attention(pool_np, Hq, Hkv, D, P, q_bits, lens, tab, window=window)
    assert rc == 0
    pool = dev(pool_np, torch.bfloat16)
    st = B.Stage(pools=[pool], layer_window=[window], num_q_heads=Hq, num_kv_heads=Hkv, head_dim=D, max_batch=len(lens),
                 max_pages_per_seq=tab.shape[1], flags=flags)
    q, kv, tb = dev(q_bits, torch.bfloat16), dev(np.asarray(lens, np.int32)), dev(tab.astype(np.int32))
    for _ in range(2):
        out = torch.full((len(lens), Hq, D), float("nan"), dtype=torch.bfloat16, device="cuda")
        lse = torch.full((len(lens), Hq), float("nan"), dtype=torch.float32, device="cuda")
        st.decode_attention(0, q, kv, tb, out, lse)
        assert st.poll_error() == B.OPW_OK
        # short rows: the bound relative to the value is the binding one (see the test of many short sequences)
        check_close(out_to_f64(out), ref, lse.cpu().numpy().astype(np.float64), ref_lse,
                    max_abs=2.0 ** -8 * float(np.abs(ref).max()) + 1e-3)
    st.close()


def test_head_dim_256_long_rows_full_and_windowed():
    """16 query / 2 KV heads at head_dim 256 (the shape of a Qwen3-Next full-attention layer)."""
    rng = np.random.default_rng(63)
    Hq, Hkv, D = 16, 2, 256
    lens = [30000, 41, 7000, 1]
    pool, tab, q, _, _ = make_case(rng, lens, Hq, Hkv, D)
    for window in (0, 4096):
        ref, ref_lse, _ = oracle.decode_attention(pool, Hq, Hkv, D, P, q, lens, tab, window=window)
        out, lse, rc, _ = gpu_attention(pool, tab, q, lens, Hq, Hkv, D, window=window)
        assert rc == B.OPW_OK
        check_close(out_to_f64(out), ref, lse, ref_lse)


def test_sixteen_query_heads_per_kv_head_on_long_rows():
    """G = 16 (both halves of the MMA tile in use) with rows long enough to be split many times."""
    rng = np.random.default_rng(62)
    Hq, Hkv, D = 32, 2, 128
    lens = [20000, 37, 9000]
    pool, tab, q, _, _ = make_case(rng, lens, Hq, Hkv, D)
    for window in (0, 5000):
        ref, ref_lse, _ = oracle.decode_attention(pool, Hq, Hkv, D, P, q, lens, tab, window=window)
        out, lse, rc, _ = gpu_attention(pool, tab, q, lens, Hq, Hkv, D, window=window)
        assert rc == B.OPW_OK
        check_close(out_to_f64(out), ref, lse, ref_lse)


def test_workspace_too_small_and_batch_too_large_are_refused():
    pool = torch.zeros(4 * 2 * 2 * 16 * 64, dtype=torch.bfloat16, device="cuda")
    cfg, keep = B.make_config(device=0, num_q_heads=8, num_kv_heads=2, head_dim=64, max_batch=2, max_pages_per_seq=2,
                              layer_window=[0], layer_num_pages=[4], layer_kv_pool=[pool.data_ptr()])
    need = B.opw_attn_stage_workspace_bytes(cfg)
    ws = torch.empty(need + 256, dtype=torch.uint8, device="cuda")
    cfg.workspace = (ws.data_ptr() + 255) // 256 * 256
    cfg.workspace_bytes = need - 256
    with pytest.raises(B.OpwError) as ei:
        B.opw_attn_stage_create(cfg)
    assert ei.value.status == B.OPW_ERR_CAPACITY
    cfg.workspace_bytes = need
    h = B.opw_attn_stage_create(cfg)
    x = pool.data_ptr()
    assert B.lib().opw_decode_step(h, 0, 3, x, x, x, x, x, x, None, None) == B.OPW_ERR_CAPACITY
    assert B.lib().opw_decode_step(h, 0, 1, x, None, x, x, x, x, None, None) == B.OPW_ERR_INVALID_ARG
    B.opw_attn_stage_destroy(h)


# ------------------------------------------------- full-size configurations ---

def compact_rows(pool, table, rows, Hkv, D):
    """Copy only the pages the sampled rows reference into a small pool (pure data movement)."""
    pe = Hkv * 2 * P * D
    pv = pool.view(-1, pe)
    sub = table[rows].clone()
    used = torch.unique(sub[sub >= 0])
    remap = torch.full((pv.shape[0],), -1, dtype=torch.int32, device=pool.device)
    remap[used.long()] = torch.arange(used.numel(), dtype=torch.int32, device=pool.device)
    small = pv[used.long()].contiguous().view(-1)
    new_tab = torch.where(sub >= 0, remap[sub.clamp(min=0).long()], torch.full_like(sub, -1))
    return oracle.as_u16(small.cpu()), new_tab.cpu().numpy()


def run_full_config(name, sample=None, sample_full=None, layers=None, tune=None, fused=True):
    """One decode step of a benchmark configuration at full size, in the launch configuration bench.py
    times, against the oracle.  sample=None compares every row of the batch; a number compares that many
    seeded rows plus the shortest and the longest (sample_full: the same, for full-attention layers of a
    stack whose window layers are compared whole)."""
    wl = synth.WORKLOADS[name]
    inp = synth.make_inputs(wl, device="cuda", growth=1, steps=1)
    st = B.Stage(pools=inp.pools, layer_window=wl.layer_window, num_q_heads=wl.num_q_heads, num_kv_heads=wl.num_kv_heads,
                 head_dim=wl.head_dim, max_batch=wl.batch, max_pages_per_seq=inp.max_pages_per_seq, **(tune or {}))
    pos, n = inp.positions(0), inp.kv_lens(0)
    order = np.argsort(n)

    def pick(k):
        if k is None or k >= wl.batch:
            return list(range(wl.batch))
        drawn = np.random.default_rng(wl.seed).choice(order[1:-1], size=k, replace=False)      # k rows besides the two extremes
        return sorted([int(order[0]), int(order[-1])] + [int(r) for r in drawn])

    stats = []
    for layer in (layers if layers is not None else range(wl.num_layers)):
        rows = pick(sample_full if (sample_full is not None and wl.layer_window[layer] == 0) else sample)
        tab = inp.page_tables[layer]
        q, k, v = inp.q[0, layer], inp.k_new[0, layer], inp.v_new[0, layer]
        small_before, small_tab = compact_rows(inp.pools[layer], tab, rows, wl.num_kv_heads, wl.head_dim)
        out = torch.full((wl.batch, wl.num_q_heads, wl.head_dim), float("nan"), dtype=torch.bfloat16, device="cuda")
        lse = torch.full((wl.batch, wl.num_q_heads), float("nan"), dtype=torch.float32, device="cuda")
        if fused:                                   # the launch configuration bench.py times
            st.decode_step(layer, q, k, v, dev(pos), tab, out, lse)
        else:
            st.kv_append(layer, k, v, dev(pos), tab)
            st.decode_attention(layer, q, dev(n), tab, out, lse)
        assert st.poll_error() == B.OPW_OK
        assert torch.isfinite(out.float()).all()    # every row was written, compared or not
        # append parity on the compared rows' pages (bit-exact), then attention on the oracle's own pool
        ref_pool = small_before
        assert oracle.kv_append(ref_pool, wl.num_kv_heads, wl.head_dim, P, k[rows].cpu(), v[rows].cpu(), pos[rows], small_tab) == 0
        small_after, _ = compact_rows(inp.pools[layer], tab, rows, wl.num_kv_heads, wl.head_dim)
        assert np.array_equal(small_after, ref_pool)
        del small_after
        ref, ref_lse, rc = oracle.decode_attention(ref_pool, wl.num_q_heads, wl.num_kv_heads, wl.head_dim, P, q[rows].cpu(),
                                                   n[rows], small_tab, window=wl.layer_window[layer])
        assert rc == 0
        stats.append((layer, len(rows)) + check_close(out_to_f64(out[rows]), ref, lse[rows].cpu().numpy().astype(np.float64), ref_lse))
        del ref_pool, small_before
    st.close()
    return stats


@pytest.mark.parametrize("fused", [True, False])
def test_config2_llama8b_shape_all_64_rows(fused):
    stats = run_full_config("c2_llama8b", fused=fused)
    assert [s[1] for s in stats] == [64]


@pytest.mark.parametrize("fused", [True, False])
def test_config3_long_context_all_16_rows(fused):
    stats = run_full_config("c3_long_context", fused=fused)
    assert [s[1] for s in stats] == [16]


@pytest.mark.parametrize("fused", [True, False])
def test_config4_large_batch_all_256_rows(fused):
    stats = run_full_config("c4_large_batch", fused=fused)
    assert [s[1] for s in stats] == [256]


def test_config5_hybrid_stack_all_eight_layers_window_layers_whole_full_layers_on_10_rows():
    """All eight layers of the stack: the six sliding-window layers on all 128 rows, the two
    full-attention layers (19 GB of KV each) on the shortest, the longest and eight seeded rows."""
    free, _ = torch.cuda.mem_get_info()
    if free < 70 * (1 << 30):
        pytest.skip("needs ~55 GB of device memory")
    stats = run_full_config("c5_hybrid_stack", sample=None, sample_full=8)
    assert [s[0] for s in stats] == list(range(8))
    assert [s[1] for s in stats] == [128, 128, 128, 10, 128, 128, 128, 10]


def test_read_probe_touches_every_word_and_validates_arguments():
    """The bandwidth probe's sink must depend on every 16-byte word (xor of all words, per block),
    otherwise the compiler or the hardware could drop loads and the ceiling would be fiction."""
    n = (1 << 20) + 48                       # not a multiple of the unrolled stride: exercises the tail loop
    buf = torch.zeros(n, dtype=torch.uint8, device="cuda")
    sink = torch.zeros(4096, dtype=torch.float32, device="cuda")
    s = torch.cuda.current_stream().cuda_stream
    B.opw_hbm_read_probe(buf.data_ptr(), n, sink.data_ptr(), s)
    torch.cuda.synchronize()
    base = sink.view(torch.int32).clone()
    assert int(base.abs().sum()) == 0
    for off in (0, 4096 + 16, n - 16):       # flip one bit in the first, a middle and the last word
        buf.zero_()
        buf[off] = 1
        sink.zero_()
        B.opw_hbm_read_probe(buf.data_ptr(), n, sink.data_ptr(), s)
        torch.cuda.synchronize()
        assert int((sink.view(torch.int32) != 0).sum()) == 1
    for args in ((0, n), (buf.data_ptr(), 0), (buf.data_ptr(), n - 8), (buf.data_ptr() + 8, n - 16)):
        with pytest.raises(B.OpwError) as e:
            B.opw_hbm_read_probe(args[0], args[1], sink.data_ptr(), s)
        assert e.value.status == B.OPW_ERR_INVALID_ARG


def test_a_warp_count_the_register_file_cannot_hold_is_refused_at_create():
    pool = torch.zeros(4 * 8 * 2 * P * 128, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(B.OpwError) as e:
        B.Stage(pools=[pool], layer_window=[0], num_q_heads=32, num_kv_heads=8, head_dim=128, max_batch=2,
                max_pages_per_seq=2, tune_warps=12)
    assert e.value.status == B.OPW_ERR_CAPACITY
    pool64 = torch.zeros(4 * 8 * 2 * P * 64, dtype=torch.bfloat16, device="cuda")
    B.Stage(pools=[pool64], layer_window=[0], num_q_heads=32, num_kv_heads=8, head_dim=64, max_batch=2,
            max_pages_per_seq=2, tune_warps=12).close()


def test_head_dim_64_at_scale_default_twelve_warps():
    """Long rows at head_dim 64 with the default tuning (twelve warps per block): sampled rows against the oracle."""
    rng = np.random.default_rng(64)
    lens = [9000, 33, 20000, 4097, 16]
    pool, tab, q, _, _ = make_case(rng, lens, 32, 8, 64)
    ref, ref_lse, rc = oracle.decode_attention(pool, 32, 8, 64, P, q, lens, tab)
    assert rc == 0
    out, lse, rc, _ = gpu_attention(pool, tab, q, lens, 32, 8, 64)
    assert rc == B.OPW_OK
    check_close(out_to_f64(out), ref, lse, ref_lse)


@pytest.mark.parametrize("lens,Hq,Hkv,D,window", [([1_000_000, 5], 32, 8, 128, 0), ([1_048_576], 16, 2, 256, 0),
                                                   ([700_001, 33, 1], 8, 8, 64, 100_000)])
def test_million_token_contexts(lens, Hq, Hkv, D, window):
    """One sequence of about a million keys (65536 pages, thousands of partials for one row, the
    two-level combine) beside tiny ones: the fused step against the oracle on the whole output."""
    wl = synth.Workload("long", len(lens), Hq, Hkv, D, [window], "const_1", 99)
    inp = synth.make_inputs(wl, device="cuda", growth=2, steps=1, lengths=np.array(lens, np.int32))
    st = B.Stage(pools=inp.pools, layer_window=[window], num_q_heads=Hq, num_kv_heads=Hkv, head_dim=D, max_batch=len(lens),
                 max_pages_per_seq=inp.max_pages_per_seq)
    out = torch.empty(len(lens), Hq, D, dtype=torch.bfloat16, device="cuda")
    lse = torch.empty(len(lens), Hq, dtype=torch.float32, device="cuda")
    pos = torch.tensor(lens, dtype=torch.int32, device="cuda")
    q = inp.q[0, 0]
    st.decode_step(0, q, inp.k_new[0, 0], inp.v_new[0, 0], pos, inp.page_tables[0], out, lse)
    assert st.poll_error() == B.OPW_OK
    ref, ref_lse, rc = oracle.decode_attention(oracle.as_u16(inp.pools[0].cpu()), Hq, Hkv, D, P, oracle.as_u16(q.cpu()),
                                               np.array(lens, np.int32) + 1, inp.page_tables[0].cpu().numpy(), window=window)
    assert rc == 0
    check_close(out_to_f64(out), ref, lse.cpu().numpy().astype(np.float64), ref_lse)
    st.close()
