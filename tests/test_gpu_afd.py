"""GPU parity of the complete attention module (projections + rotary encoding + core attention)
against its fp64 oracle, through the C ABI.

The oracle rounds only at the module's bf16 interfaces (q, k_new, v_new, the attention output); it
knows nothing of where a kernel rounds inside.  The module is checked stage by stage, each stage fed
with the GPU's own previous result so that a rounding flip upstream is not counted again downstream,
and once end to end.  Every bound below is a sum of terms, each with its reason:

  u = 2^-8 : largest relative error of one round-to-nearest bf16 rounding (8 significant bits).
  E = hidden * 2^-24 * rms(v) : allowance for the fp32 accumulation of a `hidden`-term dot product
      (products of two bf16 values are exact in fp32; each of the `hidden` additions may lose up to
      2^-24 of a running sum whose size is of the order of the result's rms; tensor-core adders may
      truncate, so the losses can add up linearly instead of cancelling).
  partner : the other element of a rotated pair (i, i + D/2); a rotation mixes the two, so an error
      of the pair's inputs shows in proportion to |ref| + |partner|, not to |ref| alone.

  v   (both paths) : one rounding on each side of values that differ by <= E:
                     |err| <= 2u |ref| + E.
  q,k (tensor-core path: the fp32 accumulators are rotated, then rounded once):
                     inputs differ by <= E each, |cos|, |sin| <= 1, the fp32 rotation itself loses
                     <= 2^-22 (|ref| + |partner|), then one rounding on each side:
                     |err| <= 2u |ref| + 2E + 2^-22 (|ref| + |partner|).
  q,k (library path: the library GEMM stores bf16, a second kernel rotates and rounds again):
                     the extra rounding moves each input by <= u |x|, which the rotation turns into
                     <= u (|x0||cos| + |x1||sin|) <= u (|ref| + |partner|) (a rotation keeps the pair's norm):
                     |err| <= 2u |ref| + u (|ref| + |partner|) + 2E + 2^-22 (|ref| + |partner|).
  append    : the pool afterwards holds the GPU's k, v rows bit for bit.
  attention : the stated core-attention tolerance, oracle run on the GPU's q and that pool.
  y         : a K-term fp32 dot product of exactly known inputs rounded to bf16 once:
              |err| <= u |ref| + 2^-10 rms(y)   (K * 2^-24 <= 2^-10 up to K = 16384).
  end to end: the interface roundings (q, k, v, attention output; relative size <= u each, independent)
              and the probabilities' bf16 rounding pass through a projection that averages them
              over Hq*D terms: max |err| <= 2^-5 rms(y) + u |ref|, mean |err| <= 2^-7 rms(y).
"""
import numpy as np
import pytest
import torch

import oracle
from helpers import P, make_case
from oracle import afd
from paper_2609_14237_b200 import binding as B

pytestmark = pytest.mark.gpu
THETA = 10000.0


@pytest.fixture(scope="module", autouse=True)
def built():
    B.build()
    assert torch.cuda.is_available()


def to_dev_bf16(bits):
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).view(torch.bfloat16).cuda()


def f64(t):
    return oracle.bf16_bits_to_f64(t.cpu().contiguous().view(torch.int16).numpy().view(np.uint16))


def tobits(t):
    return t.cpu().contiguous().view(torch.int16).numpy().view(np.uint16)


def run_module(seed, lens, Hq, Hkv, D, hidden, steps=2, inactive=(), window=0, batches=None, flags=0):
    rng = np.random.default_rng(seed)
    Bn = len(lens)
    lens = np.asarray(lens, np.int32)
    pool_np, tab, _, _, _ = make_case(rng, [int(n) + steps for n in lens], Hq, Hkv, D)
    n_qkv = (Hq + 2 * Hkv) * D
    w_qkv_bits = oracle.f32_to_bf16_bits((rng.standard_normal((n_qkv, hidden)) / np.sqrt(hidden)).astype(np.float32))
    w_o_bits = oracle.f32_to_bf16_bits((rng.standard_normal((hidden, Hq * D)) / np.sqrt(Hq * D)).astype(np.float32))
    w_qkv, w_o = oracle.bf16_bits_to_f64(w_qkv_bits), oracle.bf16_bits_to_f64(w_o_bits)

    pool = to_dev_bf16(pool_np)
    d_tab = torch.from_numpy(tab).cuda()
    stage = B.Stage(pools=[pool], layer_window=[window], num_q_heads=Hq, num_kv_heads=Hkv, head_dim=D,
                    max_batch=Bn, max_pages_per_seq=tab.shape[1])
    mod = B.AfdModule(stage, 0, to_dev_bf16(w_qkv_bits), to_dev_bf16(w_o_bits), THETA, flags)
    ref_pool = pool_np.copy()                      # the oracle's own pool, end to end
    worst = {}
    for step in range(steps):
        nb = Bn if batches is None else batches[step]
        pos = (lens[:nb] + step).astype(np.int32)
        for i in inactive:
            if i < nb:
                pos[i] = -1
        x_bits = oracle.f32_to_bf16_bits(rng.standard_normal((nb, hidden)).astype(np.float32))
        x = oracle.bf16_bits_to_f64(x_bits)
        d_x, d_pos = to_dev_bf16(x_bits), torch.from_numpy(pos).cuda()
        y = torch.full((nb, hidden), float("nan"), dtype=torch.bfloat16, device="cuda")
        before = tobits(pool).copy()
        mod.step(d_x, d_pos, d_tab[:nb].contiguous(), y)
        torch.cuda.synchronize()
        assert stage.poll_error() == B.OPW_OK and mod.poll_error() == B.OPW_OK
        gq, gk, gv, gattn = mod.intermediates(nb)
        act = pos >= 0

        # q, k, v against the oracle's projections (bounds: see the module docstring)
        rq, rk, rv = afd.project_qkv(x, w_qkv, pos, Hq, Hkv, D, THETA)
        u = 2.0 ** -8
        E = hidden * 2.0 ** -24 * float(np.sqrt(np.mean(rv[act] ** 2))) + 1e-30
        library = bool(flags & B.OPW_AFD_LIBRARY_GEMM)           # the comparison arm; everything else is the tensor-core kernel
        pre = u if library else 0.0                          # the library path's extra rounding before the rotation
        for name, got, ref in (("q", f64(gq), rq), ("k", f64(gk), rk)):
            partner = np.concatenate([ref[..., D // 2:], ref[..., :D // 2]], axis=-1)
            pair = np.abs(ref) + np.abs(partner)
            err = np.abs(got - ref)[act]
            bound = 2 * u * np.abs(ref) + (pre + 2.0 ** -22) * pair + 2 * E
            assert (err <= bound[act]).all(), (name, float((err - bound[act]).max()))
            worst[name] = max(worst.get(name, 0.0), float(err.max()))
        verr = np.abs(f64(gv) - rv)[act]
        assert (verr <= 2 * u * np.abs(rv)[act] + E).all(), float((verr - 2 * u * np.abs(rv)[act]).max())

        # append: exactly the GPU's k, v rows, nothing else changed
        expect = before.copy()
        assert oracle.kv_append(expect, Hkv, D, P, tobits(gk), tobits(gv), pos, tab[:nb]) == 0
        after = tobits(pool)
        assert (after == expect).all()

        # attention on the GPU's q and that pool
        kv_lens = np.where(act, pos + 1, 0).astype(np.int32)
        ref_attn, _, rc = oracle.decode_attention(expect, Hq, Hkv, D, P, tobits(gq), kv_lens, tab[:nb], window=window)
        assert rc == 0
        err = np.abs(f64(gattn) - ref_attn)
        # the stated 1e-2 presumes |out| < 2.56 (half a bf16 ulp there is 2^-9 * 4 = 7.8e-3); a one-key
        # context returns v itself, which can be larger, so the bound follows the largest output
        max_abs = max(1e-2, 2.0 ** -8 * float(np.abs(ref_attn).max()) + 2e-3)
        assert err.max() <= max_abs and err.mean() <= 1e-3, (err.max(), err.mean())
        assert (f64(gattn)[~act] == 0).all()

        # output projection of the GPU's attention output
        got_y = f64(y)
        assert np.isfinite(got_y).all()
        ref_y = f64(gattn).reshape(nb, Hq * D) @ w_o.T
        rms = float(np.sqrt(np.mean(ref_y[act] ** 2)))
        assert (np.abs(got_y - ref_y) <= 2.0 ** -8 * np.abs(ref_y) + 2.0 ** -10 * rms).all(), np.abs(got_y - ref_y).max()
        assert (got_y[~act] == 0).all()

        # end to end against the oracle's own module step on its own pool
        e2e_y, _, _, _ = afd.module_step(ref_pool, x, w_qkv, w_o, pos, tab[:nb], Hq, Hkv, D, THETA, window=window)
        err = np.abs(got_y - e2e_y)
        rms = float(np.sqrt(np.mean(e2e_y[act] ** 2)))
        assert (err <= 2.0 ** -5 * rms + 2.0 ** -8 * np.abs(e2e_y)).all(), (err.max(), rms)
        assert err[act].mean() <= 2.0 ** -7 * rms, (err[act].mean(), rms)
        worst["y_rel"] = max(worst.get("y_rel", 0.0), float(err.max() / rms))
    worst["launches"] = mod.launch_count() // steps
    mod.close()
    stage.close()
    return worst


BOTH = pytest.mark.parametrize("flags", [0, B.OPW_AFD_LIBRARY_GEMM], ids=["tcgen05", "library"])


@BOTH
@pytest.mark.parametrize("Hq,Hkv,D,hidden", [(8, 2, 64, 256), (16, 2, 128, 512), (8, 2, 256, 384), (6, 3, 64, 200), (4, 1, 64, 8)])
def test_module_matches_the_oracle_stage_by_stage_and_end_to_end(Hq, Hkv, D, hidden, flags):
    run_module(11 + D, [1, 15, 16, 700, 3000], Hq, Hkv, D, hidden, steps=2, inactive=(2,), flags=flags)


def test_module_on_a_sliding_window_layer():
    run_module(5, [30, 100, 2000], 8, 2, 64, 256, steps=2, window=64)


def test_module_without_programmatic_dependent_launch():
    """The projections are launched with programmatic dependent launch by default (every other test);
    this is the opt-out: same checks with plain stream order."""
    run_module(17, [40, 900, 33, 2047], 16, 4, 128, 1024, steps=3, flags=B.OPW_AFD_NO_PDL)


@pytest.mark.parametrize("Hq,Hkv,D,hidden,n", [(8, 2, 64, 256, 5), (16, 2, 128, 512, 40), (32, 8, 128, 4096, 8), (4, 2, 64, 256, 200)])
def test_module_with_the_partial_tiles_meeting_in_the_workspace(Hq, Hkv, D, hidden, n):
    """The K-splits of a weight tile run as a thread-block cluster wherever all clusters of a launch fit the
    device (every other test at these shapes); this is the hand-off through the workspace that larger launches
    and two-tile heads fall back to: last CTA of a tile up to 128 rows, the cooperative back end above."""
    rng = np.random.default_rng(50 + n)
    run_module(51 + n, list(rng.integers(1, 300, n)), Hq, Hkv, D, hidden, steps=2, inactive=(1,), flags=B.OPW_AFD_NO_CLUSTER)


@BOTH
def test_llama8b_layer_shape_and_a_batch_that_changes_between_steps(flags):
    run_module(21, [17, 900, 33, 2047, 512, 64, 5, 1200], 32, 8, 128, 4096, steps=3, batches=[8, 3, 8], flags=flags)


@pytest.mark.parametrize("D", [64, 128, 256])
def test_batch_sizes_from_one_row_to_several_batch_tiles(D):
    """One row uses the narrowest accumulator (16 columns); 96 rows is the largest batch whose angle table
    is computed inside the kernel, 97 the first that reads it from global memory; 128 and 256 fill one
    batch tile (at head_dim 256 the two-tile epilogue then runs in one and two column chunks); 300 rows
    need two batch tiles.  All on the tensor-core kernel."""
    run_module(31, [77], 8, 2, D, 512, steps=2)
    rng = np.random.default_rng(32 + D)
    for n in (64, 96, 97, 128, 256, 300):
        w = run_module(33 + n, list(rng.integers(1, 60, n)), 4, 2, D, 256, steps=1, inactive=(0, n - 1))
        assert w["launches"] == (2 if n <= 96 else 3)          # two projections, and the angle-table kernel above 96 rows


def test_library_arm_at_large_batch_and_head_dim_256():
    rng = np.random.default_rng(35)
    run_module(36, list(rng.integers(1, 60, 130)), 4, 2, 256, 256, steps=1, flags=B.OPW_AFD_LIBRARY_GEMM)


def test_the_two_projection_paths_agree():
    """Same inputs through the tensor-core kernel (rotates the fp32 accumulators, rounds once) and
    through the library path (rounds the projection, rotates, rounds again): v agrees except where the
    summation order flips a rounding; q and k differ by the library path's extra rounding, at most
    u (|ref| + |partner|) before the last rounding (see the module docstring)."""
    outs = []
    for flags in (0, B.OPW_AFD_LIBRARY_GEMM):
        rng = np.random.default_rng(41)
        lens = [100, 2000, 31, 512]
        pool_np, tab, _, _, _ = make_case(rng, [n + 1 for n in lens], 32, 8, 128)
        w1 = to_dev_bf16(oracle.f32_to_bf16_bits((rng.standard_normal((48 * 128, 1024)) / 32).astype(np.float32)))
        w2 = to_dev_bf16(oracle.f32_to_bf16_bits((rng.standard_normal((1024, 4096)) / 64).astype(np.float32)))
        x = to_dev_bf16(oracle.f32_to_bf16_bits(rng.standard_normal((4, 1024)).astype(np.float32)))
        pool = to_dev_bf16(pool_np)
        stage = B.Stage(pools=[pool], layer_window=[0], num_q_heads=32, num_kv_heads=8, head_dim=128, max_batch=4,
                        max_pages_per_seq=tab.shape[1])
        mod = B.AfdModule(stage, 0, w1, w2, THETA, flags)
        y = torch.empty(4, 1024, dtype=torch.bfloat16, device="cuda")
        mod.step(x, torch.tensor(lens, dtype=torch.int32, device="cuda"), torch.from_numpy(tab).cuda(), y)
        torch.cuda.synchronize()
        assert mod.poll_error() == B.OPW_OK and stage.poll_error() == B.OPW_OK
        outs.append([f64(t) for t in mod.intermediates(4)[:3]] + [f64(y)])
        assert mod.launch_count() == (2 if flags == 0 else 1)
        mod.close()
        stage.close()
    u = 2.0 ** -8
    for n, (a, b) in enumerate(zip(outs[0][:3], outs[1][:3])):
        if n == 2:
            assert (a != b).mean() <= 0.01                # v: the same single rounding on both paths
        partner = np.concatenate([b[..., 64:], b[..., :64]], axis=-1) if n < 2 else 0.0
        assert (np.abs(a - b) <= 2 * u * np.abs(b) + u * (np.abs(b) + np.abs(partner)) + 1e-6).all()
    rms = float(np.sqrt(np.mean(outs[1][3] ** 2)))
    assert np.abs(outs[0][3] - outs[1][3]).max() <= 2.0 ** -5 * rms


@pytest.mark.parametrize("Hq,Hkv,D,hidden,n", [(4, 2, 256, 512, 70), (8, 2, 128, 1024, 33), (4, 2, 256, 256, 200)])
def test_cluster_and_workspace_hand_offs_give_the_same_bits(Hq, Hkv, D, hidden, n):
    """Where both hand-offs cut K the same way, the partial tiles are added in the same (split) order: q, k, v and
    y come out bit for bit the same whether the K-splits met in a thread-block cluster or in the workspace."""
    outs = []
    for flags in (0, B.OPW_AFD_NO_CLUSTER):
        rng = np.random.default_rng(77)
        lens = [int(v) for v in rng.integers(1, 90, n)]
        pool_np, tab, _, _, _ = make_case(rng, [v + 1 for v in lens], Hq, Hkv, D)
        w1 = to_dev_bf16(oracle.f32_to_bf16_bits((rng.standard_normal(((Hq + 2 * Hkv) * D, hidden)) / hidden ** 0.5).astype(np.float32)))
        w2 = to_dev_bf16(oracle.f32_to_bf16_bits((rng.standard_normal((hidden, Hq * D)) / (Hq * D) ** 0.5).astype(np.float32)))
        x = to_dev_bf16(oracle.f32_to_bf16_bits(rng.standard_normal((n, hidden)).astype(np.float32)))
        stage = B.Stage(pools=[to_dev_bf16(pool_np)], layer_window=[0], num_q_heads=Hq, num_kv_heads=Hkv, head_dim=D, max_batch=n,
                        max_pages_per_seq=tab.shape[1])
        mod = B.AfdModule(stage, 0, w1, w2, THETA, flags)
        y = torch.empty(n, hidden, dtype=torch.bfloat16, device="cuda")
        mod.step(x, torch.tensor(lens, dtype=torch.int32, device="cuda"), torch.from_numpy(tab).cuda(), y)
        torch.cuda.synchronize()
        assert mod.poll_error() == B.OPW_OK and stage.poll_error() == B.OPW_OK
        outs.append([t.clone().view(torch.int16) for t in mod.intermediates(n)[:3]] + [y.view(torch.int16)])
        mod.close()
        stage.close()
    # (these launches have so few weight tiles that their clusters fit any B200 without narrowing the K-split)
    for a, b_ in zip(outs[0], outs[1]):
        assert torch.equal(a, b_)


def test_create_and_step_validate_arguments():
    pool = torch.zeros(4 * 2 * 2 * P * 64, dtype=torch.bfloat16, device="cuda")
    stage = B.Stage(pools=[pool], layer_window=[0], num_q_heads=8, num_kv_heads=2, head_dim=64, max_batch=2,
                    max_pages_per_seq=2)
    assert B.opw_attn_stage_shape(stage.handle) == dict(device=0, num_layers=1, num_q_heads=8, num_kv_heads=2,
                                                        head_dim=64, max_batch=2)
    w_qkv = torch.zeros(12 * 64, 256, dtype=torch.bfloat16, device="cuda")
    w_o = torch.zeros(256, 8 * 64, dtype=torch.bfloat16, device="cuda")
    nbytes = B.opw_afd_module_workspace_bytes(8, 2, 64, 2, 256)
    assert nbytes > 32 << 20 and B.opw_afd_module_workspace_bytes(8, 3, 64, 2, 256) == 0
    assert B.opw_afd_module_workspace_bytes(8, 2, 64, 2, 12) == 0
    ws = torch.empty(nbytes + 256, dtype=torch.uint8, device="cuda")
    base = (ws.data_ptr() + 255) // 256 * 256
    for kw, status in ((dict(layer=1), B.OPW_ERR_INVALID_ARG), (dict(hidden=12), B.OPW_ERR_INVALID_ARG),
                       (dict(rope_theta=0.0), B.OPW_ERR_INVALID_ARG), (dict(workspace=base + 8), B.OPW_ERR_INVALID_ARG),
                       (dict(flags=8), B.OPW_ERR_INVALID_ARG),
                       (dict(workspace_bytes=nbytes - 1), B.OPW_ERR_CAPACITY)):
        args = dict(stage=stage.handle, layer=0, hidden=256, w_qkv=w_qkv.data_ptr(), w_o=w_o.data_ptr(),
                    rope_theta=1e4, workspace=base, workspace_bytes=nbytes)
        args.update(kw)
        with pytest.raises(B.OpwError) as e:
            B.opw_afd_module_create(**args)
        assert e.value.status == status
    mod = B.AfdModule(stage, 0, w_qkv, w_o)
    x = torch.zeros(3, 256, dtype=torch.bfloat16, device="cuda")
    pos = torch.zeros(3, dtype=torch.int32, device="cuda")
    tab = torch.zeros(3, 2, dtype=torch.int32, device="cuda")
    with pytest.raises(B.OpwError) as e:
        mod.step(x, pos, tab, x.clone())
    assert e.value.status == B.OPW_ERR_CAPACITY
    mod.close()
    B.opw_afd_module_destroy(None)
    stage.close()


@BOTH
def test_module_at_config_2_full_size_the_shape_the_benchmark_times(flags):
    """Llama-3-8B layer, batch 64, contexts U[1024, 4096], hidden 4096, the seeded pool and page tables
    of the benchmark's workload: every row end to end against the oracle, the whole pool bitwise."""
    from paper_2609_14237_b200 import synth

    wl = synth.WORKLOADS["c2_llama8b"]
    inp = synth.make_inputs(wl, device="cuda", growth=1, steps=1)
    Hq, Hkv, D, Bn, hidden = wl.num_q_heads, wl.num_kv_heads, wl.head_dim, wl.batch, 4096
    rng = np.random.default_rng(77)
    w_qkv_bits = oracle.f32_to_bf16_bits((rng.standard_normal(((Hq + 2 * Hkv) * D, hidden)) / np.sqrt(hidden)).astype(np.float32))
    w_o_bits = oracle.f32_to_bf16_bits((rng.standard_normal((hidden, Hq * D)) / np.sqrt(Hq * D)).astype(np.float32))
    x_bits = oracle.f32_to_bf16_bits(rng.standard_normal((Bn, hidden)).astype(np.float32))
    w_qkv, w_o, x = (oracle.bf16_bits_to_f64(a) for a in (w_qkv_bits, w_o_bits, x_bits))
    pool, tab = inp.pools[0], inp.page_tables[0]
    ref_pool = oracle.as_u16(pool.cpu()).copy()
    before = ref_pool.copy()
    pos = inp.positions(0)
    stage = B.Stage(pools=[pool], layer_window=[0], num_q_heads=Hq, num_kv_heads=Hkv, head_dim=D, max_batch=Bn,
                    max_pages_per_seq=inp.max_pages_per_seq)
    mod = B.AfdModule(stage, 0, to_dev_bf16(w_qkv_bits), to_dev_bf16(w_o_bits), THETA, flags)
    y = torch.full((Bn, hidden), float("nan"), dtype=torch.bfloat16, device="cuda")
    mod.step(to_dev_bf16(x_bits), torch.from_numpy(pos).cuda(), tab, y)
    torch.cuda.synchronize()
    assert stage.poll_error() == B.OPW_OK and mod.poll_error() == B.OPW_OK
    _, gk, gv, _ = mod.intermediates(Bn)
    tab_np = tab.cpu().numpy()
    assert oracle.kv_append(before, Hkv, D, P, tobits(gk), tobits(gv), pos, tab_np) == 0
    assert (oracle.as_u16(pool.cpu()) == before).all()
    ref_y, _, _, _ = afd.module_step(ref_pool, x, w_qkv, w_o, pos, tab_np, Hq, Hkv, D, THETA)
    got = f64(y)
    err = np.abs(got - ref_y)
    rms = float(np.sqrt(np.mean(ref_y ** 2)))
    assert np.isfinite(got).all()
    assert (err <= 2.0 ** -5 * rms + 2.0 ** -8 * np.abs(ref_y)).all(), (err.max(), rms)
    assert err.mean() <= 2.0 ** -7 * rms, (err.mean(), rms)
    mod.close()
    stage.close()


@pytest.mark.parametrize("plan_flags", [0, B.OPW_PLAN_GRAPH | B.OPW_PLAN_ADVANCE])
@BOTH
def test_a_plan_of_module_steps_equals_the_same_steps_called_one_by_one(flags, plan_flags):
    """Two layers' attention modules as ops of one plan (one native submission per token), three
    tokens: outputs and both KV pools bit for bit as from opw_afd_module_step calls."""
    rng = np.random.default_rng(91)
    Hq, Hkv, D, hidden, lens = 16, 4, 128, 1024, [40, 900, 33, 2047]
    Bn, steps = len(lens), 3
    cases = [make_case(rng, [n + steps for n in lens], Hq, Hkv, D) for _ in range(2)]
    w = [(to_dev_bf16(oracle.f32_to_bf16_bits((rng.standard_normal(((Hq + 2 * Hkv) * D, hidden)) / 32).astype(np.float32))),
          to_dev_bf16(oracle.f32_to_bf16_bits((rng.standard_normal((hidden, Hq * D)) / 45).astype(np.float32)))) for _ in range(2)]
    x = to_dev_bf16(oracle.f32_to_bf16_bits(rng.standard_normal((Bn, hidden)).astype(np.float32)))
    maxp = max(c[1].shape[1] for c in cases)
    tabs = []
    for c in cases:
        t = np.full((Bn, maxp), -1, np.int32)
        t[:, :c[1].shape[1]] = c[1]
        tabs.append(torch.from_numpy(t).cuda())
    results = []
    for use_plan in (False, True):
        pools = [to_dev_bf16(c[0]) for c in cases]
        stage = B.Stage(pools=pools, layer_window=[0, 0], num_q_heads=Hq, num_kv_heads=Hkv, head_dim=D, max_batch=Bn,
                        max_pages_per_seq=maxp)
        mods = [B.AfdModule(stage, l, w[l][0], w[l][1], THETA, flags) for l in range(2)]
        pos = torch.tensor(lens, dtype=torch.int32, device="cuda")
        ys = [torch.zeros(Bn, hidden, dtype=torch.bfloat16, device="cuda") for _ in range(2)]
        outs = []
        if use_plan:
            ops = [dict(kind="afd_module", module=mods[l].handle, batch=Bn, x=(x if l == 0 else ys[0]).data_ptr(),
                        positions=pos.data_ptr(), page_table=tabs[l].data_ptr(), y=ys[l].data_ptr()) for l in range(2)]
            plan = B.opw_attn_plan_create_mixed(stage.handle, ops, plan_flags)
        for _ in range(steps):
            if use_plan:
                B.opw_attn_plan_submit(plan, torch.cuda.current_stream().cuda_stream)
                if not plan_flags & B.OPW_PLAN_ADVANCE:
                    pos.add_(1)
            else:
                mods[0].step(x, pos, tabs[0], ys[0])
                mods[1].step(ys[0], pos, tabs[1], ys[1])      # layer 1 reads layer 0's output
                pos.add_(1)
            torch.cuda.synchronize()
            outs.append(tobits(ys[1]).copy())
        assert stage.poll_error() == B.OPW_OK and all(m.poll_error() == B.OPW_OK for m in mods)
        assert pos.cpu().tolist() == [n + steps for n in lens]
        results.append((outs, [tobits(p).copy() for p in pools]))
        if use_plan:
            B.opw_attn_plan_destroy(plan)
        for m in mods:
            m.close()
        stage.close()
    for a, b in zip(results[0][0], results[1][0]):
        assert (a == b).all()
    for a, b in zip(results[0][1], results[1][1]):
        assert (a == b).all()
    assert np.isfinite(oracle.bf16_bits_to_f64(results[1][0][-1])).all() and results[1][0][-1].any()


def test_large_batch_module_steps_in_a_captured_plan_equal_the_same_steps_called_one_by_one():
    """160 rows: the projections' CTAs share their back end under a cooperative launch (with programmatic
    dependent launch on top) and the angle table comes from its own kernel; all of it captured into one CUDA graph
    must give the outputs and the KV pool of plain calls, bit for bit."""
    rng = np.random.default_rng(93)
    Hq, Hkv, D, hidden, Bn, steps = 8, 2, 128, 512, 160, 3
    lens = [int(n) for n in rng.integers(1, 200, Bn)]
    case = make_case(rng, [n + steps for n in lens], Hq, Hkv, D)
    w1 = to_dev_bf16(oracle.f32_to_bf16_bits((rng.standard_normal(((Hq + 2 * Hkv) * D, hidden)) / 22).astype(np.float32)))
    w2 = to_dev_bf16(oracle.f32_to_bf16_bits((rng.standard_normal((hidden, Hq * D)) / 32).astype(np.float32)))
    x = to_dev_bf16(oracle.f32_to_bf16_bits(rng.standard_normal((Bn, hidden)).astype(np.float32)))
    tab = torch.from_numpy(case[1]).cuda()
    results = []
    for use_plan in (False, True):
        pool = to_dev_bf16(case[0])
        stage = B.Stage(pools=[pool], layer_window=[0], num_q_heads=Hq, num_kv_heads=Hkv, head_dim=D, max_batch=Bn,
                        max_pages_per_seq=tab.shape[1])
        mod = B.AfdModule(stage, 0, w1, w2, THETA)
        pos = torch.tensor(lens, dtype=torch.int32, device="cuda")
        y = torch.zeros(Bn, hidden, dtype=torch.bfloat16, device="cuda")
        outs = []
        if use_plan:
            plan = B.opw_attn_plan_create_mixed(stage.handle, [dict(kind="afd_module", module=mod.handle, batch=Bn, x=x.data_ptr(),
                                                                    positions=pos.data_ptr(), page_table=tab.data_ptr(), y=y.data_ptr())],
                                                B.OPW_PLAN_GRAPH | B.OPW_PLAN_ADVANCE)
        for _ in range(steps):
            if use_plan:
                B.opw_attn_plan_submit(plan, torch.cuda.current_stream().cuda_stream)
            else:
                mod.step(x, pos, tab, y)
                pos.add_(1)
            torch.cuda.synchronize()
            outs.append(tobits(y).copy())
        assert stage.poll_error() == B.OPW_OK and mod.poll_error() == B.OPW_OK
        results.append((outs, tobits(pool).copy()))
        if use_plan:
            B.opw_attn_plan_destroy(plan)
        mod.close()
        stage.close()
    for a, b in zip(results[0][0], results[1][0]):
        assert (a == b).all()
    assert (results[0][1] == results[1][1]).all()
    assert np.isfinite(oracle.bf16_bits_to_f64(results[1][0][-1])).all() and results[1][0][-1].any()
