"""The allocation-free entry point against the oracle and the regular entry point (collected last on purpose).

Some users of the library may not allocate device memory at all -- a plug-in inside a
serving process whose memory is owned and pre-sized by the host framework, code that runs
once the memory budget is spent -- so they can neither create a stage nor hand over a
workspace.  `opw_decode_attention_noalloc` serves them from a fixed scratch array inside the
library.  Here it is called through the C ABI twice in a row, on different inputs, and each
result is compared element by element with the CPU oracle on the same inputs (the same checks
and tolerances as every other parity test, log-sum-exp included) and then with
`opw_decode_attention` (max |diff| <= 1e-2, mean |diff| <= 1e-3; the two paths split the keys
differently, so they agree up to rounding, not bitwise).  The second call reuses the scratch
the first one left behind, which is exactly what the test is after.
"""
import numpy as np
import pytest
import torch

import oracle
from helpers import LSE_TOL, MAX_ABS, MEAN_ABS, P, check_close, make_case
from paper_2609_14237_b200 import binding as B

pytestmark = pytest.mark.gpu


def to_dev(a, bf16=False):
    t = torch.from_numpy(np.ascontiguousarray(a))
    if bf16:
        t = t.view(torch.int16).view(torch.bfloat16)
    return t.cuda()


def f64(t):
    return oracle.bf16_bits_to_f64(t.cpu().view(torch.int16).numpy().view(np.uint16))


def run_both(seed, lens, Hq, Hkv, D, window):
    rng = np.random.default_rng(seed)
    pool_np, tab_np, q_np, _, _ = make_case(rng, lens, Hq, Hkv, D)
    pool, tab, q = to_dev(pool_np, True), to_dev(tab_np.astype(np.int32)), to_dev(q_np, True)
    kv = to_dev(np.asarray(lens, np.int32))
    B_ = len(lens)
    num_pages = pool.numel() // (Hkv * 2 * P * D)

    # the regular entry point: a stage with a caller-provided workspace
    st = B.Stage(pools=[pool], layer_window=[window], num_q_heads=Hq, num_kv_heads=Hkv, head_dim=D, max_batch=B_,
                 max_pages_per_seq=tab.shape[1])
    out_ref = torch.full((B_, Hq, D), float("nan"), dtype=torch.bfloat16, device="cuda")
    lse_ref = torch.full((B_, Hq), float("nan"), dtype=torch.float32, device="cuda")
    st.decode_attention(0, q, kv, tab, out_ref, lse_ref)
    assert st.poll_error() == B.OPW_OK
    st.close()

    # the allocation-free entry point: outputs are allocated here, by the caller, before the call
    out = torch.full((B_, Hq, D), float("nan"), dtype=torch.bfloat16, device="cuda")
    lse = torch.full((B_, Hq), float("nan"), dtype=torch.float32, device="cuda")
    torch.cuda.synchronize()
    B.opw_decode_attention_noalloc(num_q_heads=Hq, num_kv_heads=Hkv, head_dim=D, kv_pool=pool.data_ptr(),
                                   num_pages=num_pages, batch=B_, max_pages_per_seq=tab.shape[1], q=q.data_ptr(),
                                   kv_lens=kv.data_ptr(), page_table=tab.data_ptr(), out=out.data_ptr(),
                                   lse=lse.data_ptr(), window=window,
                                   stream=torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    # first against the oracle (the definition), then against the stage path
    ref, ref_l, rc = oracle.decode_attention(pool_np, Hq, Hkv, D, P, q_np, np.asarray(lens, np.int32), tab_np, window=window)
    assert rc == 0
    check_close(f64(out), ref, lse.cpu().numpy().astype(np.float64), ref_l)
    check_close(f64(out_ref), ref, lse_ref.cpu().numpy().astype(np.float64), ref_l)
    a, b = f64(out), f64(out_ref)
    assert np.isfinite(a).all()
    diff = np.abs(a - b)
    assert diff.max() <= MAX_ABS and diff.mean() <= MEAN_ABS, (diff.max(), diff.mean())
    la, lb = lse.cpu().numpy(), lse_ref.cpu().numpy()
    fin = np.isfinite(lb)
    assert (np.isneginf(la) == np.isneginf(lb)).all() and np.abs(la[fin] - lb[fin]).max() <= 2 * LSE_TOL


def test_noalloc_matches_the_stage_entry_point_on_two_calls_in_a_row():
    B.build()
    assert torch.cuda.is_available()
    # call 1: long rows that are split over many workers, an inactive row, a one-key row
    run_both(901, [9000, 33, 20000, 1, 0, 700], 32, 8, 128, window=0)
    # call 2, straight after: other shapes and lengths, a window, on the scratch call 1 left behind
    run_both(902, [300, 17, 4100, 2500], 8, 2, 64, window=1000)


def test_noalloc_rejects_sizes_beyond_its_fixed_scratch():
    B.build()
    L = B.lib()
    x = torch.zeros(1 << 16, dtype=torch.uint8, device="cuda").data_ptr()
    args = lambda Hq, Hkv, D, batch: (Hq, Hkv, D, 16, 0, 0.0, x, 4, batch, 4, x, x, x, x, None, None)   # noqa: E731
    assert L.opw_decode_attention_noalloc(*args(32, 2, 128, 4)) == B.OPW_ERR_CAPACITY      # group of 16 heads at D=128
    assert L.opw_decode_attention_noalloc(*args(32, 8, 128, 5000)) == B.OPW_ERR_CAPACITY   # batch beyond 4096
    assert L.opw_decode_attention_noalloc(*args(32, 8, 96, 4)) == B.OPW_ERR_UNSUPPORTED
    assert L.opw_decode_attention_noalloc(*args(32, 8, 128, 0)) == B.OPW_OK                # empty batch: nothing to do
