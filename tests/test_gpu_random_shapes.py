"""Seeded random shapes, lengths, windows and tunings through the C ABI against the oracle: head
counts and group sizes that are not powers of two, empty and one-key rows beside long ones, windows
shorter than a page, odd warp counts -- the corners hand-written cases tend to miss.  Appended
bytes bit-exact over the whole pool, attention within 2^-6 of each row's rms (+ half a bf16 ulp),
log-sum-exp within 2e-3."""
import numpy as np
import pytest
import torch

import oracle
from helpers import P, make_case, rand_bits
from paper_2609_14237_b200 import binding as B

pytestmark = pytest.mark.gpu


def dev(a, bf=False):
    t = torch.from_numpy(np.ascontiguousarray(a))
    if bf:
        t = t.view(torch.int16).view(torch.bfloat16)
    return t.cuda()


def draw_case(rng):
    D = int(rng.choice([64, 128, 256]))
    Hkv = int(rng.choice([1, 2, 3, 8]))
    G = int(rng.choice([g for g in (1, 2, 3, 4, 5, 8, 12, 16) if g <= (8 if D == 256 else 16)]))
    Bn = int(rng.choice([1, 2, 3, 7, 16, 40]))
    kind = int(rng.integers(0, 4))
    if kind == 0:
        lens = rng.integers(0, 70, Bn)
    elif kind == 1:
        lens = rng.integers(1, 3000, Bn)
    elif kind == 2:
        lens = np.clip(np.rint(np.exp(rng.normal(6.0, 1.5, Bn))), 0, 30000).astype(np.int64)
    else:
        lens = rng.integers(1, 200, Bn)
        lens[rng.integers(0, Bn)] = int(rng.integers(5000, 40000))
    budget = 60000 // max(1, Hkv * D // 64)                  # keeps the oracle at a fraction of a second per case
    while lens.sum() > budget:
        lens = lens // 2
    window = int(rng.choice([0, 0, 1, 16, 17, 100, 1024, 5000]))
    tune = {}
    if rng.integers(0, 3) == 0:
        tune = dict(tune_warps=int(rng.choice([1, 2, 4, 6] if D == 256 else [1, 3, 4, 8])), tune_stages=int(rng.choice([2, 3, 4])))
    if rng.integers(0, 4) == 0:
        tune["flags"] = B.OPW_FLAG_NO_PDL
    return D, Hkv * G, Hkv, [int(x) for x in lens], window, bool(rng.integers(0, 2)), tune


@pytest.mark.parametrize("block", range(8))
def test_random_cases_match_the_oracle(block):
    B.build()
    for it in range(12):
        rng = np.random.default_rng(7_000_000 + 100 * block + it)
        D, Hq, Hkv, lens, window, fused, tune = draw_case(rng)
        Bn = len(lens)
        post = [n + 1 for n in lens] if fused else lens
        pool_np, tab, q, _, _ = make_case(rng, [max(n, 1) for n in post], Hq, Hkv, D)
        pool = dev(pool_np, True)
        try:
            st = B.Stage(pools=[pool], layer_window=[window], num_q_heads=Hq, num_kv_heads=Hkv, head_dim=D, max_batch=Bn,
                         max_pages_per_seq=tab.shape[1], **tune)
        except B.OpwError as e:                             # a drawn tuning whose ring does not fit an SM
            assert e.status == B.OPW_ERR_CAPACITY and tune
            continue
        out = torch.full((Bn, Hq, D), float("nan"), dtype=torch.bfloat16, device="cuda")
        lse = torch.full((Bn, Hq), float("nan"), dtype=torch.float32, device="cuda")
        ref_pool = pool_np.copy()
        if fused:
            k_new, v_new = rand_bits(rng, (Bn, Hkv, D)), rand_bits(rng, (Bn, Hkv, D))
            pos = np.array(lens, np.int32)
            if Bn > 2 and rng.integers(0, 3) == 0:
                pos[rng.integers(0, Bn)] = -1
            st.decode_step(0, dev(q, True), dev(k_new, True), dev(v_new, True), dev(pos), dev(tab), out, lse)
            assert oracle.kv_append(ref_pool, Hkv, D, P, k_new, v_new, pos, tab) == 0
            kv = np.where(pos >= 0, pos + 1, 0).astype(np.int32)
        else:
            kv = np.array(lens, np.int32)
            st.decode_attention(0, dev(q, True), dev(kv), dev(tab), out, lse)
        what = dict(D=D, Hq=Hq, Hkv=Hkv, lens=lens[:8], window=window, fused=fused, tune=tune)
        assert st.poll_error() == B.OPW_OK, what
        assert (pool.cpu().view(torch.int16).numpy().view(np.uint16) == ref_pool).all(), what
        ref, ref_lse, rc = oracle.decode_attention(ref_pool, Hq, Hkv, D, P, q, kv, tab, window=window)
        assert rc == 0
        got = oracle.bf16_bits_to_f64(out.cpu().view(torch.int16).numpy().view(np.uint16))
        gl = lse.cpu().numpy().astype(np.float64)
        err = np.abs(got - ref)
        row_rms = np.sqrt(np.mean(ref ** 2, axis=-1, keepdims=True))
        assert np.isfinite(got).all(), what
        assert (err <= 2.0 ** -6 * row_rms + 2.0 ** -8 * np.abs(ref) + 1e-6).all(), (what, float(err.max()))
        fin = np.isfinite(ref_lse)
        assert (np.isneginf(gl) == np.isneginf(ref_lse)).all(), what
        assert (np.abs(gl[fin] - ref_lse[fin]) <= 1e-3).all(), what
        st.close()
