"""Pins for the CPU oracle (no GPU): brute force, a library routine, closed forms, invariants.

The paper prints no worked numeric example of attention, so the oracle is pinned to
the mathematics: a pure-Python restatement on tiny inputs, torch's float64
scaled_dot_product_attention on dense contiguous pages, closed forms (one key,
identical keys, two keys with known scores, uniform weights for q = 0) and the
invariants the stage must have (page permutation, window == truncated cache,
read-sharing).  Each test is chosen so that a plausible slip in the oracle -- a
dropped key, an off-by-one window, K and V swapped, the wrong head group, a missing
scale -- fails at least one of them.
"""
import math
import os
import struct

import numpy as np
import pytest
import torch

import oracle

P = 16
GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


from helpers import bits, make_case, rand_bits  # noqa: E402


def brute_force(q_bits, k_bits, v_bits, Hq, Hkv, D, lo, scale):
    """Pure-Python loops, python floats (fp64), math.exp; one sequence."""
    def f(u):
        return struct.unpack("<f", struct.pack("<I", int(u) << 16))[0]

    G = Hq // Hkv
    n = k_bits.shape[0]
    out = [[0.0] * D for _ in range(Hq)]
    lse = [0.0] * Hq
    for h in range(Hq):
        g = h // G
        s = []
        for j in range(lo, n):
            acc = 0.0
            for d in range(D):
                acc += f(q_bits[h, d]) * f(k_bits[j, g, d])
            s.append(acc * scale)
        m = max(s)
        w = [math.exp(x - m) for x in s]
        z = sum(w)
        for d in range(D):
            out[h][d] = sum(w[i] * f(v_bits[lo + i, g, d]) for i in range(len(w))) / z
        lse[h] = m + math.log(z)
    return np.array(out), np.array(lse)


# ------------------------------------------------------------------ layout ---

@pytest.mark.parametrize("Hkv,D", [(2, 64), (8, 128), (1, 64), (2, 256)])
def test_pool_index_is_a_bijection_with_contiguous_tiles(Hkv, D):
    pages = 3
    seen = np.zeros(oracle.pool_elems(pages, Hkv, P, D), dtype=np.int32)
    for p in range(pages):
        for g in range(Hkv):
            for kv in range(2):
                tile = ((p * Hkv + g) * 2 + kv) * P * D
                for t in range(P):
                    for d in range(D):
                        i = oracle.pool_index(Hkv, P, D, p, g, kv, t, d)
                        assert tile + t * D <= i < tile + (t + 1) * D      # a row stays a row
                        seen[i] += 1
    assert (seen == 1).all()


def test_pool_index_keeps_16_byte_groups_and_xors_them_with_the_slot():
    Hkv, D = 8, 128
    for t in range(P):
        for d in range(0, D, 8):
            i0 = oracle.pool_index(Hkv, P, D, 5, 3, 1, t, d)
            assert i0 % 8 == 0
            for e in range(8):
                assert oracle.pool_index(Hkv, P, D, 5, 3, 1, t, d + e) == i0 + e
            row0 = oracle.pool_index(Hkv, P, D, 5, 3, 1, t, 0) - ((0 ^ (t & 7)) * 8)
            assert (i0 - row0) // 8 == (d // 8) ^ (t & 7)


def test_numpy_row_perm_matches_the_c_index():
    for Hkv, D in [(2, 64), (8, 128)]:
        perm = oracle._row_perm(P, D)
        for t in range(P):
            for d in range(D):
                assert perm[t, d] == oracle.pool_index(Hkv, P, D, 0, 0, 0, t, d)


# ------------------------------------------------------------------ append ---

def test_append_is_bitwise_and_touches_only_the_new_rows():
    rng = np.random.default_rng(11)
    Hkv, D = 2, 64
    lens = [0, 15, 16, 255, 100]          # first slot, last slot of a page, opens a page, fills the last slot
    grown = [n + 1 for n in lens]
    pool, tab, _, ks, vs = make_case(rng, grown, 8, Hkv, D)
    before = pool.copy()
    k_new = rand_bits(rng, (len(lens), Hkv, D))
    v_new = rand_bits(rng, (len(lens), Hkv, D))
    pos = np.array(lens, dtype=np.int32)
    assert oracle.kv_append(pool, Hkv, D, P, k_new, v_new, pos, tab) == 0
    changed = np.flatnonzero(pool != before)
    assert changed.size <= len(lens) * 2 * Hkv * D
    for b, n in enumerate(lens):
        k, v = oracle.gather_logical(pool, Hkv, P, D, tab[b], 0, n + 1)
        assert (k[:n] == ks[b][:n]).all() and (v[:n] == vs[b][:n]).all()     # history untouched
        assert (k[n] == k_new[b]).all() and (v[n] == v_new[b]).all()          # new row bit-exact
    # every changed element is one of the predicted offsets
    predicted = set()
    for b, n in enumerate(lens):
        pg, t = int(tab[b, n // P]), n % P
        for g in range(Hkv):
            for kv in range(2):
                for d in range(D):
                    predicted.add(oracle.pool_index(Hkv, P, D, pg, g, kv, t, d))
    assert set(changed.tolist()) <= predicted


def test_append_skips_inactive_rows_and_reports_bad_pages():
    rng = np.random.default_rng(12)
    Hkv, D = 2, 64
    pool, tab, _, _, _ = make_case(rng, [20, 20], 8, Hkv, D)
    before = pool.copy()
    k_new = rand_bits(rng, (2, Hkv, D))
    v_new = rand_bits(rng, (2, Hkv, D))
    assert oracle.kv_append(pool, Hkv, D, P, k_new, v_new, np.array([-1, -1], np.int32), tab) == 0
    assert (pool == before).all()
    bad = tab.copy()
    bad[1, 1] = 10_000
    assert oracle.kv_append(pool, Hkv, D, P, k_new, v_new, np.array([-1, 19], np.int32), bad) == -1
    assert (pool == before).all()


# --------------------------------------------------------------- attention ---

@pytest.mark.parametrize("n", [1, 2, 15, 16, 17, 33])
def test_attention_matches_pure_python_brute_force_single_head(n):
    rng = np.random.default_rng(100 + n)
    pool, tab, q, ks, vs = make_case(rng, [n], 1, 1, 64)
    out, lse, rc = oracle.decode_attention(pool, 1, 1, 64, P, q, [n], tab)
    ref_o, ref_l = brute_force(q[0], ks[0], vs[0], 1, 1, 64, 0, 1.0 / math.sqrt(64))
    assert rc == 0
    np.testing.assert_allclose(out[0], ref_o, rtol=0, atol=1e-12)
    np.testing.assert_allclose(lse[0], ref_l, rtol=0, atol=1e-12)


def test_attention_matches_brute_force_grouped_heads_and_window():
    rng = np.random.default_rng(7)
    Hq, Hkv, D = 8, 2, 64
    lens = [18, 65, 101, 256]
    pool, tab, q, ks, vs = make_case(rng, lens, Hq, Hkv, D)
    for window in (0, 40):
        out, lse, rc = oracle.decode_attention(pool, Hq, Hkv, D, P, q, lens, tab, window=window)
        assert rc == 0
        for b, n in enumerate(lens):
            lo = max(0, n - window) if window else 0
            ref_o, ref_l = brute_force(q[b], ks[b], vs[b], Hq, Hkv, D, lo, 1.0 / math.sqrt(D))
            np.testing.assert_allclose(out[b], ref_o, rtol=0, atol=1e-12)
            np.testing.assert_allclose(lse[b], ref_l, rtol=0, atol=1e-12)


@pytest.mark.parametrize("Hq,Hkv,D,scale", [(8, 2, 64, None), (32, 8, 128, None), (16, 2, 128, 0.37), (4, 4, 64, None),
                                            (16, 2, 256, None)])
def test_attention_matches_torch_sdpa_float64_on_dense_pages(Hq, Hkv, D, scale):
    rng = np.random.default_rng(21)
    lens = [96, 96, 96]
    pool, tab, q, ks, vs = make_case(rng, lens, Hq, Hkv, D, scrambled=False)
    out, lse, rc = oracle.decode_attention(pool, Hq, Hkv, D, P, q, lens, tab, scale=scale)
    assert rc == 0
    K = torch.from_numpy(np.stack([oracle.bf16_bits_to_f64(k) for k in ks])).permute(0, 2, 1, 3)   # [B,Hkv,n,D]
    V = torch.from_numpy(np.stack([oracle.bf16_bits_to_f64(v) for v in vs])).permute(0, 2, 1, 3)
    Q = torch.from_numpy(oracle.bf16_bits_to_f64(q)).unsqueeze(2)                                  # [B,Hq,1,D]
    ref = torch.nn.functional.scaled_dot_product_attention(Q, K, V, scale=scale, enable_gqa=True).squeeze(2)
    np.testing.assert_allclose(out, ref.numpy(), rtol=0, atol=1e-12)


def test_single_key_returns_v_exactly_and_lse_is_the_score():
    rng = np.random.default_rng(3)
    Hq, Hkv, D = 8, 2, 64
    pool, tab, q, ks, vs = make_case(rng, [1, 1], Hq, Hkv, D)
    out, lse, _ = oracle.decode_attention(pool, Hq, Hkv, D, P, q, [1, 1], tab)
    G = Hq // Hkv
    for b in range(2):
        for h in range(Hq):
            assert (out[b, h] == oracle.bf16_bits_to_f64(vs[b][0, h // G])).all()
            s0 = float(oracle.bf16_bits_to_f64(q[b, h]) @ oracle.bf16_bits_to_f64(ks[b][0, h // G])) / 8.0
            assert abs(lse[b, h] - s0) < 1e-12


def test_identical_keys_give_the_mean_of_v_and_lse_s_plus_log_n():
    rng = np.random.default_rng(4)
    Hq, Hkv, D, n = 8, 2, 64, 45
    pool, tab, q, ks, vs = make_case(rng, [n], Hq, Hkv, D)
    k = np.broadcast_to(ks[0][:1], ks[0].shape).copy()
    oracle.scatter_logical(pool, Hkv, P, D, tab[0], k, vs[0])
    out, lse, _ = oracle.decode_attention(pool, Hq, Hkv, D, P, q, [n], tab)
    G = Hq // Hkv
    V = oracle.bf16_bits_to_f64(vs[0])
    for h in range(Hq):
        np.testing.assert_allclose(out[0, h], V[:, h // G].mean(axis=0), rtol=0, atol=1e-13)
        s = float(oracle.bf16_bits_to_f64(q[0, h]) @ oracle.bf16_bits_to_f64(k[0, h // G])) / 8.0
        assert abs(lse[0, h] - (s + math.log(n))) < 1e-12


def test_two_keys_with_known_scores_closed_form_golden():
    """q = 8*e0, K_0[0] = 0, K_1[0] = 1 (D = 64, scale 1/8): weights 1/(1+e), e/(1+e)."""
    with open(os.path.join(GOLDEN, "softmax_two_keys.txt")) as fh:
        vals = [float(x) for x in fh.read().split("#")[0].split()]
    w0, w1, lse_ref = vals
    Hq = Hkv = 1
    D = 64
    k = np.zeros((2, 1, D), np.float32)
    k[1, 0, 0] = 1.0
    v = np.zeros((2, 1, D), np.float32)
    v[0, 0, 0] = 1.0
    v[1, 0, 1] = 1.0
    q = np.zeros((1, 1, D), np.float32)
    q[0, 0, 0] = 8.0
    pool = np.zeros(oracle.pool_elems(1, Hkv, P, D), np.uint16)
    tab = np.zeros((1, 1), np.int32)
    oracle.scatter_logical(pool, Hkv, P, D, tab[0], bits(k), bits(v))
    out, lse, _ = oracle.decode_attention(pool, Hq, Hkv, D, P, bits(q), [2], tab)
    assert abs(out[0, 0, 0] - w0) < 1e-15 and abs(out[0, 0, 1] - w1) < 1e-15
    assert abs(lse[0, 0] - lse_ref) < 1e-15
    assert abs(out[0, 0].sum() - 1.0) < 1e-15


@pytest.mark.parametrize("window", [0, 1, 16, 17, 40, 64, 1000])
def test_q_zero_probes_count_every_visible_key_exactly_once(window):
    """q = 0 makes the weights uniform, so indicator values count the keys attended."""
    rng = np.random.default_rng(5)
    Hq, Hkv, D = 4, 2, 64
    lens = [1, 16, 17, 63, 64, 65, 130]
    pool, tab, q, ks, vs = make_case(rng, lens, Hq, Hkv, D)
    q[:] = 0
    one = bits(np.float32(1.0))
    for j0 in (0, 15, 16, 62, 129):
        for b, n in enumerate(lens):
            lo = max(0, n - window) if window else 0
            v = np.zeros((n, Hkv, D), np.uint16)
            v[:, :, 0] = one                                  # coverage: must sum to 1
            if j0 < n:
                v[j0, :, 1] = one                             # one marked key
            v[:lo, :, 2] = one                                # keys before the window
            oracle.scatter_logical(pool, Hkv, P, D, tab[b], ks[b], v)
        out, lse, _ = oracle.decode_attention(pool, Hq, Hkv, D, P, q, lens, tab, window=window)
        for b, n in enumerate(lens):
            lo = max(0, n - window) if window else 0
            n_eff = n - lo
            np.testing.assert_allclose(out[b, :, 0], 1.0, atol=1e-14)
            want = 1.0 / n_eff if lo <= j0 < n else 0.0
            np.testing.assert_allclose(out[b, :, 1], want, atol=1e-15)
            assert (out[b, :, 2] == 0.0).all()
            np.testing.assert_allclose(lse[b], math.log(n_eff), atol=1e-13)


def test_page_permutation_leaves_the_result_unchanged():
    rng = np.random.default_rng(6)
    Hq, Hkv, D = 8, 2, 64
    lens = [18, 65, 101, 256]
    pool, tab, q, ks, vs = make_case(rng, lens, Hq, Hkv, D)
    ref, ref_lse, _ = oracle.decode_attention(pool, Hq, Hkv, D, P, q, lens, tab, window=0)
    total = pool.size // (Hkv * 2 * P * D)
    perm = rng.permutation(total)                       # physical page p moves to perm[p]
    page_elems = Hkv * 2 * P * D
    pool2 = np.empty_like(pool)
    for p_old in range(total):
        pool2[perm[p_old] * page_elems:(perm[p_old] + 1) * page_elems] = pool[p_old * page_elems:(p_old + 1) * page_elems]
    tab2 = np.where(tab >= 0, perm[np.maximum(tab, 0)], -1).astype(np.int32)
    out, lse, _ = oracle.decode_attention(pool2, Hq, Hkv, D, P, q, lens, tab2, window=0)
    assert (out == ref).all() and (lse == ref_lse).all()


@pytest.mark.parametrize("W", [1, 5, 16, 33, 64])
def test_window_equals_full_attention_over_the_truncated_cache(W):
    rng = np.random.default_rng(8)
    Hq, Hkv, D = 8, 2, 64
    lens = [18, 65, 101, 256]
    pool, tab, q, ks, vs = make_case(rng, lens, Hq, Hkv, D)
    out, lse, _ = oracle.decode_attention(pool, Hq, Hkv, D, P, q, lens, tab, window=W)
    # re-page a cache that only holds the last W tokens of each sequence
    tlens = [min(n, W) for n in lens]
    pool_t, tab_t, _, _, _ = make_case(rng, tlens, Hq, Hkv, D)
    for b, n in enumerate(lens):
        oracle.scatter_logical(pool_t, Hkv, P, D, tab_t[b], ks[b][n - tlens[b]:], vs[b][n - tlens[b]:])
    ref, ref_lse, _ = oracle.decode_attention(pool_t, Hq, Hkv, D, P, q, tlens, tab_t, window=0)
    np.testing.assert_allclose(out, ref, rtol=0, atol=1e-13)
    np.testing.assert_allclose(lse, ref_lse, rtol=0, atol=1e-13)


def test_window_at_least_n_is_full_and_entries_before_the_window_are_never_read():
    rng = np.random.default_rng(9)
    Hq, Hkv, D = 8, 2, 64
    lens = [18, 65, 101, 256]
    pool, tab, q, ks, vs = make_case(rng, lens, Hq, Hkv, D)
    full, full_lse, _ = oracle.decode_attention(pool, Hq, Hkv, D, P, q, lens, tab, window=0)
    big, big_lse, _ = oracle.decode_attention(pool, Hq, Hkv, D, P, q, lens, tab, window=256)
    assert (full == big).all() and (full_lse == big_lse).all()
    W = 40
    ref, _, _ = oracle.decode_attention(pool, Hq, Hkv, D, P, q, lens, tab, window=W)
    poisoned = tab.copy()
    for b, n in enumerate(lens):
        lo = max(0, n - W)
        poisoned[b, :lo // P] = -1                     # pages wholly before the window
        poisoned[b, (n + P - 1) // P:] = -1            # and everything after the last page
    out, _, rc = oracle.decode_attention(pool, Hq, Hkv, D, P, q, lens, poisoned, window=W)
    assert rc == 0 and (out == ref).all()


def test_read_sharing_and_inactive_rows():
    rng = np.random.default_rng(10)
    Hq, Hkv, D = 8, 2, 64
    pool, tab, q, ks, vs = make_case(rng, [70, 70, 5], Hq, Hkv, D)
    tab[1] = tab[0]
    q[1] = q[0]
    out, lse, _ = oracle.decode_attention(pool, Hq, Hkv, D, P, q, [70, 70, 0], tab)
    assert (out[0] == out[1]).all() and (lse[0] == lse[1]).all()
    assert (out[2] == 0).all() and np.isneginf(lse[2]).all()


def test_head_group_map_is_contiguous_blocks():
    """Heads h and h' share keys/values iff h // G == h' // G (probed with per-group V)."""
    Hq, Hkv, D, n = 8, 2, 64, 20
    rng = np.random.default_rng(13)
    pool, tab, q, ks, vs = make_case(rng, [n], Hq, Hkv, D)
    q[:] = 0
    v = np.zeros((n, Hkv, D), np.float32)
    v[:, 0, 0] = 1.0
    v[:, 1, 0] = 2.0
    oracle.scatter_logical(pool, Hkv, P, D, tab[0], ks[0], bits(v))
    out, _, _ = oracle.decode_attention(pool, Hq, Hkv, D, P, q, [n], tab)
    np.testing.assert_allclose(out[0, :4, 0], 1.0, atol=1e-14)
    np.testing.assert_allclose(out[0, 4:, 0], 2.0, atol=1e-14)


def test_rows_argument_computes_only_the_sampled_rows():
    rng = np.random.default_rng(14)
    Hq, Hkv, D = 8, 2, 64
    lens = [18, 65, 101]
    pool, tab, q, _, _ = make_case(rng, lens, Hq, Hkv, D)
    full, _, _ = oracle.decode_attention(pool, Hq, Hkv, D, P, q, lens, tab)
    part, _, _ = oracle.decode_attention(pool, Hq, Hkv, D, P, q, lens, tab, rows=[2, 0])
    assert (part[0] == full[0]).all() and (part[2] == full[2]).all() and np.isnan(part[1]).all()
