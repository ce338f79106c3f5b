"""Test-side builders shared by the oracle pins and the GPU parity tests: random logical
K/V laid into a paged pool through the oracle's layout helpers, and the comparison of a GPU
result with the oracle's at the stated tolerance (test infrastructure)."""
import numpy as np

import oracle

P = 16


def bits(x):
    """float array -> bf16 bit patterns (RNE)."""
    return oracle.f32_to_bf16_bits(np.asarray(x, dtype=np.float32))


def rand_bits(rng, shape):
    return bits(rng.standard_normal(shape).astype(np.float32))


def make_case(rng, lens, Hq, Hkv, D, extra_pages=2, scrambled=True):
    """Random logical K/V per sequence laid into a pool through a (permuted) page table."""
    B = len(lens)
    npages = [(n + P - 1) // P for n in lens]
    total = sum(npages) + extra_pages
    order = rng.permutation(total) if scrambled else np.arange(total)
    maxp = max(npages)
    tab = np.full((B, maxp), -1, dtype=np.int32)
    pool = rand_bits(rng, oracle.pool_elems(total, Hkv, P, D))      # garbage everywhere first
    ks, vs, off = [], [], 0
    for b, n in enumerate(lens):
        tab[b, :npages[b]] = order[off:off + npages[b]]
        off += npages[b]
        k = rand_bits(rng, (n, Hkv, D))
        v = rand_bits(rng, (n, Hkv, D))
        oracle.scatter_logical(pool, Hkv, P, D, tab[b], k, v)
        ks.append(k)
        vs.append(v)
    q = rand_bits(rng, (B, Hq, D))
    return pool, tab, q, ks, vs




# ---------------------------------------------------------------- tolerances ---
MAX_ABS, MEAN_ABS = 1e-2, 1e-3          # the stated tolerance: bf16 inputs, fp32 accumulation, bf16 output
REL_RMS = 2.0 ** -6                     # max |err| / rms(row): catches a dropped chunk of a long context
LSE_TOL = 1e-3                          # fp32 log-sum-exp against fp64


def out_to_f64(t):
    """bf16 torch tensor (any device) -> float64 numpy, exactly."""
    import torch

    return oracle.bf16_bits_to_f64(t.cpu().contiguous().view(torch.int16).numpy().view(np.uint16))


def check_close(got, ref, lse_got=None, lse_ref=None, rows=None, max_abs=MAX_ABS):
    """Element-wise comparison of an attention output (float64 views) with the oracle's."""
    if rows is not None:
        got, ref = got[rows], ref[rows]
        if lse_got is not None:
            lse_got, lse_ref = lse_got[rows], lse_ref[rows]
    err = np.abs(got - ref)
    rms = float(np.sqrt(np.mean(ref ** 2)))
    assert np.isfinite(got).all()
    assert err.max() <= max_abs, err.max()
    assert err.mean() <= MEAN_ABS, err.mean()
    # per (sequence, head) relative check: error against that row's own rms (+ bf16 half-ulp slack)
    row_rms = np.sqrt(np.mean(ref ** 2, axis=-1, keepdims=True))
    assert (err <= REL_RMS * row_rms + 2.0 ** -8 * np.abs(ref) + 1e-6).all(), float((err / (row_rms + 1e-30)).max())
    if lse_got is not None:
        fin = np.isfinite(lse_ref)
        assert (np.isneginf(lse_got) == np.isneginf(lse_ref)).all()
        assert not fin.any() or np.abs(lse_got[fin] - lse_ref[fin]).max() <= LSE_TOL
    return float(err.max()), float(err.mean()), rms
