"""Test-side builders shared by the oracle pins and the GPU parity tests: random logical
K/V laid into a paged pool through the oracle's layout helpers (test infrastructure)."""
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


