"""CPU oracle of the decode attention stage -- TEST INFRASTRUCTURE, not product code.

Only the tests, the smoke check and the benchmark's CPU-baseline / reference legs may
import this package.  It wraps ``opw_oracle.c`` (plain C, fp64, OpenMP over
(sequence, head)) through ctypes and adds the few pure-numpy helpers the tests need to
lay structured keys and values into a pool.  Nothing here imports the CUDA package.

The oracle is the textbook definition of softmax attention over the keys visible to
each sequence after this step's append (the paper -- Section 3.4 and Section 4, the CAD
template -- says which operator the stage is, not how to compute it).
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "opw_oracle.c")
_LIB = os.path.join(_HERE, "libopw_oracle.so")

_i64 = ctypes.c_int64
_p = ctypes.c_void_p


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc if the shared object is missing or stale."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(
            ["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11", "-o", tmp, _SRC, "-lm"]
        )
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.opw_oracle_pool_index.restype = _i64
        _lib.opw_oracle_pool_index.argtypes = [_i64] * 8
        _lib.opw_oracle_num_threads.restype = ctypes.c_int
        _lib.opw_oracle_kv_append.restype = ctypes.c_int
        _lib.opw_oracle_kv_append.argtypes = [_p, _i64, _i64, _i64, _i64, _i64, _p, _p, _p, _p, _i64]
        _lib.opw_oracle_decode_attention.restype = ctypes.c_int
        _lib.opw_oracle_decode_attention.argtypes = (
            [_p, _i64, _i64, _i64, _i64, _i64, _i64, _p, _p, _p, _i64, _i64, ctypes.c_double, _p, _i64, _p, _p]
        )
    return _lib


def num_threads() -> int:
    return int(lib().opw_oracle_num_threads())


def as_u16(x) -> np.ndarray:
    """View a bf16 torch CPU tensor (or a uint16/int16 array) as contiguous uint16 numpy."""
    if isinstance(x, np.ndarray):
        assert x.dtype in (np.uint16, np.int16)
        return np.ascontiguousarray(x).view(np.uint16)
    import torch

    assert x.device.type == "cpu"
    if x.dtype == torch.bfloat16:
        x = x.contiguous().view(torch.int16)
    assert x.dtype == torch.int16
    return x.contiguous().numpy().view(np.uint16)


def _as_i32(x) -> np.ndarray:
    if hasattr(x, "cpu"):
        x = x.cpu().numpy()
    return np.ascontiguousarray(x, dtype=np.int32)


def _ptr(a: np.ndarray):
    return a.ctypes.data_as(_p)


def pool_index(Hkv: int, P: int, D: int, p: int, g: int, kv: int, t: int, d: int) -> int:
    return int(lib().opw_oracle_pool_index(Hkv, P, D, p, g, kv, t, d))


def pool_elems(num_pages: int, Hkv: int, P: int, D: int) -> int:
    return num_pages * Hkv * 2 * P * D


def kv_append(pool: np.ndarray, Hkv: int, D: int, P: int, k_new, v_new, positions, page_table) -> int:
    """In-place naive append into ``pool`` (1-D uint16, one layer)."""
    assert pool.dtype == np.uint16 and pool.flags.c_contiguous and pool.flags.writeable
    k = as_u16(k_new)
    v = as_u16(v_new)
    pos = _as_i32(positions)
    tab = _as_i32(page_table)
    B = pos.shape[0]
    assert tab.ndim == 2 and tab.shape[0] >= B
    assert k.size == B * Hkv * D and v.size == B * Hkv * D
    num_pages = pool.size // (Hkv * 2 * P * D)
    return int(
        lib().opw_oracle_kv_append(_ptr(pool), num_pages, Hkv, D, P, B, _ptr(k), _ptr(v), _ptr(pos), _ptr(tab), tab.shape[1])
    )


def decode_attention(pool: np.ndarray, Hq: int, Hkv: int, D: int, P: int, q, kv_lens, page_table,
                     window: int = 0, scale: float | None = None, rows=None):
    """fp64 attention of one query per sequence.  Returns (out [B,Hq,D], lse [B,Hq], rc).

    With ``rows`` (a list of batch indices) only those rows are computed; the rest of
    the returned arrays is NaN.
    """
    assert pool.dtype == np.uint16 and pool.flags.c_contiguous
    qq = as_u16(q)
    lens = _as_i32(kv_lens)
    tab = _as_i32(page_table)
    B = lens.shape[0]
    assert qq.size == B * Hq * D
    if scale is None:
        scale = 1.0 / float(np.sqrt(np.float64(D)))
    num_pages = pool.size // (Hkv * 2 * P * D)
    out = np.full((B, Hq, D), np.nan, dtype=np.float64)
    lse = np.full((B, Hq), np.nan, dtype=np.float64)
    if rows is None:
        rptr, nrows = None, 0
    else:
        r = np.ascontiguousarray(np.asarray(rows, dtype=np.int32))
        rptr, nrows = _ptr(r), r.size
    rc = lib().opw_oracle_decode_attention(
        _ptr(pool), num_pages, Hq, Hkv, D, P, B, _ptr(qq), _ptr(lens), _ptr(tab), tab.shape[1],
        int(window), float(scale), rptr, nrows, _ptr(out), _ptr(lse),
    )
    return out, lse, int(rc)


# ---------------------------------------------------------------------------
# numpy helpers for tests: lay logical keys/values into a pool and read them back
# through the oracle's own index formula.
# ---------------------------------------------------------------------------

def _row_perm(P: int, D: int) -> np.ndarray:
    """perm[t, d] = offset inside a (P x D) tile of logical element (t, d)."""
    t = np.arange(P)[:, None]
    d = np.arange(D)[None, :]
    return t * D + (((d // 8) ^ (t & 7)) * 8) + (d % 8)


def scatter_logical(pool: np.ndarray, Hkv: int, P: int, D: int, page_row, k_seq: np.ndarray, v_seq: np.ndarray):
    """Write a sequence's logical K/V (uint16 [n, Hkv, D]) into the pages listed in page_row."""
    n = k_seq.shape[0]
    perm = _row_perm(P, D)
    for j in range(n):
        pg, t = int(page_row[j // P]), j % P
        for g in range(Hkv):
            base_k = ((pg * Hkv + g) * 2 + 0) * P * D
            base_v = ((pg * Hkv + g) * 2 + 1) * P * D
            pool[base_k + perm[t]] = k_seq[j, g]
            pool[base_v + perm[t]] = v_seq[j, g]


def gather_logical(pool: np.ndarray, Hkv: int, P: int, D: int, page_row, lo: int, n: int):
    """Read back logical K/V rows [lo, n) of one sequence as uint16 [n-lo, Hkv, D] arrays."""
    perm = _row_perm(P, D)
    k = np.empty((n - lo, Hkv, D), dtype=np.uint16)
    v = np.empty((n - lo, Hkv, D), dtype=np.uint16)
    for j in range(lo, n):
        pg, t = int(page_row[j // P]), j % P
        for g in range(Hkv):
            base_k = ((pg * Hkv + g) * 2 + 0) * P * D
            base_v = ((pg * Hkv + g) * 2 + 1) * P * D
            k[j - lo, g] = pool[base_k + perm[t]]
            v[j - lo, g] = pool[base_v + perm[t]]
    return k, v


def bf16_bits_to_f64(u16: np.ndarray) -> np.ndarray:
    return (u16.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even fp32 -> bf16 bit patterns (finite inputs)."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = ((u >> 16) & 1) + np.uint32(0x7FFF)
    return ((u + r) >> 16).astype(np.uint16)
