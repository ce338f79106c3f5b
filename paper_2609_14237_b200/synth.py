"""Seeded synthetic inputs for the decode attention stage.

This module is shared by the tests (which feed the same tensors to the CPU oracle and
to the CUDA path) and by the benchmark.  It contains no attention arithmetic and does not
know where an element sits inside a pool (only how many elements a page has): pools are
filled with independent N(0,1) bf16 values, which is the same distribution under any
layout, and page tables are seeded random permutations of the physical pages dealt to the
sequences.

The five named workloads stand in for the paper's decode workloads (Section 7.1:
context-length cohorts derived from a public reasoning dataset and rescaled to 8K /
32K / 128K means on two hybrid-attention models); neither that dataset nor the model
weights are used here.
"""
from __future__ import annotations

import dataclasses
import math
from typing import List, Optional

import numpy as np
import torch

PAGE = 16


@dataclasses.dataclass
class Workload:
    name: str
    batch: int
    num_q_heads: int
    num_kv_heads: int
    head_dim: int
    layer_window: List[int]          # per layer: 0 = full attention, W > 0 = sliding window
    lengths: str                     # recipe name, see draw_lengths
    seed: int
    page_size: int = PAGE

    @property
    def num_layers(self) -> int:
        return len(self.layer_window)

    @property
    def kv_bytes_per_token(self) -> int:
        return 2 * self.num_kv_heads * self.head_dim * 2


WORKLOADS = {
    # tiny: batch 4, 8/2 heads, D=64, lengths {17, 64, 100, 255}
    "c1_tiny": Workload("c1_tiny", 4, 8, 2, 64, [0], "tiny", 1001),
    # Llama-3-8B-shaped layer: batch 64, 32/8 heads, D=128, U[1024, 4096]
    "c2_llama8b": Workload("c2_llama8b", 64, 32, 8, 128, [0], "uniform_1024_4096", 1002),
    # long context: batch 16, every sequence 32768 tokens
    "c3_long_context": Workload("c3_long_context", 16, 32, 8, 128, [0], "const_32768", 1003),
    # 70B-shaped large batch: batch 256, 64/8 heads, lognormal lengths
    "c4_large_batch": Workload("c4_large_batch", 256, 64, 8, 128, [0], "lognormal_2048", 1004),
    # hybrid stack: 8 layers, 3 sliding-window (4096) : 1 full, batch 128, U[8192, 65536]
    "c5_hybrid_stack": Workload(
        "c5_hybrid_stack", 128, 32, 8, 128, [4096, 4096, 4096, 0, 4096, 4096, 4096, 0],
        "uniform_8192_65536", 1005),
    # one sliding-window layer of the hybrid stack on its own (same shape, lengths and seed): 2.15 GB of
    # mapped pages, small enough to profile where the whole 52 GB stack is not
    "c5_window_layer": Workload("c5_window_layer", 128, 32, 8, 128, [4096], "uniform_8192_65536", 1005),
    # not one of the five benchmark configurations: a stack shaped like the paper's first evaluated
    # model (sliding-window : full = 5 : 1, 32 query / 16 KV heads of 128; the window, 1024, is an
    # assumption -- the paper prints only the ratio), batch 64, contexts U[8192, 32768]
    "m1_swa5to1_stack": Workload(
        "m1_swa5to1_stack", 64, 32, 16, 128, [1024, 1024, 1024, 1024, 1024, 0], "uniform_8192_32768", 1101),
}


def draw_lengths(recipe: str, batch: int, seed: int) -> np.ndarray:
    """Pre-append context lengths (the write position of this step's token)."""
    rng = np.random.default_rng(seed)
    if recipe == "tiny":
        base = np.array([17, 64, 100, 255], dtype=np.int64)
        return np.resize(base, batch).astype(np.int32)
    if recipe.startswith("const_"):
        return np.full(batch, int(recipe.split("_")[1]), dtype=np.int32)
    if recipe.startswith("uniform_"):
        lo, hi = (int(x) for x in recipe.split("_")[1:3])
        return rng.integers(lo, hi + 1, size=batch).astype(np.int32)
    if recipe.startswith("lognormal_"):
        # median given, sigma = 1 (natural log), clipped to [16, 16384]
        med = float(recipe.split("_")[1])
        z = rng.standard_normal(batch)
        return np.clip(np.rint(np.exp(math.log(med) + z)), 16, 16384).astype(np.int32)
    raise ValueError(recipe)


@dataclasses.dataclass
class StageInputs:
    wl: Workload
    lengths: np.ndarray              # int32 [B], pre-append
    growth: int                      # decode steps the page tables have room for
    max_pages_per_seq: int
    page_tables: List[torch.Tensor]  # per layer int32 [B, max_pages_per_seq], -1 = unmapped
    num_pages: List[int]             # per layer physical pages
    pools: List[torch.Tensor]        # per layer bf16 [num_pages * Hkv * 2 * P * D]
    q: torch.Tensor                  # bf16 [steps, layers, B, Hq, D]
    k_new: torch.Tensor              # bf16 [steps, layers, B, Hkv, D]
    v_new: torch.Tensor

    def positions(self, step: int) -> np.ndarray:
        return (self.lengths + step).astype(np.int32)

    def kv_lens(self, step: int) -> np.ndarray:
        return (self.lengths + step + 1).astype(np.int32)

    def visible_tokens(self, layer: int, step: int = 0) -> int:
        n = self.kv_lens(step).astype(np.int64)
        w = self.wl.layer_window[layer]
        return int(np.minimum(n, w).sum() if w > 0 else n.sum())

    def kv_bytes(self, layer: int, step: int = 0) -> int:
        """Algorithmic bytes: the K and V rows attention must read for one layer-step."""
        return self.visible_tokens(layer, step) * self.wl.kv_bytes_per_token


def _fill_normal_bf16(t: torch.Tensor, gen: torch.Generator, chunk: int = 1 << 26) -> None:
    flat = t.view(-1)
    for i in range(0, flat.numel(), chunk):
        flat[i:i + chunk].normal_(0.0, 1.0, generator=gen)


def make_inputs(wl: Workload, device: str = "cpu", growth: int = 1, steps: int = 1,
                lengths: Optional[np.ndarray] = None, fill_pools: bool = True,
                extra_pages: int = 3) -> StageInputs:
    """Build page tables, random pools and per-step q / k_new / v_new for a workload.

    ``growth`` decode steps fit in the mapped pages.  Sliding-window layers map only
    the pages that any of those steps can touch; earlier table entries stay -1.
    ``extra_pages`` physical pages per layer are left unreferenced by any table.
    """
    P = wl.page_size
    lens = draw_lengths(wl.lengths, wl.batch, wl.seed) if lengths is None else np.asarray(lengths, np.int32)
    B = len(lens)
    rng = np.random.default_rng(wl.seed + 7919)
    gen = torch.Generator(device=device)
    gen.manual_seed(wl.seed)
    last_page = (lens.astype(np.int64) + growth - 1) // P          # last logical page any step writes
    max_pages = int(last_page.max()) + 1
    tables, num_pages, pools = [], [], []
    for w in wl.layer_window:
        if w > 0:
            first_page = np.maximum(0, lens.astype(np.int64) + 1 - w) // P
        else:
            first_page = np.zeros(B, dtype=np.int64)
        counts = last_page - first_page + 1
        total = int(counts.sum()) + extra_pages
        perm = rng.permutation(total).astype(np.int32)
        tab = np.full((B, max_pages), -1, dtype=np.int32)
        off = 0
        for b in range(B):
            c = int(counts[b])
            tab[b, first_page[b]:first_page[b] + c] = perm[off:off + c]
            off += c
        tables.append(torch.from_numpy(tab).to(device))
        num_pages.append(total)
        pool = torch.empty(total * wl.num_kv_heads * 2 * P * wl.head_dim, dtype=torch.bfloat16, device=device)
        if fill_pools:
            _fill_normal_bf16(pool, gen)
        pools.append(pool)
    L = wl.num_layers
    q = torch.empty(steps, L, B, wl.num_q_heads, wl.head_dim, dtype=torch.bfloat16, device=device)
    k = torch.empty(steps, L, B, wl.num_kv_heads, wl.head_dim, dtype=torch.bfloat16, device=device)
    v = torch.empty_like(k)
    for t in (q, k, v):
        _fill_normal_bf16(t, gen)
    return StageInputs(wl, lens, growth, max_pages, tables, num_pages, pools, q, k, v)


def shard_rows(batch: int, rank: int, world: int) -> range:
    """Contiguous share of the batch rows owned by ``rank`` (replicas process disjoint
    subsets of the global batch; no exchange is needed between them)."""
    lo = (batch * rank) // world
    hi = (batch * (rank + 1)) // world
    return range(lo, hi)
