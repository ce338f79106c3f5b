"""Host-side pieces of the benchmark that need no GPU: the tracked traffic ratios and how
`roofline.traffic` is derived from them."""
import json
import os
import types

import numpy as np

import bench
from paper_2609_14237_b200 import synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_traffic_ratios_file_names_a_capture_for_every_benchmark_workload():
    table = json.load(open(os.path.join(ROOT, "profiles", "traffic_ratios.json")))
    caps = table["captures"]
    for name in ("c2_llama8b", "c3_long_context", "c4_large_batch", "c5_hybrid_stack", "c5_window_layer"):
        kinds = table["workloads"][name]
        for key in ("full_layers", "window_layers"):
            cap = caps[kinds[key]]
            assert 1.0 <= cap["ratio"] < 1.05                       # traffic well above the algorithmic bytes would mean re-reads
            assert os.path.exists(os.path.join(ROOT, cap["summary"]))
            assert "--clock-control none" in cap["command"] and "ncu" in cap["command"]
            assert cap["launches"]


def test_derived_traffic_weights_each_layer_by_the_ratio_of_its_kind():
    wl = synth.WORKLOADS["c5_hybrid_stack"]
    table = json.load(open(os.path.join(ROOT, "profiles", "traffic_ratios.json")))
    r_win = table["captures"][table["workloads"][wl.name]["window_layers"]]["ratio"]
    r_full = table["captures"][table["workloads"][wl.name]["full_layers"]]["ratio"]
    fake = types.SimpleNamespace(kv_bytes=lambda l, t: 100_000 if wl.layer_window[l] > 0 else 900_000)
    traffic, source = bench.derived_traffic(wl.name, wl, fake, list(range(8)), None, 0)
    want = (6 * r_win * 100_000 + 2 * r_full * 900_000) / 8
    assert abs(traffic - want) <= 1 and "window_layer" in source and "full_long_rows" in source
    assert bench.derived_traffic("c1_tiny", synth.WORKLOADS["c1_tiny"], fake, [0], None, 0) == (None, None)


def test_compact_rows_renumbers_pages_and_keeps_their_bytes():
    import torch

    page_elems = 8
    pool = torch.arange(10 * page_elems, dtype=torch.int16)
    table = torch.tensor([[7, 2, -1], [5, -1, -1], [2, 9, 0]], dtype=torch.int32)
    small, tab = bench.compact_rows(pool, table, [0, 2], page_elems)
    used = [0, 2, 7, 9]                                             # pages rows 0 and 2 reference, ascending
    assert small.numel() == len(used) * page_elems
    for new, old in enumerate(used):
        assert (small.view(-1, page_elems)[new] == pool.view(-1, page_elems)[old]).all()
    assert tab.tolist() == [[2, 1, -1], [1, 3, 0]]
