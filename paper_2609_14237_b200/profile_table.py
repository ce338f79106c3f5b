#!/usr/bin/env python
"""Profile table of the attention stage: latency and effective bandwidth over (batch, context
length, window), the operator profile a serving planner consumes for attention stages
(paper, Section 4: stage latencies come from "profiled execution latency").

    python -m paper_2609_14237_b200.profile_table [--out attn_profile.json]

Every point runs the fused decode step (append + attention + combine) through a plan (CUDA
graph, metadata advanced on the device) over enough identical layers that consecutive reads
of one pool are at least 1 GB apart (so the 126 MB L2 cannot serve them), and reports the time
per layer-step, the algorithmic KV bytes and their ratio beta_eff.  `costmodel.attention_latency`
with beta = beta_eff reproduces the measured time by construction; the table shows how far the
"KV bytes / bandwidth" model with a single beta is from the stage at small sizes.
"""
from __future__ import annotations

import argparse
import dataclasses
import json
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def measure_point(batch, seq_len, window, Hq=32, Hkv=8, D=128, submits=30, rounds=3):
    import torch

    from paper_2609_14237_b200 import binding, synth

    kvb = 2 * Hkv * D * 2
    visible = min(seq_len, window) if window else seq_len
    per_layer = batch * visible * kvb
    layers = int(min(16, max(2, -(-(1 << 30) // max(per_layer, 1)))))
    wl = synth.Workload("profile", batch, Hq, Hkv, D, [window] * layers, f"const_{seq_len}", 4242)
    inp = synth.make_inputs(wl, device="cuda", growth=rounds * submits + 8, steps=1)
    st = binding.Stage(pools=inp.pools, layer_window=wl.layer_window, num_q_heads=Hq, num_kv_heads=Hkv, head_dim=D,
                       max_batch=batch, max_pages_per_seq=inp.max_pages_per_seq)
    pos = torch.from_numpy(inp.positions(0)).cuda()
    out = torch.empty(batch, Hq, D, dtype=torch.bfloat16, device="cuda")
    items = [dict(layer=l, batch=batch, q=inp.q[0, l].data_ptr(), k_new=inp.k_new[0, l].data_ptr(),
                  v_new=inp.v_new[0, l].data_ptr(), positions=pos.data_ptr(), page_table=inp.page_tables[l].data_ptr(),
                  out=out.data_ptr()) for l in range(layers)]
    plan = binding.opw_attn_plan_create(st.handle, items, binding.OPW_PLAN_GRAPH | binding.OPW_PLAN_ADVANCE)
    stream = torch.cuda.current_stream()
    for _ in range(3):
        binding.opw_attn_plan_submit(plan, stream.cuda_stream)
    torch.cuda.synchronize()
    # the fastest of `rounds` timed rounds: a point measured right after a much larger one (its pools just
    # freed, the clocks still settling) can read several per cent slow in a single round
    times = []
    for _ in range(rounds):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(submits):
            binding.opw_attn_plan_submit(plan, stream.cuda_stream)
        e1.record(stream)
        torch.cuda.synchronize()
        times.append(e0.elapsed_time(e1) * 1e3 / (submits * layers))
    assert st.poll_error() == binding.OPW_OK
    t_us = min(times)
    first = 4 + submits * times.index(t_us)                # tokens appended before the fastest round began
    tokens = sum(min(seq_len + first + i, window) if window else seq_len + first + i for i in range(submits)) / submits
    nbytes = batch * tokens * kvb
    binding.opw_attn_plan_destroy(plan)
    st.close()
    del inp
    torch.cuda.empty_cache()
    return {"batch": batch, "seq_len": seq_len, "window": window, "layers": layers, "t_us": round(t_us, 2),
            "t_us_median": round(float(np.median(times)), 2),
            "kv_bytes": int(nbytes), "beta_eff_gbs": round(nbytes / (t_us * 1e-6) / 1e9, 1)}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--out", default="attn_profile.json")
    ap.add_argument("--batches", default="1,4,16,64,256")
    ap.add_argument("--seq-lens", default="1024,4096,16384,65536")
    ap.add_argument("--windows", default="0,4096")
    ap.add_argument("--max-gb", type=float, default=40.0, help="skip points whose pools would exceed this")
    args = ap.parse_args()
    import torch

    from paper_2609_14237_b200 import binding

    if not torch.cuda.is_available():
        raise SystemExit("profile_table needs a CUDA device")
    binding.build()
    rows = []
    for w in (int(x) for x in args.windows.split(",")):
        for s in (int(x) for x in args.seq_lens.split(",")):
            if w and s <= w:
                continue                                   # identical to the full-attention point
            for b in (int(x) for x in args.batches.split(",")):
                visible = min(s, w) if w else s
                per_layer = b * (visible + 64) * 4096
                layers = int(min(16, max(2, -(-(1 << 30) // per_layer))))
                if per_layer * layers / 1e9 > args.max_gb:
                    continue
                r = measure_point(b, s, w)
                rows.append(r)
                print(json.dumps(r), flush=True)
    if os.path.dirname(args.out):
        os.makedirs(os.path.dirname(args.out), exist_ok=True)
    # the two-parameter latency model of the stage: a floor plus bytes over bandwidth, fitted to the table
    from paper_2609_14237_b200 import costmodel

    t0_s, beta = costmodel.fit_affine_latency([(r["kv_bytes"], r["t_us"] * 1e-6) for r in rows])
    worst = max(abs(costmodel.attention_latency_affine(1, r["kv_bytes"], t0_s, beta) / (r["t_us"] * 1e-6) - 1) for r in rows)
    fit = {"t0_us": round(t0_s * 1e6, 2), "beta_gbs": round(beta / 1e9, 1), "max_rel_error": round(worst, 4),
           "model": "t = t0 + kv_bytes / beta, relative least squares"}
    print(json.dumps({"fit": fit}), flush=True)
    with open(args.out, "w") as fh:
        json.dump({"shape": {"num_q_heads": 32, "num_kv_heads": 8, "head_dim": 128, "page_size": 16}, "points": rows,
                   "fit": fit}, fh, indent=1)


if __name__ == "__main__":
    main()
