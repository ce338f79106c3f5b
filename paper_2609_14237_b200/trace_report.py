#!/usr/bin/env python
"""Per-phase timelines from the kernels' own trace records (global-timer stamps the kernels write when a
trace buffer is attached: `opw_attn_stage_set_trace`, `opw_afd_module_set_trace`).

    python -m paper_2609_14237_b200.trace_report attention [--workload c2_llama8b] [--steps 8]
    python -m paper_2609_14237_b200.trace_report module [--batch 64] [--hidden 4096]

`attention`: the split-KV kernel of the last of `--steps` back-to-back decode steps: when the workers
(warps) began, saw their first tile and ended, relative to the earliest begin.
`module`: the two projection launches of one attention-module step with the L2 flushed before it: per
CTA, when each phase was reached (set-up done, accumulator complete, accumulator read out, hand-off
barrier or ticket passed, partial tiles summed, end), relative to the launch's first CTA.
Tracing costs a few stores per warp or CTA; it is meant for reading timelines, not for benchmarking.
"""
from __future__ import annotations

import argparse
import dataclasses
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def _pct(a, qs=(0, 10, 50, 90, 100)):
    return "  ".join(f"p{q}={np.percentile(a, q):.1f}" for q in qs)


def attention(args):
    import torch

    from paper_2609_14237_b200 import binding as B, synth

    R = 4
    wl0 = synth.WORKLOADS[args.workload]
    wl = dataclasses.replace(wl0, layer_window=[wl0.layer_window[0]] * R)
    inp = synth.make_inputs(wl, device="cuda", growth=args.steps + 4, steps=1)
    st = B.Stage(pools=inp.pools, layer_window=wl.layer_window, num_q_heads=wl.num_q_heads, num_kv_heads=wl.num_kv_heads,
                 head_dim=wl.head_dim, max_batch=wl.batch, max_pages_per_seq=inp.max_pages_per_seq)
    out = torch.empty(wl.batch, wl.num_q_heads, wl.head_dim, dtype=torch.bfloat16, device="cuda")
    pos = torch.from_numpy(inp.positions(0)).cuda()
    q, k, v = inp.q[0], inp.k_new[0], inp.v_new[0]
    tr = st.enable_trace()
    for i in range(args.steps):
        st.decode_step(i % R, q[i % R], k[i % R], v[i % R], pos, inp.page_tables[i % R], out)
    torch.cuda.synchronize()
    assert st.poll_error() == B.OPW_OK
    t = tr.cpu().numpy()
    t = t[t[:, 1] > 0]
    t0 = t[:, 1].min()
    begin, first, end = (t[:, 1] - t0) / 1e3, (t[:, 2] - t0) / 1e3, (t[:, 3] - t0) / 1e3
    units = t[:, 0] >> 32
    print(f"{args.workload}: {len(t)} workers, {inp.kv_bytes(0, 0) / 1e6:.0f} MB of KV per step; microseconds after the earliest begin")
    print(f"  begin       {_pct(begin)}")
    print(f"  first tile  {_pct(first)}")
    print(f"  end         {_pct(end)}")
    print(f"  units per worker  {_pct(units)}")
    st.close()


def module(args):
    import torch

    from paper_2609_14237_b200 import binding as B, synth

    Bn, hidden = args.batch, args.hidden
    wl = dataclasses.replace(synth.WORKLOADS["c2_llama8b"], batch=Bn)
    inp = synth.make_inputs(wl, device="cuda", growth=16, steps=1)
    Hq, Hkv, D = wl.num_q_heads, wl.num_kv_heads, wl.head_dim
    stage = B.Stage(pools=inp.pools, layer_window=wl.layer_window, num_q_heads=Hq, num_kv_heads=Hkv, head_dim=D,
                    max_batch=Bn, max_pages_per_seq=inp.max_pages_per_seq)
    g = torch.Generator(device="cuda")
    g.manual_seed(1)
    w_qkv = (torch.randn((Hq + 2 * Hkv) * D, hidden, device="cuda", generator=g) / hidden ** 0.5).bfloat16()
    w_o = (torch.randn(hidden, Hq * D, device="cuda", generator=g) / (Hq * D) ** 0.5).bfloat16()
    x = torch.randn(Bn, hidden, device="cuda", generator=g).bfloat16()
    y = torch.empty_like(x)
    pos = torch.from_numpy(inp.lengths.astype(np.int32)).cuda()
    mod = B.AfdModule(stage, 0, w_qkv, w_o, 1e4, args.flags)
    tr = mod.enable_trace()
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    for _ in range(4):
        flush.zero_()
        mod.step(x, pos, inp.page_tables[0], y)
        pos.add_(1)
        torch.cuda.synchronize()
    assert mod.poll_error() == B.OPW_OK
    t = tr.cpu().numpy()
    names = ["begin", "set-up done", "accumulator complete", "accumulator read out", "hand-off passed", "tiles summed", "end"]
    for region, label in ((1, "QKV projection"), (0, "output projection")):
        r = t[region]
        r = r[r[:, 0] > 0]
        rel = (r[:, :7] - r[:, 0].min()) / 1e3
        print(f"batch {Bn}, {label}: {len(r)} CTAs, last CTA ends at {rel[:, 6].max():.2f} us; microseconds after the first CTA's begin")
        for i, n in enumerate(names):
            col = rel[:, i][r[:, i] >= r[:, 0].min()]          # (a CTA that skipped a phase keeps an older launch's stamp)
            if len(col):
                print(f"  {n:22s} min {col.min():7.2f}  median {np.median(col):7.2f}  max {col.max():7.2f}")
    mod.close()
    stage.close()


def main():
    ap = argparse.ArgumentParser(description=__doc__, formatter_class=argparse.RawDescriptionHelpFormatter)
    sub = ap.add_subparsers(dest="what", required=True)
    a = sub.add_parser("attention")
    a.add_argument("--workload", default="c2_llama8b")
    a.add_argument("--steps", type=int, default=8)
    m = sub.add_parser("module")
    m.add_argument("--batch", type=int, default=64)
    m.add_argument("--hidden", type=int, default=4096)
    m.add_argument("--flags", type=int, default=0, help="OPW_AFD_* flags of the module (4: no clusters)")
    args = ap.parse_args()
    import torch

    from paper_2609_14237_b200 import binding

    if not torch.cuda.is_available():
        raise SystemExit("trace_report needs a CUDA device")
    binding.build()
    torch.cuda.set_device(0)
    (attention if args.what == "attention" else module)(args)


if __name__ == "__main__":
    main()
