#!/usr/bin/env python
"""Benchmark of the decode attention stage: KV GB/s and sequence-steps/s per layer.

A "step" is one pass of the whole hot path over one batch: for every layer the stage
owns, the paged KV append of this step's token followed by split-KV attention and the
log-sum-exp combine.  The headline ``value`` is algorithmic KV bytes (the K and V rows the
step must read: sum over sequences of visible tokens x 2*Hkv*D*2 bytes) divided by the
step time, with all inputs resident in HBM.  ``e2e`` is the same metric through
``opw_decode_step_host`` with pinned HOST buffers: the per-step copies of q, k_new,
v_new, positions and the page table to the device and of the output back are inside the
timed region and every step ends with a stream synchronisation.  ``e2e_two_microbatches`` is the
same loop with two microbatches in flight on two streams (copies of one hide behind the other's kernels).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

For N > 1 launch with torchrun (one rank per GPU); every rank runs an independent replica
of the workload (the stage shards by sequence with no exchange), the time is the max over
ranks and the value the sum of all ranks' bytes over that time.
"""
from __future__ import annotations

import argparse
import dataclasses
import json
import os
import sys
import threading
import time

# torchrun gives every rank one OpenMP thread unless the variable is set, which suits N ranks sharing the
# host; the reference arm runs the CPU oracle on rank 0 alone (the other ranks exit), so it gets the cores
# this process may use.  Set before anything loads an OpenMP runtime.
if ("reference" in sys.argv and "TORCHELASTIC_RUN_ID" in os.environ and os.environ.get("OMP_NUM_THREADS") == "1"
        and hasattr(os, "sched_getaffinity")):
    os.environ["OMP_NUM_THREADS"] = str(len(os.sched_getaffinity(0)))

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "decode attn-stage KV GB/s"
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0
DEFAULT_WORKLOAD = "c3_long_context"
# DRAM traffic of the split-KV kernel relative to its algorithmic KV bytes comes from the ncu captures
# summarised under profiles/ (dram__bytes_read.sum + dram__bytes_write.sum per launch / algorithmic
# bytes): profiles/traffic_ratios.json lists, per kind of launch, the ratio and the capture it was read from.
PARITY_MAX_ABS, PARITY_MEAN_ABS = 1e-2, 1e-3      # the stated tolerance of the attention output
EVENT_EVERY = 4                                   # one step in four is timed call by call with CUDA events


def traffic_ratios():
    try:
        with open(os.path.join(ROOT, "profiles", "traffic_ratios.json")) as fh:
            return json.load(fh)
    except Exception:
        return {}


def derived_traffic(name, wl, inp, layers, attn_bytes_per_launch, t):
    """roofline.traffic of one launch: algorithmic bytes x the captured traffic ratio of that kind of launch
    (for a stack: the mean over its layers, each layer with the ratio of its kind)."""
    table = traffic_ratios()
    wmap = table.get("workloads", {}).get(name)
    if wmap is None:
        return None, None
    caps = table.get("captures", {})
    total, used = 0.0, []
    for l in layers:
        key = wmap["window_layers" if wl.layer_window[l % len(wl.layer_window)] > 0 else "full_layers"]
        if key not in caps:
            return None, None
        total += caps[key]["ratio"] * inp.kv_bytes(l, t)
        if key not in used:
            used.append(key)
    return int(total / len(layers)), "derived: algorithmic bytes x ratio of capture(s) " + ", ".join(
        f"{k} ({caps[k]['ratio']}, {caps[k]['summary']})" for k in used)


def measured_peak():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as fh:
            return float(json.load(fh)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons through NVML while the timed region runs."""

    def __init__(self, torch_index: int, period: float = 0.02):
        super().__init__(daemon=True)
        self.period, self.samples, self.reasons, self.stop_flag = period, [], set(), False
        self.max_mhz, self.ok = None, False
        try:
            import pynvml
            import torch

            pynvml.nvmlInit()
            uuid = str(torch.cuda.get_device_properties(torch_index).uuid)
            if not uuid.startswith("GPU-"):
                uuid = "GPU-" + uuid
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByUUID(uuid.encode() if hasattr(uuid, "encode") else uuid)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
            self.ok = True
        except Exception as e:                                   # noqa: BLE001
            self.err = repr(e)

    def sample(self):
        """One reading of the SM clock and the throttle reasons."""
        if not self.ok:
            return
        nv = self.nv
        names = {
            getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8): "hw_slowdown",
            getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40): "hw_thermal_slowdown",
            getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20): "sw_thermal_slowdown",
            getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4): "sw_power_cap",
        }
        try:
            self.samples.append(int(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)))
            try:
                mask = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self.h))
            except Exception:                                    # noqa: BLE001
                mask = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
            for bit, name in names.items():
                if mask & bit:
                    self.reasons.add(name)
        except Exception:                                        # noqa: BLE001
            pass

    def run(self):
        while self.ok and not self.stop_flag:
            self.sample()
            time.sleep(self.period)

    def result(self):
        self.stop_flag = True
        if self.is_alive():
            self.join(timeout=2)
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": [], "samples": 0}
        return {"sm_mhz": int(np.median(self.samples)), "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(self.samples)}


def measure_read_ceiling(gib=4, passes=10):
    """Read-only streaming rate of this GPU in this run: the library's read probe (16-byte evict-first
    loads, every word once) over a buffer far larger than L2, CUDA events, best of `passes`."""
    import torch

    from paper_2609_14237_b200 import binding

    free = torch.cuda.mem_get_info()[0]
    nbytes = min(gib << 30, (free // 4) & ~0xFFFFF)
    if nbytes < (1 << 30):
        return None
    buf = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    buf.fill_(1)
    sink = torch.zeros(4096, dtype=torch.float32, device="cuda")
    stream = torch.cuda.current_stream()
    best = None
    for i in range(passes + 2):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        binding.opw_hbm_read_probe(buf.data_ptr(), nbytes, sink.data_ptr(), stream.cuda_stream)
        e1.record(stream)
        torch.cuda.synchronize()
        if i >= 2:
            ms = e0.elapsed_time(e1)
            best = ms if best is None else min(best, ms)
    del buf
    torch.cuda.empty_cache()
    return {"value": round(nbytes / (best * 1e-3) / 1e9, 1), "unit": "GB/s", "bytes": int(nbytes), "passes": passes,
            "kernel": "read_probe_kernel (opw_hbm_read_probe), best pass"}


def compact_rows(pool, table, rows, page_elems):
    """Copies the pages the given rows reference into a small pool with a renumbered table (data movement only)."""
    import torch

    pv = pool.view(-1, page_elems)
    sub = table[rows].clone()
    used = torch.unique(sub[sub >= 0])
    remap = torch.full((pv.shape[0],), -1, dtype=torch.int32, device=pool.device)
    remap[used.long()] = torch.arange(used.numel(), dtype=torch.int32, device=pool.device)
    small = pv[used.long()].contiguous().view(-1)
    new_tab = torch.where(sub >= 0, remap[sub.clamp(min=0).long()], torch.full_like(sub, -1))
    return small.cpu(), new_tab.cpu().numpy()


def parity_before_timing(wl_r, inp, st, pos_all, layers, out, unfused, all_rows):
    """Step 0 of the configuration about to be timed (same stage, pools, tuning and call), compared with the
    CPU oracle on the same inputs: the appended cache bytes bit for bit, the attention output element by
    element.  Runs outside every timed region.  all_rows=False compares a seeded sample of rows (always the
    shortest and the longest) where the whole batch would take the oracle minutes."""
    import torch

    import oracle

    Hq, Hkv, D, P = wl_r.num_q_heads, wl_r.num_kv_heads, wl_r.head_dim, 16
    pe = Hkv * 2 * P * D
    pos, n = inp.positions(0), inp.kv_lens(0)
    order = np.argsort(n, kind="stable")
    Bn = len(n)
    worst_abs, sum_abs, count, worst_lse, rows_total, bitwise = 0.0, 0.0, 0, 0.0, 0, True
    lse = torch.empty(Bn, Hq, dtype=torch.float32, device=out.device)
    stream_pos = pos_all[0]
    for l in layers:
        w = wl_r.layer_window[l]
        budget = 0.7e9 if not all_rows else float("inf")          # bytes of KV the oracle is given per layer
        rows, acc = [], 0
        for r in [int(order[0]), int(order[-1])] + [int(x) for x in np.random.default_rng(7 + l).permutation(Bn)]:
            vis = min(int(n[r]), w) if w > 0 else int(n[r])
            if r in rows or (len(rows) >= 2 and acc + vis * wl_r.kv_bytes_per_token > budget):
                continue
            rows.append(r)
            acc += vis * wl_r.kv_bytes_per_token
        rows = sorted(rows)
        before, small_tab = compact_rows(inp.pools[l], inp.page_tables[l], rows, pe)
        q, k, v = inp.q[0, l], inp.k_new[0, l], inp.v_new[0, l]
        out.fill_(float("nan"))
        if unfused:
            st.kv_append(l, k, v, stream_pos, inp.page_tables[l])
            st.decode_attention(l, q, torch.from_numpy(n).to(out.device), inp.page_tables[l], out, lse)
        else:
            st.decode_step(l, q, k, v, stream_pos, inp.page_tables[l], out, lse)
        torch.cuda.synchronize()
        ref_pool = oracle.as_u16(before).copy()
        assert oracle.kv_append(ref_pool, Hkv, D, P, k[rows].cpu(), v[rows].cpu(), pos[rows], small_tab) == 0
        after, _ = compact_rows(inp.pools[l], inp.page_tables[l], rows, pe)
        bitwise = bitwise and bool(np.array_equal(oracle.as_u16(after), ref_pool))
        ref, ref_lse, rc = oracle.decode_attention(ref_pool, Hq, Hkv, D, P, q[rows].cpu(), n[rows], small_tab, window=w)
        assert rc == 0
        got = oracle.bf16_bits_to_f64(oracle.as_u16(out[rows].cpu()))
        err = np.abs(got - ref)
        if not np.isfinite(got).all():
            worst_abs = float("inf")
        worst_abs = max(worst_abs, float(err.max()))
        sum_abs += float(err.sum())
        count += err.size
        worst_lse = max(worst_lse, float(np.abs(lse[rows].cpu().numpy().astype(np.float64) - ref_lse).max()))
        rows_total += len(rows)
    res = {"max_abs": worst_abs, "mean_abs": sum_abs / max(count, 1), "lse_max_abs": worst_lse, "rows": rows_total,
           "rows_per_layer_step": rows_total // len(layers), "of_rows": Bn, "layers": len(layers), "pool_bitwise": bitwise,
           "tolerance": {"max_abs": PARITY_MAX_ABS, "mean_abs": PARITY_MEAN_ABS},
           "what": "step 0 of the timed configuration against the CPU oracle, before timing"}
    res["ok"] = bool(bitwise and worst_abs <= PARITY_MAX_ABS and res["mean_abs"] <= PARITY_MEAN_ABS)
    return res


def build_stage(wl, rotate, total_rounds, device, tune):
    """R identical copies of a one-layer workload (or the workload's own layer stack)."""
    import torch

    from paper_2609_14237_b200 import binding, synth

    if wl.num_layers == 1 and rotate > 1:
        wl_r = dataclasses.replace(wl, layer_window=list(wl.layer_window) * rotate)
    else:
        wl_r = wl
    inp = synth.make_inputs(wl_r, device=device, growth=total_rounds + 1, steps=2)
    st = binding.Stage(pools=inp.pools, layer_window=wl_r.layer_window, num_q_heads=wl.num_q_heads,
                       num_kv_heads=wl.num_kv_heads, head_dim=wl.head_dim, max_batch=wl.batch,
                       max_pages_per_seq=inp.max_pages_per_seq, **tune)
    rounds = total_rounds + 1
    pos_all = torch.from_numpy(np.stack([inp.positions(t) for t in range(rounds)])).to(device)
    len_all = torch.from_numpy(np.stack([inp.kv_lens(t) for t in range(rounds)])).to(device)
    return wl_r, inp, st, pos_all, len_all


def run_ours(name, steps, warmup, rotate, tune, want_e2e=True, want_cpu=False, world=1, rank=0, want_submit=False,
             unfused=False, want_parity=True):
    import torch

    from paper_2609_14237_b200 import binding, synth

    dev = torch.device("cuda", torch.cuda.current_device())
    wl = synth.WORKLOADS[name]
    stack = wl.num_layers > 1                       # the hybrid stack: a step runs all its layers
    R = wl.num_layers if stack else rotate
    e2e_steps = max(3, min(steps, 200)) if want_e2e else 0
    n_timed = warmup + steps + (e2e_steps + max(3, rotate) if want_e2e else 0)
    n_used = n_timed                                 # steps the call-by-call and host-buffer loops take
    # a plan submission advances every layer by one token; two plans run, each 3 warm-up submissions + n_sub timed
    n_sub = (steps if stack else max(steps // R, 10)) if want_submit else 0
    if want_e2e and world == 1 and not stack and R >= 2:
        n_used += e2e_steps + 2 * R + 8              # the two-microbatch host-buffer loop
    rounds = (n_used if stack else (n_used + R - 1) // R) + (2 * (3 + n_sub) + 2 if want_submit else 0)
    wl_r, inp, st, pos_all, len_all = build_stage(wl, R, rounds, dev, tune)
    B, Hq, Hkv, D = wl.batch, wl.num_q_heads, wl.num_kv_heads, wl.head_dim
    out = torch.empty(B, Hq, D, dtype=torch.bfloat16, device=dev)
    stream = torch.cuda.current_stream()

    def layer_round(s):                             # which layers step s runs, and at which length
        return (list(range(R)), s) if stack else ([s % R], s // R)

    def kv_bytes_of_step(s):
        layers, t = layer_round(s)
        return sum(inp.kv_bytes(l, t) for l in layers)

    def device_step(s, events=None):
        layers, t = layer_round(s)
        for l in layers:
            if events is not None:
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            if unfused:
                st.kv_append(l, inp.k_new[s & 1, l], inp.v_new[s & 1, l], pos_all[t], inp.page_tables[l])
                if events is not None:
                    e0.record(stream)
                st.decode_attention(l, inp.q[s & 1, l], len_all[t], inp.page_tables[l], out)
            else:                                   # append fused into the attention kernel: two launches
                if events is not None:
                    e0.record(stream)
                st.decode_step(l, inp.q[s & 1, l], inp.k_new[s & 1, l], inp.v_new[s & 1, l], pos_all[t],
                               inp.page_tables[l], out)
            if events is not None:
                e1.record(stream)
                events.append((e0, e1, inp.kv_bytes(l, t)))

    def barrier():
        if world > 1:
            import torch.distributed as dist

            dist.barrier()

    parity = None
    if want_parity:
        # whole batch where the oracle finishes in seconds; a sample for the 52 GB stack and under torchrun
        # (there every rank has one host thread)
        parity = parity_before_timing(wl_r, inp, st, pos_all, layer_round(0)[0], out, unfused,
                                      all_rows=(not stack and world == 1))
        if not parity["ok"] or st.poll_error() != binding.OPW_OK:
            print(json.dumps({"error": "parity check failed before timing", "workload": name, "parity": parity}), flush=True)
            raise SystemExit(1)
    for s in range(warmup):
        device_step(s)
    torch.cuda.synchronize()
    assert st.poll_error() == binding.OPW_OK
    barrier()
    sampler = ClockSampler(dev.index)
    sampler.start()
    launches0 = st.launch_count()
    ev = []
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    t0.record(stream)
    for s in range(warmup, warmup + steps):
        device_step(s, ev if (s - warmup) % EVENT_EVERY == 0 else None)
    t1.record(stream)
    sampler.sample()                                # at least one reading while the GPU is still busy
    torch.cuda.synchronize()
    barrier()
    clocks = sampler.result()
    launches = st.launch_count() - launches0
    total_ms = t0.elapsed_time(t1)
    attn_ms = [a.elapsed_time(b) for a, b, _ in ev]
    assert st.poll_error() == binding.OPW_OK
    bytes_timed = sum(kv_bytes_of_step(s) for s in range(warmup, warmup + steps))
    layers_per_step = len(layer_round(0)[0])
    attn_bytes_per_launch = float(np.mean([nb for _, _, nb in ev]))        # of the launches that were timed one by one

    if world > 1:
        import torch.distributed as dist

        tmax = torch.tensor([total_ms], dtype=torch.float64, device=dev if dist.get_backend() == "nccl" else "cpu")
        dist.all_reduce(tmax, op=dist.ReduceOp.MAX)
        total_ms = float(tmax.item())
    value = world * bytes_timed / (total_ms * 1e-3) / 1e9
    peak, peak_kind = measured_peak()
    attn_avg_ms = float(np.mean(attn_ms))
    achieved = attn_bytes_per_launch / (attn_avg_ms * 1e-3) / 1e9
    traffic, traffic_source = derived_traffic(name, wl_r, inp, layer_round(warmup)[0], attn_bytes_per_launch,
                                              layer_round(warmup + steps // 2)[1])
    step_ms = [sum(attn_ms[i * layers_per_step:(i + 1) * layers_per_step]) for i in range(len(attn_ms) // layers_per_step)]
    res = {
        "metric": METRIC, "value": round(value, 1), "unit": "GB/s", "n_gpus": world, "steps": steps, "warmup": warmup,
        "ms_per_step": round(total_ms / steps, 5), "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": {"workload": name, "batch": B, "num_q_heads": Hq, "num_kv_heads": Hkv, "head_dim": D, "page_size": 16,
                   "layers_per_step": layers_per_step, "layer_window": list(wl.layer_window),
                   "mean_context": float(np.mean(inp.lengths)),
                   "kv_bytes_per_step": int(bytes_timed // steps),
                   "l2": (f"inputs larger than L2: {'the stack of' if stack else 'rotating over'} {R} layer pools, "
                          f"{sum(inp.kv_bytes(l, 0) for l in range(R)) / 1e9:.2f} GB of KV between re-reads"),
                   "parallelism": f"replicas x{world}" if world > 1 else "1 gpu"},
        "seq_steps_per_s_per_layer": round(world * B * layers_per_step / (total_ms / steps * 1e-3), 1),
        "pct_of_nominal_8000": round(100 * value / world / NOMINAL_HBM_GBS, 2),
        "roofline": {"bound": "hbm", "achieved": round(achieved, 1), "peak": peak, "unit": "GB/s",
                     "frac": round(achieved / peak, 4), "peak_kind": peak_kind,
                     "kernel": ("attn_splitkv_kernel (+ combine_kernel, timed together per opw_decode_attention call)"
                                if unfused else
                                "attn_splitkv_kernel with fused append (+ combine_kernel, timed together per opw_decode_step call)"),
                     "kernel_ms": round(attn_avg_ms, 5), "kernel_ms_median": round(float(np.median(attn_ms)), 5),
                     "kernel_ms_min": round(float(np.min(attn_ms)), 5),
                     "kernel_ms_from": f"{len(attn_ms)} calls of the timed region, each between two CUDA events (every "
                                       f"{EVENT_EVERY}th step; the other steps run back to back, as in serving)",
                     "traffic": traffic, "traffic_source": traffic_source,
                     "note": "peak is a read+write copy rate; this kernel only reads, so frac may pass 1: see frac_of_read_ceiling"},
        "step_ms": {"mean": round(float(np.mean(step_ms)), 5), "median": round(float(np.median(step_ms)), 5),
                    "min": round(float(np.min(step_ms)), 5),
                    "what": "per sampled step, sum of its calls' CUDA-event durations (gaps between calls excluded)"},
        "gpu_launches": int(launches), "clocks": clocks,
    }
    if parity is not None:
        res["parity"] = parity

    if want_e2e:
        # q, k_new, v_new and positions of one call sit in one pinned buffer at the stage's packed
        # offsets (they travel as one copy); the output has a pinned buffer of its own.  The page table is
        # handled as a server would: sent in full when a sequence set is admitted to a layer (with nothing
        # mapped beyond the page the next token goes to; that happens in the untimed warm-up), and after that
        # only the (row, logical page, physical page) triple of every sequence whose new token opens a page.
        packs = [[st.packed_host_buffers(B) for _ in range(R)] for _ in range(2)]
        for i in range(2):
            for l in range(R):
                _, pq, pk, pv, _ = packs[i][l]
                pq.copy_(inp.q[i, l].cpu())
                pk.copy_(inp.k_new[i, l].cpu())
                pv.copy_(inp.v_new[i, l].cpu())
        hpos = pos_all.cpu()
        hpos_np = hpos.numpy()
        pos_views = {}                                 # numpy views of the packed buffers' position fields (a 64-byte host write per step)

        def write_positions(ppos, t):
            v = pos_views.get(ppos.data_ptr())
            if v is None:
                v = pos_views[ppos.data_ptr()] = ppos.numpy()
            v[:] = hpos_np[t]

        full_tab = [t.cpu().numpy() for t in inp.page_tables]
        hout = torch.empty(B, Hq, D, dtype=torch.bfloat16).pin_memory()
        base = warmup + steps
        keep_alive = []                                # pinned tables and triples of copies that may still be in flight

        def admission_table(l, t):
            tab = full_tab[l].copy()
            beyond = np.arange(tab.shape[1])[None, :] > (hpos_np[t].astype(np.int64) // 16)[:, None]
            tab[beyond] = -1
            ten = torch.from_numpy(tab).pin_memory()
            keep_alive.append(ten)
            return ten

        deltas = {}                                    # (layer, round) -> pinned int32 [n, 3], for rounds whose token opens a page

        def delta_of(l, t):
            key = (l, t)
            if key not in deltas:
                rows = np.nonzero(hpos_np[t] % 16 == 0)[0]
                if len(rows) == 0:
                    deltas[key] = None
                else:
                    lp = hpos_np[t][rows].astype(np.int64) // 16
                    tri = np.stack([rows, lp, full_tab[l][rows, lp]], axis=1).astype(np.int32)
                    deltas[key] = torch.from_numpy(tri).pin_memory()
            return deltas[key]

        for l in range(R):                             # built before any timed region
            for t in range(pos_all.shape[0]):
                delta_of(l, t)
        admitted = {}                                  # stage handle -> layers whose table it holds
        delta_bytes = [0]

        def send_table(stage, l, t):
            """The page_table_host argument of this visit, after any delta call it needs."""
            seen = admitted.setdefault(id(stage), set())
            if l not in seen:
                seen.add(l)
                return admission_table(l, t)
            tri = delta_of(l, t)
            if tri is not None:
                stage.page_table_delta_host(l, tri)
                delta_bytes[0] += tri.numel() * 4
            return None

        # The C entry point is called with addresses looked up once (a serving loop binds its buffers once, too):
        # what is left per step on the host is the positions write, the table delta if any, and one native call.
        step_host = binding.lib().opw_decode_step_host
        stream_ptr = stream.cuda_stream
        hout_ptr = hout.data_ptr()
        call_args = {}

        def args_of(stage, pack, l):
            key = (id(stage), pack[0].data_ptr(), l)
            a = call_args.get(key)
            if a is None:
                _, pq, pk, pv, ppos = pack
                a = call_args[key] = (stage.handle, l, B, pq.data_ptr(), pk.data_ptr(), pv.data_ptr(), ppos.data_ptr())
            return a

        def host_step(s):
            layers, t = layer_round(s)
            for l in layers:
                pack = packs[s & 1][l]
                write_positions(pack[4], t)          # this step's positions, written by the host
                tab = send_table(st, l, t)
                rc = step_host(*args_of(st, pack, l), None if tab is None else tab.data_ptr(), hout_ptr, None, stream_ptr)
                if rc != binding.OPW_OK:
                    raise binding.OpwError(rc, "opw_decode_step_host")
            stream.synchronize()                     # the caller reads the result every step

        warm = max(3, 1 if stack else R)             # every layer is admitted (its table sent in full) before timing
        for s in range(base, base + warm):
            host_step(s)
        barrier()
        torch.cuda.synchronize()
        delta_bytes[0] = 0
        w0 = time.perf_counter()
        t0.record(stream)
        for s in range(base + warm, base + warm + e2e_steps):
            host_step(s)
        t1.record(stream)
        torch.cuda.synchronize()
        wall_ms = (time.perf_counter() - w0) * 1e3
        e_ms = max(t0.elapsed_time(t1), wall_ms)
        if world > 1:
            import torch.distributed as dist

            tmax = torch.tensor([e_ms], dtype=torch.float64, device=dev if dist.get_backend() == "nccl" else "cpu")
            dist.all_reduce(tmax, op=dist.ReduceOp.MAX)
            e_ms = float(tmax.item())
        e_bytes = sum(kv_bytes_of_step(s) for s in range(base + warm, base + warm + e2e_steps))
        packed = layers_per_step * (B * Hq * D * 2 + 2 * B * Hkv * D * 2 + B * 4)
        h2d = packed + delta_bytes[0] / e2e_steps
        d2h = layers_per_step * hout.numel() * 2
        assert st.poll_error() == binding.OPW_OK
        table_note = ("sent in full at admission (untimed warm-up); inside the timed region 12 bytes per page a sequence opens, "
                      f"{delta_bytes[0] / e2e_steps:.1f} bytes per step on average")
        res["e2e"] = {"value": round(world * e_bytes / (e_ms * 1e-3) / 1e9, 1), "unit": "GB/s", "steps": e2e_steps,
                      "ms_per_step": round(e_ms / e2e_steps, 5), "h2d_bytes_per_step": int(round(h2d)),
                      "d2h_bytes_per_step": int(d2h), "page_table": table_note,
                      "frac_of_value": round(world * e_bytes / (e_ms * 1e-3) / 1e9 / value, 4)}
    if want_e2e and world == 1 and not stack and R >= 2:
        # The same host-buffer steps with two microbatches in flight (the paper keeps mu microbatches resident
        # on a stage so that transfers hide behind compute): even steps belong to microbatch A, odd steps to B,
        # each with a stage handle of its own (workspace, staged tables) created with OPW_FLAG_COPY_STREAMS, over
        # disjoint layer pools.  Both enqueue their kernels on ONE compute stream; each handle's copies run on its own
        # streams beside the other microbatch's kernels.  Every step still copies its inputs in and its output out;
        # the host waits for a microbatch's previous result (opw_attn_stage_wait_host_output) before it reuses that
        # microbatch's buffers.
        Re = R - R % 2                                        # an even number of pools: half for each microbatch
        flags2 = tune.get("flags", 0) | binding.OPW_FLAG_COPY_STREAMS
        tune2 = dict(tune, flags=flags2)
        mb_stages = [binding.Stage(pools=inp.pools, layer_window=wl_r.layer_window, num_q_heads=Hq, num_kv_heads=Hkv,
                                   head_dim=D, max_batch=B, max_pages_per_seq=inp.max_pages_per_seq, **tune2) for _ in range(2)]
        packs2 = [[mb_stages[l & 1].packed_host_buffers(B) for l in range(R)] for _ in range(2)]
        for i in range(2):
            for l in range(R):
                _, pq, pk, pv, _ = packs2[i][l]
                pq.copy_(inp.q[i, l].cpu())
                pk.copy_(inp.k_new[i, l].cpu())
                pv.copy_(inp.v_new[i, l].cpu())
        houts = [torch.empty(B, Hq, D, dtype=torch.bfloat16).pin_memory() for _ in range(2)]
        compute = torch.cuda.Stream()
        # This loop has its own step numbering: step s2 visits pool s2 % Re at round r0 + s2 // Re, r0 the first round
        # no pool has been appended at yet; an even pool belongs to microbatch A, an odd one to B.
        r0 = (base + warm + e2e_steps + R - 1) // R
        admitted.clear()                                      # rounds were skipped: both handles take their tables afresh
        wait_out = binding.lib().opw_attn_stage_wait_host_output

        def host_step_mb(s2):
            l, t = s2 % Re, r0 + s2 // Re
            mb = l & 1
            stage = mb_stages[mb]
            wait_out(stage.handle)                            # this microbatch's previous result is on the host now
            with torch.cuda.stream(compute):
                pack = packs2[(s2 >> 1) & 1][l]
                write_positions(pack[4], t)
                tab = send_table(stage, l, t)
                rc = step_host(*args_of(stage, pack, l), None if tab is None else tab.data_ptr(), houts[mb].data_ptr(), None,
                               compute.cuda_stream)
                if rc != binding.OPW_OK:
                    raise binding.OpwError(rc, "opw_decode_step_host")
            return inp.kv_bytes(l, t)

        warm2 = max(4, Re)
        n2 = min(e2e_steps, ((pos_all.shape[0] - 1 - r0) * Re - warm2) // 2 * 2)
        if n2 >= 4:
            for s2 in range(warm2):
                host_step_mb(s2)
            torch.cuda.synchronize()
            delta_bytes[0] = 0
            mb_bytes = 0
            w0 = time.perf_counter()
            for s2 in range(warm2, warm2 + n2):
                mb_bytes += host_step_mb(s2)
            for stg in mb_stages:
                stg.wait_host_output()
            torch.cuda.synchronize()
            mb_ms = (time.perf_counter() - w0) * 1e3
            assert all(stg.poll_error() == binding.OPW_OK for stg in mb_stages)
            v2 = mb_bytes / (mb_ms * 1e-3) / 1e9
            res["e2e_two_microbatches"] = {"value": round(v2, 1), "unit": "GB/s", "steps": n2,
                                           "ms_per_step": round(mb_ms / n2, 5), "timing": "wall clock, device synchronised at both ends",
                                           "streams": "one compute stream for both microbatches; each stage's copies on its own streams (OPW_FLAG_COPY_STREAMS)",
                                           "h2d_bytes_per_step": int(round(packed + delta_bytes[0] / n2)), "d2h_bytes_per_step": int(d2h),
                                           "frac_of_value": round(v2 / value, 4)}
        for stg in mb_stages:
            stg.close()
    if want_submit:
        # The same steps through a plan: one native call (one CUDA graph launch) per pass over
        # the stage's layers, metadata advanced on the device.
        t_now = n_used if stack else (n_used + R - 1) // R       # first length not yet appended in any pool
        gpos = pos_all[t_now].clone()
        glen = len_all[t_now].clone()
        room = int(pos_all.shape[0] - 1 - t_now)                 # decode steps the page tables still cover
        assert room >= 2 * (3 + n_sub), (room, n_sub)
        outs = [torch.empty_like(out) for _ in range(R)]        # one output buffer per item
        for mode, extra in (("plan: CUDA graph + on-device advance", 0),
                            ("plan: CUDA graph + on-device advance + combine beside the next attention",
                             binding.OPW_PLAN_OVERLAP)):
            if n_sub < 2:
                break
            items = [dict(layer=l, batch=B, q=inp.q[0, l].data_ptr(), k_new=inp.k_new[0, l].data_ptr(),
                          v_new=inp.v_new[0, l].data_ptr(), positions=gpos.data_ptr(),
                          kv_lens=glen.data_ptr() if unfused else None,
                          page_table=inp.page_tables[l].data_ptr(), out=outs[l].data_ptr()) for l in range(R)]
            plan = binding.opw_attn_plan_create(st.handle, items,
                                                binding.OPW_PLAN_GRAPH | binding.OPW_PLAN_ADVANCE | extra)
            for _ in range(3):
                binding.opw_attn_plan_submit(plan, stream.cuda_stream)
            torch.cuda.synchronize()
            first_len = gpos.cpu().numpy().astype(np.int64) + 1
            barrier()
            host = 0.0
            t0.record(stream)
            for _ in range(n_sub):
                h0 = time.perf_counter()
                binding.opw_attn_plan_submit(plan, stream.cuda_stream)
                host += time.perf_counter() - h0
            t1.record(stream)
            torch.cuda.synchronize()
            s_ms = t0.elapsed_time(t1)
            assert st.poll_error() == binding.OPW_OK
            s_bytes = 0
            for i in range(n_sub):
                n_i = first_len + i
                for l in range(R):
                    w = wl_r.layer_window[l]
                    s_bytes += int((np.minimum(n_i, w) if w > 0 else n_i).sum()) * wl.kv_bytes_per_token
            key = "submit_overlap" if extra else "submit"
            res[key] = {"mode": mode, "value": round(s_bytes / (s_ms * 1e-3) / 1e9, 1), "unit": "GB/s",
                        "submits": n_sub, "layer_steps_per_submit": R,
                        "ms_per_layer_step": round(s_ms / (n_sub * R), 5),
                        "host_us_per_submit": round(host / n_sub * 1e6, 2)}
            binding.opw_attn_plan_destroy(plan)
    if want_cpu:
        res["cpu_baseline"] = cpu_baseline(name, inp, budget_s=15.0)
    st.close()
    del inp
    torch.cuda.empty_cache()
    return res


def run_linear_layer(steps, batch=256, Hk=16, Hv=32, dk=128, dv=128, rotate=4):
    """The recurrent-state (linear attention) decode step: state bytes read + written per second."""
    import torch

    from paper_2609_14237_b200 import binding

    g = torch.Generator(device="cuda")
    g.manual_seed(2001)
    states = [torch.randn(batch, Hv, dk, dv, device="cuda", generator=g) for _ in range(rotate)]
    q = torch.randn(batch, Hk, dk, device="cuda", generator=g).to(torch.bfloat16)
    k = torch.nn.functional.normalize(torch.randn(batch, Hk, dk, device="cuda", generator=g), dim=-1).to(torch.bfloat16)
    v = torch.randn(batch, Hv, dv, device="cuda", generator=g).to(torch.bfloat16)
    a = torch.rand(batch, Hv, device="cuda", generator=g) * 0.1 + 0.9
    beta = torch.rand(batch, Hv, device="cuda", generator=g)
    slot = torch.arange(batch, dtype=torch.int32, device="cuda")
    out = torch.empty(batch, Hv, dv, dtype=torch.bfloat16, device="cuda")
    stream = torch.cuda.current_stream()

    def step(i):
        binding.opw_linear_attn_decode_step(batch=batch, num_k_heads=Hk, num_v_heads=Hv, dk=dk, dv=dv,
                                            state=states[i % rotate].data_ptr(), num_slots=batch, slot=slot.data_ptr(),
                                            q=q.data_ptr(), k=k.data_ptr(), v=v.data_ptr(), a=a.data_ptr(),
                                            beta=beta.data_ptr(), out=out.data_ptr(), stream=stream.cuda_stream)

    for i in range(5):
        step(i)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for i in range(steps):
        step(i)
    e1.record(stream)
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / steps
    nbytes = 2 * batch * Hv * dk * dv * 4
    peak, kind = measured_peak()
    gbs = nbytes / (ms * 1e-3) / 1e9
    return {"value": round(gbs, 1), "unit": "GB/s (state read + write)", "ms_per_step": round(ms, 5),
            "seq_steps_per_s_per_layer": round(batch / (ms * 1e-3), 1), "state_bytes_per_step": nbytes // 2,
            "config": {"batch": batch, "num_k_heads": Hk, "num_v_heads": Hv, "dk": dk, "dv": dv,
                       "l2": f"rotating over {rotate} state sets, {rotate * nbytes / 2e9:.2f} GB between re-reads"},
            "roofline": {"bound": "hbm", "achieved": round(gbs, 1), "peak": peak, "unit": "GB/s",
                         "frac": round(gbs / peak, 4), "peak_kind": kind, "kernel": "opw_lin::decode_step_kernel",
                         "traffic": None},
            "steps": steps}


def run_afd_module(steps, name="c2_llama8b", hidden=4096, layers=4, batch=None):
    """The complete attention module (QKV projection + rotary encoding + core attention + output
    projection) on the workload's shape: time per module step with the projections on the
    tensor-core kernel and on the library path, back to back over `layers` layers with their own
    weights and KV pools (so neither stays in L2), beside the core-attention step alone."""
    import numpy as np
    import torch

    from paper_2609_14237_b200 import binding, synth

    wl = dataclasses.replace(synth.WORKLOADS[name], layer_window=[0] * layers)
    if batch:
        wl = dataclasses.replace(wl, batch=int(batch))
    total = steps + 8
    inp = synth.make_inputs(wl, device="cuda", growth=4 * (total // layers + 4), steps=1)
    Hq, Hkv, D, Bn = wl.num_q_heads, wl.num_kv_heads, wl.head_dim, wl.batch
    stage = binding.Stage(pools=inp.pools, layer_window=wl.layer_window, num_q_heads=Hq, num_kv_heads=Hkv, head_dim=D,
                          max_batch=Bn, max_pages_per_seq=inp.max_pages_per_seq)
    g = torch.Generator(device="cuda")
    g.manual_seed(3001)
    w_qkv = [(torch.randn((Hq + 2 * Hkv) * D, hidden, device="cuda", generator=g) / hidden ** 0.5).to(torch.bfloat16)
             for _ in range(layers)]
    w_o = [(torch.randn(hidden, Hq * D, device="cuda", generator=g) / (Hq * D) ** 0.5).to(torch.bfloat16)
           for _ in range(layers)]
    x = torch.randn(Bn, hidden, device="cuda", generator=g).to(torch.bfloat16)
    y = torch.empty_like(x)
    out = torch.empty(Bn, Hq, D, dtype=torch.bfloat16, device="cuda")
    pos0 = torch.from_numpy(inp.lengths.astype(np.int32)).cuda()
    stream = torch.cuda.current_stream()

    def timed(fn):
        pos = pos0.clone()
        for i in range(8):
            fn(i % layers, pos)
            if i % layers == layers - 1:
                pos.add_(1)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for i in range(steps):
            fn(i % layers, pos)
            if i % layers == layers - 1:
                pos.add_(1)
        e1.record(stream)
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / steps

    stage_plain = binding.Stage(pools=inp.pools, layer_window=wl.layer_window, num_q_heads=Hq, num_kv_heads=Hkv, head_dim=D,
                                max_batch=Bn, max_pages_per_seq=inp.max_pages_per_seq, flags=binding.OPW_FLAG_NO_PDL)
    res = {}
    for label, st, flags in (("tcgen05", stage, 0), ("library", stage, binding.OPW_AFD_LIBRARY_GEMM),
                             ("tcgen05_no_pdl", stage_plain, binding.OPW_AFD_NO_PDL),
                             ("tcgen05_no_cluster", stage, binding.OPW_AFD_NO_CLUSTER)):
        mods = [binding.AfdModule(st, l, w_qkv[l], w_o[l], 10000.0, flags) for l in range(layers)]
        res[label] = timed(lambda l, pos: mods[l].step(x, pos, inp.page_tables[l], y))
        assert all(m.poll_error() == 0 for m in mods) and st.poll_error() == 0
        if label == "tcgen05":
            # the same steps as one plan: all layers' module steps in one CUDA graph, positions advanced on the device
            pos = pos0.clone()
            ops = [dict(kind="afd_module", module=mods[l].handle, batch=Bn, x=x.data_ptr(), positions=pos.data_ptr(),
                        page_table=inp.page_tables[l].data_ptr(), y=y.data_ptr()) for l in range(layers)]
            plan = binding.opw_attn_plan_create_mixed(st.handle, ops, binding.OPW_PLAN_GRAPH | binding.OPW_PLAN_ADVANCE)
            n_sub = max(2, steps // layers)
            for _ in range(2):
                binding.opw_attn_plan_submit(plan, stream.cuda_stream)
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            for _ in range(n_sub):
                binding.opw_attn_plan_submit(plan, stream.cuda_stream)
            e1.record(stream)
            torch.cuda.synchronize()
            res["plan"] = e0.elapsed_time(e1) / (n_sub * layers)
            assert all(m.poll_error() == 0 for m in mods) and st.poll_error() == 0
            binding.opw_attn_plan_destroy(plan)
        for m in mods:
            m.close()
    stage_plain.close()
    q, k, v = inp.q[0, 0], inp.k_new[0, 0], inp.v_new[0, 0]
    res["attention"] = timed(lambda l, pos: stage.decode_step(l, q, k, v, pos, inp.page_tables[l], out))
    stage.close()
    weight_bytes = 2 * ((Hq + 2 * Hkv) * D * hidden + hidden * Hq * D)
    return {"value": round(Bn / (res["tcgen05"] * 1e-3), 1), "unit": "sequence-steps/s per layer (whole attention module)",
            "ms_per_step": round(res["tcgen05"], 5), "ms_per_step_library_gemm": round(res["library"], 5),
            "ms_per_step_without_programmatic_dependent_launch": round(res["tcgen05_no_pdl"], 5),
            "ms_per_step_without_clusters": round(res["tcgen05_no_cluster"], 5),
            "ms_per_step_plan": round(res["plan"], 5),
            "ms_per_step_core_attention_alone": round(res["attention"], 5),
            "projection_weight_bytes_per_step": weight_bytes, "kv_bytes_per_step": int(inp.kv_bytes(0, 0)),
            "config": {"shape_of": name, "batch": Bn, "hidden": hidden, "num_q_heads": Hq, "num_kv_heads": Hkv, "head_dim": D,
                       "l2": f"{layers} layers with their own weights ({layers * weight_bytes / 1e6:.0f} MB) and KV pools, back to back"},
            "kernels": "skinny_gemm_kernel (tcgen05, rotary epilogue) x2 + attn_splitkv_kernel + combine_kernel per step",
            "steps": steps}


def cpu_baseline(name, inp=None, budget_s=15.0, device="cpu"):
    """The fp64 oracle as it stands, timed on this machine's host cores over a bounded sample of
    the workload's sequences (layer 0, step 0); value in the metric's unit."""
    import torch

    import oracle
    from paper_2609_14237_b200 import synth

    wl = synth.WORKLOADS[name]
    if inp is None:
        inp = synth.make_inputs(dataclasses.replace(wl, layer_window=wl.layer_window[:1]), device=device, growth=1, steps=1)
    Hq, Hkv, D, P = wl.num_q_heads, wl.num_kv_heads, wl.head_dim, 16
    lens = inp.kv_lens(0)
    window = inp.wl.layer_window[0]
    order = np.argsort(-lens.astype(np.int64), kind="stable")          # longest first
    pe = Hkv * 2 * P * D

    def sample(rows):
        tab = inp.page_tables[0][rows].cpu()
        used = torch.unique(tab[tab >= 0])
        remap = torch.full((inp.num_pages[0],), -1, dtype=torch.int32)
        remap[used.long()] = torch.arange(used.numel(), dtype=torch.int32)
        small = inp.pools[0].view(-1, pe)[used.to(inp.pools[0].device).long()].contiguous().view(-1).cpu()
        new_tab = torch.where(tab >= 0, remap[tab.clamp(min=0).long()], torch.full_like(tab, -1)).numpy()
        q = inp.q[0, 0][rows].cpu()
        k, v = inp.k_new[0, 0][rows].cpu(), inp.v_new[0, 0][rows].cpu()
        return oracle.as_u16(small).copy(), new_tab, q, k, v

    def timed(rows):
        pool, tab, q, k, v = sample(rows)
        n = lens[rows]
        t0 = time.perf_counter()
        oracle.kv_append(pool, Hkv, D, P, k, v, (n - 1).astype(np.int32), tab)
        oracle.decode_attention(pool, Hq, Hkv, D, P, q, n, tab, window=window)
        dt = time.perf_counter() - t0
        vis = np.minimum(n, window) if window > 0 else n
        return dt, int(vis.astype(np.int64).sum()) * wl.kv_bytes_per_token

    probe_rows = [int(order[len(order) // 2])]
    dt, nbytes = timed(probe_rows)
    rate = nbytes / max(dt, 1e-6)
    rows, acc = [], 0
    for r in order[::max(1, len(order) // 64)].tolist() + order.tolist():
        if r in rows:
            continue
        vis = min(int(lens[r]), window) if window > 0 else int(lens[r])
        if rows and (acc + vis * wl.kv_bytes_per_token) / rate > budget_s:
            break
        rows.append(int(r))
        acc += vis * wl.kv_bytes_per_token
    dt, nbytes = timed(sorted(rows))
    return {"value": round(nbytes / dt / 1e9, 4), "unit": "GB/s", "cores": oracle.num_threads(), "kind": "oracle",
            "sample": f"{len(rows)} of {len(lens)} sequences of {name}, layer 0, one append+attention step "
                      f"({nbytes / 1e6:.1f} MB of KV in {dt:.2f} s)",
            "seq_steps_per_s_per_layer": round(len(rows) / dt, 3)}


def run_reference(name, steps, warmup):
    """The reference arm: the CPU oracle, as it stands, on the host cores."""
    import oracle
    from paper_2609_14237_b200 import synth

    wl = synth.WORKLOADS[name]
    inp = synth.make_inputs(dataclasses.replace(wl, layer_window=wl.layer_window[:1]), device="cpu", growth=1, steps=1)
    total = max(1, steps + warmup)
    budget = min(20.0, 150.0 / total)
    vals = []
    for i in range(total):
        r = cpu_baseline(name, inp, budget_s=budget)
        if i >= warmup:
            vals.append(r)
    v = float(np.mean([r["value"] for r in vals]))
    ms = float(np.mean([float(r["sample"].split(" in ")[1].split(" s")[0]) for r in vals])) * 1e3
    return {"impl": "reference", "metric": METRIC, "value": round(v, 4), "unit": "GB/s", "n_gpus": 1, "steps": steps,
            "warmup": warmup, "ms_per_step": round(ms, 2), "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": name, "batch": wl.batch, "num_q_heads": wl.num_q_heads,
                       "num_kv_heads": wl.num_kv_heads, "head_dim": wl.head_dim, "page_size": 16,
                       "note": "each step is a bounded sample of the workload's sequences"},
            "cpu_baseline": {"value": round(v, 4), "unit": "GB/s", "cores": oracle.num_threads(), "kind": "oracle",
                             "sample": vals[-1]["sample"]},
            "e2e": {"value": round(v, 4), "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD)
    ap.add_argument("--rotate", type=int, default=4, help="layer pools cycled through by a one-layer workload")
    ap.add_argument("--others", default="c2_llama8b,c4_large_batch,c5_hybrid_stack",
                    help="further workloads reported under 'other_workloads' (N=1 only; '' for none)")
    ap.add_argument("--no-cpu", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--warps", type=int, default=0)
    ap.add_argument("--stages", type=int, default=0)
    ap.add_argument("--ctas", type=int, default=0)
    ap.add_argument("--unfused", action="store_true", help="separate opw_kv_append + opw_decode_attention calls")
    ap.add_argument("--module-layers", type=int, default=4, help="layers (weights and KV pools) --workload attention_module cycles through")
    ap.add_argument("--module-batch", type=int, default=0, help="batch rows of --workload attention_module (default: the shape's own)")
    ap.add_argument("--no-pdl", action="store_true", help="launch the kernels without programmatic stream serialisation")
    args = ap.parse_args()
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))

    if args.impl == "reference":
        if rank == 0:
            steps = args.steps if args.steps is not None else 3
            warmup = args.warmup if args.warmup is not None else 1
            print(json.dumps(run_reference(args.workload, steps, warmup)), flush=True)
        return

    import torch

    from paper_2609_14237_b200 import binding

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the attention stage has no CPU path")
    binding.build()
    # One rank per GPU.  OPW_BENCH_BACKEND=gloo (with fewer GPUs than ranks: ranks share devices)
    # exists to exercise the multi-rank bookkeeping on a single-GPU machine; its numbers mean nothing.
    backend = os.environ.get("OPW_BENCH_BACKEND", "nccl")
    local = local % torch.cuda.device_count() if backend != "nccl" else local
    torch.cuda.set_device(local)
    if world > 1:
        import torch.distributed as dist

        if backend == "nccl":
            dist.init_process_group("nccl", device_id=torch.device("cuda", local))
        else:
            dist.init_process_group(backend)
    steps = args.steps if args.steps is not None else 2000
    warmup = args.warmup if args.warmup is not None else 20
    if args.workload == "attention_module":         # the AFD partition's stage alone (1 GPU)
        r = run_afd_module(max(8, min(steps, 2000)), batch=args.module_batch, layers=args.module_layers)
        r.update({"metric": "attention module decode: sequence-steps/s per layer", "n_gpus": 1, "warmup": 8,
                  "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
                  "gpu_launches": r["steps"] * 4})
        r["config"]["workload"] = "attention_module"
        if rank == 0:
            print(json.dumps(r), flush=True)
        return
    if args.workload == "linear_state_layer":       # the recurrent-state layer alone (1 GPU)
        r = run_linear_layer(max(10, min(steps, 2000)))
        r.update({"metric": "recurrent-state layer decode: state GB/s (read + write)", "n_gpus": 1, "warmup": 5,
                  "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
                  "gpu_launches": r["steps"]})
        r["config"]["workload"] = "linear_state_layer"
        if rank == 0:
            print(json.dumps(r), flush=True)
        return
    tune = dict(tune_warps=args.warps, tune_stages=args.stages, tune_ctas_per_sm=args.ctas,
                flags=1 if args.no_pdl else 0)
    res = run_ours(args.workload, steps, max(3, warmup), args.rotate, tune, want_e2e=not args.no_e2e, want_submit=(world == 1), unfused=args.unfused,
                   want_cpu=(world == 1 and rank == 0 and not args.no_cpu), world=world, rank=rank)
    if world == 1 and rank == 0:
        ceil = measure_read_ceiling()
        if ceil is not None:
            res["roofline"]["read_ceiling"] = ceil
            res["roofline"]["frac_of_read_ceiling"] = round(res["roofline"]["achieved"] / ceil["value"], 4)
    if world == 1 and args.others:
        others = {}
        for name in args.others.split(","):
            if not name or name == args.workload:
                continue
            if name == "c5_hybrid_stack":
                if torch.cuda.mem_get_info()[0] < 70 * (1 << 30):
                    others[name] = {"skipped": "needs ~55 GB of device memory"}
                    continue
                k = max(10, min(steps, 100))
            else:
                k = max(10, min(steps, 1000))
            r = run_ours(name, k, max(3, min(warmup, 10)), args.rotate, tune, want_e2e=False, want_submit=True,
                         unfused=args.unfused)
            others[name] = {key: r[key] for key in ("value", "unit", "ms_per_step", "seq_steps_per_s_per_layer",
                                                    "pct_of_nominal_8000", "roofline", "step_ms", "parity", "steps",
                                                    "submit", "submit_overlap")
                            if key in r}
            others[name]["kv_bytes_per_step"] = r["config"]["kv_bytes_per_step"]
        others["linear_state_layer"] = run_linear_layer(max(10, min(steps, 500)))
        others["attention_module_llama8b_layer"] = run_afd_module(max(8, min(steps, 400)))
        res["other_workloads"] = others
    if world > 1:
        import torch.distributed as dist

        dist.barrier()
        dist.destroy_process_group()
    if rank == 0:
        print(json.dumps(res), flush=True)


if __name__ == "__main__":
    main()
