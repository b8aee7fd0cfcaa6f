#!/usr/bin/env python
"""Benchmark of the AMS-KV hot path on synthetic VAR-shaped data.

One step = one pass of the whole path over one batch: for every scale, for every layer,
amskv_append then amskv_attend (the self-attention work of generating one batch of images).
Metric: self-attention microseconds per image over all scales and layers (lower is better),
with the roofline fraction and the KV-cache bytes beside it.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload var_d30] [--impl ours|reference]

N > 1 (under torchrun) runs independent replicas, one per GPU: the path has no exchange step.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "VAR-d30 self-attn us/image (all scales+layers)"
UNIT = "us/image"
FALLBACK_HBM_GBS = 6650.0
FALLBACK_BF16_TFLOPS = 1400.0

# DRAM traffic of the dominant kernel per launch, from an ncu capture (dram__bytes_read.sum +
# dram__bytes_write.sum), keyed by (workload, policy, calls); each entry names the capture it came from and
# is valid only for the kernel as it was then -- an entry is removed whenever that kernel changes, and
# `roofline.traffic` is then null.
NCU_DOMINANT_KERNEL_TRAFFIC = {
    ("var_d30", "ams", "fused"): {
        "bytes_per_launch": 1.655e9,
        "capture": "profiles/attention_dram_traffic_var_d30.md: 64-row, 2-layer case of the same shape, every launch of "
                   "attend_pair_kernel<64, ext> of one step, scaled by rows (x 8) and by the layers of each class (21 + 9), "
                   "averaged over its 141 launches; reads exact, writes a lower bound (part of them still in L2 at that size)"},
}


def _peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return float(p["hbm_gbs"]), float(p.get("bf16_tflops_sustained", FALLBACK_BF16_TFLOPS)), "measured"
    return FALLBACK_HBM_GBS, FALLBACK_BF16_TFLOPS, "fallback"


def _kept(k, c, w, dem):
    """Segments read at scale k -- used only to count algorithmic bytes for the roofline."""
    return [s for s in range(k + 1) if dem or s < c or s > k - w]


def algorithmic_work(wl, policies, budgets=None, cache=None):
    """Per (layer, scale): bytes = Q read + out write + kept K,V read once; flops = 4 T L D per item.
    Under token budgets the attended key count comes from the library's host-side plan."""
    from paper_2511_16047_b200 import binding as B
    items = wl.rows * wl.heads
    tok = wl.tokens
    per, keys = {}, {}
    for layer, (c, w, dem) in enumerate(policies):
        for k in range(len(tok)):
            if budgets is not None and budgets[layer][0] > 0:
                L = sum(n for _, _, n in B.amskv_attended_tokens(cache, layer, k))
            else:
                L = sum(tok[s] for s in _kept(k, c, w, dem))
            per[(layer, k)] = (2 * wl.head_dim * items * (2 * tok[k] + 2 * L), 4 * tok[k] * L * wl.head_dim * items)
            keys[(layer, k)] = L
    return per, keys


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.lines = []
        self.proc = None
        self.thread = None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.FIELDS,
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, power, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.lines:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
                power.append(float(parts[2]))
            except ValueError:
                continue
            for name, val in zip(names, parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "power_w_max": max(power) if power else None, "samples": len(sm), "reasons": sorted(reasons)}


def run_ours(args):
    import torch
    import torch.distributed as dist

    from paper_2511_16047_b200 import binding as B
    from paper_2511_16047_b200 import synth

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    assert torch.cuda.is_available(), "bench.py needs a CUDA device (there is no CPU fallback)"
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    wl = synth.WORKLOADS[args.workload]
    if args.batch:
        wl = wl.replace(batch=args.batch)
    if args.layers:
        wl = wl.replace(layers=args.layers)
    if args.condensed is not None:
        wl = wl.replace(n_condensed=args.condensed)
    if args.local is not None:
        wl = wl.replace(n_local=args.local)
    if args.demanding_fraction is not None:
        wl = wl.replace(demanding_fraction=args.demanding_fraction)
    hbm_gbs, tflops, peak_kind = _peaks()
    K = len(wl.sides)
    tok = wl.tokens
    stream = torch.cuda.current_stream()

    # inputs: several Q/K/V sets per scale, used by the layers in turn.  Each layer has its own cache region,
    # so no cached K/V is shared between layers; the scale's own Q/K/V are inputs, and with one set a layer
    # could find the coarse scales' inputs (up to ~140 MB) in the 126 MB L2 where the previous layer left
    # them.  With the sets rotating, a set is touched again only after the others' bytes went through L2.
    n_sets = max(1, args.input_sets)
    qkv_sets = [[synth.qkv_for_scale(wl.rows, wl.heads, tok[k], wl.head_dim, wl.seed + 101 * i, k, "cuda") for k in range(K)]
                for i in range(n_sets)]
    qkv = qkv_sets[0]
    outs_sets = [[torch.empty_like(q) for q, _, _ in qs] for qs in qkv_sets]
    input_bytes = sum(3 * q.numel() * 2 for q, _, _ in qkv)

    def measure(policies, label, instrument, streams=None, budgets=None, fuse=None):
        streams = args.streams if streams is None else streams
        fuse = (args.fuse and streams == 1) if fuse is None else fuse
        desc, keep = B.make_desc(wl.layers, wl.heads, wl.head_dim, wl.rows, wl.sides, policies,
                                 flags=(B.FLAG_BULK_APPEND if streams == 2 else 0) |
                                 (B.FLAG_TRANSIENT_LAST_SCALE if (args.transient_last and fuse) else 0),
                                 token_budgets=budgets)
        nbytes = B.amskv_cache_required_bytes(desc)
        free_b, _ = torch.cuda.mem_get_info()
        if nbytes + (2 << 30) > free_b:
            return {"label": label, "skipped": "needs %.1f GB, %.1f GB free" % (nbytes / 1e9, free_b / 1e9)}
        arena = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
        cache = B.amskv_cache_create(desc, arena, nbytes)
        if args.path != "auto":
            B.amskv_set_attend_path(cache, {"simt": B.PATH_SIMT, "tensor": B.PATH_TENSOR, "pair": B.PATH_TENSOR_PAIR, "small": B.PATH_SMALL}[args.path])
        work, n_keys = algorithmic_work(wl, policies, budgets, cache)

        side = torch.cuda.Stream() if streams == 2 else None
        n_ev = wl.layers * K
        ev_app = [torch.cuda.Event() for _ in range(n_ev)] if side is not None else None
        ev_att = [torch.cuda.Event() for _ in range(n_ev)] if side is not None else None

        fused_launch = {}   # (layer, scale) -> the append went into the attention launch

        def step(events=None):
            """Two streams: the appends run on a side stream and overlap the attention kernels of other
            layers.  append(l, k) -> attend(l, k) and attend(l, k) -> append(l, k + 1) (which may overwrite
            the segment attend(l, k) still reads) are ordered with events."""
            stream = torch.cuda.current_stream()   # the capture stream while a graph is being recorded
            B.amskv_cache_reset(cache)
            if side is not None:
                side.wait_stream(stream)
            for k in range(K):
                for layer in range(wl.layers):
                    q, kk, v = qkv_sets[layer % n_sets][k]
                    out = outs_sets[layer % n_sets][k]
                    i = k * wl.layers + layer
                    if side is not None:
                        if k > 0:
                            side.wait_event(ev_att[i - wl.layers])
                        B.amskv_append(cache, layer, k, kk, v, side)
                        ev_app[i].record(side)
                        stream.wait_event(ev_app[i])
                    elif not fuse:
                        B.amskv_append(cache, layer, k, kk, v, stream)
                    if events is not None:
                        e0, e1 = events[(layer, k)]
                        e0.record(stream)
                    if fuse:
                        n0 = B.amskv_launch_count()
                        B.amskv_append_attend(cache, layer, k, kk, v, q, out, stream)
                        fused_launch[(layer, k)] = B.amskv_launch_count() - n0 == 1
                    else:
                        B.amskv_attend(cache, layer, k, q, out, stream)
                    if events is not None:
                        e1.record(stream)
                    if side is not None:
                        ev_att[i].record(stream)
            if side is not None:
                stream.wait_stream(side)

        for _ in range(args.warmup):
            step()
        torch.cuda.synchronize()
        assert B.amskv_status(cache) == 0
        # the launch-bound coarse scales are replayed from a CUDA graph
        graph = None
        if not args.no_graph:
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph):
                step()
            graph.replay()
            torch.cuda.synchronize()
        launches0 = B.amskv_launch_count()
        step()
        launches_per_step = B.amskv_launch_count() - launches0
        torch.cuda.synchronize()

        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()
        sampler = ClockSampler(local_rank)
        sampler.start()
        t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t0.record(stream)
        for _ in range(args.steps):
            if graph is not None:
                graph.replay()
            else:
                step()
        t1.record(stream)
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        ms = t0.elapsed_time(t1)
        result = {"label": label, "ms_per_step": ms / args.steps, "launches_per_step": launches_per_step,
                  "kv_bytes": B.amskv_cache_bytes(cache)[2], "arena_bytes": nbytes, "fused": bool(fuse)}
        # Minimum bytes of a step: Q read + out written + the kept K/V read once (`work`), plus the scale's own
        # K/V written to the cache once.  A call that ran as copy kernel + attention also reads the scale's K/V
        # a second time (the copy reads them, attention reads them again from the cache): counted apart, as
        # wasted bytes, never as work.  With --no-fuse the timed calls are the attention launches alone.
        items = wl.rows * wl.heads
        wasted = {key: 0 for key in work}
        one_launch = {key: False for key in work}
        if fuse:
            for (layer, k), (b, f) in list(work.items()):
                kv = 2 * wl.head_dim * items * 2 * tok[k]
                if args.transient_last and k == K - 1:
                    kv = 0   # attended from the caller's tensors, never written
                work[(layer, k)] = (b + kv, f)
                one_launch[(layer, k)] = bool(fused_launch.get((layer, k)))
                wasted[(layer, k)] = 0 if one_launch[(layer, k)] else kv
        result["wasted_bytes_per_step"] = sum(wasted.values())
        result["step_bytes"] = sum(b for b, _ in work.values()) + (
            0 if fuse else sum(2 * wl.head_dim * items * 2 * tok[k] for (_, k) in work))

        if instrument:
            # per-launch durations of the attention kernel: same steps, eager, CUDA events on the launch stream
            events = {key: (torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for key in work}
            att_ms = {key: 0.0 for key in work}
            t2, t3 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            eager_ms = 0.0
            for _ in range(args.steps):
                t2.record(stream)
                step(events)
                t3.record(stream)
                torch.cuda.synchronize()
                eager_ms += t2.elapsed_time(t3)
                for key, (e0, e1) in events.items():
                    att_ms[key] += e0.elapsed_time(e1)
            result["eager_ms_per_step"] = eager_ms / args.steps
            result["attend_ms_per_step"] = sum(att_ms.values()) / args.steps
            result["attend_bytes_per_step"] = sum(b for b, _ in work.values())
            result["attend_flops_per_step"] = sum(f for _, f in work.values())
            per_scale = []
            for k in range(K):
                b = sum(work[(l, k)][0] for l in range(wl.layers))
                f = sum(work[(l, k)][1] for l in range(wl.layers))
                t = sum(att_ms[(l, k)] for l in range(wl.layers)) / args.steps
                roof = sum(max(work[(l, k)][0] / (hbm_gbs * 1e9), work[(l, k)][1] / (tflops * 1e12))
                           for l in range(wl.layers)) * 1e3
                per_scale.append({"scale": k, "tokens": tok[k], "ms": round(t, 4), "gbs": round(b / t / 1e6, 1) if t else None,
                                  "tflops": round(f / t / 1e9, 1) if t else None, "roofline_ms": round(roof, 4),
                                  "frac": round(roof / t, 3) if t else None})
            result["per_scale"] = per_scale
            result["pass_roofline_ms"] = sum(p["roofline_ms"] for p in per_scale)
            # the dominant kernel alone: the calls that ran as ONE launch of the paired kernel with the append
            # fused in (every launch of that kernel in a step, and nothing else, sits between their events)
            # (scales of at most 16 queries over at most 32 keys are the warp-per-item kernel's, not this one's)
            dom = [key for key in work if one_launch[key] and (tok[key[1]] > 16 or n_keys[key] > 32)]
            if dom:
                d_ms = sum(att_ms[key] for key in dom) / args.steps
                d_bytes = sum(work[key][0] for key in dom)
                result["dominant"] = {"kernel": "attend_pair_kernel<%d, ext=true, wide=%s>" % (wl.head_dim, "true" if wl.head_dim == 128 else "false"),
                                      "launches_per_step": len(dom), "bytes_per_step": d_bytes,
                                      "flops_per_step": sum(work[key][1] for key in dom),
                                      "ms_per_step": d_ms, "scales": sorted({k for _, k in dom})}
        result["clocks"] = sampler.stop()
        torch.cuda.synchronize()
        assert B.amskv_status(cache) == 0
        result["_cache"] = (cache, arena, desc, keep)
        return result

    policies = wl.policies(full_retention=args.policy == "full")
    budgets = wl.token_budgets() if args.policy == "tokens" else None
    main = measure(policies, args.policy, instrument=True, budgets=budgets)
    if "skipped" in main:
        raise SystemExit("workload does not fit: " + main["skipped"])
    cache, arena, desc, keep = main.pop("_cache")

    # end to end through the C ABI with HOST buffers: pinned K/V/Q in, result out, every step
    e2e = None
    if not args.no_e2e:
        nst = B.amskv_step_staging_bytes(cache)
        # Two staging buffers on two streams, calls alternating between them: the device-to-host copy of one
        # call's result overlaps the host-to-device copies of the next call (the link is full duplex), and a
        # kernel can run while the other stream copies.  Per layer the calls stay ordered by events.
        stagings = [torch.empty(nst, dtype=torch.uint8, device="cuda") for _ in range(2)]
        lanes = [torch.cuda.Stream(), torch.cuda.Stream()]
        layer_done = [torch.cuda.Event() for _ in range(wl.layers)]
        hq = [q.cpu().pin_memory() for q, _, _ in qkv]
        hk = [k.cpu().pin_memory() for _, k, _ in qkv]
        hv = [v.cpu().pin_memory() for _, _, v in qkv]
        # one result buffer per lane and scale: a call's result is read back while the next call runs
        ho = [[torch.empty_like(q).pin_memory() for q in hq] for _ in range(2)]

        def host_step():
            B.amskv_cache_reset(cache)
            for lane in lanes:
                lane.wait_stream(stream)
            i = 0
            for k in range(K):
                for layer in range(wl.layers):
                    lane = i & 1
                    if k > 0:
                        lanes[lane].wait_event(layer_done[layer])   # the layer's previous scale (maybe on the other lane)
                    B.amskv_step_host(cache, layer, k, hk[k], hv[k], hq[k], ho[lane][k], stagings[lane], nst, lanes[lane])
                    layer_done[layer].record(lanes[lane])
                    i += 1
            for lane in lanes:
                stream.wait_stream(lane)

        host_step()
        torch.cuda.synchronize()
        e_steps = max(1, min(args.steps, args.e2e_steps))
        if world > 1:
            dist.barrier()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        for _ in range(e_steps):
            host_step()
        b.record(stream)
        torch.cuda.synchronize()
        e_ms = a.elapsed_time(b) / e_steps
        if world > 1:
            t = torch.tensor([e_ms], device="cuda")
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
            e_ms = float(t.item())
        h2d = wl.layers * input_bytes
        d2h = wl.layers * sum(q.numel() * 2 for q in hq)
        e2e = {"value": e_ms * 1e3 / (wl.batch * world) , "unit": UNIT, "h2d_bytes_per_step": h2d,
               "d2h_bytes_per_step": d2h, "steps": e_steps, "ms_per_step": e_ms}
        del stagings, hq, hk, hv, ho
    B.amskv_cache_destroy(cache)
    del arena
    torch.cuda.empty_cache()

    # the same pass with the appends on a side stream (they then overlap other layers' attention)
    overlap = None
    if not args.no_compare and args.streams == 1:
        overlap = measure(policies, args.policy + ", two streams", instrument=False, streams=2, budgets=budgets)
        if "_cache" in overlap:
            c3, a3, _, _ = overlap.pop("_cache")
            B.amskv_cache_destroy(c3)
            del a3
            torch.cuda.empty_cache()

    # the other policy (full retention when timing AMS-KV and vice versa): KV bytes and latency beside it
    other = None
    if not args.no_compare:
        other_name = "ams" if args.policy == "full" else "full"
        other = measure(wl.policies(full_retention=other_name == "full"), other_name, instrument=False)
        if "_cache" in other:
            c2, a2, _, _ = other.pop("_cache")
            B.amskv_cache_destroy(c2)
            del a2
            torch.cuda.empty_cache()

    ms = main["ms_per_step"]
    if world > 1:
        t = torch.tensor([ms], device="cuda")
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        ms = float(t.item())
    images = wl.batch * world
    value = ms * 1e3 / images

    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        cpu_baseline = oracle_sample(wl, policies, args.cpu_rows, budgets=budgets)

    if rank == 0:
        # whole pass: minimum bytes of a step over the graph-timed step (launch gaps and all); a workload whose
        # flops need longer at the bf16 peak than its bytes at the HBM peak is reported against the tensor peak
        achieved = main["step_bytes"] / (ms / 1e3) / 1e9
        step_flops = main["attend_flops_per_step"]
        tensor_bound = step_flops / (tflops * 1e12) > main["step_bytes"] / (hbm_gbs * 1e9)
        dom = main.get("dominant")
        traffic, traffic_note = None, None
        if (dom and not args.batch and not args.layers and args.path == "auto" and args.condensed is None
                and args.local is None and args.demanding_fraction is None):
            cap = NCU_DOMINANT_KERNEL_TRAFFIC.get((args.workload, args.policy, "fused" if main.get("fused") else "separate"))
            if cap is not None:
                traffic = cap["bytes_per_launch"]
                traffic_note = cap["capture"]
        if tensor_bound:
            ach_tf = step_flops / (ms / 1e3) / 1e12
            roofline = {"bound": "tensor", "peak": tflops, "unit": "TFLOP/s", "peak_kind": peak_kind + " (bf16, sustained)",
                        "scope": "whole step: 4 T L D flops per (row, head) of every attention launch / CUDA-graph-timed step",
                        "achieved": round(ach_tf, 1), "frac": round(ach_tf / tflops, 4), "step_flops": step_flops,
                        "step_bytes": main["step_bytes"], "hbm_gbs_achieved": round(achieved, 1),
                        "kernel": dom["kernel"] if dom else None,
                        "kernel_launches_per_step": dom["launches_per_step"] if dom else None,
                        "kernel_scales": dom["scales"] if dom else None,
                        "kernel_flops_per_launch": round(dom["flops_per_step"] / dom["launches_per_step"]) if dom else None,
                        "kernel_ms_per_launch": round(dom["ms_per_step"] / dom["launches_per_step"], 5) if dom else None,
                        "kernel_achieved": round(dom["flops_per_step"] / dom["ms_per_step"] / 1e9, 1) if dom else None,
                        "kernel_frac": round(dom["flops_per_step"] / dom["ms_per_step"] / 1e9 / tflops, 4) if dom else None,
                        "kernel_timing": "CUDA events around each call in an eager replay of the same step",
                        "traffic": None}
        else:
            roofline = {"bound": "hbm", "peak": hbm_gbs, "unit": "GB/s", "peak_kind": peak_kind,
                        "scope": "whole step: minimum bytes (Q read, out written, kept K/V read once, the scale's K/V "
                                 "written once) / CUDA-graph-timed step",
                        "achieved": round(achieved, 1), "frac": round(achieved / hbm_gbs, 4),
                        "frac_of_8TBs_nominal": round(achieved / 8000.0, 4),
                        "step_bytes": main["step_bytes"], "wasted_bytes_per_step": main["wasted_bytes_per_step"],
                        "wasted_note": "second read of a scale's K/V where a call ran as copy kernel + attention; not counted as work",
                        "kernel": dom["kernel"] if dom else None,
                        "kernel_launches_per_step": dom["launches_per_step"] if dom else None,
                        "kernel_scales": dom["scales"] if dom else None,
                        "kernel_bytes_per_launch": round(dom["bytes_per_step"] / dom["launches_per_step"]) if dom else None,
                        "kernel_ms_per_launch": round(dom["ms_per_step"] / dom["launches_per_step"], 5) if dom else None,
                        "kernel_achieved": round(dom["bytes_per_step"] / dom["ms_per_step"] / 1e6, 1) if dom else None,
                        "kernel_frac": round(dom["bytes_per_step"] / dom["ms_per_step"] / 1e6 / hbm_gbs, 4) if dom else None,
                        "kernel_timing": "CUDA events around each call in an eager replay of the same step",
                        "traffic": traffic, "traffic_note": traffic_note}
        # Exponentials: one per (query, attended key) = flops / (4 D).  The special-function unit gives 16 per
        # clock per SM (8.0 clocks per warp instruction per sub-partition, measured); with 64 channels it, not the
        # tensor pipe, is the arithmetic floor (the tensor pipe needs 4 D / 8192 = 1/32 clock per exponential).
        sm_mhz = (main["clocks"] or {}).get("sm_mhz") or 0
        sm_count = torch.cuda.get_device_properties(torch.cuda.current_device()).multi_processor_count
        sfu_peak = 16.0 * sm_count * sm_mhz * 1e6 / 1e9   # G exponentials / s at the median clock of this run
        exps = step_flops / (4.0 * wl.head_dim)
        roofline["sfu"] = {"exps_per_step": exps, "achieved": round(exps / (ms / 1e3) / 1e9, 1),
                           "peak": round(sfu_peak, 1) if sfu_peak else None, "unit": "Gexp/s",
                           "frac": round(exps / (ms / 1e3) / 1e9 / sfu_peak, 4) if sfu_peak else None,
                           "note": "all exponentials over 16 per clock per SM at the sampled median SM clock; "
                                   "3 of 16 are computed by polynomial on the FMA pipe, so the unit itself sees 13/16 of this"}
        line = {
            "metric": METRIC, "value": round(value, 3), "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": round(ms, 4), "higher_is_better": False, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": "%s: %d layers, %d heads x %d, batch %d (rows %d), sides %s, condensed %d, local %d, "
                                   "%d cache-demanding layers, policy %s" % (
                                       wl.name, wl.layers, wl.heads, wl.head_dim, wl.batch, wl.rows,
                                       "x".join(map(str, wl.sides)), wl.n_condensed, wl.n_local,
                                       sum(1 for p in policies if p[2]), args.policy),
                       "step": "append + attend for every scale and layer",
                       "calls": ("amskv_append_attend (one launch where the paired kernel takes the append in, else two)"
                                 if main.get("fused") else "amskv_append, then amskv_attend"),
                       "l2": "per-layer KV regions far larger than L2; %d input sets (Q, K, V, out per scale) used by the layers in turn; no flush" % n_sets,
                       "launch": "CUDA graph replay" if not args.no_graph else "eager",
                       "streams": "appends on a side stream, ordered with attention by events" if args.streams == 2 else "one stream",
                       "last_scale": "never stored" if (args.transient_last and main.get("fused")) else "stored",
                       "replicas": world},
            "clocks": main["clocks"],
            "e2e": e2e,
            "gpu_launches": main["launches_per_step"] * args.steps,
            "roofline": roofline,
            "pass_roofline": {"roofline_ms": round(main["pass_roofline_ms"], 3),
                              "attend_ms": round(main["attend_ms_per_step"], 3),
                              "frac": round(main["pass_roofline_ms"] / main["attend_ms_per_step"], 4),
                              "note": "sum over the timed calls of max(bytes/HBM peak, flops/bf16 peak) / their measured time"},
            "timed_calls_us_per_image": round(main["attend_ms_per_step"] * 1e3 / wl.batch, 3),
            "eager_ms_per_step": round(main["eager_ms_per_step"], 4),
            "kv_cache_gb": round(main["kv_bytes"] / 1e9, 3),
            "arena_gb": round(main["arena_bytes"] / 1e9, 3),
            "per_scale": main["per_scale"],
            "cpu_baseline": cpu_baseline,
        }
        if overlap is not None and "skipped" not in overlap:
            line["two_streams"] = {"ms_per_step": round(overlap["ms_per_step"], 4),
                                   "us_per_image": round(overlap["ms_per_step"] * 1e3 / wl.batch, 3),
                                   "note": "same pass, appends on a side stream ordered with attention by events"}
        if other is not None:
            if "skipped" in other:
                line["compare"] = other
            else:
                line["compare"] = {"policy": other["label"], "ms_per_step": round(other["ms_per_step"], 4),
                                   "us_per_image": round(other["ms_per_step"] * 1e3 / wl.batch, 3),
                                   "kv_cache_gb": round(other["kv_bytes"] / 1e9, 3)}
        print(json.dumps(line))
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


def oracle_sample(wl, policies, rows, flop_budget=1.0e12, budgets=None):
    """Times the oracle, as it stands, on a bounded sample of the workload: up to `rows` rows (and, for
    the long schedules, a subset of the heads) of one layer of each policy kind, all scales.  The sample
    is cut down to about `flop_budget` fp64 multiply-adds' worth of work.  Work is exactly linear in
    rows, heads and layers, so the per-image figure for the whole workload is the scaled, layer-weighted sum."""
    import numpy as np
    import oracle
    from paper_2511_16047_b200 import synth

    K = len(wl.sides)
    tok = wl.tokens
    kinds = {}
    for layer, pol in enumerate(policies):
        if budgets is not None and budgets[layer][0] > 0:
            pol = ("tokens",) + tuple(budgets[layer])
        kinds.setdefault(pol, 0)
        kinds[pol] += 1

    def attended(pol, k):
        """Keys of scale k's queries: segment ids (whole scales) or a (segment, token) list (token budgets)."""
        if pol[0] == "tokens":
            return oracle.attended_tokens(wl.sides, k, pol[1], pol[2])
        return oracle.keep_set(k, pol[0], pol[1], pol[2])

    per_item = 0.0   # flops of one (row, head) item over all scales and one layer of each kind
    for pol in kinds:
        for k in range(K):
            L = len(attended(pol, k)) if pol[0] == "tokens" else sum(tok[s] for s in attended(pol, k))
            per_item += 4.0 * tok[k] * L * wl.head_dim
    rows = max(2, min(rows, wl.rows))
    heads = wl.heads
    while rows > 2 and per_item * rows * heads > flop_budget:
        rows //= 2
    while heads > 1 and per_item * rows * heads > flop_budget:
        heads = (heads + 1) // 2
    qkv = [synth.qkv_for_scale(rows, heads, tok[k], wl.head_dim, wl.seed, k, "cpu") for k in range(K)]

    def items(x):
        return x.double().reshape(rows * heads, x.shape[2], wl.head_dim).numpy()

    Q = [items(q) for q, _, _ in qkv]
    Ks = [items(k) for _, k, _ in qkv]
    Vs = [items(v) for _, _, v in qkv]
    scale = 1.0 / math.sqrt(wl.head_dim)
    total_s = 0.0
    weighted = 0.0
    for pol, count in kinds.items():
        t0 = time.perf_counter()
        for k in range(K):
            if pol[0] == "tokens":
                oracle.attend_tokens(Q[k], Ks, Vs, attended(pol, k), scale)
            else:
                oracle.attend_selected(Q[k], Ks, Vs, attended(pol, k), scale)
        dt = time.perf_counter() - t0
        total_s += dt
        weighted += dt * count
    images = rows / 2.0
    head_scale = wl.heads / float(heads)
    return {"value": round(weighted * head_scale * 1e6 / images, 1), "unit": UNIT, "cores": oracle.threads(), "kind": "oracle",
            "extrapolated": True,
            "sample": "%d rows x %d of %d heads, one layer of each policy kind (%d kinds), all %d scales: %.1f s measured; "
                      "value = extrapolation (linear in rows, heads, layers) to %d heads and %d layers" % (
                          rows, heads, wl.heads, len(kinds), K, total_s, wl.heads, wl.layers),
            "measured_s": round(total_s, 2)}


def run_reference(args):
    """The reference arm: the oracle on the host cores, on the same workload, metric and unit."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from paper_2511_16047_b200 import synth
    wl = synth.WORKLOADS[args.workload]
    if args.batch:
        wl = wl.replace(batch=args.batch)
    if args.layers:
        wl = wl.replace(layers=args.layers)
    policies = wl.policies(full_retention=args.policy == "full")
    budgets = wl.token_budgets() if args.policy == "tokens" else None
    rows = max(2, args.cpu_rows // 4)
    for _ in range(max(1, min(args.warmup, 1))):
        oracle_sample(wl, policies, 2, budgets=budgets)
    vals, secs = [], 0.0
    steps = max(1, min(args.steps, 3))
    for _ in range(steps):
        r = oracle_sample(wl, policies, rows, budgets=budgets)
        vals.append(r["value"])
        secs += r["measured_s"]
    value = sum(vals) / len(vals)
    sample = r["sample"]
    line = {"impl": "reference", "metric": METRIC, "value": round(value, 1), "unit": UNIT, "n_gpus": int(os.environ.get("WORLD_SIZE", "1")),
            "steps": steps, "warmup": 1, "ms_per_step": round(value * wl.batch / 1e3, 3), "higher_is_better": False,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": wl.name, "policy": args.policy, "note": "fp64 CPU oracle, bounded sample per step"},
            "extrapolated": True, "measured_s": round(secs / steps, 2),
            "cpu_baseline": {"value": round(value, 1), "unit": UNIT, "cores": r["cores"], "kind": "oracle", "sample": sample,
                             "extrapolated": True, "measured_s": round(secs / steps, 2)},
            "e2e": {"value": round(value, 1), "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


def run_similarity(args):
    """Inter-scale key similarity (Eq. 4) over every adjacent scale pair of every layer of the workload:
    GB/s against the HBM peak, and the layer classification it yields on seeded correlated /
    independent layers.  One JSON line; not the headline metric."""
    import torch
    from paper_2511_16047_b200 import binding as B
    from paper_2511_16047_b200 import synth

    assert torch.cuda.is_available(), "bench.py needs a CUDA device (there is no CPU fallback)"
    torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
    wl = synth.WORKLOADS[args.workload]
    if args.batch:
        wl = wl.replace(batch=args.batch)
    hbm_gbs, _, peak_kind = _peaks()
    # two key sets per scale: scales share a smooth field with weight 0.9 ("correlated") or 0 ("independent")
    keys = {rho: synth.smooth_field_keys(wl.rows, wl.heads, wl.sides, wl.head_dim, wl.seed + int(rho * 10), rho, "cuda")
            for rho in (0.9, 0.0)}
    n_ws = B.amskv_similarity_workspace_bytes()
    ws = torch.empty(n_ws, dtype=torch.uint8, device="cuda")
    mask = wl.demanding_mask()   # demanding layers get the independent keys: low similarity
    K = len(wl.sides)
    out = torch.zeros((wl.layers, K - 1), dtype=torch.float64, device="cuda")
    stream = torch.cuda.current_stream()

    def step():
        for layer in range(wl.layers):
            ks = keys[0.0 if mask[layer] else 0.9]
            for i in range(1, K):
                B.amskv_layer_similarity(ks[i - 1], wl.sides[i - 1], ks[i], wl.sides[i], wl.rows, wl.heads, wl.head_dim,
                                         out[layer, i - 1:], ws, n_ws, stream)

    for _ in range(max(args.warmup, 3)):
        step()
    torch.cuda.synchronize()
    l0 = B.amskv_launch_count()
    step()
    launches = B.amskv_launch_count() - l0
    graph = torch.cuda.CUDAGraph()     # 540 small launches per pass: replayed from a graph like the attention pass
    with torch.cuda.graph(graph):
        stream = torch.cuda.current_stream()
        step()
    stream = torch.cuda.current_stream()
    graph.replay()
    torch.cuda.synchronize()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record(stream)
    for _ in range(args.steps):
        graph.replay()
    b.record(stream)
    torch.cuda.synchronize()
    ms = a.elapsed_time(b) / args.steps
    tok = wl.tokens
    bytes_step = wl.layers * sum(2 * wl.rows * wl.heads * wl.head_dim * (tok[i] + tok[i - 1]) for i in range(1, K))
    scores = (-(out.sum(dim=1)).sqrt()).tolist()     # S = -sqrt(sum of squares over all pairs)
    chosen = B.amskv_classify_lowest(scores, wl.n_demanding())
    print(json.dumps({"metric": "inter-scale key similarity, all adjacent pairs of all layers", "value": round(ms, 4), "unit": "ms/pass",
                      "higher_is_better": False, "n_gpus": 1, "steps": args.steps, "dtype": "bf16", "data": "synthetic",
                      "config": {"workload": "%s: %d layers, %d rows x %d heads x %d, %d scale pairs per layer; keys larger than L2 at the "
                                             "large scales" % (wl.name, wl.layers, wl.rows, wl.heads, wl.head_dim, K - 1)},
                      "gpu_launches": launches * args.steps,
                      "roofline": {"bound": "hbm", "achieved": round(bytes_step / ms / 1e6, 1), "peak": hbm_gbs, "unit": "GB/s",
                                   "frac": round(bytes_step / ms / 1e6 / hbm_gbs, 4), "peak_kind": peak_kind, "traffic": None,
                                   "algorithmic_bytes_per_pass": bytes_step},
                      "classification": {"lowest_similarity_layers_equal_seeded_independent_layers": chosen == mask}}))


def run_density(args):
    """Attention density as a by-product (amskv_attend_density) against the plain attend pass: the same
    append + attend steps of the workload, replayed from a CUDA graph, with and without the density output.
    One JSON line; not the headline metric."""
    import torch
    from paper_2511_16047_b200 import binding as B
    from paper_2511_16047_b200 import synth

    assert torch.cuda.is_available(), "bench.py needs a CUDA device (there is no CPU fallback)"
    torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
    wl = synth.WORKLOADS[args.workload]
    if args.batch:
        wl = wl.replace(batch=args.batch)
    wl = wl.replace(layers=args.layers or 6)
    policies = wl.policies(full_retention=args.policy == "full")
    K, tok = len(wl.sides), wl.tokens
    qkv = [synth.qkv_for_scale(wl.rows, wl.heads, tok[k], wl.head_dim, wl.seed, k, "cuda") for k in range(K)]
    outs = [torch.empty_like(q) for q, _, _ in qkv]
    desc, keep = B.make_desc(wl.layers, wl.heads, wl.head_dim, wl.rows, wl.sides, policies)
    nbytes = B.amskv_cache_required_bytes(desc)
    arena = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    cache = B.amskv_cache_create(desc, arena, nbytes)
    den = torch.zeros((wl.layers, K, wl.heads, K), dtype=torch.float64, device="cuda")

    def step(with_density, events=None):
        stream = torch.cuda.current_stream()
        B.amskv_cache_reset(cache)
        for k in range(K):
            q, kk, v = qkv[k]
            for layer in range(wl.layers):
                B.amskv_append(cache, layer, k, kk, v, stream)
                if events is not None:
                    events[k][layer][0].record(stream)
                if with_density:
                    B.amskv_attend_density(cache, layer, k, q, outs[k], den[layer, k], wl.heads * K, stream)
                else:
                    B.amskv_attend(cache, layer, k, q, outs[k], stream)
                if events is not None:
                    events[k][layer][1].record(stream)

    result = {}
    for with_density in (False, True):
        for _ in range(max(args.warmup, 3)):
            step(with_density)
        torch.cuda.synchronize()
        l0 = B.amskv_launch_count()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            step(with_density)
        launches = B.amskv_launch_count() - l0
        graph.replay()
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        stream = torch.cuda.current_stream()
        a.record(stream)
        for _ in range(args.steps):
            graph.replay()
        b.record(stream)
        torch.cuda.synchronize()
        # attention calls alone, per scale: CUDA events around each call in an eager replay
        events = [[(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(wl.layers)]
                  for _ in range(K)]
        step(with_density, events)
        torch.cuda.synchronize()
        per_scale = [round(sum(e0.elapsed_time(e1) for e0, e1 in events[k]), 4) for k in range(K)]
        result["with_density" if with_density else "plain"] = {"ms_per_step": round(a.elapsed_time(b) / args.steps, 4),
                                                               "launches_per_step": launches,
                                                               "attend_ms_per_scale": per_scale}
    assert B.amskv_status(cache) == 0
    # the density of the last scale of layer 0, per retained scale, averaged over heads (what Fig. 5 plots)
    runs = B.amskv_attended_tokens(cache, 0, K - 1)
    last = den[0, K - 1].flatten()[:wl.heads * len(runs)].view(wl.heads, len(runs)).mean(dim=0).tolist()
    B.amskv_cache_destroy(cache)
    ratio = result["with_density"]["ms_per_step"] / result["plain"]["ms_per_step"]
    print(json.dumps({"metric": "append + attend pass with the attention density as a by-product vs without", "value": round(ratio, 4),
                      "unit": "time ratio", "higher_is_better": False, "n_gpus": 1, "steps": args.steps, "dtype": "bf16",
                      "data": "synthetic",
                      "config": {"workload": "%s: %d layers, %d rows x %d heads x %d, policy %s" % (
                          wl.name, wl.layers, wl.rows, wl.heads, wl.head_dim, args.policy)},
                      "gpu_launches": (result["plain"]["launches_per_step"] + result["with_density"]["launches_per_step"]) * args.steps,
                      "plain": result["plain"], "with_density": result["with_density"],
                      "attend_ratio_per_scale": [round(d / p, 3) if p else None for p, d in zip(result["plain"]["attend_ms_per_scale"],
                                                                                                result["with_density"]["attend_ms_per_scale"])],
                      "density_of_last_scale_layer_0": {"runs": runs, "mean_over_heads": [round(x, 5) for x in last]}}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="var_d30")
    ap.add_argument("--no-fuse", dest="fuse", action="store_false",
                    help="amskv_append then amskv_attend per layer and scale instead of one amskv_append_attend call "
                         "(the append fused into the attention launch where that pays)")
    ap.add_argument("--transient-last", action="store_true",
                    help="never store the last scale (AMSKV_FLAG_TRANSIENT_LAST_SCALE): smaller arena, same results")
    ap.add_argument("--policy", default="ams", choices=["ams", "full", "tokens"],
                    help="ams: whole scales (condensed + local window); full: every scale; tokens: Algorithm 1 "
                         "and 2 with token budgets (C_cds = the condensed scales, C_min = C_cds + the penultimate "
                         "scale, C_max = C_cds + the last two scales)")
    ap.add_argument("--path", default="auto", choices=["auto", "simt", "tensor", "pair", "small"],
                    help="force one attention kernel for every scale (default: the library chooses per scale)")
    ap.add_argument("--batch", type=int, default=0, help="override the workload's batch (images)")
    ap.add_argument("--layers", type=int, default=0, help="override the workload's layer count")
    ap.add_argument("--condensed", type=int, default=None, help="override the number of condensed scales")
    ap.add_argument("--local", type=int, default=None, help="override the local window (scales)")
    ap.add_argument("--demanding-fraction", type=float, default=None, help="override the share of cache-demanding layers")
    ap.add_argument("--cpu-rows", type=int, default=256, help="rows of the oracle's timed sample")
    ap.add_argument("--e2e-steps", type=int, default=2)
    ap.add_argument("--input-sets", type=int, default=4,
                    help="Q/K/V/out sets per scale that the layers use in turn (so that a coarse scale's inputs are not "
                         "served from L2 where the previous layer left them)")
    ap.add_argument("--streams", type=int, default=1, choices=[1, 2],
                    help="2: appends on a side stream overlapping attention of other layers; 1: everything in order")
    ap.add_argument("--similarity", action="store_true", help="time amskv_layer_similarity instead of the attention pass")
    ap.add_argument("--density", action="store_true",
                    help="time the append + attend pass with and without the attention density as a by-product")
    ap.add_argument("--no-graph", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-compare", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.impl == "reference":
        run_reference(args)
    elif args.similarity:
        run_similarity(args)
    elif args.density:
        run_density(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
