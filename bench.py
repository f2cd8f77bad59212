#!/usr/bin/env python
"""Benchmark of the CoSA prefill hot path (KAP + OSK) on B200.

One "step" = one pass of the whole hot path (cosa_kap_select then cosa_osk_attention)
over one synthetic attention layer.  The headline workload is the Qwen3-8B-shaped layer
at 128K tokens (32 query / 8 KV heads, d = 128, causal, block 128, KAP budget 10 %,
OSK budget 4 %).  `value` is the visited-block TFLOP/s of the whole job: 2*128*128*128
FLOPs per block whose logits OSK formed plus the same per block it computed, summed over
all ranks, divided by the (max over ranks) time of KAP + OSK.  With N > 1 every rank
processes its own layer (independent seeds): weak scaling, no data-path collective.  With --shard kv_head
the ranks split one layer by KV-head group instead (strong scaling; still no data-path collective: the
work items of different KV heads share nothing, and the outputs stay head-sharded).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]
"""
from __future__ import annotations

import argparse
import json
import math
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

BLOCK_FLOPS = 2.0 * 128 * 128 * 128          # one 128x128x128 tile contraction
METRIC = "osk_kap_prefill_visited_block_tflops"
UNIT = "TFLOP/s"


def parse():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="qwen3_128k")
    ap.add_argument("--no-comparators", action="store_true", help="skip the dense-path and SDPA timings")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--page-size", type=int, default=0,
                    help="K and V as page pools of this many tokens per page behind a shuffled page table (Sec. C.1); not the headline config")
    ap.add_argument("--block-q", type=int, default=128, choices=[128, 256],
                    help="256: one Stage-1 ranking per 256-row query block shared by its two row tiles; not the headline config")
    ap.add_argument("--shard", default="layer", choices=["layer", "kv_head"],
                    help="with --gpus N: 'layer' gives every rank a layer of its own (weak scaling, the default); 'kv_head' splits "
                         "ONE layer by KV-head group, rank r running KAP + OSK on its heads only (strong scaling; N <= KV heads)")
    ap.add_argument("--pages-in-place", action="store_true",
                    help="with --page-size below 128: OSK reads the pages in place (cosa_options.kv_pages_in_place), no staging copy")
    ap.add_argument("--osk-impl", type=int, default=0, choices=[0, 4, 5],
                    help="4: the OSK kernel that walks two work items per CTA (cosa_options.impl = 4); 5: the same kernel on the two row "
                         "tiles of a 256-row query block, every fetched K/V tile serving both (needs --block-q 256); not the headline config")
    ap.add_argument("--no-burst", action="store_true", help="skip the five spaced single steps reported beside the timed region")
    ap.add_argument("--top-p", type=float, default=0.0,
                    help="Stage 1 by Top-p instead of the workload's budget fraction (Sec. C.1: 0.95); not the headline config")
    args = ap.parse_args()
    if args.osk_impl == 5 and args.block_q != 256:
        ap.error("--osk-impl 5 walks the lists of --block-q 256")
    return args


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return {"hbm_gbs": d["hbm_gbs"], "bf16_tflops": d["bf16_tflops"],
                "bf16_tflops_sustained": d.get("bf16_tflops_sustained", d["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples SM clock and throttle reasons of one GPU with nvidia-smi while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.proc = None
        self.lines = []
        self.index = index

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "20"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.t = threading.Thread(target=self._read, daemon=True)
            self.t.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for ln in self.lines:
            parts = [x.strip() for x in ln.split(",")]
            if len(parts) < 8:
                continue
            try:
                sm.append(float(parts[0])); mx.append(float(parts[1]))
            except ValueError:
                continue
            for name, val in zip(names, parts[4:8]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def order_pitch(cosa, budget, nqb):
    return (cosa.cosa_budget_count(budget, nqb) + 7) // 8 * 8


def cpu_oracle_sample(w, qb, kb, vb, seconds_hint=20.0):
    """Times the fp64 oracle (as it stands) on a bounded sample of the workload: KAP lists and the
    OSK walk of a few (head, query block) pairs.  Returns visited-block TFLOP/s of the sample."""
    from oracle import cosa_oracle as O
    from synth.generator import bf16_bits_to_f64
    nqb = w.n_blocks
    G = w.hq // w.hkv
    heads = [g * G + (g % G) for g in range(w.hkv)] + [h for h in range(w.hq) if h % G != (h // G) % G]
    blocks = sorted(set(int(x) for x in np.linspace(nqb // 48, nqb - 1, 48)))
    t0 = time.perf_counter()
    flops = 0.0
    n_pairs = 0
    used = []
    for h in heads:
        g = h // G
        # widen one head at a time (the full tensors would need tens of GB in fp64); widening is timed too
        q1, k1, v1 = bf16_bits_to_f64(qb[h])[None], bf16_bits_to_f64(kb[g])[None], bf16_bits_to_f64(vb[g])[None]
        used.append(h)
        order, count = O.kap_select(q1, k1, s=w.stride, budget=w.kap_budget, query_blocks=blocks,
                                    order_stride=O.budget_count(w.kap_budget, nqb))
        r = O.osk_attention(q1, k1, v1, order, count, skip_scale=w.skip_scale, tightened_budget=w.osk_budget,
                            query_blocks=blocks)
        flops += BLOCK_FLOPS * float(r["scored"].sum() + r["visited"].sum())
        n_pairs += len(blocks)
        if time.perf_counter() - t0 > seconds_hint:
            break
    dt = time.perf_counter() - t0
    try:
        from threadpoolctl import threadpool_info
        cores = max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
    except Exception:
        cores = os.cpu_count()
    return {"value": flops / dt / 1e12, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"KAP lists + OSK walk of {n_pairs} (head, query block) pairs of {w.name}: heads {used} x "
                      f"{len(blocks)} query blocks evenly spaced in [{blocks[0]}, {blocks[-1]}], {dt:.1f} s of numpy fp64",
            "seconds": dt, "flops": flops}


def run_reference(args, rank, world):
    """The base contract's reference arm: here the fp64 oracle on the host cores."""
    if rank != 0:
        return
    from synth.configs import WORKLOADS
    w = WORKLOADS[args.workload]
    qb, kb, vb, _ = w.make()
    for _ in range(max(0, min(args.warmup, 1))):
        cpu_oracle_sample(w, qb, kb, vb, seconds_hint=5.0)
    tot_flops, tot_s, last = 0.0, 0.0, None
    for _ in range(args.steps):
        last = cpu_oracle_sample(w, qb, kb, vb, seconds_hint=max(5.0, 120.0 / max(args.steps, 1)))
        tot_flops += last["flops"]; tot_s += last["seconds"]
    value = tot_flops / tot_s / 1e12
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * tot_s / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": w.name, "hq": w.hq, "hkv": w.hkv, "seq_len": w.n, "kap_budget": w.kap_budget,
                       "osk_budget": w.osk_budget, "stride": w.stride, "skip_scale": w.skip_scale,
                       "note": "each step is a bounded sample of the workload run by the fp64 oracle on host cores"},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": last["cores"], "kind": "oracle",
                             "sample": last["sample"]},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def main():
    args = parse()
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if args.impl == "reference":
        run_reference(args, rank, world)
        return

    import torch
    import torch.distributed as dist
    from paper_2607_25291_b200 import build as _build
    if rank == 0 or world == 1:
        _build.build()
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        torch.cuda.set_device(local_rank)
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
        dist.barrier()
    else:
        torch.cuda.set_device(0)
    import paper_2607_25291_b200 as cosa
    from synth.configs import WORKLOADS
    dev = torch.device("cuda", local_rank if world > 1 else 0)
    w = WORKLOADS[args.workload]
    nqb = w.n_blocks

    # ---- synthetic inputs (rank r = its own layer of the same shape: independent problems)
    t_gen = time.perf_counter()
    import dataclasses
    hq_l, hkv_l = w.hq, w.hkv                               # heads this rank works on
    if args.shard == "kv_head":
        from paper_2607_25291_b200.shard import kv_head_shard
        if world > w.hkv:
            raise SystemExit(f"--shard kv_head: {world} ranks but only {w.hkv} KV heads")
        qb, kb, vb, _ = w.make(layer=0) if w.layers > 1 else w.make()       # the same layer on every rank ...
        kv_lo, kv_hi, q_lo, q_hi = kv_head_shard(w.hq, w.hkv, world, rank)
        qb, kb, vb = qb[q_lo:q_hi], kb[kv_lo:kv_hi], vb[kv_lo:kv_hi]          # ... of which it keeps its heads
        hq_l, hkv_l = q_hi - q_lo, kv_hi - kv_lo
    else:
        qb, kb, vb, _ = w.make(layer=rank) if w.layers > 1 else dataclasses.replace(w, seed=w.seed + rank).make()
    t_gen = time.perf_counter() - t_gen
    pin = lambda bits: torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16)[None].contiguous().pin_memory()
    qh, kh, vh = pin(qb), pin(kb), pin(vb)
    q, k, v = (t.to(dev, non_blocking=True) for t in (qh, kh, vh))
    kap_budget = 1.0 if args.top_p > 0 else w.kap_budget
    pitch = order_pitch(cosa, kap_budget, nqb)
    order = torch.empty(1, hq_l, nqb, pitch, dtype=torch.int32, device=dev)
    count = torch.empty(1, hq_l, nqb, dtype=torch.int32, device=dev)
    out = torch.empty_like(q)
    lse = torch.empty(1, hq_l, w.n, dtype=torch.float32, device=dev)
    visited = torch.empty(1, hq_l, nqb, dtype=torch.int32, device=dev)
    scored = torch.empty(1, hq_l, nqb, dtype=torch.int32, device=dev)
    opt = cosa.default_options(stride=w.stride, skip_scale=w.skip_scale, order_stride=pitch, out_scored=scored,
                               top_p=args.top_p, impl=args.osk_impl)
    stream = torch.cuda.current_stream()
    k_in, v_in = k, v
    if args.page_size > 0:
        # the same K and V as page pools behind a shuffled page table (layout only: a device-side copy)
        from synth.generator import scatter_to_pages
        kpool, table = scatter_to_pages(kb, args.page_size, seed=w.seed + 31)
        vpool, _ = scatter_to_pages(vb, args.page_size, seed=w.seed + 31)
        k_in = torch.from_numpy(kpool.view(np.int16)).view(torch.bfloat16).to(dev)
        v_in = torch.from_numpy(vpool.view(np.int16)).view(torch.bfloat16).to(dev)
        page_table = torch.from_numpy(table).to(dev)[None].contiguous()
        opt.kv_page_table = page_table.data_ptr()
        opt.kv_page_size = args.page_size
        opt.kv_pages_in_place = 1 if args.pages_in_place else 0
        opt.kv_num_pages = kpool.shape[0]

    def step():
        cosa.cosa_kap_select(q, k_in, kap_budget, order, count, opt=opt, stream=stream, block_q=args.block_q)
        cosa.cosa_osk_attention(q, k_in, v_in, order, count, w.osk_budget, out, lse, visited, opt=opt, stream=stream)

    def sync_all():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(args.warmup, 3)):
        step()
    torch.cuda.synchronize()
    if cosa.cosa_device_status() != 0:
        raise RuntimeError("device status reports a timed-out wait")
    n_scored, n_computed = int(scored.sum().item()), int(visited.sum().item())
    n_listed = int(count.sum().item())
    flops_step = BLOCK_FLOPS * (n_scored + n_computed)

    # ---- timed region: K steps, CUDA events on the launching stream, max over ranks
    sampler = ClockSampler(local_rank if world > 1 else 0)
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(args.steps)]
    sync_all()
    sampler.start()
    t_wall = time.perf_counter()
    for s in range(args.steps):
        ev[s][0].record(stream)
        cosa.cosa_kap_select(q, k_in, kap_budget, order, count, opt=opt, stream=stream, block_q=args.block_q)
        ev[s][1].record(stream)
        cosa.cosa_osk_attention(q, k_in, v_in, order, count, w.osk_budget, out, lse, visited, opt=opt, stream=stream)
        ev[s][2].record(stream)
    sync_all()
    t_wall = time.perf_counter() - t_wall
    clocks = sampler.stop()
    kap_ms = float(np.mean([e[0].elapsed_time(e[1]) for e in ev]))
    osk_ms = float(np.mean([e[1].elapsed_time(e[2]) for e in ev]))
    total_ms = ev[0][0].elapsed_time(ev[-1][2])
    if cosa.cosa_device_status() != 0:
        raise RuntimeError("device status reports a timed-out wait")
    from paper_2607_25291_b200.shard import reduce_job
    total_ms, job_flops_step = reduce_job(total_ms, flops_step, dev)      # max time, summed work over ranks
    ms_per_step = total_ms / args.steps
    value = job_flops_step / (ms_per_step * 1e-3) / 1e12

    # ---- end to end through the host-buffer entry point (H2D of q,k,v and D2H of the results in the timed region)
    e2e = None
    if not args.no_e2e:
        shape = cosa.make_shape(q, k, True)
        ws = torch.empty(cosa.cosa_host_call_workspace_bytes(shape, opt), dtype=torch.uint8, device=dev)
        out_h = torch.empty(q.shape, dtype=torch.bfloat16).pin_memory()
        lse_h = torch.empty(lse.shape, dtype=torch.float32).pin_memory()
        vis_h = torch.empty(visited.shape, dtype=torch.int32).pin_memory()
        ke = max(1, min(args.steps, 3))
        cosa.cosa_prefill_host(qh, kh, vh, shape, kap_budget, w.osk_budget, out_h, lse_h, vis_h, ws, opt=opt, stream=stream)
        sync_all()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(ke):
            cosa.cosa_prefill_host(qh, kh, vh, shape, kap_budget, w.osk_budget, out_h, lse_h, vis_h, ws, opt=opt, stream=stream)
        e1.record(stream)
        sync_all()
        e2e_ms = e0.elapsed_time(e1) / ke
        t = torch.tensor([e2e_ms], dtype=torch.float64, device=dev)
        if world > 1:
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
        h2d = (qh.numel() + kh.numel() + vh.numel()) * 2
        d2h = out_h.numel() * 2 + lse_h.numel() * 4 + vis_h.numel() * 4
        e2e = {"value": job_flops_step / (float(t[0]) * 1e-3) / 1e12, "unit": UNIT, "ms_per_step": float(t[0]),
               "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": ke}
        del ws

    # ---- the same step as a burst: five launches 50 ms apart, best of five.  The K back-to-back steps above pull the SM
    # clock down within some twenty launches (sw_power_cap; 1965 -> about 1750 MHz), while the burst GEMM peak the
    # roofline is set against was taken as a best-of-ten of single products at the full clock; this is the step measured
    # the same way, reported beside the timed region's figures, never in place of them.
    burst_run = None
    if rank == 0 and world == 1 and not args.no_burst:
        bk, bo = [], []
        for _ in range(5):
            torch.cuda.synchronize()
            time.sleep(0.05)
            e3 = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
            e3[0].record(stream)
            cosa.cosa_kap_select(q, k_in, kap_budget, order, count, opt=opt, stream=stream, block_q=args.block_q)
            e3[1].record(stream)
            cosa.cosa_osk_attention(q, k_in, v_in, order, count, w.osk_budget, out, lse, visited, opt=opt, stream=stream)
            e3[2].record(stream)
            torch.cuda.synchronize()
            bk.append(e3[0].elapsed_time(e3[1])); bo.append(e3[1].elapsed_time(e3[2]))
        burst_run = {"kap_ms": min(bk), "osk_ms": min(bo), "how": "best of 5 single steps 50 ms apart (SM clock at its maximum)"}

    # ---- rooflines (fractions "of measured" unless the peaks file is absent)
    peaks = measured_peaks()
    # Which measured GEMM figure a kernel is set against follows the length of the timed region: the burst figure
    # when the region is over before the power cap pulls the clock down (under ~2 s), else the sustained one.  The
    # other fractions are given alongside, and so is the share of cycles the tensor pipe was busy at the SM clock
    # sampled during the region (8192 dense bf16 FLOPs per SM and clock), which does not move with the power state.
    burst = t_wall < 2.0
    tensor_peak = peaks["bf16_tflops"] if burst else peaks["bf16_tflops_sustained"]
    peak_name = peaks["source"] + (" (burst bf16: timed region %.2f s)" % t_wall if burst else " (sustained bf16)")
    sms = torch.cuda.get_device_properties(dev).multi_processor_count
    pipe_peak = sms * 8192 * clocks["sm_mhz"] * 1e6 / 1e12 if clocks.get("sm_mhz") else None
    osk_tflops = flops_step / (osk_ms * 1e-3) / 1e12
    pairs = hq_l * (nqb * (nqb + 1) // 2)
    R = 128 // w.stride
    kap_flops = 2.0 * R * R * 128 * pairs
    kap_tflops = kap_flops / (kap_ms * 1e-3) / 1e12
    kap_bytes = (hq_l + hkv_l) * (w.n // w.stride) * 128 * 2 + order.numel() * 4 + count.numel() * 4
    traffic = None
    tpath = os.path.join(ROOT, "profiles", "dram_traffic.json")
    if os.path.exists(tpath):
        with open(tpath) as f:
            traffic = json.load(f)

    def tensor_roof(kernel, achieved, extra):
        r = {"kernel": kernel, "bound": "tensor", "achieved": achieved, "peak": tensor_peak, "unit": "TFLOP/s",
             "frac": achieved / tensor_peak, "peak_source": peak_name,
             "frac_of_burst": achieved / peaks["bf16_tflops"], "frac_of_sustained": achieved / peaks["bf16_tflops_sustained"],
             "frac_of_nominal_2250": achieved / 2250.0,
             "tensor_pipe_busy": achieved / pipe_peak if pipe_peak else None}
        r.update(extra)
        return r

    roof_osk = tensor_roof("osk_duo_kernel" if args.osk_impl in (4, 5) else "osk_tc_kernel", osk_tflops, {"traffic": (traffic or {}).get("osk_tc_kernel")})
    if burst_run:
        b_tflops = flops_step / (burst_run["osk_ms"] * 1e-3) / 1e12
        roof_osk["as_a_burst"] = {"ms": burst_run["osk_ms"], "achieved": b_tflops, "frac_of_burst": b_tflops / peaks["bf16_tflops"],
                                  "how": burst_run["how"]}
    # KAP: the screen kernel forms the sampled logits on the tensor cores (one pass over the key tiles; whole tiles,
    # so somewhat more than the causal pairs), the sort kernel is ALU work; the algorithmic FLOPs (causal pairs only)
    # are set against the tensor peak, and the algorithmic bytes (sampled rows read once, lists written once)
    # against the copy bandwidth
    roof_kap = tensor_roof("kap_screen_kernel+kap_sort_kernel", kap_tflops,
                           {"hbm_gbs_on_algorithmic_bytes": kap_bytes / (kap_ms * 1e-3) / 1e9,
                            "hbm_frac_of_measured": kap_bytes / (kap_ms * 1e-3) / 1e9 / peaks["hbm_gbs"],
                            "traffic": ((traffic or {}).get("kap_screen_kernel", 0) + (traffic or {}).get("kap_sort_kernel", 0)) or None})
    roofline = roof_osk if osk_ms >= kap_ms else roof_kap

    extras = {}
    if rank == 0 and world == 1 and not args.no_comparators:
        # the library's own dense path: full causal lists, Stage 2 off, same kernel
        full = torch.full((1, w.hq, nqb, nqb), -1, dtype=torch.int32, device=dev)
        tri = torch.arange(nqb, device=dev, dtype=torch.int32)
        full[:] = torch.where(tri[None, :] <= tri[:, None], tri[None, :].expand(nqb, nqb), torch.full((), -1, dtype=torch.int32, device=dev))
        fcount = (tri + 1).expand(1, w.hq, nqb).contiguous()
        dopt = cosa.default_options(order_stride=nqb)
        dense_out = torch.empty_like(q)
        def dense():
            cosa.cosa_osk_attention(q, k, v, full, fcount, 1.0, dense_out, None, None, opt=dopt, stream=stream)
        def sdpa():
            return torch.nn.functional.scaled_dot_product_attention(q, k, v, is_causal=True, enable_gqa=True)
        for name, fn in (("dense_path", dense), ("sdpa", sdpa)):
            try:
                fn(); torch.cuda.synchronize()
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record(stream); fn(); fn(); b.record(stream); torch.cuda.synchronize()
                ms = a.elapsed_time(b) / 2
                dense_flops = 2 * BLOCK_FLOPS * pairs
                extras[name] = {"ms": ms, "tflops": dense_flops / (ms * 1e-3) / 1e12, "speedup_of_cosa_path": ms / ms_per_step}
            except Exception as exc:  # a comparator must not take the benchmark down
                extras[name] = {"error": str(exc)[:200]}
        del full, dense_out

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        cpu = cpu_oracle_sample(w, qb, kb, vb)
        cpu = {k_: cpu[k_] for k_ in ("value", "unit", "cores", "kind", "sample")}

    if rank == 0:
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True,
                "scaling": "strong" if args.shard == "kv_head" else "weak",
                "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
                "config": {"workload": w.name, "hq": w.hq, "hkv": w.hkv, "seq_len": w.n, "head_dim": 128, "block": 128,
                           "kap_budget": kap_budget, "top_p": args.top_p or None, "kv_page_size": args.page_size or None, "kap_block_q": args.block_q, "osk_kernel": "osk_duo_kernel" if args.osk_impl in (4, 5) else "osk_tc_kernel", "osk_budget": w.osk_budget, "stride": w.stride,
                           "skip_scale": w.skip_scale,
                           "parallelism": (f"one layer, KV heads split over {world} ranks" if args.shard == "kv_head"
                                           else f"layer-per-rank x{world}"),
                           "l2": "inputs (%.1f GB) exceed L2; no flush" % ((q.numel() + k.numel() + v.numel()) * 2 / 1e9), "blocks_listed": n_listed,
                           "blocks_scored": n_scored, "blocks_computed": n_computed,
                           "causal_block_pairs": pairs, "input_generation_s": round(t_gen, 1)},
                "latency_ms": {"kap": kap_ms, "osk": osk_ms, "kap_plus_osk": ms_per_step},
                "latency_ms_as_a_burst": ({"kap": burst_run["kap_ms"], "osk": burst_run["osk_ms"], "how": burst_run["how"]} if burst_run else None),
                "e2e": e2e, "gpu_launches": 4 * args.steps, "clocks": clocks, "roofline": roofline,
                "roofline_osk": roof_osk, "roofline_kap": roof_kap, "cpu_baseline": cpu, "comparators": extras,
                "wall_s_timed_region": t_wall}
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
