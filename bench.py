#!/usr/bin/env python
"""Benchmark of Cartridge decode attention on B200 (one JSON line on stdout).

A "step" is one decode step of the whole hot path over one batch of synthetic input: for every
layer, append each request's new KV token and attend over [Cartridge(s) ; suffix] (projections,
MLP and sampling of a real model are outside the path and not timed).  Cartridges are registered
before the timed region (the paper's throughput protocol pre-loads them, App. A.3).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c2] [--impl ours|reference]

The headline (`value`, `roofline`, `e2e`, `cpu_baseline`) is the workload named by --workload (default: the
Llama-3B-shaped batch of 64 private Cartridges).  With the default workload on one GPU the line also carries
a `workloads` array: the other benchmark workloads measured one after the other in the same process with the
paper's protocol (3 warm-up steps, then 5 timed blocks; mean and min), and the memory / throughput comparison
of a 100 k-token in-context cache against a p = 2048 Cartridge.

N > 1 is launched with torch.distributed.run: every rank runs an independent replica on its own
GPU (the path has no exchange step), timing is the maximum over ranks.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

from paper_2506_06266_b200 import replicas, synth

METRIC = "decode_attention_tokens_per_s"
UNIT = "tokens/s"

WORKLOADS = {
    "c1": synth.config1, "c2": synth.config2, "c3": synth.config3, "c4": synth.config4,
    "c5_full": synth.config5_full, "c5_cartridge": synth.config5_cartridge,
}
SIDE_WORKLOADS = ["c1", "c3", "c4", "c5_cartridge", "c5_full"]   # reported next to the headline workload
TIMED_BLOCKS = 5                                                  # App. A.3: 3 warm-up runs, 5 timed runs

KERNEL_SOURCES = ["cart_kernels.cu", "cart_shared.cu", "cart_train.cu", "cart_tc.cuh", "cart_device.cuh", "cart_internal.h"]
TRAFFIC_TABLE = os.path.join(ROOT, "profiles", "dram_traffic.txt")


def kernel_source_sha() -> str:
    """Identifies the kernels' source: DRAM counters taken from another version are not reported."""
    h = hashlib.sha256()
    for name in KERNEL_SOURCES:
        with open(os.path.join(ROOT, "paper_2506_06266_b200", "csrc", name), "rb") as f:
            h.update(f.read())
    return h.hexdigest()[:16]


def dram_traffic_ratio(workload: str):
    """DRAM bytes per algorithmic byte of a workload's launch, from the table written next to the ncu
    summaries (lines: workload, kernel, dram bytes per launch, algorithmic bytes per launch of the captured
    case, source id).  None when the workload was not captured or the kernels have changed since."""
    try:
        with open(TRAFFIC_TABLE) as f:
            for line in f:
                parts = line.split()
                if len(parts) >= 5 and not line.startswith("#") and parts[0] == workload:
                    if parts[4] != kernel_source_sha():
                        return None
                    return float(parts[2]) / float(parts[3])
    except OSError:
        pass
    return None


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            d = json.load(f)
        return float(d["hbm_gbs"]), float(d["bf16_tflops"]), float(d["bf16_tflops_sustained"]), "measured"
    except Exception:
        return 6650.0, 1590.0, 1400.0, "fallback"


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.FIELDS,
                 "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            parts = [p.strip() for p in ln.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
            except ValueError:
                continue
            for name, val in zip(names, parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None,
                "sm_max_mhz": float(max(mx)) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# ------------------------------------------------------------------------------------------------
def oracle_sample(w: synth.Workload, lw, layers, q_host_bits, reps_target_s: float = 10.0):
    """Times the CPU oracle, as it stands, on `layers` of the loaded workload (all requests)."""
    import oracle
    segs = {layer: [lw.host_segments(layer, b) for b in range(w.batch)] for layer in layers}
    oracle.decode_layer(q_host_bits[layers[0]][:1], [segs[layers[0]][0]], w.scale)   # load the library
    t0 = time.perf_counter()
    reps = 0
    while True:
        for layer in layers:
            oracle.decode_layer(q_host_bits[layer], segs[layer], w.scale)
        reps += 1
        el = time.perf_counter() - t0
        if el >= reps_target_s or reps >= 400:
            break
    per_layer = el / (reps * len(layers))
    return {"value": w.batch / (per_layer * w.n_layers), "unit": UNIT, "cores": oracle.num_threads(),
            "kind": "oracle",
            "sample": "layers %s of %d, all %d requests, %d repetition(s), %.1f s of CPU time; "
                      "extrapolated to %d layers" % (list(layers), w.n_layers, w.batch, reps, el, w.n_layers),
            "s_per_layer": per_layer}


def workload_config(w: synth.Workload) -> dict:
    """What names the workload; the same keys in both arms' lines."""
    return {"workload": w.name, "batch_per_gpu": w.batch, "layers": w.n_layers, "q_heads": w.n_q_heads,
            "kv_heads": w.n_kv_heads, "head_dim": w.head_dim, "cartridge_tokens": w.p,
            "cartridges": w.cartridges, "suffix": "uniform[%d,%d]" % (w.suffix_lo, w.suffix_hi)}


def timed_steps(lw, tensors, steps: int, blocks: int, stream, fused: bool):
    """`steps` decode steps timed as `blocks` consecutive blocks with CUDA events on the launching stream at
    the block boundaries.  Returns (total ms, ms per step of every block, sum over the steps of the unique
    and of the logical bytes per layer)."""
    q, k_new, v_new, out, lse = tensors
    blocks = max(1, min(blocks, steps))
    sizes = [steps // blocks + (1 if i < steps % blocks else 0) for i in range(blocks)]
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(blocks + 1)]
    u0, l0 = lw.unique_bytes_per_layer(), lw.algorithmic_bytes_per_layer()
    ev[0].record(stream)
    for i, n in enumerate(sizes):
        for _ in range(n):
            lw.step(q, k_new, v_new, out, lse, fused=fused)
        ev[i + 1].record(stream)
    ev[-1].synchronize()
    # every step appends one token per request, so the bytes per layer grow linearly over the steps: the sum
    # over the steps (each counted with its own token already appended) follows from the two end points
    u1, l1 = lw.unique_bytes_per_layer(), lw.algorithmic_bytes_per_layer()
    uniq = steps * ((u0 + (u1 - u0) / steps) + u1) / 2
    logical = steps * ((l0 + (l1 - l0) / steps) + l1) / 2
    per_block = [ev[i].elapsed_time(ev[i + 1]) / sizes[i] for i in range(blocks)]
    return ev[0].elapsed_time(ev[-1]), per_block, uniq, logical


def roofline_entry(w, lw, ms, steps, uniq_sum, logical_sum, launches, workload_key, share_min=4):
    """HBM roofline on the bytes the method must move (every stored Cartridge once, every suffix once) and,
    where Cartridges are shared, the tensor-core side of the same launches."""
    L = w.n_layers
    hbm_peak, tf_burst, tf_sustained, kind = measured_peaks()
    period_s = ms * 1e-3 / (steps * L)                  # one layer's launches, gaps included
    uniq = uniq_sum / steps
    logical = logical_sum / steps
    achieved = uniq / period_s / 1e9
    shared_flops = lw.shared_flops_per_layer(share_min)
    kernels = ["cart_decode_kernel"]
    if shared_flops:
        kernels = ["cart_decode_kernel", "cart_shared_kernel"] + (["cart_merge_kernel"] if launches > 2 * steps * L else [])
    ratio = dram_traffic_ratio(workload_key)
    r = {"bound": "hbm", "achieved": round(achieved, 1), "peak": hbm_peak, "unit": "GB/s",
         "frac": round(achieved / hbm_peak, 4), "peak_kind": "of " + kind,
         "frac_of_8TBs_nominal": round(achieved / 8000.0, 4),
         "traffic": None if ratio is None else int(ratio * uniq),
         "kernel": "cart_decode_kernel", "kernels_per_launch_period": kernels,
         "launches_timed": steps * L,
         "timing": "CUDA events around the timed steps / decode calls (launch period of one layer, gaps included)",
         "avg_kernel_us": round(period_s * 1e6, 2),
         "algorithmic_bytes_per_launch": int(uniq),
         "bytes": "unique: every stored Cartridge of the batch once per layer, every suffix once, q/out/lse",
         "logical_gbs": round(logical / period_s / 1e9, 1), "logical_bytes_per_launch": int(logical)}
    if shared_flops:
        tf = shared_flops / period_s / 1e12
        r["tensor"] = {"bound": "tensor", "kernel": "cart_shared_kernel", "achieved": round(tf, 1),
                       "peak": tf_sustained, "unit": "TFLOP/s", "frac": round(tf / tf_sustained, 4),
                       "peak_kind": "of %s (sustained bf16; burst %.0f)" % (kind, tf_burst),
                       "flops_per_launch": int(shared_flops),
                       "timing": "the same launch period: the tensor-core kernel runs beside the stream kernel, "
                                 "so this is a lower bound of its own rate"}
    return r


def measure_side_workload(name: str, dev, stream, warmup: int, steps_per_block: int) -> dict:
    """One of the other benchmark workloads with the paper's protocol: `warmup` steps, then 5 timed blocks."""
    from paper_2506_06266_b200 import binding, runner
    w = WORKLOADS[name]()
    L, B = w.n_layers, w.batch
    free, _ = torch.cuda.mem_get_info(dev)
    steps = TIMED_BLOCKS * steps_per_block
    need = runner.arena_bytes_for(w, warmup + steps + 40) + (6 << 30)
    if free < need:
        return {"workload": w.name, "skipped": "needs %.0f GB of device memory, %.0f GB free" % (need / 1e9, free / 1e9)}
    lw = runner.LoadedWorkload(w, dev, extra_capacity=warmup + steps + 40, stream=stream)
    try:
        q = w.queries(0, dev)
        k_new, v_new = w.appended_kv(0, dev)
        out = torch.empty_like(q)
        lse = torch.empty((L, B, w.n_q_heads), dtype=torch.float32, device=dev)
        tensors = (q, k_new, v_new, out, lse)
        for _ in range(warmup):
            lw.step(*tensors)
        binding.cart_sync_status(lw.ctx, stream)
        sampler = ClockSampler(dev.index or 0)
        sampler.start()
        n0 = binding.cart_launch_count(lw.ctx)
        ms, per_block, uniq, logical = timed_steps(lw, tensors, steps, TIMED_BLOCKS, stream, True)
        launches = binding.cart_launch_count(lw.ctx) - n0
        clocks = sampler.stop()
        binding.cart_sync_status(lw.ctx, stream)
        roof = roofline_entry(w, lw, ms, steps, uniq, logical, launches, name)
        logical_b, private_b = binding.cart_kv_bytes(lw.ctx, lw.reqs[0])
        res = {"workload": w.name, "batch": B, "layers": L, "mean_kv_tokens": round(float(lw.kv_tokens().mean()), 1),
               "steps": steps, "warmup": warmup,
               "tokens_per_s": round(B * steps / (ms * 1e-3), 1),
               "tokens_per_s_best_block": round(B / (min(per_block) * 1e-3), 1),
               "us_per_layer_mean": round(float(np.mean(per_block)) * 1e3 / L, 2),
               "us_per_layer_min": round(min(per_block) * 1e3 / L, 2),
               "unique_gbs": roof["achieved"], "frac_of_hbm_peak": roof["frac"], "logical_gbs": roof["logical_gbs"],
               "kv_bytes_per_request": int(logical_b), "kv_bytes_private_per_request": int(private_b),
               "gpu_launches": int(launches), "clocks": clocks}
        if "tensor" in roof:
            res["tensor_tflops"] = roof["tensor"]["achieved"]
            res["tensor_frac"] = roof["tensor"]["frac"]
        if L == 1:
            res["single_call"] = single_call_latency(lw, tensors, stream, dev)
        res["recorded_loop"] = recorded_loop(lw, tensors, stream, dev, 30)
        return res
    finally:
        lw.close()
        torch.cuda.empty_cache()


def recorded_loop(lw, tensors, stream, dev, steps: int) -> dict:
    """The same decode steps as one CUDA graph per step: recorded once (cart_graph_begin / cart_graph_step), replayed
    `steps` times back to back; CUDA events around the replays.  Needs room for steps + 3 more tokens per request."""
    from paper_2506_06266_b200 import binding
    q, k_new, v_new, out, lse = tensors
    L = q.shape[0]
    side = torch.cuda.Stream(device=dev)
    side.wait_stream(stream)
    with torch.cuda.stream(side):
        binding.cart_graph_begin(lw.ctx, lw.req_list, steps + 3, side)
        side.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=side):
            for layer in range(L):
                binding.cart_graph_step(lw.ctx, layer, k_new[layer], v_new[layer], q[layer], out[layer], lse[layer], side)
        for _ in range(3):
            g.replay()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(side)
        for _ in range(steps):
            g.replay()
        b.record(side)
        b.synchronize()
    ms = a.elapsed_time(b)
    binding.cart_graph_end(lw.ctx, steps + 3)
    lw.appended += steps + 3
    binding.cart_sync_status(lw.ctx, stream)
    return {"what": "one CUDA graph per decode step (all layers), recorded once and replayed",
            "steps": steps, "us_per_step": round(ms * 1e3 / steps, 2), "us_per_layer": round(ms * 1e3 / steps / L, 2)}


def single_call_latency(lw, tensors, stream, dev) -> dict:
    """The single-layer workload: one decode call by itself, L2 warm and L2 cold."""
    from paper_2506_06266_b200 import binding
    q, _, _, out, lse = tensors
    ca, cb = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

    def one_call_us(flush):
        if flush is not None:
            flush.fill_(1)                       # 256 MB written: nothing of the KV is left in L2
        else:
            torch.cuda._sleep(200000)            # keeps the GPU busy while the host enqueues the call, as the
                                                 # fill does in the cold case: the events then bracket GPU time
        ca.record(stream)
        binding.cart_decode_attention(lw.ctx, 0, lw.req_list, q[0], out[0], lse[0], stream)
        cb.record(stream)
        cb.synchronize()
        return ca.elapsed_time(cb) * 1e3

    one_call_us(None)
    warm = [one_call_us(None) for _ in range(20)]
    flush_buf = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    cold = [one_call_us(flush_buf) for _ in range(5)]
    del flush_buf
    binding.cart_sync_status(lw.ctx, stream)
    return {"what": "one cart_decode_attention call, plan cached, CUDA events around the call",
            "warm_us_mean": round(sum(warm) / len(warm), 2), "warm_us_min": round(min(warm), 2),
            "cold_us_mean": round(sum(cold) / len(cold), 2), "cold_us_min": round(min(cold), 2)}


def run_ours(args):
    from paper_2506_06266_b200 import binding, runner
    rank, world, local = replicas.setup()
    dev = torch.device("cuda", local)
    torch.cuda.set_device(dev)
    w = WORKLOADS[args.workload]()
    if args.layers:
        w = synth.shrink(w, n_layers=args.layers)
    L, B = w.n_layers, w.batch
    total_steps = args.warmup + args.steps + (0 if args.no_e2e else args.warmup + args.e2e_steps) + 2
    sample_layers = list(range(min(args.cpu_layers, L))) if (rank == 0 and world == 1 and not args.no_cpu) else []
    stream = torch.cuda.current_stream(dev)
    lw = runner.LoadedWorkload(w, dev, extra_capacity=total_steps, keep_layers=sample_layers, stream=stream,
                               paged=args.paged)
    ctx = lw.ctx
    if args.piece_cost >= 0:
        binding.cart_set_piece_cost(ctx, args.piece_cost)
    if args.side_by_side >= 0:
        binding.cart_set_side_by_side(ctx, args.side_by_side)

    q = w.queries(0, dev)
    k_new, v_new = w.appended_kv(0, dev)
    out = torch.empty_like(q)
    lse = torch.empty((L, B, w.n_q_heads), dtype=torch.float32, device=dev)
    tensors = (q, k_new, v_new, out, lse)
    torch.cuda.synchronize(dev)

    # ---- device-resident timing: exactly --steps steps, as five blocks ---------------------------
    for _ in range(args.warmup):
        lw.step(*tensors, fused=not args.unfused)
    binding.cart_sync_status(ctx, stream)
    replicas.barrier(world)
    torch.cuda.synchronize(dev)
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    launches0 = binding.cart_launch_count(ctx)
    plans0 = binding.cart_plan_count(ctx)
    ms, per_block, uniq_sum, logical_sum = timed_steps(lw, tensors, args.steps, TIMED_BLOCKS, stream, not args.unfused)
    torch.cuda.synchronize(dev)
    replicas.barrier(world)
    clocks = sampler.stop() if rank == 0 else None
    launches = binding.cart_launch_count(ctx) - launches0
    plans = binding.cart_plan_count(ctx) - plans0
    binding.cart_sync_status(ctx, stream)
    value, ms_max = replicas.whole_job_tokens_per_s(B * args.steps, ms, world, dev)

    single_call = single_call_latency(lw, tensors, stream, dev) if (L == 1 and world == 1) else None
    roofline = roofline_entry(w, lw, ms, args.steps, uniq_sum, logical_sum, launches, args.workload)

    # ---- end to end through the C ABI from pinned host buffers -------------------------------
    e2e = None
    if not args.no_e2e:
        hq = q.cpu().pin_memory()
        hk, hv = k_new.cpu().pin_memory(), v_new.cpu().pin_memory()
        hout = torch.empty(out.shape, dtype=out.dtype).pin_memory()
        hlse = torch.empty(lse.shape, dtype=lse.dtype).pin_memory()
        # Double-buffered, as a server would run it: the inputs of step i+1 cross PCIe on a copy stream
        # while step i computes, and the result of step i goes back while step i+1 computes.  Every
        # step's host-to-device and device-to-host copies are inside the timed region.
        cs_in, cs_out = torch.cuda.Stream(dev), torch.cuda.Stream(dev)
        dq = [torch.empty_like(q) for _ in range(2)]
        dk = [torch.empty_like(k_new) for _ in range(2)]
        dv = [torch.empty_like(v_new) for _ in range(2)]
        dout = [torch.empty_like(out) for _ in range(2)]
        dlse = [torch.empty_like(lse) for _ in range(2)]
        ev_in = [torch.cuda.Event() for _ in range(2)]
        ev_done = [torch.cuda.Event() for _ in range(2)]
        ev_out = [torch.cuda.Event() for _ in range(2)]

        def e2e_steps(n, start_ev):
            for i in range(n):
                b = i & 1
                with torch.cuda.stream(cs_in):
                    cs_in.wait_event(ev_done[b] if i >= 2 else start_ev)   # step i-2 has consumed buffer b
                    dq[b].copy_(hq, non_blocking=True)
                    dk[b].copy_(hk, non_blocking=True)
                    dv[b].copy_(hv, non_blocking=True)
                    ev_in[b].record(cs_in)
                stream.wait_event(ev_in[b])
                if i >= 2:
                    stream.wait_event(ev_out[b])                           # step i-2's result has left buffer b
                for layer in range(L):
                    if args.unfused:
                        binding.cart_append_kv(ctx, layer, lw.req_list, dk[b][layer], dv[b][layer], stream)
                        binding.cart_decode_attention(ctx, layer, lw.req_list, dq[b][layer], dout[b][layer],
                                                      dlse[b][layer], stream)
                    else:
                        binding.cart_decode_step(ctx, layer, lw.req_list, dk[b][layer], dv[b][layer], dq[b][layer],
                                                 dout[b][layer], dlse[b][layer], stream)
                ev_done[b].record(stream)
                with torch.cuda.stream(cs_out):
                    cs_out.wait_event(ev_done[b])
                    hout.copy_(dout[b], non_blocking=True)
                    hlse.copy_(dlse[b], non_blocking=True)
                    ev_out[b].record(cs_out)
                lw.appended += 1
            for b in range(min(n, 2)):
                stream.wait_event(ev_out[b])                               # the region ends when the results are home

        w0 = torch.cuda.Event()
        w0.record(stream)
        e2e_steps(args.warmup, w0)
        torch.cuda.synchronize(dev)
        replicas.barrier(world)
        f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        f0.record(stream)
        e2e_steps(args.e2e_steps, f0)
        f1.record(stream)
        torch.cuda.synchronize(dev)
        replicas.barrier(world)
        e2e_value, ems = replicas.whole_job_tokens_per_s(B * args.e2e_steps, f0.elapsed_time(f1), world, dev)
        h2d = L * (hq[0].numel() * 2 + hk[0].numel() * 2 + hv[0].numel() * 2)
        d2h = L * (hout[0].numel() * 2 + hlse[0].numel() * 4)
        e2e = {"value": round(e2e_value, 1), "unit": UNIT,
               "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h), "steps": args.e2e_steps,
               "pipeline": "double-buffered: copies of neighbouring steps overlap the kernels on two copy streams",
               "ms_per_step": round(ems / args.e2e_steps, 4)}
        binding.cart_sync_status(ctx, stream)

    # ---- CPU oracle on a bounded sample (rank 0, N = 1 only) ---------------------------------
    cpu = None
    if sample_layers:
        cpu = oracle_sample(w, lw, sample_layers, synth.bits(q))
        cpu["value"] = round(cpu["value"], 3)

    logical, private = binding.cart_kv_bytes(ctx, lw.reqs[0])
    kv_tokens = lw.kv_tokens()
    lw.close()
    del tensors, q, k_new, v_new, out, lse
    torch.cuda.empty_cache()

    # ---- the other workloads and the in-context-cache comparison (default run on one GPU only) --------
    side, comparison = None, None
    if world == 1 and not args.no_side and args.workload == "c2" and not args.layers:
        side = []
        for name in SIDE_WORKLOADS:
            n = {"c1": 40, "c3": 4, "c4": 4, "c5_cartridge": 2, "c5_full": 2}[name]
            side.append(measure_side_workload(name, dev, stream, 3, n))
        by = {s["workload"]: s for s in side}
        full, cart = by.get(synth.config5_full().name), by.get(synth.config5_cartridge().name)
        if full and cart and "skipped" not in full and "skipped" not in cart:
            comparison = {"what": "in-context KV cache of 100 000 tokens at batch 8 against a Cartridge of p = 2048 at "
                                  "batch 256, Llama-8B attention shapes, same GPU",
                          "kv_bytes_per_request_ratio": round(full["kv_bytes_per_request"] / cart["kv_bytes_per_request"], 2),
                          "tokens_per_s_ratio": round(cart["tokens_per_s"] / full["tokens_per_s"], 2),
                          "paper_context": "38.6x less memory, 26.4x more tokens/s on 1xH100 with a serving stack "
                                           "(whole model, not attention alone)"}
    if world > 1:
        replicas.barrier(world)
        replicas.shutdown()
    if rank != 0:
        return
    cfg = workload_config(w)
    if args.paged:
        cfg["suffix_storage"] = "pages of 64 tokens, taken as the suffixes grow"
    cfg.update({"mean_kv_tokens": round(float(kv_tokens.mean()), 1),
                "step": ("per layer: cart_append_kv, then cart_decode_attention" if args.unfused else
                         "per layer: cart_decode_step (append 1 KV token per request and attend, one call)"),
                "l2": "inputs larger than L2 (%.0f MB of KV per layer, %.1f GB per step)"
                      % (roofline["algorithmic_bytes_per_launch"] / 1e6, roofline["algorithmic_bytes_per_launch"] * L / 1e9),
                "parallelism": "replicas only" if world > 1 else "single GPU",
                "attention_us_per_layer": round(ms_max * 1e3 / args.steps / L, 2),
                "kv_bytes_per_request": int(logical), "kv_bytes_private_per_request": int(private)})
    line = {
        "metric": METRIC, "value": round(value, 1), "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": round(ms_max / args.steps, 4), "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic", "config": cfg,
        "repeats": {"blocks": len(per_block), "protocol": "warm-up steps, then the timed steps as consecutive blocks "
                                                          "(App. A.3: 3 warm-up and 5 timed runs)",
                    "ms_per_step_mean": round(float(np.mean(per_block)), 4),
                    "ms_per_step_min": round(min(per_block), 4),
                    "tokens_per_s_best_block": round(B * world / (min(per_block) * 1e-3), 1)},
        "roofline": roofline, "cpu_baseline": cpu, "e2e": e2e, "gpu_launches": int(launches),
        "plans_built_in_timed_region": int(plans), "clocks": clocks,
        **({"single_call": single_call} if single_call else {}),
        **({"workloads": side} if side is not None else {}),
        **({"comparison_100k_context_vs_cartridge": comparison} if comparison else {}),
    }
    print(json.dumps(line))


def run_prefill(args):
    """Side measurement (its own JSON line, not the headline): prefill attention of a T-token message over a
    Cartridge of the chosen workload's shape -- cart_extend_kv of the message's KV, then
    cart_prefill_attention, per layer."""
    from paper_2506_06266_b200 import binding, runner
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    w0 = WORKLOADS[args.workload]()
    T, s_old = args.prefill, 256
    w = synth.shrink(w0, batch=1, suffix_lo=s_old, suffix_hi=s_old, cartridges="private" if w0.p else "none")
    if args.layers:
        w = synth.shrink(w, n_layers=args.layers)
    L = w.n_layers
    stream = torch.cuda.current_stream(dev)
    reps = args.warmup + args.steps
    cfg = binding.make_config(L, w.n_q_heads, w.n_kv_heads, max(T, 4), 4, device=0, softmax_scale=w.scale)
    per_tok = L * w.kv_bytes_per_token_layer()
    arena_bytes = binding.cart_scratch_bytes(cfg) + (w.p + s_old + reps * T + 128) * per_tok + 4096
    arena = torch.empty(arena_bytes, dtype=torch.uint8, device=dev)
    cfg.arena, cfg.arena_bytes = arena.data_ptr(), arena_bytes
    ctx = binding.cart_create(cfg)
    k, v = w.cartridge_kv(0, dev)
    cart = binding.cart_register_cartridge(ctx, k, v, w.p, stream)
    if args.prefill_split >= 0:
        binding.cart_set_prefill_split(ctx, args.prefill_split)
    req = binding.cart_request_open(ctx, cart, s_old + reps * T)
    ks, vs = w.suffix_kv(0, s_old, dev)
    for layer in range(L):
        binding.cart_extend_kv(ctx, layer, req, ks[layer], vs[layer], s_old, stream)
    km, vm = w.suffix_kv(1, T, dev)                                   # the message's K and V, [L][T][Hkv][D]
    q = synth.normal_bf16((L, T, w.n_q_heads, 128), w.seed + 77, dev)
    out = torch.empty_like(q)

    def step():
        for layer in range(L):
            binding.cart_extend_kv(ctx, layer, req, km[layer], vm[layer], T, stream)
            binding.cart_prefill_attention(ctx, layer, req, q[layer], T, out[layer], None, stream)

    for _ in range(args.warmup):
        step()
    binding.cart_sync_status(ctx, stream)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    n0 = binding.cart_launch_count(ctx)
    e0.record(stream)
    for _ in range(args.steps):
        step()
    e1.record(stream)
    torch.cuda.synchronize(dev)
    binding.cart_sync_status(ctx, stream)
    ms = e0.elapsed_time(e1)
    launches = binding.cart_launch_count(ctx) - n0
    # the message grows the suffix by T per step: mean context of a row over the timed steps
    mean_ctx = w.p + s_old + (args.warmup + (args.steps - 1) / 2.0) * T + (T + 1) / 2.0
    flops = 4.0 * w.n_q_heads * 128 * mean_ctx * T                    # per layer
    us_layer = ms * 1e3 / args.steps / L
    _, tf_burst, tf_sustained, kind = measured_peaks()
    tflops = flops / (us_layer * 1e-6) / 1e12
    binding.cart_destroy(ctx)
    print(json.dumps({"metric": "prefill_attention_tokens_per_s", "value": round(T * args.steps / (ms * 1e-3), 1),
                      "unit": "tokens/s", "n_gpus": 1, "steps": args.steps, "warmup": args.warmup,
                      "ms_per_step": round(ms / args.steps, 4), "higher_is_better": True, "dtype": "bf16",
                      "data": "synthetic",
                      "config": {"workload": "prefill of %d tokens over %s shapes" % (T, w0.name), "layers": L,
                                 "cartridge_tokens": w.p, "suffix_before": s_old, "mean_context": round(mean_ctx, 1),
                                 "attention_us_per_layer": round(us_layer, 2),
                                 "tflops": round(tflops, 2)},
                      "roofline": {"bound": "tensor", "achieved": round(tflops, 1), "peak": tf_sustained,
                                   "unit": "TFLOP/s", "frac": round(tflops / tf_sustained, 4),
                                   "peak_kind": "of %s (sustained bf16)" % kind, "traffic": None},
                      "gpu_launches": int(launches)}))


def run_train(args):
    """Side measurement (its own JSON line, not the headline): one layer of training-time attention over a shared
    trainable Cartridge -- args.train conversations of 64 .. 512 tokens (seeded) over a Cartridge of the chosen
    workload's shape, cart_train_attention_fwd and cart_train_attention_bwd timed separately."""
    from paper_2506_06266_b200 import binding
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    w0 = WORKLOADS[args.workload]()
    Hq, Hkv, p = w0.n_q_heads, w0.n_kv_heads, w0.p
    lens = [int(x) for x in np.random.default_rng(w0.seed + 5).integers(64, 513, size=args.train)]
    T = int(sum(lens))
    cu = np.concatenate([[0], np.cumsum(lens)])
    stream = torch.cuda.current_stream(dev)
    cfg = binding.make_config(1, Hq, Hkv, T, 4, device=0, softmax_scale=w0.scale)
    per_tok = 2 * Hkv * 256
    arena_bytes = binding.cart_scratch_bytes(cfg) + (p + sum(-(-n // 64) * 64 for n in lens) + 128) * per_tok + 4096
    arena = torch.empty(arena_bytes, dtype=torch.uint8, device=dev)
    cfg.arena, cfg.arena_bytes = arena.data_ptr(), arena_bytes
    ctx = binding.cart_create(cfg)
    zk = synth.normal_bf16((1, Hkv, p, 128), w0.seed + 71, dev)
    zv = synth.normal_bf16((1, Hkv, p, 128), w0.seed + 72, dev)
    cart = binding.cart_register_cartridge(ctx, zk, zv, p, stream)
    k = synth.normal_bf16((T, Hkv, 128), w0.seed + 73, dev)
    v = synth.normal_bf16((T, Hkv, 128), w0.seed + 74, dev)
    q = synth.normal_bf16((T, Hq, 128), w0.seed + 75, dev)
    dout = synth.normal_bf16((T, Hq, 128), w0.seed + 76, dev)
    convs = []
    for c, n in enumerate(lens):
        r = binding.cart_request_open(ctx, cart, n)
        binding.cart_extend_kv(ctx, 0, r, k[cu[c]:cu[c + 1]], v[cu[c]:cu[c + 1]], n, stream)
        convs.append(r)
    convs = binding.ReqList(convs)
    out = torch.empty_like(q)
    lse = torch.empty((T, Hq), dtype=torch.float32, device=dev)
    delta = torch.empty_like(lse)
    dq = torch.empty((T, Hq, 128), dtype=torch.float32, device=dev)
    dk = torch.empty((T, Hkv, 128), dtype=torch.float32, device=dev)
    dv = torch.empty_like(dk)
    dzk = torch.empty((Hkv, p, 128), dtype=torch.float32, device=dev)
    dzv = torch.empty_like(dzk)

    def fwd():
        binding.cart_train_attention_fwd(ctx, 0, convs, q, out, lse, stream)

    def bwd():
        binding.cart_train_attention_bwd(ctx, 0, convs, q, out, lse, dout, delta, dq, dk, dv, dzk, dzv, stream)

    times = {}
    n0 = binding.cart_launch_count(ctx)
    for name, fn in (("fwd", fwd), ("bwd", bwd)):
        for _ in range(args.warmup):
            fn()
        binding.cart_sync_status(ctx, stream)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(args.steps):
            fn()
        e1.record(stream)
        torch.cuda.synchronize(dev)
        binding.cart_sync_status(ctx, stream)
        times[name] = e0.elapsed_time(e1) / args.steps
    launches = binding.cart_launch_count(ctx) - n0
    binding.cart_destroy(ctx)
    # a token of a conversation sees the Cartridge and its own conversation up to itself: 2 products forward, 5 backward
    pairs = float(T) * p + sum(n * (n + 1) / 2.0 for n in lens)
    flops_fwd = 4.0 * Hq * 128 * pairs
    flops_bwd = 10.0 * Hq * 128 * pairs
    _, tf_burst, tf_sustained, kind = measured_peaks()
    tf = {"fwd": flops_fwd / (times["fwd"] * 1e-3) / 1e12, "bwd": flops_bwd / (times["bwd"] * 1e-3) / 1e12}
    total_ms = times["fwd"] + times["bwd"]
    print(json.dumps({"metric": "train_attention_tokens_per_s", "value": round(T / (total_ms * 1e-3), 1),
                      "unit": "tokens/s", "n_gpus": 1, "steps": args.steps, "warmup": args.warmup,
                      "ms_per_step": round(total_ms, 4), "higher_is_better": True, "dtype": "bf16", "data": "synthetic",
                      "config": {"workload": "one layer of training attention, %d conversations of 64..512 tokens over a "
                                             "Cartridge of %s shape" % (args.train, w0.name),
                                 "tokens": T, "cartridge_tokens": p, "q_heads": Hq, "kv_heads": Hkv,
                                 "fwd_ms": round(times["fwd"], 4), "bwd_ms": round(times["bwd"], 4),
                                 "fwd_tflops": round(tf["fwd"], 1), "bwd_tflops": round(tf["bwd"], 1)},
                      "roofline": {"bound": "tensor", "kernel": "cart_train_bwd_kernel", "achieved": round(tf["bwd"], 1),
                                   "peak": tf_sustained, "unit": "TFLOP/s", "frac": round(tf["bwd"] / tf_sustained, 4),
                                   "peak_kind": "of %s (sustained bf16)" % kind, "traffic": None},
                      "gpu_launches": int(launches)}))


def run_reference(args):
    """The reference arm is the CPU oracle, as it stands, timed on the host cores."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    w = WORKLOADS[args.workload]()
    L, B = w.n_layers, w.batch
    n_layers = min(args.ref_layers, L)
    suffix = w.suffix_lengths()
    parts = w.request_parts()
    # the same seeded inputs as the GPU arm, generated on the host for the sampled layers only
    carts = {}
    for b in range(B):
        for c in parts[b]:
            if c not in carts:
                k, v = synth.shrink(w, n_layers=n_layers).cartridge_kv(c, "cpu")
                carts[c] = (synth.bits(k), synth.bits(v))
    segs = [[] for _ in range(n_layers)]
    ws = synth.shrink(w, n_layers=n_layers)
    for b in range(B):
        ks, vs = ws.suffix_kv(b, int(suffix[b]), "cpu")
        kb, vb = synth.bits(ks), synth.bits(vs)
        for layer in range(n_layers):
            s = [(carts[c][0][layer], carts[c][1][layer]) for c in parts[b]]
            s.append((np.ascontiguousarray(np.transpose(kb[layer], (1, 0, 2))),
                      np.ascontiguousarray(np.transpose(vb[layer], (1, 0, 2)))))
            segs[layer].append(s)
    q = synth.bits(ws.queries(0, "cpu"))

    def step():
        for layer in range(n_layers):
            oracle.decode_layer(q[layer], segs[layer], w.scale)

    for _ in range(args.warmup):
        step()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        step()
    el = time.perf_counter() - t0
    sample_ms = el / args.steps * 1e3                      # what one timed step (the sampled layers) took
    per_step_full = el / args.steps * (L / n_layers)
    value = B / per_step_full
    sample = ("each timed step = layers 0..%d of %d, all %d requests (inputs of the GPU arm's recipe, generated per "
              "sampled layer); ms_per_step is that sample's time, value is extrapolated to %d layers "
              "(%.1f ms per whole step)" % (n_layers - 1, L, B, L, per_step_full * 1e3))
    cfg = workload_config(w)
    cfg["sampled_layers_per_step"] = n_layers
    line = {"impl": "reference", "metric": METRIC, "value": round(value, 3), "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": round(sample_ms, 3),
            "ms_per_whole_step_extrapolated": round(per_step_full * 1e3, 3),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic", "config": cfg,
            "cpu_baseline": {"value": round(value, 3), "unit": UNIT, "cores": oracle.num_threads(),
                             "kind": "oracle", "sample": sample},
            "e2e": {"value": round(value, 3), "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c2", choices=sorted(WORKLOADS))
    ap.add_argument("--layers", type=int, default=0, help="override the layer count (profiling small cases)")
    ap.add_argument("--e2e-steps", type=int, default=50)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu", action="store_true")
    ap.add_argument("--no-side", action="store_true",
                    help="skip the other workloads that the default run reports next to the headline")
    ap.add_argument("--prefill", type=int, default=0,
                    help="side measurement: prefill attention of a message of this many tokens over one Cartridge "
                         "of the workload's shape (prints its own JSON line)")
    ap.add_argument("--train", type=int, default=0,
                    help="side measurement: training-time attention (forward and backward) of this many conversations "
                         "over one Cartridge of the workload's shape, one layer")
    ap.add_argument("--paged", action="store_true",
                    help="the requests' suffixes are stored in pages of 64 tokens (cart_request_open_paged)")
    ap.add_argument("--unfused", action="store_true",
                    help="append and attend with two calls per layer instead of cart_decode_step")
    ap.add_argument("--prefill-split", type=int, default=-1,
                    help="pieces a short message's chains are cut into (cart_set_prefill_split); -1 keeps the library's choice")
    ap.add_argument("--piece-cost", type=int, default=-1,
                    help="planner tuning (cart_set_piece_cost); -1 keeps the library's default")
    ap.add_argument("--side-by-side", type=int, default=-1,
                    help="planner tuning (cart_set_side_by_side): 0 = shared and stream kernel one after the other, "
                         "1 = side by side with the planner's division, N > 1 = N blocks for the shared kernel; "
                         "-1 keeps the library's default")
    ap.add_argument("--cpu-layers", type=int, default=4, help="layers the CPU oracle sample covers")
    ap.add_argument("--ref-layers", type=int, default=2, help="layers per step of the reference arm")
    ap.add_argument("--kernel-sha", action="store_true",
                    help="print the id of the kernels' source that profiles/dram_traffic.txt records, and exit")
    args = ap.parse_args()
    if args.kernel_sha:
        print(kernel_source_sha())
        return
    if args.warmup < 3 and args.impl == "ours":
        args.warmup = 3
    if args.prefill > 0:
        run_prefill(args)
    elif args.train > 0:
        run_train(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
