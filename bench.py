#!/usr/bin/env python
"""Benchmark of the multi-tenant MoE layer hot path (route -> dispatch -> experts -> combine).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload decode|prefill|pool|stack] [--impl reference]

One step is one pass of the whole layer (for `stack`: of the 24 blocks) over one batch of seeded synthetic
tokens at the Qwen1.5-MoE layer shape.  A timed block is exactly K steps between a barrier + device synchronise on
both sides; blocks are repeated until at least --min-time seconds have been timed, and the MEDIAN block gives
`ms_per_step` (the first, fastest and slowest blocks and the clocks sampled meanwhile are printed beside it), so a
burst of a few milliseconds on a cold part cannot stand for the step time.

Without --workload the headline line is the 32-token decode layer and the same JSON line carries the other
workloads (prefill, pool, stack) under "workloads".  With N > 1 every rank runs an independent replica on its own
batch (the layer has no exchange step), time is the maximum over ranks and the value the aggregate tokens/s;
`--gpus N` starts its own ranks (one process per GPU) unless a launcher already did.  Rank 0 prints one JSON line.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import math
import os
import socket
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import torch

from paper_2604_26881_b200 import replicas
from paper_2604_26881_b200 import workloads as W

METRIC = "MoE-layer tokens/s at Qwen1.5-MoE shape on 1 B200"
UNIT = "tokens/s"
DEFAULT_STEPS = {"decode": 1000, "prefill": 200, "pool": 100, "stack": 20}
EXTRA_WORKLOADS = ("prefill", "pool", "stack")     # measured beside the headline when no --workload is given


def parse_args(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--workload", default=None, choices=["decode", "prefill", "pool", "stack"],
                    help="one workload only; default: decode as the headline and the others under 'workloads'")
    ap.add_argument("--min-time", type=float, default=1.5,
                    help="seconds of timed blocks per workload (each block is exactly --steps steps)")
    ap.add_argument("--impl", default="b200", choices=["b200", "reference"])
    ap.add_argument("--path", default="auto", choices=["auto", "fma", "tcgen05"])
    ap.add_argument("--pair", default="auto", choices=["auto", "never"])
    ap.add_argument("--early-shared", default="auto", choices=["auto", "0", "1", "2"],
                    help="shared expert on the context's second stream (auto: the library's default, batches of more than 64 tokens); "
                         "the per-stage times and the roofline block always come from passes without it, where one "
                         "grouped-GEMM launch holds the shared and the routed units")
    ap.add_argument("--background", default="auto", choices=["auto", "0", "1", "2"],
                    help="background lanes of the 2-CTA grouped GEMM for short tiles (auto: the library's default)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--dry", action="store_true",
                    help="exercise the launch and reduction protocol without a GPU (gloo ranks, a sleep as the step)")
    return ap.parse_args(argv)


def _free_port() -> int:
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def spawn_ranks(n: int) -> int:
    """Re-runs this command line as n ranks (one process per GPU) under torch.distributed.run."""
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
           "--master-addr", "127.0.0.1", "--master-port", str(_free_port()), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd)


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            d = json.load(f)
        return {"hbm_gbs": float(d["hbm_gbs"]), "bf16_tflops": float(d["bf16_tflops"]),
                "bf16_tflops_sustained": float(d.get("bf16_tflops_sustained", d["bf16_tflops"])), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs (read-only queries)."""

    FIELDS = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.gpu}", f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()          # the exact process started above
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, smax, power, reasons = [], [], [], set()
        try:
            with open(self.path) as f:
                for line in f:
                    c = [v.strip() for v in line.split(",")]
                    if len(c) < 9:
                        continue
                    try:
                        sm.append(float(c[1])); smax.append(float(c[2]))
                        power.append(float(c[3]))
                    except ValueError:
                        continue
                    for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"),
                                       c[5:9]):
                        if v.lower().startswith("active"):
                            reasons.add(name)
            os.unlink(self.path)
        except Exception:
            pass
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_min_mhz=min(sm), sm_max_mhz=max(smax), samples=len(sm))
        if power:
            out["power_w_median"] = statistics.median(power)
        out["reasons"] = sorted(reasons)
        return out


def timed_blocks(step_fn, steps: int, min_time_s: float, world: int, sync, dev, make_events, max_blocks: int = 5000):
    """Times blocks of exactly `steps` calls of step_fn, each between a barrier + synchronise on both sides, until
    min_time_s seconds have been timed (every rank runs the same number of blocks: the slowest rank's first block
    decides).  Returns per-block durations in ms, already reduced to the maximum over ranks."""
    def one_block():
        replicas.barrier(world, sync)
        e0, e1 = make_events()
        e0.record()
        for _ in range(steps):
            step_fn()
        e1.record()
        replicas.barrier(world, sync)
        return e0.elapsed_time(e1)

    blocks = [one_block()]
    first = replicas.max_over_ranks([blocks[0]], world, dev)[0]
    n_more = int(min(max_blocks, math.ceil(max(0.0, min_time_s * 1e3 - first) / max(first, 1e-3))))
    for _ in range(n_more):
        blocks.append(one_block())
    return replicas.max_over_ranks(blocks, world, dev)


def block_summary(blocks_ms, steps: int) -> dict:
    return {"n": len(blocks_ms), "steps_per_block": steps, "median_ms": statistics.median(blocks_ms),
            "first_ms": blocks_ms[0], "min_ms": min(blocks_ms), "max_ms": max(blocks_ms), "timed_s": sum(blocks_ms) * 1e-3}


def kernel_source_digest() -> str:
    """SHA-256 over the grouped-GEMM sources: a DRAM-traffic figure taken from a profile is only quoted while the
    kernel it was measured on is still the one that runs."""
    h = hashlib.sha256()
    for name in ("experts_tc.cu", "tc_ptx.cuh", "plan.cuh"):
        with open(os.path.join(ROOT, "paper_2604_26881_b200", "csrc", name), "rb") as f:
            h.update(f.read())
    return h.hexdigest()[:16]


# DRAM traffic (dram__bytes_read.sum + dram__bytes_write.sum) of one launch of the dominant kernel, copied from the
# ncu summaries under profiles/ together with the digest of the kernel sources they were captured on.  bench.py prints
# the figure only while kernel_source_digest() still equals `digest`; otherwise `traffic` is null.
NCU_TRAFFIC = {
    "decode": {"bytes": 678.723072e6 + 3.447552e6, "digest": "767af1952e5f6102",
               "source": "profiles/grouped_gemm_decode_ncu.md (gate/up launch, dram__bytes_read.sum + dram__bytes_write.sum; 23.07 MB of it are the shared expert's down weights pulled into L2 for the next launch)"},
    "prefill": {"bytes": 929.690624e6 + 84.762112e6, "digest": "767af1952e5f6102",
                "source": "profiles/grouped_gemm_prefill_ncu.md (merged gate/up launch, dram__bytes_read.sum + dram__bytes_write.sum)"},
    "pool": {"bytes": 2996.817152e6 + 38.470656e6, "digest": "767af1952e5f6102",
             "source": "profiles/grouped_gemm_pool_dram.md (merged gate/up launch, dram__bytes_read.sum + dram__bytes_write.sum)"},
}


def traffic_record(workload: str, path: str):
    rec = NCU_TRAFFIC.get(workload)
    if rec is None or path != "auto":
        return None, None
    if rec["digest"] != kernel_source_digest():
        return None, f"{rec['source']} (stale: the kernel sources have changed since that capture)"
    return rec["bytes"], rec["source"]


def algorithmic_work(wl, active_experts: int, T: int):
    """Bytes and FLOPs the method itself must move / compute for one layer pass."""
    H, I, Is, E, k = wl.H, wl.I, wl.Is, wl.E, wl.k
    expert_bytes = 3 * H * I * 2
    shared_bytes = 3 * H * Is * 2 * wl.M
    router_bytes = (E * H * 2 + H * 2) * wl.M
    act_bytes = 2 * T * H * 2
    total_bytes = active_experts * expert_bytes + shared_bytes + router_bytes + act_bytes
    flops = T * (k * 6 * H * I + 6 * H * Is + 2 * H * E)
    # the gate/up grouped GEMM (the dominant kernel): two of the three matrices of every active expert
    gateup_bytes = active_experts * 2 * H * I * 2 + 2 * H * Is * 2 * wl.M + (T * k + T) * H * 2
    gateup_flops = T * (k * 4 * H * I + 4 * H * Is)
    return dict(total_bytes=total_bytes, flops=flops, gateup_bytes=gateup_bytes, gateup_flops=gateup_flops)


def oracle_sample(wl, wts, x, tenant, mot):
    """Inputs of the oracle's timed sample: the first 32 tokens of the batch."""
    n = min(x.shape[0], 32)
    xs, ts = x[:n].contiguous(), tenant[:n].contiguous()
    return n, W.as_u16(xs), ts.numpy(), mot.numpy(), W.weights_as_numpy(wts)


def run_reference(args, rank):
    """The oracle, as it stands, on the host cores: each step is a bounded sample of the workload."""
    import oracle
    if rank != 0:
        return
    wl = W.WORKLOADS[args.workload or "decode"]
    steps = args.steps if args.steps is not None else 3
    warmup = args.warmup if args.warmup is not None else 1
    steps, warmup = min(steps, 10), min(warmup, 2)      # bounded: each pass is about a second of CPU work
    wts = W.make_weights(wl, seed=0)
    x, tenant, mot = W.make_tokens(wl, seed=0)
    n, xu, ts, mn, wn = oracle_sample(wl, wts, x, tenant, mot)
    times = []
    for i in range(warmup + steps):
        t0 = time.perf_counter()
        oracle.layer_forward(xu, ts, mn, wn, k=wl.k, G=wl.G)
        if i >= warmup:
            times.append(time.perf_counter() - t0)
    total = sum(times)
    value = n * steps / total
    cores = oracle.num_threads()
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": steps,
            "warmup": warmup, "ms_per_step": 1e3 * total / steps, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": wl.name, "tokens_per_step": n, "note": "CPU oracle on a sample of the batch"},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle",
                             "sample": f"first {n} tokens of the {wl.name} batch, {steps} passes"},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


def cpu_baseline(wl, wts, x, tenant, mot):
    """The oracle timed on the host cores on a bounded sample of the same batch."""
    import oracle
    n, xu, ts, mn, wn = oracle_sample(wl, wts, x, tenant, mot)
    oracle.layer_forward(xu[:2], ts[:2], mn, wn, k=wl.k, G=wl.G)     # page in
    reps, t0 = 0, time.perf_counter()
    while reps < 3 or (time.perf_counter() - t0 < 10.0 and reps < 20):
        oracle.layer_forward(xu, ts, mn, wn, k=wl.k, G=wl.G)
        reps += 1
    dt = time.perf_counter() - t0
    return {"value": n * reps / dt, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
            "sample": f"first {n} tokens of the {wl.name} batch, {reps} passes, {dt:.1f} s"}


def apply_options(B, ctx, args):
    B.moe_set_option(ctx, B.MOE_OPT_EXPERT_PATH, {"auto": 0, "fma": 1, "tcgen05": 2}[args.path])
    B.moe_set_option(ctx, B.MOE_OPT_PAIR_MODE, {"auto": 1, "never": 0}[args.pair])
    if args.early_shared != "auto":
        B.moe_set_option(ctx, B.MOE_OPT_EARLY_SHARED, int(args.early_shared))
    if args.background != "auto":
        B.moe_set_option(ctx, B.MOE_OPT_BACKGROUND_LANES, int(args.background))


def cuda_events():
    return torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)


def dispatch_mode_report(B, ctx, step_fn, steps, world, dev):
    """Invocations and step time under a shared orchestrator and under private (per-tenant) orchestrators: the same
    work, the same results, batched across tenants or per tenant (a short timed block per mode)."""
    out = {}
    for name, mode in (("shared", B.MOE_DISPATCH_SHARED), ("private", B.MOE_DISPATCH_PRIVATE)):
        B.moe_set_option(ctx, B.MOE_OPT_DISPATCH_MODE, mode)
        for _ in range(3):
            step_fn()
        blocks = timed_blocks(step_fn, steps, 0.25, world, torch.cuda.synchronize, dev, cuda_events)
        status, n_inv, _ = B.moe_last_status(ctx)
        if status != 0:
            raise SystemExit(f"device status {status} in dispatch mode {name}")
        out[name] = {"invocations_last_layer": n_inv, "ms_per_step": statistics.median(blocks) / steps}
    B.moe_set_option(ctx, B.MOE_OPT_DISPATCH_MODE, B.MOE_DISPATCH_SHARED)
    return out


def block_formation_report(B, ctx, step_fn, steps, wl, T, world, dev):
    """Blocks of G consecutive experts against load-aware blocks formed from the observed expert loads: rows of the
    fullest block, invocations and step time (same work, same results; the blocks order and partition it)."""
    ws = B.moe_get_workspace(ctx)
    nb = -(-wl.E // wl.G)

    def measure():
        for _ in range(3):
            step_fn()
        blocks = timed_blocks(step_fn, steps, 0.25, world, torch.cuda.synchronize, dev, cuda_events)
        status, n_inv, _ = B.moe_last_status(ctx)
        if status != 0:
            raise SystemExit(f"device status {status} in the block-formation report")
        goff = B.wrap_device_pointer(ws["group_off"], (wl.M * nb + 1,), torch.int32, dev).cpu()
        rows = (goff[1:] - goff[:-1]).to(torch.float64)
        return {"invocations": n_inv, "max_rows_per_block": int(rows.max()), "mean_rows_per_block": float(rows.mean()),
                "ms_per_step": statistics.median(blocks) / steps}
    out = {"consecutive_experts": measure()}
    eoff = B.wrap_device_pointer(ws["expert_off"], (wl.M * wl.E + 1,), torch.int32, dev).cpu().to(torch.int64)
    load = (eoff[1:] - eoff[:-1]).view(wl.M, wl.E)
    B.moe_set_block_table(ctx, B.moe_form_blocks(load, wl.G), nb)
    out["load_aware"] = measure()
    B.moe_set_block_table(ctx, None)
    return out


def residency_report(B, wl, wts, x, tenant, mot, dev, n_slots):
    """On-demand residency: every expert parked in pinned host memory, n_slots device slots.  Times the first call
    (every active expert is copied in), the same batch again (all resident) and the bytes resident against the whole
    pool: what a cold start costs and what staying warm saves in device memory."""
    T = x.shape[0]
    layer = B.MoELayer(H=wl.H, E=wl.E, I=wl.I, k=wl.k, Is=wl.Is, M=wl.M, n_tenants=wl.n_tenants, max_tokens=T,
                       n_slots=n_slots, device=str(dev))
    try:
        pool = [torch.zeros((n_slots, wl.I, wl.H), dtype=torch.bfloat16, device=dev),
                torch.zeros((n_slots, wl.I, wl.H), dtype=torch.bfloat16, device=dev),
                torch.zeros((n_slots, wl.H, wl.I), dtype=torch.bfloat16, device=dev)]
        layer.set_layer_weights(0, dict(wts, pool_gate=pool[0], pool_up=pool[1], pool_down=pool[2]))
        layer.set_tables(model_of_tenant=mot)
        host = [wts[k_].contiguous().pin_memory() for k_ in ("pool_gate", "pool_up", "pool_down")]
        B.moe_residency_enable(layer.ctx, 0, host[0], host[1], host[2], pool[0], pool[1], pool[2])
        xd, td = x.to(dev), tenant.to(dev)
        out = torch.zeros_like(xd)

        def timed_call():
            torch.cuda.synchronize()
            t0 = time.perf_counter()
            st = B.moe_layer_forward_paged(layer.ctx, 0, xd, td, T, wl.G, out)
            torch.cuda.synchronize()
            return 1e3 * (time.perf_counter() - t0), st
        cold_ms, cold = timed_call()
        warm = [timed_call() for _ in range(20)]
        expert_bytes = 3 * wl.H * wl.I * 2
        return {"slots": n_slots, "experts": wl.M * wl.E, "cold_call_ms": cold_ms, "cold_loads": cold[2],
                "cold_h2d_bytes": cold[2] * expert_bytes, "warm_call_ms": statistics.median(m for m, _ in warm),
                "warm_hits": warm[-1][1][1], "active_experts": cold[0],
                "resident_bytes": n_slots * expert_bytes, "full_pool_bytes": wl.M * wl.E * expert_bytes}
    except B.MoeError as e:
        return {"skipped": str(e)}
    finally:
        layer.close()


def measure_layer(args, wl, rank, local_rank, world, dev, wts_cache, with_cpu_baseline):
    """One single-layer workload (decode, prefill, pool): device-resident throughput, per-stage times, end to end
    through the host-buffer entry point, roofline of the dominant kernel and of the whole path."""
    from paper_2604_26881_b200 import binding as B
    steps = args.steps if args.steps is not None else DEFAULT_STEPS[wl.name]
    warmup = max(args.warmup if args.warmup is not None else 20, 3)
    # every rank is an independent replica with its own batch (different seed), same weights recipe; the Qwen-shape
    # decode and prefill layers share their expert weights (prefill adds the router bias)
    key = (wl.H, wl.E, wl.I, wl.Is, wl.M)
    if key not in wts_cache:
        wts_cache[key] = W.make_weights(W.scaled(wl, zipf_bias=True), seed=0)
    wts = dict(wts_cache[key])
    if not wl.zipf_bias:
        wts["router_bias"] = None
    x, tenant, mot = W.make_tokens(wl, seed=replicas.rank_seed(0, rank))
    T = x.shape[0]
    layer = B.MoELayer(H=wl.H, E=wl.E, I=wl.I, k=wl.k, Is=wl.Is, M=wl.M, n_tenants=wl.n_tenants, max_tokens=T,
                       device=str(dev))
    try:
        layer.set_layer_weights(0, wts)
        layer.set_tables(slot_table=wts["slot_table"], model_of_tenant=mot)
        ctx = layer.ctx
        apply_options(B, ctx, args)
        xd, td = x.to(dev), tenant.to(dev)
        out = torch.zeros_like(xd)
        stream = torch.cuda.current_stream()

        # ---- device-resident throughput -----------------------------------------------------------
        for _ in range(warmup):
            B.moe_layer_forward(ctx, 0, xd, td, T, wl.G, out, stream)
        torch.cuda.synchronize()
        status, n_inv, active = B.moe_last_status(ctx)
        if status != 0:
            raise SystemExit(f"device status {status} after warm-up")
        sampler = ClockSampler(local_rank)
        sampler.start()
        l0 = B.moe_launch_count(ctx)
        blocks = timed_blocks(lambda: B.moe_layer_forward(ctx, 0, xd, td, T, wl.G, out, stream), steps, args.min_time,
                              world, torch.cuda.synchronize, dev, cuda_events)
        clocks = sampler.stop()
        launches = (B.moe_launch_count(ctx) - l0) // len(blocks)

        # ---- per-stage durations (CUDA events on the launching stream, between the kernels) ---------
        stage_ms = B.moe_stage_times(ctx, xd, td, T, wl.G, out, reps=max(10, min(steps, 100)))

        # ---- end to end through the host-buffer entry point ---------------------------------------
        xh, th = x.contiguous().pin_memory(), tenant.contiguous().pin_memory()
        oh = torch.zeros_like(xh).pin_memory()
        e2e_steps = max(10, min(steps, 200))
        for _ in range(3):
            B.moe_layer_forward_host(ctx, 0, xh, th, T, wl.G, oh, stream)
        e2e_blocks = timed_blocks(lambda: B.moe_layer_forward_host(ctx, 0, xh, th, T, wl.G, oh, stream), e2e_steps,
                                  min(args.min_time, 0.5), world, torch.cuda.synchronize, dev, cuda_events)
        # the same with two calls in flight (submit / wait): every step still copies its inputs in and its result out,
        # but the copies of neighbouring steps overlap the layer pass; timed on the host clock around whole blocks
        oh2 = torch.zeros_like(xh).pin_memory()
        outs_h = [oh, oh2]

        def pipelined_block():
            replicas.barrier(world, torch.cuda.synchronize)
            t0 = time.perf_counter()
            pending = []
            for i in range(e2e_steps):
                pending.append(B.moe_layer_forward_host_submit(ctx, 0, xh, th, T, wl.G, outs_h[i & 1], stream))
                if len(pending) > 1:
                    B.moe_layer_forward_host_wait(ctx, pending.pop(0))
            for t_ in pending:
                B.moe_layer_forward_host_wait(ctx, t_)
            dt = 1e3 * (time.perf_counter() - t0)
            replicas.barrier(world, torch.cuda.synchronize)
            return dt
        pipelined_block()
        pipe_blocks = [pipelined_block() for _ in range(max(3, int(min(args.min_time, 0.5) * 1e3 / max(e2e_blocks[0], 1e-3))))]
        pipe_blocks = replicas.max_over_ranks(pipe_blocks, world, dev)
        modes = formation = None
        step_fn = lambda: B.moe_layer_forward(ctx, 0, xd, td, T, wl.G, out, stream)
        if wl.n_tenants > 1:
            modes = dispatch_mode_report(B, ctx, step_fn, max(10, steps // 10), world, dev)
        if wl.G > 1:
            formation = block_formation_report(B, ctx, step_fn, max(10, steps // 10), wl, T, world, dev)
    finally:
        layer.close()
    residency = None
    if wl.name == "decode" and rank == 0 and world == 1:
        residency = residency_report(B, wl, wts, x, tenant, mot, dev, n_slots=wl.E - 4)

    if rank != 0:
        return None
    peaks = measured_peaks()
    work = algorithmic_work(wl, active, T)
    bs = block_summary(blocks, steps)
    ms_step = bs["median_ms"] / steps
    e2e_ms_step = statistics.median(e2e_blocks) / e2e_steps
    pipe_ms_step = statistics.median(pipe_blocks) / e2e_steps
    t_hbm = work["total_bytes"] / (peaks["hbm_gbs"] * 1e9)
    t_tc = work["flops"] / (peaks["bf16_tflops"] * 1e12)
    bound = "hbm" if t_hbm >= t_tc else "tensor"
    gu_ms = stage_ms.get("experts_gateup")            # dominant kernel: the gate/up grouped GEMM of moe_experts
    if bound == "hbm":
        achieved = work["gateup_bytes"] / (gu_ms * 1e-3) / 1e9 if gu_ms else None
        peak, runit = peaks["hbm_gbs"], "GB/s"
    else:
        achieved = work["gateup_flops"] / (gu_ms * 1e-3) / 1e12 if gu_ms else None
        peak, runit = peaks["bf16_tflops"], "TFLOP/s"
    traffic, traffic_source = traffic_record(wl.name, args.path)
    roofline = {"bound": bound, "kernel": "moe_experts gate/up grouped GEMM", "achieved": achieved, "peak": peak,
                "unit": runit, "frac": (achieved / peak) if achieved else None,
                "traffic": traffic, "traffic_source": traffic_source,
                "algorithmic": work["gateup_bytes"] if bound == "hbm" else work["gateup_flops"],
                "peak_source": peaks["source"],
                "path": {"roofline_ms": 1e3 * max(t_hbm, t_tc), "measured_ms": ms_step,
                         "frac": 1e3 * max(t_hbm, t_tc) / ms_step, "algorithmic_bytes": work["total_bytes"],
                         "flops": work["flops"], "active_experts": active},
                "stage_ms": stage_ms}
    if bound == "tensor":
        # the step is timed in long blocks, where the part has settled under its power cap: the same fractions
        # against the GEMM throughput the library reaches in that state, beside the ones against its burst
        sus = peaks["bf16_tflops_sustained"]
        roofline["peak_sustained"] = sus
        roofline["frac_of_sustained"] = (achieved / sus) if achieved else None
        roofline["path"]["frac_of_sustained"] = 1e3 * max(t_hbm, work["flops"] / (sus * 1e12)) / ms_step
    line = {"metric": METRIC, "value": world * T / (ms_step * 1e-3), "unit": UNIT, "n_gpus": world, "steps": steps,
            "warmup": warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16", "data": "synthetic",
            "config": {"workload": wl.name, "tokens_per_step_per_gpu": T, "hidden": wl.H, "experts": wl.E,
                       "inter": wl.I, "top_k": wl.k, "shared_inter": wl.Is, "G": wl.G, "tenants": wl.n_tenants,
                       "models": wl.M, "expert_path": args.path, "early_shared": args.early_shared,
                       "l2": "expert weights (about 1 GB per pass) exceed the 126 MB L2; no flush",
                       "parallelism": f"replicas x{world}"},
            "blocks": bs, "clocks": clocks, "gpu_launches": int(launches) * len(blocks),
            "gpu_launches_per_block": int(launches),
            "e2e": {"value": world * T / (pipe_ms_step * 1e-3), "unit": UNIT,
                    "h2d_bytes_per_step": int(T * wl.H * 2 + T * 4), "d2h_bytes_per_step": int(T * wl.H * 2),
                    "ms_per_step": pipe_ms_step,
                    "how": "moe_layer_forward_host_submit / _wait, two calls in flight: every step copies its inputs "
                           "from pinned host memory and its result back; host clock around blocks of steps",
                    "one_call_at_a_time": {"value": world * T / (e2e_ms_step * 1e-3), "ms_per_step": e2e_ms_step,
                                           "how": "moe_layer_forward_host (copies, layer, copies, synchronise per call)"}},
            "roofline": roofline}
    if modes:
        line["dispatch_modes"] = modes
    if formation:
        line["block_formation"] = formation
    if residency:
        line["on_demand_residency"] = residency
    if with_cpu_baseline:
        line["cpu_baseline"] = cpu_baseline(wl, wts, x, tenant, mot)
    return line


def measure_stack(args, wl, rank, local_rank, world, dev):
    """The 24-block configuration: RMSNorm -> MoE layer (+shared expert) -> residual, 26.6 GB of weights resident."""
    from paper_2604_26881_b200 import binding as B
    steps = args.steps if args.steps is not None else DEFAULT_STEPS["stack"]
    warmup = max(args.warmup if args.warmup is not None else 3, 3)
    x, tenant, mot = W.make_tokens(wl, seed=replicas.rank_seed(0, rank))
    T = x.shape[0]
    gen = torch.Generator(device=dev).manual_seed(1234)

    def rnd(*shape, std=0.02):
        return (torch.randn(*shape, generator=gen, device=dev, dtype=torch.float32) * std).to(torch.bfloat16)
    layer = B.MoELayer(H=wl.H, E=wl.E, I=wl.I, k=wl.k, Is=wl.Is, M=1, n_tenants=wl.n_tenants, max_tokens=T,
                       n_layers=wl.n_layers, device=str(dev))
    try:
        S = wl.n_slots
        for l in range(wl.n_layers):
            layer.set_layer_weights(l, {
                "router_w": rnd(1, wl.E, wl.H), "router_bias": None, "pool_gate": rnd(S, wl.I, wl.H),
                "pool_up": rnd(S, wl.I, wl.H), "pool_down": rnd(S, wl.H, wl.I), "shared_gate_w": rnd(1, wl.H),
                "ws_gate": rnd(1, wl.Is, wl.H), "ws_up": rnd(1, wl.Is, wl.H), "ws_down": rnd(1, wl.H, wl.Is),
                "rms_w": (1.0 + torch.randn(wl.H, generator=gen, device=dev) * 0.02).to(torch.bfloat16)})
        layer.set_tables(model_of_tenant=mot)
        ctx = layer.ctx
        apply_options(B, ctx, args)
        xd, td = x.to(dev), tenant.to(dev)
        xw = xd.clone()
        stream = torch.cuda.current_stream()

        def step():
            xw.copy_(xd)
            B.moe_stack_forward(ctx, xw, td, T, wl.G, None, None, stream)
        for _ in range(warmup):
            step()
        torch.cuda.synchronize()
        if B.moe_last_status(ctx)[0] != 0:
            raise SystemExit("device status set after warm-up")
        sampler = ClockSampler(local_rank)
        sampler.start()
        l0 = B.moe_launch_count(ctx)
        blocks = timed_blocks(step, steps, args.min_time, world, torch.cuda.synchronize, dev, cuda_events)
        clocks = sampler.stop()
        launches = (B.moe_launch_count(ctx) - l0) // len(blocks)
        # Realised active experts and stage times per block: one more pass keeps every block's normalised input, then
        # each block's layer is run alone on it (same kernels, same inputs) with events between its stages.
        dbg_in = torch.zeros((wl.n_layers, T, wl.H), dtype=torch.bfloat16, device=dev)
        xw.copy_(xd)
        B.moe_stack_forward(ctx, xw, td, T, wl.G, dbg_in, None, stream)
        torch.cuda.synchronize()
        out = torch.zeros_like(xd)
        active_per_block, stage_ms = [], {}
        for l in range(wl.n_layers):
            st = B.moe_stage_times(ctx, dbg_in[l], td, T, wl.G, out, reps=5, layer=l)
            for k_, v in st.items():
                stage_ms[k_] = stage_ms.get(k_, 0.0) + v
            active_per_block.append(B.moe_last_status(ctx)[2])
        modes = dispatch_mode_report(B, ctx, step, max(3, steps // 4), world, dev)
    finally:
        layer.close()
    if rank != 0:
        return None
    peaks = measured_peaks()
    expert_bytes = 3 * wl.H * wl.I * 2
    fixed_bytes = 3 * wl.H * wl.Is * 2 + (wl.E + 1) * wl.H * 2 + wl.H * 2 + 4 * T * wl.H
    total_bytes = sum(a * expert_bytes + fixed_bytes for a in active_per_block)
    flops = wl.n_layers * T * (wl.k * 6 * wl.H * wl.I + 6 * wl.H * wl.Is + 2 * wl.H * wl.E)
    t_hbm, t_tc = total_bytes / (peaks["hbm_gbs"] * 1e9), flops / (peaks["bf16_tflops"] * 1e12)
    bs = block_summary(blocks, steps)
    ms_step = bs["median_ms"] / steps
    stage_ms["rmsnorm_and_gaps"] = ms_step - sum(stage_ms.values())
    resident_bytes = wl.n_layers * (wl.E * expert_bytes + 3 * wl.H * wl.Is * 2 + (wl.E + 1) * wl.H * 2 + wl.H * 2)
    return {"metric": METRIC, "value": world * T / (ms_step * 1e-3), "unit": UNIT, "n_gpus": world,
            "steps": steps, "warmup": warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": wl.name, "blocks": wl.n_layers, "tokens_per_step_per_gpu": T, "tenants": wl.n_tenants,
                       "G": wl.G, "weights_gb": resident_bytes / 1e9,
                       "l2": "26.6 GB of weights per pass exceed the 126 MB L2; no flush",
                       "parallelism": f"replicas x{world}"},
            "blocks": bs, "clocks": clocks, "gpu_launches": int(launches) * len(blocks),
            "gpu_launches_per_block": int(launches), "dispatch_modes": modes,
            "roofline": {"bound": "hbm" if t_hbm >= t_tc else "tensor", "kernel": "whole stack",
                         "achieved": total_bytes / (ms_step * 1e-3) / 1e9, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                         "frac": 1e3 * max(t_hbm, t_tc) / ms_step, "traffic": None, "traffic_source": None,
                         "algorithmic": total_bytes, "peak_source": peaks["source"],
                         "active_experts_per_block": active_per_block,
                         "path": {"roofline_ms": 1e3 * max(t_hbm, t_tc), "measured_ms": ms_step,
                                  "frac": 1e3 * max(t_hbm, t_tc) / ms_step, "algorithmic_bytes": total_bytes,
                                  "flops": flops},
                         "stage_ms": stage_ms,
                         "stage_note": "stage times: every block's layer run alone on its own input (merged launches); "
                                       "rmsnorm_and_gaps = step time minus their sum"}}


def run_dry(args, rank, world):
    """The launch and reduction protocol without a GPU: gloo ranks, a short sleep as the step.  What the ranks do is
    what the GPU run does around its kernels: one batch per rank, blocks of exactly K steps between barriers, the
    maximum over ranks per block, the median block, one JSON line from rank 0."""
    import torch.distributed as dist
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("gloo")
    wl = W.WORKLOADS[args.workload or "decode"]
    steps = args.steps if args.steps is not None else 5
    x, _, _ = W.make_tokens(W.scaled(wl, T=min(wl.T or 64, 64), H=128), seed=replicas.rank_seed(0, rank))
    T = x.shape[0]

    class HostEvent:
        def record(self):
            self.t = time.perf_counter()

        def elapsed_time(self, other):
            return 1e3 * (other.t - self.t)

    step_s = 1e-3 * (rank + 1)                      # the last rank is the slow one
    blocks = timed_blocks(lambda: time.sleep(step_s), steps, min(args.min_time, 0.05), world, None, None,
                          lambda: (HostEvent(), HostEvent()))
    checksum = replicas.sum_over_ranks(float(x.to(torch.float64).sum()), world)
    if rank == 0:
        bs = block_summary(blocks, steps)
        ms_step = bs["median_ms"] / steps
        print(json.dumps({"metric": METRIC, "value": world * T / (ms_step * 1e-3), "unit": UNIT, "n_gpus": world,
                          "steps": steps, "warmup": 0, "ms_per_step": ms_step, "higher_is_better": True,
                          "scaling": "weak", "vs_baseline": None, "dtype": "none", "data": "synthetic", "dry": True,
                          "config": {"workload": wl.name, "tokens_per_step_per_gpu": T, "parallelism": f"replicas x{world}"},
                          "blocks": bs, "batch_checksum": checksum, "gpu_launches": 0}), flush=True)
    if world > 1:
        dist.destroy_process_group()


def main():
    args = parse_args()
    # `--gpus N` without a launcher: start the N ranks here (one process per GPU); the reference arm runs on rank 0 alone
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and args.impl != "reference":
        sys.exit(spawn_ranks(args.gpus))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))

    if args.impl == "reference":
        run_reference(args, rank)
        return
    if args.dry:
        run_dry(args, rank, world)
        return

    import torch.distributed as dist
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    dev = torch.device(f"cuda:{local_rank}")
    torch.cuda.set_device(dev)
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=dev)

    names = [args.workload] if args.workload else ["decode"] + list(EXTRA_WORKLOADS)
    wts_cache, lines = {}, {}
    for i, name in enumerate(names):
        wl = W.WORKLOADS[name]
        if wl.n_layers > 1:
            if torch.cuda.mem_get_info()[0] < 32e9:
                lines[name] = {"skipped": "needs about 30 GB of free device memory"}
                continue
            lines[name] = measure_stack(args, wl, rank, local_rank, world, dev)
        else:
            lines[name] = measure_layer(args, wl, rank, local_rank, world, dev, wts_cache,
                                        with_cpu_baseline=(i == 0 and not args.no_cpu_baseline and world == 1))
        torch.cuda.empty_cache()
    if rank == 0:
        line = lines[names[0]]
        if len(names) > 1:
            # the other workloads ride in the same line: the fields the headline has, without the CPU baseline
            line["workloads"] = {n: lines[n] for n in names[1:]}
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
