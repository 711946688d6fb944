#!/usr/bin/env python
"""Benchmark of the multi-tenant MoE layer hot path (route -> dispatch -> experts -> combine).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload decode|prefill|pool] [--impl reference]

One step is one pass of the whole layer over one batch of seeded synthetic tokens at the
Qwen1.5-MoE layer shape.  With N > 1 (launched by torch.distributed.run) every rank runs an
independent replica on its own batch (the layer has no exchange step), time is the maximum over
ranks and the value is the aggregate tokens/s.  Prints one JSON line on rank 0.
"""
from __future__ import annotations

import argparse
import json
import os
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


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--workload", default="decode", choices=["decode", "prefill", "pool", "stack"])
    ap.add_argument("--impl", default="b200", choices=["b200", "reference"])
    ap.add_argument("--path", default="auto", choices=["auto", "fma", "tcgen05"])
    ap.add_argument("--pair", default="auto", choices=["auto", "never"])
    ap.add_argument("--early-shared", default="auto", choices=["auto", "0", "1", "2"],
                    help="shared expert on the context's second stream (auto: the library's default, batches of more than 64 tokens); "
                         "the per-stage times and the roofline block always come from passes without it, where one "
                         "grouped-GEMM launch holds the shared and the routed units")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    return ap.parse_args()


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
        sm, smax, reasons = [], [], set()
        try:
            with open(self.path) as f:
                for line in f:
                    c = [v.strip() for v in line.split(",")]
                    if len(c) < 9:
                        continue
                    try:
                        sm.append(float(c[1])); smax.append(float(c[2]))
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
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(smax), samples=len(sm))
        out["reasons"] = sorted(reasons)
        return out


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


# DRAM traffic (dram__bytes_read.sum + dram__bytes_write.sum) of one launch of the dominant kernel, from the
# ncu captures summarised in profiles/grouped_gemm_decode_ncu.md and profiles/grouped_gemm_prefill_ncu.md; None where
# no capture of the current kernel exists.
NCU_TRAFFIC_BYTES = {"decode": 657.659136e6 + 4.132608e6, "prefill": 860.452352e6 + 84.881920e6}


def run_reference(args, wl, rank):
    """The oracle, as it stands, on the host cores: each step is a bounded sample of the workload."""
    import oracle
    if rank != 0:
        return
    steps = args.steps if args.steps is not None else 3
    warmup = args.warmup if args.warmup is not None else 1
    steps, warmup = min(steps, 10), min(warmup, 2)      # bounded: each pass is about a second of CPU work
    wts = W.make_weights(wl, seed=0)
    x, tenant, mot = W.make_tokens(wl, seed=0)
    n = min(x.shape[0], 32)
    xs, ts = x[:n].contiguous(), tenant[:n].contiguous()
    wn = W.weights_as_numpy(wts)
    xu = W.as_u16(xs)
    times = []
    for i in range(warmup + steps):
        t0 = time.perf_counter()
        oracle.layer_forward(xu, ts.numpy(), mot.numpy(), wn, k=wl.k, G=wl.G)
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
    n = min(x.shape[0], 32)
    xs, ts = x[:n].contiguous(), tenant[:n].contiguous()
    wn = W.weights_as_numpy(wts)
    xu = W.as_u16(xs)
    oracle.layer_forward(xu[:2], ts.numpy()[:2], mot.numpy(), wn, k=wl.k, G=wl.G)     # page in
    reps, t0 = 0, time.perf_counter()
    while reps < 3 or (time.perf_counter() - t0 < 10.0 and reps < 20):
        oracle.layer_forward(xu, ts.numpy(), mot.numpy(), wn, k=wl.k, G=wl.G)
        reps += 1
    dt = time.perf_counter() - t0
    return {"value": n * reps / dt, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
            "sample": f"first {n} tokens of the {wl.name} batch, {reps} passes, {dt:.1f} s"}


def run_stack(args, wl, rank, local_rank, world):
    """The 24-block configuration: RMSNorm -> MoE layer (+shared expert) -> residual, 26.6 GB of weights resident."""
    from paper_2604_26881_b200 import binding as B
    import torch.distributed as dist
    dev = torch.device(f"cuda:{local_rank}")
    torch.cuda.set_device(dev)
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=dev)
    steps = args.steps if args.steps is not None else 30
    warmup = max(args.warmup if args.warmup is not None else 3, 3)
    x, tenant, mot = W.make_tokens(wl, seed=replicas.rank_seed(0, rank))
    T = x.shape[0]
    gen = torch.Generator(device=dev).manual_seed(1234)

    def rnd(*shape, std=0.02):
        return (torch.randn(*shape, generator=gen, device=dev, dtype=torch.float32) * std).to(torch.bfloat16)
    layer = B.MoELayer(H=wl.H, E=wl.E, I=wl.I, k=wl.k, Is=wl.Is, M=1, n_tenants=wl.n_tenants, max_tokens=T,
                       n_layers=wl.n_layers, device=str(dev))
    S = wl.n_slots
    for l in range(wl.n_layers):
        layer.set_layer_weights(l, {
            "router_w": rnd(1, wl.E, wl.H), "router_bias": None, "pool_gate": rnd(S, wl.I, wl.H),
            "pool_up": rnd(S, wl.I, wl.H), "pool_down": rnd(S, wl.H, wl.I), "shared_gate_w": rnd(1, wl.H),
            "ws_gate": rnd(1, wl.Is, wl.H), "ws_up": rnd(1, wl.Is, wl.H), "ws_down": rnd(1, wl.H, wl.Is),
            "rms_w": (1.0 + torch.randn(wl.H, generator=gen, device=dev) * 0.02).to(torch.bfloat16)})
    layer.set_tables(model_of_tenant=mot)
    ctx = layer.ctx
    B.moe_set_option(ctx, B.MOE_OPT_PAIR_MODE, {"auto": 1, "never": 0}[args.pair])
    if args.early_shared != "auto":
        B.moe_set_option(ctx, B.MOE_OPT_EARLY_SHARED, int(args.early_shared))
    xd, td = x.to(dev), tenant.to(dev)
    xw = xd.clone()
    stream = torch.cuda.current_stream()
    for _ in range(warmup):
        xw.copy_(xd)
        B.moe_stack_forward(ctx, xw, td, T, wl.G, None, None, stream)
    torch.cuda.synchronize()
    if B.moe_last_status(ctx)[0] != 0:
        raise SystemExit("device status set after warm-up")
    sampler = ClockSampler(local_rank)
    replicas.barrier(world, torch.cuda.synchronize)
    sampler.start()
    l0 = B.moe_launch_count(ctx)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record(stream)
    for _ in range(steps):
        xw.copy_(xd)
        B.moe_stack_forward(ctx, xw, td, T, wl.G, None, None, stream)
    ev1.record(stream)
    replicas.barrier(world, torch.cuda.synchronize)
    clocks = sampler.stop()
    launches = B.moe_launch_count(ctx) - l0
    ms_total = replicas.max_over_ranks([ev0.elapsed_time(ev1)], world, dev)[0]
    if rank == 0:
        peaks = measured_peaks()
        layer_bytes = wl.E * 3 * wl.H * wl.I * 2 + 3 * wl.H * wl.Is * 2 + (wl.E + 1) * wl.H * 2 + wl.H * 2
        total_bytes = wl.n_layers * (layer_bytes + 4 * T * wl.H)          # upper bound: all experts active
        flops = wl.n_layers * T * (wl.k * 6 * wl.H * wl.I + 6 * wl.H * wl.Is + 2 * wl.H * wl.E)
        t_hbm, t_tc = total_bytes / (peaks["hbm_gbs"] * 1e9), flops / (peaks["bf16_tflops"] * 1e12)
        ms_step = ms_total / steps
        line = {"metric": METRIC, "value": world * T * steps / (ms_total * 1e-3), "unit": UNIT, "n_gpus": world,
                "steps": steps, "warmup": warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
                "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
                "config": {"workload": wl.name, "blocks": wl.n_layers, "tokens_per_step_per_gpu": T, "tenants": wl.n_tenants,
                           "G": wl.G, "weights_gb": wl.n_layers * layer_bytes / 1e9,
                           "l2": "26.6 GB of weights per pass exceed the 126 MB L2; no flush",
                           "parallelism": f"replicas x{world}"},
                "clocks": clocks, "gpu_launches": int(launches),
                "roofline": {"bound": "hbm" if t_hbm >= t_tc else "tensor", "kernel": "whole stack",
                             "achieved": total_bytes / (ms_step * 1e-3) / 1e9, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                             "frac": 1e3 * max(t_hbm, t_tc) / ms_step, "traffic": None, "peak_source": peaks["source"],
                             "note": "bytes assume every expert of every block is active"}}
        print(json.dumps(line), flush=True)
    layer.close()
    if world > 1:
        dist.destroy_process_group()


def main():
    args = parse_args()
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    wl = W.WORKLOADS[args.workload]

    if args.impl == "reference":
        run_reference(args, wl, rank)
        return

    from paper_2604_26881_b200 import binding as B
    import torch.distributed as dist

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    dev = torch.device(f"cuda:{local_rank}")
    torch.cuda.set_device(dev)
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=dev)

    if wl.n_layers > 1:
        run_stack(args, wl, rank, local_rank, world)
        return
    steps = args.steps if args.steps is not None else {"decode": 3000, "prefill": 200, "pool": 200}[args.workload]
    warmup = max(args.warmup if args.warmup is not None else 20, 3)

    # every rank is an independent replica with its own batch (different seed), same weights recipe
    wts = W.make_weights(wl, seed=0)
    x, tenant, mot = W.make_tokens(wl, seed=replicas.rank_seed(0, rank))
    T = x.shape[0]
    layer = B.MoELayer(H=wl.H, E=wl.E, I=wl.I, k=wl.k, Is=wl.Is, M=wl.M, n_tenants=wl.n_tenants, max_tokens=T,
                       device=str(dev))
    layer.set_layer_weights(0, wts)
    layer.set_tables(slot_table=wts["slot_table"], model_of_tenant=mot)
    ctx = layer.ctx
    B.moe_set_option(ctx, B.MOE_OPT_EXPERT_PATH, {"auto": 0, "fma": 1, "tcgen05": 2}[args.path])
    B.moe_set_option(ctx, B.MOE_OPT_PAIR_MODE, {"auto": 1, "never": 0}[args.pair])
    if args.early_shared != "auto":
        B.moe_set_option(ctx, B.MOE_OPT_EARLY_SHARED, int(args.early_shared))
    xd, td = x.to(dev), tenant.to(dev)
    out = torch.zeros_like(xd)
    stream = torch.cuda.current_stream()

    def barrier():
        replicas.barrier(world, torch.cuda.synchronize)

    # ---- device-resident throughput -----------------------------------------------------------
    for _ in range(warmup):
        B.moe_layer_forward(ctx, 0, xd, td, T, wl.G, out, stream)
    torch.cuda.synchronize()
    status, n_inv, active = B.moe_last_status(ctx)
    if status != 0:
        raise SystemExit(f"device status {status} after warm-up")
    sampler = ClockSampler(local_rank)
    barrier()
    sampler.start()
    l0 = B.moe_launch_count(ctx)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record(stream)
    for _ in range(steps):
        B.moe_layer_forward(ctx, 0, xd, td, T, wl.G, out, stream)
    ev1.record(stream)
    barrier()
    clocks = sampler.stop()
    launches = B.moe_launch_count(ctx) - l0
    ms_total = ev0.elapsed_time(ev1)

    # ---- per-stage durations (CUDA events on the launching stream, between the kernels) ---------
    stage_ms = B.moe_stage_times(ctx, xd, td, T, wl.G, out, reps=max(10, min(steps, 100)))

    # ---- end to end through the host-buffer entry point ---------------------------------------
    xh, th = x.contiguous().pin_memory(), tenant.contiguous().pin_memory()
    oh = torch.zeros_like(xh).pin_memory()
    e2e_steps = max(10, min(steps, 500))
    for _ in range(3):
        B.moe_layer_forward_host(ctx, 0, xh, th, T, wl.G, oh, stream)
    barrier()
    t0 = time.perf_counter()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(e2e_steps):
        B.moe_layer_forward_host(ctx, 0, xh, th, T, wl.G, oh, stream)
    e1.record(stream)
    torch.cuda.synchronize()
    e2e_ms = max(e0.elapsed_time(e1), 1e3 * (time.perf_counter() - t0))
    barrier()

    ms_total, e2e_ms = replicas.max_over_ranks([ms_total, e2e_ms], world, dev)

    if rank == 0:
        peaks = measured_peaks()
        work = algorithmic_work(wl, active, T)
        ms_step = ms_total / steps
        value = world * T * steps / (ms_total * 1e-3)
        t_hbm = work["total_bytes"] / (peaks["hbm_gbs"] * 1e9)
        t_tc = work["flops"] / (peaks["bf16_tflops"] * 1e12)
        bound = "hbm" if t_hbm >= t_tc else "tensor"
        # dominant kernel: the gate/up grouped GEMM of moe_experts
        gu_ms = stage_ms.get("experts_gateup")
        if bound == "hbm":
            achieved = work["gateup_bytes"] / (gu_ms * 1e-3) / 1e9 if gu_ms else None
            peak, runit = peaks["hbm_gbs"], "GB/s"
        else:
            achieved = work["gateup_flops"] / (gu_ms * 1e-3) / 1e12 if gu_ms else None
            peak, runit = peaks["bf16_tflops"], "TFLOP/s"
        roofline = {"bound": bound, "kernel": "moe_experts gate/up grouped GEMM", "achieved": achieved, "peak": peak,
                    "unit": runit, "frac": (achieved / peak) if achieved else None,
                    "traffic": NCU_TRAFFIC_BYTES.get(wl.name) if args.path == "auto" else None,
                    "algorithmic": work["gateup_bytes"] if bound == "hbm" else work["gateup_flops"],
                    "peak_source": peaks["source"],
                    "path": {"roofline_ms": 1e3 * max(t_hbm, t_tc), "measured_ms": ms_step,
                             "frac": 1e3 * max(t_hbm, t_tc) / ms_step, "algorithmic_bytes": work["total_bytes"],
                             "flops": work["flops"], "active_experts": active},
                    "stage_ms": stage_ms}
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": steps, "warmup": warmup,
                "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
                "dtype": "bf16", "data": "synthetic",
                "config": {"workload": wl.name, "tokens_per_step_per_gpu": T, "hidden": wl.H, "experts": wl.E,
                           "inter": wl.I, "top_k": wl.k, "shared_inter": wl.Is, "G": wl.G, "tenants": wl.n_tenants,
                           "models": wl.M, "expert_path": args.path, "early_shared": args.early_shared,
                           "l2": "expert weights (about 1 GB per pass) exceed the 126 MB L2; no flush",
                           "parallelism": f"replicas x{world}"},
                "clocks": clocks, "gpu_launches": int(launches),
                "e2e": {"value": world * T * e2e_steps / (e2e_ms * 1e-3), "unit": UNIT,
                        "h2d_bytes_per_step": int(T * wl.H * 2 + T * 4), "d2h_bytes_per_step": int(T * wl.H * 2)},
                "roofline": roofline}
        if not args.no_cpu_baseline and world == 1:
            line["cpu_baseline"] = cpu_baseline(wl, wts, x, tenant, mot)
        print(json.dumps(line), flush=True)
    layer.close()
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
