#!/usr/bin/env python
"""Benchmark of the MoE verification layer (one JSON line on stdout).

A step is one pass of the whole hot path (router, reuse-aware gating, bucketing, expert
FFNs, shared experts) over every layer of a synthetic stack for one draft batch.
Metric: verified draft tokens/s per MoE layer = B / (step time / n_layers).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg2] [--tokens B]
                  [--sigma S] [--plan P] [--impl reference] [--no-cpu-baseline]

For N > 1 launch with torch.distributed.run; every rank runs an independent replica of
the stack (own seed) and rank 0 reports the aggregate over the slowest rank's time.
"""
import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "verified draft tokens/s per MoE layer"
UNIT = "tokens/s"
FALLBACK_HBM_GBS = 6650.0


# DRAM bytes (read + write) per algorithmic byte, from the ncu captures summarised under profiles/
# (ffn_tc_kernel_cfg2_2layers.md, ffn_tc_kernel_int4_cfg4_2layers.md, ffn_stream_kernel_cfg2_2layers.md); traffic grows with the
# number of distinct experts exactly as the algorithmic bytes do.
TRAFFIC_RATIO = {"ffn_tc_kernel": 1.03, "ffn_tc_kernel/int4": 1.02, "ffn_stream_kernel": 1.005}


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="own", choices=["own", "reference"])
    ap.add_argument("--workload", default="cfg2")
    ap.add_argument("--tokens", type=int, default=None)
    ap.add_argument("--sigma", type=float, default=None)
    ap.add_argument("--layers", type=int, default=None)
    ap.add_argument("--plan", type=int, default=0)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--cpu-seconds", type=float, default=15.0)
    return ap.parse_args()


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as fh:
            return float(json.load(fh)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc, self.thread = index, [], None, None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.FIELDS}",
                 "--format=csv,noheader,nounits", "-lms", "20"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.perf_counter(), line.strip()))

    def stop(self, t0=None, t1=None):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        rows = [r for t, r in self.rows if (t0 is None or t0 <= t <= t1)] or [r for _, r in self.rows]
        sm, mx, reasons = [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for r in rows:
            p = [x.strip() for x in r.split(",")]
            try:
                sm.append(float(p[0])); mx.append(float(p[1]))
            except Exception:
                continue
            for n, v in zip(names, p[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def cpu_baseline(wl, B, sigma, seconds, seed_layers):
    """The oracle as it stands, timed on the host cores on whole layers of the same workload."""
    import numpy as np
    import oracle
    from oracle import parity
    from paper_2608_15018_b200 import workloads

    done, t_total = 0, 0.0
    for layer in seed_layers:
        T = workloads.layer_weights(wl, layer, "cpu")
        H = workloads.hidden_states(wl, layer, B, sigma, "cpu")
        conf = workloads.confidences(wl, layer, B, "cpu").double().numpy()
        ocfg, ow = parity.from_workload(wl, T)
        t0 = time.perf_counter()
        oracle.layer(ocfg, ow, workloads.raw_numpy(H), conf)
        t_total += time.perf_counter() - t0
        done += 1
        if t_total >= seconds:
            break
    return {"value": B * done / t_total, "unit": UNIT, "cores": oracle.threads(), "kind": "oracle",
            "sample": f"{done} whole layer(s) of {wl.name}, all {B} tokens, float64, OpenMP over rows"}


def run_reference(args, wl, B, sigma):
    """Reference arm: the float64 oracle on the host cores; each step is one whole layer."""
    import oracle
    from oracle import parity
    from paper_2608_15018_b200 import workloads

    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    L = wl.n_layers
    prepared = {}

    def step(i):
        layer = 0            # one layer, generated once: the untimed set-up stays short
        if layer not in prepared:
            T = workloads.layer_weights(wl, layer, "cpu")
            H = workloads.hidden_states(wl, layer, B, sigma, "cpu")
            conf = workloads.confidences(wl, layer, B, "cpu").double().numpy()
            ocfg, ow = parity.from_workload(wl, T)
            prepared.clear()
            prepared[layer] = (ocfg, ow, workloads.raw_numpy(H), conf)
        ocfg, ow, h, conf = prepared[layer]
        t0 = time.perf_counter()
        oracle.layer(ocfg, ow, h, conf)
        return time.perf_counter() - t0

    for i in range(args.warmup):
        step(0)
    times = [step(i) for i in range(args.steps)]
    t_layer = sum(times) / len(times)
    value = B / t_layer
    sample = f"each step = 1 whole layer of {wl.name} (all {B} tokens)"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * t_layer,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic", "config": {"workload": wl.name, "n_tokens": B, "n_layers": L, "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.threads(), "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def run_own(args, wl, B, sigma):
    import torch
    import torch.distributed as dist

    from paper_2608_15018_b200 import binding, replicas, workloads

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    L = args.layers or wl.n_layers
    wl_r = replicas.replica_workload(wl, rank).with_(n_layers=L)      # replicas: independent requests

    weights = [workloads.layer_weights(wl_r, l, dev) for l in range(L)]
    H = torch.stack([workloads.hidden_states(wl_r, l, B, sigma, dev) for l in range(L)]).contiguous()
    C = torch.stack([workloads.confidences(wl_r, l, B, dev) for l in range(L)]).contiguous()
    cfg = binding.Config.from_workload(wl_r, n_layers=L, kernel_plan=args.plan)
    m = binding.S2MoE(cfg, weights)
    out = m.alloc_outputs(B, stack=True)
    stream = torch.cuda.Stream()

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- warm-up, launch count, clock sampler
    with torch.cuda.stream(stream):
        for _ in range(args.warmup):
            m.verify_stack(H, C, out, stream=stream)
        stream.synchronize()
        launches_before = m.kernel_launches()
        m.verify_stack(H, C, out, stream=stream)
        stream.synchronize()
        launches_per_step = m.kernel_launches() - launches_before
    sampler = ClockSampler(local)
    sampler.start()
    time.sleep(0.3)
    t_host0 = time.perf_counter()

    # ---- timed region A (the headline): K steps, each one replay of a CUDA graph that holds one
    # s2moe_verify_stack call (every layer's kernels, nothing else); falls back to plain stream launches
    graph_ms_total = None
    timed_path = "stream launches of s2moe_verify_stack"
    try:
        with torch.cuda.stream(stream):
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=stream):
                m.verify_stack(H, C, out, stream=torch.cuda.current_stream())
            for _ in range(max(args.warmup, 3)):
                g.replay()
            barrier()
            g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            g0.record(stream)
            for _ in range(args.steps):
                g.replay()
            g1.record(stream)
            barrier()
            graph_ms_total = g0.elapsed_time(g1)
            timed_path = "CUDA graph replay of one s2moe_verify_stack call per step"
    except Exception as exc:  # pragma: no cover
        graph_ms_total = None
        print(f"graph replay skipped: {exc}", file=sys.stderr)

    # ---- timed region B: the same K steps as plain stream launches with an event pair around every
    # kernel (per-kernel durations for the roofline; the event pairs cost a few per cent)
    with torch.cuda.stream(stream):
        barrier()
        m.profile_begin(launches_per_step * args.steps)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(args.steps):
            m.verify_stack(H, C, out, stream=stream)
        e1.record(stream)
        barrier()
        stream_ms_total = e0.elapsed_time(e1)
        kernels = m.profile_end()
    t_host1 = time.perf_counter()
    clocks = sampler.stop(t_host0, t_host1)
    status = m.device_status()
    n_unique = out.n_unique.cpu().tolist()
    ms_total = graph_ms_total if graph_ms_total is not None else stream_ms_total

    # ---- end to end: host buffers through the C ABI, copies inside the timed region
    hH, hC = H.cpu().pin_memory(), C.cpu().pin_memory()
    ho = torch.empty(out.out.shape, dtype=torch.float32).pin_memory()
    hs = torch.empty(out.sel_idx.shape, dtype=torch.int32).pin_memory()
    hw = torch.empty(out.sel_w.shape, dtype=torch.float32).pin_memory()
    hu = torch.empty(out.n_unique.shape, dtype=torch.int32).pin_memory()
    with torch.cuda.stream(stream):
        for _ in range(3):
            m.verify_stack_host(hH, hC, ho, hs, hw, hu, stream=stream)
        barrier()
        t0 = time.perf_counter()
        for _ in range(args.steps):
            m.verify_stack_host(hH, hC, ho, hs, hw, hu, stream=stream)
        torch.cuda.synchronize()
        e2e_s = time.perf_counter() - t0
    h2d = hH.numel() * hH.element_size() + hC.numel() * 4
    d2h = ho.numel() * 4 + hs.numel() * 4 + hw.numel() * 4 + hu.numel() * 4

    # ---- max over ranks
    ms_total, e2e_ms_total, stream_ms_total = replicas.max_over_ranks(
        [ms_total, e2e_s * 1e3, stream_ms_total], device=dev)
    ms_step = ms_total / args.steps
    value = replicas.aggregate_tokens_per_s(world, B, L, ms_step)          # tokens/s per layer, all ranks
    e2e_value = replicas.aggregate_tokens_per_s(world, B, L, e2e_ms_total / args.steps)

    if rank == 0:
        peak, peak_kind = measured_peak()
        # dominant kernel: the one with the largest summed duration
        dom = max(kernels, key=lambda n: kernels[n]["ms"]) if kernels else None
        uniq_bytes = [m.unique_expert_bytes(u) for u in n_unique]
        step_bytes = float(sum(uniq_bytes))
        roof = None
        if dom:
            k = kernels[dom]
            per_launch_ms = k["ms"] / k["launches"]
            launches_per_layer = k["launches"] / (args.steps * L)
            # bytes one launch of the dominant kernel must move (its share of the layer's weights)
            share = {"ffn_gateup_simple": 2.0 / 3.0, "ffn_down_simple": 1.0 / 3.0}.get(dom, 1.0)
            bytes_per_launch = share * step_bytes / L / max(launches_per_layer, 1e-9)
            achieved = bytes_per_launch / (per_launch_ms * 1e-3) / 1e9
            ratio = TRAFFIC_RATIO.get(dom + "/int4" if wl.weight_dtype == workloads.Q4B32 else dom, TRAFFIC_RATIO.get(dom))
            roof = {"bound": "hbm", "kernel": dom, "achieved": achieved, "peak": peak, "unit": "GB/s",
                    "frac": achieved / peak, "peak_kind": f"of {peak_kind}",
                    "traffic": ratio * bytes_per_launch if ratio else None,
                    "traffic_source": "ncu capture of a 2-layer case, scaled by algorithmic bytes",
                    "bytes_per_launch": bytes_per_launch, "us_per_launch": per_launch_ms * 1e3}
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": {0: "f32", 1: "bf16", 2: "int4*f16 -> f32"}[wl.weight_dtype],
            "data": "synthetic",
            "config": {"workload": wl.name, "n_tokens": B, "n_layers": L, "sigma": sigma if sigma is not None else wl.sigma,
                       "d_model": wl.d_model, "d_ff": wl.d_ff, "n_experts": wl.n_experts, "top_k": wl.top_k,
                       "cap": wl.cap, "alpha": wl.alpha, "kernel_plan": args.plan,
                       "l2": f"inputs larger than L2: {step_bytes / 1e9:.2f} GB of expert weights per step",
                       "parallelism": "replicas" if world > 1 else "single GPU"},
            "stack_tokens_per_s": world * B / (ms_step * 1e-3),
            "unique_experts_mean": sum(n_unique) / len(n_unique),
            "reuse_ratio": sum(n_unique) / (len(n_unique) * B * wl.top_k),
            "unique_expert_gbs": world * step_bytes / (ms_step * 1e-3) / 1e9,
            "unique_expert_frac_of_8tbs": step_bytes / (ms_step * 1e-3) / 8e12,
            "unique_expert_frac_of_measured": step_bytes / (ms_step * 1e-3) / (peak * 1e9),
            "timed_path": timed_path,
            "stream_ms_per_step_with_kernel_events": stream_ms_total / args.steps,
            "kernels": kernels,
            "roofline": roof,
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h},
            "gpu_launches": launches_per_step * args.steps,
            "clocks": clocks,
            "device_status": status,
        }
        if world == 1 and not args.no_cpu_baseline:
            line["cpu_baseline"] = cpu_baseline(wl, B, sigma, args.cpu_seconds, range(L))
        print(json.dumps(line), flush=True)
    m.close()
    if world > 1:
        dist.destroy_process_group()


def main():
    args = parse_args()
    from paper_2608_15018_b200 import workloads

    wl = workloads.CONFIGS[args.workload]
    B = args.tokens or wl.n_tokens
    if args.impl == "reference":
        run_reference(args, wl, B, args.sigma)
    else:
        run_own(args, wl, B, args.sigma)


if __name__ == "__main__":
    main()
