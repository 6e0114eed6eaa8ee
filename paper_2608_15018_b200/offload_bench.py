"""Expert-level offloading measured (Sec. 5, "Edge memory constraints and expert-level
offloading"): the routed experts' weights live in page-locked host memory, a layer keeps
``n_slots`` of them in device memory, hot experts from a profiling pass are pinned.

For every slot count the script runs the same sequence of verification steps (a new draft batch
per step, so the active experts change from step to step) and reports the time per layer, the
hit rate of the residency cache, the bytes fetched per step and the host-to-device rate they were
fetched at, beside the fully resident context.

    python -m paper_2608_15018_b200.offload_bench [--workload cfg2] [--layers 4] [--steps 24]
                                                  [--slots 16,32,48,64] [--hot 8] [--json out.json]
"""
from __future__ import annotations

import argparse
import json
import sys
import time

import torch

from . import binding, workloads


def _host_layers(layers):
    out = []
    for lw in layers:
        d = dict(lw)
        for name in binding.OFFLOADED_FIELDS:
            if d.get(name) is not None:
                d[name] = d[name].cpu().pin_memory()
        out.append(d)
    return out


def _inputs(wl, L, B, steps, dev):
    """Per step and layer: hidden states and confidences of a fresh draft batch."""
    H, C = [], []
    for s in range(steps):
        w = wl.with_(seed=wl.seed + 1000 * (s + 1))
        H.append([workloads.hidden_states(w, l, B, None, dev) for l in range(L)])
        C.append([workloads.confidences(w, l, B, dev) for l in range(L)])
    return H, C


def _run(m, H, C, L, warm):
    """Milliseconds per step after `warm` steps (wall clock around synchronised steps: the offloaded
    path blocks on the host) and, for an offloaded context, its (hits, misses, bytes) over those steps."""
    outs = [m.alloc_outputs(H[0][0].shape[0]) for _ in range(L)]
    times, base = [], (0, 0, 0)
    for s in range(len(H)):
        if s == warm and m.offloaded:
            base = m.residency_stats()
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        for l in range(L):
            m.verify_layer(l, H[s][l], C[s][l], outputs=outs[l])
        torch.cuda.synchronize()
        if s >= warm:
            times.append((time.perf_counter() - t0) * 1e3)
    stats = tuple(a - b for a, b in zip(m.residency_stats(), base)) if m.offloaded else (0, 0, 0)
    return sum(times) / len(times), stats


def main(argv=None) -> int:
    ap = argparse.ArgumentParser(description=__doc__, formatter_class=argparse.RawDescriptionHelpFormatter)
    ap.add_argument("--workload", default="cfg2", choices=sorted(workloads.CONFIGS))
    ap.add_argument("--layers", type=int, default=4)
    ap.add_argument("--steps", type=int, default=24)
    ap.add_argument("--warmup", type=int, default=4)
    ap.add_argument("--tokens", type=int, default=0)
    ap.add_argument("--slots", default="")
    ap.add_argument("--hot", type=int, default=8, help="experts per layer pinned from the profiling pass (0: none)")
    ap.add_argument("--json", default="")
    args = ap.parse_args(argv)
    wl = workloads.CONFIGS[args.workload].with_(n_layers=args.layers)
    L, B, E = args.layers, args.tokens or wl.n_tokens, wl.n_experts
    dev = torch.device("cuda", torch.cuda.current_device())
    layers = [workloads.layer_weights(wl, l, dev) for l in range(L)]
    cfg = binding.Config.from_workload(wl, n_layers=L, kernel_plan=3)
    H, C = _inputs(wl, L, B, args.steps, dev)
    per_expert = None
    report = {"workload": wl.name, "layers": L, "tokens": B, "steps": args.steps, "rows": []}
    with binding.S2MoE(cfg, layers) as res:
        ms_res, _ = _run(res, H, C, L, args.warmup)
        per_expert = res.unique_expert_bytes(1) - res.unique_expert_bytes(0)
        # profiling pass: how often each expert of each layer is activated over the sequence
        uses = [[0] * E for _ in range(L)]
        max_u = 0
        for s in range(args.steps):
            for l in range(L):
                o = res.verify_layer(l, H[s][l], C[s][l])
                active = set(o.sel_idx.flatten().tolist())
                max_u = max(max_u, len(active))
                for e in active:
                    uses[l][e] += 1
    print(f"{wl.name}: {L} layers, B = {B}, {E} experts of {per_expert / 1e6:.1f} MB, at most {max_u} active per step; "
          f"resident: {ms_res / L * 1e3:.1f} us per layer")
    report["resident_us_per_layer"] = ms_res / L * 1e3
    host = _host_layers(layers)
    slot_list = [int(x) for x in args.slots.split(",")] if args.slots else [3 * E // 8, E // 2, 3 * E // 4, E]
    for n_slots in slot_list:
        n_hot = min(args.hot, max(0, n_slots - max_u))     # the unpinned slots must hold a whole step
        pinned = [sorted(range(E), key=lambda e: (-uses[l][e], e))[:n_hot] for l in range(L)] if n_hot else None
        try:
            m = binding.S2MoE(cfg, host, n_slots=n_slots, pinned=pinned)
        except binding.S2MoEError as exc:
            print(f"n_slots = {n_slots}: {exc}")
            continue
        with m:
            try:
                ms, (hits, misses, nbytes) = _run(m, H, C, L, args.warmup)
            except binding.S2MoEError as exc:
                print(f"n_slots = {n_slots}: {exc}")
                continue
        steps_all = args.steps - args.warmup
        row = {"n_slots": n_slots, "n_pinned": n_hot, "us_per_layer": ms / L * 1e3, "hit_rate": hits / max(1, hits + misses),
               "mb_per_step": nbytes / steps_all / 1e6,
               "pool_gb": n_slots * per_expert * L / 1e9}
        extra_ms = ms - ms_res
        row["h2d_gbs"] = (nbytes / steps_all / 1e9) / (extra_ms * 1e-3) if extra_ms > 0 and nbytes else None
        report["rows"].append(row)
        rate = f"{row['h2d_gbs']:.1f} GB/s over the extra time" if row["h2d_gbs"] else "-"
        print(f"n_slots = {n_slots:3d} ({n_hot} pinned, pool {row['pool_gb']:.2f} GB): {row['us_per_layer']:9.1f} us per layer, "
              f"hit rate {100 * row['hit_rate']:5.1f} %, {row['mb_per_step']:8.1f} MB fetched per step, {rate}")
    if args.json:
        with open(args.json, "w") as fh:
            json.dump(report, fh)
    return 0


if __name__ == "__main__":
    sys.exit(main())
