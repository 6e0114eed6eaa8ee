"""Calibration of the verification cost model on this GPU (Sec. 4.1, "Routing-aware Cost
Estimation"): the latency of the verification layer is modelled as linear in the number of
distinct experts it activates,

    t_layer(U) = T_0 + T_exp * U,

and T_exp ("the latency associated with introducing one additional expert") is what the
adaptive expansion multiplies the number of new experts by.  This script measures t_layer and
U for every layer of a stack over a sweep of draft-tree sizes and noise levels, fits the line
by least squares and reports R^2 and the mean absolute percentage error, the two figures the
paper quotes for its own calibration.

    python -m paper_2608_15018_b200.calibrate [--workload cfg5] [--layers 26] [--json out.json]
    python -m paper_2608_15018_b200.calibrate --workload cfg2 --top-k 2 --alpha 0     # draft pass

With --top-k and --alpha 0 the same measurement gives the cost of the expert-sparse draft pass
(Sec. 5.1, "Draft Experts"), the C^draft of the utility.

Every layer has its own weights, so consecutive timed layers never re-read cached weights.
"""
from __future__ import annotations

import argparse
import json
import sys

import numpy as np
import torch

from . import binding, workloads


def fit_line(u: np.ndarray, t: np.ndarray):
    """Least squares t = t0 + t_exp * u; returns (t0, t_exp, r2, mape)."""
    a = np.stack([np.ones_like(u), u], axis=1)
    (t0, t_exp), *_ = np.linalg.lstsq(a, t, rcond=None)
    pred = t0 + t_exp * u
    ss_res = float(((t - pred) ** 2).sum())
    ss_tot = float(((t - t.mean()) ** 2).sum())
    r2 = 1.0 - ss_res / ss_tot if ss_tot > 0 else 1.0
    mape = float(np.mean(np.abs((t - pred) / t)))
    return float(t0), float(t_exp), r2, mape


class _Borrowed:
    """A context that the caller owns, used where ``with`` expects one."""

    def __init__(self, m):
        self.m = m

    def __enter__(self):
        return self.m

    def __exit__(self, *exc):
        return False


def measure(wl, n_layers: int, batches, sigmas, repeats: int = 3, model=None):
    """Per-layer (B, sigma, layer, U, microseconds): median over `repeats` timed passes.  ``model``:
    a context for ``wl`` with ``n_layers`` layers that the caller has built already (its weights stay
    where they are), else one is built here."""
    dev = torch.device("cuda", torch.cuda.current_device())
    wl = wl.with_(n_layers=n_layers)
    stream = torch.cuda.Stream()
    rows = []
    if model is None:
        weights = [workloads.layer_weights(wl, l, dev) for l in range(n_layers)]
        cfg = binding.Config.from_workload(wl, n_layers=n_layers)
        holder = binding.S2MoE(cfg, weights)
    else:
        holder = _Borrowed(model)
    with holder as m, torch.cuda.stream(stream):
        for B in batches:
            for sigma in sigmas:
                H = [workloads.hidden_states(wl, l, B, sigma, dev) for l in range(n_layers)]
                C = [workloads.confidences(wl, l, B, dev) for l in range(n_layers)]
                outs = [m.alloc_outputs(B) for _ in range(n_layers)]
                times = np.zeros((repeats, n_layers))
                for rep in range(repeats + 1):                     # pass 0 warms up
                    ev = [torch.cuda.Event(enable_timing=True) for _ in range(n_layers + 1)]
                    ev[0].record(stream)
                    for l in range(n_layers):
                        m.verify_layer(l, H[l], C[l], outputs=outs[l], stream=stream)
                        ev[l + 1].record(stream)
                    stream.synchronize()
                    if rep:
                        times[rep - 1] = [ev[l].elapsed_time(ev[l + 1]) * 1e3 for l in range(n_layers)]
                med = np.median(times, axis=0)
                for l in range(n_layers):
                    rows.append((B, sigma, l, int(outs[l].n_unique.item()), float(med[l])))
        status = m.device_status()
    if status != 0:
        raise RuntimeError(f"device status {status}")
    return rows


def main(argv=None) -> int:
    ap = argparse.ArgumentParser(description=__doc__, formatter_class=argparse.RawDescriptionHelpFormatter)
    ap.add_argument("--workload", default="cfg5", choices=sorted(workloads.CONFIGS))
    ap.add_argument("--layers", type=int, default=0, help="layers of the stack (default: the workload's)")
    ap.add_argument("--batches", default="1,2,4,8,16,32,64")
    ap.add_argument("--sigmas", default="0.1,0.2,0.3,0.5,0.7,1.0")
    ap.add_argument("--top-k", type=int, default=0, help="override top-k (e.g. the draft pass: fewer experts per token)")
    ap.add_argument("--alpha", type=float, default=-1.0, help="override alpha (0 = plain top-k gating, as in the draft pass)")
    ap.add_argument("--json", default="")
    args = ap.parse_args(argv)
    wl = workloads.CONFIGS[args.workload]
    if args.top_k:
        wl = wl.with_(top_k=args.top_k, cap=max(args.top_k, min(wl.cap, wl.n_experts)))
    if args.alpha >= 0.0:
        wl = wl.with_(alpha=args.alpha)
    n_layers = args.layers or wl.n_layers
    batches = [int(x) for x in args.batches.split(",")]
    sigmas = [float(x) for x in args.sigmas.split(",")]
    rows = measure(wl, n_layers, batches, sigmas)
    arr = np.array([(r[0], r[3], r[4]) for r in rows], dtype=np.float64)
    t0, t_exp, r2, mape = fit_line(arr[:, 1], arr[:, 2])
    per_expert_mb = 3.0 * wl.d_model * wl.d_ff * {workloads.F32: 4, workloads.BF16: 2, workloads.Q4B32: 0.5625}[wl.weight_dtype] / 1e6
    report = {
        "workload": wl.name, "layers": n_layers, "points": len(rows),
        "fit_all": {"T0_us": t0, "T_exp_us": t_exp, "r2": r2, "mape": mape,
                    "implied_GBps_per_expert": per_expert_mb * 1e3 / t_exp if t_exp > 0 else None},
        "per_batch": {},
        "paper": {"r2": "0.943-0.999", "mape": "0.8-4.5 %", "note": "other hardware, other models: context only"},
    }
    print(f"{wl.name}: {len(rows)} layer timings, U from {int(arr[:, 1].min())} to {int(arr[:, 1].max())}")
    print(f"all points : t = {t0:7.2f} us + {t_exp:6.3f} us * U    R^2 = {r2:.4f}  MAPE = {100 * mape:.2f} %"
          f"   ({per_expert_mb:.1f} MB per expert -> {per_expert_mb * 1e3 / t_exp:.0f} GB/s marginal)")
    for B in batches:
        sub = arr[arr[:, 0] == B]
        if len(sub) >= 3 and sub[:, 1].max() > sub[:, 1].min():
            f = fit_line(sub[:, 1], sub[:, 2])
            report["per_batch"][str(B)] = {"T0_us": f[0], "T_exp_us": f[1], "r2": f[2], "mape": f[3],
                                           "U_min": int(sub[:, 1].min()), "U_max": int(sub[:, 1].max())}
            print(f"B = {B:3d}    : t = {f[0]:7.2f} us + {f[1]:6.3f} us * U    R^2 = {f[2]:.4f}  MAPE = {100 * f[3]:.2f} %"
                  f"   U in [{int(sub[:, 1].min())}, {int(sub[:, 1].max())}]")
    if args.json:
        with open(args.json, "w") as fh:
            json.dump({"report": report, "rows": rows}, fh)
    return 0


if __name__ == "__main__":
    sys.exit(main())
