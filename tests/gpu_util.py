"""Helpers of the GPU parity tests: run one layer through the C ABI and check it."""
import numpy as np
import torch

from oracle import parity
from paper_2608_15018_b200 import binding, workloads

TOL = {workloads.F32: 2e-3, workloads.BF16: 2e-3, workloads.Q4B32: 1e-2}


def supports(wl, plan):
    """Kernel plan 2 (mma.sync) covers bf16 weights with bf16 activations; plans 3 and 4 (tcgen05;
    4 is the whole layer in one launch) also block-int4 weights whose contraction lengths are
    multiples of 256."""
    if plan not in (2, 3, 4):
        return True
    if wl.act_dtype != workloads.BF16:
        return False
    if wl.weight_dtype == workloads.BF16:
        return True
    q4_ok = wl.d_model % 256 == 0 and wl.d_ff % 256 == 0 and (wl.n_shared == 0 or wl.d_ff_shared % 256 == 0)
    return plan in (3, 4) and wl.weight_dtype == workloads.Q4B32 and q4_ok


def run_case(wl, layer=0, n_tokens=None, sigma=None, use_conf=True, plan=0, tok_list=None,
             hidden=None, conf=None, check_lists=True, optional=False):
    """Runs one layer through the C ABI and compares it with the oracle; returns (report, outputs).
    A demanded plan that does not cover the case (format not covered, or the batch does not fit
    the streaming kernel's shared memory) is an error, unless the caller says ``optional=True``
    and handles the returned (None, None) itself (by skipping or by counting)."""
    if not supports(wl, plan):
        assert optional, f"kernel plan {plan} does not cover this case (use supports() and skip)"
        return None, None
    dev = torch.device("cuda", 0)
    T = workloads.layer_weights(wl, layer, dev)
    H = workloads.hidden_states(wl, layer, n_tokens, sigma, dev) if hidden is None else hidden.to(dev)
    if conf is None and use_conf:
        conf = workloads.confidences(wl, layer, H.shape[0], dev)
    cfg = binding.Config.from_workload(wl, n_layers=1, kernel_plan=plan)
    with binding.S2MoE(cfg, [T]) as m:
        used = m.kernel_plan(H.shape[0])
        if plan in (2, 3, 4) and used != plan:
            assert optional, f"kernel plan {plan} was demanded, the library chose {used}"
            return None, None
        assert used in (1, 2, 3, 4) and (plan == 0 or used == plan)
        o = m.verify_layer(0, H, conf)
        torch.cuda.synchronize()
        status = m.device_status()
        assert status == 0, f"device status {status}"
        lists = m.debug_lists() if check_lists else None
        launches = m.kernel_launches()
    assert launches > 0
    ocfg, ow = parity.from_workload(wl, T)
    sel = o.sel_idx.cpu().numpy()
    w = o.sel_w.cpu().numpy()
    rep = parity.check_layer(ocfg, ow, workloads.raw_numpy(H), None if conf is None else conf.cpu().numpy(),
                             o.out.cpu().numpy(), sel, w, int(o.n_unique.item()),
                             TOL[wl.weight_dtype], tok_list=tok_list)
    if lists is not None:
        parity.check_bucketing(lists, sel, w, wl.n_experts, wl.n_shared)
    rep.plan = used
    return rep, o


def check_outputs(wl, T, H, conf, o):
    """One layer's outputs `o` for hidden states H (confidences conf) against the float64 oracle run
    on the weights T (a layer dict with every tensor's values; device or host)."""
    ocfg, ow = parity.from_workload(wl, T)
    return parity.check_layer(ocfg, ow, workloads.raw_numpy(H), None if conf is None else conf.cpu().numpy(),
                              o.out.cpu().numpy(), o.sel_idx.cpu().numpy(), o.sel_w.cpu().numpy(),
                              int(o.n_unique.item()), TOL[wl.weight_dtype])
