"""The allocation-free routing entry point against the ordinary one (collected last).

s2moe_route_noalloc serves callers that may not allocate device memory while they run
(a serving loop that owns the whole device through its own pool, code running while an
allocator is locked or a stream capture is open, a path where a synchronising cudaMalloc
is not acceptable): its scratch is a fixed array inside the library image.  It must give
the selection, the mixing weights and the unique-expert count that s2moe_verify_layer
gives, call after call, although every call reuses the same scratch array.
"""
import ctypes

import numpy as np
import pytest
import torch

import oracle
from oracle import parity
from paper_2608_15018_b200 import binding, workloads
from paper_2608_15018_b200.workloads import CONFIGS

pytestmark = pytest.mark.gpu


def _reference(wl, layer, B, dev):
    T = workloads.layer_weights(wl, layer, dev)
    H = workloads.hidden_states(wl, layer, B, device=dev)
    C = workloads.confidences(wl, layer, B, device=dev)
    cfg = binding.Config.from_workload(wl, n_layers=1, kernel_plan=1)
    with binding.S2MoE(cfg, [T]) as m:
        o = m.verify_layer(0, H, C)
        torch.cuda.synchronize()
        gate = None
        if "sh_scale" in T:
            lists = m.debug_lists()
            gate = lists["slot_w"][B * wl.top_k:B * wl.top_k + B].clone()
    return cfg, T, H, C, o, gate


def test_noalloc_routing_matches_verify_layer_twice_in_a_row():
    dev = torch.device("cuda", 0)
    small3 = CONFIGS["cfg3"].with_(d_model=512, d_ff=64, d_ff_shared=64)     # gated shared expert
    small2 = CONFIGS["cfg2"].with_(d_model=256, d_ff=64)
    big = CONFIGS["e128a"].with_(d_model=256, d_ff=64)                       # 128 experts: the entry point's limit
    cases = [(small3, 0, 16), (small2, 1, 8), (small3, 1, 5), (small2.with_(alpha=0.0), 0, 64), (big, 0, 64), (big, 1, 33)]
    for wl, layer, B in cases:                      # consecutive calls share the scratch array
        cfg, T, H, C, o, gate = _reference(wl, layer, B, dev)
        binding.route_noalloc(cfg, H, T["router"], C, T.get("sh_scale"))     # (first call on the device does the set-up)
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        sel, w, nu, g = binding.route_noalloc(cfg, H, T["router"], C, T.get("sh_scale"))
        torch.cuda.synchronize()
        assert binding.route_noalloc_status() == 0
        assert torch.equal(sel, o.sel_idx)
        assert torch.equal(nu, o.n_unique)
        assert torch.allclose(w, o.sel_w, rtol=0, atol=2e-6)      # the tolerance the parity tests use for weights
        if gate is not None:
            assert torch.allclose(g.cpu(), gate, rtol=0, atol=2e-6)
        # and against the float64 oracle itself (selection in order, weights, count), under the
        # tie protocol of the parity tests
        ocfg, ow = parity.from_workload(wl, T)
        rep = parity.check_layer(ocfg, ow, workloads.raw_numpy(H), C.cpu().numpy(), None, sel.cpu().numpy(),
                                 w.cpu().numpy(), int(nu.item()), 0.0)
        assert rep.order_checked + len(rep.ties) >= B       # every token: exact order, or a reported tie
        if gate is not None:
            x = H.double().cpu().numpy() @ T["sh_scale"].double().cpu().numpy()
            assert np.allclose(g.cpu().numpy(), 1.0 / (1.0 + np.exp(-x)), rtol=0, atol=2e-6)
        # the call itself took no device memory (the output tensors above are the caller's and
        # come out of torch's cache; the driver-level figure must not have moved)
        del sel, w, nu, g
        assert torch.cuda.mem_get_info()[0] >= free_before


def test_noalloc_rejects_sizes_beyond_its_scratch():
    dev = torch.device("cuda", 0)
    lib = binding.load_library()
    wl = CONFIGS["cfg2"].with_(d_model=256, d_ff=64, n_experts=binding.NOALLOC_MAX_EXPERTS + 8)
    cfg = binding.Config.from_workload(wl, n_layers=1).c()
    buf = torch.zeros(1 << 16, dtype=torch.float32, device=dev)
    p = buf.data_ptr()
    args = lambda c, B: (ctypes.byref(c), B, p, None, p, None, p, p, p, None, None)
    assert lib.s2moe_route_noalloc(*args(cfg, 8)) == binding.ERANGE
    cfg_ok = binding.Config.from_workload(CONFIGS["cfg2"].with_(d_model=256, d_ff=64), n_layers=1).c()
    assert lib.s2moe_route_noalloc(*args(cfg_ok, binding.NOALLOC_MAX_TOKENS + 1)) == binding.ERANGE
    assert lib.s2moe_route_noalloc(*args(cfg_ok, 0)) == binding.OK
    assert lib.s2moe_route_noalloc(None, 8, p, None, p, None, p, p, p, None, None) == binding.EINVAL
    assert lib.s2moe_route_noalloc_status(None) == binding.EINVAL
    torch.cuda.synchronize()
