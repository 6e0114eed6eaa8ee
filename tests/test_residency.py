"""Expert residency (Sec. 5, "Edge memory constraints and expert-level offloading"): the host-side
replacement policy against a plain model and against a brute-force recency list; on the GPU, an
offloaded context against the float64 oracle of the layer and against its resident twin."""
import random

import pytest
import torch

from oracle import residency as oxr
from paper_2608_15018_b200 import binding


def _random_accesses(rng, n_experts, n_slots, n_pinned, steps):
    for _ in range(steps):
        n = rng.randint(0, n_slots - n_pinned) if rng.random() < 0.8 else rng.randint(0, n_slots)
        yield rng.sample(range(n_experts), n)


def test_cache_matches_the_model_on_random_sequences():
    rng = random.Random(17)
    for trial in range(40):
        E = rng.choice([4, 8, 17, 64, 128])
        n_slots = rng.randint(1, E)
        pinned = rng.sample(range(E), rng.randint(0, min(n_slots, 3)))
        lib = binding.ExpertCache(E, n_slots, pinned)
        model = oxr.ResidencyModel(E, n_slots, pinned)
        for experts in _random_accesses(rng, E, n_slots, len(pinned), 60):
            try:
                want = model.access(experts)
            except ValueError:
                with pytest.raises(binding.S2MoEError):
                    lib.access(experts)
                continue
            assert lib.access(experts) == want, (trial, experts)
        lib.close()


def test_every_access_leaves_its_experts_resident_and_pinned_experts_never_move():
    rng = random.Random(5)
    E, n_slots, pinned = 32, 9, [30, 2, 11]
    lib = binding.ExpertCache(E, n_slots, pinned)
    resident = {e: i for i, e in enumerate(pinned)}
    for experts in _random_accesses(rng, E, n_slots, len(pinned), 300):
        try:
            slots, missed = lib.access(experts)
        except binding.S2MoEError:
            continue
        assert len(set(slots)) == len(slots) and all(0 <= s < n_slots for s in slots)
        for e, s, m in zip(experts, slots, missed):
            assert m == (0 if resident.get(e) == s else 1)      # a hit is exactly "was already there"
            if m:
                assert s >= len(pinned)                           # pinned slots are never given away
                resident = {k: v for k, v in resident.items() if v != s}
                resident[e] = s
        for i, e in enumerate(pinned):
            assert resident[e] == i
    lib.close()


def test_single_expert_accesses_are_plain_lru():
    # one expert per access, no pinned experts: the classic LRU list decides hits and victims
    rng = random.Random(9)
    E, n_slots = 12, 4
    lib = binding.ExpertCache(E, n_slots)
    order, where = [], {}                      # least recent first
    for _ in range(500):
        e = rng.randrange(E)
        (slot,), (missed,) = lib.access([e])
        if e in where:
            assert missed == 0 and slot == where[e]
            order.remove(e)
        else:
            assert missed == 1
            if len(where) == n_slots:
                victim = order.pop(0)
                assert where.pop(victim) == slot
            where[e] = slot
        order.append(e)
    lib.close()


def test_cache_argument_errors():
    with pytest.raises(binding.S2MoEError):
        binding.ExpertCache(8, 0)
    with pytest.raises(binding.S2MoEError):
        binding.ExpertCache(8, 2, [1, 1])
    with pytest.raises(binding.S2MoEError):
        binding.ExpertCache(8, 2, [1, 2, 3])
    c = binding.ExpertCache(8, 3, [0])
    with pytest.raises(binding.S2MoEError):
        c.access([1, 1])
    with pytest.raises(binding.S2MoEError):
        c.access([1, 2, 3])                    # three unpinned experts, two unpinned slots
    assert c.access([0, 1, 2]) == ([0, 1, 2], [0, 1, 1])
    c.close()


# ---- GPU

def _offloaded_layers(layers):
    out = []
    for lw in layers:
        d = dict(lw)
        for name in binding.OFFLOADED_FIELDS:
            if d.get(name) is not None:
                d[name] = d[name].cpu().pin_memory()
        out.append(d)
    return out


@pytest.mark.gpu
@pytest.mark.parametrize("weights", ["bf16", "int4"])
def test_offloaded_context_matches_oracle_and_resident_context(weights):
    from gpu_util import check_outputs
    from paper_2608_15018_b200 import workloads
    from paper_2608_15018_b200.workloads import CONFIGS

    wl = CONFIGS["cfg2"].with_(d_model=512, d_ff=512, n_experts=16, top_k=2, cap=4, n_layers=2)
    if weights == "int4":
        wl = wl.with_(weight_dtype=CONFIGS["cfg4"].weight_dtype)
    dev = torch.device("cuda", 0)
    L, B = wl.n_layers, 4
    layers = [workloads.layer_weights(wl, l, dev) for l in range(L)]
    cfg = binding.Config.from_workload(wl, n_layers=L, kernel_plan=3)
    n_slots = 9                                 # B * k = 8 experts at most per step, plus one pinned
    pinned = [[3], [7]]
    with binding.S2MoE(cfg, layers) as res, binding.S2MoE(cfg, _offloaded_layers(layers), n_slots=n_slots, pinned=pinned) as off:
        total_distinct = 0
        model = [oxr.ResidencyModel(wl.n_experts, n_slots, p) for p in pinned]
        for step in range(6):
            for l in range(L):
                H = workloads.hidden_states(wl.with_(seed=wl.seed + 100 * step), l, B, 0.5, dev)
                C = workloads.confidences(wl.with_(seed=wl.seed + 100 * step), l, B, dev)
                a = off.verify_layer(l, H, C)
                b = res.verify_layer(l, H, C)
                torch.cuda.synchronize()
                assert torch.equal(a.sel_idx, b.sel_idx) and int(a.n_unique) == int(b.n_unique)
                # the same kernel on the same values: the slot a weight lies in does not change a bit
                # of what is added up, only the order of the atomic additions may
                assert torch.allclose(a.out, b.out, rtol=1e-5, atol=1e-6)
                check_outputs(wl, layers[l], H, C, a)
                active = sorted(set(a.sel_idx.flatten().tolist()))
                total_distinct += len(active)
                model[l].access(active)
        hits, misses, nbytes = off.residency_stats()
        assert hits + misses == total_distinct
        assert (hits, misses) == (sum(m.hits for m in model), sum(m.misses for m in model))
        per_expert = 3 * wl.d_model * wl.d_ff * (2 if weights == "bf16" else 0.5 + 2 / 32)
        assert nbytes == int(misses * per_expert)
        assert sum(off.residency_uses(0)) + sum(off.residency_uses(1)) == total_distinct
        assert off.device_status() == 0


@pytest.mark.gpu
def test_offloaded_context_through_the_host_buffer_stack_call():
    """The stack call with host buffers overlaps its copies with the layers; an offloaded context
    meets the host between the two kernels of every layer on top of that: same results as resident."""
    from paper_2608_15018_b200 import workloads
    from paper_2608_15018_b200.workloads import CONFIGS

    wl = CONFIGS["cfg2"].with_(d_model=512, d_ff=512, n_experts=16, top_k=2, cap=4, n_layers=5)
    dev = torch.device("cuda", 0)
    L, B = wl.n_layers, 4
    layers = [workloads.layer_weights(wl, l, dev) for l in range(L)]
    cfg = binding.Config.from_workload(wl, n_layers=L, kernel_plan=3)
    with binding.S2MoE(cfg, layers) as res, binding.S2MoE(cfg, _offloaded_layers(layers), n_slots=10) as off:
        for step in range(3):
            w = wl.with_(seed=wl.seed + 31 * step)
            H = torch.stack([workloads.hidden_states(w, l, B, 0.5, dev) for l in range(L)])
            C = torch.stack([workloads.confidences(w, l, B, dev) for l in range(L)])
            want = res.verify_stack(H, C)
            torch.cuda.synchronize()
            hh, hc = H.cpu().pin_memory(), C.cpu().pin_memory()
            ho = torch.full_like(want.out.cpu(), float("nan")).pin_memory()
            hs = torch.full_like(want.sel_idx.cpu(), -1).pin_memory()
            hw = torch.full_like(want.sel_w.cpu(), float("nan")).pin_memory()
            hu = torch.full_like(want.n_unique.cpu(), -1).pin_memory()
            off.verify_stack_host(hh, hc, ho, hs, hw, hu)
            assert torch.equal(hs, want.sel_idx.cpu()) and torch.equal(hu, want.n_unique.cpu())
            assert torch.equal(hw, want.sel_w.cpu())
            assert torch.allclose(ho, want.out.cpu(), rtol=1e-5, atol=1e-6)
        hits, misses, _ = off.residency_stats()
        assert misses > 0 and hits + misses > 0
        assert off.device_status() == 0


@pytest.mark.gpu
def test_offloaded_context_errors():
    from paper_2608_15018_b200 import workloads
    from paper_2608_15018_b200.workloads import CONFIGS

    wl = CONFIGS["cfg2"].with_(d_model=256, d_ff=256, n_experts=8, top_k=2, cap=4, n_layers=1)
    dev = torch.device("cuda", 0)
    layers = _offloaded_layers([workloads.layer_weights(wl, 0, dev)])
    cfg = binding.Config.from_workload(wl, n_layers=1, kernel_plan=3)
    with pytest.raises(binding.S2MoEError):
        binding.S2MoE(cfg, layers, n_slots=9)                       # more slots than experts
    with pytest.raises(binding.S2MoEError):
        binding.S2MoE(cfg, layers, n_slots=2, pinned=[[1, 1]])      # repeated pinned expert
    with binding.S2MoE(cfg, layers, n_slots=2) as off:               # 4 tokens x top-2 want more than 2 experts
        H = workloads.hidden_states(wl, 0, 4, 1.0, dev)
        with pytest.raises(binding.S2MoEError) as err:
            off.verify_layer(0, H, None)
        assert err.value.status == binding.ERANGE
