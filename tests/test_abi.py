"""The C-ABI library loads and exports every symbol the header declares (CPU only)."""
import ctypes
import os
import re

from paper_2608_15018_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "s2moe.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(s2moe_[a-z_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    lib = binding.load_library()
    names = declared_symbols()
    assert "s2moe_create" in names and "s2moe_verify_layer" in names and "s2moe_destroy" in names
    for n in names:
        assert hasattr(lib, n), f"{n} declared in s2moe.h but not exported"
    assert set(binding.EXPORTS) <= set(names)


def test_strerror_and_null_handling():
    lib = binding.load_library()
    assert binding.strerror(0) == "ok"
    for code in (-1, -2, -3, -4, -5):
        assert binding.strerror(code) not in ("ok", "unknown status")
    assert binding.strerror(-99) == "unknown status"
    assert lib.s2moe_destroy(None) == binding.OK
    assert lib.s2moe_kernel_launches(None) == 0
    out = ctypes.c_void_p(123)
    assert lib.s2moe_create(None, None, ctypes.byref(out)) == binding.EINVAL
    assert out.value is None


def test_create_rejects_bad_configs_before_touching_the_device():
    lib = binding.load_library()
    good = dict(d_model=256, d_ff=128, n_experts=8, top_k=2, cap=4, max_tokens=8)
    bad = [dict(d_model=100), dict(d_ff=48), dict(n_experts=0), dict(n_experts=257), dict(top_k=0),
           dict(top_k=9), dict(cap=1), dict(cap=9), dict(alpha=-1.0), dict(max_tokens=65),
           dict(max_tokens=0), dict(n_layers=0), dict(weight_dtype=3), dict(act_dtype=2),
           dict(router_dtype=2), dict(renorm=2), dict(weight_mode=2), dict(n_shared=5),
           dict(n_shared=1, d_ff_shared=40), dict(kernel_plan=5), dict(top_k=17, n_experts=32, cap=20)]
    w = (binding.LayerWeightsC * 1)()
    for change in bad:
        cfg = binding.Config(**{**good, **change}).c()
        out = ctypes.c_void_p(None)
        assert lib.s2moe_create(ctypes.byref(cfg), w, ctypes.byref(out)) == binding.EINVAL, change
        assert out.value is None
    # a valid config with null weight pointers is rejected as well
    cfg = binding.Config(**good).c()
    out = ctypes.c_void_p(None)
    assert lib.s2moe_create(ctypes.byref(cfg), w, ctypes.byref(out)) == binding.EINVAL
    # misaligned weight pointer
    for name in binding.WEIGHT_FIELDS[:4]:
        setattr(w[0], name, 4096)
    w[0].w_up = 4100
    assert lib.s2moe_create(ctypes.byref(cfg), w, ctypes.byref(out)) == binding.EINVAL
