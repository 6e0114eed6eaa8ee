"""ctypes binding of the C ABI declared in ``include/s2moe.h``.

Argument marshalling only: every step of the layer runs in the CUDA library.
There is no CPU fallback; a missing library raises at first use.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass
from typing import Dict, List, Optional, Sequence, Tuple

import torch

from . import build as _build

F32, BF16, Q4B32 = 0, 1, 2
OK, EINVAL, ERANGE, ENOMEM, ECUDA, ETIMEOUT = 0, -1, -2, -3, -4, -5
MAX_TOKENS, MAX_EXPERTS, MAX_TOP_K = 64, 256, 16

WEIGHT_FIELDS = ("router", "w_gate", "w_up", "w_down", "s_gate", "s_up", "s_down",
                 "sh_gate", "sh_up", "sh_down", "sh_s_gate", "sh_s_up", "sh_s_down", "sh_scale")

EXPORTS = ("s2moe_create", "s2moe_verify_layer", "s2moe_verify_stack", "s2moe_verify_stack_host",
           "s2moe_destroy", "s2moe_strerror", "s2moe_last_device_status", "s2moe_last_cuda_error",
           "s2moe_kernel_launches", "s2moe_unique_expert_bytes", "s2moe_debug_read",
           "s2moe_profile_begin", "s2moe_profile_end", "s2moe_kernel_class_name", "s2moe_kernel_plan",
           "s2moe_route_noalloc", "s2moe_route_noalloc_status", "s2moe_expert_masks", "s2moe_adaptive_expand", "s2moe_create_offloaded",
           "s2moe_residency_stats", "s2moe_residency_uses", "s2moe_cache_create", "s2moe_cache_access",
           "s2moe_cache_destroy")
OFFLOADED_FIELDS = ("w_gate", "w_up", "w_down", "s_gate", "s_up", "s_down")   # host tensors of an offloaded context
NOALLOC_MAX_TOKENS, NOALLOC_MAX_EXPERTS = 64, 128
KERNEL_CLASSES = 7


class LayerWeightsC(ctypes.Structure):
    _fields_ = [(n, ctypes.c_void_p) for n in WEIGHT_FIELDS]


class ResidencyC(ctypes.Structure):
    _fields_ = [("n_slots", ctypes.c_int32), ("n_pinned", ctypes.c_int32), ("pinned", ctypes.c_void_p)]


class ConfigC(ctypes.Structure):
    _fields_ = [
        ("d_model", ctypes.c_int32), ("d_ff", ctypes.c_int32), ("n_experts", ctypes.c_int32),
        ("top_k", ctypes.c_int32), ("n_shared", ctypes.c_int32), ("d_ff_shared", ctypes.c_int32),
        ("act_dtype", ctypes.c_int32), ("router_dtype", ctypes.c_int32), ("weight_dtype", ctypes.c_int32),
        ("renorm", ctypes.c_int32), ("cap", ctypes.c_int32), ("alpha", ctypes.c_float),
        ("weight_mode", ctypes.c_int32), ("max_tokens", ctypes.c_int32), ("n_layers", ctypes.c_int32),
        ("kernel_plan", ctypes.c_int32),
    ]


class S2MoEError(RuntimeError):
    def __init__(self, status: int, where: str, detail: str = ""):
        self.status = status
        super().__init__(f"{where}: status {status} ({strerror(status)}){detail}")


_lib = None


def library_path() -> str:
    return _build.LIB


def load_library(build_if_missing: bool = True) -> ctypes.CDLL:
    """Load ``libs2moe.so`` (building it with nvcc when it is missing or stale)."""
    global _lib
    if _lib is not None:
        return _lib
    override = os.environ.get("S2MOE_LIBRARY")     # e.g. a self-checking build of the same sources
    path = override or (_build.build_library() if build_if_missing else _build.LIB)
    if not os.path.exists(path):
        raise RuntimeError(f"CUDA library {path} is missing; run __graft_entry__.build()")
    lib = ctypes.CDLL(path)
    vp, i32, fp = ctypes.c_void_p, ctypes.c_int32, ctypes.c_void_p
    lib.s2moe_create.argtypes = [ctypes.POINTER(ConfigC), ctypes.POINTER(LayerWeightsC), ctypes.POINTER(vp)]
    lib.s2moe_create.restype = ctypes.c_int
    lib.s2moe_verify_layer.argtypes = [vp, i32, i32, vp, fp, fp, vp, fp, vp, vp]
    lib.s2moe_verify_layer.restype = ctypes.c_int
    lib.s2moe_verify_stack.argtypes = [vp, i32, vp, fp, fp, vp, fp, vp, vp]
    lib.s2moe_verify_stack.restype = ctypes.c_int
    lib.s2moe_verify_stack_host.argtypes = [vp, i32, vp, fp, fp, vp, fp, vp, vp]
    lib.s2moe_verify_stack_host.restype = ctypes.c_int
    lib.s2moe_destroy.argtypes = [vp]
    lib.s2moe_destroy.restype = ctypes.c_int
    lib.s2moe_strerror.argtypes = [ctypes.c_int]
    lib.s2moe_strerror.restype = ctypes.c_char_p
    lib.s2moe_last_device_status.argtypes = [vp, ctypes.POINTER(i32)]
    lib.s2moe_last_device_status.restype = ctypes.c_int
    lib.s2moe_last_cuda_error.argtypes = [vp]
    lib.s2moe_last_cuda_error.restype = ctypes.c_int
    lib.s2moe_kernel_plan.argtypes = [vp, i32]
    lib.s2moe_kernel_plan.restype = ctypes.c_int
    lib.s2moe_kernel_launches.argtypes = [vp]
    lib.s2moe_kernel_launches.restype = ctypes.c_int64
    lib.s2moe_unique_expert_bytes.argtypes = [vp, i32]
    lib.s2moe_unique_expert_bytes.restype = ctypes.c_double
    lib.s2moe_debug_read.argtypes = [vp, i32, vp, ctypes.c_size_t]
    lib.s2moe_debug_read.restype = ctypes.c_int
    lib.s2moe_route_noalloc.argtypes = [ctypes.POINTER(ConfigC), i32, vp, vp, vp, fp, vp, fp, vp, fp, vp]
    lib.s2moe_route_noalloc.restype = ctypes.c_int
    lib.s2moe_route_noalloc_status.argtypes = [ctypes.POINTER(ctypes.c_int32)]
    lib.s2moe_route_noalloc_status.restype = ctypes.c_int
    lib.s2moe_profile_begin.argtypes = [vp, i32]
    lib.s2moe_profile_begin.restype = ctypes.c_int
    lib.s2moe_profile_end.argtypes = [vp, i32, ctypes.POINTER(ctypes.c_double), ctypes.POINTER(ctypes.c_int64)]
    lib.s2moe_profile_end.restype = ctypes.c_int
    lib.s2moe_kernel_class_name.argtypes = [i32]
    lib.s2moe_kernel_class_name.restype = ctypes.c_char_p
    lib.s2moe_expert_masks.argtypes = [vp, i32, i32, i32, vp, i32, vp]
    lib.s2moe_expert_masks.restype = ctypes.c_int
    lib.s2moe_adaptive_expand.argtypes = [i32, i32, i32, vp, fp, vp, fp, ctypes.c_float, ctypes.c_float, vp, vp, vp,
                                          vp, vp]
    lib.s2moe_adaptive_expand.restype = ctypes.c_int
    lib.s2moe_create_offloaded.argtypes = [ctypes.POINTER(ConfigC), ctypes.POINTER(LayerWeightsC),
                                           ctypes.POINTER(ResidencyC), ctypes.POINTER(vp)]
    lib.s2moe_create_offloaded.restype = ctypes.c_int
    lib.s2moe_residency_stats.argtypes = [vp, ctypes.POINTER(ctypes.c_int64), ctypes.POINTER(ctypes.c_int64),
                                          ctypes.POINTER(ctypes.c_int64)]
    lib.s2moe_residency_stats.restype = ctypes.c_int
    lib.s2moe_residency_uses.argtypes = [vp, i32, vp]
    lib.s2moe_residency_uses.restype = ctypes.c_int
    lib.s2moe_cache_create.argtypes = [i32, i32, vp, i32, ctypes.POINTER(vp)]
    lib.s2moe_cache_create.restype = ctypes.c_int
    lib.s2moe_cache_access.argtypes = [vp, vp, i32, vp, vp]
    lib.s2moe_cache_access.restype = ctypes.c_int
    lib.s2moe_cache_destroy.argtypes = [vp]
    lib.s2moe_cache_destroy.restype = ctypes.c_int
    _lib = lib
    return lib


def strerror(status: int) -> str:
    return load_library().s2moe_strerror(int(status)).decode()


@dataclass
class Config:
    d_model: int
    d_ff: int
    n_experts: int
    top_k: int
    n_shared: int = 0
    d_ff_shared: int = 0
    act_dtype: int = BF16
    router_dtype: int = BF16
    weight_dtype: int = BF16
    renorm: int = 0
    cap: int = 0               # 0 -> n_experts (bias off)
    alpha: float = 0.5
    weight_mode: int = 0
    max_tokens: int = MAX_TOKENS
    n_layers: int = 1
    kernel_plan: int = 0

    def c(self) -> ConfigC:
        cap = self.cap if self.cap > 0 else self.n_experts
        return ConfigC(self.d_model, self.d_ff, self.n_experts, self.top_k, self.n_shared,
                       self.d_ff_shared, self.act_dtype, self.router_dtype, self.weight_dtype,
                       self.renorm, cap, float(self.alpha), self.weight_mode, self.max_tokens,
                       self.n_layers, self.kernel_plan)

    @staticmethod
    def from_workload(wl, max_tokens: Optional[int] = None, n_layers: Optional[int] = None,
                      kernel_plan: int = 0) -> "Config":
        return Config(wl.d_model, wl.d_ff, wl.n_experts, wl.top_k, wl.n_shared, wl.d_ff_shared,
                      wl.act_dtype, wl.router_dtype, wl.weight_dtype, wl.renorm, wl.cap, wl.alpha,
                      wl.weight_mode, max_tokens or MAX_TOKENS, n_layers or wl.n_layers, kernel_plan)


def _dptr(t: Optional[torch.Tensor]) -> Optional[int]:
    if t is None:
        return None
    if not t.is_cuda or not t.is_contiguous():
        raise ValueError("expected a contiguous CUDA tensor")
    return t.data_ptr()


def _stream_handle(stream: Optional[torch.cuda.Stream]) -> int:
    return (stream or torch.cuda.current_stream()).cuda_stream


@dataclass
class LayerOutput:
    out: torch.Tensor        # [..., B, d] float32
    sel_idx: torch.Tensor    # [..., B, k] int32
    sel_w: torch.Tensor      # [..., B, k] float32
    n_unique: torch.Tensor   # [...] int32


class S2MoE:
    """A context of the library: ``n_layers`` MoE layers whose weights stay resident."""

    def __init__(self, config: Config, layers: Sequence[Dict[str, torch.Tensor]], n_slots: int = 0,
                 pinned: Optional[Sequence[Sequence[int]]] = None):
        """``n_slots`` > 0 makes an offloaded context: the routed experts' weights (OFFLOADED_FIELDS
        of every layer dict) are host tensors, ``n_slots`` of them at a time are resident per
        layer, ``pinned[layer]`` lists the experts that are never evicted."""
        self._lib = load_library()
        self._h = ctypes.c_void_p(None)
        self.config = config
        if len(layers) != config.n_layers:
            raise ValueError("one weight dict per layer is required")
        self._keep = list(layers)          # keeps the caller's tensors alive
        arr = (LayerWeightsC * config.n_layers)()
        for i, lw in enumerate(layers):
            for name in WEIGHT_FIELDS:
                t = lw.get(name)
                if n_slots > 0 and name in OFFLOADED_FIELDS:
                    if t is not None and t.is_cuda:
                        raise ValueError(f"offloaded context: {name} must be a host tensor")
                    setattr(arr[i], name, None if t is None else t.data_ptr())
                else:
                    setattr(arr[i], name, _dptr(t))
        cfg = config.c()
        self.offloaded = n_slots > 0
        if self.offloaded:
            n_pinned = len(pinned[0]) if pinned else 0
            flat = [int(e) for row in (pinned or []) for e in row]
            if pinned and (len(pinned) != config.n_layers or len(flat) != n_pinned * config.n_layers):
                raise ValueError("pinned: one list of equal length per layer")
            self._pinned = (ctypes.c_int32 * max(1, len(flat)))(*flat)
            res = ResidencyC(int(n_slots), n_pinned, ctypes.cast(self._pinned, ctypes.c_void_p) if flat else None)
            rc = self._lib.s2moe_create_offloaded(ctypes.byref(cfg), arr, ctypes.byref(res), ctypes.byref(self._h))
        else:
            rc = self._lib.s2moe_create(ctypes.byref(cfg), arr, ctypes.byref(self._h))
        if rc != OK:
            self._h = ctypes.c_void_p(None)
            raise S2MoEError(rc, "s2moe_create_offloaded" if self.offloaded else "s2moe_create")
        self.device = layers[0]["router"].device

    def residency_stats(self) -> Tuple[int, int, int]:
        """(hits, misses, bytes fetched from host memory) since create, over all layers."""
        h, m, b = ctypes.c_int64(0), ctypes.c_int64(0), ctypes.c_int64(0)
        self._check(self._lib.s2moe_residency_stats(self._h, ctypes.byref(h), ctypes.byref(m), ctypes.byref(b)),
                    "s2moe_residency_stats")
        return h.value, m.value, b.value

    def residency_uses(self, layer: int) -> List[int]:
        """Per expert of ``layer``: the steps that activated it (the profile a hot set is chosen from)."""
        out = (ctypes.c_int64 * self.config.n_experts)()
        self._check(self._lib.s2moe_residency_uses(self._h, int(layer), ctypes.cast(out, ctypes.c_void_p)),
                    "s2moe_residency_uses")
        return list(out)

    # -- lifetime
    def close(self) -> None:
        if getattr(self, "_h", None) is not None and self._h.value:
            self._lib.s2moe_destroy(self._h)
            self._h = ctypes.c_void_p(None)

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.close()

    # -- calls
    def _check(self, rc: int, where: str) -> None:
        if rc != OK:
            detail = ""
            if rc == ECUDA:
                detail = f" cudaError={self._lib.s2moe_last_cuda_error(self._h)}"
            raise S2MoEError(rc, where, detail)

    def alloc_outputs(self, n_tokens: int, stack: bool = False) -> LayerOutput:
        c = self.config
        lead = (c.n_layers,) if stack else ()
        dev = self.device
        return LayerOutput(
            torch.empty(lead + (n_tokens, c.d_model), dtype=torch.float32, device=dev),
            torch.empty(lead + (n_tokens, c.top_k), dtype=torch.int32, device=dev),
            torch.empty(lead + (n_tokens, c.top_k), dtype=torch.float32, device=dev),
            torch.empty(lead if stack else (1,), dtype=torch.int32, device=dev),
        )

    def verify_layer(self, layer: int, hidden: torch.Tensor, conf: Optional[torch.Tensor] = None,
                     outputs: Optional[LayerOutput] = None,
                     stream: Optional[torch.cuda.Stream] = None) -> LayerOutput:
        B = hidden.shape[0]
        o = outputs or self.alloc_outputs(B)
        rc = self._lib.s2moe_verify_layer(self._h, layer, B, _dptr(hidden), _dptr(conf), _dptr(o.out),
                                          _dptr(o.sel_idx), _dptr(o.sel_w), _dptr(o.n_unique),
                                          _stream_handle(stream))
        self._check(rc, "s2moe_verify_layer")
        return o

    def verify_stack(self, hidden: torch.Tensor, conf: Optional[torch.Tensor] = None,
                     outputs: Optional[LayerOutput] = None,
                     stream: Optional[torch.cuda.Stream] = None) -> LayerOutput:
        """hidden [L][B][d]; conf [L][B] or None."""
        B = hidden.shape[1]
        o = outputs or self.alloc_outputs(B, stack=True)
        rc = self._lib.s2moe_verify_stack(self._h, B, _dptr(hidden), _dptr(conf), _dptr(o.out),
                                          _dptr(o.sel_idx), _dptr(o.sel_w), _dptr(o.n_unique),
                                          _stream_handle(stream))
        self._check(rc, "s2moe_verify_stack")
        return o

    def verify_stack_host(self, hidden: torch.Tensor, conf: Optional[torch.Tensor], out: torch.Tensor,
                          sel_idx: torch.Tensor, sel_w: torch.Tensor, n_unique: torch.Tensor,
                          stream: Optional[torch.cuda.Stream] = None) -> None:
        """All tensors are HOST tensors (pinned for best speed); returns after the results are there."""
        for t in (hidden, out, sel_idx, sel_w, n_unique):
            if t.is_cuda or not t.is_contiguous():
                raise ValueError("expected contiguous host tensors")
        B = hidden.shape[1]
        rc = self._lib.s2moe_verify_stack_host(
            self._h, B, hidden.data_ptr(), conf.data_ptr() if conf is not None else None, out.data_ptr(),
            sel_idx.data_ptr(), sel_w.data_ptr(), n_unique.data_ptr(), _stream_handle(stream))
        self._check(rc, "s2moe_verify_stack_host")

    # -- accounting and diagnostics
    def kernel_plan(self, n_tokens: int) -> int:
        """Kernel plan a batch of ``n_tokens`` runs with (0: demanded plan not runnable)."""
        return int(self._lib.s2moe_kernel_plan(self._h, int(n_tokens)))

    def kernel_launches(self) -> int:
        return int(self._lib.s2moe_kernel_launches(self._h))

    def unique_expert_bytes(self, n_unique: int) -> float:
        return float(self._lib.s2moe_unique_expert_bytes(self._h, int(n_unique)))

    def profile_begin(self, max_records: int) -> None:
        self._check(self._lib.s2moe_profile_begin(self._h, int(max_records)), "s2moe_profile_begin")

    def profile_end(self) -> Dict[str, Dict[str, float]]:
        """{kernel name: {"ms": summed duration, "launches": n}} since profile_begin."""
        ms = (ctypes.c_double * KERNEL_CLASSES)()
        n = (ctypes.c_int64 * KERNEL_CLASSES)()
        self._check(self._lib.s2moe_profile_end(self._h, KERNEL_CLASSES, ms, n), "s2moe_profile_end")
        out = {}
        for c in range(KERNEL_CLASSES):
            name = self._lib.s2moe_kernel_class_name(c)
            if name is not None and n[c] > 0:
                out[name.decode()] = {"ms": float(ms[c]), "launches": int(n[c])}
        return out

    def device_status(self) -> int:
        v = ctypes.c_int32(0)
        rc = self._lib.s2moe_last_device_status(self._h, ctypes.byref(v))
        if rc not in (OK, ETIMEOUT):
            self._check(rc, "s2moe_last_device_status")
        return int(v.value)

    def debug_read(self, what: int, count: int, dtype: torch.dtype) -> torch.Tensor:
        t = torch.zeros(max(count, 1), dtype=dtype)
        rc = self._lib.s2moe_debug_read(self._h, what, t.data_ptr(), t.numel() * t.element_size())
        self._check(rc, "s2moe_debug_read")
        return t[:count]

    def debug_lists(self) -> Dict[str, torch.Tensor]:
        """Bucketing arrays of the last call (host tensors)."""
        c = self.config
        G = c.n_experts + c.n_shared
        hdr = self.debug_read(6, 4, torch.int32)
        n_active, n_slots, U, B = (int(x) for x in hdr)
        return dict(
            n_active=n_active, n_slots=n_slots, U=U, B=B,
            logits=self.debug_read(0, B * c.n_experts, torch.float64).reshape(B, c.n_experts),
            counts=self.debug_read(1, G, torch.int32), offsets=self.debug_read(2, G + 1, torch.int32),
            slot_token=self.debug_read(3, n_slots, torch.int32), slot_w=self.debug_read(4, n_slots, torch.float32),
            active=self.debug_read(5, n_active, torch.int32))


def route_noalloc(config: Config, hidden: torch.Tensor, router: torch.Tensor,
                  conf: Optional[torch.Tensor] = None, gate_vec: Optional[torch.Tensor] = None,
                  stream: Optional[torch.cuda.Stream] = None):
    """Router logits, reuse-aware gating and the unique-expert count through
    ``s2moe_route_noalloc``: the library allocates nothing (its scratch is a fixed array in
    the library image).  For callers that may not allocate device memory while they run;
    the output tensors here are the caller's.  Returns (sel_idx, sel_w, n_unique, gate)."""
    lib = load_library()
    B = hidden.shape[0]
    dev = hidden.device
    sel_idx = torch.empty((B, config.top_k), dtype=torch.int32, device=dev)
    sel_w = torch.empty((B, config.top_k), dtype=torch.float32, device=dev)
    n_unique = torch.empty((1,), dtype=torch.int32, device=dev)
    gate = torch.empty((B,), dtype=torch.float32, device=dev) if gate_vec is not None else None
    cfg = config.c()
    rc = lib.s2moe_route_noalloc(ctypes.byref(cfg), B, _dptr(router), _dptr(gate_vec), _dptr(hidden), _dptr(conf),
                                 _dptr(sel_idx), _dptr(sel_w), _dptr(n_unique), _dptr(gate), _stream_handle(stream))
    if rc != OK:
        raise S2MoEError(rc, "s2moe_route_noalloc")
    return sel_idx, sel_w, n_unique, gate


def route_noalloc_status() -> int:
    """Device status word of the last ``route_noalloc`` call on the current device (0: no bounded
    wait gave up).  Synchronises the device."""
    out = ctypes.c_int32(0)
    rc = load_library().s2moe_route_noalloc_status(ctypes.byref(out))
    if rc not in (OK, ETIMEOUT):
        raise S2MoEError(rc, "s2moe_route_noalloc_status")
    return int(out.value)


def expert_masks(sel_idx: torch.Tensor, n_experts: int, out: Optional[torch.Tensor] = None, layer: int = 0,
                 stream: Optional[torch.cuda.Stream] = None) -> torch.Tensor:
    """Predicted expert sets as bit masks through ``s2moe_expert_masks``.  ``sel_idx`` is
    [n_tokens][top_k] int32 on the device; the result is int64 [n_tokens][n_layers][words]
    (bit e % 64 of word e / 64); with ``out`` given, layer ``layer`` of it is written."""
    lib = load_library()
    n, k = sel_idx.shape
    words = (n_experts + 63) // 64
    if out is None:
        out = torch.zeros((n, 1, words), dtype=torch.int64, device=sel_idx.device)
    n_layers = out.shape[1]
    base = out.view(-1)[layer * words:]
    rc = lib.s2moe_expert_masks(_dptr(sel_idx), n, k, n_experts, _dptr(base), n_layers * words, _stream_handle(stream))
    if rc != OK:
        raise S2MoEError(rc, "s2moe_expert_masks")
    return out


def adaptive_expand(parent: torch.Tensor, p_tok: torch.Tensor, masks: torch.Tensor, n_experts: int,
                    c_draft: Optional[torch.Tensor], t_ar: float, t_exp: float,
                    stream: Optional[torch.cuda.Stream] = None):
    """Greedy routing-aware admission through ``s2moe_adaptive_expand``.  ``masks`` is int64
    [n_cand][n_layers][words].  Returns (admitted, order, n_admitted, union) on the device."""
    lib = load_library()
    n, n_layers, words = masks.shape
    dev = masks.device
    admitted = torch.empty((n,), dtype=torch.int32, device=dev)
    order = torch.empty((n,), dtype=torch.int32, device=dev)
    n_adm = torch.empty((1,), dtype=torch.int32, device=dev)
    union = torch.empty((n_layers, words), dtype=torch.int64, device=dev)
    rc = lib.s2moe_adaptive_expand(n, n_layers, n_experts, _dptr(parent), _dptr(p_tok), _dptr(masks), _dptr(c_draft),
                                   float(t_ar), float(t_exp), _dptr(admitted), _dptr(order), _dptr(n_adm),
                                   _dptr(union), _stream_handle(stream))
    if rc != OK:
        raise S2MoEError(rc, "s2moe_adaptive_expand")
    return admitted, order, n_adm, union



class ExpertCache:
    """The replacement policy of one layer of an offloaded context, host only (``s2moe_cache_*``)."""

    def __init__(self, n_experts: int, n_slots: int, pinned: Sequence[int] = ()):
        self._lib = load_library()
        self._h = ctypes.c_void_p(None)
        arr = (ctypes.c_int32 * max(1, len(pinned)))(*[int(e) for e in pinned])
        rc = self._lib.s2moe_cache_create(int(n_experts), int(n_slots), ctypes.cast(arr, ctypes.c_void_p) if pinned else None,
                                          len(pinned), ctypes.byref(self._h))
        if rc != OK:
            self._h = ctypes.c_void_p(None)
            raise S2MoEError(rc, "s2moe_cache_create")

    def access(self, experts: Sequence[int]) -> Tuple[List[int], List[int]]:
        """Slots of ``experts`` (distinct ids) and which of them had to be fetched."""
        n = len(experts)
        ex = (ctypes.c_int32 * max(1, n))(*[int(e) for e in experts])
        sl, ms = (ctypes.c_int32 * max(1, n))(), (ctypes.c_int32 * max(1, n))()
        rc = self._lib.s2moe_cache_access(self._h, ctypes.cast(ex, ctypes.c_void_p), n, ctypes.cast(sl, ctypes.c_void_p),
                                          ctypes.cast(ms, ctypes.c_void_p))
        if rc != OK:
            raise S2MoEError(rc, "s2moe_cache_access")
        return list(sl)[:n], list(ms)[:n]

    def close(self) -> None:
        if getattr(self, "_h", None) is not None and self._h.value:
            self._lib.s2moe_cache_destroy(self._h)
            self._h = ctypes.c_void_p(None)

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
