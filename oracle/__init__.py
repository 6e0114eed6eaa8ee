"""Float64 CPU oracle of the MoE verification layer -- TEST INFRASTRUCTURE.

Only tests, the smoke check and the benchmark's CPU-baseline leg may import this
package.  It wraps ``s2moe_oracle.c`` (plain C, float64, one token and one expert
at a time) through ctypes and shares nothing with the CUDA library.

Stored number formats are passed as raw numpy arrays:
  F32   -> float32, BF16 -> uint16 (upper half of a float32),
  Q4B32 -> uint8 nibble blocks plus uint16 (binary16) scales.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass, field
from typing import Optional, Sequence

import numpy as np

F32, BF16, Q4B32 = 0, 1, 2

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "s2moe_oracle.c")
_LIB = os.path.join(_HERE, "libs2moe_oracle.so")


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O2, OpenMP).  Returns the library path."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(
            ["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-o", _LIB, _SRC, "-lm"]
        )
    return _LIB


class _Cfg(ctypes.Structure):
    _fields_ = [
        (n, ctypes.c_int32)
        for n in (
            "d_model", "d_ff", "n_experts", "top_k", "n_shared", "d_ff_shared",
            "act_dtype", "router_dtype", "weight_dtype", "renorm", "cap", "weight_mode",
        )
    ] + [("alpha", ctypes.c_double)]


class _W(ctypes.Structure):
    _fields_ = [
        (n, ctypes.c_void_p)
        for n in (
            "router", "w_gate", "w_up", "w_down", "s_gate", "s_up", "s_down",
            "sh_gate", "sh_up", "sh_down", "sh_s_gate", "sh_s_up", "sh_s_down", "sh_scale",
        )
    ]


_lib = None


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        lib.orc_threads.restype = ctypes.c_int
        lib.orc_set_threads.argtypes = [ctypes.c_int]
        _lib = lib
    return _lib


@dataclass
class Config:
    d_model: int
    d_ff: int
    n_experts: int
    top_k: int
    n_shared: int = 0
    d_ff_shared: int = 0
    act_dtype: int = F32
    router_dtype: int = F32
    weight_dtype: int = F32
    renorm: int = 1
    cap: int = 0          # 0 -> n_experts (bias off)
    weight_mode: int = 0
    alpha: float = 0.5

    def c(self) -> _Cfg:
        cap = self.cap if self.cap > 0 else self.n_experts
        return _Cfg(self.d_model, self.d_ff, self.n_experts, self.top_k, self.n_shared,
                    self.d_ff_shared, self.act_dtype, self.router_dtype, self.weight_dtype,
                    self.renorm, cap, self.weight_mode, float(self.alpha))


@dataclass
class Weights:
    """Raw arrays of one layer (see module docstring for the storage dtypes)."""
    router: np.ndarray
    w_gate: np.ndarray
    w_up: np.ndarray
    w_down: np.ndarray
    s_gate: Optional[np.ndarray] = None
    s_up: Optional[np.ndarray] = None
    s_down: Optional[np.ndarray] = None
    sh_gate: Optional[np.ndarray] = None
    sh_up: Optional[np.ndarray] = None
    sh_down: Optional[np.ndarray] = None
    sh_s_gate: Optional[np.ndarray] = None
    sh_s_up: Optional[np.ndarray] = None
    sh_s_down: Optional[np.ndarray] = None
    sh_scale: Optional[np.ndarray] = None
    _keep: list = field(default_factory=list, repr=False)

    def c(self) -> _W:
        vals = []
        for name, _ in _W._fields_:
            a = getattr(self, name)
            if a is None:
                vals.append(None)
            else:
                a = np.ascontiguousarray(a)
                self._keep.append(a)
                vals.append(a.ctypes.data)
        return _W(*vals)


def _ptr(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


@dataclass
class Gating:
    g: np.ndarray
    estar: np.ndarray
    lam: np.ndarray
    l2: np.ndarray
    sel: np.ndarray
    pw: np.ndarray
    n_unique: int
    counts: np.ndarray
    m_cap: float
    m_tok: np.ndarray


def router_logits(cfg: Config, hidden: np.ndarray, router: np.ndarray) -> np.ndarray:
    lib = _load()
    hidden = np.ascontiguousarray(hidden)
    router = np.ascontiguousarray(router)
    B = hidden.shape[0]
    out = np.empty((B, cfg.n_experts), dtype=np.float64)
    c = cfg.c()
    lib.orc_router_logits(ctypes.byref(c), B, _ptr(hidden), _ptr(router), _ptr(out))
    return out


def gating(cfg: Config, logits: np.ndarray, conf: Optional[np.ndarray] = None,
           forced_sel: Optional[np.ndarray] = None) -> Gating:
    lib = _load()
    logits = np.ascontiguousarray(logits, dtype=np.float64)
    B, E = logits.shape
    assert E == cfg.n_experts
    k = cfg.top_k
    if conf is not None:
        conf = np.ascontiguousarray(conf, dtype=np.float64)
    if forced_sel is not None:
        forced_sel = np.ascontiguousarray(forced_sel, dtype=np.int32)
    g = np.zeros(E); estar = np.zeros(E, np.int32); lam = np.zeros(B); l2 = np.zeros((B, E))
    sel = np.zeros((B, k), np.int32); pw = np.zeros((B, k)); nu = ctypes.c_int32(0)
    counts = np.zeros(E, np.int32); m_cap = ctypes.c_double(0.0); m_tok = np.zeros(B)
    c = cfg.c()
    lib.orc_gating(ctypes.byref(c), B, _ptr(logits), _ptr(conf), _ptr(forced_sel), _ptr(g),
                   _ptr(estar), _ptr(lam), _ptr(l2), _ptr(sel), _ptr(pw), ctypes.byref(nu),
                   _ptr(counts), ctypes.byref(m_cap), _ptr(m_tok))
    return Gating(g, estar, lam, l2, sel, pw, int(nu.value), counts, float(m_cap.value), m_tok)


@dataclass
class LayerResult:
    y: np.ndarray          # [n_list][d] float64 (rows follow tok_list)
    sel: np.ndarray        # [B][k] int32, selection order
    pw: np.ndarray         # [B][k] float64
    n_unique: int
    logits: np.ndarray     # [B][E] float64
    m_cap: float
    m_tok: np.ndarray


def layer(cfg: Config, w: Weights, hidden: np.ndarray, conf: Optional[np.ndarray] = None,
          forced_sel: Optional[np.ndarray] = None,
          tok_list: Optional[Sequence[int]] = None) -> LayerResult:
    """One verification layer.  ``tok_list`` limits the (expensive) expert
    evaluation to some tokens; routing always covers the whole batch."""
    lib = _load()
    hidden = np.ascontiguousarray(hidden)
    B = hidden.shape[0]
    E, k, d = cfg.n_experts, cfg.top_k, cfg.d_model
    if tok_list is None:
        tok_list = list(range(B))
    toks = np.ascontiguousarray(np.asarray(tok_list, dtype=np.int32))
    if conf is not None:
        conf = np.ascontiguousarray(conf, dtype=np.float64)
    if forced_sel is not None:
        forced_sel = np.ascontiguousarray(forced_sel, dtype=np.int32)
    y = np.zeros((len(toks), d)); sel = np.zeros((B, k), np.int32); pw = np.zeros((B, k))
    nu = ctypes.c_int32(0); logits = np.zeros((B, E)); m_cap = ctypes.c_double(0.0)
    m_tok = np.zeros(B)
    c = cfg.c(); cw = w.c()
    lib.orc_layer(ctypes.byref(c), ctypes.byref(cw), B, _ptr(hidden), _ptr(conf),
                  _ptr(forced_sel), len(toks), _ptr(toks), _ptr(y), _ptr(sel), _ptr(pw),
                  ctypes.byref(nu), _ptr(logits), ctypes.byref(m_cap), _ptr(m_tok))
    return LayerResult(y, sel, pw, int(nu.value), logits, float(m_cap.value), m_tok)


def decode_row(dtype: int, w: np.ndarray, scales: Optional[np.ndarray], row: int, K: int) -> np.ndarray:
    """Stored values of one row of a [rows][K] matrix, as the oracle reads them."""
    lib = _load()
    w = np.ascontiguousarray(w)
    if scales is not None:
        scales = np.ascontiguousarray(scales)
    out = np.zeros(K)
    lib.orc_decode_row(int(dtype), _ptr(w), _ptr(scales), ctypes.c_int64(row), int(K), _ptr(out))
    return out


def threads() -> int:
    return int(_load().orc_threads())


def set_threads(n: int) -> None:
    _load().orc_set_threads(int(n))
