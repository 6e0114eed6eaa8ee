"""Seeded synthetic inputs for the MoE verification layer.

This module only draws random numbers and stores them in the layer's input
formats (fp32, bf16, block-int4 + fp16 scales).  It contains none of the
method's arithmetic and is the one module that both the CUDA path's callers
and the CPU oracle's tests may import, so that both sides see the same bytes.

The five workloads mirror the shapes of the model families the paper evaluates
(Table 1: experts, experts per token, cap), with draft batches whose hidden
states are correlated the way neighbouring draft tokens are: a shared base plus
per-token noise (chain batches) or parent plus noise (draft trees).  They stand
in for real-model routing on the paper's evaluation tasks; no dataset item or
trained weight is involved.
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import Dict, Optional

import numpy as np
import torch

F32, BF16, Q4B32 = 0, 1, 2
_TORCH_DTYPE = {F32: torch.float32, BF16: torch.bfloat16}


@dataclass(frozen=True)
class Workload:
    name: str
    d_model: int
    d_ff: int
    n_experts: int
    top_k: int
    n_layers: int
    n_tokens: int
    structure: str              # "chain" (base + noise) or "tree" (parent + noise, heap order)
    sigma: float                # per-token noise scale
    seed: int
    n_shared: int = 0
    d_ff_shared: int = 0
    shared_gate: bool = False   # sigmoid(h . w_sg) scaling of the shared expert
    act_dtype: int = BF16
    router_dtype: int = BF16
    weight_dtype: int = BF16
    renorm: int = 0
    cap: int = 0
    alpha: float = 0.5
    weight_mode: int = 0
    weight_std: float = 0.02

    def with_(self, **kw) -> "Workload":
        return replace(self, **kw)

    # ---- byte counts used by the benchmark's roofline figures -------------
    def weight_bytes_per_element(self) -> float:
        return {F32: 4.0, BF16: 2.0, Q4B32: 0.5 + 2.0 / 32.0}[self.weight_dtype]

    def expert_bytes(self) -> float:
        return 3.0 * self.d_model * self.d_ff * self.weight_bytes_per_element()

    def shared_bytes(self) -> float:
        return self.n_shared * 3.0 * self.d_model * self.d_ff_shared * self.weight_bytes_per_element()


# cap: Table 1 where the paper lists the family (OLMoE 18, DeepSeek 16), else 2x top-k
# (inside the 1.5x-2.5x range of the cap sensitivity study).
CONFIGS: Dict[str, Workload] = {
    "cfg1": Workload("cfg1-tiny-f32", 256, 512, 8, 2, 1, 4, "chain", 0.3, 0,
                     act_dtype=F32, router_dtype=F32, weight_dtype=F32, renorm=1, cap=3),
    "cfg2": Workload("cfg2-olmoe-bf16", 2048, 1024, 64, 8, 16, 8, "chain", 0.5, 1, cap=18),
    "cfg3": Workload("cfg3-qwen15moe-bf16", 2048, 1408, 60, 4, 24, 16, "tree", 0.3, 2,
                     n_shared=1, d_ff_shared=5632, shared_gate=True, cap=8),
    "cfg4": Workload("cfg4-mixtral-q4", 4096, 14336, 8, 2, 32, 8, "chain", 0.5, 3,
                     weight_dtype=Q4B32, renorm=1, cap=4),
    "cfg5": Workload("cfg5-dsv2lite-bf16", 2048, 1408, 64, 6, 26, 16, "tree", 0.3, 4,
                     n_shared=2, d_ff_shared=1408, cap=16),
}
# 128-expert shapes of Table 1 (cap 14 and 6 as listed there): token masks and expert sets span
# two 64-bit words, the routing kernel holds four experts per lane.  Fewer layers than the models
# have, so that a stack stays within tens of GB.
CONFIGS["e128a"] = Workload("e128a-qwen3moe-like-bf16", 2048, 768, 128, 8, 12, 8, "chain", 0.5, 5, renorm=1, cap=14)
CONFIGS["e128b"] = Workload("e128b-gptoss-like-bf16", 2880, 2880, 128, 4, 4, 8, "chain", 0.5, 6, renorm=1, cap=6)
CFG4_BATCHES = (1, 2, 4, 8, 16, 32)
CFG5_TREES = (1, 2, 4, 8, 16, 32, 64)
CFG5_SIGMAS = (0.1, 0.2, 0.3, 0.5, 0.7, 1.0)

_KINDS = ("router", "w_gate", "w_up", "w_down", "sh_gate", "sh_up", "sh_down", "sh_scale",
          "hidden", "conf")


def _gen(wl: Workload, layer: int, kind: str, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed((wl.seed * 1_000_003 + layer) * 64 + _KINDS.index(kind) + 1)
    return g


def quantize_q4b32(w: torch.Tensor):
    """Symmetric block-int4 storage of a float32 tensor [..., K], K % 32 == 0.

    Blocks of 32 run along the last (contraction) dimension.  Per block:
    scale = fp16(absmax / 7); q = clamp(round_half_even(w / scale), -7, 7), q = 0
    when the scale is 0; weight i of a block is stored as q + 8 in nibble i
    (byte i // 2, low nibble for even i).  Returns (uint8 [..., K/2], fp16 [..., K/32]).
    """
    K = w.shape[-1]
    assert K % 32 == 0
    blocks = w.reshape(-1, 32).float()
    scale = (blocks.abs().amax(dim=1) / 7.0).to(torch.float16)
    sf = scale.float().unsqueeze(1)
    q = torch.where(sf > 0, torch.round(blocks / sf), torch.zeros_like(blocks)).clamp_(-7, 7)
    nib = (q + 8).to(torch.uint8)
    packed = nib[:, 0::2] | (nib[:, 1::2] << 4)
    return (packed.reshape(*w.shape[:-1], K // 2).contiguous(),
            scale.reshape(*w.shape[:-1], K // 32).contiguous())


def _normal(shape, std, gen, device):
    return torch.randn(shape, generator=gen, device=device, dtype=torch.float32) * std


def _store_matrix(wl: Workload, w: torch.Tensor, out: dict, name: str, sname: str):
    if wl.weight_dtype == Q4B32:
        parts = [quantize_q4b32(w[e]) for e in range(w.shape[0])]
        out[name] = torch.stack([p[0] for p in parts])
        out[sname] = torch.stack([p[1] for p in parts])
    else:
        out[name] = w.to(_TORCH_DTYPE[wl.weight_dtype])


def layer_weights(wl: Workload, layer: int, device="cpu") -> Dict[str, torch.Tensor]:
    """All weight tensors of one layer, in storage format, on ``device``."""
    E, d, f = wl.n_experts, wl.d_model, wl.d_ff
    out: Dict[str, torch.Tensor] = {}
    out["router"] = _normal((E, d), wl.weight_std, _gen(wl, layer, "router", device), device).to(
        _TORCH_DTYPE[wl.router_dtype])
    for name, shape in (("w_gate", (E, f, d)), ("w_up", (E, f, d)), ("w_down", (E, d, f))):
        w = _normal(shape, wl.weight_std, _gen(wl, layer, name, device), device)
        _store_matrix(wl, w, out, name, "s_" + name[2:])
        del w
    if wl.n_shared > 0:
        n, fs = wl.n_shared, wl.d_ff_shared
        for name, shape in (("sh_gate", (n, fs, d)), ("sh_up", (n, fs, d)), ("sh_down", (n, d, fs))):
            w = _normal(shape, wl.weight_std, _gen(wl, layer, name, device), device)
            _store_matrix(wl, w, out, name, "sh_s_" + name[3:])
            del w
        if wl.shared_gate:
            out["sh_scale"] = _normal((d,), wl.weight_std, _gen(wl, layer, "sh_scale", device),
                                      device).to(_TORCH_DTYPE[wl.router_dtype])
    return out


def tree_parent(i: int) -> int:
    """Heap-ordered draft tree: node 0 is the root, every node has at most two children."""
    return (i - 1) // 2


def hidden_states(wl: Workload, layer: int, n_tokens: Optional[int] = None,
                  sigma: Optional[float] = None, device="cpu") -> torch.Tensor:
    """[B][d] hidden states in the activation dtype."""
    B = wl.n_tokens if n_tokens is None else n_tokens
    s = wl.sigma if sigma is None else sigma
    gen = _gen(wl, layer, "hidden", device)
    d = wl.d_model
    base = _normal((d,), 1.0, gen, device)
    eps = _normal((B, d), 1.0, gen, device)
    if wl.structure == "chain":
        h = base.unsqueeze(0) + s * eps
    else:
        h = torch.empty((B, d), device=device, dtype=torch.float32)
        h[0] = base
        for i in range(1, B):
            h[i] = h[tree_parent(i)] + s * eps[i]
    return h.to(_TORCH_DTYPE[wl.act_dtype]).contiguous()


def confidences(wl: Workload, layer: int, n_tokens: Optional[int] = None,
                device="cpu") -> torch.Tensor:
    """[B] float32 prefix confidences: per-token c ~ U(0.5, 1), multiplied along the
    path from the first draft token (chain) or from the root (tree)."""
    B = wl.n_tokens if n_tokens is None else n_tokens
    gen = _gen(wl, layer, "conf", device)
    c = 0.5 + 0.5 * torch.rand((B,), generator=gen, device=device, dtype=torch.float32)
    c = c.cpu()
    p = torch.empty(B, dtype=torch.float32)
    for i in range(B):
        if i == 0:
            p[i] = c[i]
        else:
            par = i - 1 if wl.structure == "chain" else tree_parent(i)
            p[i] = p[par] * c[i]
    return p.to(device)


def raw_numpy(t: Optional[torch.Tensor]) -> Optional[np.ndarray]:
    """Bytes of a storage tensor as numpy: bf16/fp16 -> uint16, others unchanged."""
    if t is None:
        return None
    t = t.detach().cpu().contiguous()
    if t.dtype in (torch.bfloat16, torch.float16):
        return t.view(torch.int16).numpy().view(np.uint16)
    return t.numpy()
