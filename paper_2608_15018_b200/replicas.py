"""Multi-GPU policy of the benchmark: independent replicas, no data-path collective.

The verification layer has no exchange step, so N GPUs run N independent replicas of the
stack (each with its own seed, as independent requests would).  The only communication is
the timing protocol: a barrier around the timed region and the maximum over ranks of the
measured time.  These helpers hold that logic so that it can be tested on CPU with gloo.
"""
from __future__ import annotations

from typing import Sequence

import torch
import torch.distributed as dist


def replica_workload(wl, rank: int):
    """The workload replica ``rank`` runs: same shapes, its own seed."""
    return wl.with_(seed=wl.seed + 1000 * rank)


def max_over_ranks(values: Sequence[float], device="cpu") -> list:
    """Element-wise maximum of ``values`` over all ranks (identity without a process group)."""
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.tolist()


def aggregate_tokens_per_s(world: int, n_tokens: int, n_layers: int, ms_per_step: float) -> float:
    """Whole-job verified tokens/s per layer: every replica verifies n_tokens per layer in the
    slowest replica's step time."""
    return world * n_tokens * n_layers / (ms_per_step * 1e-3)
