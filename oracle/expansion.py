"""TEST INFRASTRUCTURE -- float64 / Python-integer oracle of the routing-aware adaptive
speculative expansion (Sec. 4.1).  Only tests, the smoke check and the CPU-baseline leg of the
benchmark may import this module; the CUDA path shares no code with it.

What it computes, in the paper's order and notation:

  * prefix confidence  p_i = prod_{j on the path to i} p_{i,j}          ("Expected Benefit")
  * expected benefit   B_i = p_i * T_AR
  * marginal verification cost (Eq. 2)
        dC(i | S) = | E_i \\ U_{j in S} E_j | * T_exp
    with the predicted expert sets given per MoE layer: the set difference is taken layer by
    layer and the new experts of all layers are added up (an expert is a (layer, id) pair)
  * utility (Eq. 3)    U_i = B_i / (dC(i | S) + C_i^draft)
  * greedy admission   candidates with U_i >= 1 are admitted until none is left

Readings where the text is silent (also listed in the design notes):
  * a candidate is eligible once its parent is admitted (roots are always eligible): a token
    can only be accepted after its ancestors, which is what p_i already expresses;
  * each step re-evaluates all eligible candidates against the current S and admits the one of
    largest utility (ties: lowest index); the loop stops when that utility is below 1;
  * a candidate whose total cost is 0 has utility +inf.

PARITY UNPINNED: the admission order (largest utility first, lowest index on ties) and the
eligibility rule are this build's readings; the arithmetic of Eq. 2 and Eq. 3 is pinned.
"""
from __future__ import annotations

import math
from typing import List, Sequence, Tuple


def expert_masks(sel_idx: Sequence[Sequence[int]]) -> List[int]:
    """Predicted expert set of every token as a Python integer bitmask (bit e = expert e)."""
    out = []
    for row in sel_idx:
        m = 0
        for e in row:
            m |= 1 << int(e)
        out.append(m)
    return out


def prefix_confidence(parent: Sequence[int], p_tok: Sequence[float]) -> List[float]:
    """p_i = p_tok[i] * p_parent(i), the root's children having parent -1 ("Expected Benefit").
    Parents come before their children."""
    p = [0.0] * len(parent)
    for i, (a, c) in enumerate(zip(parent, p_tok)):
        if a >= i:
            raise ValueError("parents must precede their children")
        p[i] = float(c) if a < 0 else p[a] * float(c)
    return p


def new_experts(masks_i: Sequence[int], union: Sequence[int]) -> int:
    """| E_i \\ union | summed over the layers (Eq. 2 without the factor T_exp)."""
    return sum(bin(m & ~u).count("1") for m, u in zip(masks_i, union))


def utility(p_i: float, n_new: int, c_draft: float, t_ar: float, t_exp: float) -> float:
    """Eq. 3; a zero total cost gives +inf."""
    cost = float(n_new) * float(t_exp) + float(c_draft)
    benefit = float(p_i) * float(t_ar)
    if cost == 0.0:
        return math.inf
    return benefit / cost


def adaptive_expand(parent: Sequence[int], p_tok: Sequence[float], masks: Sequence[Sequence[int]],
                    c_draft: Sequence[float], t_ar: float, t_exp: float) -> Tuple[List[int], List[int], List[int]]:
    """Greedy admission ("Adaptive Expansion").

    parent[i]   index of the parent candidate, -1 for children of the verified prefix
    p_tok[i]    token-level confidence p_{i,j} of candidate i
    masks[i][l] predicted expert set of candidate i in MoE layer l (integer bitmask)
    c_draft[i]  draft expansion cost C_i^draft
    Returns (admitted flags, admission order, per-layer union of the admitted sets).
    """
    n = len(parent)
    n_layers = len(masks[0]) if n else 0
    p = prefix_confidence(parent, p_tok)
    admitted = [0] * n
    order: List[int] = []
    union = [0] * n_layers
    while True:
        best, best_u = -1, -math.inf
        for i in range(n):
            if admitted[i] or (parent[i] >= 0 and not admitted[parent[i]]):
                continue
            u = utility(p[i], new_experts(masks[i], union), c_draft[i], t_ar, t_exp)
            if u > best_u:
                best, best_u = i, u
        if best < 0 or not (best_u >= 1.0):
            break
        admitted[best] = 1
        order.append(best)
        union = [u | m for u, m in zip(union, masks[best])]
    return admitted, order, union
