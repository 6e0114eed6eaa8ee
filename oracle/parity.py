"""Comparison of a layer result (plain numpy arrays, however produced) with the oracle.

TEST INFRASTRUCTURE.  Takes arrays only, so it imports nothing from the CUDA path.

Rules applied
  * selected experts are compared per token exactly and in selection order (biased
    logit descending, original logit descending, id ascending), and the unique-expert
    count exactly.  A differing token is tolerated only as a router tie: the oracle's
    margin at that decision (k-th minus (k+1)-th biased logit of the token, or the
    cap-th minus (cap+1)-th aggregated importance; for a difference in order alone, the
    gap between the two swapped biased logits) must be below ``tie_eps``; the oracle is
    then re-evaluated with the other side's choice forced, and the tie is reported.
  * mixing weights are matched by expert id, absolute tolerance ``w_tol``.
  * outputs: per token, max |y - y_ref| / max |y_ref| <= ``y_tol`` (per-token
    infinity-norm relative error; element-wise relative error is meaningless at the
    zero crossings of y); and, so that an error confined to small elements cannot
    hide under the largest one, the per-token RMS error relative to the RMS of y_ref
    must stay below ``y_tol / 4``.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Optional, Sequence

import numpy as np

from . import Config, Weights, gating as oracle_gating, layer as oracle_layer


@dataclass
class ParityReport:
    max_rel_err: float = 0.0
    rms_rel_err: float = 0.0
    max_w_err: float = 0.0
    n_unique: int = 0
    ties: List[str] = field(default_factory=list)
    tokens_checked: int = 0
    order_checked: int = 0      # tokens whose selection ORDER was compared exactly


def check_layer(cfg: Config, w: Weights, hidden_raw: np.ndarray, conf: Optional[np.ndarray],
                got_y: Optional[np.ndarray], got_sel: np.ndarray, got_w: np.ndarray, got_unique: int,
                y_tol: float, tok_list: Optional[Sequence[int]] = None, tie_eps: float = 1e-6,
                w_tol: float = 2e-6) -> ParityReport:
    B = hidden_raw.shape[0]
    k = cfg.top_k
    toks = list(range(B)) if tok_list is None else list(tok_list)
    conf64 = None if conf is None else np.asarray(conf, dtype=np.float64)
    ref = oracle_layer(cfg, w, hidden_raw, conf64, tok_list=toks if got_y is not None else [])
    rep = ParityReport(n_unique=ref.n_unique)

    got_sel = np.asarray(got_sel).reshape(B, k)
    got_w = np.asarray(got_w, dtype=np.float64).reshape(B, k)
    mism = [b for b in range(B) if set(got_sel[b].tolist()) != set(ref.sel[b].tolist())]
    # same set, other order: allowed only between experts whose biased logits differ by less
    # than the tie threshold in the oracle
    gate = None
    for b in range(B):
        if b in mism:
            continue
        if got_sel[b].tolist() == ref.sel[b].tolist():
            rep.order_checked += 1
            continue
        if gate is None:
            gate = oracle_gating(cfg, ref.logits, conf64)
        l2 = gate.l2[b]
        for j in range(k):
            a, c = int(got_sel[b, j]), int(ref.sel[b, j])
            if a != c and abs(l2[a] - l2[c]) >= tie_eps:
                raise AssertionError(f"token {b}: selection order {got_sel[b].tolist()} != oracle "
                                     f"{ref.sel[b].tolist()} (biased logits {l2[a]:.9g}, {l2[c]:.9g}: not a tie)")
        rep.ties.append(f"token {b}: order of near-equal biased logits")
    if mism:
        wsum = float(conf64.sum()) if conf64 is not None else float(B)
        cap_tie = ref.m_cap < tie_eps * max(1.0, wsum)
        for b in mism:
            if not (ref.m_tok[b] < tie_eps or cap_tie):
                raise AssertionError(
                    f"token {b}: experts {sorted(got_sel[b].tolist())} != oracle "
                    f"{sorted(ref.sel[b].tolist())} with margins m_tok={ref.m_tok[b]:.3e} "
                    f"m_cap={ref.m_cap:.3e} (not a tie)")
            rep.ties.append(f"token {b}: m_tok={ref.m_tok[b]:.3e} m_cap={ref.m_cap:.3e}")
        for b in range(B):
            assert len(set(got_sel[b].tolist())) == k and got_sel[b].min() >= 0 and got_sel[b].max() < cfg.n_experts
        ref = oracle_layer(cfg, w, hidden_raw, conf64, forced_sel=got_sel.astype(np.int32),
                           tok_list=toks if got_y is not None else [])
        rep.n_unique = ref.n_unique
    assert int(got_unique) == rep.n_unique, f"n_unique {got_unique} != oracle {rep.n_unique}"

    for b in range(B):
        order = {int(e): j for j, e in enumerate(ref.sel[b])}
        for j in range(k):
            err = abs(got_w[b, j] - ref.pw[b, order[int(got_sel[b, j])]])
            rep.max_w_err = max(rep.max_w_err, err)
    assert rep.max_w_err <= w_tol, f"mixing weight error {rep.max_w_err:.3e} > {w_tol}"

    if got_y is not None:
        got_y = np.asarray(got_y, dtype=np.float64)
        errs = []
        for n, b in enumerate(toks):
            scale = np.abs(ref.y[n]).max()
            diff = np.abs(got_y[b] - ref.y[n])
            rel = diff.max() / scale if scale > 0 else diff.max()
            errs.append(rel)
            rms = np.sqrt(np.mean(diff ** 2)) / (np.sqrt(np.mean(ref.y[n] ** 2)) + 1e-300)
            rep.rms_rel_err = max(rep.rms_rel_err, float(rms))
        rep.max_rel_err = float(max(errs)) if errs else 0.0
        rep.tokens_checked = len(toks)
        assert rep.max_rel_err <= y_tol, f"output relative error {rep.max_rel_err:.3e} > {y_tol}"
        assert rep.rms_rel_err <= y_tol / 4, f"output RMS relative error {rep.rms_rel_err:.3e} > {y_tol / 4}"
    return rep


def check_bucketing(lists: dict, sel: np.ndarray, w: np.ndarray, n_experts: int, n_shared: int) -> None:
    """Host-side validation of the bucketing arrays a layer call produced: the active
    list holds exactly the groups that have tokens, the routed ones before the shared
    ones (the order among the routed ones is the kernel's choice: not unique, so only
    its validity is checked); walking that list, the groups' slot ranges follow each
    other without gap or overlap from slot 0 on; every (token, choice) pair appears
    exactly once under its expert with its mixing weight, and tokens ascend inside an
    expert."""
    B, k = sel.shape
    counts = np.asarray(lists["counts"]); offsets = np.asarray(lists["offsets"])
    slot_token = np.asarray(lists["slot_token"]); slot_w = np.asarray(lists["slot_w"])
    active = np.asarray(lists["active"])
    G = n_experts + n_shared
    assert lists["B"] == B and lists["n_slots"] == B * k + n_shared * B
    assert counts.shape[0] == G and offsets.shape[0] == G + 1
    assert counts[:n_experts].sum() == B * k and np.all(counts[n_experts:] == B)
    assert lists["U"] == int((counts[:n_experts] > 0).sum())
    assert sorted(active.tolist()) == [g for g in range(G) if counts[g] > 0]
    assert len(set(active.tolist())) == len(active)
    routed = [g for g in active.tolist() if g < n_experts]
    assert active.tolist() == routed + list(range(n_experts, G)), "shared groups close the active list, ascending"
    at = 0
    for g in active.tolist():
        assert offsets[g] == at, f"group {g} starts at slot {offsets[g]}, expected {at}"
        at += int(counts[g])
    assert at == lists["n_slots"] and offsets[G] == at
    seen = set()
    for e in range(n_experts):
        toks = slot_token[offsets[e]:offsets[e] + counts[e]]
        assert np.all(np.diff(toks) > 0), "tokens must ascend inside an expert"
        for pos, b in zip(range(offsets[e], offsets[e] + counts[e]), toks):
            j = np.nonzero(sel[b] == e)[0]
            assert len(j) == 1, f"slot {pos}: token {b} did not select expert {e}"
            assert slot_w[pos] == w[b, j[0]]
            seen.add((int(b), e))
    assert len(seen) == B * k
    for s in range(n_shared):
        g = n_experts + s
        assert slot_token[offsets[g]:offsets[g] + counts[g]].tolist() == list(range(B))


def from_workload(wl, tensors: dict):
    """Oracle (Config, Weights) for a workload description and its storage tensors
    (torch tensors on any device; copied to host bytes)."""
    from paper_2608_15018_b200.workloads import raw_numpy  # generator module: shared by design

    cfg = Config(wl.d_model, wl.d_ff, wl.n_experts, wl.top_k, wl.n_shared, wl.d_ff_shared,
                 wl.act_dtype, wl.router_dtype, wl.weight_dtype, wl.renorm, wl.cap, wl.weight_mode,
                 float(np.float32(wl.alpha)))
    return cfg, Weights(**{n: raw_numpy(t) for n, t in tensors.items()})
