"""The comparison rules of oracle/parity.py on hand-made results (CPU only): what the GPU
parity tests accept and reject is itself checked here, with the oracle's own output as the
"other side" and deliberate defects put into it."""
import numpy as np
import pytest

import oracle
from oracle import parity


def _case(seed=0, B=5, E=9, k=3, d=8, f=6):
    rng = np.random.default_rng(seed)
    W = oracle.Weights(router=rng.normal(0, 1, (E, d)).astype(np.float32),
                       w_gate=rng.normal(0, 0.3, (E, f, d)).astype(np.float32),
                       w_up=rng.normal(0, 0.3, (E, f, d)).astype(np.float32),
                       w_down=rng.normal(0, 0.3, (E, d, f)).astype(np.float32))
    cfg = oracle.Config(d_model=d, d_ff=f, n_experts=E, top_k=k, cap=5, alpha=0.5, renorm=0, weight_mode=0)
    H = rng.normal(0, 1, (B, d)).astype(np.float32)
    conf = rng.uniform(0.5, 1.0, B)
    return cfg, W, H, conf, oracle.layer(cfg, W, H, conf)


def test_checker_accepts_the_oracle_and_counts_ordered_tokens():
    cfg, W, H, conf, r = _case()
    rep = parity.check_layer(cfg, W, H, conf, r.y, r.sel, r.pw, r.n_unique, 2e-3)
    assert rep.tokens_checked == 5 and rep.order_checked == 5 and not rep.ties
    assert rep.max_rel_err == 0.0 and rep.rms_rel_err == 0.0


def test_checker_rejects_a_wrong_selection_order():
    cfg, W, H, conf, r = _case()
    sel, pw = r.sel.copy(), r.pw.copy()
    sel[2, [0, 1]] = sel[2, [1, 0]]          # same set, same weights by expert, other order
    pw[2, [0, 1]] = pw[2, [1, 0]]
    with pytest.raises(AssertionError, match="selection order"):
        parity.check_layer(cfg, W, H, conf, r.y, sel, pw, r.n_unique, 2e-3)


def test_checker_rejects_a_wrong_expert_and_a_wrong_count():
    cfg, W, H, conf, r = _case()
    sel = r.sel.copy()
    others = [e for e in range(cfg.n_experts) if e not in sel[1]]
    sel[1, -1] = others[0]
    with pytest.raises(AssertionError, match="not a tie"):
        parity.check_layer(cfg, W, H, conf, r.y, sel, r.pw, r.n_unique, 2e-3)
    with pytest.raises(AssertionError, match="n_unique"):
        parity.check_layer(cfg, W, H, conf, r.y, r.sel, r.pw, r.n_unique + 1, 2e-3)


def test_checker_bounds_the_rms_error_as_well_as_the_largest_element():
    cfg, W, H, conf, r = _case()
    y = r.y.copy()
    scale = np.abs(y[0]).max()
    # every element off by 0.9 tolerances of the largest one: the inf-norm criterion passes,
    # the RMS criterion (a quarter of the tolerance) does not
    y[0] += 0.9 * 2e-3 * scale
    with pytest.raises(AssertionError, match="RMS"):
        parity.check_layer(cfg, W, H, conf, y, r.sel, r.pw, r.n_unique, 2e-3)
    y = r.y.copy()
    y[0, int(np.argmax(np.abs(y[0])))] *= 1 + 0.4e-3        # one element, inside both bounds
    parity.check_layer(cfg, W, H, conf, y, r.sel, r.pw, r.n_unique, 2e-3)
    y[0, 0] += 3e-3 * scale
    with pytest.raises(AssertionError, match="relative error"):
        parity.check_layer(cfg, W, H, conf, y, r.sel, r.pw, r.n_unique, 2e-3)


def test_checker_accepts_a_reported_tie_with_the_other_choice_forced():
    # two experts with identical router rows: their logits tie exactly; picking the other one
    # is accepted, reported, and the outputs are compared with that choice forced
    for seed in range(40):
        cfg, W, H, conf, _ = _case(seed)
        W.router[4] = W.router[3]
        r = oracle.layer(cfg, W, H, conf)
        b = next((b for b in range(H.shape[0]) if (3 in r.sel[b]) != (4 in r.sel[b])), None)
        if b is not None:
            break
    assert b is not None, "no seed puts the tied pair at a token's selection boundary"
    sel = r.sel.copy()
    j = int(np.nonzero((sel[b] == 3) | (sel[b] == 4))[0][0])
    sel[b, j] = 7 - sel[b, j]
    forced = oracle.layer(cfg, W, H, conf, forced_sel=sel)
    rep = parity.check_layer(cfg, W, H, conf, forced.y, sel, forced.pw, forced.n_unique, 2e-3)
    assert rep.ties
