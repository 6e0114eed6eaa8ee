"""Pins of the float64 oracle against things other than itself (CPU only).

Each test fixes the oracle to a closed form, a hand-worked example, a brute-force
definition on tiny inputs, a textbook special case evaluated with library
routines, or an invariant the method must have, chosen so that a dropped term, a
wrong sign or index, or a transposed operand fails at least one of them.
"""
import itertools
import math
import os

import numpy as np
import pytest
import torch

import oracle
from oracle import BF16, F32, Q4B32
from paper_2608_15018_b200 import workloads as wl

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ----------------------------------------------------------------- helpers

def read_fig_toy():
    vals = {"logits": {}, "standard_sel": {}, "biased_sel": {}, "weights": {}}
    with open(os.path.join(GOLDEN, "fig_toy.txt")) as fh:
        for line in fh:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            key, *rest = line.split()
            if key in vals and isinstance(vals[key], dict):
                vals[key][int(rest[0])] = [float(x) for x in rest[1:]]
            else:
                vals[key] = [float(x) for x in rest]
    return vals


def gate_cfg(E, k, cap=0, alpha=0.5, renorm=1, weight_mode=0):
    return oracle.Config(d_model=1, d_ff=1, n_experts=E, top_k=k, cap=cap, alpha=alpha,
                         renorm=renorm, weight_mode=weight_mode)


def softmax_lib(z):
    return torch.softmax(torch.from_numpy(np.asarray(z, dtype=np.float64)), dim=-1).numpy()


def silu_lib(t):
    return torch.nn.functional.silu(torch.from_numpy(np.asarray(t, dtype=np.float64))).numpy()


def dense_ffn_lib(Wg, Wu, Wd, x):
    """Textbook SwiGLU FFN with library matmuls: Wd @ (silu(Wg x) * (Wu x))."""
    return Wd @ (silu_lib(Wg @ x) * (Wu @ x))


def rand_layer(rng, E, d, f, n_sh=0, f_sh=0, gate=False, std=0.3):
    W = dict(router=rng.normal(0, 1, (E, d)).astype(np.float32),
             w_gate=rng.normal(0, std, (E, f, d)).astype(np.float32),
             w_up=rng.normal(0, std, (E, f, d)).astype(np.float32),
             w_down=rng.normal(0, std, (E, d, f)).astype(np.float32))
    if n_sh:
        W.update(sh_gate=rng.normal(0, std, (n_sh, f_sh, d)).astype(np.float32),
                 sh_up=rng.normal(0, std, (n_sh, f_sh, d)).astype(np.float32),
                 sh_down=rng.normal(0, std, (n_sh, d, f_sh)).astype(np.float32))
        if gate:
            W["sh_scale"] = rng.normal(0, 0.5, (d,)).astype(np.float32)
    return W


def standard_moe_lib(W, H, k, renorm, n_sh=0):
    """Textbook MoE layer: softmax over all experts, top-k, weighted expert sum (+ shared)."""
    H = H.astype(np.float64)
    logits = H @ W["router"].astype(np.float64).T
    P = softmax_lib(logits)
    Y = np.zeros_like(H)
    sels = []
    for b in range(H.shape[0]):
        idx = np.argsort(-logits[b], kind="stable")[:k]
        p = P[b, idx]
        if renorm:
            p = p / p.sum()
        for e, pe in zip(idx, p):
            Y[b] += pe * dense_ffn_lib(W["w_gate"][e].astype(np.float64), W["w_up"][e].astype(np.float64),
                                       W["w_down"][e].astype(np.float64), H[b])
        for s in range(n_sh):
            sc = 1.0
            if "sh_scale" in W:
                sc = 1.0 / (1.0 + math.exp(-float(H[b] @ W["sh_scale"].astype(np.float64))))
            Y[b] += sc * dense_ffn_lib(W["sh_gate"][s].astype(np.float64), W["sh_up"][s].astype(np.float64),
                                       W["sh_down"][s].astype(np.float64), H[b])
        sels.append(idx)
    return Y, np.array(sels), logits


# ------------------------------------------------- gating: hand-worked example

def test_fig_toy_golden():
    t = read_fig_toy()
    E, k, cap = int(t["E"][0]), int(t["k"][0]), int(t["cap"][0])
    L = np.array([t["logits"][b] for b in range(4)])
    conf = np.array(t["conf"])
    cfg = gate_cfg(E, k, cap, t["alpha"][0], int(t["renorm"][0]), int(t["weight_mode"][0]))
    r = oracle.gating(cfg, L, conf)
    assert np.allclose(r.g, t["g"], rtol=0, atol=1e-12)
    assert sorted(np.nonzero(r.estar)[0].tolist()) == [int(x) for x in t["estar"]]
    assert np.allclose(r.lam, t["lambda"], rtol=0, atol=1e-12)
    for b in range(4):
        assert r.sel[b].tolist() == [int(x) for x in t["biased_sel"][b]]
        assert np.allclose(r.pw[b], t["weights"][b], rtol=0, atol=1e-12)
    assert r.n_unique == int(t["biased_unique"][0])
    # the same logits without the bias: six experts, and T1/T2 (high confidence) unchanged
    r0 = oracle.gating(gate_cfg(E, k, cap, 0.0), L, conf)
    for b in range(4):
        assert r0.sel[b].tolist() == [int(x) for x in t["standard_sel"][b]]
    assert r0.n_unique == int(t["standard_unique"][0])
    assert r.sel[0].tolist() == r0.sel[0].tolist() and r.sel[1].tolist() == r0.sel[1].tolist()
    # counts follow the selection
    assert r.counts.tolist() == [2, 3, 2, 0, 0, 1, 0, 0]


# ------------------------------------------------- gating: brute-force definitions

@pytest.mark.parametrize("seed", range(6))
def test_gating_brute_force_tiny(seed):
    """TopCap = the cap-subset with the largest sum of g; top-k = the k-subset with the
    largest sum of biased logits; lambda from sorted logits.  All by enumeration."""
    rng = np.random.default_rng(seed)
    E, k, cap, B = 6, 2, 3, 5
    alpha = [0.25, 0.5, 0.9][seed % 3]
    L = rng.normal(0, 1, (B, E))
    conf = rng.uniform(0.1, 1.0, B)
    r = oracle.gating(gate_cfg(E, k, cap, alpha), L, conf)
    g = np.array([sum(conf[b] * L[b, e] for b in range(B)) for e in range(E)])
    assert np.allclose(r.g, g, atol=1e-12)
    best = max(itertools.combinations(range(E), cap), key=lambda s: sum(g[list(s)]))
    assert set(np.nonzero(r.estar)[0].tolist()) == set(best)
    for b in range(B):
        srt = np.sort(L[b])[::-1]
        lam = alpha * (srt[0] - srt[k])
        assert abs(r.lam[b] - lam) < 1e-12
        l2 = L[b] + lam * np.isin(np.arange(E), best)
        assert np.allclose(r.l2[b], l2, atol=1e-12)
        bestk = max(itertools.combinations(range(E), k), key=lambda s: sum(l2[list(s)]))
        assert set(r.sel[b].tolist()) == set(bestk)
        # selection order: descending biased logit
        assert l2[r.sel[b][0]] >= l2[r.sel[b][1]]
        p = softmax_lib(L[b])[r.sel[b]]
        assert np.allclose(r.pw[b], p / p.sum(), atol=1e-12)
    assert r.n_unique == len(set(r.sel.flatten().tolist()))
    assert r.counts.sum() == B * k


def test_lambda_closed_form_and_margins():
    # logits 0..E-1 for every token: top-1 - (k+1)-th = k exactly
    E, k, cap, B = 10, 3, 5, 4
    L = np.tile(np.arange(E, dtype=np.float64), (B, 1))
    r = oracle.gating(gate_cfg(E, k, cap, 0.5), L, None)
    assert np.allclose(r.lam, 0.5 * k)
    assert set(np.nonzero(r.estar)[0].tolist()) == set(range(E - cap, E))
    assert r.n_unique == k
    assert abs(r.m_cap - B * 1.0) < 1e-12          # g_e = B*e with unit confidences
    assert np.allclose(r.m_tok, 1.0)               # all of top-(k+1) are biased alike


def test_topcap_tie_goes_to_lower_id():
    L = np.array([[1.0, 2.0, 2.0, 0.0, 2.0]])
    r = oracle.gating(gate_cfg(5, 1, 2, 0.5), L, None)
    assert np.nonzero(r.estar)[0].tolist() == [1, 2]
    # all-zero confidences: g == 0 everywhere, E* = lowest ids
    r = oracle.gating(gate_cfg(5, 1, 2, 0.5), L, np.zeros(1))
    assert np.nonzero(r.estar)[0].tolist() == [0, 1]


def test_alpha_one_tie_keeps_original_top1():
    # alpha = 1: the (k+1)-th expert, if in E*, ties with the top-1; the original wins
    L = np.array([[3.0, 2.0, 1.0, 0.0], [0.0, 0.0, 5.0, 5.0]])
    cfg = gate_cfg(4, 1, 2, 1.0)
    r = oracle.gating(cfg, L, np.array([0.0, 1.0]))  # E* = {2, 3} from token 1
    assert np.nonzero(r.estar)[0].tolist() == [2, 3]
    # token 0: lam = 3-2 = 1 -> l' = (3, 2, 2, 1): expert 0 stays
    assert r.sel[0].tolist() == [0]
    L2 = np.array([[3.0, 1.0, 2.0, 0.0], [0.0, 0.0, 5.0, 5.0]])
    r = oracle.gating(cfg, L2, np.array([0.0, 1.0]))
    # token 0: lam = 3-2 = 1 -> l' = (3, 1, 3, 1): tie on l', original logit decides
    assert r.sel[0].tolist() == [0]


def test_full_tie_goes_to_lower_id_in_selection_order():
    """Third key of the per-token order: equal biased AND equal original logits -> lower expert id
    first, inside the selected set and at its boundary (the selection is returned in that order)."""
    # bias off: three equal logits, k = 2 -> experts 0 and 1, in that order (2 loses the tie)
    r = oracle.gating(gate_cfg(4, 2, 4, 0.0), np.array([[1.0, 1.0, 1.0, 0.0]]), None)
    assert r.sel[0].tolist() == [0, 1]
    assert r.m_tok[0] == 0.0
    r = oracle.gating(gate_cfg(4, 3, 4, 0.0), np.array([[0.0, 2.0, 2.0, 2.0]]), None)
    assert r.sel[0].tolist() == [1, 2, 3]
    # biased: token 1 (all the confidence) makes E* = {1, 3}; token 0 has l = (5, 2, 4, 2, 0),
    # k = 2: lam = 0.5 * (5 - 2) = 1.5 (the third largest is 2), l' = (5, 3.5, 4, 3.5, 0).
    # Now make the two members of E* tie with expert 2 on l' only -> original logit decides:
    L = np.array([[5.0, 2.5, 4.0, 2.5, 0.0], [0.0, 9.0, 0.0, 9.0, 0.0]])
    cfg = gate_cfg(5, 3, 2, 0.5)
    r = oracle.gating(cfg, L, np.array([0.0, 1.0]))
    assert np.nonzero(r.estar)[0].tolist() == [1, 3]
    # token 0: top-1 5, (k+1)-th = 4th largest = 2.5 -> lam = 1.25, l' = (5, 3.75, 4, 3.75, 0):
    # order 0, 2, then experts 1 and 3 tie on l' (3.75) and on l (2.5): id 1 first, 3 is left out
    assert r.lam[0] == 1.25
    assert r.sel[0].tolist() == [0, 2, 1]
    assert r.m_tok[0] == 0.0
    # and with k = 4 both are taken, lower id first
    r = oracle.gating(gate_cfg(5, 4, 2, 0.5), L, np.array([0.0, 1.0]))
    # (k+1)-th = 5th largest = 0 -> lam = 2.5, l' = (5, 5, 4, 5, 0): l' ties of 0, 1, 3 -> l: 0 first, then 1, 3 by id
    assert r.sel[0].tolist() == [0, 1, 3, 2]


# ------------------------------------------------- gating: special cases and invariants

@pytest.mark.parametrize("renorm", [0, 1])
def test_bias_off_is_textbook_topk_softmax(renorm):
    rng = np.random.default_rng(10)
    B, E, k = 7, 12, 3
    L = rng.normal(0, 2, (B, E))
    for cfg in (gate_cfg(E, k, 0, 0.5, renorm), gate_cfg(E, k, 5, 0.0, renorm), gate_cfg(E, E, 5, 0.5, renorm)):
        r = oracle.gating(cfg, L, rng.uniform(0, 1, B))
        kk = cfg.top_k
        P = softmax_lib(L)
        for b in range(B):
            idx = np.argsort(-L[b], kind="stable")[:kk]
            assert r.sel[b].tolist() == idx.tolist()
            p = P[b, idx]
            if renorm:
                p = p / p.sum()
            assert np.allclose(r.pw[b], p, atol=1e-14)
        assert math.isinf(r.m_cap)


@pytest.mark.parametrize("mode,renorm", [(0, 0), (0, 1), (1, 1)])
def test_single_token_equals_standard_gating(mode, renorm):
    rng = np.random.default_rng(11)
    E, k, cap = 16, 4, 7
    for _ in range(20):
        L = rng.normal(0, 1.5, (1, E))
        a = oracle.gating(gate_cfg(E, k, cap, 0.5, renorm, mode), L, np.array([0.7]))
        s = oracle.gating(gate_cfg(E, k, cap, 0.0, renorm, 0), L, None)
        assert a.sel.tolist() == s.sel.tolist()
        assert np.allclose(a.pw, s.pw, atol=1e-14)


def test_permutation_shift_scale_invariance():
    rng = np.random.default_rng(12)
    B, E, k, cap = 9, 20, 3, 6
    L = rng.normal(0, 1, (B, E))
    conf = rng.uniform(0.2, 1, B)
    cfg = gate_cfg(E, k, cap, 0.5, 0)
    r = oracle.gating(cfg, L, conf)
    perm = rng.permutation(B)
    rp = oracle.gating(cfg, L[perm], conf[perm])
    assert rp.sel.tolist() == r.sel[perm].tolist()
    assert np.array_equal(rp.pw, r.pw[perm])
    assert rp.n_unique == r.n_unique and rp.estar.tolist() == r.estar.tolist()
    # adding a constant to a token's logits changes nothing
    rs = oracle.gating(cfg, L + rng.normal(0, 3, (B, 1)), conf)
    assert rs.sel.tolist() == r.sel.tolist() and np.allclose(rs.pw, r.pw, atol=1e-13)
    # scaling all confidences changes nothing
    rc = oracle.gating(cfg, L, conf * 3.5)
    assert rc.sel.tolist() == r.sel.tolist() and rc.estar.tolist() == r.estar.tolist()


def test_identical_tokens_reuse_ratio():
    rng = np.random.default_rng(13)
    B, E, k, cap = 8, 32, 4, 8
    L = np.tile(rng.normal(0, 1, (1, E)), (B, 1))
    r = oracle.gating(gate_cfg(E, k, cap, 0.5), L, rng.uniform(0.1, 1, B))
    assert all(r.sel[b].tolist() == r.sel[0].tolist() for b in range(B))
    assert np.allclose(r.pw, r.pw[0])
    assert r.n_unique == k                       # reuse ratio U/(B*k) = 1/B
    assert abs(r.n_unique / (B * k) - 1.0 / B) < 1e-15


@pytest.mark.parametrize("seed", range(5))
def test_bias_monotonicity(seed):
    """The bias only lets members of E* in and only pushes non-members out; order inside
    E* and inside its complement is unchanged; for alpha < 1 the top-1 expert stays."""
    rng = np.random.default_rng(100 + seed)
    B, E, k, cap = 12, 16, 3, 6
    L = rng.normal(0, 1, (B, E))
    conf = rng.uniform(0, 1, B)
    r = oracle.gating(gate_cfg(E, k, cap, 0.75), L, conf)
    r0 = oracle.gating(gate_cfg(E, k, cap, 0.0), L, conf)
    star = set(np.nonzero(r.estar)[0].tolist())
    assert len(star) == cap
    for b in range(B):
        s1, s0 = set(r.sel[b].tolist()), set(r0.sel[b].tolist())
        assert (s1 - s0) <= star
        assert not ((s0 - s1) & star)
        assert r0.sel[b][0] in s1
        ins = [e for e in r.sel[b] if e in star]
        outs = [e for e in r.sel[b] if e not in star]
        assert ins == sorted(ins, key=lambda e: -L[b, e])
        assert outs == sorted(outs, key=lambda e: -L[b, e])
    assert r.n_unique == len(set(r.sel.flatten().tolist()))


def test_weight_mode_one_uses_biased_logits():
    rng = np.random.default_rng(14)
    B, E, k, cap = 5, 10, 2, 4
    L = rng.normal(0, 1, (B, E))
    r = oracle.gating(gate_cfg(E, k, cap, 0.5, 0, 1), L, None)
    for b in range(B):
        assert np.allclose(r.pw[b], softmax_lib(r.l2[b])[r.sel[b]], atol=1e-14)
    # with renormalisation and every selected expert inside E*, modes 0 and 1 agree
    r1 = oracle.gating(gate_cfg(E, k, cap, 0.5, 1, 1), L, None)
    r0 = oracle.gating(gate_cfg(E, k, cap, 0.5, 1, 0), L, None)
    for b in range(B):
        if all(r.estar[e] for e in r1.sel[b]):
            assert np.allclose(r1.pw[b], r0.pw[b], atol=1e-13)


def test_forced_selection():
    rng = np.random.default_rng(15)
    L = rng.normal(0, 1, (3, 6))
    forced = np.array([[5, 0], [1, 2], [3, 4]], dtype=np.int32)
    r = oracle.gating(gate_cfg(6, 2, 3, 0.5, 0), L, None, forced_sel=forced)
    assert r.sel.tolist() == forced.tolist()
    P = softmax_lib(L)
    for b in range(3):
        assert np.allclose(r.pw[b], P[b, forced[b]], atol=1e-14)


# ------------------------------------------------- number formats

def test_router_logits_against_library_matmul():
    rng = np.random.default_rng(20)
    B, E, d = 5, 7, 96
    H = torch.from_numpy(rng.normal(0, 1, (B, d)).astype(np.float32)).to(torch.bfloat16)
    R = torch.from_numpy(rng.normal(0, 1, (E, d)).astype(np.float32)).to(torch.bfloat16)
    cfg = oracle.Config(d, 1, E, 1, act_dtype=BF16, router_dtype=BF16)
    got = oracle.router_logits(cfg, wl.raw_numpy(H), wl.raw_numpy(R))
    ref = H.double().numpy() @ R.double().numpy().T      # torch's own bf16 decoding
    assert np.allclose(got, ref, rtol=0, atol=1e-12)
    assert got.shape == (B, E)
    cfg = oracle.Config(d, 1, E, 1, act_dtype=F32, router_dtype=BF16)
    got = oracle.router_logits(cfg, H.float().numpy(), wl.raw_numpy(R))
    assert np.allclose(got, ref, rtol=0, atol=1e-12)


def test_q4b32_codec_bounds():
    """Round trip through the generator's quantiser and the oracle's decoder stays within
    half a scale step; the block's largest magnitude decodes to exactly +-7 scales."""
    g = torch.Generator().manual_seed(3)
    w = torch.randn((5, 96), generator=g) * 0.02
    w[2, 32:64] = 0.0                                    # an all-zero block
    packed, scale = wl.quantize_q4b32(w)
    assert packed.shape == (5, 48) and scale.shape == (5, 3) and packed.dtype == torch.uint8
    sc = scale.double().numpy()                          # torch's own fp16 decoding
    for row in range(5):
        dec = oracle.decode_row(Q4B32, packed.numpy(), wl.raw_numpy(scale), row, 96)
        for b in range(3):
            blk = w[row, 32 * b:32 * b + 32].double().numpy()
            got = dec[32 * b:32 * b + 32]
            s = sc[row, b]
            if s == 0:
                assert np.all(got == 0)
                continue
            q = got / s
            assert np.allclose(q, np.round(q), atol=1e-9) and np.all(np.abs(q) <= 7 + 1e-9)
            inside = np.abs(blk / s) <= 7.0
            assert np.all(np.abs(got - blk)[inside] <= 0.5 * s * (1 + 1e-6))
            i = int(np.argmax(np.abs(blk)))
            assert got[i] == math.copysign(7.0, blk[i]) * s
    # nibble order: weight i sits in nibble i
    w2 = torch.zeros((1, 32)); w2[0, 0] = 7.0; w2[0, 1] = -7.0; w2[0, 31] = 3.0
    p2, s2 = wl.quantize_q4b32(w2)
    assert p2[0, 0].item() == (15 | (1 << 4)) and p2[0, 15].item() == (8 | (11 << 4))
    dec = oracle.decode_row(Q4B32, p2.numpy(), wl.raw_numpy(s2), 0, 32)
    assert dec[0] == 7.0 and dec[1] == -7.0 and dec[31] == 3.0 and dec[2] == 0.0


def test_q4b32_scale_decoding_subnormal():
    """Binary16 scales below the normal range are m * 2^-24: checked against the bit patterns'
    textbook values and against numpy's own binary16 decoding.  (Infinite and NaN scales cannot
    be read back through a dot product with unit vectors, and the quantiser never writes them:
    that branch of the decoder stays unpinned.)"""
    packed = np.full((1, 16 * 4), 0x99, dtype=np.uint8)         # every nibble 9 -> q = +1
    bits = np.array([[0x0001, 0x03ff, 0x8001, 0x0400]], dtype=np.uint16)
    dec = oracle.decode_row(Q4B32, packed, bits, 0, 32 * 4)
    assert dec[0] == 2.0 ** -24 and dec[31] == 2.0 ** -24       # smallest subnormal
    assert dec[32] == 1023 * 2.0 ** -24                         # largest subnormal
    assert dec[64] == -(2.0 ** -24)                             # sign of a subnormal
    assert dec[96] == 2.0 ** -14                                # smallest normal
    ref = bits.view(np.float16).astype(np.float64)[0]
    for b in range(4):
        assert dec[32 * b] == ref[b]
    # q = nibble - 8: nibble 1 -> -7 times a subnormal scale stays exact
    packed[0, 0] = 0x11
    assert oracle.decode_row(Q4B32, packed, bits, 0, 32 * 4)[0] == -7 * 2.0 ** -24


def test_bf16_f32_decode_rows():
    x = torch.tensor([[1.0, -2.5, 3.0e-5, 1024.0, -0.33]])
    xb = x.to(torch.bfloat16)
    assert np.array_equal(oracle.decode_row(BF16, wl.raw_numpy(xb), None, 0, 5), xb.double().numpy()[0])
    assert np.array_equal(oracle.decode_row(F32, x.numpy(), None, 0, 5), x.double().numpy()[0])


# ------------------------------------------------- expert FFN and the whole layer

def test_ffn_scalar_closed_form():
    # d = f = 1, one expert, k = 1: y = wd * silu(wg x) * (wu x)
    for wg, wu, wd, x in [(0.5, -1.5, 2.0, 3.0), (-2.0, 0.25, -1.0, 0.75)]:
        W = oracle.Weights(router=np.array([[1.0]], np.float32), w_gate=np.array([[[wg]]], np.float32),
                           w_up=np.array([[[wu]]], np.float32), w_down=np.array([[[wd]]], np.float32))
        cfg = oracle.Config(1, 1, 1, 1)
        r = oracle.layer(cfg, W, np.array([[x]], np.float32))
        t = wg * x
        assert abs(r.y[0, 0] - wd * (t / (1 + math.exp(-t))) * (wu * x)) < 1e-14
        assert r.pw[0, 0] == 1.0 and r.n_unique == 1


@pytest.mark.parametrize("renorm", [0, 1])
def test_layer_bias_off_equals_textbook_moe(renorm):
    rng = np.random.default_rng(30)
    E, d, f, k, B = 6, 24, 40, 2, 5           # d != f: a transposed operand cannot pass
    W = rand_layer(rng, E, d, f)
    H = rng.normal(0, 1, (B, d)).astype(np.float32)
    Y, sels, logits = standard_moe_lib(W, H, k, renorm)
    cfg = oracle.Config(d, f, E, k, renorm=renorm, cap=0)
    r = oracle.layer(cfg, oracle.Weights(**W), H)
    assert r.sel.tolist() == sels.tolist()
    assert np.allclose(r.logits, logits, atol=1e-12)
    assert np.allclose(r.y, Y, rtol=1e-12, atol=1e-12)


def test_layer_topk_equals_E_is_dense_weighted_sum():
    rng = np.random.default_rng(31)
    E, d, f, B = 4, 16, 24, 3
    W = rand_layer(rng, E, d, f)
    H = rng.normal(0, 1, (B, d)).astype(np.float32)
    cfg = oracle.Config(d, f, E, E, renorm=0, cap=2, alpha=0.5)
    r = oracle.layer(cfg, oracle.Weights(**W), H)
    P = softmax_lib(H.astype(np.float64) @ W["router"].astype(np.float64).T)
    for b in range(B):
        y = sum(P[b, e] * dense_ffn_lib(W["w_gate"][e].astype(np.float64), W["w_up"][e].astype(np.float64),
                                        W["w_down"][e].astype(np.float64), H[b].astype(np.float64))
                for e in range(E))
        assert np.allclose(r.y[b], y, rtol=1e-12, atol=1e-13)
    assert r.n_unique == E


@pytest.mark.parametrize("gate", [False, True])
def test_layer_shared_experts(gate):
    rng = np.random.default_rng(32)
    E, d, f, k, B, n_sh, f_sh = 5, 16, 24, 2, 4, 2, 40
    W = rand_layer(rng, E, d, f, n_sh, f_sh, gate)
    H = rng.normal(0, 1, (B, d)).astype(np.float32)
    Y, sels, _ = standard_moe_lib(W, H, k, 0, n_sh)
    cfg = oracle.Config(d, f, E, k, n_shared=n_sh, d_ff_shared=f_sh, renorm=0, cap=0)
    r = oracle.layer(cfg, oracle.Weights(**W), H)
    assert np.allclose(r.y, Y, rtol=1e-12, atol=1e-12)


def test_layer_single_token_equals_standard_decoding():
    rng = np.random.default_rng(33)
    E, d, f, k = 8, 16, 24, 2
    W = rand_layer(rng, E, d, f)
    H = rng.normal(0, 1, (1, d)).astype(np.float32)
    Y, sels, _ = standard_moe_lib(W, H, k, 0)
    r = oracle.layer(oracle.Config(d, f, E, k, renorm=0, cap=4, alpha=0.5), oracle.Weights(**W), H,
                     conf=np.array([0.3]))
    assert r.sel.tolist() == sels.tolist()
    assert np.allclose(r.y, Y, rtol=1e-12, atol=1e-13)


def test_layer_token_permutation_and_subset():
    rng = np.random.default_rng(34)
    E, d, f, k, B = 8, 16, 24, 2, 6
    W = rand_layer(rng, E, d, f)
    H = rng.normal(0, 1, (B, d)).astype(np.float32)
    conf = rng.uniform(0.2, 1, B)
    cfg = oracle.Config(d, f, E, k, renorm=1, cap=4, alpha=0.5)
    r = oracle.layer(cfg, oracle.Weights(**W), H, conf)
    perm = rng.permutation(B)
    rp = oracle.layer(cfg, oracle.Weights(**W), H[perm], conf[perm])
    assert rp.sel.tolist() == r.sel[perm].tolist()
    assert np.array_equal(rp.y, r.y[perm])
    assert rp.n_unique == r.n_unique
    # evaluating only some tokens gives the same rows
    sub = oracle.layer(cfg, oracle.Weights(**W), H, conf, tok_list=[4, 1])
    assert np.array_equal(sub.y, r.y[[4, 1]])
    # the layer's output is the gating's selection applied expert by expert
    gt = oracle.gating(cfg, r.logits, conf)
    assert gt.sel.tolist() == r.sel.tolist() and gt.n_unique == r.n_unique


def test_layer_storage_formats_agree_with_f32_of_same_values():
    """bf16 and block-int4 layers equal the fp32 layer holding the same stored values
    (values read back through the decoder pinned above; the dot loops differ)."""
    w0 = wl.Workload("t", 64, 96, 6, 2, 1, 5, "chain", 0.5, 7, n_shared=1, d_ff_shared=32,
                     shared_gate=True, renorm=1, cap=3)
    for wdt in (BF16, Q4B32):
        w = w0.with_(weight_dtype=wdt)
        T = wl.layer_weights(w, 0)
        H = wl.hidden_states(w, 0)
        conf = wl.confidences(w, 0).double().numpy()
        raw = {n: wl.raw_numpy(t) for n, t in T.items()}
        cfg = oracle.Config(64, 96, 6, 2, 1, 32, BF16, BF16, wdt, 1, 3, 0, 0.5)
        r = oracle.layer(cfg, oracle.Weights(**raw), wl.raw_numpy(H), conf)
        f32 = {}
        for name, K in (("w_gate", 64), ("w_up", 64), ("w_down", 96), ("sh_gate", 64), ("sh_up", 64),
                        ("sh_down", 32)):
            t = T[name]
            rows = t.shape[0] * t.shape[1]
            sname = ("s_" + name[2:]) if name.startswith("w_") else ("sh_s_" + name[3:])
            flat = raw[name].reshape(rows, -1)
            sc = raw[sname].reshape(rows, -1) if wdt == Q4B32 else None
            dec = np.stack([oracle.decode_row(wdt, flat, sc, i, K) for i in range(rows)])
            f32[name] = dec.reshape(t.shape[0], t.shape[1], K).astype(np.float32)
        f32["router"] = T["router"].float().numpy()
        f32["sh_scale"] = T["sh_scale"].float().numpy()
        cfg32 = oracle.Config(64, 96, 6, 2, 1, 32, F32, F32, F32, 1, 3, 0, 0.5)
        r32 = oracle.layer(cfg32, oracle.Weights(**f32), H.float().numpy(), conf)
        assert r.sel.tolist() == r32.sel.tolist()
        assert np.allclose(r.y, r32.y, rtol=1e-12, atol=1e-14)
        # and the fp32 layer is the textbook one when the bias is off
        cfg32.cap = 0
        r32 = oracle.layer(cfg32, oracle.Weights(**f32), H.float().numpy(), conf)
        Y, sels, _ = standard_moe_lib(f32, H.float().numpy(), 2, 1, 1)
        assert np.allclose(r32.y, Y, rtol=1e-11, atol=1e-13)


def test_layer_forced_selection_changes_only_what_it_should():
    rng = np.random.default_rng(35)
    E, d, f, k, B = 6, 8, 12, 2, 3
    W = rand_layer(rng, E, d, f)
    H = rng.normal(0, 1, (B, d)).astype(np.float32)
    cfg = oracle.Config(d, f, E, k, renorm=0, cap=3, alpha=0.5)
    r = oracle.layer(cfg, oracle.Weights(**W), H)
    rf = oracle.layer(cfg, oracle.Weights(**W), H, forced_sel=r.sel[:, ::-1].copy())
    assert np.allclose(rf.y, r.y, rtol=1e-13, atol=1e-15)      # same set, other order
    assert np.allclose(rf.pw, r.pw[:, ::-1])
