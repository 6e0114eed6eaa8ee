"""GPU parity of the adaptive-expansion calls (Sec. 4.1) against the oracle: bit-exact sets,
admission flags and admission order on seeded synthetic draft trees."""
import random

import numpy as np
import pytest
import torch

from oracle import expansion as ox

pytestmark = pytest.mark.gpu


def _masks_tensor(masks, words, dev):
    n, L = len(masks), len(masks[0])
    a = np.zeros((n, L, words), dtype=np.uint64)
    for i in range(n):
        for l in range(L):
            for w in range(words):
                a[i, l, w] = (masks[i][l] >> (64 * w)) & 0xFFFFFFFFFFFFFFFF
    return torch.from_numpy(a.view(np.int64)).to(dev)


def _tree(rng, n, n_layers, n_experts, k, reuse):
    """Draft tree in heap-like order; a child's predicted experts are its parent's with a few
    replaced (neighbouring draft tokens share experts), as in the paper's workloads."""
    parent = [-1 if i == 0 or rng.random() < 0.1 else rng.randrange(i) for i in range(n)]
    p_tok = [float(np.float32(rng.uniform(0.3, 1.0))) for _ in range(n)]
    sets = []
    for i in range(n):
        cand = []
        for l in range(n_layers):
            if parent[i] >= 0 and rng.random() < reuse:
                base = set(sets[parent[i]][l])
                for _ in range(rng.randint(0, 2)):
                    base.discard(rng.choice(sorted(base)))
                while len(base) < k:
                    base.add(rng.randrange(n_experts))
            else:
                base = set(rng.sample(range(n_experts), k))
            cand.append(sorted(base))
        sets.append(cand)
    return parent, p_tok, sets


@pytest.mark.parametrize("n,n_layers,n_experts,k", [(1, 1, 8, 2), (16, 4, 64, 8), (64, 16, 64, 6), (48, 3, 128, 8),
                                                  (256, 2, 256, 4), (33, 26, 64, 6)])
def test_expand_matches_oracle(n, n_layers, n_experts, k):
    from paper_2608_15018_b200 import binding

    dev = torch.device("cuda", 0)
    rng = random.Random(1000 * n + n_layers)
    words = (n_experts + 63) // 64
    for trial in range(4):
        parent, p_tok, sets = _tree(rng, n, n_layers, n_experts, k, reuse=0.7)
        masks = [[sum(1 << e for e in layer) for layer in cand] for cand in sets]
        c_draft = [float(np.float32(rng.uniform(0.0, 0.05))) for _ in range(n)]
        t_ar = float(np.float32(1.0))
        t_exp = float(np.float32(rng.choice([0.01, 0.03, 0.1]) / n_layers))
        want_adm, want_order, want_union = ox.adaptive_expand(parent, p_tok, masks, c_draft, t_ar, t_exp)

        # the sets go through the library's own mask builder, layer by layer
        out = torch.zeros((n, n_layers, words), dtype=torch.int64, device=dev)
        for l in range(n_layers):
            sel = torch.tensor([sets[i][l] for i in range(n)], dtype=torch.int32, device=dev)
            binding.expert_masks(sel, n_experts, out=out, layer=l)
        torch.cuda.synchronize()
        assert torch.equal(out.cpu(), _masks_tensor(masks, words, "cpu"))

        adm, order, n_adm, union = binding.adaptive_expand(
            torch.tensor(parent, dtype=torch.int32, device=dev), torch.tensor(p_tok, dtype=torch.float32, device=dev),
            out, n_experts, torch.tensor(c_draft, dtype=torch.float32, device=dev), t_ar, t_exp)
        torch.cuda.synchronize()
        assert adm.cpu().tolist() == want_adm
        assert n_adm.item() == len(want_order)
        assert order.cpu().tolist() == want_order + [-1] * (n - len(want_order))
        got_union = union.cpu().numpy().view(np.uint64)
        for l in range(n_layers):
            assert sum(int(got_union[l, w]) << (64 * w) for w in range(words)) == want_union[l]


def test_expand_ties_and_degenerate_cases():
    from paper_2608_15018_b200 import binding

    dev = torch.device("cuda", 0)
    # identical siblings: equal utilities, the lowest index goes first; zero cost: utility +inf
    parent = [-1, -1, -1, 0]
    p_tok = [0.5, 0.5, 0.5, 1.0]
    masks = [[0b11], [0b11], [0b11], [0b11]]
    for c, t_exp in (([0.25] * 4, 0.125), ([0.0] * 4, 0.0)):
        want = ox.adaptive_expand(parent, p_tok, masks, c, 1.0, t_exp)
        adm, order, n_adm, _ = binding.adaptive_expand(
            torch.tensor(parent, dtype=torch.int32, device=dev), torch.tensor(p_tok, dtype=torch.float32, device=dev),
            _masks_tensor(masks, 1, dev), 8, torch.tensor(c, dtype=torch.float32, device=dev), 1.0, t_exp)
        assert adm.cpu().tolist() == want[0]
        assert order.cpu().tolist()[: n_adm.item()] == want[1]
    # nothing reaches utility 1
    adm, order, n_adm, union = binding.adaptive_expand(
        torch.tensor([-1, 0], dtype=torch.int32, device=dev), torch.tensor([0.5, 0.5], dtype=torch.float32, device=dev),
        _masks_tensor([[1], [2]], 1, dev), 8, None, 0.0, 0.25)
    assert n_adm.item() == 0 and adm.cpu().tolist() == [0, 0] and order.cpu().tolist() == [-1, -1]
    assert union.cpu().tolist() == [[0]]


def test_expand_reports_a_malformed_parent_array():
    """A parent index that is not below the candidate's own is not followed: that candidate and its
    descendants are never admitted, the call reports n_admitted = -1, and the well-formed rest is
    decided as if the malformed candidates were not there."""
    from paper_2608_15018_b200 import binding

    dev = torch.device("cuda", 0)
    #          0   1   2     3 (self)  4 (forward)  5 (child of 3)  6 (beyond n)
    parent = [-1,  0,  0,    3,        5,           3,              40]
    p_tok = [0.9] * 7
    masks = [[1 << i] for i in range(7)]
    adm, order, n_adm, union = binding.adaptive_expand(
        torch.tensor(parent, dtype=torch.int32, device=dev), torch.tensor(p_tok, dtype=torch.float32, device=dev),
        _masks_tensor(masks, 1, dev), 8, None, 1.0, 0.125)
    torch.cuda.synchronize()
    want_adm, want_order, want_union = ox.adaptive_expand(parent[:3], p_tok[:3], masks[:3], [0.0] * 3, 1.0, 0.125)
    assert n_adm.item() == -1
    assert adm.cpu().tolist() == want_adm + [0, 0, 0, 0]
    assert order.cpu().tolist()[: len(want_order)] == want_order
    assert int(union.cpu().numpy().view(np.uint64)[0, 0]) == want_union[0]


def test_expand_argument_errors():
    from paper_2608_15018_b200 import binding

    dev = torch.device("cuda", 0)
    big = torch.zeros((257, 1, 1), dtype=torch.int64, device=dev)
    with pytest.raises(binding.S2MoEError):
        binding.adaptive_expand(torch.zeros(257, dtype=torch.int32, device=dev),
                                torch.ones(257, dtype=torch.float32, device=dev), big, 8, None, 1.0, 0.1)
    with pytest.raises(binding.S2MoEError):
        binding.expert_masks(torch.zeros((2, 2), dtype=torch.int32, device=dev), 1000)


def test_draft_pass_then_expansion_then_verification():
    """Expert-sparse draft pass (k_draft experts, no bias) -> predicted expert sets -> adaptive
    expansion -> the verification layer on the admitted tokens only (Sec. 4.1 and Sec. 5.1
    "Draft Experts"), every stage against the oracle."""
    import oracle
    from gpu_util import run_case
    from oracle import parity
    from paper_2608_15018_b200 import binding, workloads

    dev = torch.device("cuda", 0)
    wl = workloads.CONFIGS["cfg5"].with_(d_model=512, d_ff=352, d_ff_shared=352, n_layers=3)
    B, k_draft = 16, 3
    draft = wl.with_(top_k=k_draft, alpha=0.0)
    words = (wl.n_experts + 63) // 64
    masks = torch.zeros((B, wl.n_layers, words), dtype=torch.int64, device=dev)
    want_masks = []
    H = [workloads.hidden_states(wl, l, B, device=dev) for l in range(wl.n_layers)]
    T = [workloads.layer_weights(wl, l, dev) for l in range(wl.n_layers)]
    with binding.S2MoE(binding.Config.from_workload(draft, n_layers=wl.n_layers), T) as m:
        for l in range(wl.n_layers):
            o = m.verify_layer(l, H[l], None)
            binding.expert_masks(o.sel_idx, wl.n_experts, out=masks, layer=l)
            torch.cuda.synchronize()
            ocfg, ow = parity.from_workload(draft, T[l])
            logits = oracle.router_logits(ocfg, workloads.raw_numpy(H[l]), ow.router)
            g = oracle.gating(ocfg, logits, None)
            # the draft selection is plain top-k: sets must agree unless the k-th margin is a tie
            assert (np.sort(o.sel_idx.cpu().numpy(), axis=1) == np.sort(g.sel, axis=1)).all() or g.m_tok.min() < 1e-6
            want_masks.append(ox.expert_masks(o.sel_idx.cpu().tolist()))
    want_masks = [[want_masks[l][b] for l in range(wl.n_layers)] for b in range(B)]
    parent = [workloads.tree_parent(i) if i else -1 for i in range(B)]
    gen = torch.Generator().manual_seed(7)
    p_tok = (0.4 + 0.6 * torch.rand(B, generator=gen)).to(torch.float32)
    t_ar, t_exp = 1.0, float(np.float32(0.05))
    c_draft = torch.full((B,), float(np.float32(0.1)), dtype=torch.float32)
    want_adm, want_order, _ = ox.adaptive_expand(parent, p_tok.tolist(), want_masks, c_draft.tolist(), t_ar, t_exp)
    adm, order, n_adm, _ = binding.adaptive_expand(torch.tensor(parent, dtype=torch.int32, device=dev), p_tok.to(dev),
                                                   masks, wl.n_experts, c_draft.to(dev), t_ar, t_exp)
    torch.cuda.synchronize()
    assert adm.cpu().tolist() == want_adm and order.cpu().tolist()[: n_adm.item()] == want_order
    assert 0 < n_adm.item() < B, "the case should prune something and keep something"
    # verification of the admitted tokens only, with their prefix confidences as gating weights
    keep = [i for i in range(B) if want_adm[i]]
    conf = torch.tensor([ox.prefix_confidence(parent, p_tok.tolist())[i] for i in keep], dtype=torch.float32)
    for l in range(wl.n_layers):
        rep, out = run_case(wl, layer=l, hidden=H[l][keep], conf=conf.to(dev))
        assert rep.tokens_checked == len(keep)
