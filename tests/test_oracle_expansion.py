"""Pins of the adaptive-expansion oracle (Sec. 4.1, Eq. 2 and Eq. 3) against things other than
itself: a hand-worked tree, set arithmetic on Python sets, closed forms and invariants."""
import math
import random

import pytest

from oracle import expansion as ox


def _sets_to_masks(sets):
    return [[sum(1 << e for e in layer) for layer in cand] for cand in sets]


def test_prefix_confidence_is_the_product_along_the_path():
    parent = [-1, 0, 1, 1, -1, 4]
    p_tok = [0.5, 0.5, 0.25, 0.75, 0.125, 0.5]
    p = ox.prefix_confidence(parent, p_tok)
    # written out by hand, every value a dyadic rational (exact in binary floating point)
    assert p == [0.5, 0.25, 0.0625, 0.1875, 0.125, 0.0625]


def test_prefix_confidence_rejects_children_before_parents():
    with pytest.raises(ValueError):
        ox.prefix_confidence([1, -1], [0.5, 0.5])


def test_new_experts_is_set_difference_per_layer():
    rng = random.Random(3)
    for _ in range(200):
        n_layers = rng.randint(1, 4)
        cand = [set(rng.sample(range(70), rng.randint(0, 8))) for _ in range(n_layers)]
        seen = [set(rng.sample(range(70), rng.randint(0, 30))) for _ in range(n_layers)]
        want = sum(len(c - s) for c, s in zip(cand, seen))
        got = ox.new_experts([sum(1 << e for e in c) for c in cand], [sum(1 << e for e in s) for s in seen])
        assert got == want


def test_expert_masks_from_indices():
    assert ox.expert_masks([[0, 3], [65, 1]]) == [0b1001, (1 << 65) | 0b10]


def test_utility_formula_and_zero_cost():
    assert ox.utility(0.5, 2, 0.25, 2.0, 0.125) == 1.0 / 0.5          # 0.5*2 / (2*0.125 + 0.25)
    assert ox.utility(0.5, 0, 0.0, 1.0, 0.25) == math.inf
    assert ox.utility(0.0, 3, 0.5, 1.0, 0.25) == 0.0


def test_hand_worked_tree():
    # five candidates, one layer; all numbers dyadic so that every utility below is exact
    parent = [-1, 0, 0, 1, -1]
    p_tok = [0.875, 0.75, 0.5, 0.875, 0.25]
    sets = [[{0, 1}], [{1, 2}], [{0, 1}], [{5, 6}], [{0}]]
    adm, order, union = ox.adaptive_expand(parent, p_tok, _sets_to_masks(sets), [0.125] * 5, t_ar=1.0, t_exp=0.25)
    # step 1: U0 = 0.875 / (2*0.25 + 0.125) = 1.4 ; U4 = 0.25 / (0.25 + 0.125) = 0.667     -> admit 0
    # step 2: U1 = 0.65625 / 0.375 = 1.75 ; U2 = 0.4375 / 0.125 = 3.5 ; U4 = 0.25 / 0.125 = 2 -> admit 2
    # step 3: U1 = 1.75 ; U4 = 2                                                             -> admit 4
    # step 4: U1 = 1.75                                                                      -> admit 1
    # step 5: U3 = 0.57421875 / (2*0.25 + 0.125) = 0.91875 < 1                               -> stop
    assert order == [0, 2, 4, 1]
    assert adm == [1, 1, 1, 0, 1]
    assert union == [0b111]
    # candidate 4 was below 1 on its own and became worth verifying once expert 0 was paid for:
    # the effect that confidence-only pruning cannot see
    alone = ox.utility(0.25, 1, 0.125, 1.0, 0.25)
    assert alone < 1.0


def test_without_expert_cost_it_is_confidence_pruning():
    # empty predicted sets: the cost is C_draft alone, so (prefix confidences never grow along a
    # path) the admitted set is exactly { i : p_i * T_AR >= C_draft }
    rng = random.Random(11)
    for _ in range(50):
        n = rng.randint(1, 24)
        parent = [-1 if i == 0 or rng.random() < 0.2 else rng.randrange(i) for i in range(n)]
        p_tok = [rng.choice([0.25, 0.5, 0.75, 0.875, 1.0]) for _ in range(n)]
        adm, order, _ = ox.adaptive_expand(parent, p_tok, [[0]] * n, [0.125] * n, t_ar=1.0, t_exp=0.25)
        p = ox.prefix_confidence(parent, p_tok)
        assert adm == [1 if pi >= 0.125 else 0 for pi in p]
        # largest utility first means non-increasing prefix confidence here
        assert [p[i] for i in order] == sorted((p[i] for i in order), reverse=True)


def test_free_verification_admits_everything_with_zero_draft_cost():
    parent = [-1, 0, 1, 2]
    adm, order, _ = ox.adaptive_expand(parent, [0.5] * 4, [[1], [2], [4], [8]], [0.0] * 4, t_ar=1.0, t_exp=0.0)
    assert adm == [1, 1, 1, 1] and order == [0, 1, 2, 3]


def test_no_benefit_admits_nothing():
    adm, order, union = ox.adaptive_expand([-1, 0], [0.5, 0.5], [[1], [2]], [0.125, 0.125], t_ar=0.0, t_exp=0.25)
    assert adm == [0, 0] and order == [] and union == [0]


def test_invariants_on_random_trees():
    rng = random.Random(5)
    for _ in range(100):
        n = rng.randint(1, 30)
        n_layers = rng.randint(1, 3)
        parent = [-1 if i == 0 or rng.random() < 0.15 else rng.randrange(i) for i in range(n)]
        p_tok = [rng.uniform(0.2, 1.0) for _ in range(n)]
        masks = [[sum(1 << e for e in rng.sample(range(64), 4)) for _ in range(n_layers)] for _ in range(n)]
        c_draft = [rng.uniform(0.0, 0.2) for _ in range(n)]
        t_ar, t_exp = 1.0, rng.uniform(0.01, 0.2)
        adm, order, union = ox.adaptive_expand(parent, p_tok, masks, c_draft, t_ar, t_exp)
        p = ox.prefix_confidence(parent, p_tok)
        # ancestor-closed, each admitted exactly once, in an order that respects ancestry
        pos = {i: k for k, i in enumerate(order)}
        assert sorted(order) == [i for i in range(n) if adm[i]]
        for i in order:
            assert parent[i] < 0 or (adm[parent[i]] and pos[parent[i]] < pos[i])
        # replay: every admission had utility >= 1 against the set admitted before it and was the
        # best eligible candidate; at the end nobody eligible reaches 1
        seen = [0] * n_layers
        done = set()
        for i in order:
            elig = [j for j in range(n) if j not in done and (parent[j] < 0 or parent[j] in done)]
            us = {j: ox.utility(p[j], ox.new_experts(masks[j], seen), c_draft[j], t_ar, t_exp) for j in elig}
            assert us[i] >= 1.0 and us[i] == max(us.values())
            seen = [s | m for s, m in zip(seen, masks[i])]
            done.add(i)
        assert seen == union
        elig = [j for j in range(n) if j not in done and (parent[j] < 0 or parent[j] in done)]
        assert all(ox.utility(p[j], ox.new_experts(masks[j], seen), c_draft[j], t_ar, t_exp) < 1.0 for j in elig)
