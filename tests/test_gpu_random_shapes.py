"""Seeded random shapes through the tcgen05 kernels (two launches per layer, and the fused one) (bf16 and block-int4 weights) against the
oracle: expert counts from 1 to 256, ragged widths, shared experts with and without the sigmoid
gate, every batch size class, all gating variants."""
import random

import pytest

from gpu_util import run_case
from paper_2608_15018_b200.workloads import BF16, CONFIGS, Q4B32

pytestmark = pytest.mark.gpu


def _case(rng, trial):
    q4 = rng.random() < 0.4
    E = rng.choice([1, 2, 3, 8, 17, 60, 64, 100, 128, 256])
    k = rng.randint(1, min(E, 16))
    n_sh = rng.choice([0, 0, 1, 2])
    wl = CONFIGS["cfg3"].with_(
        d_model=rng.choice([256, 512, 768]) if q4 else rng.choice([64, 192, 512, 1024]),
        d_ff=rng.choice([256, 512]) if q4 else rng.choice([32, 96, 352, 512]),
        n_experts=E, top_k=k, cap=rng.randint(k, E), n_shared=n_sh,
        d_ff_shared=((rng.choice([256, 768]) if q4 else rng.choice([64, 352, 736])) if n_sh else 0),
        shared_gate=bool(n_sh and rng.random() < 0.5), weight_dtype=Q4B32 if q4 else BF16,
        renorm=rng.randint(0, 1), weight_mode=rng.randint(0, 1), alpha=rng.choice([0.0, 0.5, 1.0]),
        structure=rng.choice(["chain", "tree"]), sigma=rng.choice([0.0, 0.1, 1.0]), seed=trial)
    return wl, rng.choice([1, 2, 3, 7, 8, 9, 16, 31, 33, 64]), rng.random() < 0.7


@pytest.mark.parametrize("plan", [3, 4])
@pytest.mark.parametrize("seed", [11, 12])
def test_random_shapes_on_the_tensor_core_plan(seed, plan):
    rng = random.Random(seed)
    ran = 0
    for trial in range(25):
        wl, B, use_conf = _case(rng, trial)
        rep, _ = run_case(wl, n_tokens=B, plan=plan, use_conf=use_conf, optional=True)
        if rep is not None:
            assert rep.plan == plan and rep.tokens_checked == B
            ran += 1
    assert ran >= 20
