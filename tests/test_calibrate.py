"""The cost-model fit of Sec. 4.1 ("Routing-aware Cost Estimation": verification latency linear in
the number of activated experts): the least-squares helper on CPU, and a small sweep on the GPU."""
import numpy as np
import pytest

from paper_2608_15018_b200 import calibrate


def test_fit_line_on_an_exact_line():
    u = np.array([4.0, 9.0, 16.0, 31.0, 64.0])
    t0, t_exp, r2, mape = calibrate.fit_line(u, 31.5 + 1.75 * u)
    assert abs(t0 - 31.5) < 1e-9 and abs(t_exp - 1.75) < 1e-10
    assert abs(r2 - 1.0) < 1e-12 and mape < 1e-12


def test_fit_line_on_three_noisy_points_by_hand():
    # u = 0, 1, 2; t = 1, 4, 5: slope = cov / var = 4 / 2 = 2, intercept = mean(t) - 2 * mean(u) = 10/3 - 2 = 4/3
    u, t = np.array([0.0, 1.0, 2.0]), np.array([1.0, 4.0, 5.0])
    t0, t_exp, r2, mape = calibrate.fit_line(u, t)
    assert abs(t_exp - 2.0) < 1e-12 and abs(t0 - 4.0 / 3.0) < 1e-12
    # residuals -1/3, 2/3, -1/3: SS_res = 2/3, SS_tot = 26/3 -> R^2 = 1 - 1/13
    assert abs(r2 - (1.0 - 1.0 / 13.0)) < 1e-12
    assert abs(mape - (1.0 / 3.0 / 1.0 + 2.0 / 3.0 / 4.0 + 1.0 / 3.0 / 5.0) / 3.0) < 1e-12


def test_fit_line_with_constant_latency():
    t0, t_exp, r2, mape = calibrate.fit_line(np.array([1.0, 2.0, 3.0]), np.array([7.0, 7.0, 7.0]))
    assert abs(t0 - 7.0) < 1e-12 and abs(t_exp) < 1e-12 and r2 == 1.0 and mape < 1e-12


@pytest.mark.gpu
def test_mini_sweep_counts_match_the_oracle_and_the_slope_is_positive():
    """Two layers, two batch sizes, two noise levels of the DeepSeek-like shape at reduced width:
    the U of every timed layer equals the oracle's count, every latency is positive and the
    fitted cost of one more expert is positive."""
    import torch

    import oracle
    from oracle import parity
    from paper_2608_15018_b200 import workloads

    wl = workloads.CONFIGS["cfg5"].with_(d_model=1024, d_ff=704, d_ff_shared=704, n_layers=2)
    rows = calibrate.measure(wl, 2, [4, 32], [0.1, 1.0], repeats=3)
    assert len(rows) == 8
    for B, sigma, layer, U, us in rows:
        T = workloads.layer_weights(wl, layer, "cuda")
        H = workloads.hidden_states(wl, layer, B, sigma, "cuda")
        C = workloads.confidences(wl, layer, B, "cuda")
        ocfg, ow = parity.from_workload(wl, T)
        logits = oracle.router_logits(ocfg, workloads.raw_numpy(H), ow.router)
        ref = oracle.gating(ocfg, logits, C.double().cpu().numpy())
        assert U == ref.n_unique or min(ref.m_tok.min(), ref.m_cap) < 1e-6
        assert us > 0
    arr = np.array([(r[3], r[4]) for r in rows], dtype=np.float64)
    assert arr[:, 0].max() > arr[:, 0].min()
    t0, t_exp, r2, mape = calibrate.fit_line(arr[:, 0], arr[:, 1])
    assert t_exp > 0 and t0 > 0
    torch.cuda.empty_cache()
