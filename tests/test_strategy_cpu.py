"""Per-block strategy on the CPU: Algorithm 1 (C host function and oracle) against a hand-worked case, and the
oracle's sensitivity scan (Sec. 4.2.1) against what the block designs fix."""
import numpy as np
import pytest

import oracle
import oracle.strategy as ostrat
import paper_2502_20727_b200 as spd
import spd_inputs as si
from paper_2502_20727_b200 import build as spd_build


@pytest.fixture(scope="module", autouse=True)
def lib():
    spd_build.build()
    return spd.load_library()


def test_algorithm_1_hand_worked():
    # ascending order of S: block 1 (0.1), 3 (0.2), 0 (0.5), 4 (1.0), 2 (3.0); budget 4 leaves block 2 a TP block
    S = [0.5, 0.1, 3.0, 0.2, 1.0]
    want_mask = [0, 0, 1, 0, 0]
    want_tier = [ostrat.SB, ostrat.ISB, ostrat.TP, ostrat.ISB, ostrat.SB]  # tau1 = 0.3, tau2 = 1.0 (inclusive)
    assert ostrat.alg1_plan(S, 4, 0.3, 1.0) == (want_mask, want_tier)
    assert spd.alg1_plan(S, 4, 0.3, 1.0) == (want_mask, want_tier)
    # the whole budget: the most sensitive block is dropped last and is extremely sensitive
    assert spd.alg1_plan(S, 5, 0.3, 1.0) == ([0] * 5, [ostrat.SB, ostrat.ISB, ostrat.ESB, ostrat.ISB, ostrat.SB])
    assert spd.alg1_plan(S, 0, 0.3, 1.0) == ([1] * 5, [ostrat.TP] * 5)


def test_algorithm_1_matches_the_oracle_on_random_lists_with_ties():
    rng = np.random.default_rng(3)
    for _ in range(50):
        n = int(rng.integers(1, 12))
        S = [float(v) for v in rng.integers(0, 5, n) * 0.25]  # many ties
        n_spd = int(rng.integers(0, n + 1))
        assert spd.alg1_plan(S, n_spd, 0.25, 0.75) == ostrat.alg1_plan(S, n_spd, 0.25, 0.75)


def test_algorithm_1_rejects_bad_arguments():
    with pytest.raises(spd.SpdError):
        spd.alg1_plan([0.1, 0.2], 3, 0.1, 0.2)
    with pytest.raises(spd.SpdError):
        spd.alg1_plan([0.1, 0.2], 1, 0.5, 0.2)


def small(T, L=3, scale=8.0):
    w = si.Workload("scan", "fp32", L, 64, 4, 4, 16, 128, T, (0,) * L, 2, 9, 0)
    layers = si.to_oracle_layers(si.make_stack(w, "cpu", 5))
    for lw in layers:  # make the attention branch matter
        lw["wo"] = lw["wo"] * scale
    dims = oracle.Dims(L, 64, 4, 4, 16, 128, T)
    x = si.make_hidden(w, (2, 9, 64), "cpu", 5, 0).double().numpy()
    return dims, layers, x


def test_scan_is_zero_for_one_device():
    dims, layers, x = small(T=1)
    sens, metric = ostrat.sensitivity_scan(dims, layers, x)
    assert max(abs(v) for v in metric) < 1e-24  # T = 1: an SPD block is a TP block


def test_scan_telescopes_to_the_all_spd_metric_and_skips_a_block_without_attention_output():
    dims, layers, x = small(T=4)
    layers[1]["wo"] = np.zeros_like(layers[1]["wo"])  # block 1: Y_i = 0, so SPD == TP there
    sens, metric = ostrat.sensitivity_scan(dims, layers, x)
    L = dims.n_layers
    out_tp, _, _ = oracle.stack_forward(dims, [1] * L, layers, x, np.zeros(2, np.int32), oracle.Cache(dims, 2, 9))
    out_spd, _, _ = oracle.stack_forward(dims, [0] * L, layers, x, np.zeros(2, np.int32), oracle.Cache(dims, 2, 9))
    assert abs(sum(sens) - np.mean((out_spd - out_tp) ** 2)) < 1e-12 * metric[0]
    assert abs(sens[1]) < 1e-20 and sens[0] > 1e-9 and sens[2] > 1e-9
    assert metric[L] == 0.0
