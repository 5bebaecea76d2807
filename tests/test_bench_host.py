"""Host-side logic of bench.py that needs no GPU: the masks a configuration is run with, the bounded oracle sample, and the byte / flop counts of the roofline."""
import os
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

import bench  # noqa: E402
import spd_inputs as si  # noqa: E402


def test_masks_per_configuration():
    assert set(bench.masks_of(si.WORKLOADS["c2"])) == {"sync", "spd"}            # its own mask is all-SPD
    m = bench.masks_of(si.WORKLOADS["c3_t4"])
    assert m["config"] == (1, 0, 0, 0, 0, 0, 0, 1) and m["sync"] == (1,) * 8 and m["spd"] == (0,) * 8
    m5 = bench.masks_of(si.WORKLOADS["c5"])
    assert sum(m5["config"]) == 10 and len(m5["config"]) == 40


def test_oracle_sample_is_bounded_and_keeps_the_mask_mix():
    w = si.WORKLOADS["c5"]
    layers, B, scale = bench.oracle_sample(w, w.mask)
    assert len(layers) == 4 and scale == 4 / 40 and 1 <= B <= w.batch
    assert sum(w.mask[l] for l in layers) == 1                                    # 25 % TP blocks, as in the mask
    assert 2.0 * w.params_per_layer() / 1e9 * len(layers) * B <= 60.0             # a few seconds per step
    layers, B, scale = bench.oracle_sample(w, (1,) * 40)
    assert all(l < 40 for l in layers) and len(layers) == 4
    w2 = si.WORKLOADS["c2"]
    assert bench.oracle_sample(w2, w2.mask) == ([0, 1, 2, 3], 8, 1.0)             # small enough: the whole step


def test_algorithmic_bytes_and_flops():
    w = si.WORKLOADS["c2"]
    gw = bench.gemm_weight_bytes(w)
    assert gw["gemm_qkv"] == 3 * 4096 * 4096 * 2 and gw["gemm_gate_up"] == 2 * 11008 * 4096 * 2
    weights, kv = bench.decode_bytes(w, 8, 576)
    assert weights == 4 * w.params_per_layer() * 2 and kv == 4 * 8 * 576 * 2 * 32 * 128 * 2
    # 2 flops per weight and token, plus causal attention (half of 4 S^2 nq d)
    assert bench.prefill_flops(w, 1, 512) == 4 * (2.0 * sum(gw.values()) / 2 * 512 + 2.0 * 512 * 512 * 32 * 128)
