"""GPU parity of the decoder block with bias (OPT-style, Sec. 4.1.2) through the C ABI against the oracle."""
import numpy as np
import pytest
import torch

import oracle
import spd_inputs as si
from parity_util import TOL, Pair, rel_err
from test_parity_gpu import run_case

pytestmark = pytest.mark.gpu


def opt(name, dtype, L, H, nq, nkv, d, F, T, mask, B, S, steps):
    return si.Workload(name, dtype, L, H, nq, nkv, d, F, T, mask, B, S, steps, block="opt")


@pytest.mark.parametrize("T", [1, 2, 4])
@pytest.mark.parametrize("mask", [(0, 0), (1, 1), (1, 0)])
def test_fp32_two_layers_any_T(T, mask):
    w = opt("opt32", "fp32", 2, 256, 4, 4, 64, 688, T, mask, 3, 21, 3)
    run_case(w, mask, 3, 21, 3)


@pytest.mark.parametrize("mask", [(0, 1, 0), (1, 1, 1)])
def test_bf16_small_ragged(mask):
    w = opt("optbf", "bf16", 3, 512, 8, 8, 64, 1376, 4, mask, 3, 37, 3)
    run_case(w, mask, 3, 37, 3)


def test_opt_6_7b_dims_reduced_tokens():
    """hidden 4096, 32 heads x 128, ffn 16384 (OPT-6.7B, Sec. 5.1), T = 8, one SPD block, few tokens."""
    w = opt("opt67", "bf16", 1, 4096, 32, 32, 128, 16384, 8, (0,), 2, 20, 2)
    run_case(w, (0,), 2, 20, 2, check_cache=False)


def test_bias_placement_is_the_papers_not_the_rejected_one():
    """The GPU's SPD block must match the design of Sec. 4.1.2 (b after the sum, once) and must NOT match the
    rejected design of Table 1(b) (b before the sum, T times), nor the synchronous block."""
    T = 4
    w = opt("optbias", "fp32", 1, 256, 4, 4, 64, 512, T, (0,), 2, 12, 0)
    lay = si.make_stack(w, "cpu", 0)
    for lw in lay:
        lw["wo"] = lw["wo"] * 20  # make the attention branch count
    p = Pair(w, mask=(0,), B=2, max_len=12, layers=lay)
    got, ref, _ = p.prefill(12)
    assert rel_err(got, ref) <= TOL["fp32"]
    x = si.make_hidden(w, (2, 12, w.hidden), "cpu", 0, 0).double().numpy()
    rej, _, _ = oracle.bias_block_forward(p.dims, p.layers_np[0], 2, x, np.zeros(2, np.int32), oracle.Cache(p.dims, 2, 12))
    syn, _, _ = oracle.bias_block_forward(p.dims, p.layers_np[0], 1, x, np.zeros(2, np.int32), oracle.Cache(p.dims, 2, 12))
    assert rel_err(got, rej) > 100 * TOL["fp32"]
    assert rel_err(got, syn) > 100 * TOL["fp32"]
