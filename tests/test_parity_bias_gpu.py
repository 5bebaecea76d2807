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


@pytest.mark.parametrize("mask", [(0, 1, 0), (1, 1, 1)])
def test_bf16_on_the_unfused_sequence(mask):
    """The K-split GEMMs with separate LayerNorm / bias kernels stay selectable (tuning key bias_fused = 0)."""
    w = opt("optbf", "bf16", 3, 512, 8, 8, 64, 1376, 4, mask, 3, 37, 3)
    run_case(w, mask, 3, 37, 3, tuning={"bias_fused": 0})


@pytest.mark.parametrize("mask", [(0, 0), (1, 1), (0, 1)])
def test_bf16_prompt_over_several_token_tiles_and_a_ragged_fc1_tile(mask):
    """300 prompt tokens (CTA pairs, a ragged last tile), 688 fc1 rows per shard (not a multiple of the fc1 tile),
    then decode steps at a batch of 2; LayerNorm is folded into the QKV and fc1 tails on this path."""
    w = opt("optbf2", "bf16", 2, 1024, 8, 8, 128, 2752, 4, mask, 2, 150, 3)
    run_case(w, mask, 2, 150, 3)


def test_bf16_decode_batch_of_several_token_boxes():
    """Decode at a batch of 40 (token box 64) after a short prompt, both block kinds in one stack."""
    w = opt("optbf3", "bf16", 2, 1024, 8, 8, 128, 2048, 8, (0, 1), 40, 9, 2)
    run_case(w, (0, 1), 40, 9, 2)


def test_fused_and_unfused_sequences_agree():
    """Same stack, same inputs: folding LayerNorm into the tails changes rounding, nothing else."""
    w = opt("optbf4", "bf16", 2, 1024, 8, 8, 128, 2752, 4, (0, 1), 2, 150, 0)
    outs = []
    for fused in (1, 0):
        p = Pair(w, mask=(0, 1), B=2, max_len=150)
        p.stack.set_tuning(bias_fused=fused)
        got, ref, _ = p.prefill(150)
        assert rel_err(got, ref) <= TOL["bf16"]
        outs.append(got)
        p.stack.close()
    assert rel_err(outs[0], outs[1]) <= TOL["bf16"]


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
