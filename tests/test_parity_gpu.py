"""GPU parity: the CUDA library through its C ABI against the CPU oracle, element by element,
on the same seeded inputs.  Bound: max|gpu-ref|/max|ref| <= 1e-4 (float32), 2e-2 (bfloat16)."""
import numpy as np
import pytest
import torch

import spd_inputs as si
from parity_util import TOL, Pair, rel_err

pytestmark = pytest.mark.gpu


def run_case(w, mask, B, S, steps, max_prefill_tokens=None, check_cache=True, tuning=None):
    p = Pair(w, mask=mask, B=B, max_len=S + steps, max_prefill_tokens=max_prefill_tokens)
    if tuning:
        p.stack.set_tuning(**tuning)
    tol = TOL[w.dtype]
    got, ref, syncs = p.prefill(S)
    assert got.shape == ref.shape
    e = rel_err(got, ref)
    assert e <= tol, f"prefill rel err {e}"
    assert p.stack.sync_points() == syncs
    for t in range(steps):
        got, ref = p.decode(t)
        e = rel_err(got, ref)
        assert e <= tol, f"decode step {t} rel err {e}"
    if check_cache:
        n = S + steps
        for l in (0, w.n_layers - 1):
            for which in ("k", "v"):
                ref_c = getattr(p.cache, which)[l, B - 1, :n]
                e = rel_err(p.gpu_cache(l, which, B - 1, n), ref_c)
                assert e <= tol, f"{which} cache layer {l} rel err {e}"
    assert p.stack.device_error() == 0
    p.stack.close()


@pytest.mark.parametrize("mask", [(0,), (1,)])
def test_c1_tiny_fp32_full(mask):
    """configs[0]: 1 layer, hidden 256, 4 heads x 64, FFN 688, T=2, batch 1, 16 prompt + 8 decode."""
    w = si.WORKLOADS["c1"]
    run_case(w, mask, w.batch, w.prompt, w.decode_steps)


@pytest.mark.parametrize("T", [1, 2, 4])
@pytest.mark.parametrize("mask", [(0, 0), (1, 1), (1, 0)])
def test_fp32_two_layers_any_T(T, mask):
    w = si.WORKLOADS["c1"].with_(n_layers=2, T=T, mask=mask)
    run_case(w, mask, 3, 21, 3)


def test_fp32_without_rope_and_head_dim_32():
    w = si.WORKLOADS["c1"].with_(rope_base=0.0, head_dim=32, n_q_heads=8, n_kv_heads=4, T=4)
    run_case(w, (0,), 2, 19, 2)


@pytest.mark.parametrize("mask", [(0, 1, 0), (1, 1, 1)])
def test_bf16_small_ragged(mask):
    """Odd sizes: 5 tokens over a page boundary, FFN/T = 344 (not a tile multiple), GQA 8/4."""
    w = si.Workload("small", "bf16", 3, 512, 8, 4, 64, 1376, 4, mask, 3, 37, 3)
    run_case(w, mask, 3, 37, 3)


def test_bf16_chunked_prefill_inside_a_sequence():
    """max_prefill_tokens smaller than the prompt: later chunks attend to cached earlier ones."""
    w = si.Workload("small", "bf16", 2, 256, 4, 4, 64, 512, 2, (0, 1), 2, 50, 1)
    run_case(w, (0, 1), 2, 50, 1, max_prefill_tokens=16)


def test_bf16_chunked_prefill_by_sequences():
    w = si.Workload("small", "bf16", 2, 256, 4, 4, 64, 512, 2, (0, 0), 5, 20, 1)
    run_case(w, (0, 0), 5, 20, 1, max_prefill_tokens=45)


@pytest.mark.parametrize("name,layers,B,S", [("c2", 2, 2, 24), ("c3_t4", 1, 2, 20), ("c3_t8", 1, 1, 20),
                                             ("c4_b32", 1, 2, 18)])
def test_full_model_dims_reduced_tokens(name, layers, B, S):
    """Full hidden / head / FFN sizes of configs[1..3] with few tokens and layers."""
    w0 = si.WORKLOADS[name]
    mask = tuple(w0.mask[:layers]) if name != "c3_t4" else (0,)
    w = w0.with_(n_layers=layers, mask=mask)
    run_case(w, mask, B, S, 2, check_cache=False)


def test_mask_is_honoured_on_the_gpu():
    """An SPD mask on the GPU must NOT match the oracle's synchronous stack."""
    w = si.Workload("small", "bf16", 2, 256, 4, 4, 64, 512, 4, (0, 0), 2, 12, 0)
    lay = si.make_stack(w, "cpu", 0)
    for lw in lay:  # make the attention and MLP branches as large as the residual stream
        lw["wo"] = (lw["wo"].float() * 20).to(torch.bfloat16)
        for n in ("w_gate", "w_up", "w_down"):
            lw[n] = (lw[n].float() * 5).to(torch.bfloat16)
    p_spd = Pair(w, mask=(0, 0), B=2, max_len=12, layers=lay)
    got_spd, ref_spd, _ = p_spd.prefill(12)
    p_sync = Pair(w, mask=(1, 1), B=2, max_len=12, layers=lay)
    got_sync, ref_sync, _ = p_sync.prefill(12)
    assert rel_err(got_spd, ref_spd) <= TOL["bf16"]
    assert rel_err(got_sync, ref_sync) <= TOL["bf16"]
    assert rel_err(got_spd, ref_sync) > 5 * TOL["bf16"]


def test_decode_at_bench_size_on_synthetic_cache():
    """configs[1] at its full decode shape (4 layers, batch 8, context 512+) with the KV cache
    pre-filled with seeded values on both sides, so the oracle only pays for the decode step."""
    w = si.WORKLOADS["c2"]
    p = Pair(w, B=8, max_len=w.prompt + 4)
    lens = np.array([512, 512, 500, 512, 17, 512, 1, 511], dtype=np.int32)
    p.fill_cache(lens)
    for t in range(2):
        got, ref = p.decode(t)
        e = rel_err(got, ref)
        assert e <= TOL["bf16"], f"step {t}: {e}"
    assert p.stack.device_error() == 0


@pytest.mark.parametrize("nq,nkv,T", [(8, 2, 2), (16, 2, 2), (8, 1, 1)])
def test_bf16_grouped_query_head_dim_128(nq, nkv, T):
    """GQA groups of 4, 8 (tensor-core decode attention) with head_dim 128, ragged prompt over pages."""
    w = si.Workload("gqa", "bf16", 2, 512, nq, nkv, 128, 1024, T, (0, 1), 3, 45, 4)
    run_case(w, (0, 1), 3, 45, 4)


def test_gqa_decode_long_ragged_context_on_synthetic_cache():
    """configs[3] dims (64 query / 8 KV heads), one layer, contexts up to 2100 tokens with ragged
    lengths: several context splits and partially filled last pages."""
    w = si.WORKLOADS["c4_b32"].with_(n_layers=1, mask=(0,))
    p = Pair(w, B=4, max_len=2112)
    lens = np.array([2100, 17, 1, 1030], dtype=np.int32)
    p.fill_cache(lens)
    for t in range(2):
        got, ref = p.decode(t)
        e = rel_err(got, ref)
        assert e <= TOL["bf16"], f"step {t}: {e}"
    assert p.stack.device_error() == 0


@pytest.mark.parametrize("mask", [(0,), (1,)])
def test_prefill_over_several_tiles_at_full_width(mask):
    """configs[1] dims, one layer, one 300-token prompt: three 128-token GEMM tiles with a ragged
    tail, three 128-row attention tiles, every column tile of the real widths."""
    w = si.WORKLOADS["c2"].with_(n_layers=1, mask=mask)
    run_case(w, mask, 1, 300, 1, check_cache=True)


def test_single_token_prompt_and_single_sequence():
    """Degenerate sizes: a one-token prompt (prefill of M = 1), then decode with batch 1."""
    w = si.Workload("tiny", "bf16", 2, 256, 4, 2, 64, 512, 2, (0, 1), 1, 1, 3)
    run_case(w, (0, 1), 1, 1, 3)


def test_context_up_to_the_last_slot_of_the_last_page():
    """Decode until the cache is exactly full (max_seq_len = pages * 16): the last step writes the last slot."""
    w = si.Workload("tiny", "bf16", 1, 256, 4, 4, 64, 512, 2, (0,), 2, 29, 3)
    run_case(w, (0,), 2, 29, 3)  # 29 + 3 = 32 = two full pages


def test_out_of_range_page_is_flagged_not_followed():
    """A block-table entry outside [0, n_pages) must set the device error flag; the kernels skip or
    clamp the access instead of touching memory outside the page tensors."""
    w = si.Workload("tiny", "bf16", 1, 256, 4, 4, 64, 512, 2, (0,), 2, 20, 1)
    p = Pair(w, B=2, max_len=24)
    p.prefill(20)
    assert p.stack.device_error() == 0
    bad = p.block_table.clone()
    bad[1, 1] = p.n_pages + 7  # the page the next token of sequence 1 would go to
    x = si.make_hidden(w, (2, w.hidden), "cpu", 0, 1).to(p.device)
    seq = torch.full((2,), 20, dtype=torch.int32, device=p.device)
    p.stack.set_graphs(False)
    p.stack.decode_step(x, seq, bad, 21)
    torch.cuda.synchronize()
    assert p.stack.device_error() & 1
    assert p.stack.device_error() == 0  # reading clears it
    # the stack is still usable
    out = p.stack.decode_step(x, seq, p.block_table, 21)
    torch.cuda.synchronize()
    assert torch.isfinite(out.float()).all() and p.stack.device_error() == 0


@pytest.mark.parametrize("B", [40, 70])
def test_bf16_decode_batches_beyond_32(B):
    """Decode token tiles of 64 (batch 40) and two token tiles (batch 70), SPD and TP blocks."""
    w = si.Workload("wide", "bf16", 2, 256, 4, 4, 64, 512, 2, (0, 1), B, 18, 2)
    run_case(w, (0, 1), B, 18, 2, check_cache=False)


def test_bf16_head_dim_32_without_rope():
    """Eight heads per 256-row prefill tile, four per 128-row decode tile, rotary embedding off."""
    w = si.Workload("d32", "bf16", 2, 256, 8, 4, 32, 512, 4, (0, 1), 3, 21, 2).with_(rope_base=0.0)
    run_case(w, (0, 1), 3, 21, 2)


def test_bf16_hidden_not_a_multiple_of_16_takes_the_unfused_prefill():
    w = si.Workload("h264", "bf16", 1, 264, 4, 4, 64, 512, 2, (0,), 2, 10, 1)
    run_case(w, (0,), 2, 10, 1)


def test_run_twice_bitwise_identical():
    w = si.Workload("small", "bf16", 2, 512, 8, 8, 64, 1024, 4, (0, 1), 4, 33, 2)
    outs = []
    for _ in range(2):
        p = Pair(w, B=4, max_len=40)
        a, _, _ = p.prefill(33)
        b, _ = p.decode(0)
        outs.append((a, b))
    assert np.array_equal(outs[0][0], outs[1][0]) and np.array_equal(outs[0][1], outs[1][1])


@pytest.mark.parametrize("rescale_log2", [0, 2])
def test_prefill_attention_rescale_path(rescale_log2):
    """The tensor-core prefill attention rescales its accumulated output in tensor memory whenever the running
    row maximum outgrows the one in use by more than 2^rescale_log2: with 0 every growth goes through that path
    (with the default of 8 and N(0,1) inputs it hardly ever runs).  700 tokens = 6 key tiles with a ragged last
    one, GQA group of 4, head_dim 128, second sequence chunked inside the prompt."""
    w = si.Workload("fa_rescale", "bf16", 2, 512, 8, 2, 128, 1024, 2, (0, 1), 2, 700, 1)
    p = Pair(w, mask=(0, 1), B=2, max_len=704, max_prefill_tokens=512)
    p.stack.set_tuning(prefill_rescale_log2=rescale_log2)
    got, ref, _ = p.prefill(700)
    e = rel_err(got, ref)
    assert e <= TOL["bf16"], f"prefill rel err {e}"
    got, ref = p.decode(0)
    assert rel_err(got, ref) <= TOL["bf16"]
    assert p.stack.device_error() == 0
    p.stack.close()


def test_prefill_attention_long_prompt_many_key_tiles():
    """1500-token prompts: up to 12 key tiles per query tile (each K / V ring slot reused six times, a ragged last
    tile), GQA group of 4, head_dim 128, prompt cut into chunks of 1024 tokens that attend to the cache."""
    w = si.Workload("fa_long", "bf16", 1, 512, 8, 2, 128, 1024, 2, (0,), 2, 1500, 1)
    p = Pair(w, mask=(0,), B=2, max_len=1504, max_prefill_tokens=1024)
    got, ref, _ = p.prefill(1500)
    e = rel_err(got, ref)
    assert e <= TOL["bf16"], f"prefill rel err {e}"
    got, ref = p.decode(0)
    assert rel_err(got, ref) <= TOL["bf16"]
    assert p.stack.device_error() == 0
    p.stack.close()


@pytest.mark.parametrize("stages", [3, 4, 5])
def test_decode_ring_depth_is_only_a_schedule(stages):
    """The weight tiles of a decode projection stream through a ring of 3, 4 or 5 stages (chosen per launch by
    default): any depth gives the same numbers, bit for bit."""
    w = si.Workload("ring", "bf16", 2, 1024, 8, 4, 128, 2752, 4, (0, 1), 5, 40, 2)
    outs = []
    for st in (0, stages):
        p = Pair(w, mask=(0, 1), B=5, max_len=48)
        p.fill_cache(np.array([40, 7, 16, 33, 1], dtype=np.int32))
        p.stack.set_tuning(decode_ring_stages=st)
        got, ref = p.decode(0)
        assert rel_err(got, ref) <= TOL["bf16"]
        got2, ref2 = p.decode(1)
        assert rel_err(got2, ref2) <= TOL["bf16"]
        assert p.stack.device_error() == 0
        outs.append((got, got2))
        p.stack.close()
    assert np.array_equal(outs[0][0], outs[1][0]) and np.array_equal(outs[0][1], outs[1][1])


@pytest.mark.parametrize("mask", [(1, 1), (0, 0), (0, 1)])
def test_prefill_on_cta_pairs_equals_prefill_on_single_blocks(mask):
    """Launches with more than 128 tokens run their projections on pairs of thread blocks (256-token tiles, one
    tensor-core instruction over two SMs, each block loading half of the tile's weight rows).  Same K order, same
    accumulators: the output is bit-identical to the one-block-per-tile schedule, and both match the oracle.
    520 tokens = two full 256-token tiles and a third whose second block has only 8 valid rows; FFN / T = 344."""
    w = si.Workload("pairs", "bf16", 2, 512, 8, 4, 64, 1376, 4, mask, 2, 260, 1)
    outs = []
    for pairs in (1, 0):
        p = Pair(w, mask=mask, B=2, max_len=264, max_prefill_tokens=1024)
        p.stack.set_tuning(prefill_pairs=pairs)
        got, ref, _ = p.prefill(260)
        assert rel_err(got, ref) <= TOL["bf16"]
        got_d, ref_d = p.decode(0)
        assert rel_err(got_d, ref_d) <= TOL["bf16"]
        assert p.stack.device_error() == 0
        outs.append((got, got_d))
        p.stack.close()
    assert np.array_equal(outs[0][0], outs[1][0]) and np.array_equal(outs[0][1], outs[1][1])
