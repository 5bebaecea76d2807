"""GPU parity of the rank-mode decode step (tensor parallelism across GPUs, Sec. 3 / Sec. 4.1.1):
all T ranks of a group executed on one GPU - every launch covers all ranks' data, and the shard
sums are exchanges through per-rank receive planes and arrival flags in global memory, the same
kernels and protocol a group of T GPUs runs over peer-mapped memory - against the CPU oracle's
sharded block, element by element.  Bound: max|gpu-ref|/max|ref| <= 2e-2 (bfloat16)."""
import time

import numpy as np
import pytest
import torch

import spd_inputs as si
from parity_util import TOL, Pair, rel_err

pytestmark = pytest.mark.gpu


def run_tp_case(w, mask, B, lens, steps):
    p = Pair(w, mask=mask, B=B, max_len=int(max(lens)) + steps + 1)
    p.fill_cache(np.asarray(lens, dtype=np.int32))
    p.stack.tp_attach_local()
    torch.cuda.synchronize()
    for t in range(steps):
        got, ref = p.tp_decode(t)
        assert got.shape == (w.T,) + ref.shape
        for r in range(w.T):
            e = rel_err(got[r], ref)
            assert e <= TOL["bf16"], f"step {t} rank {r}: rel err {e}"
        # every rank adds the same planes in the same order: the copies are bit-identical
        for r in range(1, w.T):
            assert np.array_equal(got[r], got[0]), f"step {t}: rank {r} differs from rank 0"
    assert p.stack.device_error() == 0
    return p


@pytest.mark.parametrize("mask", [(0, 0), (1, 1), (0, 1, 0)])
@pytest.mark.parametrize("T", [2, 4])
def test_rank_mode_small(T, mask):
    """Ragged contexts over page boundaries, FFN/T not a tile multiple, GQA 8/4, mixed masks."""
    w = si.Workload("tp_small", "bf16", len(mask), 512, 8, 4, 64, 1376, T, mask, 3, 37, 3)
    p = run_tp_case(w, mask, 3, [37, 5, 16], 5)   # (0, 1, 0): 4 exchanges a step; (0, 0): 2; (1, 1): 4
    p.stack.close()


def test_rank_mode_odd_number_of_exchanges_alternates_two_graphs():
    """One SPD block = one exchange a step: consecutive steps use the two receive buffers in turn, each
    phase replaying its own captured graph."""
    mask = (0,)
    w = si.Workload("tp_odd", "bf16", 1, 512, 8, 4, 64, 1376, 4, mask, 3, 37, 3)
    p = run_tp_case(w, mask, 3, [20, 5, 16], 6)
    p.stack.close()


def test_rank_mode_eight_ranks_head_dim_128():
    """T = 8 at head_dim 128 (tensor-core decode attention for the GQA group of 4), batch 5."""
    mask = (1, 0)
    w = si.Workload("tp8", "bf16", 2, 1024, 32, 8, 128, 2048, 8, mask, 5, 70, 2)
    p = run_tp_case(w, mask, 5, [70, 1, 33, 64, 17], 2)
    p.stack.close()


@pytest.mark.parametrize("mask,T,S", [((0, 1, 0), 4, 37), ((1, 0), 2, 150)])
def test_rank_mode_prompts_then_decode(mask, T, S):
    """Prompts through the rank-mode step (several 64-token tiles, chunks that attend to the chunks before them),
    then decode steps on the caches it filled."""
    w = si.Workload("tp_prompt", "bf16", len(mask), 512, 8, 4, 64, 1376, T, mask, 3, S, 2)
    p = Pair(w, mask=mask, B=3, max_len=S + 2)
    p.stack.tp_attach_local()
    torch.cuda.synchronize()
    got, ref, _ = p.tp_prefill(S)
    for r in range(T):
        e = rel_err(got[r], ref)
        assert e <= TOL["bf16"], f"prompt, rank {r}: rel err {e}"
        assert np.array_equal(got[r], got[0])
    for t in range(2):
        got, ref = p.tp_decode(t)
        for r in range(T):
            assert rel_err(got[r], ref) <= TOL["bf16"]
    assert p.stack.device_error() == 0
    p.stack.close()


def test_rank_mode_prompt_head_dim_128_chunked():
    """head_dim 128 (tensor-core prompt attention), 8 ranks: 128 tiles per 64 tokens, so the prompt goes in
    chunks of 192 tokens; 300-token prompts are cut inside the sequence."""
    mask = (0, 1)
    w = si.Workload("tp_prompt128", "bf16", 2, 1024, 16, 8, 128, 2048, 8, mask, 2, 300, 1)
    p = Pair(w, mask=mask, B=2, max_len=304)
    p.stack.tp_attach_local()
    torch.cuda.synchronize()
    got, ref, _ = p.tp_prefill(300)
    for r in (0, 3, 7):
        e = rel_err(got[r], ref)
        assert e <= TOL["bf16"], f"prompt, rank {r}: rel err {e}"
    got, ref = p.tp_decode(0)
    assert rel_err(got[0], ref) <= TOL["bf16"]
    assert p.stack.device_error() == 0
    p.stack.close()


@pytest.mark.parametrize("B", [20, 40])
def test_rank_mode_larger_batches(B):
    """Token tiles of 32 and 64 (other instantiations of the exchange tail), ragged contexts, mixed mask."""
    mask = (1, 0)
    w = si.Workload("tp_batch", "bf16", 2, 512, 8, 4, 64, 1376, 4, mask, B, 40, 2)
    lens = [1 + (7 * i) % 40 for i in range(B)]
    p = run_tp_case(w, mask, B, lens, 2)
    p.stack.close()


def test_rank_mode_matches_the_single_launch_emulation():
    """The same stack through spd_decode_step (shards as one cluster per tile) and through the rank-mode
    step: two implementations of one function, equal to rounding."""
    mask = (0, 1)
    w = si.Workload("tp_vs", "bf16", 2, 1024, 16, 16, 64, 2752, 4, mask, 4, 50, 2)
    p = Pair(w, mask=mask, B=4, max_len=64)
    lens = np.array([50, 3, 31, 48], dtype=np.int32)
    p.fill_cache(lens)
    x = si.make_hidden(w, (4, w.hidden), "cpu", 0, 1).to("cuda:0")
    seq = torch.from_numpy(lens.copy()).to("cuda:0")
    a = p.stack.decode_step(x, seq, p.block_table, 51).float().cpu().numpy()
    # the step appended K/V at position lens[b]; the rank-mode step rewrites the same slots
    p.stack.tp_attach_local()
    b = p.stack.tp_decode_step(x, seq, p.block_table, 51).float().cpu().numpy()
    torch.cuda.synchronize()
    assert rel_err(b[0], a) <= 1e-2
    assert p.stack.device_error() == 0
    p.stack.close()


def test_configs1_shape_one_layer_all_ranks():
    """configs[1] dims (hidden 4096, 32 heads x 128, FFN 11008, T = 8), one TP and one SPD layer, batch 8 on a
    synthetic cache: 256 thread blocks per exchange launch, all resident at once."""
    mask = (1, 0)
    w = si.WORKLOADS["c2"].with_(n_layers=2, mask=mask)
    p = run_tp_case(w, mask, 8, [200, 17, 1, 130, 64, 199, 100, 5], 1)
    p.stack.close()


def test_a_rank_that_never_arrives_is_reported_not_waited_for():
    """Rank 0 of a group of two whose peer never runs: the wait for the peer's partial sums ends after
    its time limit, the step returns, the error flag says so, and the context stays usable."""
    import paper_2502_20727_b200 as spd
    mask = (0,)
    full = si.Workload("tp_alone", "bf16", 1, 256, 4, 4, 64, 512, 2, mask, 2, 8, 1)
    layers = si.make_stack(full, "cpu", 0)
    shard = [{n: t.to("cuda:0") for n, t in spd.shard_layer(lw, 0, 2).items()} for lw in layers]
    one = full.with_(n_q_heads=2, n_kv_heads=2, ffn=256, T=1)
    with torch.cuda.stream(torch.cuda.Stream(device="cuda:0")):   # the previous current stream comes back afterwards
        stack = spd.stack_from_workload(one, shard, sync_mask=mask, max_batch=2, max_seq_len=16, n_pages=4,
                                        max_prefill_tokens=64, device="cuda:0")
        nbytes = (stack.tp_region_bytes(2) + 1023) // 1024 * 1024
        regions = torch.zeros(2 * nbytes + 1024, dtype=torch.uint8, device="cuda:0")
        base = (regions.data_ptr() + 1023) // 1024 * 1024
        stack.tp_attach(2, 0, [base, base + nbytes], nbytes)   # rank 1's region exists, but nobody plays rank 1
        stack.set_tuning(peer_wait_ms=20)                      # the limit is a tuning key: fail fast here
        x = si.make_hidden(one, (2, one.hidden), "cpu", 0, 1).to("cuda:0")
        seq = torch.zeros(2, dtype=torch.int32, device="cuda:0")
        bt = torch.tensor([[0], [1]], dtype=torch.int32, device="cuda:0")
        t0 = time.perf_counter()
        out = stack.tp_decode_step(x, seq, bt, 1)
        torch.cuda.synchronize()
        waited = time.perf_counter() - t0
        assert out.shape == (1, 2, 256)
        assert stack.device_error() & 8
        assert waited < 0.5, f"gave up after {waited:.3f} s with a 20 ms limit"
        # usable afterwards: the ordinary single-GPU step of the shard's stack runs clean
        stack.tp_detach()
        y = stack.decode_step(x, seq, bt, 1)
        torch.cuda.synchronize()
        assert torch.isfinite(y.float()).all()
        assert stack.device_error() == 0
        stack.close()


def test_attach_argument_checks_and_mask_change_while_attached():
    """Bad groups / regions are refused with a status code; the per-block mask may change between steps of an
    attached context (every rank does so at the same step): the exchanges keep alternating their buffers."""
    import paper_2502_20727_b200 as spd
    mask = (0, 0)
    w = si.Workload("tp_args", "bf16", 2, 512, 8, 4, 64, 1376, 4, mask, 3, 20, 4)
    p = Pair(w, mask=mask, B=3, max_len=32)
    st = p.stack
    with pytest.raises(spd.SpdError):                      # not attached yet
        st.tp_decode_step(torch.zeros((3, 512), dtype=torch.bfloat16, device="cuda:0"),
                          torch.zeros(3, dtype=torch.int32, device="cuda:0"), p.block_table, 1)
    nbytes = (st.tp_region_bytes(4) + 1023) // 1024 * 1024
    buf = torch.zeros(4 * nbytes + 2048, dtype=torch.uint8, device="cuda:0")
    base = (buf.data_ptr() + 1023) // 1024 * 1024
    good = [base + j * nbytes for j in range(4)]
    with pytest.raises(spd.SpdError):                      # a context of 4 shards is ranks 0..3 of a group of 4, nothing else
        st.tp_attach(8, 0, good + good, nbytes)
    with pytest.raises(spd.SpdError):                      # misaligned region
        st.tp_attach(4, 0, [g + 16 for g in good], nbytes)
    with pytest.raises(spd.SpdError):                      # region too small
        st.tp_attach(4, 0, good, nbytes // 2)
    with pytest.raises(spd.SpdError):                      # regions of the local ranks not at equal distances
        st.tp_attach(4, 0, [good[0], good[1], good[3], good[2]], nbytes)
    st.tp_attach(4, 0, good, nbytes)
    torch.cuda.synchronize()
    p.fill_cache(np.array([20, 3, 11], dtype=np.int32))
    for t, m in enumerate([(0, 0), (1, 0), (1, 1), (0, 1)]):   # 2, 3, 4, 3 exchanges per step
        st.set_mask(m)
        p.mask = list(m)
        got, ref = p.tp_decode(t)
        for r in range(4):
            assert rel_err(got[r], ref) <= TOL["bf16"], f"mask {m}, rank {r}"
    assert st.device_error() == 0
    st.close()


def test_a_launch_whose_ranks_cannot_all_be_resident_is_refused():
    """8 ranks at hidden 16384: 1024 thread blocks per exchange launch wait on one another, more than the GPU holds at
    once - refused before anything runs, not left to time out."""
    import paper_2502_20727_b200 as spd
    mask = (0,)
    w = si.Workload("tp_big", "bf16", 1, 16384, 8, 8, 128, 2048, 8, mask, 1, 4, 1)
    p = Pair(w, mask=mask, B=1, max_len=16)
    p.fill_cache(np.array([4], dtype=np.int32))
    p.stack.tp_attach_local()
    x = torch.zeros((1, 16384), dtype=torch.bfloat16, device="cuda:0")
    with pytest.raises(spd.SpdError) as e:
        p.stack.tp_decode_step(x, torch.full((1,), 4, dtype=torch.int32, device="cuda:0"), p.block_table, 5)
    assert e.value.status == -5   # SPD_ECUDA (cooperative launch too large)
    torch.cuda.synchronize()
    p.stack.tp_detach()
    assert p.stack.device_error() == 0
    p.stack.close()


@pytest.mark.parametrize("T,mask,B,S,chunk", [(4, (1, 0, 1), 2, 300, 4096), (2, (0, 0), 3, 200, 256), (8, (1,), 1, 130, 4096)])
def test_rank_mode_prompts_over_many_tiles(T, mask, B, S, chunk):
    """Prompts at tensor-core speed in rank mode: the prompt projections on CTA pairs per rank, the kept shard sums as
    two-shot exchanges over 128-token tiles dealt round-robin to the ranks.  600 tokens = five tiles for four ranks (one
    rank owns two); chunks of 256 tokens cut prompts inside the sequence; 130 tokens for 8 ranks leave six ranks without
    a tile.  Every rank against the oracle, ranks bit-identical, then decode steps on the caches."""
    w = si.Workload("tp_fast", "bf16", len(mask), 512, 8, 8, 64, 1024, T, mask, B, S, 2)
    p = Pair(w, mask=mask, B=B, max_len=S + 2, max_prefill_tokens=chunk)
    p.stack.tp_attach_local()
    torch.cuda.synchronize()
    got, ref, _ = p.tp_prefill(S)
    for r in range(T):
        e = rel_err(got[r], ref)
        assert e <= TOL["bf16"], f"prompt, rank {r}: rel err {e}"
        assert np.array_equal(got[r], got[0])
    for t in range(2):
        got, ref = p.tp_decode(t)
        for r in range(T):
            assert rel_err(got[r], ref) <= TOL["bf16"]
    assert p.stack.device_error() == 0
    p.stack.close()


def test_a_prompt_whose_peer_never_runs_is_reported_not_waited_for():
    """Rank 0 of a group of two, its peer absent: the owner's wait for the peer's partial rows and the wait for the
    peer's finished tile both run out (20 ms each), the call returns, error bit 8 is set, the context stays usable."""
    import paper_2502_20727_b200 as spd
    mask = (1,)
    full = si.Workload("tp_alone_p", "bf16", 1, 256, 4, 4, 64, 512, 2, mask, 1, 200, 0)
    layers = si.make_stack(full, "cpu", 0)
    shard = [{n: t.to("cuda:0") for n, t in spd.shard_layer(lw, 0, 2).items()} for lw in layers]
    one = full.with_(n_q_heads=2, n_kv_heads=2, ffn=256, T=1)
    with torch.cuda.stream(torch.cuda.Stream(device="cuda:0")):
        stack = spd.stack_from_workload(one, shard, sync_mask=mask, max_batch=1, max_seq_len=208, n_pages=14,
                                        max_prefill_tokens=256, device="cuda:0")
        nbytes = (stack.tp_region_bytes(2) + 1023) // 1024 * 1024
        regions = torch.zeros(2 * nbytes + 1024, dtype=torch.uint8, device="cuda:0")
        base = (regions.data_ptr() + 1023) // 1024 * 1024
        stack.tp_attach(2, 0, [base, base + nbytes], nbytes)
        stack.set_tuning(peer_wait_ms=20)
        x = si.make_hidden(one, (1, 200, one.hidden), "cpu", 0, 0).to("cuda:0")
        bt = torch.arange(13, dtype=torch.int32, device="cuda:0")[None]
        t0 = time.perf_counter()
        out = stack.tp_prefill(x, bt)
        torch.cuda.synchronize()
        waited = time.perf_counter() - t0
        assert out.shape == (1, 1, 200, 256)
        assert stack.device_error() & 8
        assert waited < 1.0, f"gave up after {waited:.3f} s with a 20 ms limit"
        stack.tp_detach()
        y = stack.prefill(x, bt)
        torch.cuda.synchronize()
        assert torch.isfinite(y.float()).all() and stack.device_error() == 0
        stack.close()
