"""Baseline of the rank mode (spd_tp_baseline_*): one shard's stack per rank, the shard sums the block keeps done by a
collective BETWEEN kernels.  Here the T ranks are T host threads on one GPU, each with its own context, stream and
KV pages; their all-reduce is a host-side rendezvous (nothing on the device waits for another rank).  Every rank's
output is compared with the CPU oracle's sharded block, element by element (2e-2, bfloat16), the ranks with each
other (bit-identical: same sums in the same order), and the number of all-reduces with the sync-points of the mask."""
import threading

import numpy as np
import pytest
import torch

import oracle
import paper_2502_20727_b200 as spd
import spd_inputs as si
from parity_util import TOL, oracle_dims, rel_err, to_np

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


class ThreadAllReduce:
    """Sum over the T threads' views in rank order; each thread gets the same bits."""

    def __init__(self, T):
        self.T, self.barrier, self.views, self.calls = T, threading.Barrier(T), [None] * T, [0] * T

    def for_rank(self, r):
        def all_reduce(view):
            torch.cuda.current_stream().synchronize()  # this rank's partial sums are complete
            self.views[r] = view
            self.barrier.wait()
            total = self.views[0].clone()
            for j in range(1, self.T):
                total += self.views[j]
            torch.cuda.current_stream().synchronize()
            self.barrier.wait()                           # nobody overwrites before everybody has read
            view.copy_(total)
            self.calls[r] += 1
        return all_reduce


@pytest.mark.parametrize("T,mask", [(2, (1, 0)), (4, (0, 1, 0)), (2, (1, 1))])
def test_ranks_with_a_collective_between_kernels_match_the_oracle(T, mask):
    L = len(mask)
    w = si.Workload("tp_base", "bf16", L, 512, 8, 4, 64, 1024, T, mask, 3, 37, 2)
    layers = si.make_stack(w, "cpu", 0)
    B, S, steps = 3, 37, 2
    dims = oracle_dims(w)
    cache = oracle.Cache(dims, B, S + steps)
    lnp = si.to_oracle_layers(layers)
    x = si.make_hidden(w, (B, S, w.hidden), "cpu", 0, 0)
    ref_p, syncs, _ = oracle.stack_forward(dims, list(mask), lnp, to_np(x), np.zeros(B, np.int32), cache)
    xs = [si.make_hidden(w, (B, w.hidden), "cpu", 0, 1 + t) for t in range(steps)]
    ref_d = [oracle.stack_forward(dims, list(mask), lnp, to_np(xs[t])[:, None, :], np.full(B, S + t, np.int32), cache)[0][:, 0]
             for t in range(steps)]
    one = w.with_(n_q_heads=w.n_q_heads // T, n_kv_heads=w.n_kv_heads // T, ffn=w.ffn // T, T=1)
    pages = (S + steps + w.kv_block - 1) // w.kv_block
    reducer = ThreadAllReduce(T)
    results, errors = [None] * T, []

    def rank_main(r):
        try:
            with torch.cuda.stream(torch.cuda.Stream(device=DEV)):
                shard = [{n: t.to(DEV) for n, t in spd.shard_layer(lw, r, T).items()} for lw in layers]
                stack = spd.stack_from_workload(one, shard, sync_mask=mask, max_batch=B, max_seq_len=S + steps,
                                                n_pages=B * pages + 2, max_prefill_tokens=64, device=DEV)  # prompts in chunks
                bt = si.make_block_table(B, pages, B * pages + 2, r).to(DEV)
                ar = reducer.for_rank(r)
                outs = [to_np(stack.tp_baseline_prefill(x.to(DEV), bt, ar))]
                for t in range(steps):
                    seq = torch.full((B,), S + t, dtype=torch.int32, device=DEV)
                    outs.append(to_np(stack.tp_baseline_decode_step(xs[t].to(DEV), seq, bt, S + t + 1, ar)))
                torch.cuda.current_stream().synchronize()
                assert stack.device_error() == 0
                stack.close()
                results[r] = outs
        except Exception as e:  # a failing rank must not leave the others at the rendezvous
            errors.append(e)
            reducer.barrier.abort()

    threads = [threading.Thread(target=rank_main, args=(r,)) for r in range(T)]
    for th in threads:
        th.start()
    for th in threads:
        th.join(timeout=300)
    assert not errors, errors
    for r in range(T):
        assert rel_err(results[r][0], ref_p) <= TOL["bf16"]
        for t in range(steps):
            assert rel_err(results[r][1 + t], ref_d[t]) <= TOL["bf16"]
        for a, b in zip(results[0], results[r]):
            assert np.array_equal(a, b)                     # all ranks hold the same bits
    # one all-reduce per kept sync-point and launch: 37 tokens in chunks of 64 -> 3 sequences x 1 chunk ... count launches
    per_launch = sum(2 if m else 1 for m in mask)
    assert syncs == per_launch
    launches = B + steps                                    # max_prefill_tokens 64 < 2 prompts: one prompt per launch
    assert reducer.calls == [per_launch * launches] * T


def test_a_failing_all_reduce_is_reported_and_a_full_stack_is_refused():
    w = si.Workload("tp_base1", "bf16", 1, 256, 4, 4, 64, 512, 1, (1,), 1, 8, 0)
    layers = [{n: t.to(DEV) for n, t in lw.items()} for lw in si.make_stack(w, "cpu", 0)]
    with torch.cuda.stream(torch.cuda.Stream(device=DEV)):
        stack = spd.stack_from_workload(w, layers, sync_mask=(1,), max_batch=1, max_seq_len=8, n_pages=2, device=DEV)
        bt = torch.tensor([[0]], dtype=torch.int32, device=DEV)
        x = si.make_hidden(w, (1, 8, w.hidden), "cpu", 0, 0).to(DEV)

        def broken(view):
            raise RuntimeError("link down")
        with pytest.raises(RuntimeError, match="link down"):
            stack.tp_baseline_prefill(x, bt, broken)
        torch.cuda.synchronize()
        # a group of one: the all-reduce is the identity and the result is the plain stack's
        got = stack.tp_baseline_prefill(x, bt, lambda view: None)
        ref = stack.prefill(x, bt)
        torch.cuda.synchronize()
        assert rel_err(to_np(got), to_np(ref)) <= 1e-2
        stack.close()
        w2 = w.with_(T=2)
        two = spd.stack_from_workload(w2, layers, sync_mask=(1,), max_batch=1, max_seq_len=8, n_pages=2, device=DEV)
        with pytest.raises(spd.SpdError) as ei:
            two.tp_baseline_prefill(x, bt, lambda view: None)
        assert ei.value.status == -1
        two.close()
