"""The launch timeline (spd_timeline_*): kernels stamp their start and end inside the replayed decode graph, a
small kernel at the end of each step folds the stamps into every launch's own share of the step.  Checked here:
the launch list, that the shares never exceed the steps' spans, that the spans agree with the event-timed
duration of the same back-to-back steps, and that stamping changes no result."""
import numpy as np
import pytest
import torch

import spd_inputs as si
from parity_util import Pair

pytestmark = pytest.mark.gpu


def test_decode_step_shares_add_up_to_the_step():
    w = si.Workload("tl", "bf16", 3, 1024, 8, 4, 128, 2752, 4, (0, 1, 0), 5, 40, 2)
    p = Pair(w, mask=(0, 1, 0), B=5, max_len=96)
    p.fill_cache(np.array([40, 7, 16, 33, 1], dtype=np.int32))
    x = si.make_hidden(w, (5, w.hidden), "cpu", 0, 1).to(p.device)
    seq = torch.tensor([40, 7, 16, 33, 1], dtype=torch.int32, device=p.device)
    out_plain, out_tl = torch.empty_like(x), torch.empty_like(x)
    for _ in range(2):  # capture, then replay
        p.stack.decode_step(x, seq, p.block_table, 41, out_plain)
    torch.cuda.synchronize()

    p.stack.timeline_begin()
    for _ in range(3):
        p.stack.decode_step(x, seq, p.block_table, 41, out_tl)
    torch.cuda.synchronize()
    p.stack.timeline_begin()  # totals of the warm-up steps cleared, graph kept
    n = 20
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(n):
        p.stack.decode_step(x, seq, p.block_table, 41, out_tl)
    e1.record()
    torch.cuda.synchronize()
    launches, span_ns, calls = p.stack.timeline_read()
    p.stack.timeline_end()

    assert calls == n
    per_block = ["gemm_qkv", "attention", "gemm_o_proj", "gemm_gate_up", "gemm_down"]
    assert [k for k, _ in launches] == ["residual_rmsnorm"] + per_block * 3
    assert all(ns > 0 for _, ns in launches)
    own = sum(ns for _, ns in launches)
    assert own <= span_ns                                     # overlap is never counted twice
    assert own >= 0.5 * span_ns                               # and the launches cover most of the step
    event_ns = e0.elapsed_time(e1) * 1e6
    assert span_ns <= event_ns * 1.02                         # the steps' spans fit inside the event-timed region ...
    assert span_ns >= 0.5 * event_ns                          # ... and make up most of it (the rest: graph launch gaps)
    assert torch.equal(out_plain, out_tl)                     # stamping changes nothing
    # after spd_timeline_end the step runs (and is captured) without slots again
    out_after = torch.empty_like(x)
    p.stack.decode_step(x, seq, p.block_table, 41, out_after)
    torch.cuda.synchronize()
    assert torch.equal(out_plain, out_after) and p.stack.device_error() == 0
    p.stack.close()


def test_prefill_launch_list_and_read_without_begin():
    import paper_2502_20727_b200 as spd
    w = si.Workload("tlp", "bf16", 2, 512, 8, 2, 128, 1024, 2, (0, 1), 2, 150, 1)
    p = Pair(w, mask=(0, 1), B=2, max_len=160)
    with pytest.raises(spd.SpdError):
        p.stack.timeline_read()
    x = si.make_hidden(w, (2, 150, w.hidden), "cpu", 0, 0).to(p.device)
    ref = p.stack.prefill(x, p.block_table)
    p.stack.timeline_begin()
    got = p.stack.prefill(x, p.block_table)
    launches, span_ns, calls = p.stack.timeline_read()
    p.stack.timeline_end()
    assert calls == 1 and span_ns > 0
    per_block = ["gemm_qkv", "attention", "gemm_o_proj", "gemm_gate_up", "gemm_down"]
    assert [k for k, _ in launches] == ["rope_table", "residual_rmsnorm"] + per_block * 2
    assert 0 < sum(ns for _, ns in launches) <= span_ns
    assert torch.equal(ref, got)
    p.stack.close()
