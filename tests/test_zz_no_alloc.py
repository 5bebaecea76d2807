"""spd_gemm_bf16_sum_static - the entry point for callers that cannot allocate device memory
while they call the library (an engine whose allocator owns the GPU, a plugin under a
no-cudaMalloc rule).  Its split planes live in a fixed array inside the library, shared by all
calls, so the check runs it twice in a row with different shapes (the second call finds the
first one's leftovers in the array) and compares each result with the sum of the planes that the
ordinary entry point, spd_gemm_bf16, writes to caller memory - and with the CPU oracle's linear layer.
A further check watches the device allocator around a call: nothing may be allocated.  Collected last
on purpose."""
import numpy as np
import pytest
import torch

import oracle
import paper_2502_20727_b200 as spd
from parity_util import rel_err

pytestmark = pytest.mark.gpu


def rand_bf16(shape, seed):
    g = torch.Generator().manual_seed(seed)
    return torch.randn(shape, generator=g).to(torch.bfloat16)


def oracle_linear(a, w):
    """The oracle's linear layer per shard block: [M, batches*N] (a, w on the host)."""
    wb = w if w.dim() == 3 else w[None]
    cols = [oracle.linear((a[z] if a.dim() == 3 else a).double().numpy(), wb[z].float().numpy()) for z in range(wb.shape[0])]
    return np.concatenate(cols, axis=1)


def both(a, w, splits, swap):
    batches = w.shape[0] if w.dim() == 3 else 1
    M, N = a.shape[-2], w.shape[-2]
    out = torch.full((M, batches * N), float("nan"), dtype=torch.float32, device="cuda")
    err = torch.zeros(1, dtype=torch.int32, device="cuda")
    spd.gemm_bf16_sum_static(a, w, out, err, splits=splits, swap=swap)
    ref = spd.gemm_bf16(a, w, splits=splits, swap=swap).sum(0)
    torch.cuda.synchronize()
    assert int(err.item()) == 0
    return out.double().cpu().numpy(), ref.double().cpu().numpy()


@pytest.mark.parametrize("swap", [True, False])
def test_two_calls_in_a_row_match_the_allocating_entry_point_and_the_oracle(swap):
    # first call: 4 shard blocks of 344 rows with one input per shard, 3 splits (ragged tiles)
    a1, w1 = rand_bf16((4, 24, 512), 11), rand_bf16((4, 344, 512), 12)
    got, ref = both(a1.cuda(), w1.cuda(), 3, swap)
    assert rel_err(got, ref) < 2e-5
    assert rel_err(got, oracle_linear(a1, w1)) < 2e-5  # fp32 accumulation of exact bf16 products
    # second call: smaller and differently shaped, so stale planes of the first call lie around it
    a2, w2 = rand_bf16((8, 1376), 13), rand_bf16((200, 1376), 14)
    got, ref = both(a2.cuda(), w2.cuda(), 5, swap)
    assert rel_err(got, ref) < 2e-5
    assert rel_err(got, oracle_linear(a2, w2)) < 2e-5


def test_a_call_allocates_no_device_memory():
    """What the entry point is for: once the first call on the device has looked up the array's address, a call
    leaves the torch allocator's and the driver's view of device memory exactly as it found them."""
    a, w = rand_bf16((8, 1376), 21).cuda(), rand_bf16((200, 1376), 22).cuda()
    out = torch.empty((8, 200), dtype=torch.float32, device="cuda")
    err = torch.zeros(1, dtype=torch.int32, device="cuda")
    spd.gemm_bf16_sum_static(a, w, out, err, splits=4, swap=True)  # warm-up: symbol look-up, kernel images
    torch.cuda.synchronize()
    before = (torch.cuda.memory_allocated(), torch.cuda.memory_reserved(), torch.cuda.mem_get_info()[0])
    spd.gemm_bf16_sum_static(a, w, out, err, splits=4, swap=True)
    torch.cuda.synchronize()
    after = (torch.cuda.memory_allocated(), torch.cuda.memory_reserved(), torch.cuda.mem_get_info()[0])
    assert before == after
    assert int(err.item()) == 0
    assert rel_err(out.double().cpu().numpy(), oracle_linear(a.cpu(), w.cpu())) < 2e-5


def test_a_problem_larger_than_the_array_is_refused():
    a, w = rand_bf16((128, 64), 15).cuda(), rand_bf16((8192, 64), 16).cuda()  # 128*8192*4 B = the whole array
    out = torch.empty((128, 8192), dtype=torch.float32, device="cuda")
    err = torch.zeros(1, dtype=torch.int32, device="cuda")
    spd.gemm_bf16_sum_static(a, w, out, err, splits=1)  # exactly fits
    a2 = rand_bf16((129, 64), 17).cuda()
    out2 = torch.empty((129, 8192), dtype=torch.float32, device="cuda")
    with pytest.raises(spd.SpdError) as ei:
        spd.gemm_bf16_sum_static(a2, w, out2, err, splits=1)
    assert ei.value.status == -3
    torch.cuda.synchronize()
