"""The tensor-core projection GEMM on its own against the oracle's linear layer."""
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


def ref_linear(a, w):
    return oracle.linear(a.double().numpy(), w.float().numpy())


@pytest.mark.parametrize("swap", [True, False])
@pytest.mark.parametrize("M,N,K,splits", [(8, 256, 512, 1), (8, 256, 512, 4), (1, 128, 64, 1), (33, 384, 1376, 3),
                                          (64, 1000, 4096, 5), (130, 344, 256, 2), (300, 200, 8 * 37, 1)])
def test_plain_gemm(swap, M, N, K, splits):
    a, w = rand_bf16((M, K), 1), rand_bf16((N, K), 2)
    c = spd.gemm_bf16(a.cuda(), w.cuda(), splits=splits, swap=swap)
    got = c.sum(0).double().cpu().numpy()
    ref = ref_linear(a, w)
    assert rel_err(got, ref) < 2e-5  # fp32 accumulation of exact bf16 products
    if splits > 1:  # every plane is a partial sum over its own K range, none is empty
        assert all(float(c[s].abs().max()) > 0 for s in range(splits))


@pytest.mark.parametrize("swap", [True, False])
@pytest.mark.parametrize("a_batched", [False, True])
def test_shard_batched_gemm(swap, a_batched):
    """T weight row-blocks of 344 rows (not a tile multiple); optionally one input per shard."""
    T, M, N, K = 4, 24, 344, 512
    w = rand_bf16((T, N, K), 3)
    a = rand_bf16((T, M, K) if a_batched else (M, K), 4)
    c = spd.gemm_bf16(a.cuda(), w.cuda(), splits=2, swap=swap).sum(0).double().cpu().numpy()
    for z in range(T):
        ref = ref_linear(a[z] if a_batched else a, w[z])
        assert rel_err(c[:, z * N:(z + 1) * N], ref) < 2e-5
