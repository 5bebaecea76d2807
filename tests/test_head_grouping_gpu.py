"""Head grouping measurements (Sec. 4.2.4) through the C ABI against the oracle: head distances of Eq. 2,
MLP output norms of Eq. 3, and the decisions taken from them."""
import numpy as np
import pytest
import torch

import oracle.head_grouping as ohg
import paper_2502_20727_b200 as spd
import spd_inputs as si
from parity_util import Pair

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("nq,nkv,d,T,layer", [(8, 8, 64, 4, 1), (8, 2, 128, 2, 0)])
def test_measurements_match_the_oracle(nq, nkv, d, T, layer):
    w = si.Workload("hg", "bf16", 2, 256, nq, nkv, d, 512, T, (0, 0), 2, 24, 0)
    layers = si.make_stack(w, "cpu", 9)
    for lw in layers:  # sharper attention and a visible attention branch
        lw["wq"] = (lw["wq"].float() * 6).to(torch.bfloat16)
        lw["wo"] = (lw["wo"].float() * 6).to(torch.bfloat16)
    p = Pair(w, B=2, max_len=24, layers=layers)
    x = si.make_hidden(w, (2, 24, w.hidden), "cpu", 9, 0)
    dist, norms = p.stack.head_grouping_stats(layer, x.to(p.device), p.block_table)
    assert p.stack.device_error() == 0
    xin = ohg.block_input(p.dims, p.layers_np, x.double().numpy(), layer)
    ref_d = ohg.head_distances(ohg.head_scores(p.dims, p.layers_np[layer], xin))
    ref_n = ohg.mlp_norms(p.dims, p.layers_np[layer], xin)
    # Both quantities are Euclidean norms (of a difference of two score vectors, of an MLP output), so by the triangle
    # inequality their error is at most the norm of the error of the vectors they are taken of: the rms-relative error
    # of a block-level bf16 tensor, measured at 0.6e-2 ... 0.8e-2 per block against the 2e-2 bound on its largest
    # element (twice that for a distance, which has two vectors in it; the scores add the bf16 rounding of q and k
    # in the exponent, relative 2^-9 * |score|).  3e-2 of the largest entry leaves a factor of two over that.
    assert np.max(np.abs(dist - ref_d)) <= 3e-2 * ref_d.max()
    assert np.max(np.abs(norms - ref_n)) <= 3e-2 * ref_n.max()
    # decisions: the library's searches on its own measurements reach the optimum of the oracle's measurements
    group = nq // nkv
    dev, _ = spd.head_scatter(dist, group, T)
    _, best = ohg.scatter_bruteforce(ref_d, group, T)
    assert ohg.scatter_objective(ref_d, group, dev) >= best * (1 - 5e-2)
    perm, _ = spd.mlp_match(norms)
    _, best_m = ohg.mlp_match_bruteforce(ref_n)
    assert sum(ref_n[i, perm[i]] for i in range(T)) >= best_m * (1 - 5e-2)


def test_fp32_and_oversized_batches_are_refused():
    w = si.Workload("hg", "fp32", 1, 256, 4, 4, 64, 512, 2, (0,), 1, 8, 0)
    p = Pair(w, B=1, max_len=8)
    x = si.make_hidden(w, (1, 8, w.hidden), "cpu", 0, 0).to(p.device)
    with pytest.raises(spd.SpdError) as ei:
        p.stack.head_grouping_stats(0, x, p.block_table)
    assert ei.value.status == -1
