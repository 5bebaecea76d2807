"""The sensitivity scan of Sec. 4.2.1 through the C ABI against the oracle's scan, and the block
selection that follows from it."""
import numpy as np
import pytest
import torch

import oracle
import oracle.strategy as ostrat
import paper_2502_20727_b200 as spd
import spd_inputs as si
from parity_util import Pair

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("dtype,tol", [("fp32", 2e-3), ("bf16", 0.1)])
def test_scan_matches_the_oracle_and_gives_the_same_plan(dtype, tol):
    L, T = 4, 4
    w = si.Workload("scan", dtype, L, 256, 8, 8, 32, 512, T, (0,) * L, 2, 40, 0)
    layers = si.make_stack(w, "cpu", 7)
    for i, lw in enumerate(layers):  # blocks differ in how much their attention branch matters
        lw["wo"] = (lw["wo"].float() * (2.0 + 6.0 * i)).to(w.torch_dtype)
    layers[2]["wo"] = torch.zeros_like(layers[2]["wo"])  # block 2: SPD == TP
    p = Pair(w, B=2, max_len=40, layers=layers)
    x = si.make_hidden(w, (2, 40, w.hidden), "cpu", 7, 0)
    sens, metric = p.stack.sensitivity_scan(x.to(p.device), p.block_table)
    ref_s, ref_m = ostrat.sensitivity_scan(p.dims, p.layers_np, x.double().numpy())
    scale = max(ref_m)
    assert scale > 0
    assert np.max(np.abs(np.array(metric) - np.array(ref_m))) <= tol * scale
    assert np.max(np.abs(np.array(sens) - np.array(ref_s))) <= tol * scale
    assert abs(sens[2]) <= tol * scale
    # thresholds in the gaps of the oracle's values: both sides must take the same decisions
    order = np.sort(ref_s)
    tau1, tau2 = (order[0] + order[1]) / 2, (order[2] + order[3]) / 2
    assert spd.alg1_plan(sens, 3, tau1, tau2) == ostrat.alg1_plan(ref_s, 3, tau1, tau2)
    # the context still runs its own mask afterwards
    assert list(p.stack.mask) == [0] * L
    assert p.stack.device_error() == 0


def test_scan_needs_the_spd_workspace():
    w = si.Workload("scan", "bf16", 2, 256, 4, 4, 64, 512, 2, (1, 1), 1, 8, 0)
    p = Pair(w, mask=(1, 1), B=1, max_len=8)
    x = si.make_hidden(w, (1, 8, w.hidden), "cpu", 0, 0).to(p.device)
    with pytest.raises(spd.SpdError) as ei:
        p.stack.sensitivity_scan(x, p.block_table)
    assert ei.value.status == -3
    with pytest.raises(spd.SpdError):
        p.stack.set_mask([0, 1])
    p.stack.set_mask([1, 1])
