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


def metric_tolerance(dtype, ref_out, scale):
    """Absolute tolerance of a metric = mean((out_a - out_b)^2) of two stack outputs.
    bf16: each output element v is rounded once more to bf16 on its way out, an error uniform within +-u|v|, u = 2^-8,
    independent between the two passes wherever they differ; it does not cancel in the difference but adds its variance,
    2 u^2 mean(v^2) / 3, to the mean square (the cross term with the true difference averages out over the elements).
    The bf16 roundings inside the blocks that differ between the passes are of the same size: the floor is doubled.
    That is what the outputs can resolve, not a margin of the kernels - here about a tenth of the largest metric, because
    the SPD / TP difference (rms 0.02) is small against the outputs themselves (up to 7).
    fp32: the same floor with u = 2^-24 is nil; 2e-3 of the largest metric covers the fp32 reassociation of the sums."""
    if dtype == "fp32":
        return 2e-3 * scale
    u = 2.0 ** -8
    return 2 * (2 * u * u * float(np.mean(np.square(ref_out))) / 3)


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
def test_scan_matches_the_oracle_and_gives_the_same_plan(dtype):
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
    ref_out, _, _ = oracle.stack_forward(p.dims, [1] * L, p.layers_np, x.double().numpy(), np.zeros(2, np.int32),
                                         oracle.Cache(p.dims, 2, 40))
    tol = metric_tolerance(dtype, ref_out, scale)
    assert tol <= 0.15 * scale                                 # the floor stays a fraction of what is being measured
    assert np.max(np.abs(np.array(metric) - np.array(ref_m))) <= tol
    assert np.max(np.abs(np.array(sens) - np.array(ref_s))) <= 2 * tol   # a difference of two metrics
    assert abs(sens[2]) <= 2 * tol
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
