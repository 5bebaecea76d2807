"""Oracle of the per-block strategy (test infrastructure, like the rest of this folder): the
progressive sensitivity scan of Sec. 4.2.1 on the oracle's own forward pass, with the mean
squared difference from the all-TP output as the metric in place of perplexity, and the block
selection of Algorithm 1.  Plain loops over the paper's steps; shares nothing with the CUDA path."""
from __future__ import annotations

import numpy as np

from . import Cache, Dims, stack_forward

TP, ISB, SB, ESB = 0, 1, 2, 3


def sensitivity_scan(dims: Dims, layers, x):
    """x: [B, S, H].  metric[i] = MSE(output with blocks i..L-1 SPD and 0..i-1 TP, all-TP output),
    metric[L] = 0; S[i] = metric[i] - metric[i+1] (Sec. 4.2.1: the change from also applying SPD to
    block i when all later blocks are SPD blocks already)."""
    L = dims.n_layers
    B, S, _ = x.shape
    pos0 = np.zeros(B, np.int32)

    def run(mask):
        out, _, _ = stack_forward(dims, mask, layers, x, pos0, Cache(dims, B, S))
        return out

    ref = run([1] * L)
    metric = [0.0] * (L + 1)
    for i in range(L - 1, -1, -1):
        mask = [1] * i + [0] * (L - i)
        metric[i] = float(np.mean((run(mask) - ref) ** 2))
    sens = [metric[i] - metric[i + 1] for i in range(L)]
    return sens, metric


def alg1_plan(S, n_spd, tau1, tau2):
    """Algorithm 1: B = block indices in ascending order of S; the first n_spd become SPD blocks,
    labelled ISB (S <= tau1), SB (S <= tau2) or ESB."""
    n = len(S)
    B = sorted(range(n), key=lambda b: (S[b], b))
    mask, tier = [1] * n, [TP] * n
    for i in range(n_spd):
        blk = B[i]
        mask[blk] = 0
        if S[blk] <= tau1:
            tier[blk] = ISB
        elif S[blk] <= tau2:
            tier[blk] = SB
        else:
            tier[blk] = ESB
    return mask, tier
