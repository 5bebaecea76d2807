"""Oracle of the SPD-aware attention head grouping measurements and searches (Sec. 4.2.4; test
infrastructure like the rest of this folder).  Plain numpy over the paper's definitions: attention
scores per head, their pairwise Euclidean distances (Eq. 2), exhaustive head scattering, the norms
of MLP_m(A_i) and the exhaustive matching of Eq. 3."""
from __future__ import annotations

import itertools

import numpy as np

from . import Cache, Dims, block_forward, linear, rmsnorm, rope, stack_forward


def block_input(dims: Dims, layers, x, layer: int):
    """Hidden states entering block `layer` when the blocks before it are TP blocks (Sec. 4.2.3)."""
    if layer == 0:
        return np.asarray(x, dtype=np.float64)
    B, S, H = x.shape
    sub = Dims(layer, dims.hidden, dims.n_q_heads, dims.n_kv_heads, dims.head_dim, dims.ffn, dims.T, dims.rms_eps, dims.rope_base)
    out, _, _ = stack_forward(sub, [1] * layer, layers[:layer], x, np.zeros(B, np.int32), Cache(sub, B, S))
    return out


def head_scores(dims: Dims, lw, xin):
    """sigma[h, b, i, j]: causal softmax of q_i . k_j / sqrt(d) of head h (0 above the diagonal)."""
    B, S, H = xin.shape
    d, nq, nkv = dims.head_dim, dims.n_q_heads, dims.n_kv_heads
    h = rmsnorm(xin.reshape(B * S, H), lw["attn_norm"], dims.rms_eps)
    Q = linear(h, lw["wq"]).reshape(B, S, nq, d)
    K = linear(h, lw["wk"]).reshape(B, S, nkv, d)
    if dims.rope_base > 0:
        for b in range(B):
            for s in range(S):
                for j in range(nq):
                    Q[b, s, j] = rope(Q[b, s, j], s, dims.rope_base)
                for j in range(nkv):
                    K[b, s, j] = rope(K[b, s, j], s, dims.rope_base)
    sigma = np.zeros((nq, B, S, S))
    group = nq // nkv
    for hq in range(nq):
        for b in range(B):
            sc = Q[b, :, hq] @ K[b, :, hq // group].T / np.sqrt(d)
            for i in range(S):
                row = sc[i, : i + 1]
                p = np.exp(row - row.max())
                sigma[hq, b, i, : i + 1] = p / p.sum()
    return sigma


def head_distances(sigma):
    n = sigma.shape[0]
    flat = sigma.reshape(n, -1)
    D = np.zeros((n, n))
    for a in range(n):
        for b in range(n):
            D[a, b] = np.sqrt(np.sum((flat[a] - flat[b]) ** 2))
    return D


def unit_distances(D, heads_per_unit):
    n = D.shape[0] // heads_per_unit
    U = np.zeros((n, n))
    for a in range(n):
        for b in range(n):
            if a != b:
                U[a, b] = D[a * heads_per_unit:(a + 1) * heads_per_unit, b * heads_per_unit:(b + 1) * heads_per_unit].sum()
    return (U + U.T) / 2


def scatter_objective(D, heads_per_unit, device_of_unit):
    U = unit_distances(D, heads_per_unit)
    n = U.shape[0]
    return sum(U[a, b] for a in range(n) for b in range(a + 1, n) if device_of_unit[a] == device_of_unit[b])


def scatter_bruteforce(D, heads_per_unit, T):
    """Eq. 2 by brute force: every way of dealing the units to T devices in equal shares."""
    U = unit_distances(D, heads_per_unit)
    n = U.shape[0]
    cap = n // T
    best, best_assign = -1.0, None
    for assign in itertools.product(range(T), repeat=n):
        if any(assign.count(t) != cap for t in range(T)):
            continue
        obj = sum(U[a, b] for a in range(n) for b in range(a + 1, n) if assign[a] == assign[b])
        if obj > best + 1e-15:
            best, best_assign = obj, assign
    return list(best_assign), best


def mlp_norms(dims: Dims, lw, xin):
    """norms[i, m] = || MLP_m(rmsnorm(X + Y_i)) ||_F: partition m's slice of gate/up/down on device i's input (Eq. 3)."""
    B, S, H = xin.shape
    T, F = dims.T, dims.ffn
    Fs = F // T
    one = Dims(1, dims.hidden, dims.n_q_heads, dims.n_kv_heads, dims.head_dim, dims.ffn, dims.T, dims.rms_eps, dims.rope_base)
    _, y, _ = block_forward(one, lw, 0, xin, np.zeros(B, np.int32), Cache(one, B, S))
    X = xin.reshape(B * S, H)
    out = np.zeros((T, T))
    for i in range(T):
        u = rmsnorm(X + y[i], lw["mlp_norm"], dims.rms_eps)
        for m in range(T):
            g = linear(u, lw["w_gate"][m * Fs:(m + 1) * Fs])
            up = linear(u, lw["w_up"][m * Fs:(m + 1) * Fs])
            a = g / (1.0 + np.exp(-g)) * up
            z = linear(a, np.ascontiguousarray(lw["w_down"][:, m * Fs:(m + 1) * Fs]))
            out[i, m] = np.sqrt(np.sum(z * z))
    return out


def mlp_match_bruteforce(N):
    T = N.shape[0]
    best, best_perm = -1.0, None
    for perm in itertools.permutations(range(T)):
        s = sum(N[i, perm[i]] for i in range(T))
        if s > best + 1e-15:
            best, best_perm = s, perm
    return list(best_perm), best
