"""Head grouping on the CPU: the host searches of Eq. 2 / Eq. 3 (C ABI) against brute force, and the oracle's
measurements against what their definitions fix."""
import itertools

import numpy as np
import pytest

import oracle
import oracle.head_grouping as ohg
import paper_2502_20727_b200 as spd
import spd_inputs as si
from paper_2502_20727_b200 import build as spd_build


@pytest.fixture(scope="module", autouse=True)
def lib():
    spd_build.build()
    return spd.load_library()


def random_dist(n, seed):
    pts = np.random.default_rng(seed).standard_normal((n, 5))
    return np.sqrt(((pts[:, None] - pts[None]) ** 2).sum(-1))


def test_two_identical_pairs_are_split_across_devices():
    # heads 0,1 identical and heads 2,3 identical: the even distribution puts one of each on a device
    D = np.array([[0, 0, 5, 5], [0, 0, 5, 5], [5, 5, 0, 0], [5, 5, 0, 0]], dtype=np.float64)
    dev, obj = spd.head_scatter(D, 1, 2)
    assert dev[0] != dev[1] and dev[2] != dev[3] and obj == 10.0


@pytest.mark.parametrize("n,T,hpu", [(8, 4, 1), (6, 3, 1), (8, 2, 1), (16, 4, 2), (12, 3, 1)])
def test_scatter_is_the_brute_force_optimum(n, T, hpu):
    """8 heads on 4 devices is the case the paper draws; also GQA units of two heads."""
    D = random_dist(n, n * 7 + T)
    dev, obj = spd.head_scatter(D, hpu, T)
    ref_dev, ref_obj = ohg.scatter_bruteforce(D, hpu, T)
    assert sorted(np.bincount(dev, minlength=T)) == [n // hpu // T] * T
    assert abs(obj - ref_obj) <= 1e-5 * ref_obj
    assert abs(ohg.scatter_objective(D, hpu, dev) - ref_obj) <= 1e-5 * ref_obj


def test_scatter_heuristic_for_many_heads_is_balanced_and_beats_the_contiguous_split():
    n, T = 32, 8
    D = random_dist(n, 11)
    dev, obj = spd.head_scatter(D, 1, T)
    assert sorted(np.bincount(dev, minlength=T)) == [4] * T
    contiguous = [u // 4 for u in range(n)]
    assert obj >= ohg.scatter_objective(D, 1, contiguous)
    assert abs(obj - ohg.scatter_objective(D, 1, dev)) <= 1e-5 * obj
    # no single swap improves it (local optimum)
    for a, b in itertools.combinations(range(n), 2):
        if dev[a] != dev[b]:
            sw = list(dev)
            sw[a], sw[b] = sw[b], sw[a]
            assert ohg.scatter_objective(D, 1, sw) <= obj * (1 + 1e-6)


@pytest.mark.parametrize("T", [1, 2, 4, 6])
def test_match_is_the_brute_force_optimum(T):
    N = np.random.default_rng(T).uniform(1, 2, (T, T))
    perm, obj = spd.mlp_match(N)
    ref_perm, ref_obj = ohg.mlp_match_bruteforce(N)
    assert sorted(perm) == list(range(T)) and abs(obj - ref_obj) < 1e-12 and perm == ref_perm


def test_bad_arguments():
    with pytest.raises(spd.SpdError):
        spd.head_scatter(np.zeros((6, 6)), 1, 4)  # 6 units on 4 devices
    with pytest.raises(spd.SpdError):
        spd.mlp_match(np.zeros((9, 9)))


def small():
    w = si.Workload("hg", "fp32", 2, 64, 4, 2, 16, 128, 2, (0, 0), 2, 7, 0)
    layers = si.to_oracle_layers(si.make_stack(w, "cpu", 3))
    dims = oracle.Dims(2, 64, 4, 2, 16, 128, 2)
    x = si.make_hidden(w, (2, 7, 64), "cpu", 3, 0).double().numpy()
    return dims, layers, x


def test_oracle_scores_are_causal_distributions_and_equal_heads_are_at_distance_zero():
    dims, layers, x = small()
    lw = dict(layers[0])
    lw["wq"] = lw["wq"].copy()
    lw["wq"][16:32] = lw["wq"][0:16]  # head 1 = head 0 (same KV head): identical scores
    sigma = ohg.head_scores(dims, lw, x)
    assert np.allclose(sigma.sum(-1), 1.0) and np.all(np.triu(sigma[0, 0], 1) == 0)
    D = ohg.head_distances(sigma)
    assert D[0, 1] < 1e-12 and D[0, 2] > 1e-3 and np.allclose(D, D.T) and np.all(np.diag(D) == 0)


def test_oracle_mlp_norms_reassemble_the_spd_block():
    """sum_i MLP_i(X + Y_i) with the diagonal pairing is the MLP sum of the SPD block (Sec. 4.1.1)."""
    dims, layers, x = small()
    one = oracle.Dims(1, 64, 4, 2, 16, 128, 2)
    N = ohg.mlp_norms(dims, layers[0], x)
    assert N.shape == (2, 2) and np.all(N > 0)
    # zeroing MLP partition 1 zeroes column 1 only
    lw = dict(layers[0])
    lw["w_down"] = lw["w_down"].copy()
    lw["w_down"][:, 64:] = 0
    N2 = ohg.mlp_norms(dims, lw, x)
    assert np.all(N2[:, 1] == 0) and np.allclose(N2[:, 0], N[:, 0])
    # block input of block 1 is the TP output of block 0
    xin = ohg.block_input(dims, layers, x, 1)
    ref, _, _ = oracle.stack_forward(one, [1], layers[:1], x, np.zeros(2, np.int32), oracle.Cache(one, 2, 7))
    assert np.array_equal(xin, ref)


def test_reordering_keeps_the_tp_block_and_changes_the_spd_block():
    """Sec. 4.2.4: the re-ordering only decides which heads and MLP partition share a device."""
    import torch
    dims, layers, x = small()
    lw_t = {k: torch.from_numpy(np.ascontiguousarray(v)) for k, v in layers[0].items()}
    order = spd.head_order_from_devices([1, 0], 2, 2)  # the two KV groups swap devices
    assert order == [2, 3, 0, 1]
    new = spd.permute_layer(lw_t, n_q_heads=4, n_kv_heads=2, head_dim=16, T=2, head_order=order, mlp_of_device=[1, 0])
    new_np = {k: v.numpy() for k, v in new.items()}
    one = oracle.Dims(1, 64, 4, 2, 16, 128, 2)
    def run(lw, mask):
        out, _, _ = oracle.stack_forward(one, mask, [lw], x, np.zeros(2, np.int32), oracle.Cache(one, 2, 7))
        return out
    assert np.max(np.abs(run(new_np, [1]) - run(layers[0], [1]))) < 1e-12
    # swapping both the head sets and the MLP partitions is a whole-device swap: SPD unchanged too
    assert np.max(np.abs(run(new_np, [0]) - run(layers[0], [0]))) < 1e-12
    # moving only the MLP partitions re-pairs <A_i, MLP_m>: the SPD block changes
    only_mlp = {k: v.numpy() for k, v in spd.permute_layer(lw_t, n_q_heads=4, n_kv_heads=2, head_dim=16, T=2, mlp_of_device=[1, 0]).items()}
    assert np.max(np.abs(run(only_mlp, [1]) - run(layers[0], [1]))) < 1e-12
    assert np.max(np.abs(run(only_mlp, [0]) - run(layers[0], [0]))) > 1e-6
