"""Pins of the oracle's decoder block with bias (OPT-style, Sec. 4.1.2) to things other than itself: the
`transformers` OPT decoder layer, torch's LayerNorm, and what the paper fixes about where the bias goes."""
import numpy as np
import pytest
import torch

import oracle
import spd_inputs as si
from oracle import Cache, Dims


def rel_err(a, b):
    return float(np.max(np.abs(a - b)) / np.max(np.abs(b)))


def layer_np(w, seed=1):
    return {k: v.float().numpy() for k, v in si.make_bias_layer(w, 0, "cpu", seed).items()}


def work(nq=4, nkv=4, T=1, L=1):
    return si.Workload("opt", "fp32", L, 32, nq, nkv, 8, 48, T, (0,) * L, 2, 6, 0, block="opt")


def x_of(B, S, H, seed=0):
    return np.random.default_rng(seed).standard_normal((B, S, H))


def dims_of(w):
    return Dims(w.n_layers, w.hidden, w.n_q_heads, w.n_kv_heads, w.head_dim, w.ffn, w.T, 1e-5, 0.0)


def test_layernorm_matches_torch():
    x = x_of(1, 5, 32)[0] * 3 + 1
    g, b = np.linspace(0.5, 1.5, 32).astype(np.float32), np.linspace(-1, 1, 32).astype(np.float32)
    ref = torch.nn.functional.layer_norm(torch.from_numpy(x), (32,), torch.from_numpy(g).double(), torch.from_numpy(b).double(), 1e-5)
    assert rel_err(oracle.layernorm(x, g, b, 1e-5), ref.numpy()) < 1e-13


def test_unsharded_block_matches_transformers_opt_layer():
    """The single-device block is the OPT decoder layer (pre-LayerNorm, ReLU, biases everywhere)."""
    from transformers.models.opt.modeling_opt import OPTConfig, OPTDecoderLayer
    w = work()
    lw = layer_np(w)
    cfg = OPTConfig(hidden_size=32, num_attention_heads=4, ffn_dim=48, num_hidden_layers=1, vocab_size=8, word_embed_proj_dim=32,
                    do_layer_norm_before=True, activation_function="relu", enable_bias=True, dropout=0.0, attention_dropout=0.0,
                    layer_norm_elementwise_affine=True)
    cfg._attn_implementation = "sdpa"
    layer = OPTDecoderLayer(cfg, layer_idx=0).double().eval()
    names = {"self_attn.q_proj.weight": "wq", "self_attn.q_proj.bias": "bq", "self_attn.k_proj.weight": "wk", "self_attn.k_proj.bias": "bk",
             "self_attn.v_proj.weight": "wv", "self_attn.v_proj.bias": "bv", "self_attn.out_proj.weight": "wo", "self_attn.out_proj.bias": "bo",
             "self_attn_layer_norm.weight": "attn_norm", "self_attn_layer_norm.bias": "attn_norm_b", "fc1.weight": "w_fc1", "fc1.bias": "b_fc1",
             "fc2.weight": "w_fc2", "fc2.bias": "b_fc2", "final_layer_norm.weight": "mlp_norm", "final_layer_norm.bias": "mlp_norm_b"}
    with torch.no_grad():
        for n, p in layer.named_parameters():
            p.copy_(torch.from_numpy(lw[names[n]]).double())
    B, S = 2, 6
    x = x_of(B, S, 32)
    mask = torch.full((S, S), float("-inf"), dtype=torch.float64).triu(1)[None, None].expand(B, 1, S, S)
    with torch.no_grad():
        ref = layer(torch.from_numpy(x), attention_mask=mask)
    ref = (ref[0] if isinstance(ref, tuple) else ref).numpy()
    got = oracle.bias_unsharded_stack_forward(dims_of(w), [lw], x, np.zeros(B, np.int32), Cache(dims_of(w), B, S))
    assert rel_err(got, ref) < 1e-10


@pytest.mark.parametrize("T", [1, 2, 4])
def test_all_sync_stack_equals_unsharded_stack(T):
    w = work(T=T, L=2)
    layers = [{k: v.float().numpy() for k, v in lw.items()} for lw in si.make_stack(w, "cpu", 2)]
    x = x_of(2, 6, 32, 1)
    d = dims_of(w)
    ref = oracle.bias_unsharded_stack_forward(d, layers, x, np.zeros(2, np.int32), Cache(d, 2, 6))
    got, syncs = oracle.bias_stack_forward(d, [1, 1], layers, x, np.zeros(2, np.int32), Cache(d, 2, 6))
    assert rel_err(got, ref) < 1e-12 and syncs == 4


def test_t1_spd_equals_sync():
    w = work(T=1)
    lw = layer_np(w)
    x = x_of(2, 6, 32, 2)
    d = dims_of(w)
    a, _, _ = oracle.bias_block_forward(d, lw, 0, x, np.zeros(2, np.int32), Cache(d, 2, 6))
    b, _, _ = oracle.bias_block_forward(d, lw, 1, x, np.zeros(2, np.int32), Cache(d, 2, 6))
    assert rel_err(a, b) < 1e-13


@pytest.mark.parametrize("T", [2, 4])
def test_spd_block_closed_form_from_library_primitives(T):
    """out = X + sum_i P_i + b + sum_i fc2_i(relu(fc1_i(LN(X + P_i + b)))) + b_fc2 (Sec. 4.1.2), rebuilt with torch."""
    w = work(T=T)
    lw = layer_np(w)
    x = x_of(2, 6, 32, 3)
    d = dims_of(w)
    out, p, syncs = oracle.bias_block_forward(d, lw, 0, x, np.zeros(2, np.int32), Cache(d, 2, 6))
    assert syncs == 1
    X = torch.from_numpy(x.reshape(12, 32))
    t = {k: torch.from_numpy(v).double() for k, v in lw.items()}
    Fs = 48 // T
    acc = X + t["bo"] + t["b_fc2"]
    for i in range(T):
        Pi = torch.from_numpy(p[i])
        u = torch.nn.functional.layer_norm(X + Pi + t["bo"], (32,), t["mlp_norm"], t["mlp_norm_b"], 1e-5)
        a = torch.relu(u @ t["w_fc1"][i * Fs:(i + 1) * Fs].T + t["b_fc1"][i * Fs:(i + 1) * Fs])
        acc = acc + Pi + a @ t["w_fc2"][:, i * Fs:(i + 1) * Fs].T
    assert rel_err(out.reshape(12, 32), acc.numpy()) < 1e-12
    # the partial products add up to the unsharded out_proj (without its bias) of the sync block
    sync, p2, syncs2 = oracle.bias_block_forward(d, lw, 1, x, np.zeros(2, np.int32), Cache(d, 2, 6))
    assert syncs2 == 2 and np.array_equal(p, p2)
    assert rel_err(out, sync) > 1e-4  # SPD is a different function for T > 1


@pytest.mark.parametrize("T", [2, 4])
def test_rejected_design_of_table_1b_counts_the_bias_t_times(T):
    w = work(T=T)
    lw = layer_np(w)
    x = x_of(2, 6, 32, 4)
    d = dims_of(w)
    spd, _, _ = oracle.bias_block_forward(d, lw, 0, x, np.zeros(2, np.int32), Cache(d, 2, 6))
    rej, _, _ = oracle.bias_block_forward(d, lw, 2, x, np.zeros(2, np.int32), Cache(d, 2, 6))
    assert np.max(np.abs((rej - spd) - (T - 1) * lw["bo"].astype(np.float64))) < 1e-12
    assert rel_err(rej, spd) > 1e-3


def test_spd_equals_sync_when_the_attention_product_vanishes():
    w = work(T=4)
    lw = layer_np(w)
    lw["wo"] = np.zeros_like(lw["wo"])  # P_i = 0: every device sees X + b, as the sync block does
    x = x_of(2, 6, 32, 5)
    d = dims_of(w)
    a, _, _ = oracle.bias_block_forward(d, lw, 0, x, np.zeros(2, np.int32), Cache(d, 2, 6))
    b, _, _ = oracle.bias_block_forward(d, lw, 1, x, np.zeros(2, np.int32), Cache(d, 2, 6))
    assert rel_err(a, b) < 1e-13


def test_decode_steps_reproduce_the_rows_of_a_prefill():
    w = work(T=2, L=2)
    layers = [{k: v.float().numpy() for k, v in lw.items()} for lw in si.make_stack(w, "cpu", 6)]
    d = dims_of(w)
    x = x_of(2, 5, 32, 6)
    full, _ = oracle.bias_stack_forward(d, [0, 1], layers, x, np.zeros(2, np.int32), Cache(d, 2, 5))
    cache = Cache(d, 2, 5)
    for t in range(5):
        step, _ = oracle.bias_stack_forward(d, [0, 1], layers, x[:, t:t + 1], np.full(2, t, np.int32), cache)
        assert rel_err(step[:, 0], full[:, t]) < 1e-12
