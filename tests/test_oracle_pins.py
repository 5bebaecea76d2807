"""Pins of the CPU oracle against things other than itself.

Each test names the statement it checks.  Library routines (the `transformers`
LLaMA decoder layer, torch's attention / RMSNorm / SiLU / linear) stand for the
textbook definitions; invariants come from the paper: TP equals single-device
execution (Sec. 1, Sec. 3), the SPD block's output form X + sum Y_i + sum Z_i with
MLP input X + Y_i (Sec. 4.1.1), the rejected design of Table 1(a), head
re-ordering (Sec. 4.2.4) and the halving of sync-points (Sec. 3).
"""
import itertools

import numpy as np
import pytest
import torch
import torch.nn.functional as Fn

import oracle
from oracle import Cache, Dims

torch.manual_seed(0)


def small_layer(dims: Dims, seed: int, std: float = 0.35):
    g = torch.Generator().manual_seed(seed)
    H, qd, kd, F = dims.hidden, dims.n_q_heads * dims.head_dim, dims.n_kv_heads * dims.head_dim, dims.ffn
    shp = {"wq": (qd, H), "wk": (kd, H), "wv": (kd, H), "wo": (H, qd), "w_gate": (F, H), "w_up": (F, H),
           "w_down": (H, F)}
    lw = {n: (torch.randn(s, generator=g) * std).numpy() for n, s in shp.items()}
    lw["attn_norm"] = (torch.rand(H, generator=g) + 0.5).numpy()
    lw["mlp_norm"] = (torch.rand(H, generator=g) + 0.5).numpy()
    return lw


def rel_err(a, b):
    return float(np.max(np.abs(a - b)) / max(np.max(np.abs(b)), 1e-300))


DIMS_GQA = dict(hidden=32, n_q_heads=8, n_kv_heads=4, head_dim=8, ffn=48)


def x_of(B, S, H, seed=1):
    return torch.randn(B, S, H, generator=torch.Generator().manual_seed(seed), dtype=torch.float64).numpy()


# ---------------------------------------------------------------- primitives

def test_rmsnorm_matches_torch_library():
    x = x_of(1, 7, 40)[0]
    g = np.linspace(0.5, 1.5, 40).astype(np.float32)
    ref = Fn.rms_norm(torch.from_numpy(x), (40,), torch.from_numpy(g).double(), eps=1e-5).numpy()
    assert rel_err(oracle.rmsnorm(x, g, 1e-5), ref) < 1e-14


def test_linear_matches_numpy_matmul():
    rng = np.random.default_rng(0)
    x, w = rng.standard_normal((5, 37)), rng.standard_normal((11, 37)).astype(np.float32)
    assert rel_err(oracle.linear(x, w), x @ w.astype(np.float64).T) < 1e-14


def test_rope_is_a_rotation_by_pos_times_theta():
    d, base = 8, 10000.0
    v = np.arange(1.0, d + 1.0)
    # position 0 is the identity
    assert np.allclose(oracle.rope(v, 0, base), v, rtol=0, atol=0)
    out = oracle.rope(v, 3, base)
    # pair (j, j+d/2) rotated by angle 3 * base^(-2j/d): check through complex multiplication
    for j in range(d // 2):
        z = complex(v[j], v[j + d // 2]) * np.exp(1j * 3 * base ** (-2.0 * j / d))
        assert abs(out[j] - z.real) < 1e-12 and abs(out[j + d // 2] - z.imag) < 1e-12
    # rotations compose: <rope(q,m), rope(k,n)> depends on m-n only
    q, k = np.cos(np.arange(d)), np.sin(np.arange(d) + 0.3)
    a = oracle.rope(q, 9, base) @ oracle.rope(k, 4, base)
    b = oracle.rope(q, 5, base) @ oracle.rope(k, 0, base)
    assert abs(a - b) < 1e-12


def hf_layer(dims: Dims, lw):
    from transformers.models.llama.modeling_llama import LlamaConfig, LlamaDecoderLayer, LlamaRotaryEmbedding
    cfg = LlamaConfig(hidden_size=dims.hidden, intermediate_size=dims.ffn, num_attention_heads=dims.n_q_heads,
                      num_key_value_heads=dims.n_kv_heads, head_dim=dims.head_dim, rms_norm_eps=dims.rms_eps,
                      rope_theta=dims.rope_base, attention_bias=False, mlp_bias=False, num_hidden_layers=1,
                      vocab_size=8)
    cfg._attn_implementation = "sdpa"  # the eager path rounds its softmax to float32
    layer = LlamaDecoderLayer(cfg, 0).double()
    names = {"self_attn.q_proj.weight": "wq", "self_attn.k_proj.weight": "wk", "self_attn.v_proj.weight": "wv",
             "self_attn.o_proj.weight": "wo", "mlp.gate_proj.weight": "w_gate", "mlp.up_proj.weight": "w_up",
             "mlp.down_proj.weight": "w_down", "input_layernorm.weight": "attn_norm",
             "post_attention_layernorm.weight": "mlp_norm"}
    with torch.no_grad():
        for n, p in layer.named_parameters():
            p.copy_(torch.from_numpy(lw[names[n]]).double())
    return layer, LlamaRotaryEmbedding(cfg)


@pytest.mark.parametrize("nq,nkv", [(4, 4), (8, 4), (8, 2)])
def test_unsharded_block_matches_transformers_llama_layer(nq, nkv):
    """The single-device block is the LLaMA-2 decoder layer (library implementation)."""
    dims = Dims(1, 32, nq, nkv, 8, 48, 1)
    lw = small_layer(dims, 3)
    B, S = 2, 6
    x = x_of(B, S, 32)
    layer, rot = hf_layer(dims, lw)
    xt = torch.from_numpy(x)
    pos = torch.arange(S)[None].expand(B, S)
    # the library's rotary module evaluates cos/sin in float32; feed it float64 tables of the
    # same definition (angle = pos * base^(-2j/d), duplicated over both halves) and check them
    cos32, sin32 = rot(xt, pos)
    inv = dims.rope_base ** (-torch.arange(0, dims.head_dim, 2, dtype=torch.float64) / dims.head_dim)
    ang = pos[..., None].double() * inv
    cos, sin = torch.cat([ang, ang], -1).cos(), torch.cat([ang, ang], -1).sin()
    assert torch.allclose(cos, cos32.double(), atol=1e-6) and torch.allclose(sin, sin32.double(), atol=1e-6)
    mask = torch.full((S, S), float("-inf"), dtype=torch.float64).triu(1)[None, None]
    with torch.no_grad():
        ref = layer(xt, attention_mask=mask, position_ids=pos, position_embeddings=(cos, sin)).numpy()
    got = oracle.unsharded_stack_forward(dims, [lw], x, np.zeros(B, np.int32), Cache(dims, B, S))
    # the library layer rounds inside its RMSNorm to float32 whatever the module dtype, hence
    # 1e-6 and not 1e-12; a structural mistake shows at 1e-2 and above
    assert rel_err(got, ref) < 2e-6


def test_attention_with_zero_queries_is_a_running_mean():
    """Closed form: W_Q = 0 makes every causal softmax uniform, so with W_V = W_O = I and
    unit gains the attention branch returns the running mean of the normalised input."""
    H = 16
    dims = Dims(1, H, 2, 2, 8, 4, 1, rope_base=10000.0)
    lw = small_layer(dims, 5)
    lw["wq"][:] = 0
    lw["wv"] = np.eye(H, dtype=np.float32)
    lw["wo"] = np.eye(H, dtype=np.float32)
    lw["attn_norm"][:] = 1
    lw["w_down"][:] = 0  # MLP contributes nothing
    x = x_of(1, 5, H)
    out = oracle.unsharded_stack_forward(dims, [lw], x, np.zeros(1, np.int32), Cache(dims, 1, 5))
    h = x[0] / np.sqrt((x[0] ** 2).mean(-1, keepdims=True) + 1e-5)
    run_mean = np.cumsum(h, 0) / np.arange(1, 6)[:, None]
    assert rel_err(out[0], x[0] + run_mean) < 1e-13


# ---------------------------------------------------------------- TP == single device

@pytest.mark.parametrize("T", [1, 2, 4])
def test_all_sync_stack_equals_unsharded_stack(T):
    """TP keeps parity with single-device execution (Sec. 1, Sec. 3)."""
    dims = Dims(3, T=T, **DIMS_GQA)
    layers = [small_layer(dims, 10 + l) for l in range(3)]
    B, S = 2, 5
    x = x_of(B, S, 32)
    ref = oracle.unsharded_stack_forward(dims, layers, x, np.zeros(B, np.int32), Cache(dims, B, S))
    got, syncs, _ = oracle.stack_forward(dims, [1, 1, 1], layers, x, np.zeros(B, np.int32), Cache(dims, B, S))
    assert rel_err(got, ref) < 1e-12
    assert syncs == 6


def test_t1_spd_equals_sync():
    """One device: there is nothing to drop, X + (Y + Z) = (X + Y) + Z."""
    dims = Dims(2, T=1, **DIMS_GQA)
    layers = [small_layer(dims, 20 + l) for l in range(2)]
    x = x_of(2, 4, 32)
    z = np.zeros(2, np.int32)
    a, _, _ = oracle.stack_forward(dims, [1, 1], layers, x, z, Cache(dims, 2, 4))
    b, _, _ = oracle.stack_forward(dims, [0, 0], layers, x, z, Cache(dims, 2, 4))
    assert rel_err(b, a) < 1e-13


# ---------------------------------------------------------------- the SPD block

def torch_attention_heads(dims: Dims, lw, x):
    """Per-head attention outputs A[B,S,nq,d] from torch library routines only."""
    from transformers.models.llama.modeling_llama import apply_rotary_pos_emb
    B, S, H = x.shape
    d, nq, nkv = dims.head_dim, dims.n_q_heads, dims.n_kv_heads
    xt = torch.from_numpy(x)
    h = Fn.rms_norm(xt, (H,), torch.from_numpy(lw["attn_norm"]).double(), eps=dims.rms_eps)
    q = Fn.linear(h, torch.from_numpy(lw["wq"]).double()).view(B, S, nq, d).transpose(1, 2)
    k = Fn.linear(h, torch.from_numpy(lw["wk"]).double()).view(B, S, nkv, d).transpose(1, 2)
    v = Fn.linear(h, torch.from_numpy(lw["wv"]).double()).view(B, S, nkv, d).transpose(1, 2)
    inv = dims.rope_base ** (-torch.arange(0, d, 2, dtype=torch.float64) / d)
    ang = torch.arange(S, dtype=torch.float64)[:, None] * inv[None]
    emb = torch.cat([ang, ang], -1)[None]
    q, k = apply_rotary_pos_emb(q, k, emb.cos(), emb.sin())
    k = k.repeat_interleave(nq // nkv, 1)
    v = v.repeat_interleave(nq // nkv, 1)
    a = Fn.scaled_dot_product_attention(q, k, v, is_causal=True)
    return a.transpose(1, 2)  # [B,S,nq,d]


@pytest.mark.parametrize("T", [2, 4])
def test_spd_block_closed_form_from_library_primitives(T):
    """Sec. 4.1.1: out = X + sum_i Y_i + sum_i Z_i with Z_i = MLP_i(norm(X + Y_i)),
    Y_i = (heads of device i) x (their rows of W_O^T)."""
    dims = Dims(1, T=T, **DIMS_GQA)
    lw = small_layer(dims, 31)
    B, S, H, d = 2, 5, 32, 8
    x = x_of(B, S, H)
    A = torch_attention_heads(dims, lw, x)
    wo = torch.from_numpy(lw["wo"]).double()
    wg, wu, wd = (torch.from_numpy(lw[n]).double() for n in ("w_gate", "w_up", "w_down"))
    gm = torch.from_numpy(lw["mlp_norm"]).double()
    qh, Fs = dims.n_q_heads // T, dims.ffn // T
    xt = torch.from_numpy(x)
    total = xt.clone()
    ys = []
    for i in range(T):
        Ai = A[:, :, i * qh:(i + 1) * qh].reshape(B, S, qh * d)
        Yi = Ai @ wo[:, i * qh * d:(i + 1) * qh * d].T
        ui = Fn.rms_norm(xt + Yi, (H,), gm, eps=dims.rms_eps)
        Zi = (Fn.silu(ui @ wg[i * Fs:(i + 1) * Fs].T) * (ui @ wu[i * Fs:(i + 1) * Fs].T)) @ wd[:, i * Fs:(i + 1) * Fs].T
        total = total + Yi + Zi
        ys.append(Yi.reshape(B * S, H).numpy())
    out, y, syncs = oracle.block_forward(dims, lw, 0, x, np.zeros(B, np.int32), Cache(dims, B, S))
    assert syncs == 1
    assert rel_err(out, total.numpy()) < 1e-12
    assert rel_err(y, np.stack(ys)) < 1e-12


def test_spd_equals_sync_when_attention_output_vanishes():
    """W_O = 0: every Y_i = 0, all devices feed X to the MLP, nothing was dropped."""
    dims = Dims(1, T=4, **DIMS_GQA)
    lw = small_layer(dims, 40)
    lw["wo"][:] = 0
    x = x_of(1, 4, 32)
    z = np.zeros(1, np.int32)
    a, _, _ = oracle.block_forward(dims, lw, 1, x, z, Cache(dims, 1, 4))
    b, _, _ = oracle.block_forward(dims, lw, 0, x, z, Cache(dims, 1, 4))
    assert rel_err(b, a) < 1e-13


def test_spd_equals_sync_when_one_device_holds_everything():
    """Only device 1 has a non-zero W_O slice and a non-zero W_D slice: the devices whose
    MLP input lacks Y_1 contribute Z_i = 0, so SPD reproduces the synchronous block.
    (Catches a device feeding some other device's Y into its MLP.)"""
    dims = Dims(1, T=4, **DIMS_GQA)
    lw = small_layer(dims, 41)
    qd, Fs = (8 // 4) * 8, 48 // 4
    keep = lw["wo"][:, qd:2 * qd].copy()
    lw["wo"][:] = 0
    lw["wo"][:, qd:2 * qd] = keep
    keep = lw["w_down"][:, Fs:2 * Fs].copy()
    lw["w_down"][:] = 0
    lw["w_down"][:, Fs:2 * Fs] = keep
    x = x_of(2, 3, 32)
    z = np.zeros(2, np.int32)
    a, _, _ = oracle.block_forward(dims, lw, 1, x, z, Cache(dims, 2, 3))
    b, _, _ = oracle.block_forward(dims, lw, 0, x, z, Cache(dims, 2, 3))
    assert rel_err(b, a) < 1e-13


def permute_heads(lw, dims: Dims, perm_q, perm_kv):
    """Head re-ordering of Sec. 4.2.4: rows of W_Q/W_K/W_V and the matching columns of W_O."""
    d = dims.head_dim
    out = {k: v.copy() for k, v in lw.items()}
    rq = np.concatenate([np.arange(h * d, (h + 1) * d) for h in perm_q])
    rk = np.concatenate([np.arange(h * d, (h + 1) * d) for h in perm_kv])
    out["wq"] = lw["wq"][rq]
    out["wo"] = lw["wo"][:, rq]
    out["wk"] = lw["wk"][rk]
    out["wv"] = lw["wv"][rk]
    return out


def test_head_regrouping_keeps_sync_and_changes_spd():
    """Moving heads between devices is invisible to the synchronous block and visible to SPD."""
    dims = Dims(1, 32, 4, 4, 8, 48, 2)
    lw = small_layer(dims, 50)
    lw2 = permute_heads(lw, dims, [0, 2, 1, 3], [0, 2, 1, 3])  # swap a head across the two devices
    x = x_of(1, 5, 32)
    z = np.zeros(1, np.int32)
    s1, _, _ = oracle.block_forward(dims, lw, 1, x, z, Cache(dims, 1, 5))
    s2, _, _ = oracle.block_forward(dims, lw2, 1, x, z, Cache(dims, 1, 5))
    p1, _, _ = oracle.block_forward(dims, lw, 0, x, z, Cache(dims, 1, 5))
    p2, _, _ = oracle.block_forward(dims, lw2, 0, x, z, Cache(dims, 1, 5))
    assert rel_err(s2, s1) < 1e-13
    assert rel_err(p2, p1) > 1e-3


def test_ffn_column_regrouping_keeps_sync_and_changes_spd():
    dims = Dims(1, 32, 4, 4, 8, 48, 2)
    lw = small_layer(dims, 51)
    perm = np.arange(48)
    perm[[3, 30]] = perm[[30, 3]]  # one FFN unit changes device
    lw2 = {k: v.copy() for k, v in lw.items()}
    lw2["w_gate"], lw2["w_up"], lw2["w_down"] = lw["w_gate"][perm], lw["w_up"][perm], lw["w_down"][:, perm]
    x = x_of(1, 5, 32)
    z = np.zeros(1, np.int32)
    s1, _, _ = oracle.block_forward(dims, lw, 1, x, z, Cache(dims, 1, 5))
    s2, _, _ = oracle.block_forward(dims, lw2, 1, x, z, Cache(dims, 1, 5))
    p1, _, _ = oracle.block_forward(dims, lw, 0, x, z, Cache(dims, 1, 5))
    p2, _, _ = oracle.block_forward(dims, lw2, 0, x, z, Cache(dims, 1, 5))
    assert rel_err(s2, s1) < 1e-13
    assert rel_err(p2, p1) > 1e-4


def test_whole_device_permutation_leaves_spd_unchanged():
    """Devices are independent mini-blocks until the final sum (Sec. 4.2.4): renumbering
    devices (heads and MLP slice together) changes nothing."""
    dims = Dims(1, 32, 4, 4, 8, 48, 2)
    lw = small_layer(dims, 52)
    lw2 = permute_heads(lw, dims, [2, 3, 0, 1], [2, 3, 0, 1])
    perm = np.concatenate([np.arange(24, 48), np.arange(0, 24)])
    lw2["w_gate"], lw2["w_up"], lw2["w_down"] = lw2["w_gate"][perm], lw2["w_up"][perm], lw2["w_down"][:, perm]
    x = x_of(2, 4, 32)
    z = np.zeros(2, np.int32)
    p1, y1, _ = oracle.block_forward(dims, lw, 0, x, z, Cache(dims, 2, 4))
    p2, y2, _ = oracle.block_forward(dims, lw2, 0, x, z, Cache(dims, 2, 4))
    assert rel_err(p2, p1) < 1e-13
    assert rel_err(y2[::-1], y1) < 1e-13


def test_rejected_design_of_table_1a_differs():
    """Adding Y_i after the MLP all-reduce leaves each device with a different output that
    lacks the other devices' Y: it must differ from the shipped design, and the mean over
    devices of its outputs relates to it by  out - mean_i(var_i) = (1 - 1/T) sum_i Y_i."""
    T = 4
    dims = Dims(1, T=T, **DIMS_GQA)
    lw = small_layer(dims, 60)
    x = x_of(1, 5, 32)
    z = np.zeros(1, np.int32)
    good, y, _ = oracle.block_forward(dims, lw, 0, x, z, Cache(dims, 1, 5))
    bad, _, _ = oracle.block_forward(dims, lw, 2, x, z, Cache(dims, 1, 5))
    assert bad.shape == (T, 1, 5, 32)
    for i in range(T):
        assert rel_err(bad[i], good) > 1e-3
    for i, j in itertools.combinations(range(T), 2):
        assert rel_err(bad[i], bad[j]) > 1e-3
    ysum = y.sum(0).reshape(1, 5, 32)
    assert rel_err(good - bad.mean(0), (1 - 1 / T) * ysum) < 1e-12


def test_sync_point_count_follows_the_mask():
    """A sync block has two shard sums, an SPD block one; all-SPD halves the total (Sec. 3)."""
    dims = Dims(4, T=2, **DIMS_GQA)
    layers = [small_layer(dims, 70 + l) for l in range(4)]
    x = x_of(1, 3, 32)
    z = np.zeros(1, np.int32)
    counts = {}
    for mask in ([1, 1, 1, 1], [0, 0, 0, 0], [1, 0, 0, 1]):
        _, n, _ = oracle.stack_forward(dims, mask, layers, x, z, Cache(dims, 1, 3))
        counts[tuple(mask)] = n
    assert counts[(1, 1, 1, 1)] == 8 and counts[(0, 0, 0, 0)] == 4 and counts[(1, 0, 0, 1)] == 6


def test_mask_is_honoured_per_layer():
    dims = Dims(2, T=2, **DIMS_GQA)
    layers = [small_layer(dims, 80 + l) for l in range(2)]
    x = x_of(1, 4, 32)
    z = np.zeros(1, np.int32)
    outs = {m: oracle.stack_forward(dims, list(m), layers, x, z, Cache(dims, 1, 4), True) for m in
            [(1, 1), (1, 0), (0, 1), (0, 0)]}
    # first layer output depends on mask[0] only
    assert rel_err(outs[(1, 0)][2][0], outs[(1, 1)][2][0]) == 0
    assert rel_err(outs[(0, 1)][2][0], outs[(1, 1)][2][0]) > 1e-3
    finals = [outs[m][0] for m in outs]
    for a, b in itertools.combinations(finals, 2):
        assert rel_err(a, b) > 1e-4


def test_layer_streamed_stack_is_the_stack():
    """Feeding the blocks one layer at a time (deep, wide stacks whose weights do not fit in host
    memory at once) is the same chain of blocks: outputs, per-layer outputs, caches and the
    sync-point count are bit-identical to the whole-stack routine, prompt and decode step alike."""
    dims = Dims(5, T=4, **DIMS_GQA)
    layers = [small_layer(dims, 60 + l) for l in range(5)]
    mask = [1, 0, 0, 1, 0]
    B, S = 2, 5
    x, x1 = x_of(B, S, 32), x_of(B, 1, 32, seed=3)
    ca, cb = Cache(dims, B, S + 1), Cache(dims, B, S + 1)
    asked = []

    def source(l):
        asked.append(l)
        return layers[l]

    z = np.zeros(B, np.int32)
    a = oracle.stack_forward(dims, mask, layers, x, z, ca, True)
    b = oracle.stack_forward_streamed(dims, mask, source, x, z, cb, True)
    assert asked == [0, 1, 2, 3, 4]
    assert np.array_equal(a[0], b[0]) and a[1] == b[1] == 7 and np.array_equal(a[2], b[2])
    a1 = oracle.stack_forward(dims, mask, layers, x1, np.full(B, S, np.int32), ca)
    b1 = oracle.stack_forward_streamed(dims, mask, source, x1, np.full(B, S, np.int32), cb)
    assert np.array_equal(a1[0], b1[0]) and np.array_equal(ca.k, cb.k) and np.array_equal(ca.v, cb.v)


# ---------------------------------------------------------------- cache consistency

@pytest.mark.parametrize("mask", [[1, 1], [0, 0], [0, 1]])
def test_decode_steps_reproduce_the_rows_of_a_prefill(mask):
    """Causality: processing tokens one at a time against the cache gives the same rows as
    processing them together."""
    dims = Dims(2, T=2, **DIMS_GQA)
    layers = [small_layer(dims, 90 + l) for l in range(2)]
    B, S = 2, 6
    x = x_of(B, S, 32)
    full, _, _ = oracle.stack_forward(dims, mask, layers, x, np.zeros(B, np.int32), Cache(dims, B, S))
    cache = Cache(dims, B, S)
    first, _, _ = oracle.stack_forward(dims, mask, layers, x[:, :3], np.zeros(B, np.int32), cache)
    assert rel_err(first, full[:, :3]) < 1e-13
    for t in range(3, S):
        step, _, _ = oracle.stack_forward(dims, mask, layers, x[:, t:t + 1], np.full(B, t, np.int32), cache)
        assert rel_err(step, full[:, t:t + 1]) < 1e-12


def test_sequences_in_a_batch_are_independent_and_ragged_positions_work():
    dims = Dims(1, T=2, **DIMS_GQA)
    lw = small_layer(dims, 95)
    x = x_of(2, 4, 32)
    both, _, _ = oracle.stack_forward(dims, [0], [lw], x, np.zeros(2, np.int32), Cache(dims, 2, 4))
    for b in range(2):
        one, _, _ = oracle.stack_forward(dims, [0], [lw], x[b:b + 1], np.zeros(1, np.int32), Cache(dims, 1, 4))
        assert rel_err(one, both[b:b + 1]) < 1e-13
    # ragged: sequence 0 has 3 cached tokens, sequence 1 has 1
    cache = Cache(dims, 2, 8)
    oracle.stack_forward(dims, [0], [lw], x[:, :1], np.zeros(2, np.int32), cache)
    c0 = Cache(dims, 1, 8)
    oracle.stack_forward(dims, [0], [lw], x[:1, :3], np.zeros(1, np.int32), c0)
    cache.k[:, 0], cache.v[:, 0] = c0.k[:, 0], c0.v[:, 0]
    xn = x_of(2, 1, 32, seed=7)
    step, _, _ = oracle.stack_forward(dims, [0], [lw], xn, np.array([3, 1], np.int32), cache)
    ref0, _, _ = oracle.stack_forward(dims, [0], [lw], np.concatenate([x[:1, :3], xn[:1]], 1),
                                      np.zeros(1, np.int32), Cache(dims, 1, 8))
    ref1, _, _ = oracle.stack_forward(dims, [0], [lw], np.concatenate([x[1:, :1], xn[1:]], 1),
                                      np.zeros(1, np.int32), Cache(dims, 1, 8))
    assert rel_err(step[0], ref0[0, 3:]) < 1e-12
    assert rel_err(step[1], ref1[0, 1:]) < 1e-12


def test_bad_dims_are_rejected():
    with pytest.raises(ValueError):
        dims = Dims(1, 32, 6, 3, 8, 48, 4)  # 6 heads over 4 devices
        oracle.stack_forward(dims, [0], [small_layer(dims, 1)], x_of(1, 2, 32), np.zeros(1, np.int32), Cache(dims, 1, 2))
