"""Seeded synthetic inputs shared by the CPU oracle's tests and the CUDA path.

This module only DRAWS numbers and describes workloads; it contains none of the
method's arithmetic.  The workloads take the shapes of the LLaMA-2 models the
paper evaluates (Sec. 5.1); weights and activations are random because neither
the checkpoints nor the calibration text are available.

Recipe (per layer l, generator seeded with ``seed * 1000003 + l``; draws in the
order below):
  wq, wk, wv, wo, w_gate, w_up, w_down ~ N(0, 0.02^2)
  attn_norm, mlp_norm                  ~ U(0.5, 1.5)
Hidden states (prompt and per-step decode inputs) ~ N(0, 1).
For bf16 workloads every tensor is rounded to bf16 once, here, so both sides
read identical values.
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import Dict, List, Sequence, Tuple

import numpy as np
import torch

WEIGHT_NAMES = ("attn_norm", "wq", "wk", "wv", "wo", "mlp_norm", "w_gate", "w_up", "w_down")


@dataclass(frozen=True)
class Workload:
    name: str
    dtype: str              # "fp32" | "bf16"  (storage type of weights / activations / KV)
    n_layers: int
    hidden: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    ffn: int
    T: int
    mask: Tuple[int, ...]   # per layer, 1 = sync (TP block), 0 = SPD block
    batch: int
    prompt: int
    decode_steps: int
    rms_eps: float = 1e-5
    rope_base: float = 10000.0
    kv_block: int = 16
    block: str = "llama"    # "llama": RMSNorm / rotary / SwiGLU, no bias; "opt": LayerNorm / biases / ReLU (Sec. 4.1.2)
    prefill_batch: int = 0  # prompts of the prefill measurement when they differ from the decode batch (0: batch x prompt)
    prefill_len: int = 0

    @property
    def torch_dtype(self):
        return torch.float32 if self.dtype == "fp32" else torch.bfloat16

    def with_(self, **kw) -> "Workload":
        w = replace(self, **kw)
        if len(w.mask) != w.n_layers:
            w = replace(w, mask=tuple(w.mask[: w.n_layers]) + (0,) * max(0, w.n_layers - len(w.mask)))
        return w

    def shape_of(self, name: str) -> Tuple[int, ...]:
        H, qd, kd, F = self.hidden, self.n_q_heads * self.head_dim, self.n_kv_heads * self.head_dim, self.ffn
        return {"attn_norm": (H,), "mlp_norm": (H,), "wq": (qd, H), "wk": (kd, H), "wv": (kd, H),
                "wo": (H, qd), "w_gate": (F, H), "w_up": (F, H), "w_down": (H, F)}[name]

    def params_per_layer(self) -> int:
        if self.block == "opt":
            H, qd, kd, F = self.hidden, self.n_q_heads * self.head_dim, self.n_kv_heads * self.head_dim, self.ffn
            return qd * H + 2 * kd * H + H * qd + 2 * F * H + (qd + 2 * kd + H + F + H) + 4 * H
        return sum(int(np.prod(self.shape_of(n))) for n in WEIGHT_NAMES)


def c5_mask(n_layers: int = 40, n_sync: int = 10, seed: int = 0) -> Tuple[int, ...]:
    """25 % sync blocks at seeded random positions, the rest SPD."""
    pos = np.sort(np.random.default_rng(seed).permutation(n_layers)[:n_sync])
    m = np.zeros(n_layers, dtype=np.int64)
    m[pos] = 1
    return tuple(int(v) for v in m)


WORKLOADS: Dict[str, Workload] = {
    "c1": Workload("c1", "fp32", 1, 256, 4, 4, 64, 688, 2, (0,), 1, 16, 8),
    "c2": Workload("c2", "bf16", 4, 4096, 32, 32, 128, 11008, 8, (0,) * 4, 8, 512, 128),
    "c3_t4": Workload("c3_t4", "bf16", 8, 5120, 40, 40, 128, 13824, 4, (1, 0, 0, 0, 0, 0, 0, 1), 16, 1024, 256),
    "c3_t8": Workload("c3_t8", "bf16", 8, 5120, 40, 40, 128, 13824, 8, (1, 0, 0, 0, 0, 0, 0, 1), 16, 1024, 256),
    "c4_b1": Workload("c4_b1", "bf16", 8, 8192, 64, 8, 128, 28672, 8, (0,) * 8, 1, 2048, 256),
    "c4_b32": Workload("c4_b32", "bf16", 8, 8192, 64, 8, 128, 28672, 8, (0,) * 8, 32, 2048, 256),
    # prefill of 4 x 4096 tokens; decode of batch 64 for 512 steps on caches pre-filled to 512 tokens
    "c5": Workload("c5", "bf16", 40, 8192, 64, 8, 128, 28672, 8, c5_mask(), 64, 512, 512, prefill_batch=4, prefill_len=4096),
    # the block with bias (Sec. 4.1.2) at OPT-6.7B's shape (Sec. 5.1): 4 layers, hidden 4096, 32 heads x 128, ffn 16384
    "opt67": Workload("opt67", "bf16", 4, 4096, 32, 32, 128, 16384, 8, (0,) * 4, 8, 512, 128, block="opt"),
}


def _gen(device, seed: int) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def make_layer(w: Workload, layer: int, device="cpu", seed: int = 0) -> Dict[str, torch.Tensor]:
    """Weights of one layer in the workload's storage dtype, torch.nn.Linear layout [out, in]."""
    g = _gen(device, seed * 1000003 + layer)
    out: Dict[str, torch.Tensor] = {}
    for n in ("wq", "wk", "wv", "wo", "w_gate", "w_up", "w_down"):
        t = torch.randn(w.shape_of(n), generator=g, device=device, dtype=torch.float32) * 0.02
        out[n] = t.to(w.torch_dtype).contiguous()
    for n in ("attn_norm", "mlp_norm"):
        t = torch.rand(w.shape_of(n), generator=g, device=device, dtype=torch.float32) + 0.5
        out[n] = t.to(w.torch_dtype).contiguous()
    return out


BIAS_WEIGHT_NAMES = ("attn_norm", "attn_norm_b", "wq", "bq", "wk", "bk", "wv", "bv", "wo", "bo", "mlp_norm", "mlp_norm_b",
                     "w_fc1", "b_fc1", "w_fc2", "b_fc2")


def make_bias_layer(w: Workload, layer: int, device="cpu", seed: int = 0) -> Dict[str, torch.Tensor]:
    """One OPT-style layer (shapes of the OPT models of Sec. 5.1): matrices ~ N(0, 0.02^2), biases and
    LayerNorm shifts ~ N(0, 0.1^2) (large enough that a misplaced bias shows), LayerNorm gains ~ U(0.5, 1.5).
    Draw order: wq, wk, wv, wo, w_fc1, w_fc2, then bq, bk, bv, bo, b_fc1, b_fc2, attn_norm_b, mlp_norm_b, then the gains."""
    g = _gen(device, seed * 1000003 + layer + 500009)
    H, qd, kd, F = w.hidden, w.n_q_heads * w.head_dim, w.n_kv_heads * w.head_dim, w.ffn
    shapes = {"wq": (qd, H), "wk": (kd, H), "wv": (kd, H), "wo": (H, qd), "w_fc1": (F, H), "w_fc2": (H, F),
              "bq": (qd,), "bk": (kd,), "bv": (kd,), "bo": (H,), "b_fc1": (F,), "b_fc2": (H,), "attn_norm_b": (H,), "mlp_norm_b": (H,)}
    out: Dict[str, torch.Tensor] = {}
    for n in ("wq", "wk", "wv", "wo", "w_fc1", "w_fc2"):
        out[n] = (torch.randn(shapes[n], generator=g, device=device, dtype=torch.float32) * 0.02).to(w.torch_dtype).contiguous()
    for n in ("bq", "bk", "bv", "bo", "b_fc1", "b_fc2", "attn_norm_b", "mlp_norm_b"):
        out[n] = (torch.randn(shapes[n], generator=g, device=device, dtype=torch.float32) * 0.1).to(w.torch_dtype).contiguous()
    for n in ("attn_norm", "mlp_norm"):
        out[n] = (torch.rand((H,), generator=g, device=device, dtype=torch.float32) + 0.5).to(w.torch_dtype).contiguous()
    return out


def make_stack(w: Workload, device="cpu", seed: int = 0) -> List[Dict[str, torch.Tensor]]:
    if w.block == "opt":
        return [make_bias_layer(w, l, device, seed) for l in range(w.n_layers)]
    return [make_layer(w, l, device, seed) for l in range(w.n_layers)]


def make_hidden(w: Workload, shape: Sequence[int], device="cpu", seed: int = 0, stream: int = 0) -> torch.Tensor:
    """N(0,1) hidden states; ``stream`` separates the prompt (0) from decode step t (1 + t)."""
    g = _gen(device, seed * 7919 + 104729 * (stream + 1))
    return torch.randn(tuple(shape), generator=g, device=device, dtype=torch.float32).to(w.torch_dtype)


def make_kv_fill(w: Workload, shape: Sequence[int], device="cpu", seed: int = 0, stream: int = 0) -> torch.Tensor:
    """N(0,1) stand-in cache contents for tests that start a decode step at a long context
    without paying for the prefill in the oracle."""
    g = _gen(device, seed * 613 + 15485863 * (stream + 1))
    return torch.randn(tuple(shape), generator=g, device=device, dtype=torch.float32).to(w.torch_dtype)


def make_block_table(batch: int, pages_per_seq: int, n_pages: int, seed: int = 0) -> torch.Tensor:
    """int32 [batch, pages_per_seq]: a seeded random permutation of page ids, so that the
    pages of a sequence are scattered (non-contiguous on purpose)."""
    assert batch * pages_per_seq <= n_pages
    perm = np.random.default_rng(seed + 17).permutation(n_pages)[: batch * pages_per_seq]
    return torch.from_numpy(perm.astype(np.int32).reshape(batch, pages_per_seq))


def to_oracle_layers(layers: List[Dict[str, torch.Tensor]]) -> List[Dict[str, np.ndarray]]:
    """Up-cast stored weights to float32 numpy for the oracle (exact for bf16 and fp32)."""
    return [{n: t.detach().to("cpu", torch.float32).numpy() for n, t in lw.items()} for lw in layers]
