"""Shared plumbing of the GPU parity tests: run the CUDA library and the CPU oracle on the
same seeded inputs and compare.  No arithmetic of the method lives here."""
from __future__ import annotations

import numpy as np
import torch

import oracle
import spd_inputs as si

TOL = {"fp32": 1e-4, "bf16": 2e-2}


def stack_tol(dtype: str, depth: int) -> float:
    """Bound on the output of `depth` blocks run one after the other on their own outputs.  The stated
    tolerances are those of a block's output.  Behind one another the blocks' rounding errors (each at most
    TOL, independent of each other) travel down the residual stream and add in quadrature: TOL * sqrt(depth).
    (Measured at the 70B shape: 0.4-0.8e-2 per block fed with the oracle's input at every depth, 2.8e-2 after
    eight blocks on their own outputs - about 1e-2 * sqrt(depth).)"""
    return TOL[dtype] * float(np.sqrt(depth))
_STREAM = None


def rel_err(got, ref) -> float:
    """max |got - ref| / max |ref| over the tensor: the bound the tolerances are stated on."""
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    return float(np.max(np.abs(got - ref)) / max(float(np.max(np.abs(ref))), 1e-30))


def oracle_dims(w: si.Workload) -> oracle.Dims:
    return oracle.Dims(w.n_layers, w.hidden, w.n_q_heads, w.n_kv_heads, w.head_dim, w.ffn, w.T, w.rms_eps,
                       w.rope_base)


def to_np(t: torch.Tensor) -> np.ndarray:
    return t.detach().to("cpu", torch.float64).numpy()


class Pair:
    """One workload instantiated on both sides."""

    def __init__(self, w: si.Workload, *, mask=None, B=None, max_len=None, max_prefill_tokens=None, seed=0,
                 device="cuda:0", n_pages=None, layers=None, weights_on="cpu", stream_oracle=False):
        """weights_on: where the seeded generator of ``spd_inputs`` draws the weights ("cpu", or the CUDA
        device for wide layers: torch's device generator, seconds instead of minutes per 70B-shaped layer).
        stream_oracle: the oracle gets the layers one at a time (up-cast copies of one layer in host memory
        instead of the whole stack)."""
        import paper_2502_20727_b200 as spd
        # a non-default stream: the legacy default stream cannot be captured into the graphs
        # that replay decode steps
        global _STREAM
        if _STREAM is None:
            _STREAM = torch.cuda.Stream(device=device)
        torch.cuda.set_stream(_STREAM)
        self.w = w
        self.B = B or w.batch
        self.max_len = max_len or (w.prompt + w.decode_steps)
        self.mask = list(w.mask if mask is None else mask)
        self.device = device
        self.layers = layers if layers is not None else si.make_stack(w, weights_on, seed)
        self.layers_gpu = [{n: t.to(device) for n, t in lw.items()} for lw in self.layers]
        self.layers_np = None if stream_oracle else si.to_oracle_layers(self.layers)
        self.layer_out = None  # the oracle's per-layer outputs of the last call made with want_layers
        self.dims = oracle_dims(w)
        self.cache = oracle.Cache(self.dims, self.B, self.max_len)
        pages_per_seq = (self.max_len + w.kv_block - 1) // w.kv_block
        self.n_pages = n_pages or (self.B * pages_per_seq + 3)
        self.block_table = si.make_block_table(self.B, pages_per_seq, self.n_pages, seed).to(device)
        self.stack = spd.stack_from_workload(w, self.layers_gpu, sync_mask=self.mask, max_batch=self.B,
                                             max_seq_len=self.max_len, n_pages=self.n_pages,
                                             max_prefill_tokens=max_prefill_tokens or 4096, device=device)
        self.pos = np.zeros(self.B, dtype=np.int32)

    def _oracle(self, x, want_layers=False):
        """The oracle's forward pass of the workload's block kind: (out, sync_points)."""
        if getattr(self.w, "block", "llama") == "opt":
            return oracle.bias_stack_forward(self.dims, self.mask, self.layers_np, x, self.pos, self.cache)
        if self.layers_np is None:
            out, syncs, self.layer_out = oracle.stack_forward_streamed(
                self.dims, self.mask, lambda l: si.to_oracle_layers([self.layers[l]])[0], x, self.pos, self.cache, want_layers)
        else:
            out, syncs, self.layer_out = oracle.stack_forward(self.dims, self.mask, self.layers_np, x, self.pos, self.cache,
                                                              want_layers)
        return out, syncs

    def prefill(self, S, seed=0, want_layers=False):
        x = si.make_hidden(self.w, (self.B, S, self.w.hidden), "cpu", seed, 0)
        ref, syncs = self._oracle(to_np(x), want_layers)
        got = self.stack.prefill(x.to(self.device), self.block_table)
        torch.cuda.synchronize()
        self.pos = self.pos + S
        return to_np(got), ref, syncs

    def decode(self, t, seed=0):
        x = si.make_hidden(self.w, (self.B, self.w.hidden), "cpu", seed, 1 + t)
        ref, _ = self._oracle(to_np(x)[:, None, :])
        # fixed device buffers, as a serving loop has them: after the first step the library
        # replays its captured graph, so both the capture and the replay path are compared
        if not hasattr(self, "x_dev"):
            self.x_dev = torch.empty((self.B, self.w.hidden), dtype=self.w.torch_dtype, device=self.device)
            self.seq_dev = torch.empty(self.B, dtype=torch.int32, device=self.device)
            self.out_dev = torch.empty_like(self.x_dev)
        self.x_dev.copy_(x)
        self.seq_dev.copy_(torch.from_numpy(self.pos.copy()))
        got = self.stack.decode_step(self.x_dev, self.seq_dev, self.block_table, int(self.pos.max()) + 1, self.out_dev)
        torch.cuda.synchronize()
        self.pos = self.pos + 1
        return to_np(got), ref[:, 0, :]

    def prefix_prefill(self, depth, S, seed=0):
        """The GPU's output after the first `depth` blocks for the prompts of prefill(S, seed): a second context
        over the same weight tensors and block table with pages of its own (compare with layer_out[depth - 1])."""
        import paper_2502_20727_b200 as spd
        w = self.w.with_(n_layers=depth, mask=tuple(self.mask[:depth]))
        st = spd.stack_from_workload(w, self.layers_gpu[:depth], sync_mask=self.mask[:depth], max_batch=self.B,
                                     max_seq_len=self.max_len, n_pages=self.n_pages, max_prefill_tokens=self.B * S,
                                     device=self.device)
        x = si.make_hidden(self.w, (self.B, S, self.w.hidden), "cpu", seed, 0)
        got = st.prefill(x.to(self.device), self.block_table)
        torch.cuda.synchronize()
        err = st.device_error()
        st.close()
        assert err == 0
        return to_np(got).reshape(self.B * S, self.w.hidden)

    def block_prefill(self, l, x_in, S):
        """Block l alone on the GPU, fed with x_in [B*S, H] (the oracle's input of that block, rounded to the storage
        dtype): its output [B*S, H] - the comparison that the per-block tolerance is stated for, at any depth."""
        import paper_2502_20727_b200 as spd
        w = self.w.with_(n_layers=1, mask=(self.mask[l],))
        st = spd.stack_from_workload(w, self.layers_gpu[l:l + 1], sync_mask=[self.mask[l]], max_batch=self.B,
                                     max_seq_len=self.max_len, n_pages=self.n_pages, max_prefill_tokens=self.B * S,
                                     device=self.device)
        x = torch.from_numpy(np.ascontiguousarray(x_in).reshape(self.B, S, self.w.hidden)).to(self.w.torch_dtype).to(self.device)
        got = st.prefill(x, self.block_table)
        torch.cuda.synchronize()
        err = st.device_error()
        st.close()
        assert err == 0
        return to_np(got).reshape(self.B * S, self.w.hidden)

    def tp_prefill(self, S, seed=0):
        """Prompts in rank mode: every rank's output [T, B, S, H] and the oracle's."""
        x = si.make_hidden(self.w, (self.B, S, self.w.hidden), "cpu", seed, 0)
        ref, syncs = self._oracle(to_np(x))
        got = self.stack.tp_prefill(x.to(self.device), self.block_table)
        torch.cuda.synchronize()
        self.pos = self.pos + S
        return to_np(got), ref, syncs

    def tp_decode(self, t, seed=0):
        """One decode step in rank mode (the stack attached as all T ranks of a group on this GPU):
        every rank's output [T, B, H] and the oracle's."""
        x = si.make_hidden(self.w, (self.B, self.w.hidden), "cpu", seed, 1 + t)
        ref, _ = self._oracle(to_np(x)[:, None, :])
        # fixed device buffers: later steps replay the captured graphs (one per receive-buffer phase)
        if not hasattr(self, "tp_x"):
            self.tp_x = torch.empty((self.B, self.w.hidden), dtype=self.w.torch_dtype, device=self.device)
            self.tp_seq = torch.empty(self.B, dtype=torch.int32, device=self.device)
            self.tp_out = torch.empty((self.w.T, self.B, self.w.hidden), dtype=self.w.torch_dtype, device=self.device)
        self.tp_x.copy_(x)
        self.tp_seq.copy_(torch.from_numpy(self.pos.copy()))
        got = self.stack.tp_decode_step(self.tp_x, self.tp_seq, self.block_table, int(self.pos.max()) + 1, self.tp_out)
        torch.cuda.synchronize()
        self.pos = self.pos + 1
        return to_np(got), ref[:, 0, :]

    def fill_cache(self, lens, seed=0):
        """Put the same synthetic K/V (N(0,1), storage dtype) into the GPU pages and the oracle's
        cache for positions [0, lens[b]) of every sequence and layer."""
        w = self.w
        bs, kvw = w.kv_block, w.n_kv_heads * w.head_dim
        bt = self.block_table.cpu().numpy()
        for l in range(w.n_layers):
            for which, pages in (("k", self.stack.k_pages[l]), ("v", self.stack.v_pages[l])):
                fill = si.make_kv_fill(w, (self.B, self.max_len, w.n_kv_heads, w.head_dim), "cpu", seed,
                                       2 * l + (which == "v"))
                host_pages = torch.zeros(pages.shape, dtype=pages.dtype)
                for b in range(self.B):
                    n = int(lens[b])
                    getattr(self.cache, which)[l, b, :n] = to_np(fill[b, :n]).reshape(n, kvw)
                    for j in range((n + bs - 1) // bs):
                        cnt = min(bs, n - j * bs)
                        host_pages[bt[b, j], :, :cnt] = fill[b, j * bs:j * bs + cnt].transpose(0, 1)
                pages.copy_(host_pages)
        self.pos = np.asarray(lens, dtype=np.int32).copy()

    def gpu_cache(self, layer, which, b, n):
        """K or V of sequence b, positions [0, n), gathered from the GPU pages -> [n, nkv*d]."""
        w = self.w
        pages = (self.stack.k_pages if which == "k" else self.stack.v_pages)[layer].cpu()
        bt = self.block_table.cpu().numpy()
        rows = [pages[bt[b, t // w.kv_block], :, t % w.kv_block, :].reshape(-1) for t in range(n)]
        return to_np(torch.stack(rows))
