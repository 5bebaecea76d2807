"""Thin Python binding of the SPD block library (``include/spd.h``).

Argument marshalling only: PyTorch supplies device memory and streams, every step of the
block runs in the CUDA library.  There is no fallback: if ``libspd_b200.so`` is missing or a
call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os
from typing import Dict, List, Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libspd_b200.so")

SPD_OK = 0
STATUS_NAMES = {0: "SPD_OK", -1: "SPD_EINVAL", -2: "SPD_ENULL", -3: "SPD_EWORKSPACE", -4: "SPD_ECAPACITY",
                -5: "SPD_ECUDA", -6: "SPD_EDEVICE", -7: "SPD_ECALLBACK"}
ALLREDUCE_FN = ctypes.CFUNCTYPE(ctypes.c_int, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_size_t, ctypes.c_void_p)
WEIGHT_NAMES = ("attn_norm", "wq", "wk", "wv", "wo", "mlp_norm", "w_gate", "w_up", "w_down")
BIAS_FIELDS = ("attn_norm_b", "bq", "bk", "bv", "bo", "mlp_norm_b", "b_fc1", "b_fc2")
# tensors of a layer of the block with bias (Sec. 4.1.2) -> fields of spd_layer
BIAS_LAYER_FIELDS = {"attn_norm": "attn_norm", "attn_norm_b": "attn_norm_b", "wq": "wq", "bq": "bq", "wk": "wk", "bk": "bk", "wv": "wv",
                     "bv": "bv", "wo": "wo", "bo": "bo", "mlp_norm": "mlp_norm", "mlp_norm_b": "mlp_norm_b", "w_fc1": "w_gate",
                     "b_fc1": "b_fc1", "w_fc2": "w_down", "b_fc2": "b_fc2"}
EXPORTS = ("spd_workspace_bytes", "spd_create", "spd_prefill", "spd_decode_step", "spd_sync_points",
           "spd_launches_per_decode_step", "spd_device_error", "spd_destroy", "spd_status_string",
           "spd_last_cuda_error", "spd_profile_begin", "spd_profile_end", "spd_profile_kinds",
           "spd_profile_kind_name", "spd_gemm_bf16", "spd_set_graphs", "spd_gemm_bf16_sum_static",
           "spd_set_tuning", "spd_set_mask", "spd_sensitivity_scan", "spd_alg1_plan",
           "spd_head_grouping_stats", "spd_head_scatter", "spd_mlp_match", "spd_timeline_begin", "spd_timeline_read",
           "spd_timeline_end", "spd_tp_region_bytes", "spd_tp_attach", "spd_tp_detach", "spd_tp_decode_step",
           "spd_tp_prefill", "spd_tp_baseline_decode_step", "spd_tp_baseline_prefill")


class SpdError(RuntimeError):
    def __init__(self, where: str, status: int, detail: str = ""):
        self.status = status
        super().__init__(f"{where}: {STATUS_NAMES.get(status, status)} {detail}".strip())


class spd_dims(ctypes.Structure):
    _fields_ = [("n_layers", ctypes.c_int32), ("hidden", ctypes.c_int32), ("n_q_heads", ctypes.c_int32),
                ("n_kv_heads", ctypes.c_int32), ("head_dim", ctypes.c_int32), ("ffn", ctypes.c_int32),
                ("T", ctypes.c_int32), ("dtype", ctypes.c_int32), ("rms_eps", ctypes.c_float),
                ("rope_base", ctypes.c_float), ("kv_block_size", ctypes.c_int32), ("max_batch", ctypes.c_int32),
                ("max_seq_len", ctypes.c_int32), ("max_prefill_tokens", ctypes.c_int32), ("block_kind", ctypes.c_int32)]


class spd_layer(ctypes.Structure):
    _fields_ = [(n, ctypes.c_void_p) for n in WEIGHT_NAMES] + [("k_pages", ctypes.c_void_p), ("v_pages", ctypes.c_void_p)] + \
               [(n, ctypes.c_void_p) for n in BIAS_FIELDS]


_lib = None


def load_library() -> ctypes.CDLL:
    """Load the in-tree CUDA library; raise if it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: run `python -m paper_2502_20727_b200.build` "
                          "(there is no CPU or PyTorch fallback)")
    lib = ctypes.CDLL(LIB_PATH)
    vp, i32, sz = ctypes.c_void_p, ctypes.c_int32, ctypes.c_size_t
    lib.spd_workspace_bytes.argtypes = [ctypes.POINTER(spd_dims), vp, ctypes.POINTER(sz)]
    lib.spd_create.argtypes = [ctypes.POINTER(spd_dims), vp, ctypes.POINTER(spd_layer), i32, vp, sz,
                               ctypes.POINTER(vp)]
    lib.spd_prefill.argtypes = [vp, vp, i32, i32, vp, i32, vp, vp]
    lib.spd_decode_step.argtypes = [vp, vp, i32, vp, vp, i32, i32, vp, vp]
    lib.spd_sync_points.argtypes = [vp]
    lib.spd_launches_per_decode_step.argtypes = [vp]
    lib.spd_device_error.argtypes = [vp, vp, ctypes.POINTER(i32)]
    lib.spd_destroy.argtypes = [vp]
    lib.spd_destroy.restype = None
    lib.spd_status_string.argtypes = [ctypes.c_int]
    lib.spd_status_string.restype = ctypes.c_char_p
    lib.spd_last_cuda_error.argtypes = []
    lib.spd_gemm_bf16.argtypes = [vp, vp, vp, i32, i32, i32, i32, i32, i32, i32, vp, vp]
    lib.spd_set_graphs.argtypes = [vp, i32]
    lib.spd_set_mask.argtypes = [vp, vp]
    lib.spd_sensitivity_scan.argtypes = [vp, vp, i32, i32, vp, i32, vp, vp, ctypes.POINTER(ctypes.c_double),
                                         ctypes.POINTER(ctypes.c_double), vp]
    lib.spd_head_grouping_stats.argtypes = [vp, i32, vp, i32, i32, vp, i32, vp, vp, ctypes.POINTER(ctypes.c_float),
                                            ctypes.POINTER(ctypes.c_double), vp]
    lib.spd_head_scatter.argtypes = [ctypes.POINTER(ctypes.c_float), i32, i32, i32, ctypes.POINTER(i32), ctypes.POINTER(ctypes.c_double)]
    lib.spd_mlp_match.argtypes = [ctypes.POINTER(ctypes.c_double), i32, ctypes.POINTER(i32), ctypes.POINTER(ctypes.c_double)]
    lib.spd_alg1_plan.argtypes = [ctypes.POINTER(ctypes.c_double), i32, i32, ctypes.c_double, ctypes.c_double, vp, vp]
    lib.spd_set_tuning.argtypes = [vp, ctypes.c_char_p, i32]
    lib.spd_gemm_bf16_sum_static.argtypes = [vp, vp, vp, i32, i32, i32, i32, i32, i32, i32, vp, vp]
    lib.spd_tp_region_bytes.argtypes = [vp, i32, ctypes.POINTER(sz)]
    lib.spd_tp_attach.argtypes = [vp, i32, i32, ctypes.POINTER(vp), sz, vp]
    lib.spd_tp_detach.argtypes = [vp]
    lib.spd_tp_decode_step.argtypes = [vp, vp, i32, vp, vp, i32, i32, vp, vp]
    lib.spd_tp_prefill.argtypes = [vp, vp, i32, i32, vp, i32, vp, vp]
    lib.spd_tp_baseline_decode_step.argtypes = [vp, vp, i32, vp, vp, i32, i32, vp, vp, sz, ALLREDUCE_FN, vp, vp]
    lib.spd_tp_baseline_prefill.argtypes = [vp, vp, i32, i32, vp, i32, vp, vp, sz, ALLREDUCE_FN, vp, vp]
    lib.spd_profile_begin.argtypes = [vp]
    lib.spd_profile_end.argtypes = [vp, vp, ctypes.POINTER(ctypes.c_float), ctypes.POINTER(i32)]
    lib.spd_timeline_begin.argtypes = [vp, vp]
    lib.spd_timeline_end.argtypes = [vp]
    lib.spd_timeline_read.argtypes = [vp, vp, i32, ctypes.POINTER(i32), ctypes.POINTER(ctypes.c_uint64), ctypes.POINTER(i32),
                                      ctypes.POINTER(ctypes.c_uint64), ctypes.POINTER(ctypes.c_uint64)]
    lib.spd_profile_kinds.argtypes = []
    lib.spd_profile_kind_name.argtypes = [ctypes.c_int]
    lib.spd_profile_kind_name.restype = ctypes.c_char_p
    for n in EXPORTS:
        if n not in ("spd_destroy", "spd_status_string", "spd_profile_kind_name", "spd_gemm_bf16"):
            getattr(lib, n).restype = ctypes.c_int
    _lib = lib
    return lib


def _check(where: str, rc: int):
    if rc != SPD_OK:
        lib = load_library()
        detail = lib.spd_status_string(rc).decode()
        if rc == -5:
            detail += f" (cudaError {lib.spd_last_cuda_error()})"
        raise SpdError(where, rc, detail)


def _stream_ptr() -> ctypes.c_void_p:
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def gemm_bf16(a: torch.Tensor, w: torch.Tensor, *, splits: int = 1, swap: bool = False) -> torch.Tensor:
    """The projection GEMM on its own.  a: bf16 [M,K] or [batches,M,K]; w: bf16 [N,K] or [batches,N,K].
    Returns fp32 [splits, M, batches*N]."""
    lib = load_library()
    wb = w if w.dim() == 3 else w[None]
    a_batched = a.dim() == 3
    batches, N, K = wb.shape
    M = a.shape[-2]
    if a_batched and a.shape[0] != batches:
        raise ValueError("a and w disagree on the batch count")
    for t in (a, w):
        if not (t.is_cuda and t.is_contiguous() and t.dtype == torch.bfloat16):
            raise ValueError("contiguous CUDA bf16 tensors expected")
    c = torch.empty((splits, M, batches * N), dtype=torch.float32, device=a.device)
    err = torch.zeros(1, dtype=torch.int32, device=a.device)
    with torch.cuda.device(a.device):
        _check("spd_gemm_bf16", lib.spd_gemm_bf16(a.data_ptr(), w.data_ptr(), c.data_ptr(), M, N, K, batches,
                                                   1 if a_batched else 0, splits, 1 if swap else 0, err.data_ptr(),
                                                   _stream_ptr()))
    if int(err.item()) != 0:
        raise SpdError("spd_gemm_bf16", -6, f"device flag {int(err.item())}")
    return c


STATIC_SCRATCH_BYTES = 4 << 20


def gemm_bf16_sum_static(a: torch.Tensor, w: torch.Tensor, out: torch.Tensor, err: torch.Tensor, *, splits: int = 1,
                         swap: bool = False) -> torch.Tensor:
    """spd_gemm_bf16_sum_static: the split-K GEMM summed over its splits, for callers that must
    not allocate device memory during the call.  The caller passes the output (fp32
    [M, batches*N]) and the int32 error flag; the split planes sit in the library's own fixed
    array (``STATIC_SCRATCH_BYTES``; larger problems raise SPD_EWORKSPACE).  Nothing is
    allocated here either, and the flag is not read back: check ``err`` when convenient."""
    lib = load_library()
    wb = w if w.dim() == 3 else w[None]
    a_batched = a.dim() == 3
    batches, N, K = wb.shape
    M = a.shape[-2]
    if a_batched and a.shape[0] != batches:
        raise ValueError("a and w disagree on the batch count")
    for t in (a, w):
        if not (t.is_cuda and t.is_contiguous() and t.dtype == torch.bfloat16):
            raise ValueError("contiguous CUDA bf16 tensors expected")
    if not (out.is_cuda and out.is_contiguous() and out.dtype == torch.float32 and tuple(out.shape) == (M, batches * N)):
        raise ValueError("out: contiguous CUDA float32 [M, batches*N]")
    if not (err.is_cuda and err.dtype == torch.int32 and err.numel() >= 1):
        raise ValueError("err: CUDA int32 tensor")
    with torch.cuda.device(a.device):
        _check("spd_gemm_bf16_sum_static",
               lib.spd_gemm_bf16_sum_static(a.data_ptr(), w.data_ptr(), out.data_ptr(), M, N, K, batches,
                                            1 if a_batched else 0, splits, 1 if swap else 0, err.data_ptr(),
                                            _stream_ptr()))
    return out


TIER_NAMES = ("TP", "ISB", "SB", "ESB")


def alg1_plan(sensitivity: Sequence[float], n_spd: int, tau1: float, tau2: float):
    """Algorithm 1 on a list of block sensitivities; returns (sync_mask, tiers), see spd_alg1_plan."""
    lib = load_library()
    n = len(sensitivity)
    s = (ctypes.c_double * n)(*[float(v) for v in sensitivity])
    mask = (ctypes.c_uint8 * n)()
    tier = (ctypes.c_uint8 * n)()
    _check("spd_alg1_plan", lib.spd_alg1_plan(s, n, int(n_spd), float(tau1), float(tau2), mask, tier))
    return [int(v) for v in mask], [int(v) for v in tier]


def head_scatter(dist, heads_per_unit: int, T: int):
    """Eq. 2 on a [n_heads, n_heads] distance matrix; returns (device of every unit, objective); see spd_head_scatter."""
    import numpy as np
    lib = load_library()
    d = np.ascontiguousarray(dist, dtype=np.float32)
    n = d.shape[0]
    out = (ctypes.c_int32 * (n // heads_per_unit))()
    obj = ctypes.c_double(0.0)
    _check("spd_head_scatter", lib.spd_head_scatter(d.ctypes.data_as(ctypes.POINTER(ctypes.c_float)), n, int(heads_per_unit), int(T), out,
                                                     ctypes.byref(obj)))
    return [int(v) for v in out], obj.value


def mlp_match(norms):
    """Eq. 3 on a [T, T] matrix of output norms; returns (MLP partition of every device, objective); see spd_mlp_match."""
    import numpy as np
    lib = load_library()
    nm = np.ascontiguousarray(norms, dtype=np.float64)
    T = nm.shape[0]
    out = (ctypes.c_int32 * T)()
    obj = ctypes.c_double(0.0)
    _check("spd_mlp_match", lib.spd_mlp_match(nm.ctypes.data_as(ctypes.POINTER(ctypes.c_double)), T, out, ctypes.byref(obj)))
    return [int(v) for v in out], obj.value


def head_order_from_devices(device_of_unit: Sequence[int], heads_per_unit: int, T: int) -> List[int]:
    """Query-head order that puts the units of device 0 first, then device 1, ... (units keep their order inside a
    device): position p of the result names the old head that moves to p."""
    order: List[int] = []
    for dev in range(T):
        for u, du in enumerate(device_of_unit):
            if du == dev:
                order.extend(range(u * heads_per_unit, (u + 1) * heads_per_unit))
    return order


def permute_layer(lw: Dict[str, torch.Tensor], *, n_q_heads: int, n_kv_heads: int, head_dim: int, T: int,
                  head_order: Optional[Sequence[int]] = None, mlp_of_device: Optional[Sequence[int]] = None) -> Dict[str, torch.Tensor]:
    """The weight re-ordering of Sec. 4.2.4 (index moves only): rows of wq / wk / wv and columns of wo by head so that
    the heads of A_i sit on device i, and the MLP partitions (row blocks of w_gate / w_up, column blocks of w_down) so
    that device i holds partition mlp_of_device[i].  The function a TP block computes does not change."""
    out = dict(lw)
    dev = lw["wq"].device
    if head_order is not None:
        group = n_q_heads // n_kv_heads
        q_idx = torch.tensor([h * head_dim + e for h in head_order for e in range(head_dim)], device=dev)
        kv_order = [head_order[i] // group for i in range(0, n_q_heads, group)]
        kv_idx = torch.tensor([h * head_dim + e for h in kv_order for e in range(head_dim)], device=dev)
        out["wq"] = lw["wq"].index_select(0, q_idx).contiguous()
        out["wk"] = lw["wk"].index_select(0, kv_idx).contiguous()
        out["wv"] = lw["wv"].index_select(0, kv_idx).contiguous()
        out["wo"] = lw["wo"].index_select(1, q_idx).contiguous()
    if mlp_of_device is not None:
        F = lw["w_gate"].shape[0]
        Fs = F // T
        f_idx = torch.tensor([m * Fs + e for m in mlp_of_device for e in range(Fs)], device=dev)
        out["w_gate"] = lw["w_gate"].index_select(0, f_idx).contiguous()
        out["w_up"] = lw["w_up"].index_select(0, f_idx).contiguous()
        out["w_down"] = lw["w_down"].index_select(1, f_idx).contiguous()
    return out


def tp_tile_owner(tile: int, T: int):
    """Rank-mode prompts: (owner rank, slot in the owner's receive planes) of the 128-token tile `tile` of a launch -
    tiles are dealt round-robin, so tile i is summed and redistributed by rank i % T (spd_tp_prefill)."""
    return tile % T, tile // T


def shard_layer(lw: Dict[str, torch.Tensor], r: int, T: int) -> Dict[str, torch.Tensor]:
    """The tensors rank r of a T-GPU group holds of one LLaMA-style layer (Sec. 3): rows r of the
    column-parallel matrices, columns r of the row-parallel ones (as contiguous matrices), the norm gains whole."""
    def rows(t):
        n = t.shape[0] // T
        return t[r * n:(r + 1) * n].contiguous()

    def cols(t):
        n = t.shape[1] // T
        return t[:, r * n:(r + 1) * n].contiguous()

    return {"attn_norm": lw["attn_norm"], "mlp_norm": lw["mlp_norm"], "wq": rows(lw["wq"]), "wk": rows(lw["wk"]),
            "wv": rows(lw["wv"]), "wo": cols(lw["wo"]), "w_gate": rows(lw["w_gate"]), "w_up": rows(lw["w_up"]),
            "w_down": cols(lw["w_down"])}


class CollectiveAllReduce:
    """The all-reduce of the rank-mode baseline as a torch.distributed collective (NCCL on GPUs, gloo on CPU tensors):
    sums the view over the group in place on the current stream and counts the calls - one per sync-point the
    blocks keep (Sec. 3: two per TP block; Sec. 4.1.1: one per SPD block)."""

    def __init__(self, group=None):
        self.group, self.calls, self.elements = group, 0, 0

    def __call__(self, view: torch.Tensor):
        import torch.distributed as dist
        dist.all_reduce(view, op=dist.ReduceOp.SUM, group=self.group)
        self.calls += 1
        self.elements += view.numel()


class SpdStack:
    """A stack of TP / SPD decoder blocks over caller-held weights and paged KV tensors.

    layers: one dict per layer with the tensors of ``WEIGHT_NAMES`` (CUDA, contiguous, dtype
    float32 or bfloat16, torch.nn.Linear layout).  sync_mask[l] = 1 runs layer l as the
    synchronous TP block, 0 as the SPD block.
    """

    def __init__(self, *, hidden: int, n_q_heads: int, n_kv_heads: int, head_dim: int, ffn: int, T: int,
                 sync_mask: Sequence[int], layers: List[Dict[str, torch.Tensor]], n_pages: int,
                 max_batch: int, max_seq_len: int, max_prefill_tokens: int, rms_eps: float = 1e-5,
                 rope_base: float = 10000.0, kv_block_size: int = 16, device: Optional[torch.device] = None, block: str = "llama"):
        self.lib = load_library()
        self.device = torch.device(device if device is not None else "cuda:0")
        dt = layers[0]["wq"].dtype
        if dt not in (torch.float32, torch.bfloat16):
            raise ValueError("weights must be float32 or bfloat16")
        self.dtype = dt
        if block not in ("llama", "opt"):
            raise ValueError("block: 'llama' (no bias) or 'opt' (with bias)")
        self.block = block
        # tensor name -> spd_layer field
        self.fields = {n: n for n in WEIGHT_NAMES} if block == "llama" else dict(BIAS_LAYER_FIELDS)
        self.dims = spd_dims(len(layers), hidden, n_q_heads, n_kv_heads, head_dim, ffn, T,
                             0 if dt == torch.float32 else 1, rms_eps, rope_base, kv_block_size, max_batch,
                             max_seq_len, max_prefill_tokens, 0 if block == "llama" else 1)
        self.mask = (ctypes.c_uint8 * len(layers))(*[1 if m else 0 for m in sync_mask])
        if len(sync_mask) != len(layers):
            raise ValueError("one mask entry per layer")
        self.layers = layers
        self.n_pages = n_pages
        for lw in layers:
            for n in self.fields:
                t = lw[n]
                if not (t.is_cuda and t.is_contiguous() and t.dtype == dt):
                    raise ValueError(f"{n}: need a contiguous CUDA tensor of dtype {dt}")
        with torch.cuda.device(self.device):
            page_shape = (n_pages, n_kv_heads, kv_block_size, head_dim)
            self.k_pages = [torch.zeros(page_shape, dtype=dt, device=self.device) for _ in layers]
            self.v_pages = [torch.zeros(page_shape, dtype=dt, device=self.device) for _ in layers]
            nbytes = ctypes.c_size_t(0)
            _check("spd_workspace_bytes", self.lib.spd_workspace_bytes(ctypes.byref(self.dims), self.mask,
                                                                         ctypes.byref(nbytes)))
            self.workspace = torch.empty(nbytes.value + 256, dtype=torch.uint8, device=self.device)
            base = (self.workspace.data_ptr() + 255) // 256 * 256
            arr = (spd_layer * len(layers))()
            for i, lw in enumerate(layers):
                for n, field in self.fields.items():
                    setattr(arr[i], field, lw[n].data_ptr())
                arr[i].k_pages = self.k_pages[i].data_ptr()
                arr[i].v_pages = self.v_pages[i].data_ptr()
            self._ctx = ctypes.c_void_p()
            _check("spd_create", self.lib.spd_create(ctypes.byref(self.dims), self.mask, arr, n_pages,
                                                      ctypes.c_void_p(base), nbytes.value, ctypes.byref(self._ctx)))
        self.workspace_bytes = nbytes.value

    # -- calls ---------------------------------------------------------------------------
    def prefill(self, x: torch.Tensor, block_table: torch.Tensor, out: Optional[torch.Tensor] = None) -> torch.Tensor:
        B, S, H = x.shape
        self._check_io(x, block_table)
        out = torch.empty_like(x) if out is None else out
        with torch.cuda.device(self.device):
            _check("spd_prefill", self.lib.spd_prefill(self._ctx, x.data_ptr(), B, S, block_table.data_ptr(),
                                                        block_table.shape[1], out.data_ptr(), _stream_ptr()))
        return out

    def decode_step(self, x: torch.Tensor, seq_lens: torch.Tensor, block_table: torch.Tensor, max_context: int,
                    out: Optional[torch.Tensor] = None) -> torch.Tensor:
        B, H = x.shape
        self._check_io(x, block_table)
        if not (seq_lens.is_cuda and seq_lens.dtype == torch.int32 and seq_lens.numel() == B):
            raise ValueError("seq_lens: int32 CUDA tensor [B]")
        out = torch.empty_like(x) if out is None else out
        with torch.cuda.device(self.device):
            _check("spd_decode_step", self.lib.spd_decode_step(self._ctx, x.data_ptr(), B, seq_lens.data_ptr(),
                                                                block_table.data_ptr(), block_table.shape[1],
                                                                int(max_context), out.data_ptr(), _stream_ptr()))
        return out

    def device_error(self) -> int:
        flag = ctypes.c_int32(0)
        with torch.cuda.device(self.device):
            _check("spd_device_error", self.lib.spd_device_error(self._ctx, _stream_ptr(), ctypes.byref(flag)))
        return flag.value

    def profile_begin(self):
        _check("spd_profile_begin", self.lib.spd_profile_begin(self._ctx))

    def profile_end(self) -> Dict[str, Dict[str, float]]:
        """Returns {kind: {"ms": total, "launches": n}} for the calls since profile_begin."""
        n = self.lib.spd_profile_kinds()
        ms = (ctypes.c_float * n)()
        cnt = (ctypes.c_int32 * n)()
        with torch.cuda.device(self.device):
            _check("spd_profile_end", self.lib.spd_profile_end(self._ctx, _stream_ptr(), ms, cnt))
        return {self.lib.spd_profile_kind_name(i).decode(): {"ms": float(ms[i]), "launches": int(cnt[i])}
                for i in range(n)}

    def timeline_begin(self):
        """Stamp every kernel of the following calls and fold the stamps into per-launch totals; see spd_timeline_begin."""
        with torch.cuda.device(self.device):
            _check("spd_timeline_begin", self.lib.spd_timeline_begin(self._ctx, _stream_ptr()))

    def timeline_end(self):
        _check("spd_timeline_end", self.lib.spd_timeline_end(self._ctx))

    def timeline_read(self):
        """([(kind name, own_ns summed over the calls)] in launch order, span_ns summed, number of calls) since
        timeline_begin; see spd_timeline_read."""
        cap = 6 * self.dims.n_layers + 16
        kinds = (ctypes.c_int32 * cap)()
        own = (ctypes.c_uint64 * cap)()
        n = ctypes.c_int32(0)
        span, calls = ctypes.c_uint64(0), ctypes.c_uint64(0)
        with torch.cuda.device(self.device):
            _check("spd_timeline_read", self.lib.spd_timeline_read(self._ctx, _stream_ptr(), cap, kinds, own, ctypes.byref(n),
                                                                    ctypes.byref(span), ctypes.byref(calls)))
        names = [self.lib.spd_profile_kind_name(i).decode() for i in range(self.lib.spd_profile_kinds())]
        return [(names[kinds[i]], int(own[i])) for i in range(n.value)], int(span.value), int(calls.value)

    def set_mask(self, sync_mask: Sequence[int]):
        """Replace the per-block mask (1 = TP block, 0 = SPD block); see spd_set_mask."""
        if len(sync_mask) != self.dims.n_layers:
            raise ValueError("one mask entry per layer")
        m = (ctypes.c_uint8 * len(sync_mask))(*[1 if v else 0 for v in sync_mask])
        _check("spd_set_mask", self.lib.spd_set_mask(self._ctx, m))
        self.mask = m

    def sensitivity_scan(self, x: torch.Tensor, block_table: torch.Tensor):
        """Sec. 4.2.1 scan on prompt batch x [B, S, hidden]; returns (sensitivity[L], metric[L+1]);
        see spd_sensitivity_scan."""
        B, S, H = x.shape
        self._check_io(x, block_table)
        L = self.dims.n_layers
        ref, tmp = torch.empty_like(x), torch.empty_like(x)
        sens = (ctypes.c_double * L)()
        met = (ctypes.c_double * (L + 1))()
        with torch.cuda.device(self.device):
            _check("spd_sensitivity_scan",
                   self.lib.spd_sensitivity_scan(self._ctx, x.data_ptr(), B, S, block_table.data_ptr(), block_table.shape[1],
                                                 ref.data_ptr(), tmp.data_ptr(), sens, met, _stream_ptr()))
        return [float(v) for v in sens], [float(v) for v in met]

    def head_grouping_stats(self, layer: int, x: torch.Tensor, block_table: torch.Tensor):
        """Head distances (Eq. 2) and MLP output norms (Eq. 3) of block `layer` on prompt batch x [B, S, hidden];
        returns (dist [nq, nq], norms [T, T]) as numpy arrays; see spd_head_grouping_stats."""
        import numpy as np
        B, S, H = x.shape
        self._check_io(x, block_table)
        nq, T = self.dims.n_q_heads, self.dims.T
        sigma = torch.empty(nq * B * S * S, dtype=torch.float32, device=self.device)
        dist_dev = torch.empty(nq * nq, dtype=torch.float32, device=self.device)
        dist = np.zeros((nq, nq), dtype=np.float32)
        norms = np.zeros((T, T), dtype=np.float64)
        with torch.cuda.device(self.device):
            _check("spd_head_grouping_stats",
                   self.lib.spd_head_grouping_stats(self._ctx, int(layer), x.data_ptr(), B, S, block_table.data_ptr(),
                                                    block_table.shape[1], sigma.data_ptr(), dist_dev.data_ptr(),
                                                    dist.ctypes.data_as(ctypes.POINTER(ctypes.c_float)),
                                                    norms.ctypes.data_as(ctypes.POINTER(ctypes.c_double)), _stream_ptr()))
        return dist, norms

    def set_graphs(self, enabled: bool):
        """Replay decode steps from captured CUDA graphs (default on); see spd_set_graphs."""
        _check("spd_set_graphs", self.lib.spd_set_graphs(self._ctx, 1 if enabled else 0))

    def set_tuning(self, **kw: int):
        """Tuning knobs of the decode step, e.g. ``set_tuning(qkv_splits=4, l2_prefetch_blocks=8)``;
        see spd_set_tuning."""
        for k, v in kw.items():
            _check("spd_set_tuning", self.lib.spd_set_tuning(self._ctx, k.encode(), int(v)))

    # -- tensor parallelism across GPUs (spd_tp_*) ------------------------------------------
    def tp_region_bytes(self, T: int) -> int:
        n = ctypes.c_size_t(0)
        _check("spd_tp_region_bytes", self.lib.spd_tp_region_bytes(self._ctx, int(T), ctypes.byref(n)))
        return n.value

    def tp_attach(self, T: int, rank_base: int, region_ptrs: Sequence[int], region_bytes: int):
        """Make this context rank ``rank_base`` (and the following ones, if it holds several shards) of a
        group of T ranks; region_ptrs[j] = device address of rank j's region as mapped in this process."""
        if len(region_ptrs) != T:
            raise ValueError("one region per rank")
        arr = (ctypes.c_void_p * T)(*[ctypes.c_void_p(int(p)) for p in region_ptrs])
        with torch.cuda.device(self.device):
            _check("spd_tp_attach", self.lib.spd_tp_attach(self._ctx, int(T), int(rank_base), arr, int(region_bytes),
                                                            _stream_ptr()))

    def tp_attach_local(self):
        """All T ranks of the group on this GPU (every launch covers all ranks' data): regions in one tensor."""
        T = self.dims.T
        stride = (self.tp_region_bytes(T) + 1023) // 1024 * 1024
        with torch.cuda.device(self.device):
            self._tp_regions = torch.empty(T * stride + 1024, dtype=torch.uint8, device=self.device)
        base = (self._tp_regions.data_ptr() + 1023) // 1024 * 1024
        self.tp_attach(T, 0, [base + j * stride for j in range(T)], stride)

    def tp_attach_symmetric(self, rank: int, world: int, group=None):
        """Rank ``rank`` of a real group of ``world`` GPUs (one process per GPU, torch.distributed initialised
        with NCCL): the region is a symmetric-memory allocation whose peer mappings the rendezvous returns."""
        import torch.distributed as dist
        import torch.distributed._symmetric_memory as symm
        group = group if group is not None else dist.group.WORLD
        nbytes = (self.tp_region_bytes(world) + 1023) // 1024 * 1024
        with torch.cuda.device(self.device):
            self._tp_regions = symm.empty(nbytes, dtype=torch.uint8, device=self.device)
            handle = symm.rendezvous(self._tp_regions, group.group_name if hasattr(group, "group_name") else group)
            ptrs = [int(p) for p in handle.buffer_ptrs]
            self.tp_attach(world, rank, ptrs, nbytes)
            torch.cuda.current_stream().synchronize()
        dist.barrier(group=group)
        self._tp_handle = handle

    def tp_detach(self):
        _check("spd_tp_detach", self.lib.spd_tp_detach(self._ctx))

    def tp_prefill(self, x: torch.Tensor, block_table: torch.Tensor, out: Optional[torch.Tensor] = None) -> torch.Tensor:
        """Prompts in rank mode; returns [ranks held by this context, B, S, hidden]."""
        B, S, H = x.shape
        self._check_io(x, block_table)
        if out is None:
            out = torch.empty((self.dims.T, B, S, H), dtype=x.dtype, device=x.device)
        with torch.cuda.device(self.device):
            _check("spd_tp_prefill", self.lib.spd_tp_prefill(self._ctx, x.data_ptr(), B, S, block_table.data_ptr(),
                                                              block_table.shape[1], out.data_ptr(), _stream_ptr()))
        return out

    def tp_decode_step(self, x: torch.Tensor, seq_lens: torch.Tensor, block_table: torch.Tensor, max_context: int,
                       out: Optional[torch.Tensor] = None) -> torch.Tensor:
        """One decode step in rank mode; returns [ranks held by this context, B, hidden]."""
        B, H = x.shape
        self._check_io(x, block_table)
        if not (seq_lens.is_cuda and seq_lens.dtype == torch.int32 and seq_lens.numel() == B):
            raise ValueError("seq_lens: int32 CUDA tensor [B]")
        if out is None:
            out = torch.empty((self.dims.T, B, H), dtype=x.dtype, device=x.device)
        with torch.cuda.device(self.device):
            _check("spd_tp_decode_step", self.lib.spd_tp_decode_step(self._ctx, x.data_ptr(), B, seq_lens.data_ptr(),
                                                                      block_table.data_ptr(), block_table.shape[1],
                                                                      int(max_context), out.data_ptr(), _stream_ptr()))
        return out

    # -- baseline of the rank mode: the shard sums as a collective between kernels (spd_tp_baseline_*) ---------
    def _baseline_hook(self, all_reduce, tokens):
        """(ctypes callback, scratch tensor) for one call: the library hands the callback a pointer into `scratch`;
        the caller's all_reduce gets the matching fp32 view and sums it over the ranks in place."""
        need = 2 * tokens * self.dims.hidden
        if getattr(self, "_baseline_scratch", None) is None or self._baseline_scratch.numel() < need:
            self._baseline_scratch = torch.empty(need, dtype=torch.float32, device=self.device)
        scratch, self._baseline_error = self._baseline_scratch, None

        def hook(user, buf, count, stream):
            try:
                first = (int(buf) - scratch.data_ptr()) // 4
                all_reduce(scratch[first:first + int(count)])
                return 0
            except Exception as e:  # surfaces as SPD_ECALLBACK; the exception itself is re-raised by the caller
                self._baseline_error = e
                return 1
        return ALLREDUCE_FN(hook), scratch

    def tp_baseline_decode_step(self, x, seq_lens, block_table, max_context, all_reduce, out=None):
        """One decode step of ONE shard's stack (this context: T = 1, the shard's weights) with the block's kept shard
        sums done by ``all_reduce(view)`` - an in-place sum of a float32 CUDA view over all ranks, enqueued on the
        current stream (e.g. ``torch.distributed.all_reduce``); see spd_tp_baseline_decode_step."""
        B, H = x.shape
        self._check_io(x, block_table)
        out = torch.empty_like(x) if out is None else out
        fn, scratch = self._baseline_hook(all_reduce, B)
        with torch.cuda.device(self.device):
            rc = self.lib.spd_tp_baseline_decode_step(self._ctx, x.data_ptr(), B, seq_lens.data_ptr(), block_table.data_ptr(),
                                                      block_table.shape[1], int(max_context), out.data_ptr(), scratch.data_ptr(),
                                                      scratch.numel(), fn, None, _stream_ptr())
        if self._baseline_error is not None:
            raise self._baseline_error
        _check("spd_tp_baseline_decode_step", rc)
        return out

    def tp_baseline_prefill(self, x, block_table, all_reduce, out=None):
        """Prompts through ONE shard's stack with the kept shard sums done by ``all_reduce``; see spd_tp_baseline_prefill."""
        B, S, H = x.shape
        self._check_io(x, block_table)
        out = torch.empty_like(x) if out is None else out
        fn, scratch = self._baseline_hook(all_reduce, min(B * S, self.dims.max_prefill_tokens))
        with torch.cuda.device(self.device):
            rc = self.lib.spd_tp_baseline_prefill(self._ctx, x.data_ptr(), B, S, block_table.data_ptr(), block_table.shape[1],
                                                  out.data_ptr(), scratch.data_ptr(), scratch.numel(), fn, None, _stream_ptr())
        if self._baseline_error is not None:
            raise self._baseline_error
        _check("spd_tp_baseline_prefill", rc)
        return out

    def sync_points(self) -> int:
        return self.lib.spd_sync_points(self._ctx)

    def launches_last_call(self) -> int:
        return self.lib.spd_launches_per_decode_step(self._ctx)

    def _check_io(self, x, block_table):
        if not (x.is_cuda and x.is_contiguous() and x.dtype == self.dtype and x.shape[-1] == self.dims.hidden):
            raise ValueError("x: contiguous CUDA tensor [..., hidden] of the weights' dtype")
        if not (block_table.is_cuda and block_table.dtype == torch.int32 and block_table.is_contiguous()
                and block_table.shape[0] == x.shape[0]):
            raise ValueError("block_table: contiguous int32 CUDA tensor [B, max_pages]")

    def close(self):
        if getattr(self, "_ctx", None) is not None and self._ctx.value:
            self.lib.spd_destroy(self._ctx)
            self._ctx = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def stack_from_workload(w, layers, *, sync_mask=None, max_batch=None, max_seq_len=None, max_prefill_tokens=None,
                        n_pages=None, device="cuda:0") -> SpdStack:
    """Build an SpdStack for a ``spd_inputs.Workload``-like object (duck-typed: the binding does
    not import the input generators)."""
    max_batch = max_batch or w.batch
    max_seq_len = max_seq_len or (w.prompt + w.decode_steps)
    pages_per_seq = (max_seq_len + w.kv_block - 1) // w.kv_block
    n_pages = n_pages or max_batch * pages_per_seq
    return SpdStack(hidden=w.hidden, n_q_heads=w.n_q_heads, n_kv_heads=w.n_kv_heads, head_dim=w.head_dim,
                    ffn=w.ffn, T=w.T, sync_mask=list(w.mask if sync_mask is None else sync_mask), layers=layers,
                    n_pages=n_pages, max_batch=max_batch, max_seq_len=max_seq_len,
                    max_prefill_tokens=max_prefill_tokens or min(w.batch * w.prompt, 8192), rms_eps=w.rms_eps,
                    rope_base=w.rope_base, kv_block_size=w.kv_block, device=device, block=getattr(w, "block", "llama"))
