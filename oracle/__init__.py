"""Python face of the CPU oracle (``spd_oracle.c``).

Test infrastructure only: the tests, the smoke check and the benchmark's CPU
baseline import this; the CUDA library and its binding never do.  Everything
here is argument marshalling (numpy -> C pointers); the arithmetic lives in the
C file.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "spd_oracle.c")
_LIB = os.path.join(_HERE, "libspd_oracle.so")

WEIGHT_NAMES = ("attn_norm", "wq", "wk", "wv", "wo", "mlp_norm", "w_gate", "w_up", "w_down")


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (OpenMP over independent rows)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-fopenmp", "-fno-fast-math", "-shared", "-fPIC", "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


class _Dims(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in
                ("n_layers", "hidden", "n_q_heads", "n_kv_heads", "head_dim", "ffn", "T")] + \
               [("rms_eps", ctypes.c_double), ("rope_base", ctypes.c_double)]


class _Layer(ctypes.Structure):
    _fields_ = [(n, ctypes.c_void_p) for n in WEIGHT_NAMES]


@dataclass
class Dims:
    n_layers: int
    hidden: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    ffn: int
    T: int
    rms_eps: float = 1e-5
    rope_base: float = 10000.0

    def c(self) -> _Dims:
        return _Dims(self.n_layers, self.hidden, self.n_q_heads, self.n_kv_heads, self.head_dim,
                     self.ffn, self.T, self.rms_eps, self.rope_base)


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.oracle_stack_forward.restype = ctypes.c_int
        _lib.oracle_unsharded_stack_forward.restype = ctypes.c_int
        _lib.oracle_block_forward.restype = ctypes.c_int
    return _lib


def _f32(a):
    a = np.ascontiguousarray(np.asarray(a), dtype=np.float32)
    return a


def _pack_layers(layers):
    """layers: list of dicts name -> array.  Returns (ctypes array, keep-alive list)."""
    keep = []
    arr = (_Layer * len(layers))()
    for i, lw in enumerate(layers):
        for n in WEIGHT_NAMES:
            a = _f32(lw[n])
            keep.append(a)
            setattr(arr[i], n, a.ctypes.data)
    return arr, keep


def _p(a):
    return ctypes.c_void_p(a.ctypes.data) if a is not None else None


class Cache:
    """The oracle's own KV cache: contiguous double [L, B, max_len, nkv*d]."""

    def __init__(self, dims: Dims, B: int, max_len: int):
        shape = (dims.n_layers, B, max_len, dims.n_kv_heads * dims.head_dim)
        self.k = np.zeros(shape, dtype=np.float64)
        self.v = np.zeros(shape, dtype=np.float64)
        self.max_len = max_len
        self.B = B


def stack_forward(dims: Dims, mask, layers, x, pos0, cache: Cache, want_layers: bool = False):
    """Run the masked stack (mask[l] = 1 sync, 0 SPD) on S new tokens per sequence.

    x: [B, S, H]; pos0: [B] tokens already cached.  Returns (out float64 [B,S,H],
    sync_points, layer_out or None)."""
    x = np.ascontiguousarray(x, dtype=np.float64)
    B, S, H = x.shape
    assert H == dims.hidden and B == cache.B
    mask = np.ascontiguousarray(mask, dtype=np.uint8)
    assert mask.shape == (dims.n_layers,)
    pos0 = np.ascontiguousarray(pos0, dtype=np.int32)
    arr, keep = _pack_layers(layers)
    out = np.empty_like(x)
    lo = np.empty((dims.n_layers, B * S, H), dtype=np.float64) if want_layers else None
    d = dims.c()
    rc = lib().oracle_stack_forward(ctypes.byref(d), _p(mask), arr, _p(x), B, S, _p(pos0),
                                    _p(cache.k), _p(cache.v), cache.max_len, _p(out), _p(lo))
    if rc < 0:
        raise ValueError("oracle: bad dims or positions")
    del keep
    return out, rc, lo


def unsharded_stack_forward(dims: Dims, layers, x, pos0, cache: Cache):
    x = np.ascontiguousarray(x, dtype=np.float64)
    B, S, H = x.shape
    pos0 = np.ascontiguousarray(pos0, dtype=np.int32)
    arr, keep = _pack_layers(layers)
    out = np.empty_like(x)
    d = dims.c()
    rc = lib().oracle_unsharded_stack_forward(ctypes.byref(d), arr, _p(x), B, S, _p(pos0),
                                              _p(cache.k), _p(cache.v), cache.max_len, _p(out))
    if rc < 0:
        raise ValueError("oracle: bad dims or positions")
    del keep
    return out


def block_forward(dims: Dims, layer, mode: int, x, pos0, cache: Cache, layer_index: int = 0):
    """One block.  mode 1 = sync, 0 = SPD, 2 = rejected design of Table 1(a)
    (output [T,B,S,H]).  Returns (out, y [T, B*S, H], sync_points)."""
    x = np.ascontiguousarray(x, dtype=np.float64)
    B, S, H = x.shape
    pos0 = np.ascontiguousarray(pos0, dtype=np.int32)
    arr, keep = _pack_layers([layer])
    out = np.empty((dims.T, B, S, H) if mode == 2 else (B, S, H), dtype=np.float64)
    y = np.empty((dims.T, B * S, H), dtype=np.float64)
    d = dims.c()
    rc = lib().oracle_block_forward(ctypes.byref(d), arr, mode, _p(x), B, S, _p(pos0),
                                    _p(cache.k[layer_index]), _p(cache.v[layer_index]),
                                    cache.max_len, _p(out), _p(y))
    if rc < 0:
        raise ValueError("oracle: bad dims or positions")
    del keep
    return out, y, rc


def stack_forward_streamed(dims: Dims, mask, layer_source, x, pos0, cache: Cache, want_layers: bool = False):
    """The masked stack of ``stack_forward`` with the weights supplied one layer at a time:
    ``layer_source(l)`` returns the dict of layer l, which is dropped again before layer l+1 is
    asked for, so a deep stack of wide layers never sits in host memory as a whole.  Block l's
    output is block l+1's input, nothing else (Algorithm 1's block list, run in order).

    Returns (out [B,S,H], sync_points, layer_out [L, B*S, H] or None)."""
    cur = np.ascontiguousarray(x, dtype=np.float64)
    B, S, H = cur.shape
    lo = np.empty((dims.n_layers, B * S, H), dtype=np.float64) if want_layers else None
    syncs = 0
    for l in range(dims.n_layers):
        cur, _, n = block_forward(dims, layer_source(l), 1 if mask[l] else 0, cur, pos0, cache, layer_index=l)
        syncs += n
        if lo is not None:
            lo[l] = cur.reshape(B * S, H)
    return cur, syncs, lo


def rmsnorm(x, g, eps):
    x = np.ascontiguousarray(x, dtype=np.float64)
    g = _f32(g)
    out = np.empty_like(x)
    lib().oracle_rmsnorm(_p(x), _p(g), x.shape[0], x.shape[1], ctypes.c_double(eps), _p(out))
    return out


def rope(v, pos: int, base: float):
    v = np.array(v, dtype=np.float64).copy()
    lib().oracle_rope(_p(v), v.shape[0], int(pos), ctypes.c_double(base))
    return v


def linear(x, w):
    """y = x @ w.T in float64 (x float64 [M,K], w float32 [N,K])."""
    x = np.ascontiguousarray(x, dtype=np.float64)
    w = _f32(w)
    out = np.empty((x.shape[0], w.shape[0]), dtype=np.float64)
    lib().oracle_linear(_p(x), _p(w), x.shape[0], w.shape[0], x.shape[1], _p(out))
    return out


# ---- the decoder block with bias (OPT-style), Sec. 4.1.2 ------------------------------------------
BIAS_WEIGHT_NAMES = ("attn_norm", "attn_norm_b", "wq", "bq", "wk", "bk", "wv", "bv", "wo", "bo", "mlp_norm", "mlp_norm_b",
                     "w_fc1", "b_fc1", "w_fc2", "b_fc2")


class _BiasLayer(ctypes.Structure):
    _fields_ = [(n, ctypes.c_void_p) for n in BIAS_WEIGHT_NAMES]


def _pack_bias_layers(layers):
    keep = []
    arr = (_BiasLayer * len(layers))()
    for i, lw in enumerate(layers):
        for n in BIAS_WEIGHT_NAMES:
            a = _f32(lw[n])
            keep.append(a)
            setattr(arr[i], n, a.ctypes.data)
    return arr, keep


def bias_stack_forward(dims: Dims, mask, layers, x, pos0, cache: Cache):
    """Masked stack of OPT-style blocks (mask[l] = 1 TP, 0 SPD with bias).  dims.rms_eps is the LayerNorm eps;
    dims.rope_base is ignored.  Returns (out [B,S,H], sync_points)."""
    x = np.ascontiguousarray(x, dtype=np.float64)
    B, S, H = x.shape
    mask = np.ascontiguousarray(mask, dtype=np.uint8)
    pos0 = np.ascontiguousarray(pos0, dtype=np.int32)
    arr, keep = _pack_bias_layers(layers)
    out = np.empty_like(x)
    d = dims.c()
    L = lib()
    L.oracle_bias_stack_forward.restype = ctypes.c_int
    rc = L.oracle_bias_stack_forward(ctypes.byref(d), _p(mask), arr, _p(x), B, S, _p(pos0), _p(cache.k), _p(cache.v), cache.max_len, _p(out))
    if rc < 0:
        raise ValueError("oracle: bad dims or positions")
    del keep
    return out, rc


def bias_unsharded_stack_forward(dims: Dims, layers, x, pos0, cache: Cache):
    x = np.ascontiguousarray(x, dtype=np.float64)
    B, S, H = x.shape
    pos0 = np.ascontiguousarray(pos0, dtype=np.int32)
    arr, keep = _pack_bias_layers(layers)
    out = np.empty_like(x)
    d = dims.c()
    L = lib()
    L.oracle_bias_unsharded_stack_forward.restype = ctypes.c_int
    rc = L.oracle_bias_unsharded_stack_forward(ctypes.byref(d), arr, _p(x), B, S, _p(pos0), _p(cache.k), _p(cache.v), cache.max_len, _p(out))
    if rc < 0:
        raise ValueError("oracle: bad dims or positions")
    del keep
    return out


def bias_block_forward(dims: Dims, layer, mode: int, x, pos0, cache: Cache):
    """One OPT-style block.  mode 1 sync, 0 SPD (Sec. 4.1.2), 2 the rejected design of Table 1(b).
    Returns (out [B,S,H], p [T, B*S, H], sync_points)."""
    x = np.ascontiguousarray(x, dtype=np.float64)
    B, S, H = x.shape
    pos0 = np.ascontiguousarray(pos0, dtype=np.int32)
    arr, keep = _pack_bias_layers([layer])
    out = np.empty((B, S, H), dtype=np.float64)
    p = np.empty((dims.T, B * S, H), dtype=np.float64)
    d = dims.c()
    L = lib()
    L.oracle_bias_block_forward.restype = ctypes.c_int
    rc = L.oracle_bias_block_forward(ctypes.byref(d), arr, mode, _p(x), B, S, _p(pos0), _p(cache.k[0]), _p(cache.v[0]), cache.max_len,
                                     _p(out), _p(p))
    if rc < 0:
        raise ValueError("oracle: bad dims or positions")
    del keep
    return out, p, rc


def layernorm(x, g, b, eps):
    x = np.ascontiguousarray(x, dtype=np.float64)
    out = np.empty_like(x)
    lib().oracle_layernorm(_p(x), _p(_f32(g)), _p(_f32(b)), x.shape[0], x.shape[1], ctypes.c_double(eps), _p(out))
    return out
