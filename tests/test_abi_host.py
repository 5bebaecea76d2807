"""Host-side checks that need no GPU: the C-ABI library loads, exports every symbol the header
declares, and validates dimensions before touching a device."""
import ctypes
import os
import re

import pytest

import paper_2502_20727_b200 as spd
from paper_2502_20727_b200 import build as spd_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    spd_build.build()
    return spd.load_library()


def declared_symbols():
    out = set()
    for fn in os.listdir(os.path.join(ROOT, "include")):
        if fn.endswith(".h"):
            text = open(os.path.join(ROOT, "include", fn)).read()
            text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
            out |= set(re.findall(r"\b(spd_[a-z_0-9]+)\s*\(", text))
    return out


def test_every_declared_symbol_is_exported(lib):
    names = declared_symbols()
    assert {"spd_create", "spd_prefill", "spd_decode_step", "spd_destroy"} <= names
    for n in names:
        assert hasattr(lib, n), n
    assert names == set(spd.EXPORTS) | names  # binding knows nothing the header does not declare
    assert set(spd.EXPORTS) <= names


def dims(**kw):
    base = dict(n_layers=2, hidden=256, n_q_heads=4, n_kv_heads=4, head_dim=64, ffn=688, T=2, dtype=1,
                rms_eps=1e-5, rope_base=10000.0, kv_block_size=16, max_batch=4, max_seq_len=64,
                max_prefill_tokens=64)
    base.update(kw)
    return spd.spd_dims(**base)


def ws_bytes(lib, d, mask=(0, 1)):
    m = (ctypes.c_uint8 * len(mask))(*mask)
    n = ctypes.c_size_t(0)
    rc = lib.spd_workspace_bytes(ctypes.byref(d), m, ctypes.byref(n))
    return rc, n.value


def test_workspace_size_is_positive_and_grows(lib):
    rc, n1 = ws_bytes(lib, dims())
    assert rc == 0 and n1 > 0
    rc, n2 = ws_bytes(lib, dims(max_prefill_tokens=128))
    assert rc == 0 and n2 > n1
    rc, n_sync = ws_bytes(lib, dims(), mask=(1, 1))
    assert rc == 0 and n_sync < n1  # no per-shard MLP-input planes without an SPD block


@pytest.mark.parametrize("bad", [dict(n_q_heads=6, n_kv_heads=3, T=4), dict(n_kv_heads=2, T=4), dict(ffn=690, T=4),
                                 dict(T=0), dict(T=16), dict(head_dim=48), dict(dtype=3), dict(n_layers=0),
                                 dict(n_q_heads=4, n_kv_heads=3), dict(rms_eps=0.0), dict(max_batch=0)])
def test_bad_dims_are_rejected_on_the_host(lib, bad):
    rc, _ = ws_bytes(lib, dims(**bad))
    assert rc == -1


def test_null_pointers(lib):
    n = ctypes.c_size_t(0)
    d = dims()
    assert lib.spd_workspace_bytes(None, None, ctypes.byref(n)) == -2
    assert lib.spd_workspace_bytes(ctypes.byref(d), None, ctypes.byref(n)) == -2
    assert lib.spd_create(ctypes.byref(d), None, None, 1, None, 0, None) == -2
    assert lib.spd_prefill(None, None, 1, 1, None, 1, None, None) == -2
    assert lib.spd_decode_step(None, None, 1, None, None, 1, 1, None, None) == -2
    assert lib.spd_sync_points(None) == -2
    lib.spd_destroy(None)  # no-op


def test_status_strings(lib):
    for code in range(0, -7, -1):
        s = lib.spd_status_string(code)
        assert s and s != b"unknown status"
    assert lib.spd_status_string(-99) == b"unknown status"


def test_binding_fails_loudly_without_the_library(monkeypatch, tmp_path):
    monkeypatch.setattr(spd, "_lib", None)
    monkeypatch.setattr(spd, "LIB_PATH", str(tmp_path / "missing.so"))
    with pytest.raises(ImportError):
        spd.load_library()
