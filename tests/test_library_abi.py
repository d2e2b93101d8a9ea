"""The C-ABI library loads, exports every symbol the header declares, and its
host-only layout queries agree with the oracle's layout.  No GPU needed."""
import ctypes
import os
import re

import pytest

from oracle import layout as ol
from paper_2502_15075_b200 import build as kvq_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def kvq():
    kvq_build.build()
    from paper_2502_15075_b200 import kvq as mod
    return mod


def declared_functions():
    names = set()
    for fn in os.listdir(os.path.join(ROOT, "include")):
        if fn.endswith(".h"):
            text = open(os.path.join(ROOT, "include", fn)).read()
            text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
            names |= set(re.findall(r"\b(kvq_[a-z_0-9]+)\s*\(", text))
    return sorted(names)


def test_every_declared_symbol_is_exported(kvq):
    lib = ctypes.CDLL(kvq.LIB_PATH)
    names = declared_functions()
    assert len(names) >= 9
    for n in names:
        assert hasattr(lib, n), f"{n} declared in include/ but not exported"
    assert set(kvq.EXPORTS) <= set(names)
    assert kvq.kvq_layout_version() == 2


@pytest.mark.parametrize("D,kb,vb,gk,gv,k_axis", [
    (64, 4, 2, 32, 32, 0), (64, 4, 2, 64, 64, 0), (128, 4, 2, 128, 128, 0), (128, 2, 4, 128, 128, 0),
    (128, 4, 4, 128, 128, 0), (128, 8, 4, 128, 128, 0), (128, 4, 2, 128, 128, 1), (128, 8, 2, 128, 128, 1),
    (128, 16, 16, 128, 128, 0), (128, 4, 2, 32, 64, 0)])
def test_page_and_cache_bytes_match_oracle_layout(kvq, D, kb, vb, gk, gv, k_axis):
    cfg = kvq.make_config(3, 8, 2, D, kb, vb, gk, gv, k_axis, "bf16", 512)
    L = ol.Layout(D, kb, vb, gk, gv, k_axis)
    assert kvq.kvq_page_bytes(cfg) == L.page_bytes
    pages, tail = kvq.kvq_cache_bytes(cfg)
    assert pages == 3 * 2 * 4 * L.page_bytes
    assert tail == (3 * 2 * 128 * D * 2 if k_axis else 0)
    assert kvq.kvq_workspace_bytes(cfg) >= 3 * 8 * (D + 2) * 4


def test_k4v2_page_is_104_bytes_per_token(kvq):
    cfg = kvq.make_config(1, 32, 8, 128, 4, 2, 128, 128, 0, "bf16", 128)
    assert kvq.kvq_page_bytes(cfg) == 128 * 104
    cfg44 = kvq.make_config(1, 32, 8, 128, 4, 4, 128, 128, 0, "bf16", 128)
    assert kvq.kvq_page_bytes(cfg44) == 128 * 136


@pytest.mark.parametrize("kw,code", [
    (dict(head_dim=96), -2), (dict(kb=7), -2), (dict(vb=5), -2), (dict(gk=16), -2), (dict(gv=256), -2),
    (dict(capacity_tokens=100), -1), (dict(n_q_heads=9), -1), (dict(batch=0), -1), (dict(in_dtype=7), -1),
    (dict(k_axis=1, kb=16), -2), (dict(n_q_heads=32, n_kv_heads=2), -2), (dict(k_axis=2), -1)])
def test_invalid_configs_are_rejected_on_the_host(kvq, kw, code):
    base = dict(batch=2, n_q_heads=8, n_kv_heads=2, head_dim=128, kb=4, vb=2, gk=128, gv=128, k_axis=0,
                in_dtype=1, capacity_tokens=256)
    base.update(kw)
    cfg = kvq.kvq_config(**base)
    with pytest.raises(kvq.KvqError) as e:
        kvq.kvq_page_bytes(cfg)
    assert e.value.code == code
    assert "kvq" in str(e.value) and kvq.kvq_strerror(code) != "unknown kvq error"


def test_null_and_misaligned_arguments_fail_before_any_launch(kvq):
    cfg = kvq.make_config(1, 8, 2, 128, 4, 2, 128, 128, 0, "bf16", 256)
    lib = ctypes.CDLL(kvq.LIB_PATH)
    lib.kvq_decode_attention.argtypes = kvq._lib.kvq_decode_attention.argtypes
    lib.kvq_quantize_append.argtypes = kvq._lib.kvq_quantize_append.argtypes
    null_cache = kvq.kvq_cache(None, None, None, None)
    assert lib.kvq_decode_attention(ctypes.byref(cfg), ctypes.byref(null_cache), 16, 16, 2, 0.0, 16, 1 << 20, None) == -1
    fake = kvq.kvq_cache(4096 + 8, None, 4096, 4096)     # misaligned pages pointer (never dereferenced)
    assert lib.kvq_quantize_append(ctypes.byref(cfg), ctypes.byref(fake), 4096, 4096, 0, 0, 128, 1, None) == -3
    ok = kvq.kvq_cache(4096, None, 4096, 4096)
    assert lib.kvq_quantize_append(ctypes.byref(cfg), ctypes.byref(ok), 4096, 4096, 0, 0, 100, 1, None) == -1   # stride < D
    assert lib.kvq_quantize_append(ctypes.byref(cfg), ctypes.byref(ok), 4096, 4096, 0, 0, 132, 1, None) == -3   # row not 16 B
    assert lib.kvq_quantize_append(ctypes.byref(cfg), ctypes.byref(ok), 4096, 4096, 0, 0, 128, 257, None) == -5  # > capacity
    assert lib.kvq_decode_attention(ctypes.byref(cfg), ctypes.byref(ok), 4096, 4096, 2, 0.0, 4096, 8, None) == -4
    assert lib.kvq_decode_attention(ctypes.byref(cfg), ctypes.byref(ok), 4096, 4096, 9, 0.0, 4096, 1 << 20, None) == -1


def test_bit_balance_is_the_log_ratio_of_the_frobenius_norms(kvq):
    assert kvq.kvq_bit_balance(16.0, 1.0) == 2.0          # ||K||_F = 4 ||V||_F -> two more bits for keys
    assert kvq.kvq_bit_balance(1.0, 1.0) == 0.0
    assert kvq.kvq_bit_balance(1.0, 4.0) == -1.0
    with pytest.raises(kvq.KvqError):
        kvq.kvq_bit_balance(0.0, 1.0)
