"""The C-ABI library loads without a GPU and exports every symbol the header declares."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def libpath():
    from paper_2603_04411_b200 import build
    return build.build()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "twkv.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(twkv_[a-z_]+)\s*\(", text)))


def test_header_symbols_are_exported(libpath):
    L = ctypes.CDLL(libpath)
    names = declared_symbols()
    assert "twkv_compress" in names and "twkv_decode_attn" in names and len(names) >= 12
    for n in names:
        assert hasattr(L, n), n


def test_binding_lists_the_same_entry_points(libpath):
    from paper_2603_04411_b200 import binding
    assert sorted(binding.EXPORTS) == declared_symbols()
    for n in binding.EXPORTS:
        assert callable(getattr(binding, n)), n


def test_host_only_calls(libpath):
    from paper_2603_04411_b200 import binding as B
    assert B.twkv_status_string(0) == "ok"
    assert "capacity" in B.twkv_status_string(3)
    cfg = B.make_config(n_layers=1, n_q_heads=32, n_kv_heads=8, max_seqs=4, max_tokens_per_seq=4096)
    small = B.twkv_cache_required_bytes(cfg, 0)
    big = B.twkv_cache_required_bytes(cfg, 1 << 30)
    assert small > 0 and big - small == 1 << 30
    bad = B.make_config(n_layers=1, n_q_heads=32, n_kv_heads=8, head_dim=64, max_seqs=4, max_tokens_per_seq=4096)
    assert B.twkv_cache_required_bytes(bad, 0) == 0
    bad = B.make_config(n_layers=1, n_q_heads=24, n_kv_heads=8, max_seqs=4, max_tokens_per_seq=4096)
    assert B.twkv_cache_required_bytes(bad, 0) == 0
    # null handles are refused on the host
    assert B.lib.twkv_cache_destroy(None) == B.TWKV_ERR_INVALID_ARG
    assert B.lib.twkv_compress(None, 0, None, None, None, None, 0, None, None, 0, None) == B.TWKV_ERR_INVALID_ARG
    assert B.lib.twkv_decode_attn(None, 0, None, None, 0, None, 0, None) == B.TWKV_ERR_INVALID_ARG
    assert B.twkv_launch_count() == 0


def test_projector_argument_checks_need_no_device():
    """Sizes and pointers are validated before any CUDA call."""
    from paper_2603_04411_b200 import binding as B
    import ctypes
    assert B.twkv_projector_required_bytes(1024) == 256 + 2 * 1024 * 1024 * 2
    assert B.twkv_projector_required_bytes(1000) == 0 and B.twkv_projector_required_bytes(64) == 0
    h = ctypes.c_void_p()
    one = ctypes.c_void_p(256)
    assert B.lib.twkv_projector_create(1000, B.TWKV_F16, one, one, one, 1 << 30, None, ctypes.byref(h)) == B.TWKV_ERR_UNSUPPORTED
    assert B.lib.twkv_projector_create(1024, B.TWKV_F32, one, one, one, 1 << 30, None, ctypes.byref(h)) == B.TWKV_ERR_UNSUPPORTED
    assert B.lib.twkv_projector_create(1024, B.TWKV_F16, None, None, one, 1 << 30, None, ctypes.byref(h)) == B.TWKV_ERR_INVALID_ARG
    assert B.lib.twkv_projector_create(1024, B.TWKV_F16, one, one, None, 1 << 30, None, ctypes.byref(h)) == B.TWKV_ERR_INVALID_ARG
    assert B.lib.twkv_projector_create(1024, B.TWKV_F16, one, one, ctypes.c_void_p(264), 1 << 30, None, ctypes.byref(h)) == B.TWKV_ERR_INVALID_ARG
    assert B.lib.twkv_projector_create(1024, B.TWKV_F16, one, one, one, 1024, None, ctypes.byref(h)) == B.TWKV_ERR_CAPACITY
    assert B.lib.twkv_project(None, one, one, one, one, 4, None) == B.TWKV_ERR_INVALID_ARG
    assert h.value is None
