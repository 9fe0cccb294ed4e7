"""CPU-only checks of the C-ABI boundary: the library loads, exports every symbol the header
declares, and its host-side validation returns status codes (no kernel is launched)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "wersa.h")


@pytest.fixture(scope="module")
def lib():
    from paper_2507_08637_b200 import build
    path = build.build()
    return ctypes.CDLL(path)


def declared_symbols():
    text = open(HEADER).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(wersa_[a-z_0-9]+)\s*\(", text)))


def test_header_declares_the_four_core_entry_points():
    syms = declared_symbols()
    for name in ("wersa_create", "wersa_forward", "wersa_backward", "wersa_destroy"):
        assert name in syms


def test_library_exports_every_declared_symbol(lib):
    for name in declared_symbols():
        assert hasattr(lib, name), name


def _cfg(**kw):
    from paper_2507_08637_b200 import make_config
    base = dict(batch=1, heads=8, seq_len=131072, head_dim=64, levels=8, features=256)
    base.update(kw)
    return make_config(**base)


def test_workspace_bytes_and_validation():
    import paper_2507_08637_b200 as w
    full = w.wersa_workspace_bytes(_cfg())
    fwd_only = w.wersa_workspace_bytes(_cfg(flags=w.WERSA_FLAG_FORWARD_ONLY))
    assert full % 256 == 0 and 0 < fwd_only < full
    # invalid or unsupported configurations give 0
    for bad in (dict(batch=0), dict(heads=-1), dict(seq_len=1), dict(head_dim=128), dict(head_dim=20), dict(levels=0),
                dict(levels=9), dict(features=100), dict(features=1280), dict(features=512, dtype="f32"),
                dict(features=512, flags=w.WERSA_FLAG_SIMT_ONLY), dict(seq_len=100, levels=8), dict(eps=-1.0),
                dict(bw_floor=0.0)):
        assert w.wersa_workspace_bytes(_cfg(**bad)) == 0, bad
    # narrower heads run zero-padded (more workspace); feature maps up to 1024 run in groups of 256 (bf16)
    assert w.wersa_workspace_bytes(_cfg(head_dim=32)) > full
    assert w.wersa_workspace_bytes(_cfg(head_dim=16, dtype="f32", features=64)) > 0
    assert w.wersa_workspace_bytes(_cfg(features=1024)) > fwd_only
    assert w.wersa_workspace_bytes(_cfg(features=512, head_dim=32)) > 0
    # 2^L may reach the next power of two above n (zero padding of the wavelet transform)
    assert w.wersa_workspace_bytes(_cfg(seq_len=200, levels=8)) > 0


def test_create_rejects_bad_arguments_without_a_device(lib):
    import paper_2507_08637_b200 as w
    lib.wersa_create.restype = ctypes.c_int
    lib.wersa_create.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_size_t, ctypes.c_void_p]
    handle = ctypes.c_void_p()
    cfg = _cfg()
    need = w.wersa_workspace_bytes(cfg)
    assert lib.wersa_create(None, None, 0, ctypes.byref(handle)) == 1
    assert lib.wersa_create(ctypes.byref(cfg), None, need, ctypes.byref(handle)) == 3
    assert lib.wersa_create(ctypes.byref(cfg), ctypes.c_void_p(256), need - 1, ctypes.byref(handle)) == 3
    assert lib.wersa_create(ctypes.byref(cfg), ctypes.c_void_p(257), need, ctypes.byref(handle)) == 3
    bad = _cfg(features=100)
    assert lib.wersa_create(ctypes.byref(bad), ctypes.c_void_p(256), 1 << 40, ctypes.byref(handle)) == 2
    bad = _cfg(levels=0)
    assert lib.wersa_create(ctypes.byref(bad), ctypes.c_void_p(256), 1 << 40, ctypes.byref(handle)) == 1
    assert handle.value is None
    # a context is host memory only: creating and destroying one touches no device
    assert lib.wersa_create(ctypes.byref(cfg), ctypes.c_void_p(256), need, ctypes.byref(handle)) == 0
    lib.wersa_launch_count.argtypes = [ctypes.c_void_p, ctypes.c_int]
    assert lib.wersa_launch_count(handle, 0) == 0
    lib.wersa_forward.restype = ctypes.c_int
    lib.wersa_forward.argtypes = [ctypes.c_void_p] * 11
    assert lib.wersa_forward(handle, None, None, None, None, None, None, None, None, None, None) == 1
    lib.wersa_forward_host.restype = ctypes.c_int
    lib.wersa_forward_host.argtypes = [ctypes.c_void_p] * 15
    assert lib.wersa_forward_host(handle, *([None] * 14)) == 1
    assert lib.wersa_forward_host(None, *([ctypes.c_void_p(256)] * 14)) == 1
    lib.wersa_destroy.argtypes = [ctypes.c_void_p]
    assert lib.wersa_destroy(handle) == 0
    assert lib.wersa_destroy(None) == 0


def test_status_strings(lib):
    lib.wersa_status_string.restype = ctypes.c_char_p
    seen = {lib.wersa_status_string(i) for i in range(7)}
    assert len(seen) == 7 and all(s for s in seen)
