"""The C-ABI library: it loads without a GPU, exports every symbol the header declares,
and rejects bad arguments on the host before touching the device."""
import ctypes
import re
from pathlib import Path

import pytest

ROOT = Path(__file__).resolve().parent.parent


@pytest.fixture(scope="module")
def api():
    from paper_2406_05317_b200 import build
    build.build()
    from paper_2406_05317_b200 import api as _api
    return _api


def declared_symbols():
    text = (ROOT / "include" / "lococo.h").read_text()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(lococo_[a-z_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(api):
    names = declared_symbols()
    assert "lococo_compress_step" in names and "lococo_chunk_attention" in names
    assert "lococo_process_sequence" in names and len(names) >= 15
    lib = ctypes.CDLL(str(ROOT / "paper_2406_05317_b200" / "liblococo.so"))
    for n in names:
        assert hasattr(lib, n), n


def test_binding_covers_every_entry_point(api):
    bound = set(api._SIGNATURES) | {"lococo_status_string"}
    assert set(declared_symbols()) == bound


def make(api, **kw):
    cfg = dict(batch=1, heads=2, head_dim=64, M=16, k=5, c_in=64, weights_per_head=0, dtype=api.F32,
               softmax_scale=0.0, norm_eps=1e-6, max_chunk=16, path=api.PATH_AUTO)
    cfg.update(kw)
    c = api.Config(**cfg)
    h = ctypes.c_void_p()
    st = api.raw().lococo_create(ctypes.byref(c), ctypes.byref(h))
    return st, h


def test_create_validates_on_the_host(api):
    st, h = make(api)
    assert st == api.OK and h.value
    n = ctypes.c_size_t()
    assert api.raw().lococo_workspace_bytes(h, ctypes.byref(n)) == api.OK and n.value > 0
    assert api.raw().lococo_destroy(h) == api.OK
    for bad in (dict(k=4), dict(k=0), dict(c_in=96), dict(M=0), dict(max_chunk=0), dict(dtype=7),
                dict(weights_per_head=2), dict(batch=0), dict(norm_eps=-1.0), dict(path=9)):
        st, h = make(api, **bad)
        assert st == api.ERR_INVALID_ARG and not h.value, bad
    for bad in (dict(head_dim=96, c_in=96), dict(k=65), dict(batch=4096, heads=32)):
        st, h = make(api, **bad)
        assert st == api.ERR_UNSUPPORTED_SHAPE and not h.value, bad
    assert api.raw().lococo_create(None, None) == api.ERR_INVALID_ARG


def test_calls_without_workspace_or_weights_are_refused(api):
    st, h = make(api)
    T = api.Tensor(ctypes.c_void_p(4096), 1024, 1024, 64)
    n = ctypes.c_int32()
    lib = api.raw()
    assert lib.lococo_compress_step(h, T, T, 0, T, T, 4, T, T, ctypes.byref(n), None, None) == api.ERR_WORKSPACE
    assert lib.lococo_process_sequence(h, T, T, T, 8, 4, T, T, T, ctypes.byref(n), None, None) == api.ERR_WORKSPACE
    assert lib.lococo_set_weights(h, ctypes.c_void_p(4096), None, None) == api.ERR_WORKSPACE
    assert lib.lococo_set_workspace(h, ctypes.c_void_p(4097), 1 << 30, None) == api.ERR_INVALID_ARG
    assert lib.lococo_set_workspace(h, ctypes.c_void_p(4096), 16, None) == api.ERR_WORKSPACE
    # attention needs no weights, but its arguments are still checked
    bad = api.Tensor(ctypes.c_void_p(4100), 1024, 1024, 64)
    assert lib.lococo_chunk_attention(h, bad, T, T, 0, T, T, 4, T, None, None) == api.ERR_INVALID_ARG
    assert lib.lococo_chunk_attention(h, T, T, T, 17, T, T, 4, T, None, None) == api.ERR_INVALID_ARG
    assert lib.lococo_chunk_attention(h, T, T, T, 0, T, T, 17, T, None, None) == api.ERR_INVALID_ARG
    assert lib.lococo_chunk_attention(h, T, T, T, 0, T, T, 4, api.Tensor(None, 0, 0, 0), None, None) == api.ERR_INVALID_ARG
    lib.lococo_destroy(h)


def test_host_entry_point_checks_the_chunk_size_before_anything_else(api):
    # a chunk size of 0 would divide by zero on the host, one above max_chunk would overrun the scratch
    st, h = make(api)
    lib = api.raw()
    buf = ctypes.c_void_p(4096)
    n = ctypes.c_int32()
    for B in (0, -3, 17):
        assert lib.lococo_process_sequence_host(h, buf, buf, buf, 64, B, buf, None, None, ctypes.byref(n), buf,
                                                1 << 30, None) == api.ERR_INVALID_ARG, B
    # a valid chunk size gets as far as the missing workspace
    assert lib.lococo_process_sequence_host(h, buf, buf, buf, 64, 16, buf, None, None, ctypes.byref(n), buf,
                                            1 << 30, None) == api.ERR_WORKSPACE
    T = api.Tensor(ctypes.c_void_p(4096), 1024, 1024, 64)
    lib.lococo_destroy(h)


def test_status_strings(api):
    seen = {api.status_string(s) for s in range(6)}
    assert len(seen) == 6 and "ok" in seen
