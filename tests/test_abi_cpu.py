"""CPU-only checks of the C-ABI library: it loads, exports every declared symbol, and rejects
bad arguments on the host before anything could be launched (no GPU is touched)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def B():
    from paper_2506_17286_b200 import build, binding
    build.build()
    binding.lib()
    return binding


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "gta.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"GTA_API[^;(]*?\b(gta_\w+)\s*\(", text)))


def test_every_declared_symbol_is_exported(B):
    names = _declared_symbols()
    assert set(names) >= {"gta_prefill", "gta_decode", "gta_cache_append"}
    L = ctypes.CDLL(B.LIB_PATH)
    for n in names:
        assert hasattr(L, n), f"{n} declared in include/gta.h but not exported"
    assert set(names) == set(B.EXPORTS)


def test_version_and_status_strings(B):
    assert B.version() >= 100
    seen = {B.status_string(i) for i in range(9)}
    assert len(seen) == 9 and B.status_string(0) == "ok"
    assert B.status_string(99) == "unknown status"


def _shape(B, **kw):
    base = dict(batch=2, seq=64, d_model=64, n_heads=4, n_q=2, n_k=2, n_c=1, d_h=32, d_l=64, dtype=B.GTA_BF16)
    base.update(kw)
    return B.make_shape(**base)


def test_workspace_sizes(B):
    s = _shape(B)
    assert B.prefill_workspace_bytes(s) >= 2 * 2 * 64 * 64 * 2
    assert B.prefill_workspace_bytes(s) % 256 == 0
    assert B.decode_workspace_bytes(s, 1000) > 0 and B.decode_workspace_bytes(s, 1000) % 256 == 0
    assert B.decode_workspace_bytes(s, 4000) > B.decode_workspace_bytes(s, 1000)
    assert B.prefill_workspace_bytes(_shape(B, n_q=3)) == 0       # n_q does not divide n_h
    assert B.decode_workspace_bytes(s, -1) == 0


def test_bad_arguments_are_rejected_on_the_host(B):
    L = B.lib()
    good = _shape(B)
    buf = (ctypes.c_char * 4096)()
    base = ctypes.addressof(buf)
    p = ctypes.c_void_p((base + 255) & ~255)          # an aligned (host) address: never dereferenced
    odd = ctypes.c_void_p(((base + 255) & ~255) + 2)
    args = [p] * 7

    def prefill(shape, a=args, ws=p, ws_bytes=1 << 40):
        return L.gta_prefill(ctypes.byref(shape), *a, ws, ws_bytes, None, None)

    assert L.gta_prefill(None, *args, p, 1 << 40, None, None) == B.GTA_ERR_INVALID_ARG
    assert prefill(good, [None] + args[1:]) == B.GTA_ERR_INVALID_ARG
    assert prefill(good, [odd] + args[1:]) == B.GTA_ERR_INVALID_ARG
    assert prefill(_shape(B, n_k=3)) == B.GTA_ERR_INVALID_ARG          # n_k must divide n_q
    assert prefill(_shape(B, n_c=4)) == B.GTA_ERR_INVALID_ARG          # n_c must divide n_q
    assert prefill(_shape(B, dtype=7)) == B.GTA_ERR_INVALID_ARG
    assert prefill(_shape(B, seq=-1)) == B.GTA_ERR_INVALID_ARG
    assert prefill(_shape(B, softmax_scale=-1.0)) == B.GTA_ERR_INVALID_ARG
    assert prefill(_shape(B, d_h=20)) == B.GTA_ERR_UNSUPPORTED         # rows must be 16-byte vectors
    assert prefill(_shape(B, d_h=512, d_l=512)) == B.GTA_ERR_UNSUPPORTED
    assert prefill(good, ws=None) == B.GTA_ERR_WORKSPACE
    assert prefill(good, ws_bytes=16) == B.GTA_ERR_WORKSPACE
    assert prefill(_shape(B, seq=0)) == B.GTA_OK                       # empty problem: no-op
    assert prefill(_shape(B, batch=0)) == B.GTA_OK

    def chunk(shape, kv_len, kv_cap):
        return L.gta_prefill_chunk(ctypes.byref(shape), kv_len, kv_cap, *args, p, 1 << 40, None, None)

    n = good.seq
    assert chunk(good, n - 1, n) == B.GTA_ERR_INVALID_ARG              # fewer keys than queries
    assert chunk(good, n + 8, n + 4) == B.GTA_ERR_INVALID_ARG          # more keys than the buffers hold
    assert L.gta_prefill_chunk(None, 8, 8, *args, p, 1 << 40, None, None) == B.GTA_ERR_INVALID_ARG
    assert chunk(_shape(B, seq=0), 16, 16) == B.GTA_OK                 # no queries: no-op

    def decode(shape, s_cap=128, ws=p, ws_bytes=1 << 40, lens=p):
        return L.gta_decode(ctypes.byref(shape), p, p, p, lens, s_cap, p, p, p, p, ws, ws_bytes, None, None)

    assert decode(good, s_cap=-1) == B.GTA_ERR_INVALID_ARG
    assert decode(good, lens=None) == B.GTA_ERR_INVALID_ARG
    assert decode(good, ws_bytes=8) == B.GTA_ERR_WORKSPACE
    assert decode(_shape(B, d_l=4096)) == B.GTA_ERR_UNSUPPORTED
    assert decode(_shape(B, batch=0)) == B.GTA_OK

    def decode_host(shape, s_cap=128, ws=p, ws_bytes=1 << 40, lens=p):
        return L.gta_decode_hostcache(ctypes.byref(shape), p, p, p, lens, s_cap, p, p, p, p, ws, ws_bytes, None, None)

    assert decode_host(good, s_cap=-1) == B.GTA_ERR_INVALID_ARG
    assert decode_host(good, lens=None) == B.GTA_ERR_INVALID_ARG
    assert decode_host(good, ws_bytes=8) == B.GTA_ERR_WORKSPACE
    assert decode_host(_shape(B, batch=0)) == B.GTA_OK
    assert B.decode_hostcache_workspace_bytes(good, 1000) > 0

    def append(shape, n_new=1, lens=p):
        return L.gta_cache_append(ctypes.byref(shape), p, p, 128, p, p, n_new, lens, None, None)

    assert append(good, n_new=-1) == B.GTA_ERR_INVALID_ARG
    assert append(good, lens=None) == B.GTA_ERR_INVALID_ARG
    assert append(good, n_new=0) == B.GTA_OK

    def decode_paged(shape, table=p, page_size=64, n_pages=10, max_pages=4, ws_bytes=1 << 40):
        return L.gta_decode_paged(ctypes.byref(shape), p, p, p, table, page_size, n_pages, max_pages, p, p, p, p, p,
                                  p, ws_bytes, None, None)

    assert decode_paged(good, table=None) == B.GTA_ERR_INVALID_ARG
    assert decode_paged(good, table=odd) == B.GTA_ERR_INVALID_ARG
    assert decode_paged(good, page_size=0) == B.GTA_ERR_INVALID_ARG
    assert decode_paged(good, n_pages=0) == B.GTA_ERR_INVALID_ARG
    assert decode_paged(good, max_pages=-3) == B.GTA_ERR_INVALID_ARG
    assert decode_paged(good, page_size=1 << 20, max_pages=1 << 12) == B.GTA_ERR_INVALID_ARG   # capacity over int32
    assert decode_paged(good, ws_bytes=8) == B.GTA_ERR_WORKSPACE
    assert decode_paged(_shape(B, batch=0)) == B.GTA_OK
    assert B.decode_paged_workspace_bytes(good, 64, 4) == B.decode_workspace_bytes(good, 256)
    assert B.decode_paged_workspace_bytes(good, 0, 4) == 0

    def layer_prefill(shape, pos0=0, s_cap=128, base=10000.0, ws_bytes=1 << 40):
        return L.gta_layer_prefill(ctypes.byref(shape), pos0, s_cap, ctypes.c_float(base), p, p, p, p, p, p, p, p, p,
                                   ws_bytes, None, None)

    lay = _shape(B, d_model=128, n_heads=4, n_q=2, n_k=2, n_c=1, d_h=64, d_l=128)     # (2 + 2) 64 + 128 = 384 columns
    assert layer_prefill(lay, pos0=-1) == B.GTA_ERR_INVALID_ARG
    assert layer_prefill(lay, pos0=65) == B.GTA_ERR_INVALID_ARG           # 65 + 64 tokens do not fit 128 rows
    assert layer_prefill(lay, base=1.0) == B.GTA_ERR_INVALID_ARG
    assert layer_prefill(_shape(B, d_model=128, n_heads=4, n_q=2, n_k=2, n_c=1, d_h=64, d_l=128, causal=0)) \
        == B.GTA_ERR_INVALID_ARG
    assert layer_prefill(_shape(B, d_model=128, n_heads=4, n_q=2, n_k=1, n_c=1, d_h=64, d_l=128)) \
        == B.GTA_ERR_UNSUPPORTED                                          # 320 projection columns: no multiple of 128
    assert layer_prefill(_shape(B, d_model=128, n_heads=4, n_q=2, n_k=2, n_c=1, d_h=64, d_l=128, dtype=B.GTA_F32)) \
        == B.GTA_ERR_UNSUPPORTED
    assert layer_prefill(lay, ws_bytes=8) == B.GTA_ERR_WORKSPACE
    assert layer_prefill(_shape(B, d_model=128, n_heads=4, n_q=2, n_k=2, n_c=1, d_h=64, d_l=128, seq=0)) == B.GTA_OK
    assert B.layer_prefill_workspace_bytes(lay) > B.prefill_workspace_bytes(lay)

    def layer_decode(shape, s_cap=128, base=10000.0, lens=p, ws_bytes=1 << 40):
        return L.gta_layer_decode(ctypes.byref(shape), s_cap, ctypes.c_float(base), p, p, p, p, p, p, p, lens, p, p,
                                  ws_bytes, None, None)

    assert layer_decode(lay, s_cap=0) == B.GTA_ERR_INVALID_ARG
    assert layer_decode(lay, base=0.5) == B.GTA_ERR_INVALID_ARG
    assert layer_decode(lay, lens=None) == B.GTA_ERR_INVALID_ARG
    assert layer_decode(lay, ws_bytes=8) == B.GTA_ERR_WORKSPACE
    assert layer_decode(_shape(B, d_model=128, n_heads=4, n_q=2, n_k=2, n_c=1, d_h=64, d_l=128, batch=0)) == B.GTA_OK
    assert L.gta_layer_decode_paged(ctypes.byref(lay), None, 64, 10, 4, ctypes.c_float(1e4), p, p, p, p, p, p, p, p, p,
                                    p, 1 << 40, None, None) == B.GTA_ERR_INVALID_ARG
    assert L.gta_layer_decode_paged(ctypes.byref(lay), p, 0, 10, 4, ctypes.c_float(1e4), p, p, p, p, p, p, p, p, p,
                                    p, 1 << 40, None, None) == B.GTA_ERR_INVALID_ARG
    assert B.layer_decode_paged_workspace_bytes(lay, 64, 2) == B.layer_decode_workspace_bytes(lay, 128)

    def append_paged(shape, table=p, page_size=64, n_new=1):
        return L.gta_cache_append_paged(ctypes.byref(shape), p, p, table, page_size, 10, 4, p, p, n_new, p, None, None)

    assert append_paged(good, table=None) == B.GTA_ERR_INVALID_ARG
    assert append_paged(good, page_size=-1) == B.GTA_ERR_INVALID_ARG
    assert append_paged(good, n_new=-1) == B.GTA_ERR_INVALID_ARG
    assert append_paged(good, n_new=0) == B.GTA_OK

    def chunk_paged(shape, kv_len, table=p, page_size=64, n_pages=10, max_pages=4, ws_bytes=1 << 40):
        return L.gta_prefill_chunk_paged(ctypes.byref(shape), kv_len, p, p, p, table, page_size, n_pages, max_pages,
                                         p, p, p, p, p, ws_bytes, None, None)

    assert chunk_paged(good, n, table=None) == B.GTA_ERR_INVALID_ARG
    assert chunk_paged(good, n, table=odd) == B.GTA_ERR_INVALID_ARG
    assert chunk_paged(good, n, page_size=0) == B.GTA_ERR_INVALID_ARG
    assert chunk_paged(good, n - 1) == B.GTA_ERR_INVALID_ARG             # fewer keys than queries
    assert chunk_paged(good, 64 * 4 + 1) == B.GTA_ERR_INVALID_ARG        # more keys than the block table covers
    assert chunk_paged(good, n, ws_bytes=8) == B.GTA_ERR_WORKSPACE
    assert chunk_paged(_shape(B, seq=0), 16) == B.GTA_OK                 # no queries: no-op
    assert L.gta_prefill_chunk_paged(None, 8, p, p, p, p, 64, 10, 4, p, p, p, p, p, 1 << 40, None,
                                     None) == B.GTA_ERR_INVALID_ARG

    def layer_prefill_paged(shape, pos0=0, table=p, page_size=64, max_pages=2, base=10000.0, ws_bytes=1 << 40):
        return L.gta_layer_prefill_paged(ctypes.byref(shape), pos0, ctypes.c_float(base), p, p, p, p, p, p, p, table,
                                         page_size, 10, max_pages, p, p, ws_bytes, None, None)

    assert layer_prefill_paged(lay, table=None) == B.GTA_ERR_INVALID_ARG
    assert layer_prefill_paged(lay, page_size=-4) == B.GTA_ERR_INVALID_ARG
    assert layer_prefill_paged(lay, pos0=65) == B.GTA_ERR_INVALID_ARG     # 65 + 64 tokens do not fit two pages
    assert layer_prefill_paged(lay, base=1.0) == B.GTA_ERR_INVALID_ARG
    assert layer_prefill_paged(lay, ws_bytes=8) == B.GTA_ERR_WORKSPACE


def test_binding_rejects_cpu_tensors_and_missing_library(B, monkeypatch):
    import torch
    t = torch.zeros(1, 1, 8, 8)
    with pytest.raises(ValueError):
        B.gta_prefill(t, t, t, torch.zeros(1, 8, 8), torch.zeros(1, 8, 8), torch.zeros(8, 8))
    monkeypatch.setattr(B, "_lib", None)
    monkeypatch.setattr(B, "LIB_PATH", os.path.join(ROOT, "does_not_exist.so"))
    with pytest.raises(RuntimeError, match="no CPU or PyTorch fallback"):
        B.lib()
