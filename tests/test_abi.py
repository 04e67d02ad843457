"""CPU-only checks of the C-ABI library: it loads without a GPU, exports every
symbol include/pda.h declares, and its host-side validation rejects bad
arguments before anything is enqueued."""
import ctypes as C
import os
import re

import pytest

from paper_2605_06068_b200 import binding as pda
from paper_2605_06068_b200 import build as pda_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    pda_build.build()
    return pda.lib()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "pda.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    names = re.findall(r"^\s*(?:const\s+)?[A-Za-z_][\w\s\*]*?\b(\w+)\s*\([^;{]*\)\s*;", text, flags=re.M)
    return sorted(set(names))


def test_every_declared_symbol_is_exported(lib):
    names = declared_functions()
    assert set(pda.EXPORTS) == set(names), (names, pda.EXPORTS)
    for n in names:
        assert getattr(lib, n) is not None


def test_version_and_strings(lib):
    assert lib.pda_version() == 100
    assert pda.status_string(0) == "ok"
    assert "align" in pda.status_string(-3)
    assert pda.max_chunks(131072, 2048) == 64 and pda.max_chunks(1, 2048) == 1
    assert pda.max_chunks(0, 16) == 0 and pda.max_chunks(5, 0) == -1


def desc(**kw):
    d = dict(page_stride=8 * 16 * 128, head_stride=16 * 128, slot_stride=128, num_pages=10,
             page_size=16, num_kv_heads=8, head_dim=128, dtype=0)
    d.update(kw)
    return pda.CacheDesc(**d)


def call_attention(lib, d, q=0x1000, k=0x2000, v=0x3000, bt=0x4000, sl=0x5000, out=0x6000,
                   batch=1, hq=32, chunk=0, po=None, pl=None, mc=0, ks=None, vs=None, bts=4):
    return lib.paged_decode_attention(q, k, v, C.byref(d), ks, vs, bt, bts, sl, batch, hq, 0.1,
                                      chunk, out, po, pl, mc, 0, None, None)


def test_attention_validation_without_a_gpu(lib):
    # every call below must be refused on the host (fake non-null pointers are never dereferenced)
    assert call_attention(lib, desc(page_size=32)) == -2
    assert call_attention(lib, desc(head_dim=100, slot_stride=100)) == -2
    assert call_attention(lib, desc(head_dim=512, slot_stride=512)) == -2
    assert call_attention(lib, desc(dtype=7)) == -2
    assert call_attention(lib, desc(), hq=30) == -1            # not a multiple of kv heads
    assert call_attention(lib, desc(), q=None) == -1
    assert call_attention(lib, desc(), out=None) == -1
    assert call_attention(lib, desc(), q=0x1008) == -3
    assert call_attention(lib, desc(slot_stride=132)) == -3     # 264-byte rows
    assert call_attention(lib, desc(slot_stride=64)) == -1      # rows overlap
    assert call_attention(lib, desc(), chunk=24, po=0x7000, pl=0x8000, mc=4) == -1
    assert call_attention(lib, desc(), chunk=32) == -1          # partial buffers missing
    assert call_attention(lib, desc(dtype=1)) == -1             # e4m3 without scales
    assert call_attention(lib, desc(), batch=-1) == -1
    assert call_attention(lib, desc(), batch=70000) == -4
    assert call_attention(lib, desc(), bts=0) == -1
    assert call_attention(lib, desc(), batch=0) == 0            # empty batch: nothing to do


def test_append_and_reduce_validation_without_a_gpu(lib):
    d = desc()
    assert lib.kv_append(0x1000, 0x2000, 0x3000, 0x4000, C.byref(d), 0x5000, 4, 0x6000, 0, None, None) == 0
    assert lib.kv_append(None, 0x2000, 0x3000, 0x4000, C.byref(d), 0x5000, 4, 0x6000, 2, None, None) == -1
    assert lib.kv_append(0x1004, 0x2000, 0x3000, 0x4000, C.byref(d), 0x5000, 4, 0x6000, 2, None, None) == -3
    d8 = desc(dtype=1)
    assert lib.kv_append(0x1000, 0x2000, 0x3000, 0x4000, C.byref(d8), 0x5000, 4, 0x6000, 2, None, None) == -2
    assert lib.kv_append(0x1000, 0x2000, 0x3000, 0x4000, None, 0x5000, 4, 0x6000, 2, None, None) == -1
    assert lib.paged_decode_reduce(0x1000, 0x2000, 0x3000, 0, 8, 128, 16, 4, 0x4000, None) == 0
    assert lib.paged_decode_reduce(None, 0x2000, 0x3000, 1, 8, 128, 16, 4, 0x4000, None) == -1
    assert lib.paged_decode_reduce(0x1000, 0x2000, 0x3000, 1, 8, 128, 0, 4, 0x4000, None) == -1
    assert lib.pda_debug_e4m3_decode(None, None) == -1


def test_missing_library_fails_loudly(monkeypatch):
    monkeypatch.setattr(pda, "_lib", None)
    monkeypatch.setattr(pda, "LIB_PATH", "/nonexistent/libpda.so")
    with pytest.raises(RuntimeError, match="no CPU or PyTorch fallback"):
        pda.lib()


def test_new_entry_points_validate_without_a_gpu(lib):
    d = desc()
    P = 0x1000
    # paged_decode_step: k_new without v_new, missing out, e4m3 cache with an append
    step = lambda **kw: lib.paged_decode_step(
        kw.get("q", P), kw.get("kn", P), kw.get("vn", P), P, P, C.byref(kw.get("d", d)), None, None, P, 4, P,
        kw.get("batch", 1), 32, 0.1, kw.get("chunk", 0), kw.get("out", P), None, None, 0, None, None, None)
    assert step(vn=None) == -1
    assert step(out=None) == -1
    assert step(batch=0) == 0
    assert step(chunk=8) == -1
    # window must be non-negative
    assert lib.paged_window_decode_attention(P, P, P, C.byref(d), None, None, P, 4, P, 1, 32, 0.1, -1, 0,
                                             P, None, None, 0, 0, None, None) == -1
    # verify: token count, batch * tokens limit
    ver = lambda T, batch=1: lib.paged_verify_attention(P, P, P, C.byref(d), None, None, P, 4, P, batch, 32, T,
                                                        0.1, 0, P, None, None, 0, 0, None, None)
    assert ver(0) == -1 and ver(5000) == -1 and ver(16, batch=5000) == -4 and ver(16, batch=0) == 0
    # shared prefix: prefix must be page-aligned, chunks positive, max_chunks must leave room for suffixes
    pre = lambda prefix, pchunk, chunk, mc: lib.paged_prefix_decode_attention(
        P, P, P, C.byref(d), None, None, P, 64, P, 2, 32, 0.1, prefix, pchunk, chunk, P, P, P, mc, 0, None, None)
    assert pre(100, 64, 64, 8) == -1
    assert pre(128, 0, 64, 8) == -1
    assert pre(128, 64, 0, 8) == -1
    assert pre(128, 64, 64, 2) == -1
    assert pre(4096, 64, 64, 100) == -1       # prefix longer than the block table can hold
    # fp8 append needs an e4m3 cache and both scale arrays
    assert lib.kv_append_fp8(P, P, P, P, C.byref(d), P, P, P, 4, P, 1, None, None) == -2
    d8 = desc(dtype=1, page_stride=8 * 16 * 128, head_stride=16 * 128)
    assert lib.kv_append_fp8(P, P, P, P, C.byref(d8), None, P, P, 4, P, 1, None, None) == -1
    assert lib.kv_append_tokens(P, P, P, P, C.byref(d), P, 4, P, 1, -1, None, None) == -1
    assert lib.kv_append_tokens(P, P, P, P, C.byref(d), P, 4, P, 1, 0, None, None) == 0
    assert lib.pda_workspace_ints(64, 8) == 514 and lib.pda_workspace_ints(-1, 8) == -1
    assert lib.pda_advance_seq_lens(None, 4, 1, None) == -1 and lib.pda_advance_seq_lens(None, 0, 1, None) == 0
    # the allocation-free entry point rejects oversize problems before touching the device
    assert lib.paged_decode_attention_static(P, P, P, C.byref(d), None, None, P, 4, P, 64, 32, 0.1, 16,
                                             4096, P, None, None) == -4


def test_diagnostic_calls_check_their_arguments_without_a_gpu(lib):
    assert lib.pda_debug_wait_timeout(0, 0x1000, None, None) == -1
    assert lib.pda_debug_wait_timeout((1 << 20) + 1, 0x1000, None, None) == -1
    assert lib.pda_debug_wait_timeout(100, None, None, None) == -1
    assert lib.pda_debug_wait_timeout(100, 0x1000, 0x2004, None) == -3
    assert lib.pda_debug_read_probe(None, 1 << 20, 0x1000, None) == -1
    assert lib.pda_debug_read_probe(0x1000, 24, 0x2000, None) == -1
    assert lib.pda_debug_read_probe(0x1008, 32, 0x2000, None) == -3
