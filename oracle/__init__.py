"""ctypes front end of the fp64 CPU oracle (``pda_oracle.cpp``).

TEST INFRASTRUCTURE ONLY: imported by the tests, the smoke check and the
benchmark's CPU-baseline / reference legs. Nothing here touches CUDA, and the
CUDA package never imports this module.

Arrays are numpy: bf16 data as ``uint16`` bit patterns, e4m3 data as ``uint8``.
Caches are ``[num_pages, Hkv, P, D]`` arrays (any strides with a unit inner
stride are accepted; strides are passed on in elements).
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "pda_oracle.cpp")
_LIB = os.path.join(_HERE, "libpda_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with g++ (no fast-math) into ``libpda_oracle.so``."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = f"{_LIB}.{os.getpid()}.tmp"
        subprocess.check_call(
            ["g++", "-O2", "-std=c++17", "-fPIC", "-shared", "-pthread", "-o", tmp, _SRC])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.oracle_hardware_threads.restype = C.c_int
    return _lib


def hardware_threads() -> int:
    return int(_load().oracle_hardware_threads())


def _p(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _cache_strides(cache: np.ndarray):
    assert cache.ndim == 4, "cache must be [num_pages, Hkv, P, D]"
    es = cache.itemsize
    st = [s // es for s in cache.strides]
    assert st[3] == 1, "inner (head_dim) stride must be 1"
    return st[0], st[1], st[2]


def e4m3_decode_table() -> np.ndarray:
    t = np.empty(256, dtype=np.float64)
    _load().oracle_e4m3_decode_table(_p(t))
    return t


def kv_append(k_new, v_new, k_cache, v_cache, block_table, seq_lens):
    """In-place append into ``k_cache``/``v_cache`` (uint16 views of bf16)."""
    assert k_cache.dtype == np.uint16 and v_cache.dtype == np.uint16
    assert k_new.dtype == np.uint16 and v_new.dtype == np.uint16
    k_new = np.ascontiguousarray(k_new)
    v_new = np.ascontiguousarray(v_new)
    block_table = np.ascontiguousarray(block_table, dtype=np.int32)
    seq_lens = np.ascontiguousarray(seq_lens, dtype=np.int32)
    ps, hs, ss = _cache_strides(k_cache)
    assert (ps, hs, ss) == _cache_strides(v_cache)
    _, Hkv, P, D = k_cache.shape
    B = seq_lens.shape[0]
    _load().oracle_kv_append(
        _p(k_new), _p(v_new), _p(k_cache), _p(v_cache), C.c_int64(ps), C.c_int64(hs),
        C.c_int64(ss), C.c_int32(P), C.c_int32(Hkv), C.c_int32(D), C.c_int32(2),
        _p(block_table), C.c_int32(block_table.shape[1]), _p(seq_lens), C.c_int32(B))


def paged_decode_attention(q, k_cache, v_cache, block_table, seq_lens, scale,
                           k_scale=None, v_scale=None, chunk_tokens=0, max_chunks=0,
                           n_threads=0, window=0):
    """Returns ``(out, lse)`` in float64.

    ``window > 0`` attends only each sequence's last ``window`` tokens.
    Unsplit: ``out [B,Hq,D]``, ``lse [B,Hq]``. Split (``chunk_tokens > 0``):
    ``out [B,Hq,max_chunks,D]`` (NaN where no chunk exists) and
    ``lse [B,Hq,max_chunks]`` (NaN likewise).
    """
    q = np.ascontiguousarray(q)
    assert q.dtype == np.uint16 and q.ndim == 3
    B, Hq, D = q.shape
    if k_cache.dtype == np.uint16:
        dtype = 0
    elif k_cache.dtype == np.uint8:
        dtype = 1
        assert k_scale is not None and v_scale is not None
        k_scale = np.ascontiguousarray(k_scale, dtype=np.float32)
        v_scale = np.ascontiguousarray(v_scale, dtype=np.float32)
    else:
        raise TypeError("cache dtype must be uint16 (bf16 bits) or uint8 (e4m3)")
    assert v_cache.dtype == k_cache.dtype
    ps, hs, ss = _cache_strides(k_cache)
    assert (ps, hs, ss) == _cache_strides(v_cache)
    _, Hkv, P, Dc = k_cache.shape
    assert Dc == D and Hq % Hkv == 0
    block_table = np.ascontiguousarray(block_table, dtype=np.int32)
    seq_lens = np.ascontiguousarray(seq_lens, dtype=np.int32)
    assert seq_lens.shape[0] == B and block_table.shape[0] == B
    if chunk_tokens == 0:
        out = np.zeros((B, Hq, D), dtype=np.float64)
        lse = np.zeros((B, Hq), dtype=np.float64)
    else:
        assert max_chunks > 0
        out = np.full((B, Hq, max_chunks, D), np.nan, dtype=np.float64)
        lse = np.full((B, Hq, max_chunks), np.nan, dtype=np.float64)
    if n_threads <= 0:
        n_threads = hardware_threads()
    _load().oracle_paged_decode_attention(
        _p(q), _p(k_cache), _p(v_cache), C.c_int32(dtype), _p(k_scale), _p(v_scale),
        C.c_int64(ps), C.c_int64(hs), C.c_int64(ss), C.c_int32(P), C.c_int32(Hkv),
        C.c_int32(D), _p(block_table), C.c_int32(block_table.shape[1]), _p(seq_lens),
        C.c_int32(B), C.c_int32(Hq), C.c_float(np.float32(scale)), C.c_int32(chunk_tokens),
        C.c_int32(max_chunks), C.c_int32(window), _p(out), _p(lse), C.c_int32(n_threads))
    return out, lse


def kv_append_tokens(k_new, v_new, k_cache, v_cache, block_table, seq_lens):
    """In-place append of ``n_new`` tokens per sequence; ``k_new`` is ``[B,n_new,Hkv,D]``."""
    assert k_cache.dtype == np.uint16 and k_new.dtype == np.uint16 and k_new.ndim == 4
    k_new, v_new = np.ascontiguousarray(k_new), np.ascontiguousarray(v_new)
    block_table = np.ascontiguousarray(block_table, dtype=np.int32)
    seq_lens = np.ascontiguousarray(seq_lens, dtype=np.int32)
    ps, hs, ss = _cache_strides(k_cache)
    _, Hkv, P, D = k_cache.shape
    _load().oracle_kv_append_tokens(
        _p(k_new), _p(v_new), _p(k_cache), _p(v_cache), C.c_int64(ps), C.c_int64(hs),
        C.c_int64(ss), C.c_int32(P), C.c_int32(Hkv), C.c_int32(D), C.c_int32(2),
        _p(block_table), C.c_int32(block_table.shape[1]), _p(seq_lens),
        C.c_int32(seq_lens.shape[0]), C.c_int32(k_new.shape[1]))


def kv_append_e4m3(k_new, v_new, k_cache, v_cache, k_scale, v_scale, block_table, seq_lens):
    """In-place quantising append into uint8 (e4m3) caches and their fp32 scale arrays."""
    assert k_cache.dtype == np.uint8 and v_cache.dtype == np.uint8 and k_new.dtype == np.uint16
    assert k_scale.dtype == np.float32 and k_scale.flags.c_contiguous and v_scale.flags.c_contiguous
    k_new, v_new = np.ascontiguousarray(k_new), np.ascontiguousarray(v_new)
    block_table = np.ascontiguousarray(block_table, dtype=np.int32)
    seq_lens = np.ascontiguousarray(seq_lens, dtype=np.int32)
    ps, hs, ss = _cache_strides(k_cache)
    _, Hkv, P, D = k_cache.shape
    _load().oracle_kv_append_e4m3(
        _p(k_new), _p(v_new), _p(k_cache), _p(v_cache), _p(k_scale), _p(v_scale), C.c_int64(ps),
        C.c_int64(hs), C.c_int64(ss), C.c_int32(P), C.c_int32(Hkv), C.c_int32(D), _p(block_table),
        C.c_int32(block_table.shape[1]), _p(seq_lens), C.c_int32(seq_lens.shape[0]))


def kv_append_tokens_e4m3(k_new, v_new, k_cache, v_cache, k_scale, v_scale, block_table, seq_lens):
    """In-place quantising append of ``k_new, v_new [B,T,Hkv,D]`` (bf16 bits): the one-token rule of
    ``kv_append_e4m3`` applied to the block's tokens in order (``seq_lens`` = lengths after the append)."""
    assert k_cache.dtype == np.uint8 and v_cache.dtype == np.uint8 and k_new.dtype == np.uint16
    assert k_new.ndim == 4 and k_scale.dtype == np.float32 and k_scale.flags.c_contiguous and v_scale.flags.c_contiguous
    k_new, v_new = np.ascontiguousarray(k_new), np.ascontiguousarray(v_new)
    block_table = np.ascontiguousarray(block_table, dtype=np.int32)
    seq_lens = np.ascontiguousarray(seq_lens, dtype=np.int32)
    ps, hs, ss = _cache_strides(k_cache)
    _, Hkv, P, D = k_cache.shape
    _load().oracle_kv_append_tokens_e4m3(
        _p(k_new), _p(v_new), _p(k_cache), _p(v_cache), _p(k_scale), _p(v_scale), C.c_int64(ps),
        C.c_int64(hs), C.c_int64(ss), C.c_int32(P), C.c_int32(Hkv), C.c_int32(D), _p(block_table),
        C.c_int32(block_table.shape[1]), _p(seq_lens), C.c_int32(seq_lens.shape[0]), C.c_int32(k_new.shape[1]))


def paged_verify_attention(q, k_cache, v_cache, block_table, seq_lens, scale,
                           k_scale=None, v_scale=None, n_threads=0):
    """Causal attention of a block of query tokens: ``q [B,T,Hq,D]`` -> ``(out, lse)`` fp64;
    query ``i`` attends tokens ``j <= L - T + i`` (the cache already holds the block)."""
    q = np.ascontiguousarray(q)
    assert q.dtype == np.uint16 and q.ndim == 4
    B, T, Hq, D = q.shape
    dtype = 0 if k_cache.dtype == np.uint16 else 1
    if dtype == 1:
        k_scale = np.ascontiguousarray(k_scale, dtype=np.float32)
        v_scale = np.ascontiguousarray(v_scale, dtype=np.float32)
    ps, hs, ss = _cache_strides(k_cache)
    _, Hkv, P, _ = k_cache.shape
    block_table = np.ascontiguousarray(block_table, dtype=np.int32)
    seq_lens = np.ascontiguousarray(seq_lens, dtype=np.int32)
    out = np.zeros((B, T, Hq, D), dtype=np.float64)
    lse = np.zeros((B, T, Hq), dtype=np.float64)
    if n_threads <= 0:
        n_threads = hardware_threads()
    _load().oracle_paged_verify_attention(
        _p(q), _p(k_cache), _p(v_cache), C.c_int32(dtype), _p(k_scale), _p(v_scale),
        C.c_int64(ps), C.c_int64(hs), C.c_int64(ss), C.c_int32(P), C.c_int32(Hkv), C.c_int32(D),
        _p(block_table), C.c_int32(block_table.shape[1]), _p(seq_lens), C.c_int32(B),
        C.c_int32(Hq), C.c_int32(T), C.c_float(np.float32(scale)), _p(out), _p(lse),
        C.c_int32(n_threads))
    return out, lse


def paged_decode_reduce(part_o, part_lse, seq_lens, chunk_tokens):
    """Merge ``[B,Hq,C,D]`` / ``[B,Hq,C]`` partials; returns ``(out, lse)`` fp64."""
    part_o = np.ascontiguousarray(part_o, dtype=np.float64)
    part_lse = np.ascontiguousarray(part_lse, dtype=np.float64)
    seq_lens = np.ascontiguousarray(seq_lens, dtype=np.int32)
    B, Hq, Cm, D = part_o.shape
    out = np.zeros((B, Hq, D), dtype=np.float64)
    lse = np.zeros((B, Hq), dtype=np.float64)
    _load().oracle_paged_decode_reduce(
        _p(part_o), _p(part_lse), _p(seq_lens), C.c_int32(B), C.c_int32(Hq), C.c_int32(D),
        C.c_int32(chunk_tokens), C.c_int32(Cm), _p(out), _p(lse))
    return out, lse


def quantize_pages_e4m3(src_bf16_bits, valid_slots):
    """Quantise a contiguous bf16 ``[num_pages,Hkv,P,D]`` cache per (page, head).

    Returns ``(bytes uint8 [num_pages,Hkv,P,D], scales fp32 [num_pages,Hkv])``;
    slots at or beyond ``valid_slots[page]`` are zero bytes.
    """
    src = np.ascontiguousarray(src_bf16_bits)
    assert src.dtype == np.uint16 and src.ndim == 4
    n, Hkv, P, D = src.shape
    valid_slots = np.ascontiguousarray(valid_slots, dtype=np.int32)
    dst = np.zeros(src.shape, dtype=np.uint8)
    scales = np.ones((n, Hkv), dtype=np.float32)
    _load().oracle_quantize_pages_e4m3(
        _p(src), _p(valid_slots), C.c_int32(n), C.c_int32(Hkv), C.c_int32(P), C.c_int32(D),
        _p(dst), _p(scales))
    return dst, scales
