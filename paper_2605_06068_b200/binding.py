"""ctypes binding of ``libpda.so`` with the C ABI's own names.

Argument marshalling only: tensors are torch CUDA tensors whose ``data_ptr``s,
shapes and strides are passed straight to the C entry points declared in
``include/pda.h``. There is no fallback: if the library is missing or a call
fails, a ``RuntimeError`` is raised.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libpda.so")

PDA_BF16, PDA_FP8_E4M3 = 0, 1
PDA_FLAG_FORCE_GENERIC = 1
PDA_FLAG_MQ_MMA_SYNC = 2
PDA_FLAG_MQ_ONE_UNIT = 4
DEV_STATUS = {0: "ok", 1: "bad page id", 2: "seq_len exceeds block table", 3: "copy wait timed out"}

EXPORTS = ["pda_version", "pda_status_string", "pda_max_chunks", "kv_append",
           "paged_decode_attention", "paged_decode_reduce", "paged_decode_step_host",
           "pda_debug_e4m3_decode", "paged_decode_attention_static", "pda_workspace_ints",
           "paged_decode_step", "pda_advance_seq_lens", "paged_window_decode_attention", "kv_append_tokens",
           "paged_verify_attention", "paged_prefix_decode_attention", "kv_append_fp8", "kv_append_tokens_fp8",
           "pda_set_persistent_threshold", "pda_debug_wait_timeout", "pda_debug_read_probe"]
STATIC_SCRATCH_BYTES = 16 * 1024 * 1024


class CacheDesc(C.Structure):
    _fields_ = [("page_stride", C.c_int64), ("head_stride", C.c_int64), ("slot_stride", C.c_int64),
                ("num_pages", C.c_int32), ("page_size", C.c_int32), ("num_kv_heads", C.c_int32),
                ("head_dim", C.c_int32), ("dtype", C.c_int32)]


_lib = None


def lib():
    """Loads ``libpda.so`` on first use; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                f"{LIB_PATH} not found: build it with `python -m paper_2605_06068_b200.build` "
                "(there is no CPU or PyTorch fallback)")
        L = C.CDLL(LIB_PATH)
        L.pda_status_string.restype = C.c_char_p
        L.pda_status_string.argtypes = [C.c_int]
        vp, i32, f32, u32 = C.c_void_p, C.c_int32, C.c_float, C.c_uint32
        dp = C.POINTER(CacheDesc)
        L.pda_max_chunks.argtypes = [i32, i32]
        L.kv_append.argtypes = [vp, vp, vp, vp, dp, vp, i32, vp, i32, vp, vp]
        L.paged_decode_attention.argtypes = [vp, vp, vp, dp, vp, vp, vp, i32, vp, i32, i32, f32,
                                             i32, vp, vp, vp, i32, u32, vp, vp]
        L.paged_decode_reduce.argtypes = [vp, vp, vp, i32, i32, i32, i32, i32, vp, vp]
        L.paged_decode_step_host.argtypes = [vp] * 5 + [vp] * 5 + [vp, vp, dp, i32, i32, i32, f32,
                                                                 i32, vp, vp, i32, vp, vp, vp, vp, vp]
        L.pda_workspace_ints.argtypes = [i32, i32]
        L.pda_set_persistent_threshold.argtypes = [i32]
        L.kv_append_fp8.argtypes = [vp, vp, vp, vp, dp, vp, vp, vp, i32, vp, i32, vp, vp]
        L.kv_append_tokens_fp8.argtypes = [vp, vp, vp, vp, dp, vp, vp, vp, i32, vp, i32, i32, vp, vp]
        L.kv_append_tokens.argtypes = [vp, vp, vp, vp, dp, vp, i32, vp, i32, i32, vp, vp]
        L.paged_verify_attention.argtypes = [vp, vp, vp, dp, vp, vp, vp, i32, vp, i32, i32, i32, f32,
                                             i32, vp, vp, vp, i32, u32, vp, vp]
        L.paged_prefix_decode_attention.argtypes = [vp, vp, vp, dp, vp, vp, vp, i32, vp, i32, i32, f32,
                                                    i32, i32, i32, vp, vp, vp, i32, u32, vp, vp]
        L.paged_window_decode_attention.argtypes = [vp, vp, vp, dp, vp, vp, vp, i32, vp, i32, i32, f32,
                                                    i32, i32, vp, vp, vp, i32, u32, vp, vp]
        L.pda_advance_seq_lens.argtypes = [vp, i32, i32, vp]
        L.paged_decode_step.argtypes = [vp, vp, vp, vp, vp, dp, vp, vp, vp, i32, vp, i32, i32, f32,
                                        i32, vp, vp, vp, i32, vp, vp, vp]
        L.pda_debug_e4m3_decode.argtypes = [vp, vp]
        L.pda_debug_wait_timeout.argtypes = [u32, vp, vp, vp]
        L.pda_debug_read_probe.argtypes = [vp, C.c_uint64, vp, vp]
        L.paged_decode_attention_static.argtypes = [vp, vp, vp, dp, vp, vp, vp, i32, vp, i32, i32,
                                                    f32, i32, i32, vp, vp, vp]
        _lib = L
    return _lib


def status_string(code: int) -> str:
    return lib().pda_status_string(int(code)).decode()


def _check(rc: int, what: str):
    if rc != 0:
        raise RuntimeError(f"{what} failed with code {rc}: {status_string(rc)}")


def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


_raw_stream = getattr(torch._C, "_cuda_getCurrentRawStream", None)


def _stream(stream):
    if stream is not None:
        return C.c_void_p(stream.cuda_stream)
    if _raw_stream is not None:   # the current stream's handle without building a Stream object (~10x cheaper)
        return C.c_void_p(_raw_stream(torch.cuda.current_device()))
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def cache_desc(cache: torch.Tensor) -> CacheDesc:
    """Descriptor of a ``[num_pages, Hkv, P, D]`` cache tensor (bf16, or uint8 /
    float8_e4m3fn for e4m3)."""
    assert cache.dim() == 4 and cache.stride(3) == 1
    if cache.dtype == torch.bfloat16:
        dt = PDA_BF16
    elif cache.dtype in (torch.uint8, torch.float8_e4m3fn):
        dt = PDA_FP8_E4M3
    else:
        raise TypeError(f"unsupported cache dtype {cache.dtype}")
    n, Hkv, P, D = cache.shape
    return CacheDesc(cache.stride(0), cache.stride(1), cache.stride(2), n, P, Hkv, D, dt)


def max_chunks(max_seq_len: int, chunk_tokens: int) -> int:
    return int(lib().pda_max_chunks(max_seq_len, chunk_tokens))


def kv_append(k_new, v_new, k_cache, v_cache, block_table, seq_lens, status=None, stream=None):
    desc = cache_desc(k_cache)
    assert k_new.is_contiguous() and v_new.is_contiguous() and block_table.stride(1) == 1
    assert v_cache.stride() == k_cache.stride() and v_cache.shape == k_cache.shape
    rc = lib().kv_append(_ptr(k_new), _ptr(v_new), _ptr(k_cache), _ptr(v_cache), C.byref(desc),
                         _ptr(block_table), block_table.stride(0), _ptr(seq_lens),
                         seq_lens.shape[0], _ptr(status), _stream(stream))
    _check(rc, "kv_append")


def paged_decode_attention(q, k_cache, v_cache, block_table, seq_lens, scale, chunk_tokens=0,
                           out=None, part_o=None, part_lse=None, k_scale=None, v_scale=None,
                           flags=0, status=None, stream=None):
    """Unsplit (``chunk_tokens == 0``): fills and returns ``out`` ``[B,Hq,D]`` bf16.
    Split: fills ``part_o`` ``[B,Hq,C,D]`` / ``part_lse`` ``[B,Hq,C]`` fp32 and returns them."""
    desc = cache_desc(k_cache)
    assert q.is_contiguous() and q.dtype == torch.bfloat16 and block_table.stride(1) == 1
    assert v_cache.stride() == k_cache.stride() and v_cache.shape == k_cache.shape
    B, Hq, D = q.shape
    mc = 0
    if chunk_tokens == 0:
        if out is None:
            out = torch.empty_like(q)
    else:
        assert part_o is not None and part_lse is not None
        assert part_o.is_contiguous() and part_lse.is_contiguous()
        mc = part_o.shape[2]
        assert tuple(part_o.shape) == (B, Hq, mc, D) and tuple(part_lse.shape) == (B, Hq, mc)
    rc = lib().paged_decode_attention(
        _ptr(q), _ptr(k_cache), _ptr(v_cache), C.byref(desc), _ptr(k_scale), _ptr(v_scale),
        _ptr(block_table), block_table.stride(0), _ptr(seq_lens), B, Hq, float(scale),
        chunk_tokens, _ptr(out), _ptr(part_o), _ptr(part_lse), mc, flags, _ptr(status),
        _stream(stream))
    _check(rc, "paged_decode_attention")
    return out if chunk_tokens == 0 else (part_o, part_lse)


def paged_window_decode_attention(q, k_cache, v_cache, block_table, seq_lens, scale, window,
                                  chunk_tokens=0, out=None, part_o=None, part_lse=None,
                                  k_scale=None, v_scale=None, flags=0, status=None, stream=None):
    """``paged_decode_attention`` over each sequence's last ``window`` tokens only."""
    desc = cache_desc(k_cache)
    B, Hq, D = q.shape
    mc = 0
    if chunk_tokens == 0:
        if out is None:
            out = torch.empty_like(q)
    else:
        mc = part_o.shape[2]
        assert tuple(part_o.shape) == (B, Hq, mc, D) and tuple(part_lse.shape) == (B, Hq, mc)
    rc = lib().paged_window_decode_attention(
        _ptr(q), _ptr(k_cache), _ptr(v_cache), C.byref(desc), _ptr(k_scale), _ptr(v_scale),
        _ptr(block_table), block_table.stride(0), _ptr(seq_lens), B, Hq, float(scale), int(window),
        chunk_tokens, _ptr(out), _ptr(part_o), _ptr(part_lse), mc, flags, _ptr(status),
        _stream(stream))
    _check(rc, "paged_window_decode_attention")
    return out if chunk_tokens == 0 else (part_o, part_lse)


def paged_decode_reduce(part_o, part_lse, seq_lens, chunk_tokens, out=None, stream=None):
    B, Hq, mc, D = part_o.shape
    if out is None:
        out = torch.empty((B, Hq, D), dtype=torch.bfloat16, device=part_o.device)
    rc = lib().paged_decode_reduce(_ptr(part_o), _ptr(part_lse), _ptr(seq_lens), B, Hq, D,
                                   chunk_tokens, mc, _ptr(out), _stream(stream))
    _check(rc, "paged_decode_reduce")
    return out


def workspace_ints(batch: int, num_kv_heads: int) -> int:
    return int(lib().pda_workspace_ints(batch, num_kv_heads))


def new_workspace(batch: int, num_kv_heads: int, device="cuda") -> torch.Tensor:
    """Zeroed int32 workspace for ``paged_decode_step`` (zero it once; calls leave it zeroed)."""
    return torch.zeros(workspace_ints(batch, num_kv_heads), dtype=torch.int32, device=device)


def paged_decode_step(q, k_new, v_new, k_cache, v_cache, block_table, seq_lens, scale,
                      chunk_tokens=0, out=None, part_o=None, part_lse=None, workspace=None,
                      k_scale=None, v_scale=None, status=None, stream=None):
    """Fused append + attention (+ reduce) in one launch; fills and returns ``out``."""
    desc = cache_desc(k_cache)
    assert q.is_contiguous() and q.dtype == torch.bfloat16 and block_table.stride(1) == 1
    B, Hq, D = q.shape
    if out is None:
        out = torch.empty_like(q)
    mc = 0
    if chunk_tokens:
        mc = part_o.shape[2]
        assert tuple(part_o.shape) == (B, Hq, mc, D) and tuple(part_lse.shape) == (B, Hq, mc)
    rc = lib().paged_decode_step(
        _ptr(q), _ptr(k_new), _ptr(v_new), _ptr(k_cache), _ptr(v_cache), C.byref(desc),
        _ptr(k_scale), _ptr(v_scale), _ptr(block_table), block_table.stride(0), _ptr(seq_lens),
        B, Hq, float(scale), chunk_tokens, _ptr(out), _ptr(part_o), _ptr(part_lse), mc,
        _ptr(workspace), _ptr(status), _stream(stream))
    _check(rc, "paged_decode_step")
    return out


def paged_decode_step_host(q_host, k_new_host, v_new_host, block_table_host, seq_lens_host,
                           q_dev, k_new_dev, v_new_dev, block_table_dev, seq_lens_dev,
                           k_cache, v_cache, scale, chunk_tokens, part_o, part_lse,
                           out_dev, out_host, workspace=None, status=None, stream=None):
    """Fused decode step from pinned host inputs to a host output. ``q_dev``, ``k_new_dev``,
    ``v_new_dev`` and ``out_dev`` may be None: the kernel then works on the pinned host buffers in
    place (see ``include/pda.h``)."""
    desc = cache_desc(k_cache)
    B, Hq, _ = q_host.shape
    mc = 0 if part_o is None else part_o.shape[2]
    rc = lib().paged_decode_step_host(
        _ptr(q_host), _ptr(k_new_host), _ptr(v_new_host), _ptr(block_table_host),
        _ptr(seq_lens_host), _ptr(q_dev), _ptr(k_new_dev), _ptr(v_new_dev), _ptr(block_table_dev),
        _ptr(seq_lens_dev), _ptr(k_cache), _ptr(v_cache), C.byref(desc),
        block_table_host.stride(0), B, Hq, float(scale), chunk_tokens, _ptr(part_o),
        _ptr(part_lse), mc, _ptr(workspace), _ptr(out_dev), _ptr(out_host), _ptr(status),
        _stream(stream))
    _check(rc, "paged_decode_step_host")
    return out_host


def debug_e4m3_decode(stream=None):
    out = torch.empty(256, dtype=torch.float32, device="cuda")
    _check(lib().pda_debug_e4m3_decode(_ptr(out), _stream(stream)), "pda_debug_e4m3_decode")
    return out


def paged_decode_attention_static(q, k_cache, v_cache, block_table, seq_lens, scale, chunk_tokens,
                                  max_chunks, out=None, k_scale=None, v_scale=None, status=None,
                                  stream=None):
    """Split-KV attention + reduce using the library's built-in scratch array, for
    callers that cannot allocate partial buffers (see ``include/pda.h``). ``out`` should
    be passed in by such callers; it is only created here as a convenience. Raises if
    ``batch*Hq*max_chunks*(D+1)*4`` bytes exceed ``STATIC_SCRATCH_BYTES``."""
    desc = cache_desc(k_cache)
    B, Hq, _ = q.shape
    if out is None:
        out = torch.empty_like(q)
    rc = lib().paged_decode_attention_static(
        _ptr(q), _ptr(k_cache), _ptr(v_cache), C.byref(desc), _ptr(k_scale), _ptr(v_scale),
        _ptr(block_table), block_table.stride(0), _ptr(seq_lens), B, Hq, float(scale),
        chunk_tokens, max_chunks, _ptr(out), _ptr(status), _stream(stream))
    _check(rc, "paged_decode_attention_static")
    return out


def debug_wait_timeout(polls, status, result=None, stream=None):
    """Runs the kernels' two bounded waits on a barrier nobody arrives at, with ``polls`` as the limit;
    ``status`` (int32[1]) receives PDA_DEV_TIMEOUT, ``result`` (int64[3]) the two durations in ns and the
    mask of waits that wrongly reported completion."""
    _check(lib().pda_debug_wait_timeout(int(polls), _ptr(status), _ptr(result), _stream(stream)),
           "pda_debug_wait_timeout")


def debug_read_probe(buf, sink, stream=None):
    """Enqueues one read-only pass over ``buf`` (any dtype, contiguous, a multiple of 16 bytes)."""
    nbytes = buf.numel() * buf.element_size()
    _check(lib().pda_debug_read_probe(_ptr(buf), nbytes, _ptr(sink), _stream(stream)), "pda_debug_read_probe")


def advance_seq_lens(seq_lens, delta=1, stream=None):
    """``seq_lens += delta`` on the device, in stream order (graph-capturable)."""
    _check(lib().pda_advance_seq_lens(_ptr(seq_lens), seq_lens.shape[0], int(delta), _stream(stream)),
           "pda_advance_seq_lens")


def kv_append_tokens(k_new, v_new, k_cache, v_cache, block_table, seq_lens, status=None, stream=None):
    """Append ``k_new``/``v_new`` ``[B,n_new,Hkv,D]``; ``seq_lens`` is the length after the append."""
    desc = cache_desc(k_cache)
    assert k_new.is_contiguous() and v_new.is_contiguous() and k_new.dim() == 4
    rc = lib().kv_append_tokens(_ptr(k_new), _ptr(v_new), _ptr(k_cache), _ptr(v_cache), C.byref(desc),
                                _ptr(block_table), block_table.stride(0), _ptr(seq_lens),
                                seq_lens.shape[0], k_new.shape[1], _ptr(status), _stream(stream))
    _check(rc, "kv_append_tokens")


def paged_verify_attention(q, k_cache, v_cache, block_table, seq_lens, scale, chunk_tokens=0, out=None,
                           part_o=None, part_lse=None, k_scale=None, v_scale=None, flags=0, status=None,
                           stream=None):
    """Causal attention of a block of query tokens ``q [B,T,Hq,D]``; returns ``out [B,T,Hq,D]``."""
    desc = cache_desc(k_cache)
    assert q.is_contiguous() and q.dim() == 4
    B, T, Hq, D = q.shape
    if out is None:
        out = torch.empty_like(q)
    mc = 0
    if chunk_tokens:
        mc = part_o.shape[3]
        assert tuple(part_o.shape) == (B, T, Hq, mc, D) and tuple(part_lse.shape) == (B, T, Hq, mc)
    rc = lib().paged_verify_attention(
        _ptr(q), _ptr(k_cache), _ptr(v_cache), C.byref(desc), _ptr(k_scale), _ptr(v_scale),
        _ptr(block_table), block_table.stride(0), _ptr(seq_lens), B, Hq, T, float(scale),
        chunk_tokens, _ptr(out), _ptr(part_o), _ptr(part_lse), mc, flags, _ptr(status),
        _stream(stream))
    _check(rc, "paged_verify_attention")
    return out


def paged_prefix_decode_attention(q, k_cache, v_cache, block_table, seq_lens, scale, prefix_tokens,
                                  prefix_chunk_tokens, chunk_tokens, part_o, part_lse, out=None,
                                  k_scale=None, v_scale=None, flags=0, status=None, stream=None):
    """Decode attention of a batch sharing its first ``prefix_tokens`` tokens' pages."""
    desc = cache_desc(k_cache)
    B, Hq, D = q.shape
    if out is None:
        out = torch.empty_like(q)
    mc = part_o.shape[2]
    assert tuple(part_o.shape) == (B, Hq, mc, D) and tuple(part_lse.shape) == (B, Hq, mc)
    rc = lib().paged_prefix_decode_attention(
        _ptr(q), _ptr(k_cache), _ptr(v_cache), C.byref(desc), _ptr(k_scale), _ptr(v_scale),
        _ptr(block_table), block_table.stride(0), _ptr(seq_lens), B, Hq, float(scale),
        int(prefix_tokens), int(prefix_chunk_tokens), int(chunk_tokens), _ptr(out), _ptr(part_o),
        _ptr(part_lse), mc, flags, _ptr(status), _stream(stream))
    _check(rc, "paged_prefix_decode_attention")
    return out


def kv_append_fp8(k_new, v_new, k_cache, v_cache, k_scale, v_scale, block_table, seq_lens,
                  status=None, stream=None):
    """Quantising append of bf16 rows into e4m3 caches (scale fixed by each page's first row)."""
    desc = cache_desc(k_cache)
    assert k_new.is_contiguous() and v_new.is_contiguous() and k_scale.is_contiguous()
    rc = lib().kv_append_fp8(_ptr(k_new), _ptr(v_new), _ptr(k_cache), _ptr(v_cache), C.byref(desc),
                             _ptr(k_scale), _ptr(v_scale), _ptr(block_table), block_table.stride(0),
                             _ptr(seq_lens), seq_lens.shape[0], _ptr(status), _stream(stream))
    _check(rc, "kv_append_fp8")


def kv_append_tokens_fp8(k_new, v_new, k_cache, v_cache, k_scale, v_scale, block_table, seq_lens,
                         status=None, stream=None):
    """Quantising append of a block ``k_new, v_new [B,T,Hkv,D]`` bf16 into e4m3 caches."""
    desc = cache_desc(k_cache)
    assert k_new.is_contiguous() and v_new.is_contiguous() and k_scale.is_contiguous() and k_new.dim() == 4
    rc = lib().kv_append_tokens_fp8(_ptr(k_new), _ptr(v_new), _ptr(k_cache), _ptr(v_cache), C.byref(desc),
                                    _ptr(k_scale), _ptr(v_scale), _ptr(block_table), block_table.stride(0),
                                    _ptr(seq_lens), seq_lens.shape[0], k_new.shape[1], _ptr(status),
                                    _stream(stream))
    _check(rc, "kv_append_tokens_fp8")


def set_persistent_threshold(min_units_per_cta: int):
    """Units per resident CTA from which the unsplit fused step uses the persistent kernel (0: always)."""
    _check(lib().pda_set_persistent_threshold(int(min_units_per_cta)), "pda_set_persistent_threshold")
