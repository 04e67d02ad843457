"""The allocation-free entry point (paged_decode_attention_static) against the
ordinary split attention + reduce calls.

It serves callers that cannot obtain device memory when they call -- a process
that has already given all of HBM to its KV pool, a plug-in without an
allocator, a loop that must not trigger an allocation's synchronisation -- by
keeping the split-KV partials in an array built into the library. This file
sorts last so that a run stopping at the first failure has run everything else.
"""
import numpy as np
import pytest
import torch

from paper_2605_06068_b200 import binding as pda
from paper_2605_06068_b200 import workloads as W

from util import DeviceWorkload, assert_close, bf16_to_bits, bf16_to_f64, oracle_out

pytestmark = pytest.mark.gpu


def run_both(w, chunk):
    dw = DeviceWorkload(w)
    if w.kv_dtype == "bf16":
        dw.append()
    expect = dw.attend(chunk_tokens=chunk)           # existing entry points, torch-owned partials
    mc = dw.part_o.shape[2]
    out = torch.full_like(dw.q, float("nan"))        # caller-provided output
    got = pda.paged_decode_attention_static(dw.q, dw.k_cache, dw.v_cache, dw.block_table,
                                            dw.seq_lens, float(w.scale), chunk, mc, out=out,
                                            k_scale=dw.k_scale, v_scale=dw.v_scale,
                                            status=dw.status)
    torch.cuda.synchronize()
    assert int(dw.status.item()) == 0
    return got, expect


def test_static_scratch_matches_ordinary_path_on_two_calls_in_a_row(oracle):
    # first call: a larger batch that leaves its partials behind in the shared array
    w1 = W.make_workload("na1", [900, 17, 2049, 333, 64, 1500], 32, 8, 128, seed=101)
    got1, exp1 = run_both(w1, 256)
    assert_close(bf16_to_f64(got1), bf16_to_f64(exp1), what="static scratch, call 1", norm=False)
    assert_close(bf16_to_f64(got1), oracle_out(oracle, w1), what="static scratch against the oracle")
    assert (bf16_to_bits(got1) == bf16_to_bits(exp1)).all()   # same kernels, same order of operations
    # second call straight after: other shapes, other chunking, fewer live chunks
    w2 = W.make_workload("na2", [100, 33, 700], 8, 2, 64, seed=102)
    got2, exp2 = run_both(w2, 64)
    assert_close(bf16_to_f64(got2), bf16_to_f64(exp2), what="static scratch, call 2", norm=False)
    assert (bf16_to_bits(got2) == bf16_to_bits(exp2)).all()
    # and the first workload again: stale contents of the second call must not matter
    got3, exp3 = run_both(w1, 512)
    assert_close(bf16_to_f64(got3), bf16_to_f64(exp3), what="static scratch, call 3", norm=False)


def test_static_scratch_rejects_sizes_beyond_its_maximum():
    w = W.make_workload("na3", [40, 50], 32, 8, 128, seed=103)
    dw = DeviceWorkload(w)
    out = torch.empty_like(dw.q)
    # 2 * 32 * max_chunks * 129 * 4 bytes > 16 MiB  <=>  max_chunks > 508
    with pytest.raises(RuntimeError, match="fixed maximum"):
        pda.paged_decode_attention_static(dw.q, dw.k_cache, dw.v_cache, dw.block_table,
                                          dw.seq_lens, float(w.scale), 16, 600, out=out)
    # just inside the limit is accepted
    pda.paged_decode_attention_static(dw.q, dw.k_cache, dw.v_cache, dw.block_table, dw.seq_lens,
                                      float(w.scale), 16, 500, out=out, status=dw.status)
    torch.cuda.synchronize()
    assert int(dw.status.item()) == 0


def test_static_scratch_reserves_nothing_after_its_first_call():
    """What the caller without an allocator relies on: once the start-up call has run on the device (it
    loads the device image that holds the array), further calls take no device memory at all. The
    runtime's free-memory figure must be the same before and after them."""
    w = W.make_workload("na4", [700, 90, 1300], 32, 8, 128, seed=104)
    dw = DeviceWorkload(w)
    dw.append()
    out = torch.empty_like(dw.q)
    mc = pda.max_chunks(1300, 128)
    # the start-up call: an empty batch is enough and enqueues nothing
    pda.paged_decode_attention_static(dw.q[:0], dw.k_cache, dw.v_cache, dw.block_table[:0], dw.seq_lens[:0],
                                      float(w.scale), 128, mc, out=out)
    # one full call, so that the kernels it launches are loaded too (the runtime loads code on first use)
    pda.paged_decode_attention_static(dw.q, dw.k_cache, dw.v_cache, dw.block_table, dw.seq_lens,
                                      float(w.scale), 128, mc, out=out, status=dw.status)
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info()
    for _ in range(3):
        pda.paged_decode_attention_static(dw.q, dw.k_cache, dw.v_cache, dw.block_table, dw.seq_lens,
                                          float(w.scale), 128, mc, out=out, status=dw.status)
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info()
    assert free_after == free_before, (free_before, free_after)
    assert int(dw.status.item()) == 0
