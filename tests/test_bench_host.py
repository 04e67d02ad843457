"""CPU-only checks of bench.py's host-side byte accounting (the numerators of its roofline figures)."""
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

import bench  # noqa: E402
from paper_2605_06068_b200 import workloads as W  # noqa: E402


def test_distinct_bytes_equal_logical_bytes_without_shared_pages():
    w = W.make_workload("plain", [17, 33, 64, 100], 8, 2, 64, seed=3)
    # every valid K and V element once: sum(L) tokens x kv heads x head_dim x (K and V) x 2 bytes
    assert w.kv_bytes == (17 + 33 + 64 + 100) * 2 * 64 * 2 * 2
    assert bench.unique_kv_bytes(w) == w.kv_bytes


def test_distinct_bytes_count_a_shared_prefix_once():
    lens = [64 + 5, 64 + 16, 64 + 33]
    w = W.make_workload("shared", lens, 8, 2, 64, kv_dtype="e4m3", seed=4, shared_prefix_tokens=64)
    per_token = 2 * 64 * 2 * 1                      # kv heads x head_dim x (K and V) x 1 byte
    per_page_scales = 2 * 2 * 4                     # kv heads x (K and V scale) x fp32
    pages = sum((L + 15) // 16 for L in lens)
    assert w.kv_bytes == sum(lens) * per_token + pages * per_page_scales
    distinct_tokens = 64 + 5 + 16 + 33              # the prefix once, every suffix once
    distinct_pages = 4 + 1 + 1 + 3
    assert bench.unique_kv_bytes(w) == distinct_tokens * per_token + distinct_pages * per_page_scales
    cfg = bench.config_of(w, 0, 1)
    assert cfg["unique_kv_bytes_per_gpu"] < cfg["kv_bytes_per_gpu"] and "flushed" in cfg["l2"]


def test_traffic_table_covers_the_workloads_of_the_default_line():
    for name in ["llama8b"] + bench.DEFAULT_ALSO:
        assert bench.NCU_TRAFFIC_BYTES.get(name), name
        assert name in bench.DEFAULT_CHUNK


def test_prefix_chunk_rule():
    """The cascade's default prefix chunk: at most one prefix CTA per SM, at least 1024 tokens, a power of two."""
    class Shape:
        def __init__(self, batch, hq, hkv):
            self.batch, self.num_q_heads, self.num_kv_heads = batch, hq, hkv
    assert bench.prefix_chunk_tokens(Shape(20, 32, 8), 32768) == 2048      # 8 units a chunk: 16 chunks, 128 CTAs
    assert bench.prefix_chunk_tokens(Shape(128, 32, 8), 2048) == 1024      # 32 units a chunk: 4 chunks would be 512 tokens
    assert bench.prefix_chunk_tokens(Shape(1, 8, 8), 100) == 1024
    assert bench.prefix_chunk_tokens(Shape(4096, 64, 8), 1 << 20) == 1 << 20  # more units a chunk than SMs: one chunk
