"""Seeded synthetic decode batches (host side, numpy only).

This module only *draws inputs*: sequence lengths, page placement, random
q/K/V values and their storage encodings. It contains none of the attention
arithmetic and is the one piece shared by the CUDA path's callers and the CPU
oracle's callers: both receive the very same host arrays.

bf16 tensors are carried as ``uint16`` bit patterns, e4m3 tensors as ``uint8``.

Recipe common to all workloads (one ``numpy.random.Generator(PCG64(seed))``,
draws in this order): lengths -> page permutation -> q -> K, V (pages in order of
first use, in slabs of 1024 pages, slab s from the s-th spawned child generator)
-> k_new, v_new. Values are N(0,1) rounded to bf16
(round to nearest even). ``seq_lens`` is the length AFTER this step's append;
the caches hold tokens ``0 .. L-2`` and the slot of token ``L-1`` is poisoned
until ``kv_append`` writes ``k_new``/``v_new`` there. Physical pages come from a
pool of ``ceil(1.25 * pages_needed)`` pages; a seeded permutation of the pool
is dealt out in (sequence, logical page) order; never-used pages, the unused
slots of each last page and the block-table tail are poison (0xFF bytes, a NaN
in both encodings, and -1 page ids).

The workload shapes stand in for the serving regimes the paper evaluates
(Appendix A: Llama-3.1-8B with 32 query / 8 kv heads and a 128k window under a
Poisson load with seed 42; the shared-prefix prompt-caching scenario); the
paper's prompt pool is not available, so lengths are drawn from the stated
distributions instead.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import Optional

import numpy as np

POISON_BYTE = 0xFF
BASE_SEED = 42  # the seed the paper's load generator uses (Appendix A, Scenario A)


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """float32 -> bf16 bit patterns, round to nearest even (finite inputs)."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    if x.size >= (1 << 16):  # library cast (same rounding), multi-threaded
        import torch
        return torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    u = x.view(np.uint32)
    r = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + r) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


@dataclass
class Workload:
    name: str
    batch: int
    num_q_heads: int
    num_kv_heads: int
    head_dim: int
    page_size: int
    scale: np.float32
    kv_dtype: str                      # "bf16" | "e4m3"
    num_pages: int
    q: np.ndarray                      # [B,Hq,D] uint16
    k_cache: np.ndarray                # [num_pages,Hkv,P,D] uint16 | uint8
    v_cache: np.ndarray
    block_table: np.ndarray            # [B,max_pages] int32, -1 padded
    seq_lens: np.ndarray               # [B] int32, length after append
    k_new: Optional[np.ndarray] = None  # [B,Hkv,D] uint16 (bf16 caches only)
    v_new: Optional[np.ndarray] = None
    k_scale: Optional[np.ndarray] = None  # [num_pages,Hkv] float32 (e4m3 only)
    v_scale: Optional[np.ndarray] = None
    chunk_tokens: int = 0              # split-KV chunk the workload prescribes (0: caller's choice)
    seed: int = BASE_SEED
    notes: dict = field(default_factory=dict)

    @property
    def elem_bytes(self) -> int:
        return 2 if self.kv_dtype == "bf16" else 1

    @property
    def total_tokens(self) -> int:
        return int(np.maximum(self.seq_lens, 0).astype(np.int64).sum())

    @property
    def kv_bytes(self) -> int:
        """Algorithmic KV traffic of one attention pass: every valid K and V
        element once, plus (e4m3) both scale arrays' entries of every page used."""
        n = self.total_tokens * self.num_kv_heads * self.head_dim * 2 * self.elem_bytes
        if self.kv_dtype == "e4m3":
            pages = int(np.ceil(np.maximum(self.seq_lens, 0) / self.page_size).sum())
            n += pages * self.num_kv_heads * 2 * 4
        return n


def _deal_pages(rng, pages_per_seq, shared_prefix_pages=0):
    """Returns (block_table, num_pages). With a shared prefix, the first
    ``shared_prefix_pages`` logical pages of every row alias the same ids."""
    B = len(pages_per_seq)
    private = [int(n) - shared_prefix_pages for n in pages_per_seq]
    needed = shared_prefix_pages + sum(private)
    pool = int(math.ceil(1.25 * needed))
    perm = rng.permutation(pool).astype(np.int32)
    max_pages = max(int(n) for n in pages_per_seq) if B else 0
    table = np.full((B, max(max_pages, 1)), -1, dtype=np.int32)
    cursor = 0
    shared = perm[:shared_prefix_pages]
    cursor += shared_prefix_pages
    for b in range(B):
        table[b, :shared_prefix_pages] = shared
        table[b, shared_prefix_pages:shared_prefix_pages + private[b]] = perm[cursor:cursor + private[b]]
        cursor += private[b]
    return table, pool


def _fill_normal_bf16(rng, dst_u16_2d, rows_idx, slab=1024):
    """dst[rows_idx[i]] = bf16(N(0,1)). Rows are cut into slabs of ``slab`` rows;
    slab s is drawn from the s-th child generator spawned from ``rng`` (so the
    result does not depend on how many threads fill the slabs)."""
    width = dst_u16_2d.shape[1]
    starts = list(range(0, len(rows_idx), slab))
    children = rng.spawn(len(starts)) if starts else []

    def work(i):
        idx = rows_idx[starts[i]:starts[i] + slab]
        x = children[i].standard_normal((len(idx), width), dtype=np.float32)
        dst_u16_2d[idx] = f32_to_bf16_bits(x)

    if len(starts) <= 1:
        for i in range(len(starts)):
            work(i)
    else:
        from concurrent.futures import ThreadPoolExecutor
        import os
        with ThreadPoolExecutor(max_workers=min(16, os.cpu_count() or 1)) as ex:
            list(ex.map(work, range(len(starts))))


def make_workload(name, seq_lens, num_q_heads, num_kv_heads, head_dim, page_size=16,
                  kv_dtype="bf16", seed=BASE_SEED, shared_prefix_tokens=0, chunk_tokens=0,
                  rng=None, value_scale=1.0) -> Workload:
    """Build a decode batch for explicit lengths (``seq_lens`` = after append)."""
    rng = np.random.default_rng(np.random.PCG64(seed)) if rng is None else rng
    seq_lens = np.asarray(seq_lens, dtype=np.int32)
    B, Hq, Hkv, D, P = len(seq_lens), num_q_heads, num_kv_heads, head_dim, page_size
    assert shared_prefix_tokens % P == 0
    pages_per_seq = [(max(int(L), 0) + P - 1) // P for L in seq_lens]
    sp = shared_prefix_tokens // P
    assert all(n >= sp for n in pages_per_seq) or sp == 0
    table, num_pages = _deal_pages(rng, pages_per_seq, sp)

    q = f32_to_bf16_bits(rng.standard_normal((B, Hq, D), dtype=np.float32))

    # K, V as bf16 for every used page, in order of first use.
    used = []
    seen = set()
    for b in range(B):
        for p in table[b, :pages_per_seq[b]]:
            if int(p) not in seen:
                seen.add(int(p))
                used.append(int(p))
    used = np.asarray(used, dtype=np.int64)
    tile = Hkv * P * D
    kb = np.empty((num_pages, tile), dtype=np.uint16)
    vb = np.empty((num_pages, tile), dtype=np.uint16)
    unused = np.setdiff1d(np.arange(num_pages, dtype=np.int64), used)
    kb[unused] = 0xFFFF
    vb[unused] = 0xFFFF
    _fill_normal_bf16(rng, kb, used)
    _fill_normal_bf16(rng, vb, used)
    if value_scale != 1.0:
        kb[used] = f32_to_bf16_bits(bf16_bits_to_f32(kb[used]) * np.float32(value_scale))
    kb = kb.reshape(num_pages, Hkv, P, D)
    vb = vb.reshape(num_pages, Hkv, P, D)

    k_new = f32_to_bf16_bits(rng.standard_normal((B, Hkv, D), dtype=np.float32))
    v_new = f32_to_bf16_bits(rng.standard_normal((B, Hkv, D), dtype=np.float32))

    # number of valid slots per physical page (max over the rows that use it)
    valid = np.zeros(num_pages, dtype=np.int32)
    for b in range(B):
        L = int(seq_lens[b])
        for i in range(pages_per_seq[b]):
            n = min(P, L - i * P)
            p = int(table[b, i])
            valid[p] = max(valid[p], n)

    scale = np.float32(1.0 / math.sqrt(D))
    if kv_dtype == "bf16":
        # poison the tail of each last page and the slot kv_append will fill
        for b in range(B):
            L = int(seq_lens[b])
            if L <= 0:
                continue
            last = int(table[b, (L - 1) // P])
            s = (L - 1) % P
            kb[last, :, s:, :] = 0xFFFF
            vb[last, :, s:, :] = 0xFFFF
        return Workload(name, B, Hq, Hkv, D, P, scale, "bf16", num_pages, q, kb, vb, table,
                        seq_lens, k_new, v_new, None, None, chunk_tokens, seed)

    assert kv_dtype == "e4m3"
    # e4m3 caches hold all L tokens (a quantising append is not part of this path).
    import torch  # library cast used as the storage encoder

    def quant(bits):
        x = torch.from_numpy(bf16_bits_to_f32(bits).reshape(num_pages, Hkv, P, D).copy())
        slot = torch.arange(P).view(1, 1, P, 1)
        ok = slot < torch.from_numpy(valid).view(-1, 1, 1, 1)
        x = torch.where(ok, x, torch.zeros(()))
        amax = x.abs().amax(dim=(2, 3))
        sc = torch.where(amax > 0, amax / 448.0, torch.ones(()))
        y = (x / sc[:, :, None, None]).to(torch.float8_e4m3fn).view(torch.uint8)
        y = torch.where(ok.expand_as(y), y, torch.full((), POISON_BYTE, dtype=torch.uint8))
        sc = torch.where(torch.from_numpy(valid).view(-1, 1) > 0, sc, torch.full((), float("nan")))
        return y.numpy(), sc.numpy().astype(np.float32)

    k8, ks = quant(kb)
    v8, vs = quant(vb)
    return Workload(name, B, Hq, Hkv, D, P, scale, "e4m3", num_pages, q, k8, v8, table,
                    seq_lens, None, None, ks, vs, chunk_tokens, seed,
                    notes={"k_bf16": kb, "v_bf16": vb, "valid_slots": valid})


# ---- the five named workloads ------------------------------------------------------------

def tiny(seed=BASE_SEED + 0) -> Workload:
    """batch 4, lengths {17,33,64,100}, 8 q / 2 kv heads, head_dim 64."""
    return make_workload("tiny", [17, 33, 64, 100], 8, 2, 64, seed=seed)


def llama8b(seed=BASE_SEED + 1, batch=64) -> Workload:
    """batch 64, 32 q / 8 kv heads, head_dim 128, lengths uniform in [512,4096]."""
    rng = np.random.default_rng(np.random.PCG64(seed))
    L = rng.integers(512, 4096, size=batch, endpoint=True)
    return make_workload("llama8b", L, 32, 8, 128, seed=seed, rng=rng)


def longctx(seed=BASE_SEED + 2, batch=8) -> Workload:
    """batch 8, 32 q / 8 kv heads, lengths uniform in [32768,131072], 2048-token chunks."""
    rng = np.random.default_rng(np.random.PCG64(seed))
    L = rng.integers(32768, 131072, size=batch, endpoint=True)
    return make_workload("longctx", L, 32, 8, 128, seed=seed, rng=rng, chunk_tokens=2048)


def chat70b(seed=BASE_SEED + 3, batch=256) -> Workload:
    """batch 256, 64 q / 8 kv heads, lengths lognormal(median 1024, sigma 0.8) in [16,8192]."""
    rng = np.random.default_rng(np.random.PCG64(seed))
    L = np.clip(np.rint(np.exp(rng.normal(math.log(1024.0), 0.8, size=batch))), 16, 8192)
    return make_workload("chat70b", L.astype(np.int32), 64, 8, 128, seed=seed, rng=rng)


def prefix_fp8(seed=BASE_SEED + 4, batch=128) -> Workload:
    """batch 128, 32 q / 8 kv heads, shared 2048-token prefix + suffix in [64,1024], e4m3 KV."""
    rng = np.random.default_rng(np.random.PCG64(seed))
    L = 2048 + rng.integers(64, 1024, size=batch, endpoint=True)
    return make_workload("prefix_fp8", L, 32, 8, 128, kv_dtype="e4m3", seed=seed, rng=rng,
                         shared_prefix_tokens=2048)


def scenario_c(seed=BASE_SEED + 5, batch=20) -> Workload:
    """Shared-prefix prompt caching shaped like the paper's Scenario C: 20 concurrent
    sequences, one 32768-token shared prefix plus a private suffix of 128..256 tokens
    (its 128-token suffix plus up to 128 generated tokens), 32 q / 8 kv heads, head_dim 128."""
    rng = np.random.default_rng(np.random.PCG64(seed))
    L = 32768 + rng.integers(128, 256, size=batch, endpoint=True)
    return make_workload("scenario_c", L, 32, 8, 128, seed=seed, rng=rng, shared_prefix_tokens=32768)


WORKLOADS = {"tiny": tiny, "llama8b": llama8b, "longctx": longctx, "chat70b": chat70b,
             "prefix_fp8": prefix_fp8, "scenario_c": scenario_c}
