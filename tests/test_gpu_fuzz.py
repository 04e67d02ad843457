"""Seeded random sweeps over shapes, lengths, chunkings and entry points: every case is compared
with the oracle element by element. The fixed cases elsewhere cover the named edge cases; this file
covers combinations nobody thought of (lengths straddling pages and chunks in every way, batches of
one, group sizes 1..8, both kv dtypes), with the seeds fixed so that a failure reproduces."""
import numpy as np
import pytest
import torch

from paper_2605_06068_b200 import binding as pda
from paper_2605_06068_b200 import workloads as W

from util import DeviceWorkload, assert_close, bf16_tensor, bf16_to_bits, bf16_to_f64, host_appended, oracle_out

pytestmark = pytest.mark.gpu

SHAPES = [(8, 2, 64), (32, 8, 128), (8, 8, 128), (16, 2, 128), (4, 4, 64), (64, 8, 128)]


def random_lens(rng, batch):
    kinds = rng.integers(0, 4, size=batch)
    lens = np.where(kinds == 0, rng.integers(1, 40, size=batch),
                    np.where(kinds == 1, rng.integers(1, 12, size=batch) * 16 + rng.integers(-1, 2, size=batch),
                             np.where(kinds == 2, rng.integers(100, 700, size=batch), rng.integers(700, 2500, size=batch))))
    return np.maximum(lens, 1).astype(np.int64)


@pytest.mark.parametrize("seed", range(12))
def test_random_decode_steps(oracle, seed):
    rng = np.random.default_rng(1000 + seed)
    Hq, Hkv, D = SHAPES[seed % len(SHAPES)]
    fp8 = D == 128 and seed % 3 == 2
    batch = int(rng.integers(1, 10))
    lens = random_lens(rng, batch)
    w = W.make_workload("fuzz", lens, Hq, Hkv, D, kv_dtype="e4m3" if fp8 else "bf16", seed=2000 + seed)
    k_ref, v_ref = host_appended(oracle, w)
    ref = oracle_out(oracle, w, k_ref, v_ref)
    what = f"seed {seed} Hq{Hq} kv{Hkv} D{D} {'e4m3' if fp8 else 'bf16'} lens {list(lens)}"
    for chunk in (0, int(rng.choice([16, 32, 64, 128, 512]))):
        dw = DeviceWorkload(w)
        # separate calls
        if not fp8:
            dw.append()
        out = dw.attend(chunk_tokens=chunk)
        assert_close(bf16_to_f64(out), ref, w.kv_dtype, what=f"{what} chunk {chunk} separate")
        # the fused step
        dw2 = DeviceWorkload(w)
        ws = pda.new_workspace(w.batch, Hkv)
        po = pl = None
        if chunk:
            mc = pda.max_chunks(int(lens.max()), chunk)
            po = torch.full((w.batch, Hq, mc, D), float("nan"), dtype=torch.float32, device="cuda")
            pl = torch.full((w.batch, Hq, mc), float("nan"), dtype=torch.float32, device="cuda")
        out2 = pda.paged_decode_step(dw2.q, dw2.k_new, dw2.v_new, dw2.k_cache, dw2.v_cache, dw2.block_table,
                                     dw2.seq_lens, float(w.scale), chunk_tokens=chunk, part_o=po, part_lse=pl,
                                     workspace=ws, k_scale=dw2.k_scale, v_scale=dw2.v_scale, status=dw2.status)
        torch.cuda.synchronize()
        assert_close(bf16_to_f64(out2), ref, w.kv_dtype, what=f"{what} chunk {chunk} fused")
        assert (ws == 0).all() and int(dw2.status.item()) == 0 and int(dw.status.item()) == 0
        if not fp8:
            assert (bf16_to_bits(dw2.k_cache) == k_ref).all() and (bf16_to_bits(dw2.v_cache) == v_ref).all()


@pytest.mark.parametrize("seed", range(10))
def test_random_verification_blocks(oracle, seed):
    rng = np.random.default_rng(3000 + seed)
    Hq, Hkv, D = SHAPES[seed % len(SHAPES)]
    fp8 = D == 128 and seed % 4 == 1
    batch = int(rng.integers(1, 7))
    T = int(rng.integers(1, 24))
    lens = np.maximum(random_lens(rng, batch) // 2, T)        # every sequence holds its whole block
    w = W.make_workload("fuzzv", lens, Hq, Hkv, D, kv_dtype="e4m3" if fp8 else "bf16", seed=4000 + seed)
    q = W.f32_to_bf16_bits(rng.standard_normal((batch, T, Hq, D), dtype=np.float32))
    kn = W.f32_to_bf16_bits(rng.standard_normal((batch, T, Hkv, D), dtype=np.float32))
    vn = W.f32_to_bf16_bits(rng.standard_normal((batch, T, Hkv, D), dtype=np.float32))
    k, v = w.k_cache.copy(), w.v_cache.copy()
    dw = DeviceWorkload(w)
    if fp8:
        ks, vs = w.k_scale.copy(), w.v_scale.copy()
        oracle.kv_append_tokens_e4m3(kn, vn, k, v, ks, vs, w.block_table, w.seq_lens)
        pda.kv_append_tokens_fp8(bf16_tensor(kn), bf16_tensor(vn), dw.k_cache, dw.v_cache, dw.k_scale, dw.v_scale,
                                 dw.block_table, dw.seq_lens, status=dw.status)
        assert (dw.k_cache.cpu().numpy() == k).all() and (dw.v_cache.cpu().numpy() == v).all()
        ref, _ = oracle.paged_verify_attention(q, k, v, w.block_table, w.seq_lens, w.scale, ks, vs)
    else:
        oracle.kv_append_tokens(kn, vn, k, v, w.block_table, w.seq_lens)
        pda.kv_append_tokens(bf16_tensor(kn), bf16_tensor(vn), dw.k_cache, dw.v_cache, dw.block_table,
                             dw.seq_lens, status=dw.status)
        assert (bf16_to_bits(dw.k_cache) == k).all() and (bf16_to_bits(dw.v_cache) == v).all()
        ref, _ = oracle.paged_verify_attention(q, k, v, w.block_table, w.seq_lens, w.scale)
    what = f"seed {seed} Hq{Hq} kv{Hkv} D{D} {'e4m3' if fp8 else 'bf16'} T{T} lens {list(lens)}"
    for flags in (0, pda.PDA_FLAG_MQ_MMA_SYNC, pda.PDA_FLAG_MQ_ONE_UNIT):
        for chunk in (0, int(rng.choice([32, 64, 256]))):
            po = pl = None
            if chunk:
                mc = pda.max_chunks(int(lens.max()), chunk)
                po = torch.full((batch, T, Hq, mc, D), float("nan"), dtype=torch.float32, device="cuda")
                pl = torch.full((batch, T, Hq, mc), float("nan"), dtype=torch.float32, device="cuda")
            out = pda.paged_verify_attention(bf16_tensor(q), dw.k_cache, dw.v_cache, dw.block_table, dw.seq_lens,
                                             float(w.scale), chunk_tokens=chunk, part_o=po, part_lse=pl,
                                             k_scale=dw.k_scale, v_scale=dw.v_scale, flags=flags, status=dw.status)
            assert_close(bf16_to_f64(out), ref, w.kv_dtype, what=f"{what} chunk {chunk} flags {flags}")
    assert int(dw.status.item()) == 0
