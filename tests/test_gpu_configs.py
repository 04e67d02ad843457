"""GPU parity at the full sizes of the five named workloads, in the launch
configuration bench.py times (the fused paged_decode_step with the same chunk
choices) and through the three separate calls, against the full oracle."""
import numpy as np
import pytest
import torch

from paper_2605_06068_b200 import binding as pda
from paper_2605_06068_b200 import workloads as W

from util import DeviceWorkload, assert_close, bf16_to_bits, bf16_to_f64, host_appended, oracle_out

pytestmark = pytest.mark.gpu

# (workload, chunk_tokens bench.py uses for the fused step, chunk_tokens for the separate calls)
CASES = [("llama8b", 0, 512), ("longctx", 2048, 2048), ("chat70b", 0, 512), ("prefix_fp8", 0, 512)]


@pytest.mark.parametrize("name,chunk,chunk_sep", CASES)
def test_full_size_config(oracle, name, chunk, chunk_sep):
    w = W.WORKLOADS[name]()
    if w.chunk_tokens:
        assert chunk == w.chunk_tokens
    k, v = host_appended(oracle, w)
    ref = oracle_out(oracle, w, k, v)
    ref_rms = np.sqrt((ref ** 2).mean())

    # ---- the fused step, as timed by bench.py
    dw = DeviceWorkload(w)
    ws = pda.new_workspace(w.batch, w.num_kv_heads)
    po = pl = None
    if chunk:
        mc = pda.max_chunks(int(w.seq_lens.max()), chunk)
        po = torch.empty((w.batch, w.num_q_heads, mc, w.head_dim), dtype=torch.float32, device="cuda")
        pl = torch.empty((w.batch, w.num_q_heads, mc), dtype=torch.float32, device="cuda")
    out = pda.paged_decode_step(dw.q, dw.k_new, dw.v_new, dw.k_cache, dw.v_cache, dw.block_table,
                                dw.seq_lens, float(w.scale), chunk_tokens=chunk, part_o=po, part_lse=pl,
                                workspace=ws, k_scale=dw.k_scale, v_scale=dw.v_scale, status=dw.status)
    torch.cuda.synchronize()
    if w.kv_dtype == "bf16":
        assert (bf16_to_bits(dw.k_cache) == k).all() and (bf16_to_bits(dw.v_cache) == v).all()
    got = bf16_to_f64(out)
    worst, nerr = assert_close(got, ref, w.kv_dtype, what=f"{name} fused chunk {chunk}")
    print(f"{name}: fused chunk {chunk}: max err/tol {worst:.3f}, max err/rms {nerr:.3e}")
    assert (ws == 0).all() and int(dw.status.item()) == 0
    # the output is not trivially small: the stated tolerance alone cannot tell at long context
    assert np.sqrt((got ** 2).mean()) > 0.5 * ref_rms

    # ---- the three separate calls (kv_append, split attention, reduce)
    dw = DeviceWorkload(w)
    if w.kv_dtype == "bf16":
        dw.append()
        assert (bf16_to_bits(dw.k_cache) == k).all() and (bf16_to_bits(dw.v_cache) == v).all()
    got = bf16_to_f64(dw.attend(chunk_tokens=chunk_sep))
    worst, nerr = assert_close(got, ref, w.kv_dtype, what=f"{name} separate chunk {chunk_sep}")
    print(f"{name}: separate chunk {chunk_sep}: max err/tol {worst:.3f}, max err/rms {nerr:.3e}")
    assert int(dw.status.item()) == 0


@pytest.mark.parametrize("name", ["llama8b", "chat70b", "prefix_fp8"])
def test_full_size_verification_sampled(oracle, name):
    """16-token verification at the full size of a workload, in the configuration `bench.py --mode verify`
    times (unsplit; the persistent tcgen05 kernel for bf16, with chat70b's 2048 units partly claimed from the
    counter; the e4m3 tensor-core kernel for prefix_fp8), against the oracle on a sample of the sequences:
    the longest, the shortest and ten others."""
    T = 16
    w = W.WORKLOADS[name]()
    rng = np.random.default_rng(77)
    q = W.f32_to_bf16_bits(rng.standard_normal((w.batch, T, w.num_q_heads, w.head_dim), dtype=np.float32))
    dw = DeviceWorkload(w)
    k, v = w.k_cache, w.v_cache
    if w.kv_dtype == "bf16":   # (a bf16 workload's last slots are filled by the append)
        k, v = host_appended(oracle, w)
        dw.append()
    out = pda.paged_verify_attention(torch.from_numpy(q.view(np.int16)).cuda().view(torch.bfloat16), dw.k_cache,
                                     dw.v_cache, dw.block_table, dw.seq_lens, float(w.scale),
                                     k_scale=dw.k_scale, v_scale=dw.v_scale, status=dw.status)
    got = bf16_to_f64(out)
    assert int(dw.status.item()) == 0
    order = np.argsort(w.seq_lens)
    pick = np.unique(np.concatenate([order[:1], order[-1:], rng.choice(w.batch, size=10, replace=False)]))
    scales = (w.k_scale, w.v_scale) if w.kv_dtype == "e4m3" else ()
    ref, _ = oracle.paged_verify_attention(q[pick], k, v, w.block_table[pick], w.seq_lens[pick], w.scale, *scales)
    worst, nerr = assert_close(got[pick], ref, w.kv_dtype, what=f"{name} verification of {T} tokens, sampled")
    print(f"{name}: verify {T}: max err/tol {worst:.3f}, max err/rms {nerr:.3e}")
    # every other sequence: finite and of the same scale as the sampled ones
    assert np.isfinite(got).all()
    assert np.sqrt((got ** 2).mean()) > 0.3 * np.sqrt((ref ** 2).mean())


@pytest.mark.parametrize("name,prefix,pchunk,chunk", [("scenario_c", 32768, 2048, 256), ("prefix_fp8", 2048, 512, 256)])
def test_full_size_shared_prefix_cascade_sampled(oracle, name, prefix, pchunk, chunk):
    """The shared-prefix cascade at full size, with the chunk sizes `bench.py --mode cascade` uses, against
    the plain oracle (the cascade is an exact reorganisation of decode attention) on sampled sequences."""
    w = W.WORKLOADS[name]()
    dw = DeviceWorkload(w)
    k, v = w.k_cache, w.v_cache
    if w.kv_dtype == "bf16":
        k, v = host_appended(oracle, w)
        dw.append()
    mc = (prefix + pchunk - 1) // pchunk + pda.max_chunks(int(w.seq_lens.max()) - prefix + 1, chunk)
    po = torch.full((w.batch, w.num_q_heads, mc, w.head_dim), float("nan"), dtype=torch.float32, device="cuda")
    pl = torch.full((w.batch, w.num_q_heads, mc), float("nan"), dtype=torch.float32, device="cuda")
    out = pda.paged_prefix_decode_attention(dw.q, dw.k_cache, dw.v_cache, dw.block_table, dw.seq_lens,
                                            float(w.scale), prefix, pchunk, chunk, po, pl,
                                            k_scale=dw.k_scale, v_scale=dw.v_scale, status=dw.status)
    got = bf16_to_f64(out)
    assert int(dw.status.item()) == 0 and np.isfinite(got).all()
    rng = np.random.default_rng(78)
    order = np.argsort(w.seq_lens)
    pick = np.unique(np.concatenate([order[:1], order[-1:], rng.choice(w.batch, size=4, replace=False)]))
    scales = (w.k_scale, w.v_scale) if w.kv_dtype == "e4m3" else ()
    ref, _ = oracle.paged_decode_attention(w.q[pick], k, v, w.block_table[pick], w.seq_lens[pick], w.scale, *scales)
    worst, nerr = assert_close(got[pick], ref, w.kv_dtype, what=f"{name} cascade, sampled")
    print(f"{name}: cascade {pchunk}/{chunk}: max err/tol {worst:.3f}, max err/rms {nerr:.3e}")
