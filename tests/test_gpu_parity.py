"""GPU parity: the CUDA path (through the C ABI) against the fp64 CPU oracle on
the same seeded inputs. Integer / byte work is compared bit-exactly, floating
point within |err| <= atol + rtol*|ref| with (5e-3, 1e-2) for bf16 KV and
(2e-2, 2e-2) for e4m3 KV, plus a normalised-error gate (see util.py)."""
import numpy as np
import pytest
import torch

from paper_2605_06068_b200 import binding as pda
from paper_2605_06068_b200 import workloads as W

from util import (DeviceWorkload, assert_close, bf16_tensor, bf16_to_bits, bf16_to_f64,
                  host_appended, oracle_out)

pytestmark = pytest.mark.gpu

PATHS = [pytest.param(0, id="tma"), pytest.param(pda.PDA_FLAG_FORCE_GENERIC, id="generic")]


def status_of(dw):
    return int(dw.status.item())


# ---- kv_append ---------------------------------------------------------------------------

@pytest.mark.parametrize("seed", [42, 43, 44, 45])
def test_kv_append_bit_exact_whole_cache(oracle, seed):
    w = W.tiny(seed=seed)
    dw = DeviceWorkload(w)
    dw.append()
    k_ref, v_ref = host_appended(oracle, w)
    assert (bf16_to_bits(dw.k_cache) == k_ref).all()
    assert (bf16_to_bits(dw.v_cache) == v_ref).all()
    assert status_of(dw) == 0


def test_kv_append_strided_cache_and_guard_regions(oracle):
    """[pages, slot, head, D] storage viewed as [pages, head, slot, D]; sentinel bytes
    around the cache must survive."""
    w = W.make_workload("nhd", [1, 16, 17, 250], 4, 4, 128, seed=5)
    k_ref, v_ref = host_appended(oracle, w)
    guard = 4096
    n = w.k_cache.size
    bufs = []
    for host in (w.k_cache, w.v_cache):
        raw = torch.full((n + 2 * guard,), -21555, dtype=torch.int16, device="cuda")
        body = raw[guard:guard + n].view(w.num_pages, 16, w.num_kv_heads, w.head_dim)
        body.copy_(torch.from_numpy(host.view(np.int16)).cuda().permute(0, 2, 1, 3))
        bufs.append((raw, body.permute(0, 2, 1, 3).view(torch.bfloat16)))
    dw = DeviceWorkload(w)
    pda.kv_append(dw.k_new, dw.v_new, bufs[0][1], bufs[1][1], dw.block_table, dw.seq_lens,
                  status=dw.status)
    assert (bf16_to_bits(bufs[0][1]) == k_ref).all() and (bf16_to_bits(bufs[1][1]) == v_ref).all()
    for raw, _ in bufs:
        assert (raw[:guard] == -21555).all() and (raw[-guard:] == -21555).all()
    # attention through the same strided view
    out = pda.paged_decode_attention(dw.q, bufs[0][1], bufs[1][1], dw.block_table, dw.seq_lens,
                                     float(w.scale), status=dw.status)
    assert_close(bf16_to_f64(out), oracle_out(oracle, w, k_ref, v_ref), what="strided")
    assert status_of(dw) == 0


def test_kv_append_bad_inputs_set_status_and_touch_nothing(oracle):
    w = W.tiny(seed=42)
    dw = DeviceWorkload(w)
    before_k = bf16_to_bits(dw.k_cache).copy()
    bt = dw.block_table.clone()
    bt[0, 1] = w.num_pages          # row 0 appends into logical page 1 (L=17)
    bt[1, 2] = -1                   # row 1 appends into logical page 2 (L=33)
    sl = dw.seq_lens.clone()
    sl[3] = bt.shape[1] * 16 + 1    # beyond the table
    pda.kv_append(dw.k_new, dw.v_new, dw.k_cache, dw.v_cache, bt, sl, status=dw.status)
    torch.cuda.synchronize()
    assert status_of(dw) == 2       # the larger of BAD_PAGE (1) and BAD_SEQ_LEN (2)
    after = bf16_to_bits(dw.k_cache)
    # only row 2 (L=64) was appended
    page = w.block_table[2, 3]
    expect = before_k.copy()
    expect[page, :, 15, :] = w.k_new[2]
    assert (after == expect).all()


# ---- attention: tiny config and small ragged cases ----------------------------------------

@pytest.mark.parametrize("flags", PATHS)
@pytest.mark.parametrize("seed", [42, 43, 44, 45])
def test_tiny_unsplit_and_split(oracle, seed, flags):
    w = W.tiny(seed=seed)
    dw = DeviceWorkload(w)
    dw.append()
    ref = oracle_out(oracle, w)
    out = dw.attend(flags=flags)
    assert_close(bf16_to_f64(out), ref, what="tiny unsplit")
    for chunk in (16, 32, 48, 128):
        out_s = dw.attend(chunk_tokens=chunk, flags=flags)
        assert_close(bf16_to_f64(out_s), ref, what=f"tiny chunk {chunk}")
        # partials themselves against the oracle's per-chunk results
        k, v = host_appended(oracle, w)
        mc = dw.part_o.shape[2]
        po, pl = oracle.paged_decode_attention(w.q, k, v, w.block_table, w.seq_lens, w.scale,
                                               chunk_tokens=chunk, max_chunks=mc)
        live = ~np.isnan(pl)
        g_po, g_pl = dw.part_o.cpu().numpy().astype(np.float64), dw.part_lse.cpu().numpy().astype(np.float64)
        assert np.isnan(g_pl[~live]).all(), "entries of chunks that do not exist must stay untouched"
        np.testing.assert_allclose(g_pl[live], pl[live], rtol=0, atol=2e-3)
        assert np.abs(g_po[live] - po[live]).max() < 5e-3
    assert status_of(dw) == 0


RAGGED = [
    # (lengths, Hq, Hkv, D)
    ([1, 2, 15, 16, 17, 31, 32, 33, 255, 256, 257, 1000], 8, 2, 64),
    ([1, 16, 17, 129, 640, 2049], 32, 8, 128),
    ([5, 48, 300, 777], 64, 8, 128),     # G = 8
    ([3, 100, 513], 8, 8, 128),          # G = 1
    ([7, 64, 200], 6, 3, 64),            # G = 2
    ([9, 130], 24, 2, 96),               # G = 12, head_dim 96: generic kernel only
    ([4, 33, 260, 1030], 12, 4, 128),    # G = 3
    ([4, 33, 260, 1030], 20, 4, 128),    # G = 5
    ([6, 70, 515], 28, 4, 128),          # G = 7
]


@pytest.mark.parametrize("flags", PATHS)
@pytest.mark.parametrize("case", RAGGED, ids=lambda c: f"Hq{c[1]}kv{c[2]}D{c[3]}")
def test_ragged_batches(oracle, case, flags):
    lens, Hq, Hkv, D = case
    w = W.make_workload("ragged", lens, Hq, Hkv, D, seed=77)
    dw = DeviceWorkload(w)
    dw.append()
    ref = oracle_out(oracle, w)
    assert_close(bf16_to_f64(dw.attend(flags=flags)), ref, what="ragged unsplit")
    for chunk in (64, 512):
        assert_close(bf16_to_f64(dw.attend(chunk_tokens=chunk, flags=flags)), ref,
                     what=f"ragged chunk {chunk}")
    assert status_of(dw) == 0


@pytest.mark.parametrize("flags", PATHS)
def test_fp8_small(oracle, flags):
    w = W.prefix_fp8(seed=46, batch=5)
    dw = DeviceWorkload(w)
    ref = oracle_out(oracle, w)
    assert_close(bf16_to_f64(dw.attend(flags=flags)), ref, "e4m3", what="fp8 unsplit")
    assert_close(bf16_to_f64(dw.attend(chunk_tokens=256, flags=flags)), ref, "e4m3", what="fp8 split")
    w2 = W.make_workload("fp8r", [1, 15, 16, 17, 100, 333], 16, 2, 64, kv_dtype="e4m3", seed=8)
    dw2 = DeviceWorkload(w2)
    assert_close(bf16_to_f64(dw2.attend(flags=flags)), oracle_out(oracle, w2), "e4m3", what="fp8 D64")
    assert status_of(dw) == 0 and status_of(dw2) == 0


def test_e4m3_device_decoder_matches_table(oracle):
    t = oracle.e4m3_decode_table()
    g = pda.debug_e4m3_decode().cpu().numpy().astype(np.float64)
    ok = ~np.isnan(t)
    assert (g[ok] == t[ok]).all() and np.isnan(g[~ok]).all()
    assert (np.signbit(g[ok]) == np.signbit(t[ok])).all()


# ---- invariants and anti-shortcut checks ---------------------------------------------------

@pytest.mark.parametrize("flags", PATHS)
def test_single_token_returns_v_bits(oracle, flags):
    w = W.make_workload("one", [1, 1, 1, 1], 8, 2, 64, seed=3)
    dw = DeviceWorkload(w)
    dw.append()
    out = bf16_to_bits(dw.attend(flags=flags))
    for b in range(4):
        for h in range(8):
            assert (out[b, h] == w.v_new[b, h // 4]).all()
    w = W.make_workload("one", [1, 1], 32, 8, 128, seed=4)
    dw = DeviceWorkload(w)
    dw.append()
    out = bf16_to_bits(dw.attend(flags=flags))
    for b in range(2):
        for h in range(32):
            assert (out[b, h] == w.v_new[b, h // 4]).all()


@pytest.mark.parametrize("flags", PATHS)
def test_equal_scores_give_mean_and_empty_sequence_gives_zero(oracle, flags):
    w = W.make_workload("mean", [0, 40, 700, 0, 16], 32, 8, 128, seed=6)
    dw = DeviceWorkload(w)
    dw.append()
    dw.q.zero_()
    k, v = host_appended(oracle, w)
    ref = oracle_out(oracle, type(w)(**{**w.__dict__, "q": np.zeros_like(w.q)}), k, v)
    for chunk in (0, 128):
        out = bf16_to_f64(dw.attend(chunk_tokens=chunk, flags=flags))
        assert (out[0] == 0).all() and (out[3] == 0).all()
        assert_close(out, ref, what="equal scores")
        # independent of the oracle: the mean of the gathered V rows
        L = 700
        pages = w.block_table[2, :(L + 15) // 16]
        V = W.bf16_bits_to_f32(v[pages]).astype(np.float64).transpose(1, 0, 2, 3).reshape(8, -1, 128)[:, :L]
        assert np.abs(out[2, 5] - V[1].mean(axis=0)).max() < 1e-3


@pytest.mark.parametrize("flags", PATHS)
@pytest.mark.parametrize("chunk", [0, 512])
def test_needle_tokens(oracle, flags, chunk):
    """One key at score 40 with V = 1..D: a dropped, duplicated or misplaced token shows at O(1)."""
    L, D = 1500, 128
    w = W.make_workload("needle", [L], 4, 1, D, seed=13)
    dw = DeviceWorkload(w)
    dw.append()
    q = w.q.copy(); q[0, 1:] = q[0, 0]
    dw.q = bf16_tensor(q)
    qf = W.bf16_bits_to_f32(q[0, 0]).astype(np.float64)
    k0, v0 = dw.k_cache.clone(), dw.v_cache.clone()
    needle_k = W.f32_to_bf16_bits((40.0 / (float(w.scale) * (qf @ qf)) * qf).astype(np.float32))
    needle_v = W.f32_to_bf16_bits(np.arange(1, D + 1, dtype=np.float32))
    for j in (0, 1, 15, 16, 17, 511, 512, 513, 1023, 1024, L - 17, L - 16, L - 2, L - 1):
        dw.k_cache.copy_(k0); dw.v_cache.copy_(v0)
        page, slot = int(w.block_table[0, j // 16]), j % 16
        dw.k_cache[page, 0, slot] = bf16_tensor(needle_k)
        dw.v_cache[page, 0, slot] = bf16_tensor(needle_v)
        out = bf16_to_f64(dw.attend(chunk_tokens=chunk, flags=flags))
        for h in range(4):
            assert np.abs(out[0, h] - np.arange(1, D + 1)).max() <= 0.5, f"needle at {j}"


@pytest.mark.parametrize("flags", PATHS)
def test_structured_v(oracle, flags):
    """V_j[d] = 1 + d/D for every token => out[d] = 1 + d/D (normalisation by l);
    V_j[0] = j/L => out[0] = sum_j p_j j/L (token <-> weight pairing, via the oracle)."""
    L, D = 2100, 128
    w = W.make_workload("sv", [L, 333], 8, 2, D, seed=17, value_scale=3.0)
    k, v = host_appended(oracle, w)
    ramp = W.f32_to_bf16_bits(1.0 + np.arange(D, dtype=np.float32) / D)
    for b, Lb in enumerate((L, 333)):
        for j in range(Lb):
            page = w.block_table[b, j // 16]
            v[page, :, j % 16, :] = ramp
            v[page, :, j % 16, 0] = W.f32_to_bf16_bits(np.float32(j // 16) / 256)
    w.k_cache, w.v_cache = k, v
    w.k_new = np.stack([k[w.block_table[b, (Lb - 1) // 16], :, (Lb - 1) % 16] for b, Lb in enumerate((L, 333))])
    w.v_new = np.stack([v[w.block_table[b, (Lb - 1) // 16], :, (Lb - 1) % 16] for b, Lb in enumerate((L, 333))])
    dw = DeviceWorkload(w)
    ref = oracle_out(oracle, w, k, v)
    for chunk in (0, 256):
        out = bf16_to_f64(dw.attend(chunk_tokens=chunk, flags=flags))
        assert np.abs(out[:, :, 1:] - (1.0 + np.arange(1, D) / D)).max() < 8e-3
        assert np.abs(out[:, :, 0] - ref[:, :, 0]).max() < 5e-3
        assert_close(out, ref, what="structured V")


@pytest.mark.parametrize("flags", PATHS)
def test_page_permutation_poison_and_determinism(oracle, flags):
    w = W.make_workload("perm", [17, 33, 64, 100, 900], 32, 8, 128, seed=42)
    dw = DeviceWorkload(w)
    dw.append()
    out1 = bf16_to_bits(dw.attend(flags=flags)).copy()
    out1b = bf16_to_bits(dw.attend(flags=flags))
    assert (out1 == out1b).all(), "run-to-run determinism"
    split1 = bf16_to_bits(dw.attend(chunk_tokens=64, flags=flags)).copy()
    # re-deal the physical pages under a consistent block table
    rng = np.random.default_rng(1)
    perm = rng.permutation(w.num_pages)
    k, v = host_appended(oracle, w)
    k2 = np.empty_like(k); v2 = np.empty_like(v)
    k2[perm] = k; v2[perm] = v
    # change every poison pattern on the way: unused slots, unused pages, table tail
    used = np.zeros(w.num_pages, bool)
    for b in range(w.batch):
        L = int(w.seq_lens[b]); n = (L + 15) // 16
        used[perm[w.block_table[b, :n]]] = True
        if L % 16:
            k2[perm[w.block_table[b, n - 1]], :, L % 16:, :] = 0x7F80   # +inf
            v2[perm[w.block_table[b, n - 1]], :, L % 16:, :] = 0x7FC0   # NaN
    k2[~used] = 0x7F80; v2[~used] = 0xFF80
    table2 = np.where(w.block_table >= 0, perm[np.maximum(w.block_table, 0)], 2 ** 31 - 1).astype(np.int32)
    w2 = type(w)(**{**w.__dict__, "k_cache": k2, "v_cache": v2, "block_table": table2})
    dw2 = DeviceWorkload(w2)
    out2 = bf16_to_bits(dw2.attend(flags=flags))
    assert (out2 == out1).all(), "page placement and poison must not change a single bit"
    assert (bf16_to_bits(dw2.attend(chunk_tokens=64, flags=flags)) == split1).all()
    assert status_of(dw) == 0 and status_of(dw2) == 0


@pytest.mark.parametrize("flags", PATHS)
def test_bad_block_table_sets_status_and_zero_fills(oracle, flags):
    w = W.make_workload("bad", [100, 200, 300], 8, 2, 64, seed=9)
    dw = DeviceWorkload(w)
    dw.append()
    good = bf16_to_bits(dw.attend(flags=flags)).copy()
    guard_q = dw.q.clone()
    dw.block_table[0, 3] = -1
    dw.block_table[1, 0] = w.num_pages
    out = bf16_to_bits(dw.attend(flags=flags))
    torch.cuda.synchronize()
    assert status_of(dw) == 1
    assert (out[0] == 0).all() and (out[1] == 0).all() and (out[2] == good[2]).all()
    assert torch.equal(dw.q, guard_q)
    dw.status.zero_()
    dw.seq_lens[2] = dw.block_table.shape[1] * 16 + 5
    out = bf16_to_bits(dw.attend(chunk_tokens=64, flags=flags, max_chunks=8))
    torch.cuda.synchronize()
    assert status_of(dw) == 2
    assert (out[2] == 0).all()


# ---- the fused step (append + attention + reduce in one launch) -----------------------------

@pytest.fixture(params=["persistent", "per_unit"])
def step_kernel(request):
    """Runs a test with the unsplit fused step forced onto the persistent kernel, then onto the
    one-CTA-per-unit kernel (the library picks by units per resident CTA otherwise)."""
    pda.set_persistent_threshold(0 if request.param == "persistent" else 1 << 30)
    yield request.param
    pda.set_persistent_threshold(6)


STEP_CASES = [
    ([17, 33, 64, 100], 8, 2, 64),
    ([1, 16, 17, 129, 640, 2049, 0, 5], 32, 8, 128),
    ([5, 48, 300, 777, 1], 64, 8, 128),
    ([3, 100, 513], 8, 8, 128),
]


@pytest.mark.parametrize("case", STEP_CASES, ids=lambda c: f"Hq{c[1]}kv{c[2]}D{c[3]}")
def test_fused_step_matches_oracle_and_appends_bit_exactly(oracle, case, step_kernel):
    lens, Hq, Hkv, D = case
    w = W.make_workload("step", lens, Hq, Hkv, D, seed=123)
    k_ref, v_ref = host_appended(oracle, w)
    ref = oracle_out(oracle, w, k_ref, v_ref)
    ws = pda.new_workspace(w.batch, Hkv)
    for chunk in (0, 64, 512):
        dw = DeviceWorkload(w)
        po = pl = None
        if chunk:
            mc = pda.max_chunks(max(lens), chunk)
            po = torch.full((w.batch, Hq, mc, D), float("nan"), dtype=torch.float32, device="cuda")
            pl = torch.full((w.batch, Hq, mc), float("nan"), dtype=torch.float32, device="cuda")
        out = torch.full_like(dw.q, float("nan"))
        for rep in range(2):   # the second call re-appends the same rows and reuses the workspace
            pda.paged_decode_step(dw.q, dw.k_new, dw.v_new, dw.k_cache, dw.v_cache, dw.block_table,
                                  dw.seq_lens, float(w.scale), chunk_tokens=chunk, out=out,
                                  part_o=po, part_lse=pl, workspace=ws, status=dw.status)
            torch.cuda.synchronize()
            assert (bf16_to_bits(dw.k_cache) == k_ref).all() and (bf16_to_bits(dw.v_cache) == v_ref).all()
            assert_close(bf16_to_f64(out), ref, what=f"fused step chunk {chunk} rep {rep}")
            assert (ws == 0).all(), "the workspace must be left zeroed"
            assert status_of(dw) == 0
        # the three separate calls agree to the last bits (other kernels may merge warps in another order)
        dw3 = DeviceWorkload(w)
        dw3.append()
        sep = bf16_to_f64(dw3.attend(chunk_tokens=chunk))
        assert np.abs(sep - bf16_to_f64(out)).max() <= 2.0 ** -7 * max(1e-30, np.abs(sep).max())


@pytest.mark.parametrize("case", [([5000, 33, 700], 32, 8, 128, 16),      # 313 chunks: weights in shared memory
                                  ([26000, 40], 8, 1, 64, 16)],             # 1625 chunks x 8 heads: do not fit, plain loop
                         ids=["313chunks", "1625chunks"])
def test_fused_step_merge_of_many_chunks(oracle, case):
    lens, Hq, Hkv, D, chunk = case
    w = W.make_workload("manychunks", lens, Hq, Hkv, D, seed=77)
    k_ref, v_ref = host_appended(oracle, w)
    ref = oracle_out(oracle, w, k_ref, v_ref)
    dw = DeviceWorkload(w)
    ws = pda.new_workspace(w.batch, Hkv)
    mc = pda.max_chunks(max(lens), chunk)
    po = torch.full((w.batch, Hq, mc, D), float("nan"), dtype=torch.float32, device="cuda")
    pl = torch.full((w.batch, Hq, mc), float("nan"), dtype=torch.float32, device="cuda")
    out = pda.paged_decode_step(dw.q, dw.k_new, dw.v_new, dw.k_cache, dw.v_cache, dw.block_table,
                                dw.seq_lens, float(w.scale), chunk_tokens=chunk, part_o=po, part_lse=pl,
                                workspace=ws, status=dw.status)
    torch.cuda.synchronize()
    assert_close(bf16_to_f64(out), ref, what=f"fused step, {mc} chunks")
    assert (ws == 0).all() and status_of(dw) == 0
    assert (bf16_to_bits(dw.k_cache) == k_ref).all()


def test_fused_step_fp8_and_no_append(oracle):
    w = W.prefix_fp8(seed=46, batch=6)
    dw = DeviceWorkload(w)
    ref = oracle_out(oracle, w)
    ws = pda.new_workspace(w.batch, w.num_kv_heads)
    mc = pda.max_chunks(int(w.seq_lens.max()), 256)
    po = torch.empty((w.batch, 32, mc, 128), dtype=torch.float32, device="cuda")
    pl = torch.empty((w.batch, 32, mc), dtype=torch.float32, device="cuda")
    out = pda.paged_decode_step(dw.q, None, None, dw.k_cache, dw.v_cache, dw.block_table, dw.seq_lens,
                                float(w.scale), chunk_tokens=256, part_o=po, part_lse=pl, workspace=ws,
                                k_scale=dw.k_scale, v_scale=dw.v_scale, status=dw.status)
    assert_close(bf16_to_f64(out), ref, "e4m3", what="fused fp8 step")
    assert (ws == 0).all() and status_of(dw) == 0
    # without a workspace the split step falls back to separate launches, same result
    out2 = pda.paged_decode_step(dw.q, None, None, dw.k_cache, dw.v_cache, dw.block_table, dw.seq_lens,
                                 float(w.scale), chunk_tokens=256, part_o=po, part_lse=pl,
                                 k_scale=dw.k_scale, v_scale=dw.v_scale, status=dw.status)
    assert (bf16_to_bits(out2) == bf16_to_bits(out)).all()


def test_fused_step_bad_inputs(oracle, step_kernel):
    w = W.make_workload("bad", [100, 200, 300], 8, 2, 64, seed=9)
    dw = DeviceWorkload(w)
    ws = pda.new_workspace(3, 2)
    mc = 8
    po = torch.empty((3, 8, mc, 64), dtype=torch.float32, device="cuda")
    pl = torch.empty((3, 8, mc), dtype=torch.float32, device="cuda")
    good = bf16_to_bits(pda.paged_decode_step(dw.q, dw.k_new, dw.v_new, dw.k_cache, dw.v_cache, dw.block_table,
                                              dw.seq_lens, float(w.scale), chunk_tokens=64, part_o=po,
                                              part_lse=pl, workspace=ws, status=dw.status)).copy()
    k_before = bf16_to_bits(dw.k_cache).copy()
    dw.block_table[0, 3] = -1
    dw.block_table[1, 12] = w.num_pages      # the page row 1 appends into (L=200 -> logical page 12)
    out = bf16_to_bits(pda.paged_decode_step(dw.q, dw.k_new, dw.v_new, dw.k_cache, dw.v_cache, dw.block_table,
                                             dw.seq_lens, float(w.scale), chunk_tokens=64, part_o=po,
                                             part_lse=pl, workspace=ws, status=dw.status))
    torch.cuda.synchronize()
    assert status_of(dw) == 1 and (ws == 0).all()
    assert (out[2] == good[2]).all()
    # rows with a bad page: only the chunks that hit it are dropped, nothing is written out of range
    assert np.isfinite(bf16_to_f64(torch.from_numpy(out.view(np.int16)).view(torch.bfloat16))).all()
    assert (bf16_to_bits(dw.k_cache) == k_before).all()
    # unsplit: a unit with a bad page or an impossible length is zero-filled, the others are untouched
    dw.status.zero_()
    good_u = bf16_to_bits(pda.paged_decode_step(dw.q, None, None, dw.k_cache, dw.v_cache, torch.from_numpy(w.block_table).cuda(),
                                                dw.seq_lens, float(w.scale), workspace=ws, status=dw.status)).copy()
    assert status_of(dw) == 0
    dw.seq_lens[2] = dw.block_table.shape[1] * 16 + 5
    out_u = bf16_to_bits(pda.paged_decode_step(dw.q, dw.k_new, dw.v_new, dw.k_cache, dw.v_cache, dw.block_table,
                                               dw.seq_lens, float(w.scale), workspace=ws, status=dw.status))
    torch.cuda.synchronize()
    assert status_of(dw) == 2 and (ws == 0).all()
    assert (out_u == 0).all() and good_u.any()    # every row has a bad page or an impossible length
    assert (bf16_to_bits(dw.k_cache) == k_before).all()


# ---- reduce on synthetic partials ----------------------------------------------------------

def test_reduce_alone(oracle):
    rng = np.random.default_rng(0)
    B, Hq, Cm, D = 3, 8, 7, 128
    po = rng.standard_normal((B, Hq, Cm, D)).astype(np.float32)
    pl = (rng.standard_normal((B, Hq, Cm)) * 3).astype(np.float32)
    seq = np.array([7 * 32, 33, 0], np.int32)
    po[1, :, 2:] = np.nan; pl[1, :, 2:] = np.nan   # chunks that do not exist: never read
    ref, _ = oracle.paged_decode_reduce(po.astype(np.float64), pl.astype(np.float64), seq, 32)
    out = pda.paged_decode_reduce(torch.from_numpy(po).cuda(), torch.from_numpy(pl).cuda(),
                                  torch.from_numpy(seq).cuda(), 32)
    assert_close(bf16_to_f64(out), ref, what="reduce", norm=False)
    assert (bf16_to_f64(out)[2] == 0).all()
    # a single chunk is the identity (up to the bf16 rounding of the output)
    out1 = pda.paged_decode_reduce(torch.from_numpy(po).cuda(), torch.from_numpy(pl).cuda(),
                                   torch.tensor([5, 32, 1], dtype=torch.int32).cuda(), 32)
    expect = torch.from_numpy(po[:, :, 0]).to(torch.bfloat16)
    assert torch.equal(out1.cpu(), expect)


@pytest.mark.parametrize("D", [64, 128, 256])
@pytest.mark.parametrize("Cm", [1, 33, 300])
def test_reduce_many_chunks_and_widths(oracle, D, Cm):
    """Chunk counts on both sides of the kernel's register-held weight blocks (32 per block, 256 in
    registers, more recomputed), ragged per sequence, for every vector width of a row."""
    rng = np.random.default_rng(Cm * 1000 + D)
    B, Hq, chunk = 5, 3, 16
    po = rng.standard_normal((B, Hq, Cm, D)).astype(np.float32)
    pl = (rng.standard_normal((B, Hq, Cm)) * 4).astype(np.float32)
    seq = np.array([Cm * chunk, max(Cm * chunk - 17, 1), (Cm // 2) * chunk + 1, 1, 0], np.int32)
    for b in range(B):                      # chunks past a sequence's end hold poison and are never read
        n = (int(seq[b]) + chunk - 1) // chunk
        po[b, :, n:] = np.nan
        pl[b, :, n:] = np.nan
    pl[0, 1, 0] = -np.inf                   # an empty chunk inside the range: weight 0
    po[0, 1, 0] = 0.0
    # a row whose chunks are ALL empty (what a unit skipped for a bad length leaves behind): zeros, also
    # where the weights are recomputed beyond the register-held blocks
    pl[1, 2, :] = -np.inf
    po[1, 2, :] = 0.0
    ref, _ = oracle.paged_decode_reduce(po.astype(np.float64), pl.astype(np.float64), seq, chunk)
    out = pda.paged_decode_reduce(torch.from_numpy(po).cuda(), torch.from_numpy(pl).cuda(),
                                  torch.from_numpy(seq).cuda(), chunk)
    assert_close(bf16_to_f64(out), ref, what=f"reduce Cm={Cm} D={D}", norm=False)
    assert (bf16_to_f64(out)[4] == 0).all()
    assert (bf16_to_f64(out)[1, 2] == 0).all() and (ref[1, 2] == 0).all()


# ---- the end-to-end host call ---------------------------------------------------------------

def test_step_host_matches_device_calls(oracle):
    w = W.make_workload("host", [17, 33, 64, 100, 1200], 32, 8, 128, seed=42)
    dw = DeviceWorkload(w)
    ref = oracle_out(oracle, w)
    pin = lambda a: torch.from_numpy(a.view(np.int16) if a.dtype == np.uint16 else a).pin_memory()
    hq, hk, hv = pin(w.q), pin(w.k_new), pin(w.v_new)
    hbt, hsl = pin(w.block_table), pin(w.seq_lens)
    dq, dk, dv = torch.empty_like(dw.q), torch.empty_like(dw.k_new), torch.empty_like(dw.v_new)
    dbt, dsl = torch.empty_like(dw.block_table), torch.empty_like(dw.seq_lens)
    for chunk in (0, 256):
        dw = DeviceWorkload(w)
        mc = pda.max_chunks(1200, chunk) if chunk else 0
        po = torch.empty((w.batch, 32, mc, 128), dtype=torch.float32, device="cuda") if chunk else None
        pl = torch.empty((w.batch, 32, mc), dtype=torch.float32, device="cuda") if chunk else None
        out_dev = torch.empty_like(dw.q)
        out_host = torch.zeros(w.q.shape, dtype=torch.int16).pin_memory()
        pda.paged_decode_step_host(hq.view(torch.bfloat16), hk, hv, hbt, hsl, dq, dk, dv, dbt, dsl,
                                   dw.k_cache, dw.v_cache, float(w.scale), chunk, po, pl,
                                   out_dev, out_host, workspace=pda.new_workspace(w.batch, 8),
                                   status=dw.status)
        torch.cuda.synchronize()
        got = W.bf16_bits_to_f32(out_host.numpy().view(np.uint16)).astype(np.float64)
        assert_close(got, ref, what=f"step_host chunk {chunk}")
        k_ref, _ = host_appended(oracle, w)
        assert (bf16_to_bits(dw.k_cache) == k_ref).all()
        # in place: no staging buffers, the kernel reads q / k_new / v_new from and writes the result to
        # the pinned (device-mapped) host buffers; same result, and a plain (unmapped) buffer is refused
        dw = DeviceWorkload(w)
        out_host2 = torch.zeros(w.q.shape, dtype=torch.int16).pin_memory()
        pda.paged_decode_step_host(hq.view(torch.bfloat16), hk, hv, hbt, hsl, None, None, None, dbt, dsl,
                                   dw.k_cache, dw.v_cache, float(w.scale), chunk, po, pl,
                                   None, out_host2, workspace=pda.new_workspace(w.batch, 8),
                                   status=dw.status)
        torch.cuda.synchronize()
        got2 = W.bf16_bits_to_f32(out_host2.numpy().view(np.uint16)).astype(np.float64)
        assert_close(got2, ref, what=f"step_host in place chunk {chunk}")
        assert (bf16_to_bits(dw.k_cache) == k_ref).all()
        assert int(dw.status.item()) == 0
        # everything in place: block_table and seq_lens are read from the pinned host buffers too, so
        # the step is the kernel launch and nothing else
        dw = DeviceWorkload(w)
        out_host3 = torch.zeros(w.q.shape, dtype=torch.int16).pin_memory()
        pda.paged_decode_step_host(hq.view(torch.bfloat16), hk, hv, hbt, hsl, None, None, None, None, None,
                                   dw.k_cache, dw.v_cache, float(w.scale), chunk, po, pl,
                                   None, out_host3, workspace=pda.new_workspace(w.batch, 8),
                                   status=dw.status)
        torch.cuda.synchronize()
        got3 = W.bf16_bits_to_f32(out_host3.numpy().view(np.uint16)).astype(np.float64)
        assert_close(got3, ref, what=f"step_host all in place chunk {chunk}")
        assert (got3 == got2).all()
        assert (bf16_to_bits(dw.k_cache) == k_ref).all()
        assert int(dw.status.item()) == 0
    with pytest.raises(RuntimeError):
        pda.paged_decode_step_host(hq.view(torch.bfloat16), hk, hv, hbt, hsl, None, None, None, dbt, dsl,
                                   dw.k_cache, dw.v_cache, float(w.scale), 0, None, None,
                                   None, torch.zeros(w.q.shape, dtype=torch.int16), status=dw.status)


# ---- sliding window -------------------------------------------------------------------------

@pytest.mark.parametrize("flags", PATHS)
@pytest.mark.parametrize("shape", [(8, 2, 64), (32, 8, 128)])
def test_sliding_window(oracle, flags, shape):
    Hq, Hkv, D = shape
    lens = [1, 15, 16, 17, 40, 100, 333, 1000]
    w = W.make_workload("win", lens, Hq, Hkv, D, seed=61)
    dw = DeviceWorkload(w)
    dw.append()
    k, v = host_appended(oracle, w)
    for window in (1, 7, 16, 33, 128, 5000):
        ref, _ = oracle.paged_decode_attention(w.q, k, v, w.block_table, w.seq_lens, w.scale, window=window)
        # pages wholly before the window may be evicted: poison their table entries
        bt = dw.block_table.clone()
        for b, L in enumerate(lens):
            first_live = max(0, L - window) // 16
            bt[b, :first_live] = -7
        out = pda.paged_window_decode_attention(dw.q, dw.k_cache, dw.v_cache, bt, dw.seq_lens,
                                                float(w.scale), window, flags=flags, status=dw.status)
        assert_close(bf16_to_f64(out), ref, what=f"window {window} unsplit")
        if window == 1:   # the last V row, bit for bit
            got = bf16_to_bits(out)
            for b in range(len(lens)):
                assert (got[b, 0] == w.v_new[b, 0]).all()
        for chunk in (32, 256):
            mc = pda.max_chunks(max(lens), chunk)
            po = torch.full((w.batch, Hq, mc, D), float("nan"), dtype=torch.float32, device="cuda")
            pl = torch.full((w.batch, Hq, mc), float("nan"), dtype=torch.float32, device="cuda")
            pda.paged_window_decode_attention(dw.q, dw.k_cache, dw.v_cache, bt, dw.seq_lens, float(w.scale),
                                              window, chunk_tokens=chunk, part_o=po, part_lse=pl, flags=flags,
                                              status=dw.status)
            out_s = pda.paged_decode_reduce(po, pl, dw.seq_lens, chunk)
            assert_close(bf16_to_f64(out_s), ref, what=f"window {window} chunk {chunk}")
    assert status_of(dw) == 0


# ---- quantising append into e4m3 caches ------------------------------------------------------

@pytest.mark.parametrize("shape", [(8, 2, 64), (32, 8, 128)])
def test_fp8_append_bit_exact_and_attention_on_the_grown_cache(oracle, shape):
    Hq, Hkv, D = shape
    B, T = 5, 40
    start = np.array([0, 3, 15, 16, 31], np.int32)
    rng = np.random.default_rng(11)
    pages_per_seq = (int(start.max()) + T + 15) // 16
    n_pages = B * pages_per_seq + 3
    table = rng.permutation(n_pages)[:B * pages_per_seq].reshape(B, pages_per_seq).astype(np.int32)
    hk = np.full((n_pages, Hkv, 16, D), 0xFF, np.uint8); hv = hk.copy()
    hks = np.full((n_pages, Hkv), np.nan, np.float32); hvs = hks.copy()
    # caches start empty except for `start` tokens appended through the oracle itself
    dk, dv = torch.from_numpy(hk.copy()).cuda(), torch.from_numpy(hv.copy()).cuda()
    dks, dvs = torch.from_numpy(hks.copy()).cuda(), torch.from_numpy(hvs.copy()).cuda()
    bt = torch.from_numpy(table).cuda()
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    lens = np.zeros(B, np.int32)
    for t in range(int(start.max()) + T):
        active = (t < start + T)
        lens = lens + active.astype(np.int32)
        cur = np.where(active, lens, 0).astype(np.int32)      # inactive rows append nothing
        scale_up = 1.0 + 5.0 * (t % 7 == 3)                     # some rows exceed their page's range
        kn = W.f32_to_bf16_bits((rng.standard_normal((B, Hkv, D)) * scale_up).astype(np.float32))
        vn = W.f32_to_bf16_bits(rng.standard_normal((B, Hkv, D)).astype(np.float32))
        oracle.kv_append_e4m3(kn, vn, hk, hv, hks, hvs, table, cur)
        pda.kv_append_fp8(bf16_tensor(kn), bf16_tensor(vn), dk, dv, dks, dvs, bt,
                          torch.from_numpy(cur).cuda(), status=status)
    assert (dk.cpu().numpy() == hk).all() and (dv.cpu().numpy() == hv).all()
    gks, gvs = dks.cpu().numpy(), dvs.cpu().numpy()
    live = ~np.isnan(hks)
    assert (np.isnan(gks) == np.isnan(hks)).all() and (gks[live] == hks[live]).all() and (gvs[live] == hvs[live]).all()
    assert int(status.item()) == 0
    # attention over the grown cache
    q = W.f32_to_bf16_bits(rng.standard_normal((B, Hq, D), dtype=np.float32))
    ref, _ = oracle.paged_decode_attention(q, hk, hv, table, lens, np.float32(1 / np.sqrt(D)), hks, hvs)
    out = pda.paged_decode_attention(bf16_tensor(q), dk, dv, bt, torch.from_numpy(lens).cuda(),
                                     float(np.float32(1 / np.sqrt(D))), k_scale=dks, v_scale=dvs, status=status)
    assert_close(bf16_to_f64(out), ref, "e4m3", what="attention after fp8 appends")


@pytest.mark.parametrize("shape", [(8, 2, 64), (32, 8, 128)])
def test_fp8_block_append_bit_exact_and_verified(oracle, shape):
    """Blocks of T tokens quantised into e4m3 caches: bytes and scales equal the oracle's (which is the
    one-token rule in order), over several blocks that open pages in their middle, start from empty
    sequences and include a sequence shorter than a block; then the block is verified over that cache."""
    Hq, Hkv, D = shape
    B, T, n_blocks = 4, 7, 5
    rng = np.random.default_rng(21)
    first = np.array([7, 20, 3, 16], np.int32)      # lengths after the first block (3 < T: partial block)
    max_len = int(first.max()) + T * (n_blocks - 1)
    pages_per_seq = (max_len + 15) // 16
    n_pages = B * pages_per_seq + 2
    table = rng.permutation(n_pages)[:B * pages_per_seq].reshape(B, pages_per_seq).astype(np.int32)
    hk = np.full((n_pages, Hkv, 16, D), 0xFF, np.uint8); hv = hk.copy()
    hks = np.full((n_pages, Hkv), np.nan, np.float32); hvs = hks.copy()
    # sequence 1 has 13 earlier tokens (so that its first block lands in the middle of a page it did not open)
    pre = np.array([0, 13, 0, 9], np.int32)
    for t in range(int(pre.max())):
        cur = np.where(t < pre, t + 1, 0).astype(np.int32)
        kn1 = W.f32_to_bf16_bits(rng.standard_normal((B, Hkv, D)).astype(np.float32))
        vn1 = W.f32_to_bf16_bits(rng.standard_normal((B, Hkv, D)).astype(np.float32))
        oracle.kv_append_e4m3(kn1, vn1, hk, hv, hks, hvs, table, cur)
    dk, dv = torch.from_numpy(hk.copy()).cuda(), torch.from_numpy(hv.copy()).cuda()
    dks, dvs = torch.from_numpy(hks.copy()).cuda(), torch.from_numpy(hvs.copy()).cuda()
    bt = torch.from_numpy(table).cuda()
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    lens = first.copy()
    for blk in range(n_blocks):
        amp = 1.0 + 4.0 * (blk == 2)
        kn = W.f32_to_bf16_bits((rng.standard_normal((B, T, Hkv, D)) * amp).astype(np.float32))
        vn = W.f32_to_bf16_bits(rng.standard_normal((B, T, Hkv, D)).astype(np.float32))
        oracle.kv_append_tokens_e4m3(kn, vn, hk, hv, hks, hvs, table, lens)
        pda.kv_append_tokens_fp8(bf16_tensor(kn), bf16_tensor(vn), dk, dv, dks, dvs, bt,
                                 torch.from_numpy(lens).cuda(), status=status)
        assert (dk.cpu().numpy() == hk).all() and (dv.cpu().numpy() == hv).all(), f"block {blk}"
        gks, gvs = dks.cpu().numpy(), dvs.cpu().numpy()
        live = ~np.isnan(hks)
        assert (np.isnan(gks) == np.isnan(hks)).all() and (gks[live] == hks[live]).all() and (gvs[live] == hvs[live]).all()
        if blk < n_blocks - 1:
            lens = lens + T
    assert int(status.item()) == 0
    if D != 128:
        return      # multi-query attention over e4m3 caches is built for head_dim 128
    # the last block's queries over the cache that now holds it
    scale = np.float32(1 / np.sqrt(D))
    q = W.f32_to_bf16_bits(rng.standard_normal((B, T, Hq, D), dtype=np.float32))
    ref, _ = oracle.paged_verify_attention(q, hk, hv, table, lens, scale, hks, hvs)
    out = pda.paged_verify_attention(bf16_tensor(q), dk, dv, bt, torch.from_numpy(lens).cuda(), float(scale),
                                     k_scale=dks, v_scale=dvs, status=status)
    assert_close(bf16_to_f64(out), ref, "e4m3", what="verify after fp8 block appends")
    assert int(status.item()) == 0


@pytest.mark.parametrize("kv_dtype", ["bf16", "e4m3"])
@pytest.mark.parametrize("B", [2, 31, 33, 128, 129, 200, 256, 257])
def test_longest_first_order_visits_every_sequence_once(oracle, B, kv_dtype):
    """Unsplit launches of up to 256 sequences serve the sequences by decreasing length: 64 length buckets,
    by index inside a bucket, every CTA computing the same order. Batches on either side of a warp's 32
    sequences and of the 128 threads, with many equal lengths, empty sequences, and one sequence far longer
    than the rest (which sets the bucket width): every row must be right, i.e. every sequence was taken by
    exactly one CTA per kv head. 257 sequences: no ordering."""
    rng = np.random.default_rng(900 + B)
    lens = rng.integers(0, 40, size=B)
    lens[rng.integers(0, B, size=max(B // 8, 1))] = 17          # ties
    lens[rng.integers(0, B)] = 2100                             # one long sequence
    w = W.make_workload("order", lens, 8, 2, 128, kv_dtype=kv_dtype, seed=901 + B)
    dw = DeviceWorkload(w)
    if kv_dtype == "bf16":
        dw.append()
    ref = oracle_out(oracle, w)
    for rep in range(2):
        assert_close(bf16_to_f64(dw.attend()), ref, kv_dtype, what=f"B={B} {kv_dtype} launch {rep}")
    assert status_of(dw) == 0
