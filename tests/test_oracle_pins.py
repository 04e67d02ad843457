"""Pins for the fp64 CPU oracle (no GPU): each check ties the oracle to
something fixed outside it -- a library routine on densely gathered pages,
closed forms, invariants, bit definitions -- so that a dropped term, a wrong
index or a transposed operand fails at least one of them."""
import math
import os

import numpy as np
import pytest
import torch

from paper_2605_06068_b200 import workloads as W

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def appended(oracle, w):
    """Caches after this step's kv_append (host copy)."""
    k, v = w.k_cache.copy(), w.v_cache.copy()
    oracle.kv_append(w.k_new, w.v_new, k, v, w.block_table, w.seq_lens)
    return k, v


def dense_kv(w, k, v, b):
    """Gather sequence b's pages to dense float64 [Hkv, L, D] (independent of the oracle)."""
    L, P = int(w.seq_lens[b]), w.page_size
    n = (L + P - 1) // P
    pages = w.block_table[b, :n]
    if w.kv_dtype == "bf16":
        K = W.bf16_bits_to_f32(k[pages]).astype(np.float64)
        V = W.bf16_bits_to_f32(v[pages]).astype(np.float64)
    else:
        K = torch.from_numpy(k[pages].copy()).view(torch.float8_e4m3fn).to(torch.float64).numpy()
        V = torch.from_numpy(v[pages].copy()).view(torch.float8_e4m3fn).to(torch.float64).numpy()
        K = K * w.k_scale[pages].astype(np.float64)[:, :, None, None]
        V = V * w.v_scale[pages].astype(np.float64)[:, :, None, None]
    # [n, Hkv, P, D] -> [Hkv, n*P, D] -> first L tokens
    K = K.transpose(1, 0, 2, 3).reshape(w.num_kv_heads, n * P, w.head_dim)[:, :L]
    V = V.transpose(1, 0, 2, 3).reshape(w.num_kv_heads, n * P, w.head_dim)[:, :L]
    return K, V


def sdpa_reference(w, k, v):
    """torch's scaled_dot_product_attention (fp64, CPU, GQA by repeat) per sequence."""
    out = np.zeros((w.batch, w.num_q_heads, w.head_dim))
    G = w.num_q_heads // w.num_kv_heads
    for b in range(w.batch):
        K, V = dense_kv(w, k, v, b)
        q = torch.from_numpy(W.bf16_bits_to_f32(w.q[b]).astype(np.float64))[None, :, None, :]
        Kt = torch.from_numpy(K).repeat_interleave(G, dim=0)[None]
        Vt = torch.from_numpy(V).repeat_interleave(G, dim=0)[None]
        o = torch.nn.functional.scaled_dot_product_attention(q, Kt, Vt, scale=float(w.scale))
        out[b] = o[0, :, 0, :].numpy()
    return out


@pytest.mark.parametrize("seed", [42, 43, 44, 45])
def test_matches_library_sdpa_on_tiny(oracle, seed):
    w = W.tiny(seed=seed)
    k, v = appended(oracle, w)
    out, lse = oracle.paged_decode_attention(w.q, k, v, w.block_table, w.seq_lens, w.scale)
    ref = sdpa_reference(w, k, v)
    assert np.isfinite(out).all()
    np.testing.assert_allclose(out, ref, rtol=0, atol=1e-12)
    # lse against a dense logsumexp
    G = w.num_q_heads // w.num_kv_heads
    for b in range(w.batch):
        K, _ = dense_kv(w, k, v, b)
        q = W.bf16_bits_to_f32(w.q[b]).astype(np.float64)
        for h in range(w.num_q_heads):
            s = float(w.scale) * (K[h // G] @ q[h])
            ref_lse = float(torch.logsumexp(torch.from_numpy(s), 0))
            assert abs(lse[b, h] - ref_lse) < 1e-12


@pytest.mark.parametrize("shape", [(1, 1, 32), (4, 4, 64), (8, 1, 128), (6, 2, 96)])
def test_matches_library_sdpa_other_head_layouts(oracle, shape):
    """G = 1 (MHA), Hkv = 1 (MQA) and an odd group size reduce to textbook attention."""
    Hq, Hkv, D = shape
    w = W.make_workload("x", [1, 5, 16, 31, 48], Hq, Hkv, D, seed=7)
    k, v = appended(oracle, w)
    out, _ = oracle.paged_decode_attention(w.q, k, v, w.block_table, w.seq_lens, w.scale)
    np.testing.assert_allclose(out, sdpa_reference(w, k, v), rtol=0, atol=1e-12)


def test_single_token_returns_v_exactly(oracle):
    w = W.make_workload("one", [1, 1, 1], 8, 2, 64, seed=3)
    k, v = appended(oracle, w)
    out, lse = oracle.paged_decode_attention(w.q, k, v, w.block_table, w.seq_lens, w.scale)
    for b in range(3):
        page = w.block_table[b, 0]
        for h in range(8):
            expect = W.bf16_bits_to_f32(v[page, h // 4, 0]).astype(np.float64)
            assert (out[b, h] == expect).all()
            # and that value is the appended row
            assert (v[page, h // 4, 0] == w.v_new[b, h // 4]).all()
            kq = float(w.scale) * np.dot(W.bf16_bits_to_f32(k[page, h // 4, 0]).astype(np.float64),
                                         W.bf16_bits_to_f32(w.q[b, h]).astype(np.float64))
            assert abs(lse[b, h] - kq) < 1e-13


def test_equal_scores_give_mean_of_v(oracle):
    w = W.tiny(seed=11)
    k, v = appended(oracle, w)
    zero_q = np.zeros_like(w.q)
    out, lse = oracle.paged_decode_attention(zero_q, k, v, w.block_table, w.seq_lens, w.scale)
    for b in range(w.batch):
        _, V = dense_kv(w, k, v, b)
        for h in range(w.num_q_heads):
            np.testing.assert_allclose(out[b, h], V[h // 4].mean(axis=0), rtol=0, atol=1e-13)
            assert abs(lse[b, h] - math.log(int(w.seq_lens[b]))) < 1e-13
    # scale = 0 has the same effect with a non-zero q
    out2, _ = oracle.paged_decode_attention(w.q, k, v, w.block_table, w.seq_lens, 0.0)
    np.testing.assert_allclose(out2, out, rtol=0, atol=1e-13)


def test_two_token_logistic_closed_form(oracle):
    w = W.make_workload("two", [2, 2], 4, 2, 32, seed=5)
    k, v = appended(oracle, w)
    out, _ = oracle.paged_decode_attention(w.q, k, v, w.block_table, w.seq_lens, w.scale)
    for b in range(2):
        K, V = dense_kv(w, k, v, b)
        for h in range(4):
            q = W.bf16_bits_to_f32(w.q[b, h]).astype(np.float64)
            s0, s1 = float(w.scale) * (K[h // 2] @ q)
            sig = 1.0 / (1.0 + math.exp(-(s0 - s1)))
            expect = sig * V[h // 2, 0] + (1.0 - sig) * V[h // 2, 1]
            np.testing.assert_allclose(out[b, h], expect, rtol=0, atol=1e-13)


def test_hand_worked_example(oracle):
    """A case worked by hand: D=2... stored under tests/golden with its derivation."""
    rows = [l.split() for l in open(os.path.join(GOLD, "two_token_example.txt")) if l[:1] not in "#\n"]
    vals = {r[0]: [float(x) for x in r[1:]] for r in rows}
    D, P = 32, 16
    # one sequence, one head, two tokens; only the first two dims are non-zero
    q = np.zeros((1, 1, D), np.float32); q[0, 0, :2] = vals["q"]
    K = np.zeros((1, 1, P, D), np.float32); V = np.zeros((1, 1, P, D), np.float32)
    K[0, 0, 0, :2] = vals["k0"]; K[0, 0, 1, :2] = vals["k1"]
    V[0, 0, 0, :2] = vals["v0"]; V[0, 0, 1, :2] = vals["v1"]
    out, lse = oracle.paged_decode_attention(
        W.f32_to_bf16_bits(q), W.f32_to_bf16_bits(K), W.f32_to_bf16_bits(V),
        np.array([[0]], np.int32), np.array([2], np.int32), vals["scale"][0])
    np.testing.assert_allclose(out[0, 0, :2], vals["out"], rtol=0, atol=1e-15)
    assert abs(lse[0, 0] - vals["lse"][0]) < 1e-15
    assert (out[0, 0, 2:] == 0).all()


def test_page_placement_invariance_and_poison(oracle):
    w = W.tiny(seed=42)
    k, v = appended(oracle, w)
    out, lse = oracle.paged_decode_attention(w.q, k, v, w.block_table, w.seq_lens, w.scale)
    rng = np.random.default_rng(1)
    perm = rng.permutation(w.num_pages)            # new id of old page p is perm[p]
    k2 = np.empty_like(k); v2 = np.empty_like(v)
    k2[perm] = k; v2[perm] = v
    table2 = np.where(w.block_table >= 0, perm[np.maximum(w.block_table, 0)], -1).astype(np.int32)
    out2, lse2 = oracle.paged_decode_attention(w.q, k2, v2, table2, w.seq_lens, w.scale)
    assert (out2 == out).all() and (lse2 == lse).all()
    # changing the poison (unused slots, unused pages, table tail) changes nothing
    k3, v3 = k.copy(), v.copy()
    used = np.zeros(w.num_pages, bool)
    for b in range(w.batch):
        L = int(w.seq_lens[b]); n = (L + 15) // 16
        used[w.block_table[b, :n]] = True
        if L % 16:
            k3[w.block_table[b, n - 1], :, L % 16:, :] = 0x1234
            v3[w.block_table[b, n - 1], :, L % 16:, :] = 0x7F80  # +inf
    k3[~used] = 0; v3[~used] = 0x7F80
    table3 = np.where(w.block_table >= 0, w.block_table, 2 ** 31 - 1).astype(np.int32)
    out3, _ = oracle.paged_decode_attention(w.q, k3, v3, table3, w.seq_lens, w.scale)
    assert (out3 == out).all()


def test_convexity_and_gqa_sharing(oracle):
    w = W.tiny(seed=9)
    k, v = appended(oracle, w)
    q = w.q.copy()
    q[:, 1] = q[:, 0]; q[:, 2] = q[:, 0]; q[:, 3] = q[:, 0]   # heads 0..3 share kv head 0
    out, _ = oracle.paged_decode_attention(q, k, v, w.block_table, w.seq_lens, w.scale)
    assert (out[:, 1] == out[:, 0]).all() and (out[:, 3] == out[:, 0]).all()
    assert not (out[:, 4] == out[:, 0]).all()
    for b in range(w.batch):
        _, V = dense_kv(w, k, v, b)
        for h in range(w.num_q_heads):
            lo, hi = V[h // 4].min(axis=0), V[h // 4].max(axis=0)
            assert (out[b, h] >= lo - 1e-12).all() and (out[b, h] <= hi + 1e-12).all()


def test_needle_token_dominates(oracle):
    """One key aligned with q at score 30 above the rest pulls out its own V row."""
    w = W.make_workload("needle", [100], 4, 1, 64, seed=13)
    k, v = appended(oracle, w)
    qf = W.bf16_bits_to_f32(w.q[0, 0]).astype(np.float64)
    for j in (0, 15, 16, 98, 99):
        k2, v2 = k.copy(), v.copy()
        page, slot = w.block_table[0, j // 16], j % 16
        coef = 40.0 / (float(w.scale) * float(qf @ qf))
        k2[page, 0, slot] = W.f32_to_bf16_bits((coef * qf).astype(np.float32))
        v2[page, 0, slot] = W.f32_to_bf16_bits(np.arange(1, 65, dtype=np.float32))
        out, _ = oracle.paged_decode_attention(w.q, k2, v2, w.block_table, w.seq_lens, w.scale)
        np.testing.assert_allclose(out[0, 0], np.arange(1, 65), rtol=0, atol=1e-6)


def test_empty_sequence(oracle):
    w = W.make_workload("empty", [0, 3], 2, 1, 32, seed=2)
    k, v = appended(oracle, w)
    out, lse = oracle.paged_decode_attention(w.q, k, v, w.block_table, w.seq_lens, w.scale)
    assert (out[0] == 0).all() and np.isneginf(lse[0]).all()
    assert np.isfinite(out[1]).all()


# ---- kv_append ---------------------------------------------------------------------------

def test_kv_append_is_a_copy_into_the_right_slot():
    import oracle
    w = W.tiny(seed=42)
    k, v = w.k_cache.copy(), w.v_cache.copy()
    oracle.kv_append(w.k_new, w.v_new, k, v, w.block_table, w.seq_lens)
    # numpy restatement by fancy indexing on the flattened token axis
    expect_k, expect_v = w.k_cache.copy(), w.v_cache.copy()
    for b, L in enumerate([17, 33, 64, 100]):
        page = w.block_table[b, (L - 1) // 16]
        expect_k[page, :, (L - 1) % 16, :] = w.k_new[b]
        expect_v[page, :, (L - 1) % 16, :] = w.v_new[b]
    assert (k == expect_k).all() and (v == expect_v).all()
    changed = (k != w.k_cache).sum()
    assert changed <= 4 * 2 * 64 and changed > 0
    # the lengths exercise: first slot of a fresh page, last slot of a page, mid-page
    assert [(L - 1) % 16 for L in (17, 33, 64, 100)] == [0, 0, 15, 3]


def test_append_then_attend_equals_cache_built_directly(oracle):
    w = W.tiny(seed=21)
    k, v = appended(oracle, w)
    out, _ = oracle.paged_decode_attention(w.q, k, v, w.block_table, w.seq_lens, w.scale)
    ref = sdpa_reference(w, k, v)
    np.testing.assert_allclose(out, ref, rtol=0, atol=1e-12)
    # the last token seen by attention is the appended one
    for b in range(w.batch):
        K, V = dense_kv(w, k, v, b)
        np.testing.assert_array_equal(K[:, -1], W.bf16_bits_to_f32(w.k_new[b]).astype(np.float64))
        np.testing.assert_array_equal(V[:, -1], W.bf16_bits_to_f32(w.v_new[b]).astype(np.float64))


# ---- split + reduce ----------------------------------------------------------------------

@pytest.mark.parametrize("chunk", [16, 32, 48, 256])
def test_split_then_reduce_equals_unsplit(oracle, chunk):
    w = W.tiny(seed=42)
    k, v = appended(oracle, w)
    out, lse = oracle.paged_decode_attention(w.q, k, v, w.block_table, w.seq_lens, w.scale)
    mc = (100 + chunk - 1) // chunk
    po, pl = oracle.paged_decode_attention(w.q, k, v, w.block_table, w.seq_lens, w.scale,
                                           chunk_tokens=chunk, max_chunks=mc)
    # chunks that do not exist are untouched (NaN-filled by the wrapper)
    for b in range(w.batch):
        n = (int(w.seq_lens[b]) + chunk - 1) // chunk
        assert np.isfinite(po[b, :, :n]).all() and np.isnan(po[b, :, n:]).all()
    out2, lse2 = oracle.paged_decode_reduce(po, pl, w.seq_lens, chunk)
    np.testing.assert_allclose(out2, out, rtol=0, atol=1e-12)
    np.testing.assert_allclose(lse2, lse, rtol=0, atol=1e-12)
    # each chunk on its own is plain attention over that token range (library routine)
    G = 4
    for b in range(w.batch):
        K, V = dense_kv(w, k, v, b)
        L = int(w.seq_lens[b])
        for c in range((L + chunk - 1) // chunk):
            t0, t1 = c * chunk, min((c + 1) * chunk, L)
            for h in (0, 5):
                q = torch.from_numpy(W.bf16_bits_to_f32(w.q[b, h]).astype(np.float64))
                s = float(w.scale) * (torch.from_numpy(K[h // G, t0:t1]) @ q)
                p = torch.softmax(s, 0)
                np.testing.assert_allclose(po[b, h, c], (p @ torch.from_numpy(V[h // G, t0:t1])).numpy(),
                                           rtol=0, atol=1e-12)


def test_reduce_special_cases(oracle):
    rng = np.random.default_rng(0)
    po = rng.standard_normal((2, 3, 4, 8))
    # a single chunk is the identity
    out, lse = oracle.paged_decode_reduce(po, np.full((2, 3, 4), 1.5), np.array([7, 16]), 16)
    np.testing.assert_array_equal(out, po[:, :, 0])
    assert (lse == 1.5).all()
    # equal lse over n chunks gives the plain average and lse + log n
    out, lse = oracle.paged_decode_reduce(po, np.full((2, 3, 4), -2.0), np.array([64, 33]), 16)
    np.testing.assert_allclose(out[0], po[0].mean(axis=1), atol=1e-15)
    np.testing.assert_allclose(out[1], po[1, :, :3].mean(axis=1), atol=1e-15)
    np.testing.assert_allclose(lse[0], -2.0 + math.log(4), atol=1e-15)
    # a chunk whose lse is far below the others has no weight
    pl = np.zeros((2, 3, 4)); pl[:, :, 1] = -800.0
    out, _ = oracle.paged_decode_reduce(po, pl, np.array([32, 32]), 16)
    np.testing.assert_allclose(out, po[:, :, 0], atol=1e-15)
    # no chunk at all
    out, lse = oracle.paged_decode_reduce(po, pl, np.array([0, 0]), 16)
    assert (out == 0).all() and np.isneginf(lse).all()


# ---- e4m3 --------------------------------------------------------------------------------

def test_e4m3_table_against_bit_definition_and_library_cast(oracle):
    t = oracle.e4m3_decode_table()
    lib = torch.arange(256, dtype=torch.uint8).view(torch.float8_e4m3fn).to(torch.float64).numpy()
    assert np.isnan(t[0x7F]) and np.isnan(t[0xFF]) and np.isnan(t).sum() == 2
    ok = ~np.isnan(t)
    assert (t[ok] == lib[ok]).all() and np.isnan(lib[~ok]).all()
    # spot values fixed by the format definition (tests/golden/e4m3_values.txt)
    for line in open(os.path.join(GOLD, "e4m3_values.txt")):
        if line.startswith("#") or not line.strip():
            continue
        code, val = line.split()
        assert t[int(code, 16)] == float(val), line
    # monotone over the positive finite codes, antisymmetric in the sign bit
    assert (np.diff(t[:0x7F]) > 0).all()
    assert (t[0x80:0xFF] == -t[0x00:0x7F]).all()


def test_quantiser_matches_library_cast_and_round_trip(oracle):
    w = W.prefix_fp8(seed=46, batch=3)
    kb, valid = w.notes["k_bf16"], w.notes["valid_slots"]
    q8, sc = oracle.quantize_pages_e4m3(kb, valid)
    used = valid > 0
    P = w.page_size
    slot_ok = np.arange(P)[None, :] < valid[:, None]                     # [pages, P]
    m = np.broadcast_to(slot_ok[:, None, :, None], q8.shape)
    # same bytes and scales as the workload's library-cast encoder
    assert (q8[m] == w.k_cache[m]).all()
    assert (sc[used] == w.k_scale[used]).all()
    # round trip within half an e4m3 ulp of the scaled value; amax maps to +-448
    t = oracle.e4m3_decode_table()
    x = W.bf16_bits_to_f32(kb).astype(np.float64)
    y = x / sc.astype(np.float64)[:, :, None, None]
    deq = t[q8]
    ulp = np.where(np.abs(y) < 2.0 ** -6, 2.0 ** -9, 2.0 ** (np.floor(np.log2(np.maximum(np.abs(y), 1e-300))) - 3))
    assert (np.abs(deq - y)[m] <= 0.5 * ulp[m] * (1 + 1e-6)).all()
    amax_code = np.abs(deq).max(axis=(2, 3), where=m, initial=0.0)
    assert (amax_code[used] == 448.0).all()
    z = (x == 0) & m
    assert (deq[z] == 0).all()


def test_fp8_attention_matches_library_sdpa_on_dequantised_cache(oracle):
    w = W.prefix_fp8(seed=46, batch=3)
    out, _ = oracle.paged_decode_attention(w.q, w.k_cache, w.v_cache, w.block_table, w.seq_lens,
                                           w.scale, w.k_scale, w.v_scale)
    ref = sdpa_reference(w, w.k_cache, w.v_cache)
    np.testing.assert_allclose(out, ref, rtol=0, atol=1e-12)
    # all rows alias the same prefix pages
    assert (w.block_table[:, :128] == w.block_table[0, :128]).all()


# ---- sliding window ----------------------------------------------------------------------

@pytest.mark.parametrize("window", [1, 5, 16, 17, 40, 1000])
def test_window_matches_library_sdpa_on_the_last_tokens(oracle, window):
    w = W.tiny(seed=42)
    k, v = appended(oracle, w)
    out, lse = oracle.paged_decode_attention(w.q, k, v, w.block_table, w.seq_lens, w.scale, window=window)
    G = w.num_q_heads // w.num_kv_heads
    for b in range(w.batch):
        K, V = dense_kv(w, k, v, b)
        lo = max(0, int(w.seq_lens[b]) - window)
        q = torch.from_numpy(W.bf16_bits_to_f32(w.q[b]).astype(np.float64))[None, :, None, :]
        Kt = torch.from_numpy(K[:, lo:]).repeat_interleave(G, dim=0)[None]
        Vt = torch.from_numpy(V[:, lo:]).repeat_interleave(G, dim=0)[None]
        o = torch.nn.functional.scaled_dot_product_attention(q, Kt, Vt, scale=float(w.scale))
        np.testing.assert_allclose(out[b], o[0, :, 0, :].numpy(), rtol=0, atol=1e-12)
    # window = 1 returns the last V row exactly; a window covering everything changes nothing
    if window == 1:
        for b in range(w.batch):
            assert (out[b, 0] == W.bf16_bits_to_f32(w.v_new[b, 0]).astype(np.float64)).all()
    if window == 1000:
        full, _ = oracle.paged_decode_attention(w.q, k, v, w.block_table, w.seq_lens, w.scale)
        assert (out == full).all()
    # split + reduce under a window equals the unsplit windowed result
    po, pl = oracle.paged_decode_attention(w.q, k, v, w.block_table, w.seq_lens, w.scale,
                                           chunk_tokens=32, max_chunks=4, window=window)
    out2, lse2 = oracle.paged_decode_reduce(po, pl, w.seq_lens, 32)
    np.testing.assert_allclose(out2, out, rtol=0, atol=1e-12)
    np.testing.assert_allclose(lse2, lse, rtol=0, atol=1e-12)


# ---- multi-token append and verification (causal block) attention -------------------------

def verify_case(oracle, lens, T, Hq, Hkv, D, seed):
    """A workload whose last T tokens per sequence are appended as a block; returns the pieces."""
    w = W.make_workload("verify", lens, Hq, Hkv, D, seed=seed)
    rng = np.random.default_rng(seed + 1)
    B = len(lens)
    q = W.f32_to_bf16_bits(rng.standard_normal((B, T, Hq, D), dtype=np.float32))
    kn = W.f32_to_bf16_bits(rng.standard_normal((B, T, Hkv, D), dtype=np.float32))
    vn = W.f32_to_bf16_bits(rng.standard_normal((B, T, Hkv, D), dtype=np.float32))
    k, v = w.k_cache.copy(), w.v_cache.copy()
    oracle.kv_append_tokens(kn, vn, k, v, w.block_table, w.seq_lens)
    return w, q, kn, vn, k, v


def test_multi_token_append_places_each_token(oracle):
    w, q, kn, vn, k, v = verify_case(oracle, [16, 17, 40, 100], 16, 8, 2, 64, seed=3)
    expect_k, expect_v = w.k_cache.copy(), w.v_cache.copy()
    for b, L in enumerate([16, 17, 40, 100]):
        for i in range(16):
            pos = L - 16 + i
            page = w.block_table[b, pos // 16]
            expect_k[page, :, pos % 16, :] = kn[b, i]
            expect_v[page, :, pos % 16, :] = vn[b, i]
    assert (k == expect_k).all() and (v == expect_v).all()
    # one token per sequence is the single-token append
    k1, v1 = w.k_cache.copy(), w.v_cache.copy()
    k2, v2 = w.k_cache.copy(), w.v_cache.copy()
    oracle.kv_append(w.k_new, w.v_new, k1, v1, w.block_table, w.seq_lens)
    oracle.kv_append_tokens(w.k_new[:, None], w.v_new[:, None], k2, v2, w.block_table, w.seq_lens)
    assert (k1 == k2).all() and (v1 == v2).all()


@pytest.mark.parametrize("T", [1, 4, 16])
def test_verify_attention_matches_library_sdpa_with_causal_mask(oracle, T):
    lens = [16, 17, 40, 100]
    w, q, kn, vn, k, v = verify_case(oracle, lens, T, 8, 2, 64, seed=9)
    out, lse = oracle.paged_verify_attention(q, k, v, w.block_table, w.seq_lens, w.scale)
    G = 4
    for b, L in enumerate(lens):
        K, V = dense_kv(w, k, v, b)
        qq = torch.from_numpy(W.bf16_bits_to_f32(q[b]).astype(np.float64)).permute(1, 0, 2)[None]  # [1,Hq,T,D]
        Kt = torch.from_numpy(K).repeat_interleave(G, dim=0)[None]
        Vt = torch.from_numpy(V).repeat_interleave(G, dim=0)[None]
        mask = torch.arange(L)[None, :] <= (L - T + torch.arange(T))[:, None]               # [T, L]
        o = torch.nn.functional.scaled_dot_product_attention(qq, Kt, Vt, attn_mask=mask, scale=float(w.scale))
        np.testing.assert_allclose(out[b], o[0].permute(1, 0, 2).numpy(), rtol=0, atol=1e-12)
    # the last query token sees everything: it equals plain decode attention with that q
    full, lse_full = oracle.paged_decode_attention(q[:, -1], k, v, w.block_table, w.seq_lens, w.scale)
    assert (out[:, -1] == full).all() and (lse[:, -1] == lse_full).all()
    # the first query token of a block that starts the sequence sees only itself: out = its V row
    if T == 16:
        assert (out[0, 0, 0] == W.bf16_bits_to_f32(vn[0, 0, 0]).astype(np.float64)).all()


# ---- quantising append ---------------------------------------------------------------------

def test_e4m3_append_policy_against_library_cast(oracle):
    """Scale is set by the page's first row (amax*2/448); later rows reuse it and saturate."""
    rng = np.random.default_rng(3)
    Hkv, D, P = 2, 64, 16
    n_pages = 4
    kc = np.full((n_pages, Hkv, P, D), 0xFF, np.uint8); vc = kc.copy()
    ks = np.full((n_pages, Hkv), np.nan, np.float32); vs = ks.copy()
    table = np.array([[2, 0], [3, 1]], np.int32)
    hist = {}
    for step in range(20):                       # lengths 1..20: pages opened at L=1 and L=17
        lens = np.array([step + 1, step + 1], np.int32)
        kn = W.f32_to_bf16_bits((rng.standard_normal((2, Hkv, D)) * (1 + 3 * (step % 5 == 4))).astype(np.float32))
        vn = W.f32_to_bf16_bits(rng.standard_normal((2, Hkv, D)).astype(np.float32))
        if step == 7:
            kn[0, 0] = 0                          # an all-zero row
        oracle.kv_append_e4m3(kn, vn, kc, vc, ks, vs, table, lens)
        hist[step] = (kn, vn)
    # restate with torch's cast (saturating by clamp) page by page
    for b in range(2):
        for step in range(20):
            page, slot = table[b, step // 16], step % 16
            first = hist[(step // 16) * 16]
            for g in range(Hkv):
                for src, cache, scales in ((0, kc, ks), (1, vc, vs)):
                    x0 = torch.from_numpy(W.bf16_bits_to_f32(first[src][b, g]))
                    sc = (x0.abs().max() * 2.0) / 448.0
                    assert scales[page, g] == np.float32(sc)
                    x = torch.from_numpy(W.bf16_bits_to_f32(hist[step][src][b, g]))
                    y = (x / sc).clamp(-448.0, 448.0).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
                    got = cache[page, g, slot]
                    same = (got == y) | ((got & 0x7F) == 0) & ((y & 0x7F) == 0)   # +-0 alike
                    assert same.all(), (b, step, g, src)
    # untouched slots keep their fill; the zero row quantises to zero codes
    assert (kc[table[0, 1], :, 4:, :] == 0xFF).all()
    assert ((kc[table[0, 0], 0, 7] & 0x7F) == 0).all()
    # a row 4x larger than the page's first row saturates at +-448 somewhere
    t = oracle.e4m3_decode_table()
    assert np.abs(t[kc[table[0, 0], :, 4]]).max() == 448.0


def test_e4m3_block_append_is_the_one_token_rule_in_order(oracle):
    """A block of T tokens appended at once must leave exactly what T one-token appends (pinned
    above against the library cast) leave: same bytes, same scales, including pages opened inside
    the block (their scale comes from the block's own row in slot 0) and sequences shorter than T."""
    rng = np.random.default_rng(11)
    Hkv, D, P, T = 2, 64, 16, 7
    n_pages = 8
    table = np.array([[2, 0, 5], [3, 1, 6], [4, 7, 0]], np.int32)
    final = np.array([21, 16, 3], np.int32)       # crosses a page boundary / ends on one / shorter than the block
    kn = W.f32_to_bf16_bits((rng.standard_normal((3, T, Hkv, D)) * 2).astype(np.float32))
    vn = W.f32_to_bf16_bits(rng.standard_normal((3, T, Hkv, D)).astype(np.float32))

    def fresh():
        kc = np.full((n_pages, Hkv, P, D), 0xFF, np.uint8)
        ks = np.full((n_pages, Hkv), np.nan, np.float32)
        return kc, kc.copy(), ks, ks.copy()

    # history before the block: one-token appends up to final - T
    kc, vc, ks, vs = fresh()
    kc2, vc2, ks2, vs2 = fresh()
    for step in range(int((final - T).max())):
        lens = np.minimum(step + 1, np.maximum(final - T, 0)).astype(np.int32)
        if step >= lens.max():
            break
        hk = W.f32_to_bf16_bits(np.random.default_rng(100 + step).standard_normal((3, Hkv, D)).astype(np.float32))
        hv = W.f32_to_bf16_bits(np.random.default_rng(200 + step).standard_normal((3, Hkv, D)).astype(np.float32))
        active = (step + 1) <= np.maximum(final - T, 0)
        lens = np.where(active, step + 1, 0).astype(np.int32)      # length 0: no append for that sequence
        for args in ((kc, vc, ks, vs), (kc2, vc2, ks2, vs2)):
            oracle.kv_append_e4m3(hk, hv, args[0], args[1], args[2], args[3], table, lens)
    # the block at once ...
    oracle.kv_append_tokens_e4m3(kn, vn, kc, vc, ks, vs, table, final)
    # ... against token by token
    for i in range(T):
        at = final - T + i                          # position of token i
        lens = np.where(at >= 0, at + 1, 0).astype(np.int32)
        oracle.kv_append_e4m3(np.ascontiguousarray(kn[:, i]), np.ascontiguousarray(vn[:, i]),
                              kc2, vc2, ks2, vs2, table, lens)
    assert (kc == kc2).all() and (vc == vc2).all()
    assert np.array_equal(ks, ks2, equal_nan=True) and np.array_equal(vs, vs2, equal_nan=True)
    # a block of one token is the one-token append
    a, b = fresh(), fresh()
    lens1 = np.array([1, 17, 5], np.int32)
    oracle.kv_append_tokens_e4m3(kn[:, :1], vn[:, :1], a[0], a[1], a[2], a[3], table, lens1)
    oracle.kv_append_e4m3(np.ascontiguousarray(kn[:, 0]), np.ascontiguousarray(vn[:, 0]), b[0], b[1], b[2], b[3], table, lens1)
    assert (a[0] == b[0]).all() and (a[1] == b[1]).all()
