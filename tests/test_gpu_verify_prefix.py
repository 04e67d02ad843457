"""GPU parity of the multi-query kernel's two uses: verification attention over a
block of draft tokens (causal inside the block) and the shared-prefix cascade."""
import numpy as np
import pytest
import torch

from paper_2605_06068_b200 import binding as pda
from paper_2605_06068_b200 import workloads as W

from util import DeviceWorkload, assert_close, bf16_tensor, bf16_to_bits, bf16_to_f64, oracle_out

pytestmark = pytest.mark.gpu

# the multi-query kernels: tcgen05 + TMEM where it applies (bf16, head_dim 128), else / forced mma.sync
MQ = [pytest.param(0, id="tcgen05"), pytest.param(pda.PDA_FLAG_MQ_MMA_SYNC, id="mma_sync"),
      pytest.param(pda.PDA_FLAG_MQ_ONE_UNIT, id="tcgen05_one_unit")]


def verify_inputs(w, T, seed):
    rng = np.random.default_rng(seed)
    B = w.batch
    q = W.f32_to_bf16_bits(rng.standard_normal((B, T, w.num_q_heads, w.head_dim), dtype=np.float32))
    kn = W.f32_to_bf16_bits(rng.standard_normal((B, T, w.num_kv_heads, w.head_dim), dtype=np.float32))
    vn = W.f32_to_bf16_bits(rng.standard_normal((B, T, w.num_kv_heads, w.head_dim), dtype=np.float32))
    return q, kn, vn


@pytest.mark.parametrize("flags", MQ)
@pytest.mark.parametrize("T", [1, 4, 16, 40])
@pytest.mark.parametrize("shape", [(8, 2, 64), (32, 8, 128), (64, 8, 128), (8, 8, 128)],
                         ids=lambda s: f"Hq{s[0]}kv{s[1]}D{s[2]}")
def test_verify_attention_and_block_append(oracle, shape, T, flags):
    Hq, Hkv, D = shape
    lens = [40, 41, 63, 64, 100, 640, 1300]
    w = W.make_workload("verify", lens, Hq, Hkv, D, seed=19)
    q, kn, vn = verify_inputs(w, T, 20)
    k, v = w.k_cache.copy(), w.v_cache.copy()
    oracle.kv_append_tokens(kn, vn, k, v, w.block_table, w.seq_lens)
    ref, _ = oracle.paged_verify_attention(q, k, v, w.block_table, w.seq_lens, w.scale)

    dw = DeviceWorkload(w)
    pda.kv_append_tokens(bf16_tensor(kn), bf16_tensor(vn), dw.k_cache, dw.v_cache, dw.block_table,
                         dw.seq_lens, status=dw.status)
    assert (bf16_to_bits(dw.k_cache) == k).all() and (bf16_to_bits(dw.v_cache) == v).all()
    dq = bf16_tensor(q)
    out = pda.paged_verify_attention(dq, dw.k_cache, dw.v_cache, dw.block_table, dw.seq_lens,
                                     float(w.scale), flags=flags, status=dw.status)
    assert_close(bf16_to_f64(out), ref, what=f"verify T={T} unsplit")
    for chunk in (64, 256):
        mc = pda.max_chunks(max(lens), chunk)
        po = torch.full((w.batch, T, Hq, mc, D), float("nan"), dtype=torch.float32, device="cuda")
        pl = torch.full((w.batch, T, Hq, mc), float("nan"), dtype=torch.float32, device="cuda")
        out_s = pda.paged_verify_attention(dq, dw.k_cache, dw.v_cache, dw.block_table, dw.seq_lens,
                                           float(w.scale), chunk_tokens=chunk, part_o=po, part_lse=pl,
                                           flags=flags, status=dw.status)
        assert_close(bf16_to_f64(out_s), ref, what=f"verify T={T} chunk {chunk}")
    # the last query token sees the whole sequence: same as plain decode attention (up to rounding)
    plain = pda.paged_decode_attention(dq[:, -1].contiguous(), dw.k_cache, dw.v_cache, dw.block_table,
                                       dw.seq_lens, float(w.scale), status=dw.status)
    assert np.abs(bf16_to_f64(plain) - bf16_to_f64(out)[:, -1]).max() < 1e-2
    assert int(dw.status.item()) == 0


def test_verify_attention_fp8_and_causal_needle(oracle):
    w = W.prefix_fp8(seed=46, batch=4)
    T = 16
    q, _, _ = verify_inputs(w, T, 21)
    ref, _ = oracle.paged_verify_attention(q, w.k_cache, w.v_cache, w.block_table, w.seq_lens, w.scale,
                                           w.k_scale, w.v_scale)
    dw = DeviceWorkload(w)
    out = pda.paged_verify_attention(bf16_tensor(q), dw.k_cache, dw.v_cache, dw.block_table, dw.seq_lens,
                                     float(w.scale), k_scale=dw.k_scale, v_scale=dw.v_scale, status=dw.status)
    assert_close(bf16_to_f64(out), ref, "e4m3", what="verify fp8")
    assert int(dw.status.item()) == 0

    # causal structure: make the LAST key of a block dominant for every query; only the last
    # query may see it, every earlier one must not
    lens = [200]
    w = W.make_workload("needle", lens, 4, 1, 128, seed=23)
    q, kn, vn = verify_inputs(w, T, 24)
    q[:] = q[:, :1, :1]                       # one q row everywhere
    qf = W.bf16_bits_to_f32(q[0, 0, 0]).astype(np.float64)
    kn[0, -1, 0] = W.f32_to_bf16_bits((40.0 / (float(w.scale) * (qf @ qf)) * qf).astype(np.float32))
    vn[0, -1, 0] = W.f32_to_bf16_bits(np.arange(1, 129, dtype=np.float32))
    dw = DeviceWorkload(w)
    pda.kv_append_tokens(bf16_tensor(kn), bf16_tensor(vn), dw.k_cache, dw.v_cache, dw.block_table, dw.seq_lens)
    out = bf16_to_f64(pda.paged_verify_attention(bf16_tensor(q), dw.k_cache, dw.v_cache, dw.block_table,
                                                 dw.seq_lens, float(w.scale)))
    assert np.abs(out[0, -1, 0] - np.arange(1, 129)).max() <= 0.5
    assert np.abs(out[0, :-1]).max() < 3.0    # N(0,1) averages, nowhere near 1..128


@pytest.mark.parametrize("T", [1, 16, 40])
def test_verify_more_units_than_sms(oracle, T):
    """Enough (sequence, kv head, row block) units that the persistent kernel carries several per CTA: units
    of one iteration and of many, odd page counts, ragged tails, one and two row blocks, and (T = 16) a share
    of the units claimed from the counter rather than dealt."""
    rng = np.random.default_rng(300 + T)
    B = 40 if T != 16 else 90
    lens = np.maximum(rng.integers(1, 900, size=B), T)
    lens[:4] = [T, 64, 65, 128]
    w = W.make_workload("many_units", lens, 32, 8, 128, seed=301 + T)
    q, kn, vn = verify_inputs(w, T, 302 + T)
    k, v = w.k_cache.copy(), w.v_cache.copy()
    oracle.kv_append_tokens(kn, vn, k, v, w.block_table, w.seq_lens)
    ref, _ = oracle.paged_verify_attention(q, k, v, w.block_table, w.seq_lens, w.scale)
    dw = DeviceWorkload(w)
    pda.kv_append_tokens(bf16_tensor(kn), bf16_tensor(vn), dw.k_cache, dw.v_cache, dw.block_table, dw.seq_lens)
    for rep in range(3):   # repeated launches: the claim counter is back at zero each time
        out = pda.paged_verify_attention(bf16_tensor(q), dw.k_cache, dw.v_cache, dw.block_table, dw.seq_lens,
                                         float(w.scale), status=dw.status)
        assert_close(bf16_to_f64(out), ref, what=f"verify, {B * 8} units, T={T}, launch {rep}")
    # split calls: units are (sequence, chunk, kv head, row block); partials merged by the reduce launch
    for chunk in (64, 208, 512):
        mc = pda.max_chunks(int(lens.max()), chunk)
        po = torch.full((B, T, 32, mc, 128), float("nan"), dtype=torch.float32, device="cuda")
        pl = torch.full((B, T, 32, mc), float("nan"), dtype=torch.float32, device="cuda")
        for flags in (0, pda.PDA_FLAG_MQ_ONE_UNIT):
            po.fill_(float("nan"))
            out = pda.paged_verify_attention(bf16_tensor(q), dw.k_cache, dw.v_cache, dw.block_table, dw.seq_lens,
                                             float(w.scale), chunk_tokens=chunk, part_o=po, part_lse=pl,
                                             flags=flags, status=dw.status)
            assert_close(bf16_to_f64(out), ref, what=f"verify split {chunk}, T={T}, flags {flags}")
    assert int(dw.status.item()) == 0


@pytest.mark.parametrize("flags", MQ)
def test_verify_bad_table_entries_and_lengths_set_status(oracle, flags):
    """A page id outside the pool and a length beyond the block table: the status word reports them (the
    larger code wins), nothing is read outside the caches, and the other sequences' rows are right."""
    lens = [300, 90, 200, 47, 130, 64] + [40 + 7 * i for i in range(18)]   # 24 x 8 units: more than SMs
    T = 4
    w = W.make_workload("bad", lens, 32, 8, 128, seed=61)
    q, kn, vn = verify_inputs(w, T, 62)
    k, v = w.k_cache.copy(), w.v_cache.copy()
    oracle.kv_append_tokens(kn, vn, k, v, w.block_table, w.seq_lens)
    ref, _ = oracle.paged_verify_attention(q, k, v, w.block_table, w.seq_lens, w.scale)
    dw = DeviceWorkload(w)
    pda.kv_append_tokens(bf16_tensor(kn), bf16_tensor(vn), dw.k_cache, dw.v_cache, dw.block_table, dw.seq_lens)
    bt = dw.block_table.clone()
    bt[1, 2] = w.num_pages + 7      # sequence 1: a page id past the pool
    bt[4, 0] = -1                   # sequence 4: a negative page id
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    out = pda.paged_verify_attention(bf16_tensor(q), dw.k_cache, dw.v_cache, bt, dw.seq_lens, float(w.scale),
                                     flags=flags, status=st)
    got = bf16_to_f64(out)
    assert int(st.item()) == 1      # PDA_DEV_BAD_PAGE
    good = [b for b in range(len(lens)) if b not in (1, 4)]
    assert np.isfinite(got[good]).all()
    for b in good:
        assert_close(got[b:b + 1], ref[b:b + 1], what=f"sequence {b} beside a bad table row, flags {flags}")
    sl = dw.seq_lens.clone()
    sl[2] = bt.shape[1] * 16 + 5    # sequence 2: longer than its table row can describe
    st.zero_()
    out = pda.paged_verify_attention(bf16_tensor(q), dw.k_cache, dw.v_cache, dw.block_table, sl, float(w.scale),
                                     flags=flags, status=st)
    got = bf16_to_f64(out)
    assert int(st.item()) == 2      # PDA_DEV_BAD_SEQ_LEN
    for b in [b for b in range(len(lens)) if b != 2]:
        assert_close(got[b:b + 1], ref[b:b + 1], what=f"sequence {b} beside a bad length, flags {flags}")
    assert (got[2] == 0).all()      # the misdescribed sequence's rows are zero


@pytest.mark.parametrize("kv_dtype", ["bf16", "e4m3"])
def test_verify_batch_beyond_the_ranked_range(oracle, kv_dtype):
    """More than 128 sequences: the CTAs take the sequences in index order instead of longest first;
    lengths from one token to a few pages, so that single-iteration CTAs and odd page counts occur."""
    rng = np.random.default_rng(91)
    B, T = 150, 3
    lens = np.maximum(rng.integers(1, 200, size=B), T)
    w = W.make_workload("big_batch", lens, 32, 8, 128, kv_dtype=kv_dtype, seed=92)
    q, kn, vn = verify_inputs(w, T, 93)
    dw = DeviceWorkload(w)
    if kv_dtype == "bf16":  # (a bf16 workload's last slots are filled by the append)
        k, v = w.k_cache.copy(), w.v_cache.copy()
        oracle.kv_append_tokens(kn, vn, k, v, w.block_table, w.seq_lens)
        pda.kv_append_tokens(bf16_tensor(kn), bf16_tensor(vn), dw.k_cache, dw.v_cache, dw.block_table, dw.seq_lens)
        ref, _ = oracle.paged_verify_attention(q, k, v, w.block_table, w.seq_lens, w.scale)
    else:
        ref, _ = oracle.paged_verify_attention(q, w.k_cache, w.v_cache, w.block_table, w.seq_lens, w.scale,
                                               w.k_scale, w.v_scale)
    for chunk, flags in ((0, 0), (64, 0), (0, pda.PDA_FLAG_MQ_ONE_UNIT)):
        po = pl = None
        if chunk:
            mc = pda.max_chunks(int(lens.max()), chunk)
            po = torch.full((B, T, 32, mc, 128), float("nan"), dtype=torch.float32, device="cuda")
            pl = torch.full((B, T, 32, mc), float("nan"), dtype=torch.float32, device="cuda")
        out = pda.paged_verify_attention(bf16_tensor(q), dw.k_cache, dw.v_cache, dw.block_table, dw.seq_lens,
                                         float(w.scale), chunk_tokens=chunk, part_o=po, part_lse=pl,
                                         k_scale=dw.k_scale, v_scale=dw.v_scale, flags=flags, status=dw.status)
        assert_close(bf16_to_f64(out), ref, kv_dtype, what=f"verify batch {B} {kv_dtype} chunk {chunk} flags {flags}")
    assert int(dw.status.item()) == 0


@pytest.mark.parametrize("flags", MQ)
@pytest.mark.parametrize("spread", ["moderate", "extreme"])
def test_verify_fp8_under_unequal_scales(oracle, flags, spread):
    """e4m3 caches whose page scales differ by powers of two (the tensor-core path folds the K scale into
    the score factor and the V scale into the exponent and divides it out of the row sum), pages with a
    zero scale, query rows of very different magnitude (Q is split into two e4m3 parts after a per-row
    power-of-two scaling), and a lone dominant key (P = 1 next to tiny weights).
    moderate: V scales within 2^-3 .. 2^3 of each other; extreme: V scales over 2^-12 .. 2^8, values in
    the hundreds, where an output element can be small by cancellation between large terms. Both are
    checked element by element against the stated e4m3 tolerance, on every kernel choice."""
    rng = np.random.default_rng(77)
    lens = [1000, 333, 64, 17]
    T = 8
    w = W.make_workload("fp8_scales", lens, 32, 8, 128, kv_dtype="e4m3", seed=78)
    used = np.unique(w.block_table[w.block_table >= 0])
    ks, vs = w.k_scale.copy(), w.v_scale.copy()
    vexp = (-3, 4) if spread == "moderate" else (-12, 9)
    ks[used] *= np.exp2(rng.integers(-3, 2, size=ks[used].shape)).astype(np.float32)
    vs[used] *= np.exp2(rng.integers(*vexp, size=vs[used].shape)).astype(np.float32)
    vs[used[3]] = 0.0                                   # a page whose values all decode to zero
    vs[used[10], 2] = 0.0
    q = W.bf16_bits_to_f32(verify_inputs(w, T, 79)[0])
    q *= np.exp2(rng.integers(-8, 3, size=q.shape[:3])).astype(np.float32)[..., None]   # per (b, t, head)
    # a dominant key: row (b=0, t=T-1, head 5) points at the cache row of token 500 of sequence 0
    page, slot, g = int(w.block_table[0, 500 // 16]), 500 % 16, 5 // 4
    dec = np.asarray(oracle.e4m3_decode_table(), dtype=np.float64)
    krow = (dec[w.k_cache[page, g, slot]] * float(ks[page, g])).astype(np.float32)
    q[0, T - 1, 5] = (60.0 / (float(w.scale) * float(krow @ krow))) * krow
    q = W.f32_to_bf16_bits(q.astype(np.float32))
    ref, _ = oracle.paged_verify_attention(q, w.k_cache, w.v_cache, w.block_table, w.seq_lens, w.scale, ks, vs)
    dw = DeviceWorkload(w)
    out = pda.paged_verify_attention(bf16_tensor(q), dw.k_cache, dw.v_cache, dw.block_table, dw.seq_lens,
                                     float(w.scale), k_scale=torch.from_numpy(ks).cuda(),
                                     v_scale=torch.from_numpy(vs).cuda(), flags=flags, status=dw.status)
    got = bf16_to_f64(out)
    assert_close(got, ref, "e4m3", what=f"fp8 unequal scales ({spread}) flags {flags}")
    # the dominant key's row is that value row (times its scale), to the rounding of the output
    vrow = dec[w.v_cache[page, g, slot]] * float(vs[page, g])
    assert np.abs(got[0, T - 1, 5] - vrow).max() <= 2e-2 + 2e-2 * np.abs(vrow).max()
    assert int(dw.status.item()) == 0


@pytest.mark.parametrize("flags", MQ)
@pytest.mark.parametrize("kv_dtype", ["bf16", "e4m3"])
@pytest.mark.parametrize("B", [3, 40])
def test_shared_prefix_cascade(oracle, kv_dtype, B, flags):
    rng = np.random.default_rng(7)
    prefix = 512
    lens = prefix + rng.integers(0, 300, size=B)
    lens[0] = prefix                        # a sequence with an empty suffix
    w = W.make_workload("cascade", lens, 32, 8, 128, kv_dtype=kv_dtype, seed=29, shared_prefix_tokens=prefix)
    assert (w.block_table[:, :prefix // 16] == w.block_table[0, :prefix // 16]).all()
    dw = DeviceWorkload(w)
    if kv_dtype == "bf16":
        dw.append()
    from util import host_appended
    k, v = host_appended(oracle, w)
    ref = oracle_out(oracle, w, k, v)
    for pchunk, chunk in ((128, 64), (512, 256)):
        mc = (prefix + pchunk - 1) // pchunk + pda.max_chunks(int(lens.max()) - prefix + 1, chunk)
        po = torch.full((B, 32, mc, 128), float("nan"), dtype=torch.float32, device="cuda")
        pl = torch.full((B, 32, mc), float("nan"), dtype=torch.float32, device="cuda")
        out = pda.paged_prefix_decode_attention(dw.q, dw.k_cache, dw.v_cache, dw.block_table, dw.seq_lens,
                                                float(w.scale), prefix, pchunk, chunk, po, pl,
                                                k_scale=dw.k_scale, v_scale=dw.v_scale, flags=flags,
                                                status=dw.status)
        assert_close(bf16_to_f64(out), ref, kv_dtype, what=f"cascade {kv_dtype} B={B} chunks {pchunk}/{chunk}")
    plain = dw.attend()
    assert np.abs(bf16_to_f64(plain) - bf16_to_f64(out)).max() < 2e-2
    assert int(dw.status.item()) == 0


def test_shared_prefix_cascade_in_a_cuda_graph(oracle):
    """The cascade forks its suffix launch onto a library-owned stream; captured in a graph the fork
    and join become graph edges. Replays must give the eager (and the oracle's) result."""
    rng = np.random.default_rng(8)
    prefix, B = 1024, 12
    lens = prefix + rng.integers(1, 200, size=B)
    w = W.make_workload("cascade_graph", lens, 32, 8, 128, seed=30, shared_prefix_tokens=prefix)
    dw = DeviceWorkload(w)
    dw.append()
    from util import host_appended
    k, v = host_appended(oracle, w)
    ref = oracle_out(oracle, w, k, v)
    pchunk, chunk = 256, 64
    mc = prefix // pchunk + pda.max_chunks(int(lens.max()) - prefix + 1, chunk)
    po = torch.empty((B, 32, mc, 128), dtype=torch.float32, device="cuda")
    pl = torch.empty((B, 32, mc), dtype=torch.float32, device="cuda")
    out = torch.empty_like(dw.q)

    def run(stream=None):
        pda.paged_prefix_decode_attention(dw.q, dw.k_cache, dw.v_cache, dw.block_table, dw.seq_lens,
                                          float(w.scale), prefix, pchunk, chunk, po, pl, out=out,
                                          status=dw.status, stream=stream)
    run()                      # eager once: creates the side stream outside any capture
    torch.cuda.synchronize()
    eager = out.clone()
    assert_close(bf16_to_f64(eager), ref, what="cascade eager")
    s = torch.cuda.Stream()
    g = torch.cuda.CUDAGraph()
    s.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(s):
        with torch.cuda.graph(g, stream=s):
            run(s)
    for _ in range(3):
        out.zero_()
        po.fill_(float("nan"))
        g.replay()
        torch.cuda.synchronize()
        assert torch.equal(out.view(torch.int16), eager.view(torch.int16))
    assert int(dw.status.item()) == 0


def test_verify_persistent_kernel_in_a_cuda_graph(oracle):
    """The persistent kernel shares out its last units through a counter the library owns; a captured launch
    keeps its counter, which every replay must find at zero and leave at zero."""
    rng = np.random.default_rng(401)
    B, T = 120, 8
    lens = np.maximum(rng.integers(1, 700, size=B), T)
    w = W.make_workload("graph_units", lens, 32, 8, 128, seed=402)
    q, kn, vn = verify_inputs(w, T, 403)
    k, v = w.k_cache.copy(), w.v_cache.copy()
    oracle.kv_append_tokens(kn, vn, k, v, w.block_table, w.seq_lens)
    ref, _ = oracle.paged_verify_attention(q, k, v, w.block_table, w.seq_lens, w.scale)
    dw = DeviceWorkload(w)
    pda.kv_append_tokens(bf16_tensor(kn), bf16_tensor(vn), dw.k_cache, dw.v_cache, dw.block_table, dw.seq_lens)
    dq = bf16_tensor(q)
    out = torch.empty_like(dq)

    def run(stream=None):
        pda.paged_verify_attention(dq, dw.k_cache, dw.v_cache, dw.block_table, dw.seq_lens, float(w.scale),
                                   out=out, status=dw.status, stream=stream)
    run()
    torch.cuda.synchronize()
    eager = out.clone()
    assert_close(bf16_to_f64(eager), ref, what="verify eager")
    s = torch.cuda.Stream()
    g = torch.cuda.CUDAGraph()
    s.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(s):
        with torch.cuda.graph(g, stream=s):
            run(s)
    for _ in range(3):
        out.zero_()
        g.replay()
        torch.cuda.synchronize()
        assert torch.equal(out.view(torch.int16), eager.view(torch.int16))
        run()                  # eager launches between the replays take other counters
        torch.cuda.synchronize()
        assert torch.equal(out.view(torch.int16), eager.view(torch.int16))
    assert int(dw.status.item()) == 0


@pytest.mark.parametrize("T", [8, 40])
def test_verify_fp8_persistent_kernel_edge_cases(oracle, T):
    """The persistent e4m3 kernel (the default for unsplit calls on e4m3 caches): more units than SMs, so
    that every CTA walks through several; sequences that are empty, shorter than the block, and one
    token on either side of a page and of an iteration; 32 query rows per kv head (rows held twice, T = 8)
    and 160 (two row blocks, T = 40). Then a page id outside the pool and a length beyond the table: the
    status word reports them, those sequences' rows are zero and every other row is right. Last, the
    launch captured in a CUDA graph and replayed."""
    lens = [0, 3, 16, 17, 63, 64, 65, 700, 1, 129, 256, 300] + [30 + 11 * i for i in range(28)]   # 40 x 8 units
    w = W.make_workload("fp8_units", lens, 32, 8, 128, kv_dtype="e4m3", seed=171)
    q, _, _ = verify_inputs(w, T, 172)
    ref, _ = oracle.paged_verify_attention(q, w.k_cache, w.v_cache, w.block_table, w.seq_lens, w.scale,
                                           w.k_scale, w.v_scale)
    dw = DeviceWorkload(w)
    dq = bf16_tensor(q)
    out = pda.paged_verify_attention(dq, dw.k_cache, dw.v_cache, dw.block_table, dw.seq_lens, float(w.scale),
                                     k_scale=dw.k_scale, v_scale=dw.v_scale, status=dw.status)
    got = bf16_to_f64(out)
    assert_close(got, ref, "e4m3", what=f"persistent e4m3 verify T={T}")
    assert (got[0] == 0).all() and int(dw.status.item()) == 0        # the empty sequence's rows are zero
    one_unit = pda.paged_verify_attention(dq, dw.k_cache, dw.v_cache, dw.block_table, dw.seq_lens, float(w.scale),
                                          k_scale=dw.k_scale, v_scale=dw.v_scale, flags=pda.PDA_FLAG_MQ_ONE_UNIT)
    # the same arithmetic unit by unit (which softmax set takes which iteration differs, so not bit for bit)
    assert_close(bf16_to_f64(one_unit), ref, "e4m3", what=f"one-unit e4m3 verify T={T}")
    assert np.abs(bf16_to_f64(one_unit) - got).max() <= 4e-3
    # bad inputs
    bt = dw.block_table.clone()
    bt[7, 5] = w.num_pages + 3
    bt[10, 0] = -1
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    bad = bf16_to_f64(pda.paged_verify_attention(dq, dw.k_cache, dw.v_cache, bt, dw.seq_lens, float(w.scale),
                                                 k_scale=dw.k_scale, v_scale=dw.v_scale, status=st))
    assert int(st.item()) == 1      # PDA_DEV_BAD_PAGE
    good = [b for b in range(len(lens)) if b not in (7, 10)]
    assert_close(bad[good], ref[good], "e4m3", what="rows beside a bad table row")
    assert (bad[[7, 10]] == 0).all()
    sl = dw.seq_lens.clone()
    sl[11] = bt.shape[1] * 16 + 9
    st.zero_()
    bad = bf16_to_f64(pda.paged_verify_attention(dq, dw.k_cache, dw.v_cache, dw.block_table, sl, float(w.scale),
                                                 k_scale=dw.k_scale, v_scale=dw.v_scale, status=st))
    assert int(st.item()) == 2      # PDA_DEV_BAD_SEQ_LEN
    good = [b for b in range(len(lens)) if b != 11]
    assert_close(bad[good], ref[good], "e4m3", what="rows beside a bad length")
    assert (bad[11] == 0).all()
    # captured and replayed
    res = torch.empty_like(dq)
    s = torch.cuda.Stream()
    g = torch.cuda.CUDAGraph()
    s.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(s):
        with torch.cuda.graph(g, stream=s):
            pda.paged_verify_attention(dq, dw.k_cache, dw.v_cache, dw.block_table, dw.seq_lens, float(w.scale),
                                       out=res, k_scale=dw.k_scale, v_scale=dw.v_scale, status=dw.status, stream=s)
    for _ in range(3):
        res.zero_()
        g.replay()
        torch.cuda.synchronize()
        assert torch.equal(res.view(torch.int16), out.view(torch.int16))
    assert int(dw.status.item()) == 0


@pytest.mark.parametrize("kv_dtype", ["bf16", "e4m3"])
@pytest.mark.parametrize("shape", [(6, 2), (20, 4), (28, 4), (12, 1)], ids=lambda s: f"Hq{s[0]}kv{s[1]}")
def test_verify_group_sizes_that_are_not_powers_of_two(oracle, shape, kv_dtype):
    """Query row r of a (sequence, kv head) unit is (draft token r / G, head r % G): G = 3, 5, 7 and 12, with
    row counts that end inside a warp's 32 rows (T = 5: 15, 25, 35, 60 rows), fill one block exactly or not
    (T = 16: 48, 80, 112, 192 rows) and need two blocks. Enough sequences that the persistent kernels carry
    several units per CTA; the one-unit and the mma.sync kernels on the same inputs."""
    Hq, Hkv = shape
    rng = np.random.default_rng(500 + Hq)
    B = -(-330 // Hkv)                      # more than 2 x 148 units
    lens = np.maximum(rng.integers(1, 500, size=B), 16)
    lens[:3] = [16, 64, 65]
    w = W.make_workload("odd_group", lens, Hq, Hkv, 128, kv_dtype=kv_dtype, seed=501 + Hq)
    for T in (5, 16):
        q, kn, vn = verify_inputs(w, T, 502 + T)
        k, v = w.k_cache.copy(), w.v_cache.copy()
        dw = DeviceWorkload(w)
        if kv_dtype == "bf16":
            oracle.kv_append_tokens(kn, vn, k, v, w.block_table, w.seq_lens)
            pda.kv_append_tokens(bf16_tensor(kn), bf16_tensor(vn), dw.k_cache, dw.v_cache, dw.block_table, dw.seq_lens)
        ref, _ = oracle.paged_verify_attention(q, k, v, w.block_table, w.seq_lens, w.scale, w.k_scale, w.v_scale)
        for flags in (0, pda.PDA_FLAG_MQ_ONE_UNIT, pda.PDA_FLAG_MQ_MMA_SYNC):
            out = pda.paged_verify_attention(bf16_tensor(q), dw.k_cache, dw.v_cache, dw.block_table, dw.seq_lens,
                                             float(w.scale), k_scale=dw.k_scale, v_scale=dw.v_scale, flags=flags,
                                             status=dw.status)
            assert_close(bf16_to_f64(out), ref, kv_dtype, what=f"G={Hq // Hkv} T={T} {kv_dtype} flags {flags}")
    assert int(dw.status.item()) == 0


@pytest.mark.parametrize("flags", MQ)
def test_verify_sequences_shorter_than_the_block(oracle, flags):
    """A sequence with fewer tokens than the block has query tokens (position L - n + i < 0 for the first
    n - L of them): those rows attend nothing and are zero, the others follow the rule; an empty sequence
    gives zero rows. Among them enough ordinary sequences for several units per CTA."""
    T = 16
    lens = [0, 1, 5, 15, 16, 17, 0, 3] + [20 + 7 * i for i in range(40)]
    w = W.make_workload("short", lens, 32, 8, 128, seed=610)
    q, _, _ = verify_inputs(w, T, 611)
    k, v = w.k_cache.copy(), w.v_cache.copy()
    oracle.kv_append(w.k_new, w.v_new, k, v, w.block_table, w.seq_lens)   # (the workload's last token)
    ref, _ = oracle.paged_verify_attention(q, k, v, w.block_table, w.seq_lens, w.scale)
    for b, L in enumerate(lens[:8]):
        assert (ref[b, :max(T - L, 0)] == 0).all() and (L == 0 or np.abs(ref[b, T - 1]).max() > 0)
    dw = DeviceWorkload(w)
    dw.append()
    out = pda.paged_verify_attention(bf16_tensor(q), dw.k_cache, dw.v_cache, dw.block_table, dw.seq_lens,
                                     float(w.scale), flags=flags, status=dw.status)
    got = bf16_to_f64(out)
    assert_close(got, ref, what="verify with sequences shorter than the block")
    for b, L in enumerate(lens[:8]):
        assert (got[b, :max(T - L, 0)] == 0).all()
    assert int(dw.status.item()) == 0
