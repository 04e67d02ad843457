"""A multi-token decode loop captured ONCE in a CUDA graph: each replay advances
seq_lens on the device and runs the fused step (append + attention + reduce).
Every step's output and the final caches are checked against the oracle run on
a host copy that grows the same way. Lengths cross page and chunk boundaries."""
import numpy as np
import pytest
import torch

from paper_2605_06068_b200 import binding as pda
from paper_2605_06068_b200 import workloads as W

from util import assert_close, bf16_tensor, bf16_to_bits, bf16_to_f64

pytestmark = pytest.mark.gpu


@pytest.fixture(params=["persistent", "per_unit"])
def step_kernel(request):
    pda.set_persistent_threshold(0 if request.param == "persistent" else 1 << 30)
    yield request.param
    pda.set_persistent_threshold(6)


@pytest.mark.parametrize("chunk", [0, 32])
@pytest.mark.parametrize("shape", [(8, 2, 64), (32, 8, 128)])
def test_graph_replayed_decode_loop(oracle, chunk, shape, step_kernel):
    if chunk and step_kernel == "persistent":
        pytest.skip("the persistent kernel serves unsplit launches only")
    Hq, Hkv, D = shape
    T = 20
    start = np.array([1, 14, 15, 16, 30, 47, 200], np.int32)
    w = W.make_workload("loop", start + T, Hq, Hkv, D, seed=31)     # tables sized for the final lengths
    rng = np.random.default_rng(5)
    q_t = W.f32_to_bf16_bits(rng.standard_normal((T, len(start), Hq, D), dtype=np.float32))
    k_t = W.f32_to_bf16_bits(rng.standard_normal((T, len(start), Hkv, D), dtype=np.float32))
    v_t = W.f32_to_bf16_bits(rng.standard_normal((T, len(start), Hkv, D), dtype=np.float32))

    # device state (static addresses: the graph bakes them in)
    kc, vc = bf16_tensor(w.k_cache), bf16_tensor(w.v_cache)
    bt = torch.from_numpy(w.block_table).cuda()
    sl = torch.from_numpy(start - 1).cuda()          # the first replay advances to `start`
    q, kn, vn = bf16_tensor(q_t[0]), bf16_tensor(k_t[0]), bf16_tensor(v_t[0])
    dq, dk, dv = bf16_tensor(q_t), bf16_tensor(k_t), bf16_tensor(v_t)
    out = torch.empty_like(q)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    ws = pda.new_workspace(len(start), Hkv)
    po = pl = None
    if chunk:
        mc = pda.max_chunks(int((start + T).max()), chunk)
        po = torch.empty((len(start), Hq, mc, D), dtype=torch.float32, device="cuda")
        pl = torch.empty((len(start), Hq, mc), dtype=torch.float32, device="cuda")

    def step(stream):
        pda.advance_seq_lens(sl, 1, stream=stream)
        pda.paged_decode_step(q, kn, vn, kc, vc, bt, sl, float(w.scale), chunk_tokens=chunk, out=out,
                              part_o=po, part_lse=pl, workspace=ws, status=status, stream=stream)

    s = torch.cuda.Stream()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.stream(s):
        # warm-up outside capture (first-use set-up), then undo its effect on the state
        step(s)
        s.synchronize()
        sl.copy_(torch.from_numpy(start - 1).cuda())
        kc.copy_(bf16_tensor(w.k_cache)); vc.copy_(bf16_tensor(w.v_cache))
        s.synchronize()
        with torch.cuda.graph(g, stream=s):
            step(s)
    torch.cuda.synchronize()

    # host mirror
    hk, hv = w.k_cache.copy(), w.v_cache.copy()
    lens = start.copy() - 1
    for t in range(T):
        q.copy_(dq[t]); kn.copy_(dk[t]); vn.copy_(dv[t])
        g.replay()
        torch.cuda.synchronize()
        lens = lens + 1
        oracle.kv_append(k_t[t], v_t[t], hk, hv, w.block_table, lens)
        ref, _ = oracle.paged_decode_attention(q_t[t], hk, hv, w.block_table, lens, w.scale)
        assert (sl.cpu().numpy() == lens).all()
        assert_close(bf16_to_f64(out), ref, what=f"graph step {t}")
    assert (bf16_to_bits(kc) == hk).all() and (bf16_to_bits(vc) == hv).all()
    assert int(status.item()) == 0 and (ws == 0).all()
