"""GPU parity at the full sizes of the five named workloads, in the launch
configuration bench.py times (same chunk choices), against the full oracle."""
import numpy as np
import pytest

from paper_2605_06068_b200 import binding as pda
from paper_2605_06068_b200 import workloads as W

from util import DeviceWorkload, assert_close, bf16_to_bits, bf16_to_f64, host_appended, oracle_out

pytestmark = pytest.mark.gpu

# (workload, chunk_tokens used by bench.py; 0 = unsplit as well)
CASES = [("llama8b", 512), ("longctx", 2048), ("chat70b", 512), ("prefix_fp8", 512)]


@pytest.mark.parametrize("name,chunk", CASES)
def test_full_size_config(oracle, name, chunk):
    w = W.WORKLOADS[name]()
    if w.chunk_tokens:
        assert chunk == w.chunk_tokens
    dw = DeviceWorkload(w)
    k, v = host_appended(oracle, w)
    if w.kv_dtype == "bf16":
        dw.append()
        assert (bf16_to_bits(dw.k_cache) == k).all() and (bf16_to_bits(dw.v_cache) == v).all()
    ref = oracle_out(oracle, w, k, v)
    out = bf16_to_f64(dw.attend(chunk_tokens=chunk))
    worst, nerr = assert_close(out, ref, w.kv_dtype, what=f"{name} chunk {chunk}")
    print(f"{name}: chunk {chunk}: max err/tol {worst:.3f}, max err/rms {nerr:.3e}")
    if name != "longctx":   # one unit per (sequence, kv head) would serialise 131k tokens
        out_u = bf16_to_f64(dw.attend())
        assert_close(out_u, ref, w.kv_dtype, what=f"{name} unsplit")
    assert int(dw.status.item()) == 0
    # the output is not trivially small: the stated tolerance alone cannot tell at long context
    assert np.sqrt((out ** 2).mean()) > 0.5 * np.sqrt((ref ** 2).mean())
