"""The library's failure handling on the device, exercised without a fault: the bounded waits of the
attention kernels are made to run out on a barrier that nobody arrives at, and the device stays usable."""
import numpy as np
import pytest
import torch

from paper_2605_06068_b200 import binding as pda
from paper_2605_06068_b200 import workloads as W

from util import DeviceWorkload, assert_close, bf16_to_f64, oracle_out

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("polls", [1, 2000, 50000])
def test_bounded_waits_expire_and_report(oracle, polls):
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    result = torch.full((3,), -1, dtype=torch.int64, device="cuda")
    pda.debug_wait_timeout(polls, status, result)
    torch.cuda.synchronize()                      # the kernel returned: neither wait hung
    assert int(status.item()) == 3                # PDA_DEV_TIMEOUT
    assert pda.status_string(3).startswith("device: bounded wait")
    t_suspended, t_spinning, wrongly_done = (int(x) for x in result.cpu())
    assert wrongly_done == 0                      # neither wait claimed a phase that never completed
    assert 0 < t_suspended < 2_000_000_000 and 0 < t_spinning < 2_000_000_000
    if polls >= 2000:                             # a suspended poll may sleep up to 1 us, never longer
        assert t_suspended / polls < 5_000, t_suspended / polls
        assert t_spinning / polls < 5_000, t_spinning / polls
    # the context is intact: an ordinary call on the same stream right after gives the oracle's result
    w = W.make_workload("after_timeout", [300, 17, 1025], 32, 8, 128, seed=7)
    dw = DeviceWorkload(w)
    dw.append()
    out = dw.attend()
    assert_close(bf16_to_f64(out), oracle_out(oracle, w), what="decode after an expired wait")
    assert int(dw.status.item()) == 0


def test_wait_timeout_argument_checks():
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    for polls in (0, (1 << 20) + 1):
        with pytest.raises(RuntimeError, match="invalid argument"):
            pda.debug_wait_timeout(polls, status)
    with pytest.raises(RuntimeError, match="invalid argument"):
        pda.debug_wait_timeout(10, None)
    assert int(status.item()) == 0


def test_read_probe_reads_without_writing():
    buf = torch.arange(1 << 22, dtype=torch.int32, device="cuda")      # 16 MiB
    before = buf.clone()
    sink = torch.zeros(1, dtype=torch.int32, device="cuda")
    pda.debug_read_probe(buf, sink)
    pda.debug_read_probe(buf[: (1 << 22) - 4 * 37], sink)              # a length that is no multiple of the stride
    torch.cuda.synchronize()
    assert torch.equal(buf, before)
