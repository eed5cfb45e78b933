"""Failure reporting: a wait that runs out inside a kernel is seen by the host without hanging anything.

The production kernels bound every mbarrier wait (about 1 s).  This test does not touch them: it runs
the library's self-test kernel, whose one wait (on a barrier that nothing arrives at) has a 1 ms limit,
and follows the report through the C ABI: status word, error code of the next call, clearing, and a
correct result afterwards.  Nothing here faults, traps or hangs the GPU; the kernel returns normally.
"""
import pytest
import torch

import paper_2603_15619_b200 as moda
from paper_2603_15619_b200 import binding, synthetic

from parity import assert_forward_close, oracle_forward

pytestmark = pytest.mark.gpu


def test_expired_wait_is_reported_by_the_next_call_and_cleared():
    w = synthetic.Workload("st", 1, 200, 2, 64, 0)
    x = synthetic.make(w, seed=5, device="cuda")
    moda.moda_attn_fwd(x["Q"], x["K"], x["V"], None, 0, w.scale)          # sets up the host mirror of the status word
    assert moda.moda_last_status() == 0
    try:
        moda.moda_selftest_wait_timeout()
        torch.cuda.synchronize()                                          # the kernel returned by itself
        with pytest.raises(binding.ModaError) as e:
            moda.moda_attn_fwd(x["Q"], x["K"], x["V"], None, 0, w.scale)
        assert e.value.code == binding.MODA_ERR_DEVICE_TIMEOUT
        assert moda.moda_last_status() == binding.MODA_SELFTEST_WAIT_STATUS   # site 255, reason 1 (wait ran out)
    finally:
        moda.moda_last_status(clear=True)
    assert moda.moda_last_status() == 0
    O, LSE = moda.moda_attn_fwd(x["Q"], x["K"], x["V"], None, 0, w.scale)
    assert_forward_close(O, LSE, *oracle_forward(x, w.scale), "after clearing the status word")
