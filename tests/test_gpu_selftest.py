"""The bounded wait of the kernels, made to run out on purpose: a kernel waits on a barrier that nothing signals,
gives up after the limit it was handed, reports ARB_DEV_WAIT_TIMEOUT and ends normally.  Nothing faults or hangs;
the context must serve the next call correctly."""
import numpy as np
import pytest
import torch

from paper_2512_05033_b200 import workloads as wl
from tests import helpers as H

pytestmark = pytest.mark.gpu


def test_wait_gives_up_reports_and_leaves_the_context_usable():
    from paper_2512_05033_b200 import binding
    c = H.ctx()
    assert c.poll_status() == 0
    limit = 2_000_000                      # about a millisecond of SM cycles
    report = c.selftest_wait_timeout(limit)
    torch.cuda.synchronize()               # returns: the kernel ended by itself
    ended, gave_up, waited = (int(x) for x in report.cpu())
    assert ended == 1
    assert gave_up == 64                   # warp 0 by its own limit, warp 1 through the abort flag
    assert limit < waited < 50 * limit     # it did wait, and not much longer than asked
    assert c.poll_status() == binding.DEV_WAIT_TIMEOUT
    assert c.poll_status() == 0            # reading clears the word
    # the same context, next call: decode through the tensor-core kernel and the CUDA-core kernel, and a chunk
    for ql, flags in (([1, 1, 1], 0), ([1, 1, 1], binding.ATTN_NO_TENSOR_CORES), ([1, 9, 40], 0)):
        inp = wl.small_attn_case(3, 12, 2, 128, torch.bfloat16, [3000, 150, 1024], ql, seed=611)
        out, bits = H.gpu_attn(inp, flags=flags)
        ref, _ = H.oracle_attn(inp)
        assert bits == 0
        H.assert_close(out, ref, torch.bfloat16, tight=3e-3)


def test_wait_limit_is_validated_on_the_host():
    from paper_2512_05033_b200 import binding
    c = H.ctx()
    report = torch.zeros(3, dtype=torch.int32, device="cuda")
    for bad in (0, -5, (1 << 31) + 1):
        st = binding.lib.arb_selftest_wait_timeout(c._h, bad, report.data_ptr(), None)
        assert st == binding.ARB_ERR_INVALID_ARG
    assert binding.lib.arb_selftest_wait_timeout(c._h, 1000, None, None) == binding.ARB_ERR_INVALID_ARG
    torch.cuda.synchronize()
    assert int(report[0]) == 0 and c.poll_status() == 0
