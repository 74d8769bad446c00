"""Failure detection without a GPU fault: the producer of the tensor-core prefill is told (on
the host, through a test-only symbol) to load nothing, so every device-side wait runs into its limit.  The kernel must
unwind by itself, report SP_ERR_TIMEOUT through the workspace status word, and leave the
context usable: the next ordinary call gives the same result as before."""
import math

import numpy as np
import pytest
import torch

import paper_2404_06910_b200 as sp
from helpers import dev, workspace
from workloads import build_layout

pytestmark = pytest.mark.gpu


def test_prefill_bounded_waits_report_timeout_and_context_survives():
    lay = build_layout([32], [[100, 40]], [[24, 24]])
    H, D = 2, 128
    g = torch.Generator().manual_seed(5)
    q, k, v = (torch.randn(lay.total_tokens, H, D, generator=g).bfloat16() for _ in range(3))
    dl = sp.DeviceLayout.from_host(lay)
    qd, kd, vd = dev(q), dev(k), dev(v)
    ws = workspace(sp.sp_prefill_workspace_bytes(dl, H, D, sp.SP_BF16))

    def run():
        out = torch.zeros_like(qd)
        sp.sp_superpose_prefill(qd, kd, vd, dl, 1 / math.sqrt(D), out, None, ws)
        return out

    good = run()
    sp.sp_check_status(ws)

    sp.lib.sp_test_stall_producer(1)            # test-only symbol: the producer loads nothing from now on
    try:
        run()
        with pytest.raises(sp.SpError) as e:
            sp.sp_check_status(ws)
        assert e.value.code == sp.SP_ERR_TIMEOUT
    finally:
        sp.lib.sp_test_stall_producer(0)

    again = run()
    sp.sp_check_status(ws)                      # status word is cleared by the next call
    torch.cuda.synchronize()
    assert torch.equal(good, again)
