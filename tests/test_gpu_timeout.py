"""A bounded device-side wait that runs out: the kernel returns normally, the context reports
JUPITER_ERR_TIMEOUT exactly once, and the context keeps computing correctly afterwards.  The wait that runs out is
jupiter_wait_probe's: one CTA waiting, with a short limit, on a barrier that nobody arrives at -- nothing faults."""
import numpy as np
import pytest

import oracle
from workloads import synth
from tests.helpers import assert_close, run_gpu_prefill

pytestmark = pytest.mark.gpu


def test_wait_runs_out_is_reported_once_and_the_context_stays_usable():
    import torch
    import paper_2504_08242_b200 as J
    ctx = J.Context(0)
    try:
        assert ctx.poll_device_status() == J.OK
        n0 = ctx.launch_count()
        ctx.wait_probe(1_000_000)  # about half a millisecond of SM clocks
        assert ctx.launch_count() == n0 + 1
        assert ctx.poll_device_status() == J.ERR_TIMEOUT
        assert ctx.poll_device_status() == J.OK  # the poll cleared the word
        # the next real calls (tensor-core prefill, fused form) pass parity
        B, S, Hq, Hkv, D = 1, 300, 4, 2, 128
        q = synth.normal_bf16(31, 1, (B, S, Hq, D))
        k, v = synth.normal_bf16(31, 2, (B, S, Hkv, D)), synth.normal_bf16(31, 3, (B, S, Hkv, D))
        scale = 1.0 / np.sqrt(D)
        out = run_gpu_prefill(ctx, q, k, v, [130, 170], 320, scale, fused=True)[0]
        assert_close(out, oracle.full_causal(q, k, v, scale), "after a timeout")
        assert ctx.poll_device_status() == J.OK
        torch.cuda.synchronize()
    finally:
        ctx.close()


def test_two_timeouts_before_a_poll_report_once():
    import paper_2504_08242_b200 as J
    ctx = J.Context(0)
    try:
        ctx.wait_probe(200_000)
        ctx.wait_probe(200_000)  # sees the word already set and gives up at once
        assert ctx.poll_device_status() == J.ERR_TIMEOUT
        assert ctx.poll_device_status() == J.OK
    finally:
        ctx.close()


def test_wait_probe_arguments():
    import paper_2504_08242_b200 as J
    ctx = J.Context(0)
    try:
        for bad in (0, -5, 3_000_000_000):
            with pytest.raises(J.JupiterError) as e:
                ctx.wait_probe(bad)
            assert e.value.status == J.ERR_INVALID_ARG
        assert ctx.poll_device_status() == J.OK
    finally:
        ctx.close()
