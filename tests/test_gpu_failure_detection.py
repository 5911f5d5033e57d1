"""Failure detection without a GPU fault: every device-side wait of the tensor-core pipelines is bounded and
reports through a status word.  The self-test makes one such wait run out (a barrier nothing arrives at,
limit of about a millisecond) and the host must see the code, clear it, and find the context fully usable."""
import time

import numpy as np
import pytest
import torch

from oracle import muon_oracle as orc
from paper_2609_21594_b200 import workloads as wl
from gpu_util import QUINTIC, bf16_input, host_f64, rel

pytestmark = pytest.mark.gpu


def test_expired_wait_is_reported_and_the_context_survives():
    from paper_2609_21594_b200 import binding as mb

    ctx = mb.Context()
    assert ctx.muon_last_device_status() == 0
    t0 = time.perf_counter()
    ctx.muon_self_test_bounded_wait()
    assert ctx.muon_last_device_status() == 100           # the wait gave up and said so
    assert time.perf_counter() - t0 < 5.0                  # ... within its limit, not after a hang
    assert ctx.muon_synchronize_and_check() == mb.ERR_DEVICE_TIMEOUT   # the opt-in synchronous check turns it into a status
    ctx.muon_clear_device_status()
    assert ctx.muon_last_device_status() == 0
    assert ctx.muon_synchronize_and_check() == mb.OK
    # the device and the context are fine: a normal orthogonalisation still matches the oracle
    shape = (256, 384)
    x, v = bf16_input(wl.grad_np("after_timeout", 0, 0, shape))
    out = torch.empty_like(x)
    ctx.ensure_workspace([shape])
    ctx.muon_orthogonalize_batched([x], [out], [shape], 5, QUINTIC)
    torch.cuda.synchronize()
    assert ctx.muon_last_device_status() == 0
    assert rel(host_f64(out), orc.newton_schulz(v, 5, QUINTIC, 1e-7, "bf16")) <= 1e-2
    ctx.close()
