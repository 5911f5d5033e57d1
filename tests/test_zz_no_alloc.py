"""GPU test of muon_orthogonalize_static, the entry point for callers that cannot allocate device
memory (allocator callbacks, processes whose device memory another runtime has fully handed out,
sections that must not hit an allocation's implicit synchronisation).  It takes no context and keeps
all its scratch in a fixed array inside the library, so the test checks it against the ordinary
entry point, muon_orthogonalize_batched, on two calls in a row: the second call runs on whatever the
first one left in the shared scratch and must still be right.  Because both entry points run the same
kernels, agreeing with each other is not enough: every result is also held against the CPU oracle, and
the device's free memory is read before and after the calls to see that nothing was allocated.

This file sorts last on purpose: if it fails under `pytest -x`, every other test has already run.
"""
import numpy as np
import pytest
import torch

from oracle import muon_oracle as orc
from paper_2609_21594_b200 import workloads as wl
from gpu_util import QUINTIC, bf16_input, dev_f32, host_f64, rel

pytestmark = pytest.mark.gpu


def _reference(mb, precision, x_dev, shape):
    """The existing entry point on the same device tensor."""
    ctx = mb.Context(mb.muon_default_options(ns_precision=precision))
    ctx.ensure_workspace([shape])
    out = torch.full_like(x_dev, float("nan"))
    ctx.muon_orthogonalize_batched([x_dev], [out], [shape], 5, QUINTIC)
    torch.cuda.synchronize()
    assert ctx.muon_last_device_status() == 0
    ctx.close()
    return out


@pytest.mark.parametrize("precision", ["bf16", "fp32"])
def test_static_scratch_matches_regular_entry_point_twice_in_a_row(precision):
    from paper_2609_21594_b200 import binding as mb

    prec = mb.NS_BF16 if precision == "bf16" else mb.NS_FP32
    # first a tall multi-tile matrix, then a smaller ragged one that leaves most of the old scratch in place
    for call, shape in enumerate([(1024, 256), (200, 264)]):
        g = wl.grad_np("noalloc", call, 0, shape)
        x, vals = bf16_input(g) if precision == "bf16" else (dev_f32(g), g.astype(np.float64))
        expect = _reference(mb, prec, x, shape)
        out = torch.full_like(x, float("nan"))
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        mb.muon_orthogonalize_static(x, out, shape[0], shape[1], prec, 5, QUINTIC, 1e-7, 0, status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        got, ref = host_f64(out), host_f64(expect)
        assert np.isfinite(got).all()
        # same kernels on the same data: the engine is deterministic, so the results are identical;
        # the tolerance of the other parity tests (1e-2 bf16 / 1e-4 fp32) is the stated bar
        tol = 1e-2 if precision == "bf16" else 1e-4
        assert np.linalg.norm(got - ref) <= tol * np.linalg.norm(ref)
        assert np.array_equal(got, ref)
        # ... and right, not merely equal: the oracle in the matching arithmetic, at the benchmark spec's tolerances
        want = orc.newton_schulz(vals, 5, QUINTIC, 1e-7, "bf16" if precision == "bf16" else "fp64")
        assert rel(got, want) <= tol, (shape, rel(got, want))


def test_static_scratch_allocates_no_device_memory():
    """After the first call on the device (which resolves the array's address), further calls must leave the
    amount of free device memory exactly as they found it: nothing is allocated, nothing is freed."""
    from paper_2609_21594_b200 import binding as mb

    shape = (384, 640)
    x, _ = bf16_input(wl.grad_np("noalloc", 7, 0, shape))
    outs = [torch.empty_like(x) for _ in range(3)]
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    mb.muon_orthogonalize_static(x, outs[0], shape[0], shape[1], mb.NS_BF16, 5, QUINTIC, 1e-7, 0, status)   # set-up call
    torch.cuda.synchronize()
    free_before, total = torch.cuda.mem_get_info()
    for out in outs[1:]:
        mb.muon_orthogonalize_static(x, out, shape[0], shape[1], mb.NS_BF16, 5, QUINTIC, 1e-7, 0, status)
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info()
    assert free_after == free_before, (free_before, free_after)
    assert int(status.item()) == 0
    assert torch.equal(outs[0], outs[1]) and torch.equal(outs[1], outs[2])


def test_static_scratch_rejects_what_does_not_fit_and_bad_arguments():
    from paper_2609_21594_b200 import binding as mb

    x = torch.zeros(8, 8, dtype=torch.bfloat16, device="cuda")
    y = torch.zeros(8, 8, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(mb.MuonError) as e:      # 2048 x 2048 bf16 needs 32 MiB of workspace: beyond the fixed array
        mb.muon_orthogonalize_static(x, y, 2048, 2048, mb.NS_BF16, 5, QUINTIC)
    assert e.value.code == mb.ERR_TOO_LARGE
    with pytest.raises(mb.MuonError) as e:
        mb.muon_orthogonalize_static(x, x, 8, 8, mb.NS_BF16, 5, QUINTIC)       # in == out
    assert e.value.code == mb.ERR_INVALID_ARG
    with pytest.raises(mb.MuonError) as e:
        mb.muon_orthogonalize_static(x, y, 8, 8, mb.NS_BF16, 0, QUINTIC)       # no iterations
    assert e.value.code == mb.ERR_INVALID_ARG
    mb.muon_orthogonalize_static(x, y, 0, 8, mb.NS_BF16, 5, QUINTIC)           # empty matrix: a no-op
    torch.cuda.synchronize()
