"""GPU parity of muon_step_batched_views: logical matrices updated in place inside larger physical
parameters (fused QKV rows, side-by-side column factors, [E, M, N] expert planes, ragged sub-blocks).
The strided result must equal, bit for bit, the ordinary step on contiguous copies of the same
blocks, leave everything outside the views untouched, and match the oracle within the bf16 tolerance."""
import numpy as np
import pytest
import torch

from oracle import muon_oracle as orc
from paper_2609_21594_b200 import workloads as wl
from gpu_util import QUINTIC, host_f64, rel

pytestmark = pytest.mark.gpu

LR, MU, WD = 0.02, 0.95, 0.01


def _physical(name, shape):
    w = torch.from_numpy(wl.param_np(name, 0, shape)).cuda()
    g = torch.from_numpy(wl.grad_np(name, 0, 0, shape)).cuda().to(torch.bfloat16)
    m = torch.from_numpy(wl.grad_np(name, 1, 0, shape)).cuda()          # a non-trivial momentum state
    return w, g, m


def _check(mb, physical_shape, views_fn, name):
    ctx = mb.Context()
    W, G, M = _physical(name, physical_shape)
    U = torch.full(physical_shape, -3.0, dtype=torch.bfloat16, device="cuda")
    W0, M0 = W.clone(), M.clone()
    views = views_fn(W)
    vshapes = [v for _, v in views]
    shapes = [(r, c) for (r, c, _) in vshapes]
    ctx.ensure_workspace(shapes)

    def block(t, off, v):
        r, c, ld = v
        flat = t.reshape(-1)
        return torch.as_strided(flat, (r, c), (ld, 1), off)

    # reference: the ordinary step on contiguous copies
    Wc = [block(W0, off, v).clone().contiguous() for off, v in views]
    Gc = [block(G, off, v).clone().contiguous() for off, v in views]
    Mc = [block(M0, off, v).clone().contiguous() for off, v in views]
    Mc0 = [host_f64(m) for m in Mc]
    Oc = [torch.empty(s, dtype=torch.bfloat16, device="cuda") for s in shapes]
    Wc0 = [host_f64(w) for w in Wc]
    ctx.muon_step_batched_out(Wc, Gc, Mc, Oc, shapes, LR, MU, WD, 5, QUINTIC)
    # strided, in place
    ctx.muon_step_batched_views(mb.view_addresses(W, views), mb.view_addresses(G, views), mb.view_addresses(M, views),
                                mb.view_addresses(U, views), vshapes, LR, MU, WD, 5, QUINTIC)
    torch.cuda.synchronize()
    assert ctx.muon_last_device_status() == 0
    covered = torch.zeros(physical_shape, dtype=torch.bool, device="cuda")
    for i, (off, v) in enumerate(views):
        assert torch.equal(block(W, off, v), Wc[i]), (name, i)
        assert torch.equal(block(M, off, v), Mc[i]), (name, i)
        assert torch.equal(block(U, off, v).view(torch.int16), Oc[i].view(torch.int16)), (name, i)
        block(covered, off, v).fill_(True)
        ref = orc.muon_step(Wc0[i], host_f64(Gc[i]), Mc0[i], LR, MU, WD, 5, QUINTIC, 1e-7, True, "bf16")
        assert rel(host_f64(Oc[i]), ref[2]) <= 1e-2, (name, i)
        assert rel(host_f64(Mc[i]), ref[1]) <= 1e-6
    # nothing outside the views moved
    assert torch.equal(W[~covered], W0[~covered]) and torch.equal(M[~covered], M0[~covered])
    assert bool((U[~covered] == -3.0).all())
    ctx.close()


def test_fused_qkv_row_blocks():
    from paper_2609_21594_b200 import binding as mb

    # 6 query heads, 2 key and 2 value heads of dim 64 on d = 256: one [640, 256] projection
    _check(mb, (640, 256), lambda t: mb.views_of_rows(t, [384, 128, 128]), "qkv")


def test_side_by_side_column_factors():
    from paper_2609_21594_b200 import binding as mb

    _check(mb, (256, 320), lambda t: mb.views_of_cols(t, [192, 128]), "mla")


def test_expert_planes_are_independent_matrices():
    from paper_2609_21594_b200 import binding as mb

    _check(mb, (3, 128, 192), lambda t: mb.views_of_planes(t), "experts")
    _check(mb, (2, 320, 128), lambda t: mb.views_of_planes(t), "experts_tall")       # tall planes: transposed path


def test_ragged_sub_block_leaves_its_surroundings_alone():
    from paper_2609_21594_b200 import binding as mb

    # a 97 x 53 block at rows 3.., columns 8.. of a [100, 72] tensor: odd sizes force the element-wise path
    _check(mb, (100, 72), lambda t: [(3 * t.stride(0) + 8, (97, 53, t.stride(0)))], "ragged")


def test_row_interleaved_gate_up():
    """Gate and up projections stored as alternating rows of one [2m, n] tensor: two views with row stride 2n, the second
    offset by n elements.  Also three-way interleaving with an odd row count per view."""
    from paper_2609_21594_b200 import binding as mb

    _check(mb, (512, 384), lambda t: mb.views_of_interleaved_rows(t, 2), "gate_up")          # wide logical matrices
    _check(mb, (1536, 256), lambda t: mb.views_of_interleaved_rows(t, 2), "gate_up_tall")    # tall: transposed path
    _check(mb, (3 * 131, 200), lambda t: mb.views_of_interleaved_rows(t, 3), "three_way")


def test_overlapping_views_are_rejected_before_any_launch():
    from paper_2609_21594_b200 import binding as mb

    ctx = mb.Context()
    W, G, M = _physical("overlap", (128, 256))
    W0, M0 = W.clone(), M.clone()
    ctx.ensure_workspace([(64, 256), (65, 256)])
    es = W.element_size()
    n0 = ctx.muon_launch_count()
    # rows 0..63 and rows 63..127: one shared row
    views = [(64, 256, 256), (65, 256, 256)]
    with pytest.raises(mb.MuonError) as e:
        ctx.muon_step_batched_views([W.data_ptr(), W.data_ptr() + 63 * 256 * es], [G.data_ptr(), G.data_ptr() + 63 * 256 * 2],
                                    [M.data_ptr(), M.data_ptr() + 64 * 256 * es], None, views, LR, MU, WD, 5, QUINTIC)
    assert e.value.code == mb.ERR_INVALID_ARG
    # the same momentum twice
    with pytest.raises(mb.MuonError) as e:
        ctx.muon_step_batched_views([W.data_ptr(), W.data_ptr() + 64 * 256 * es], [G.data_ptr(), G.data_ptr() + 64 * 256 * 2],
                                    [M.data_ptr(), M.data_ptr()], None, [(64, 256, 256)] * 2, LR, MU, WD, 5, QUINTIC)
    assert e.value.code == mb.ERR_INVALID_ARG
    torch.cuda.synchronize()
    assert ctx.muon_launch_count() == n0 and torch.equal(W, W0) and torch.equal(M, M0)
    ctx.close()


def test_views_reject_bad_strides():
    from paper_2609_21594_b200 import binding as mb

    ctx = mb.Context()
    W, G, M = _physical("bad", (64, 64))
    ctx.ensure_workspace([(64, 64)])
    with pytest.raises(mb.MuonError) as e:
        ctx.muon_step_batched_views([W.data_ptr()], [G.data_ptr()], [M.data_ptr()], None, [(64, 64, 32)], LR, MU, WD, 5, QUINTIC)
    assert e.value.code == mb.ERR_INVALID_ARG
    ctx.close()
