"""GPU parity of muon_step_flat, the sharded-state flow: parameters, momenta and gradients stay in flat
shard buffers; the gather is fused into the momentum/cast kernel and the scatter into the update kernel.
It must reproduce, bit for bit, muon_materialize + muon_step_batched_out + muon_scatter on the same
data, never touch padding, and (through that path) match the oracle."""
import numpy as np
import pytest
import torch

from oracle import muon_oracle as orc
from paper_2609_21594_b200 import workloads as wl
from gpu_util import QUINTIC, host_f64, rel

pytestmark = pytest.mark.gpu

LR, MU, WD = 0.02, 0.95, 0.01
PAD_F32 = -777.0
PAD_BF16 = 0x7B7B


def _flat_from(mats_np, lay, segs, dtype, fill):
    flat = np.full(lay.flat_len, fill, dtype=dtype)
    return orc.scatter(flat, list(lay.shapes), segs, mats_np)


def _case(mb, shapes, lay, name, two_steps=True):
    segs = [(s.matrix, s.elem_begin, s.elem_count, s.flat_offset) for s in lay.segments]
    ctx = mb.Context()
    ctx.ensure_workspace(shapes)
    L4, L2 = mb.Layout(ctx, lay, 4), mb.Layout(ctx, lay, 2)
    Wn = [wl.param_np(name, i, s) for i, s in enumerate(shapes)]
    Mn = [wl.grad_np(name, 9, i, s) for i, s in enumerate(shapes)]
    flatW = torch.from_numpy(_flat_from(Wn, lay, segs, np.float32, PAD_F32)).cuda()
    flatM = torch.from_numpy(_flat_from(Mn, lay, segs, np.float32, PAD_F32)).cuda()
    flatO = torch.full((lay.flat_len,), PAD_BF16, dtype=torch.int16, device="cuda").view(torch.bfloat16)
    # reference state as whole matrices
    W = [torch.from_numpy(w).cuda() for w in Wn]
    M = [torch.from_numpy(m).cuda() for m in Mn]
    O = [torch.zeros(s, dtype=torch.bfloat16, device="cuda") for s in shapes]
    for step in range(2 if two_steps else 1):
        g_bits = [wl.to_bf16_bits(wl.grad_np(name, step, i, s)) for i, s in enumerate(shapes)]
        flatG = torch.from_numpy(_flat_from(g_bits, lay, segs, np.uint16, PAD_BF16).view(np.int16)).cuda().view(torch.bfloat16)
        ctx.muon_step_flat(L2, flatW, flatG, flatM, flatO, LR, MU, WD, 5, QUINTIC)
        G = [torch.zeros(s, dtype=torch.bfloat16, device="cuda") for s in shapes]
        ctx.muon_materialize(flatG, L2, G)
        ctx.muon_step_batched_out(W, G, M, O, shapes, LR, MU, WD, 5, QUINTIC)
        torch.cuda.synchronize()
        assert ctx.muon_last_device_status() == 0
        refW = torch.full((lay.flat_len,), PAD_F32, dtype=torch.float32, device="cuda")
        refM = torch.full((lay.flat_len,), PAD_F32, dtype=torch.float32, device="cuda")
        refO = torch.full((lay.flat_len,), PAD_BF16, dtype=torch.int16, device="cuda").view(torch.bfloat16)
        ctx.muon_scatter(refW, L4, W)
        ctx.muon_scatter(refM, L4, M)
        ctx.muon_scatter(refO, L2, O)
        torch.cuda.synchronize()
        assert torch.equal(flatW, refW), (name, step)            # payload identical, padding still the fill value
        assert torch.equal(flatM, refM), (name, step)
        assert torch.equal(flatO.view(torch.int16), refO.view(torch.int16)), (name, step)
    L4.close()
    L2.close()
    ctx.close()
    return W, Wn


@pytest.mark.parametrize("shards", [1, 3, 8])
def test_flat_state_matches_the_materialised_path(shards):
    from paper_2609_21594_b200 import binding as mb

    shapes = wl.shapes_tiny() + wl.shapes_odd() + [(0, 5), (200, 264)]
    _case(mb, shapes, wl.layout_per_param(shapes, shards), f"flat{shards}")


def test_flat_state_one_llama_layer():
    from paper_2609_21594_b200 import binding as mb

    shapes = wl.shapes_llama8b(layers=1)
    _case(mb, shapes, wl.layout_per_param(shapes, 8), "flatllama", two_steps=False)


@pytest.mark.parametrize("align", [1, 2, 4])
def test_flat_state_with_segment_offsets_that_are_not_vector_aligned(align):
    """A row-aligned layout may start a segment on any multiple of align_elems.  With align 1, 2 or 4 a small odd
    matrix ahead of a 64 x 64 one leaves the latter's rows at offsets that are no multiple of 8 (or 4) elements:
    the step kernels must then give up their 16-byte accesses on the flat buffers, not fault or mis-read."""
    from paper_2609_21594_b200 import binding as mb

    shapes = [(3, 5), (64, 64), (7, 9), (128, 256), (256, 128)]
    lay = wl.layout_per_param(shapes, 2, align=align)
    offs = {s.flat_offset % 8 for s in lay.segments if shapes[s.matrix][1] % 8 == 0}
    assert any(o != 0 for o in offs)                     # the interesting case really occurs
    W, Wn = _case(mb, shapes, lay, f"flatalign{align}")
    # ... and the shared result is right: two oracle steps on the 64 x 64 matrix
    Wo, Mo = Wn[1].astype(np.float64), wl.grad_np(f"flatalign{align}", 9, 1, shapes[1]).astype(np.float64)
    for step in range(2):
        g = wl.bf16_bits_to_f32(wl.to_bf16_bits(wl.grad_np(f"flatalign{align}", step, 1, shapes[1]))).astype(np.float64)
        Wprev = Wo
        Wo, Mo, _ = orc.muon_step(Wo, g, Mo, LR, MU, WD, 5, QUINTIC, 1e-7, True, "bf16")
    # teacher forcing is not needed at this size: two steps stay well inside the tolerance on dW of the last step
    assert rel(host_f64(W[1]) - Wprev, Wo - Wprev) <= 3e-2


def test_flat_state_needs_whole_row_segments():
    from paper_2609_21594_b200 import binding as mb

    shapes = [(37, 53), (130, 7), (64, 64)]
    lay = wl.layout_flat_concat(shapes, 4)                      # cut points fall inside rows
    assert any(s.elem_begin % shapes[s.matrix][1] for s in lay.segments)
    ctx = mb.Context()
    ctx.ensure_workspace(shapes)
    L = mb.Layout(ctx, lay, 2)
    fw = torch.zeros(lay.flat_len, device="cuda")
    fg = torch.zeros(lay.flat_len, device="cuda", dtype=torch.bfloat16)
    before = ctx.muon_launch_count()
    with pytest.raises(mb.MuonError) as e:
        ctx.muon_step_flat(L, fw, fg, fw.clone(), None, LR, MU, WD, 5, QUINTIC)
    assert e.value.code == mb.ERR_UNSUPPORTED and ctx.muon_launch_count() == before
    L.close()
    ctx.close()


def test_head_interleaved_fused_qkv_as_a_layout():
    """A permuting transform of the model adapter (Section 6.6), expressed as a layout: a grouped-query fused QKV projection
    stored group by group -- [q heads of group 0 | k0 | v0 | q heads of group 1 | k1 | v1 | ...] along the rows of one
    physical [G * 6 * 64, d] tensor.  The logical matrices Wq (all q heads), Wk and Wv are made of row runs that alternate
    through the physical tensor, so no single strided view describes them; a segment table does.  The physical tensor IS
    the flat buffer: parameters, momenta and gradients are updated in place, bit-identical to the ordinary step on
    contiguous copies of the three logical matrices."""
    from paper_2609_21594_b200 import binding as mb

    groups, hd, d = 4, 64, 256
    q_rows, kv_rows = 4 * hd, hd                       # per group: four query heads, one key head, one value head
    per_group = q_rows + 2 * kv_rows
    shapes = [(groups * q_rows, d), (groups * kv_rows, d), (groups * kv_rows, d)]
    segs = []
    for g in range(groups):
        base = g * per_group * d
        segs.append(wl.Segment(0, g * q_rows * d, q_rows * d, base))
        segs.append(wl.Segment(1, g * kv_rows * d, kv_rows * d, base + q_rows * d))
        segs.append(wl.Segment(2, g * kv_rows * d, kv_rows * d, base + (q_rows + kv_rows) * d))
    lay = wl.Layout(tuple(shapes), 1, groups * per_group * d, 8, tuple(segs))
    assert mb.muon_layout_validate(mb.make_layout_desc(lay, 2)) == mb.OK
    W, Wn = _case(mb, shapes, lay, "gqa_qkv")
    # and against the oracle (two steps were taken; check that the parameters moved and stayed finite)
    for w, w0 in zip(W, Wn):
        assert bool(torch.isfinite(w).all()) and not np.array_equal(w.cpu().numpy(), w0)
