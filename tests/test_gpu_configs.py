"""GPU parity at the benchmark configurations' full sizes, in the launch configuration bench.py times
(flat bf16 gradient shards -> muon_materialize -> muon_step_batched_out -> muon_scatter).

The oracle cannot run a whole set in reasonable time, so each test checks (i) sampled matrices -- one per
distinct shape plus the first and last matrix and chunk-boundary matrices -- element by element against the
bf16-emulating oracle (relative Frobenius error <= 1e-2 on O and dW, 1e-6 on M'), and (ii) properties
that hold at any size for every matrix: bit-exact gather/scatter, M' == G on the first step, finite
outputs, and ||O||_F inside the band the quintic's singular-value interval implies."""
import numpy as np
import pytest
import torch

from oracle import muon_oracle as orc
from paper_2609_21594_b200 import workloads as wl
from gpu_util import QUINTIC, host_f64, rel

pytestmark = pytest.mark.gpu

LR, MU, WD = 0.02, 0.95, 0.01
TOL_BF16 = 1e-2


def _run_config(config, shapes, row_scaled, sample_idx, layout_gen, shards=8):
    from paper_2609_21594_b200 import binding as mb

    dev = torch.device("cuda", 0)
    ctx = mb.Context()
    ctx.ensure_workspace(shapes)
    layout = layout_gen(shapes, shards)
    L = mb.Layout(ctx, layout, 2)
    W = [wl.device_draw(config, 0, i, "param", s, dev, std=0.02, dtype=torch.float32) for i, s in enumerate(shapes)]
    M = [torch.zeros(s, dtype=torch.float32, device=dev) for s in shapes]
    G_src = [wl.device_draw(config, 0, i, "grad", s, dev, std=1e-3, dtype=torch.bfloat16, row_scaled=row_scaled)
             for i, s in enumerate(shapes)]
    O = [torch.full(s, float("nan"), dtype=torch.bfloat16, device=dev) for s in shapes]
    sampled = {i: (host_f64(W[i]), host_f64(G_src[i])) for i in sample_idx}
    flat = torch.full((layout.flat_len,), 0x7B7B, dtype=torch.int16, device=dev).view(torch.bfloat16)
    ctx.muon_scatter(flat, L, G_src)
    G = [torch.zeros_like(g) for g in G_src]
    ctx.muon_materialize(flat, L, G)
    ctx.muon_step_batched_out(W, G, M, O, shapes, LR, MU, WD, wl.NS_STEPS, QUINTIC)
    flat_o = torch.full((layout.flat_len,), 0x7B7B, dtype=torch.int16, device=dev).view(torch.bfloat16)
    ctx.muon_scatter(flat_o, L, O)
    torch.cuda.synchronize()
    assert ctx.muon_last_device_status() == 0
    # ---- properties for every matrix
    pad_mask = torch.ones(layout.flat_len, dtype=torch.bool, device=dev)
    for sg in layout.segments:
        pad_mask[sg.flat_offset:sg.flat_offset + sg.elem_count] = False
        a = O[sg.matrix].view(-1)[sg.elem_begin:sg.elem_begin + sg.elem_count].view(torch.int16)
        b = flat_o[sg.flat_offset:sg.flat_offset + sg.elem_count].view(torch.int16)
        assert torch.equal(a, b)
    assert bool((flat_o.view(torch.int16)[pad_mask] == 0x7B7B).all())     # padding never written
    for i, s in enumerate(shapes):
        assert torch.equal(G[i].view(torch.int16), G_src[i].view(torch.int16)), i    # gather bit-exact
        assert torch.equal(M[i], G[i].float()), i                                     # M0 = 0  =>  M' = G
        of = O[i].float()
        assert bool(torch.isfinite(of).all()) and bool(torch.isfinite(W[i]).all()), i
        nrm = float(of.norm()) / np.sqrt(min(s))
        assert 0.25 < nrm < 1.21, (i, s, nrm)          # singular values end in [~0, 1.2024], most of them near 0.7-1.1
    # ---- sampled matrices against the oracle
    worst = 0.0
    for i in sample_idx:
        W0, Gv = sampled[i]
        Wn, Mn, Oref = orc.muon_step(W0, Gv, np.zeros(shapes[i]), LR, MU, WD, wl.NS_STEPS, QUINTIC, 1e-7, True, "bf16")
        eO = rel(host_f64(O[i]), Oref)
        eW = rel(host_f64(W[i]) - W0, Wn - W0)
        assert rel(host_f64(M[i]), Mn) <= 1e-6
        assert eO <= TOL_BF16 and eW <= TOL_BF16 + 1e-4, (i, shapes[i], eO, eW)
        worst = max(worst, eO)
    L.close()
    ctx.close()
    return worst


def test_1b_class_stack_16_layers():
    shapes = wl.shapes_1b()
    assert len(shapes) == 112
    sample = list(range(7)) + [len(shapes) - 1]           # one full layer (every distinct shape) + the last matrix
    _run_config("1b", shapes, False, sample, wl.layout_per_param)


def test_moe_784_matrices_flat_concat_layout():
    from paper_2609_21594_b200 import binding as mb

    shapes = wl.shapes_moe()
    assert len(shapes) == 784
    n, chunk_of = mb.muon_plan_describe(mb.muon_default_options(), shapes)
    # first and last matrix, one of each shape, and the two matrices on either side of a chunk boundary
    boundary = next(i for i in range(1, len(shapes)) if chunk_of[i] != chunk_of[i - 1]
                    and (min(shapes[i]), max(shapes[i])) == (min(shapes[i - 1]), max(shapes[i - 1])))
    same_group = [i for i in range(len(shapes)) if (min(shapes[i]), max(shapes[i])) == (1408, 2048)]
    edge = next(j for j in range(1, len(same_group)) if chunk_of[same_group[j]] != chunk_of[same_group[j - 1]])
    sample = sorted({0, 128, 192, len(shapes) - 1, same_group[edge - 1], same_group[edge], boundary})
    _run_config("moe", shapes, False, sample, wl.layout_flat_concat)


def test_llama3_8b_set_in_8_flat_shards():
    """The benchmark workload itself: 224 matrices, 6.98 G elements, per-parameter row-split layout."""
    shapes = wl.shapes_llama8b()
    assert len(shapes) == 224
    # Wq of layer 0, Wk of layer 0 (1024 x 4096), a gate matrix at a chunk boundary (14336 x 4096, tall),
    # the last matrix (down, 4096 x 14336)
    sample = [0, 2, 7 * 1 + 4, len(shapes) - 1]
    _run_config("llama8b", shapes, True, sample, wl.layout_per_param)


def test_llama3_8b_flat_concat_round_trip_bit_exact():
    """The layout generator whose shard cuts fall inside matrices (the flat concatenation cut at aligned points), at the
    benchmark's full size: scatter then gather must reproduce every matrix bit for bit, every segment must sit where the
    table says, and the padding of the flat buffer must never be written."""
    from paper_2609_21594_b200 import binding as mb

    dev = torch.device("cuda", 0)
    shapes = wl.shapes_llama8b()
    # 32 equal layers over 8 shards would put every cut on a layer boundary; 7 shards cut inside matrices, mid-row
    layout = wl.layout_flat_concat(shapes, 7)
    inside = [sg for sg in layout.segments if sg.elem_begin != 0]
    assert len(inside) >= 6 and any(sg.elem_begin % shapes[sg.matrix][1] for sg in inside)
    ctx = mb.Context()
    L = mb.Layout(ctx, layout, 2)
    src = [wl.device_draw("llama8b_fc", 0, i, "grad", s, dev, std=1e-3, dtype=torch.bfloat16) for i, s in enumerate(shapes)]
    flat = torch.full((layout.flat_len,), 0x7B7B, dtype=torch.int16, device=dev).view(torch.bfloat16)
    ctx.muon_scatter(flat, L, src)
    back = [torch.full(s, float("nan"), dtype=torch.bfloat16, device=dev) for s in shapes]
    ctx.muon_materialize(flat, L, back)
    torch.cuda.synchronize()
    pad_mask = torch.ones(layout.flat_len, dtype=torch.bool, device=dev)
    for sg in layout.segments:
        pad_mask[sg.flat_offset:sg.flat_offset + sg.elem_count] = False
        a = src[sg.matrix].view(-1)[sg.elem_begin:sg.elem_begin + sg.elem_count].view(torch.int16)
        assert torch.equal(a, flat[sg.flat_offset:sg.flat_offset + sg.elem_count].view(torch.int16)), sg
    assert bool((flat.view(torch.int16)[pad_mask] == 0x7B7B).all())
    for i in range(len(shapes)):
        assert torch.equal(back[i].view(torch.int16), src[i].view(torch.int16)), i
    L.close()
    ctx.close()


def test_host_buffer_pipeline_with_ramp_sets_matches_the_device_resident_step():
    """muon_step_flat_host on a set large enough for its plan to ramp (8 layers of the 1B-class stack, 360 M elements:
    small sets first and last, full-size sets in between).  Different batching,
    same results: parameters, momenta, updates and the host-side flat update buffer are bit-identical to scatter-free
    device-resident muon_step_batched_out on the same gradients."""
    from paper_2609_21594_b200 import binding as mb

    dev = torch.device("cuda", 0)
    shapes = wl.shapes_1b(8)
    opt = mb.muon_default_options()
    set_of, order = mb.muon_plan_pipeline(opt, shapes)
    assert len(order) >= mb.muon_plan_launch_sets(opt, shapes)[0] + 2         # the ramps are really there
    ctx = mb.Context()
    ctx.ensure_workspace(shapes)
    layout = wl.layout_per_param(shapes, 8)
    L = mb.Layout(ctx, layout, 2)
    W0 = [wl.device_draw("pipe", 0, i, "param", s, dev, std=0.02, dtype=torch.float32) for i, s in enumerate(shapes)]
    G = [wl.device_draw("pipe", 0, i, "grad", s, dev, std=1e-3, dtype=torch.bfloat16) for i, s in enumerate(shapes)]
    M0 = [wl.device_draw("pipe", 1, i, "grad", s, dev, std=1e-3, dtype=torch.float32) for i, s in enumerate(shapes)]
    flat = torch.zeros(layout.flat_len, dtype=torch.bfloat16, device=dev)
    ctx.muon_scatter(flat, L, G)
    host_in = torch.empty(layout.flat_len, dtype=torch.bfloat16).pin_memory()
    host_in.copy_(flat)
    host_out = torch.zeros(layout.flat_len, dtype=torch.bfloat16).pin_memory()
    # device-resident reference
    Wa, Ma = [w.clone() for w in W0], [m.clone() for m in M0]
    Oa = [torch.empty(s, dtype=torch.bfloat16, device=dev) for s in shapes]
    ctx.muon_step_batched_out(Wa, G, Ma, Oa, shapes, LR, MU, WD, wl.NS_STEPS, QUINTIC)
    # host-buffer pipeline (gradients arrive by copy engine into Gb)
    Wb, Mb = [w.clone() for w in W0], [m.clone() for m in M0]
    Gb = [torch.zeros(s, dtype=torch.bfloat16, device=dev) for s in shapes]
    Ob = [torch.zeros(s, dtype=torch.bfloat16, device=dev) for s in shapes]
    ctx.muon_step_flat_host(host_in, host_out, L, Wb, Gb, Mb, Ob, LR, MU, WD, wl.NS_STEPS, QUINTIC)
    torch.cuda.synchronize()
    assert ctx.muon_last_device_status() == 0
    for i in range(len(shapes)):
        assert torch.equal(Gb[i].view(torch.int16), G[i].view(torch.int16)), i
        assert torch.equal(Wb[i], Wa[i]) and torch.equal(Mb[i], Ma[i]), i
        assert torch.equal(Ob[i].view(torch.int16), Oa[i].view(torch.int16)), i
    flat_o = torch.zeros(layout.flat_len, dtype=torch.bfloat16, device=dev)
    ctx.muon_scatter(flat_o, L, Oa)
    assert torch.equal(host_out.view(torch.int16), flat_o.cpu().view(torch.int16))
    L.close()
    ctx.close()
