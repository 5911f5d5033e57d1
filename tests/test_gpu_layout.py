"""GPU parity: muon_materialize / muon_scatter against the oracle, bit for bit, through the C ABI."""
import numpy as np
import pytest
import torch

from oracle import muon_oracle as orc
from paper_2609_21594_b200 import workloads as wl

pytestmark = pytest.mark.gpu

GUARD = 64  # canary elements before and after every device buffer


def _np_dtype(es):
    return np.uint16 if es == 2 else np.uint32


def _t_dtype(es):
    return torch.int16 if es == 2 else torch.int32


def _guarded(n, es, fill):
    buf = torch.full((n + 2 * GUARD,), fill, dtype=_t_dtype(es), device="cuda")
    return buf, buf[GUARD:GUARD + n]


def _run_case(mb, shapes, lay, es):
    ctx = mb.Context()
    L = mb.Layout(ctx, lay, es)
    segs = [(s.matrix, s.elem_begin, s.elem_count, s.flat_offset) for s in lay.segments]
    rng = np.random.default_rng(lay.flat_len + es)
    flat_np = rng.integers(0, 1 << (8 * es), size=lay.flat_len, dtype=np.uint64).astype(_np_dtype(es))
    flat_full, flat = _guarded(lay.flat_len, es, 0x1111)
    flat.copy_(torch.from_numpy(flat_np.view(np.int16 if es == 2 else np.int32)))
    canary = 0x5A5A
    fulls, mats = [], []
    for (m, n) in shapes:
        f, v = _guarded(max(m * n, 1), es, canary)
        fulls.append(f)
        mats.append(v[:m * n] if m * n else None)
    ctx.muon_materialize(flat, L, mats)
    torch.cuda.synchronize()
    expect = orc.materialize(flat_np, shapes, segs)
    for i, (m, n) in enumerate(shapes):
        got = fulls[i].cpu().numpy().view(_np_dtype(es))
        assert np.array_equal(got[GUARD:GUARD + m * n], expect[i].reshape(-1)), f"matrix {i}"
        assert (got[:GUARD] == canary).all() and (got[GUARD + max(m * n, 1) if m * n else GUARD + 1:] == canary).all()
    # scatter into a canary-filled flat buffer: payload arrives, padding and guards stay
    out_full, out = _guarded(lay.flat_len, es, 0x7B7B)
    ctx.muon_scatter(out, L, mats)
    torch.cuda.synchronize()
    canary_flat = np.full(lay.flat_len, 0x7B7B, dtype=_np_dtype(es))
    expect_flat = orc.scatter(canary_flat, shapes, segs, expect)
    got = out_full.cpu().numpy().view(_np_dtype(es))
    assert np.array_equal(got[GUARD:GUARD + lay.flat_len], expect_flat)
    assert (got[:GUARD] == 0x7B7B).all() and (got[GUARD + lay.flat_len:] == 0x7B7B).all()
    # round trip on the original buffer reproduces every payload element
    ctx.muon_scatter(flat, L, mats)
    torch.cuda.synchronize()
    assert np.array_equal(flat_full.cpu().numpy().view(_np_dtype(es))[GUARD:GUARD + lay.flat_len], flat_np)
    L.close()
    ctx.close()


@pytest.mark.parametrize("es", [2, 4])
@pytest.mark.parametrize("shards", [1, 3, 8])
@pytest.mark.parametrize("gen", ["per_param", "flat_concat"])
def test_odd_shapes_bit_exact(es, shards, gen):
    from paper_2609_21594_b200 import binding as mb

    shapes = wl.shapes_odd() + [(0, 9), (257, 130)]
    lay = (wl.layout_per_param if gen == "per_param" else wl.layout_flat_concat)(shapes, shards)
    _run_case(mb, shapes, lay, es)


def test_small_alignment_forces_elementwise_path():
    from paper_2609_21594_b200 import binding as mb

    shapes = [(37, 53), (129, 3), (64, 64)]
    lay = wl.layout_flat_concat(shapes, 5, align=1)
    _run_case(mb, shapes, lay, 2)
    lay = wl.layout_per_param(shapes, 5, align=3)
    _run_case(mb, shapes, lay, 4)


def test_multi_tile_set_bit_exact():
    from paper_2609_21594_b200 import binding as mb

    shapes = wl.shapes_tiny() + [(1408, 2048), (2048, 1408)]
    _run_case(mb, shapes, wl.layout_per_param(shapes, 8), 2)
    _run_case(mb, shapes, wl.layout_flat_concat(shapes, 8), 2)


def test_llama_layer_layout_round_trip_sampled():
    """One full-size Llama-3-8B layer (7 matrices, 218M elements) in 8 shards: properties that hold at any
    size plus sampled segments checked against the oracle's per-segment definition."""
    from paper_2609_21594_b200 import binding as mb

    shapes = wl.shapes_llama8b(layers=1)
    lay = wl.layout_per_param(shapes, 8)
    ctx = mb.Context()
    L = mb.Layout(ctx, lay, 2)
    g = torch.Generator(device="cuda")
    g.manual_seed(5)
    flat = torch.randint(-32768, 32767, (lay.flat_len,), dtype=torch.int16, device="cuda", generator=g)
    mats = [torch.full((m * n,), 0x0BAD, dtype=torch.int16, device="cuda") for (m, n) in shapes]
    ctx.muon_materialize(flat, L, mats)
    out = torch.zeros_like(flat)
    ctx.muon_scatter(out, L, mats)
    torch.cuda.synchronize()
    assert torch.equal(out, flat)          # no padding in this layout: the round trip is the identity
    rng = np.random.default_rng(0)
    for k in rng.choice(len(lay.segments), size=12, replace=False):
        s = lay.segments[k]
        a = mats[s.matrix][s.elem_begin:s.elem_begin + s.elem_count]
        b = flat[s.flat_offset:s.flat_offset + s.elem_count]
        assert torch.equal(a, b)
    L.close()
    ctx.close()


def test_argument_errors_launch_nothing():
    from paper_2609_21594_b200 import binding as mb

    ctx = mb.Context()
    shapes = [(8, 16)]
    lay = wl.layout_per_param(shapes, 2)
    L = mb.Layout(ctx, lay, 2)
    flat = torch.zeros(lay.flat_len, dtype=torch.int16, device="cuda")
    before = ctx.muon_launch_count()
    with pytest.raises(mb.MuonError) as e:
        ctx.muon_materialize(flat, L, [None])
    assert e.value.code == mb.ERR_INVALID_ARG
    with pytest.raises(mb.MuonError) as e:
        ctx.muon_materialize(flat[1:], L, [torch.zeros(128, dtype=torch.int16, device="cuda")])
    assert e.value.code == mb.ERR_INVALID_ARG
    assert ctx.muon_launch_count() == before
    bad = wl.Layout(lay.shapes, 2, lay.shard_len, lay.align, lay.segments[:-1])
    with pytest.raises(mb.MuonError) as e:
        mb.Layout(ctx, bad, 2)
    assert e.value.code == mb.ERR_BAD_LAYOUT
    L.close()
    ctx.close()
