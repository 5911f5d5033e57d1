"""Host-side checks of the C ABI that need no GPU: the library loads, exports every symbol the
header declares, validates layouts, plans batches and sizes workspaces; compute entry points are
not called."""
import ctypes as C
import os
import re

import numpy as np
import pytest
import torch

from oracle import muon_oracle as orc
from paper_2609_21594_b200 import binding as mb
from paper_2609_21594_b200 import workloads as wl

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def header_functions():
    text = open(os.path.join(ROOT, "include", "muon_b200.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(muon_[a-z_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    names = header_functions()
    assert len(names) >= 18
    for n in names:
        assert hasattr(mb.lib, n), n
    assert sorted(mb.EXPORTED) == names


def test_struct_sizes_match_the_header():
    assert C.sizeof(mb.Shape) == 8
    assert C.sizeof(mb.View) == 16
    assert C.sizeof(mb.Segment) == 32
    assert C.sizeof(mb.LayoutDesc) == 48
    assert C.sizeof(mb.Options) == 40


def test_status_strings():
    assert mb.lib.muon_status_string(0) == b"ok"
    for code in range(-6, 0):
        assert mb.lib.muon_status_string(code) not in (b"ok", b"unknown status")
    assert mb.lib.muon_status_string(-99) == b"unknown status"


@pytest.mark.skipif(torch.cuda.is_available(), reason="checks the no-device error path")
def test_create_fails_loudly_without_a_device():
    with pytest.raises(mb.MuonError) as e:
        mb.Context()
    assert e.value.code == mb.ERR_CUDA


def test_default_options():
    o = mb.muon_default_options()
    assert (o.grad_dtype, o.ns_precision, o.nesterov, o.coeffs_per_step, o.engine) == (0, 0, 1, 0, 0)
    assert o.eps == pytest.approx(1e-7) and o.chunk_elems == 1 << 29
    assert (o.coeffs_per_matrix, o.launch_per_product) == (0, 0)


@pytest.mark.parametrize("gen", [wl.layout_per_param, wl.layout_flat_concat])
@pytest.mark.parametrize("shards", [1, 2, 8])
@pytest.mark.parametrize("setname", ["odd", "tiny"])
def test_layout_validate_accepts_generated_layouts(gen, shards, setname):
    shapes = wl.shapes_odd() if setname == "odd" else wl.shapes_tiny()
    lay = gen(shapes, shards)
    assert mb.muon_layout_validate(mb.make_layout_desc(lay, 2)) == mb.OK
    segs = [(s.matrix, s.elem_begin, s.elem_count, s.flat_offset) for s in lay.segments]
    assert orc.layout_is_valid(lay.flat_len, shapes, segs, lay.align, lay.num_shards, lay.shard_len)


def _mutated(lay, fn):
    segs = [wl.Segment(s.matrix, s.elem_begin, s.elem_count, s.flat_offset) for s in lay.segments]
    segs = fn(segs)
    return wl.Layout(lay.shapes, lay.num_shards, lay.shard_len, lay.align, tuple(segs))


def test_layout_validate_rejects_malformed_layouts_like_the_bruteforce_checker():
    base = wl.layout_per_param(wl.shapes_odd(), 4)
    S = wl.Segment
    cases = {
        "gap": lambda s: s[:-1],
        "overlap_matrix": lambda s: s + [s[0]],
        "misaligned": lambda s: [S(s[0].matrix, s[0].elem_begin, s[0].elem_count, s[0].flat_offset + 1)] + s[1:],
        "out_of_matrix": lambda s: s[:-1] + [S(s[-1].matrix, s[-1].elem_begin, s[-1].elem_count + 1, s[-1].flat_offset)],
        "bad_matrix": lambda s: s[:-1] + [S(99, s[-1].elem_begin, s[-1].elem_count, s[-1].flat_offset)],
        "flat_overlap": lambda s: [S(s[0].matrix, s[0].elem_begin, s[0].elem_count, s[1].flat_offset)] + s[1:],
        "beyond_flat": lambda s: s[:-1] + [S(s[-1].matrix, s[-1].elem_begin, s[-1].elem_count, base.flat_len)],
        "negative": lambda s: [S(s[0].matrix, -1, s[0].elem_count, s[0].flat_offset)] + s[1:],
    }
    for name, fn in cases.items():
        bad = _mutated(base, fn)
        assert mb.muon_layout_validate(mb.make_layout_desc(bad, 2)) == mb.ERR_BAD_LAYOUT, name
        segs = [(s.matrix, s.elem_begin, s.elem_count, s.flat_offset) for s in bad.segments]
        assert not orc.layout_is_valid(bad.flat_len, list(bad.shapes), segs, bad.align, bad.num_shards, bad.shard_len), name
    # a segment that straddles two shards
    lay = wl.layout_per_param([(4, 64)], 2, align=8)
    strad = wl.Layout(lay.shapes, 2, lay.shard_len, 8, (wl.Segment(0, 0, 256, 0),))
    if strad.shard_len < 256:
        assert mb.muon_layout_validate(mb.make_layout_desc(strad, 2)) == mb.ERR_BAD_LAYOUT
    # the same hand-built table the oracle's own pin uses: 1 x 12 matrix, two shards of 8, one piece at offset 4
    one_piece = wl.Layout(((1, 12),), 2, 8, 4, (wl.Segment(0, 0, 12, 4),))
    cut = wl.Layout(((1, 12),), 2, 8, 4, (wl.Segment(0, 0, 4, 4), wl.Segment(0, 4, 8, 8)))
    assert mb.muon_layout_validate(mb.make_layout_desc(one_piece, 2)) == mb.ERR_BAD_LAYOUT
    assert mb.muon_layout_validate(mb.make_layout_desc(cut, 2)) == mb.OK
    assert mb.muon_layout_validate(mb.make_layout_desc(wl.Layout(((1, 12),), 1, 16, 4, (wl.Segment(0, 0, 12, 4),)), 2)) == mb.OK
    d = mb.make_layout_desc(base, 3)
    assert mb.muon_layout_validate(d) == mb.ERR_INVALID_ARG      # element size must be 2 or 4
    d = mb.make_layout_desc(base, 2)
    d.segments[0].reserved = 7
    assert mb.muon_layout_validate(d) == mb.ERR_BAD_LAYOUT


def test_full_size_llama_layout_validates_quickly():
    lay = wl.layout_per_param(wl.shapes_llama8b(), 8)
    assert mb.muon_layout_validate(mb.make_layout_desc(lay, 2)) == mb.OK
    lay = wl.layout_flat_concat(wl.shapes_moe(), 8)
    assert mb.muon_layout_validate(mb.make_layout_desc(lay, 2)) == mb.OK
    # the flat-concat cuts really fall inside matrices for the MoE set
    assert any(s.elem_begin != 0 for s in lay.segments)


def test_plan_groups_by_core_shape_and_caps_chunks():
    opt = mb.muon_default_options()
    shapes = wl.shapes_moe()
    n, chunk_of = mb.muon_plan_describe(opt, shapes)
    # 1408x2048 and 2048x1408 share the core shape (1408, 2048): 768 matrices, 186 per 2^29-element chunk
    per = (1 << 29) // (1408 * 2048)
    assert per == 186
    assert n == -(-768 // per) + 1
    by_chunk = {}
    for i, c in enumerate(chunk_of):
        by_chunk.setdefault(c, []).append(i)
    for c, idx in by_chunk.items():
        cores = {(min(shapes[i]), max(shapes[i])) for i in idx}
        assert len(cores) == 1
        s, l = next(iter(cores))
        assert len(idx) == 1 or len(idx) * s * l <= 1 << 29
    # the Llama set: a single 14336x4096 matrix is 58.7M elements -> 9 per chunk
    n, chunk_of = mb.muon_plan_describe(opt, wl.shapes_llama8b())
    sizes = np.bincount(chunk_of)
    assert sizes.max() <= 64 and n == -(-64 // 32) + 1 + -(-96 // 9)
    # zero-sized matrices are skipped
    n, chunk_of = mb.muon_plan_describe(opt, [(0, 5), (3, 4), (7, 0)])
    assert n == 1 and chunk_of == [-1, 0, -1]
    # a tiny cap still puts one matrix per chunk
    opt.chunk_elems = 1
    n, chunk_of = mb.muon_plan_describe(opt, wl.shapes_tiny())
    assert n == 6 and sorted(chunk_of) == list(range(6))


def test_workspace_bytes_grows_with_the_largest_chunk():
    opt = mb.muon_default_options()
    small = mb.muon_workspace_bytes(opt, wl.shapes_tiny())
    # X, X' (bf16) + A, B (bf16) for the biggest group, plus partial sums: at least 2*X + 2*A
    assert small >= 2 * (4 * 256 * 256 * 2) + 2 * (4 * 256 * 256 * 2)
    big = mb.muon_workspace_bytes(opt, wl.shapes_llama8b())
    assert big >= 2 * (1 << 29) * 2 * 0.98
    assert big < 6 * (1 << 30)
    opt32 = mb.muon_default_options(ns_precision=mb.NS_FP32)
    assert mb.muon_workspace_bytes(opt32, wl.shapes_tiny()) > 1.9 * small
    assert mb.muon_workspace_bytes(opt, []) == 0
    bad = mb.muon_default_options(ns_precision=5)
    with pytest.raises(mb.MuonError):
        mb.muon_workspace_bytes(bad, wl.shapes_tiny())
