"""Property test of the C library's host-side layout validation against the oracle's brute-force checker:
random segment tables -- valid ones produced by the generators and then perturbed in random ways -- must be
accepted or rejected identically by both."""
import numpy as np
from hypothesis import HealthCheck, given, settings
from hypothesis import strategies as st

from oracle import muon_oracle as orc
from paper_2609_21594_b200 import binding as mb
from paper_2609_21594_b200 import workloads as wl

shape_st = st.tuples(st.integers(0, 9), st.integers(0, 9))


@settings(max_examples=300, deadline=None, suppress_health_check=[HealthCheck.too_slow])
@given(shapes=st.lists(shape_st, min_size=1, max_size=5), shards=st.integers(1, 4), align=st.sampled_from([1, 2, 4, 8]),
       flat=st.booleans(), mutations=st.lists(st.tuples(st.integers(0, 5), st.integers(0, 63), st.integers(-3, 3)), max_size=3))
def test_validate_agrees_with_bruteforce(shapes, shards, align, flat, mutations):
    gen = wl.layout_flat_concat if flat else wl.layout_per_param
    lay = gen(shapes, shards, align)
    segs = [[s.matrix, s.elem_begin, s.elem_count, s.flat_offset] for s in lay.segments]
    shard_len = lay.shard_len
    for kind, which, delta in mutations:
        if kind == 5:
            shard_len = max(0, shard_len + delta * align)
            continue
        if not segs:
            continue
        k = which % len(segs)
        if kind == 0:
            segs[k][1] += delta                      # elem_begin
        elif kind == 1:
            segs[k][2] += delta                      # elem_count
        elif kind == 2:
            segs[k][3] += delta * (align if which % 2 else 1)   # flat_offset, aligned or not
        elif kind == 3:
            segs.append(list(segs[k]))               # duplicate
        elif kind == 4:
            segs.pop(k)                              # drop
    mutated = wl.Layout(tuple(shapes), shards, shard_len, align, tuple(wl.Segment(*s) for s in segs))
    got = mb.muon_layout_validate(mb.make_layout_desc(mutated, 2))
    expect = orc.layout_is_valid(shards * shard_len, list(shapes), [tuple(s) for s in segs], align, shards, shard_len)
    assert (got == mb.OK) == expect, (got, expect, shapes, shards, align, segs, shard_len)
    assert got in (mb.OK, mb.ERR_BAD_LAYOUT)
