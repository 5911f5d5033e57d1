"""Host-side planning logic of the library, checked on a CPU: the tile lists of the symmetric products and
the packing of shape groups into launch sets.  Both are pure host arithmetic behind the C ABI."""
import itertools

import numpy as np
import pytest

from paper_2609_21594_b200 import binding as mb
from paper_2609_21594_b200 import workloads as wl

NONE = 0xFFFF


def _blocks_of(tiles):
    """Every (row block, column block) a tile list computes, in order."""
    out = []
    for ra, rb, cc, cd in tiles:
        for r in (ra, rb):
            for c in (cc, cd):
                if r != NONE and c != NONE:
                    out.append((r, c))
    return out


@pytest.mark.parametrize("nb", list(range(0, 41)) + [56, 112])
def test_symmetric_tiles_cover_every_unordered_block_pair(nb):
    tiles = mb.muon_symmetric_tiles(nb)
    blocks = _blocks_of(tiles)
    for ra, rb, cc, cd in tiles:
        assert ra != NONE and cc != NONE and ra < nb and cc < nb
        assert rb == NONE or (rb < nb and rb != ra)
        assert cd == NONE or (cd < nb and cd != cc)
    # brute force over every block the list computes
    seen = {}
    for r, c in blocks:
        seen[(min(r, c), max(r, c))] = seen.get((min(r, c), max(r, c)), 0) + 1
    want = {(x, y) for x in range(nb) for y in range(x, nb)}
    assert set(seen) == want                                     # nothing missing, nothing outside the matrix
    # the only pairs computed twice are (2j, 2j+1): the lower-left block of a diagonal 2 x 2 tile
    twice = sorted(k for k, v in seen.items() if v > 1)
    assert all(v <= 2 for v in seen.values())
    assert twice == [(2 * j, 2 * j + 1) for j in range(nb // 2)]
    # each ordered block position is written by at most one tile (a mirrored block is written by its source tile)
    assert len(set(blocks)) == len(blocks)
    # a last odd column is covered by 128-wide tiles, everything else by 256-wide ones
    narrow = [t for t in tiles if t[3] == NONE]
    assert len(narrow) == (nb // 2 + 1 if nb % 2 else 0)
    assert all(t[2] == nb - 1 for t in narrow)
    half_empty = [t for t in tiles if t[1] == NONE]
    assert len(half_empty) == nb % 2
    # cost in 128 x 128 block products: the triangle, one redundant block per diagonal tile, one idle half at most
    paid = sum(2 * (1 if t[3] == NONE else 2) for t in tiles)
    assert paid == nb * (nb + 1) // 2 + nb // 2 + nb % 2


def test_symmetric_tiles_cost_at_the_benchmark_sizes():
    def cost(nb):                                  # in 256 x 256 tile equivalents
        return sum(0.5 if t[3] == NONE else 1.0 for t in mb.muon_symmetric_tiles(nb))
    assert cost(32) == 136                         # 4096 rows: the plain upper triangle of 2 x 2 tiles
    assert cost(11) == 18                          # 1408 rows: 15 full tiles + 6 half-width ones (21 before)
    assert cost(16) == 36 and cost(8) == 10 and cost(2) == 1


def test_launch_sets_pack_shape_groups_under_the_cap():
    opt = mb.muon_default_options()
    cap = 1 << 29

    def sets_of(shapes):
        n, set_of = mb.muon_plan_launch_sets(opt, shapes)
        nch, chunk_of = mb.muon_plan_describe(opt, shapes)
        elems = np.zeros(n, dtype=np.int64)
        chunks_in = [set() for _ in range(n)]
        for (m, k), s, c in zip(shapes, set_of, chunk_of):
            if s >= 0:
                elems[s] += m * k
                chunks_in[s].add(c)
        return n, nch, elems, chunks_in

    n, nch, elems, chunks_in = sets_of(wl.shapes_tiny())
    assert n == 1 and nch == 2                    # both core shapes of the d=256 layer share every launch
    n, nch, elems, chunks_in = sets_of(wl.shapes_1b())
    assert nch == 4 and n == 2 and (elems <= cap).all()
    n, nch, elems, chunks_in = sets_of(wl.shapes_moe())
    assert nch == 6 and n == 5 and (elems <= cap).all()      # the attention group rides with one expert chunk
    n, nch, elems, chunks_in = sets_of(wl.shapes_llama8b())
    assert nch == 14 and n == 14                  # every Llama-3-8B chunk already fills the cap on its own
    # a chunk belongs to exactly one set
    all_chunks = list(itertools.chain.from_iterable(chunks_in))
    assert len(all_chunks) == len(set(all_chunks)) == nch
    # one matrix larger than the cap still gets a set of its own
    big = mb.muon_default_options(chunk_elems=1000)
    n, set_of = mb.muon_plan_launch_sets(big, [(64, 64), (8, 8), (8, 8), (100, 100)])
    assert n == 3 and set_of[1] == set_of[2] and len({set_of[0], set_of[1], set_of[3]}) == 3
    n, set_of = mb.muon_plan_launch_sets(opt, [(0, 5), (3, 4)])
    assert n == 1 and set_of == [-1, 0]


def test_workspace_is_the_largest_launch_set():
    opt = mb.muon_default_options()
    # tiny: both groups resident together: 2 X + 2 A for each, bf16
    need = mb.muon_workspace_bytes(opt, wl.shapes_tiny())
    x = (4 * 256 * 256 + 2 * 256 * 1024) * 2
    a = (4 * 256 * 256 + 2 * 256 * 256) * 2
    assert 2 * x + 2 * a <= need <= 2 * x + 2 * a + 16384


# ----------------------------------------------------------------------------- strided views: overlap check
def _brute_overlap(bases, views, es):
    seen = set()
    for b, (r, c, ld) in zip(bases, views):
        if not b or r == 0 or c == 0:
            continue
        mine = set()
        for i in range(r):
            lo = b + i * ld * es
            mine.update(range(lo, lo + c * es))
        if seen & mine:
            return True
        seen |= mine
    return False


def test_views_overlap_known_cases():
    base, es = 1 << 20, 4
    # fused QKV: three row blocks of one [3*64, 96] tensor
    qkv = [(64, 96, 96)] * 3
    assert not mb.muon_views_overlap([base + k * 64 * 96 * es for k in range(3)], qkv, es)
    assert mb.muon_views_overlap([base, base + 63 * 96 * es, base + 128 * 96 * es], qkv, es)        # second starts one row early
    # gate/up stored row-interleaved in one [2*m, n] tensor: row stride 2n, second view offset by n
    m, n = 40, 24
    assert not mb.muon_views_overlap([base, base + n * es], [(m, n, 2 * n)] * 2, es)
    assert mb.muon_views_overlap([base, base + (n - 1) * es], [(m, n, 2 * n)] * 2, es)               # offset one element short
    # side-by-side column factors of one [m, 3n] tensor
    assert not mb.muon_views_overlap([base + k * n * es for k in range(3)], [(m, n, 3 * n)] * 3, es)
    assert mb.muon_views_overlap([base, base + n * es], [(m, n + 1, 3 * n), (m, n, 3 * n)], es)
    # bounding intervals nest but no element is shared: a narrow view in the padding columns of a wide one
    assert not mb.muon_views_overlap([base, base + 16 * es], [(10, 16, 32), (10, 8, 32)], es)
    # identical views, empty views, null bases
    assert mb.muon_views_overlap([base, base], [(3, 5, 5)] * 2, es)
    assert not mb.muon_views_overlap([base, base], [(3, 5, 5), (0, 5, 5)], es)
    assert not mb.muon_views_overlap([base, 0], [(3, 5, 5)] * 2, es)
    with pytest.raises(mb.MuonError):
        mb.muon_views_overlap([base], [(3, 5, 4)], es)                                                # ld < cols


def test_views_overlap_against_brute_force():
    rng = np.random.default_rng(5)
    hits = 0
    for case in range(300):
        es = int(rng.choice([2, 4]))
        k = int(rng.integers(2, 6))
        views, bases = [], []
        for _ in range(k):
            r, c = int(rng.integers(0, 7)), int(rng.integers(0, 7))
            ld = c + int(rng.integers(0, 9))
            views.append((r, c, max(ld, 1)))
            bases.append(4096 + es * int(rng.integers(0, 60)))
        want = _brute_overlap(bases, views, es)
        hits += want
        assert mb.muon_views_overlap(bases, views, es) == want, (case, bases, views, es)
    assert 30 < hits < 270          # the sample exercises both answers


# ----------------------------------------------------------------------------- host-buffer pipeline plan
@pytest.mark.parametrize("name", ["llama8b", "moe", "1b", "tiny", "odd"])
def test_pipeline_plan_ramps(name):
    """What muon_step_flat_host runs: every matrix in exactly one set, every set within the cap and within 8 core
    shapes, and -- when the work is large enough to ramp -- sets listed in running order that open and close with about
    2^24 elements and grow no faster than the kernels of the sets before them can cover the next copy (65536 flops of
    Newton-Schulz work per element copied), so that the copies no kernel overlaps stay short."""
    shapes = {"llama8b": wl.shapes_llama8b, "moe": wl.shapes_moe, "1b": wl.shapes_1b, "tiny": wl.shapes_tiny,
              "odd": wl.shapes_odd}[name]()
    opt = mb.muon_default_options()
    set_of, order = mb.muon_plan_pipeline(opt, shapes)
    nsets = len(order)
    assert sorted(order) == list(range(nsets))
    assert all(0 <= s < nsets for s in set_of) and len(set_of) == len(shapes)
    elems, work = [0] * nsets, [0.0] * nsets
    kinds = [set() for _ in range(nsets)]
    for (m, n), s in zip(shapes, set_of):
        sm, lg = min(m, n), max(m, n)
        elems[s] += m * n
        work[s] += 10.0 * sm * sm * (3 * lg + sm)
        kinds[s].add((sm, lg))
    cap, edge = 1 << 29, 1 << 24
    assert all(0 < e <= cap or len(k) == 1 for e, k in zip(elems, kinds))
    assert all(len(k) <= 8 for k in kinds)
    total = sum(elems)
    if total < 16 * edge:                                   # too little work to ramp: the ordinary plan
        assert (nsets, set_of) == mb.muon_plan_launch_sets(opt, shapes)
        return
    assert order == list(range(nsets))                      # listed in running order
    biggest = max(m * n for m, n in shapes)
    assert elems[0] <= max(edge, biggest) and elems[-1] <= max(edge, biggest)

    def ramp_length(seq):
        done, k = 0.0, 0
        while k < len(seq) and elems[seq[k]] < cap // 2:
            target = edge + done / 65536.0
            if elems[seq[k]] > max(target, edge, min(m * n for m, n in shapes)):
                break
            done += work[seq[k]]
            k += 1
        return k

    up, down = ramp_length(list(range(nsets))), ramp_length(list(range(nsets - 1, -1, -1)))
    assert up >= 2 and down >= 2, (up, down, elems)
    # the ramps are made of the matrices with the most work per element
    dens = sorted({(10.0 * min(m, n) ** 2 * (3 * max(m, n) + min(m, n))) / (m * n) for m, n in shapes}, reverse=True)
    assert work[0] / elems[0] == pytest.approx(dens[0])
    # and leave most of the work to full-size sets
    assert sum(e for e in elems if e >= cap // 4) >= total // 2
